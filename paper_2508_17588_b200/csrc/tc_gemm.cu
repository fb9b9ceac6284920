// bf16 GEMM of the refresh path on the 5th-generation tensor cores:
//   C[M, Nout] = A[M, K] * W[Nout, K]^T + bias   (fp32 accumulation in TMEM)
// followed by the epilogue of Eq. 2 / Eq. 3: optional GELU-tanh or gate, bf16 rounding, and
// rows written either compactly or straight into their slots of a [B, N, D] cache.
//
// Persistent kernel, one CTA per SM, 128 x 256 output tile, K in steps of 64:
//   warp 0      TMA producer: A tile (128x64) and W tile (256x64) per stage, 128-byte swizzle
//   warp 1      MMA issuer:   4 x tcgen05.mma (M128 N256 K16) per stage, commit frees the stage
//   warps 2..5  epilogue:     tcgen05.ld of the finished accumulator, bias/act, global stores
// Two 256-column accumulators in TMEM let the epilogue of tile i overlap the MMAs of tile i+1.
#include <cuda.h>

#include <mutex>

#include "hero_internal.h"
#include "tc_common.cuh"

namespace hero {

// ---------------------------------------------------------------------------
// Driver entry point for tensor-map encoding (resolved at run time: no -lcuda needed)
// ---------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;
static std::once_flag g_encode_once;

int tc_init_driver_api() {
  std::call_once(g_encode_once, [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  });
  if (!g_encode) {
    set_cuda_error(cudaErrorUnknown, "cuTensorMapEncodeTiled not available");
    return HERO_ERR_CUDA;
  }
  return HERO_OK;
}

// bf16 tensor [.., rows, cols] with cols contiguous; box = box_rows x 64 columns (128 bytes), 128B swizzle,
// out-of-range elements read as zero.
int make_tmap_bf16(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                   const uint32_t* box) {
  HERO_TRY(tc_init_driver_api());
  cuuint64_t gdim[3];
  cuuint64_t gstr[2];
  cuuint32_t bx[3], es[3];
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
  CUresult r = g_encode(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr,
                        bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    set_cuda_error(cudaErrorInvalidValue, "cuTensorMapEncodeTiled");
    return HERO_ERR_CUDA;
  }
  return HERO_OK;
}

namespace {
using namespace tc;

#ifndef HERO_GEMM_BN
#define HERO_GEMM_BN 256
#endif
#ifndef HERO_GEMM_STAGES
#define HERO_GEMM_STAGES 4
#endif
constexpr int kBM = 128, kBN = HERO_GEMM_BN, kBK = 64, kStages = HERO_GEMM_STAGES;
constexpr int kABytes = kBM * kBK * 2;                 // 16 KB
constexpr int kBBytes = kBN * kBK * 2;                 // 32 KB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kGemmThreads = 192;
constexpr int kTmemCols = 512;                         // two accumulators of 256 fp32 columns
constexpr size_t kGemmSmem = 1024 /*alignment slack*/ + (size_t)kStages * kStageBytes + 256 /*barriers*/;

__device__ __forceinline__ float gelu_tanh_f(float t) {
  // 0.5 t (1 + tanh(sqrt(2/pi) (t + 0.044715 t^3))) with the hardware tanh (one special-function
  // instruction, relative error 2^-11: below the bf16 rounding of the result).  The epilogue shares the
  // SM's power budget with the tensor core, so every instruction saved here is tensor clock gained.
  const float t2 = t * t;
  const float u = t * fmaf(0.0356774081f, t2, 0.7978845608f);
  float th;
  asm("tanh.approx.f32 %0, %1;" : "=f"(th) : "f"(u));
  const float h = 0.5f * t;
  return fmaf(h, th, h);
}

// Tile order of the persistent CTAs.  Consecutive tile numbers run down kGroupM row tiles before moving
// to the next column tile, and only then to the next band of rows: the ~148 tiles in flight at any time
// then cover about 24 x 6 tiles, whose operands (24 row panels of A, 6 of W) stay in L2 and are shared by
// the CTAs working on them, instead of every CTA streaming its own panel of A from DRAM.  Bands of 16 to 48
// row tiles time within a percent of each other in the step, 24 slightly ahead (12: 1 % slower, 6: 3 %, one
// band over all rows: 3 %).
constexpr int kGroupM = 24;
__device__ __forceinline__ void tile_coords(int tile, int m_tiles, int n_tiles, int& mt, int& nt) {
  const int per_group = kGroupM * n_tiles;
  const int group = tile / per_group;
  const int first_m = group * kGroupM;
  const int rows = min(kGroupM, m_tiles - first_m);
  const int r = tile - group * per_group;
  mt = first_m + r % rows;
  nt = r / rows;
}

__global__ void __launch_bounds__(kGemmThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tm_a, const __grid_constant__ CUtensorMap tm_w,
               const __nv_bfloat16* __restrict__ bias, const GemmOut out, int M, int Nout, int K,
               int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)kStages * kStageBytes);
  uint64_t* full = bars;                    // [kStages] TMA -> MMA
  uint64_t* empty = bars + kStages;         // [kStages] MMA -> TMA
  uint64_t* acc_full = bars + 2 * kStages;  // [2] MMA -> epilogue
  uint64_t* acc_empty = acc_full + 2;       // [2] epilogue -> MMA
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m_tiles = (M + kBM - 1) / kBM, n_tiles = (Nout + kBN - 1) / kBN;
  const int n_tiles_total = m_tiles * n_tiles;
  const int k_blocks = (K + kBK - 1) / kBK;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 4); }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 0 && lane == 0) { tma_prefetch_desc(&tm_a); tma_prefetch_desc(&tm_w); }
  if (warp == 1) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < n_tiles_total && ok; tile += gridDim.x) {
        int mt, nt;
        tile_coords(tile, m_tiles, n_tiles, mt, nt);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait(&empty[stage], phase ^ 1, abort_flag))) break;
          uint8_t* sa = smem + (size_t)stage * kStageBytes;
          mbar_expect_tx(&full[stage], kStageBytes);
          tma_load_2d(sa, &tm_a, &full[stage], kb * kBK, mt * kBM);
          tma_load_2d(sa + kABytes, &tm_w, &full[stage], kb * kBK, nt * kBN);
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
      }
      // On the way out make sure every stage that was armed has landed (bounded): the CTA must
      // not retire with bulk copies still writing its shared memory.
      for (int i = 0; i < kStages; ++i) {
        if (!mbar_wait(&empty[stage], phase ^ 1, abort_flag)) break;
        if (++stage == kStages) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    // All 32 lanes run the loop and one elected lane issues: tile counters, stage addresses and descriptors
    // then stay warp-uniform values instead of one diverged lane's private registers, which is what the
    // tensor-core instructions are fed from.
    {
      const bool leader = elect_one();
      constexpr uint32_t idesc = idesc_bf16(kBM, kBN, 0);
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      int t = 0;
      for (int tile = blockIdx.x; tile < n_tiles_total && ok; tile += gridDim.x, ++t) {
        const int acc = t & 1;
        if (!(ok = mbar_wait_warp(&acc_empty[acc], ((t >> 1) & 1) ^ 1, abort_flag))) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)acc * kBN;
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!(ok = mbar_wait_warp(&full[stage], phase, abort_flag))) break;
          tc_fence_after();
          const uint32_t sa = smem_u32(smem + (size_t)stage * kStageBytes);
          const uint64_t da = smem_desc_sw128(sa, 1024), db = smem_desc_sw128(sa + kABytes, 1024);
          if (leader) {
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)   // +32 bytes (encoded >>4) per K step of 16 inside the swizzle atom
              mma_ss(d_tmem, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
            mma_commit(&empty[stage]);
          }
          if (++stage == kStages) { stage = 0; phase ^= 1; }
        }
        if (ok && leader) mma_commit(&acc_full[acc]);
      }
    }
  } else {
    // ------------------------------------------------------------ epilogue (warps 2..5)
    const int quad = warp & 3;                 // TMEM lane quadrant this warp may read
    bool ok = true;
    int t = 0;
    for (int tile = blockIdx.x; tile < n_tiles_total && ok; tile += gridDim.x, ++t) {
      int mt, nt;
      tile_coords(tile, m_tiles, n_tiles, mt, nt);
      const int acc = t & 1;
      ok = mbar_wait(&acc_full[acc], (t >> 1) & 1, abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const int m = mt * kBM + quad * 32 + lane;
      const bool row_ok = m < M;
      int b = 0, li = 0;
      if (row_ok) { b = m / out.n_sel; li = m - b * out.n_sel; }
      long long scat_row = 0;
      if (row_ok) scat_row = (long long)b * out.n_rows + (out.idx ? out.idx[li] : li);
      const uint32_t t_row = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)acc * kBN;
#pragma unroll 1
      for (int c = 0; c < kBN / 32; ++c) {
        const int n0 = nt * kBN + c * 32;
        if (n0 >= Nout) break;                 // warp-uniform
        uint32_t r[32];
        tmem_ld32(t_row + c * 32, r);
        tmem_ld_wait();
        if (row_ok) {
          const int seg = n0 / out.seg_cols, col0 = n0 - seg * out.seg_cols;
          const long long drow = out.scatter[seg] ? scat_row : (long long)m;
          __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(out.ptr[seg]) + drow * out.ld[seg] + col0;
          const float* gate = out.gate ? out.gate + (long long)b * out.gate_ld + col0 : nullptr;
          const float seg_scale = (seg == 0 && out.seg0_scale != 0.f) ? out.seg0_scale : 1.0f;   // warp-uniform
#pragma unroll
          for (int v = 0; v < 4; ++v) {        // 8 columns = one 16-byte store
            if (n0 + v * 8 < Nout) {
              const uint4 braw = __ldg(reinterpret_cast<const uint4*>(bias + n0 + v * 8));
              const uint32_t bw[4] = {braw.x, braw.y, braw.z, braw.w};
              uint32_t packed[4];
#pragma unroll
              for (int q = 0; q < 4; ++q) {
                float f0 = __uint_as_float(r[v * 8 + 2 * q]) + __uint_as_float(bw[q] << 16);
                float f1 = __uint_as_float(r[v * 8 + 2 * q + 1]) + __uint_as_float(bw[q] & 0xFFFF0000u);
                if (out.act == 1) { f0 = gelu_tanh_f(f0); f1 = gelu_tanh_f(f1); }
                if (seg_scale != 1.0f) { f0 *= seg_scale; f1 *= seg_scale; }
                if (gate) { f0 *= gate[v * 8 + 2 * q]; f1 *= gate[v * 8 + 2 * q + 1]; }
                const __nv_bfloat162 p = __floats2bfloat162_rn(f0, f1);
                packed[q] = *reinterpret_cast<const uint32_t*>(&p);
              }
              *reinterpret_cast<uint4*>(dst + v * 8) = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[acc]);
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, 1);
  if (warp == 1) { tc_fence_after(); tmem_dealloc(tmem_base, kTmemCols); }
}

// Self-test of the bounded wait: the barrier below is initialised for one arrival that never comes.
__global__ void wait_timeout_selftest_kernel(int* __restrict__ status, unsigned long long budget_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); abort_flag = 0; mbar_fence_init(); }
  __syncthreads();
  const bool ok = mbar_wait_warp(&bar, 0, &abort_flag, budget_ns);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || abort_flag)) atomicExch(status, 1);
}

}  // namespace

int launch_wait_timeout_selftest(int* d_status, int budget_us, cudaStream_t s) {
  wait_timeout_selftest_kernel<<<1, 64, 0, s>>>(d_status, (unsigned long long)budget_us * 1000ull);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

int launch_tc_gemm(const void* a, const void* w, const void* bias, int M, int Nout, int K, const GemmOut& out,
                   int* d_status, cudaStream_t s) {
  if (M <= 0) return HERO_OK;
  if (K % 8 || Nout % 8 || out.seg_cols % 32) return HERO_ERR_ALIGN;
  if (!aligned16(a) || !aligned16(w) || !aligned16(bias)) return HERO_ERR_ALIGN;
  for (int i = 0; i < 3; ++i)
    if (out.ptr[i] && (!aligned16(out.ptr[i]) || out.ld[i] % 8)) return HERO_ERR_ALIGN;
  CUtensorMap tm_a, tm_w;
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)M};
    const uint64_t str[1] = {(uint64_t)K * 2};
    const uint32_t box[2] = {(uint32_t)kBK, (uint32_t)kBM};
    HERO_TRY(make_tmap_bf16(&tm_a, a, 2, dims, str, box));
  }
  {
    const uint64_t dims[2] = {(uint64_t)K, (uint64_t)Nout};
    const uint64_t str[1] = {(uint64_t)K * 2};
    const uint32_t box[2] = {(uint32_t)kBK, (uint32_t)kBN};
    HERO_TRY(make_tmap_bf16(&tm_w, w, 2, dims, str, box));
  }
  static PerDeviceOnce attr_once;            // the opt-in is a property of the kernel ON a device
  HERO_TRY(per_device_once(attr_once, [](int) {
    HERO_CUDA_TRY(cudaFuncSetAttribute(tc_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGemmSmem));
    return HERO_OK;
  }));
  const int tiles = ((M + kBM - 1) / kBM) * ((Nout + kBN - 1) / kBN);
  const int grid = tiles < num_sms() ? tiles : num_sms();
  tc_gemm_kernel<<<grid, kGemmThreads, kGemmSmem, s>>>(tm_a, tm_w, (const __nv_bfloat16*)bias, out, M, Nout, K,
                                                       d_status);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

}  // namespace hero
