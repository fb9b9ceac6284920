// Flash-attention for the refresh path (Eq. 3 with the refreshed queries attending to the
// full cached K/V): O = softmax(Q K^T / sqrt(64)) V per (batch, head), bf16 in, fp32 softmax,
// no score matrix ever leaves the SM.
//
// One CTA = 256 query rows (two tiles of 128) of one (batch, head); it streams all N cached
// keys in tiles of 128 through a 4-stage TMA ring shared by both query tiles.
//   warp 0      TMA: both Q tiles once, then K/V tiles (128-byte swizzle)
//   warp 1      tcgen05.mma issuer: S = Q K^T (M128 N128 K64) into TMEM, then P V (M128 N64 K128)
//               with P read from TMEM and V as an N-contiguous shared-memory operand
//   warps 2..5  softmax group of query tile 0, warps 6..9 of query tile 1: one thread per
//               query row; running max / sum in registers, P written back over S in TMEM as
//               bf16, the running output rescaled and accumulated in registers
// TMEM holds four 128-column buffers, (query tile) x (key tile parity).  A buffer first receives
// S; the softmax overwrites columns [0,64) with P; the P V product lands in columns [64,128).
// Two softmax groups keep every SM sub-partition busy while the other group waits on the
// tensor core.
#include <cuda.h>

#include <mutex>

#include "hero_internal.h"
#include "tc_common.cuh"

namespace hero {

int make_tmap_bf16(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                   const uint32_t* box);

namespace {
using namespace tc;

constexpr int kQT = 128, kQTiles = 2, kKT = 128, kHD = 64, kKvStages = 4;
constexpr int kQBytes = kQT * kHD * 2;       // 16 KB per query tile
constexpr int kKBytes = kKT * kHD * 2;       // 16 KB
constexpr int kKvStageBytes = 2 * kKBytes;   // K tile then V tile
constexpr int kAttThreads = 64 + 128 * kQTiles;
constexpr size_t kAttSmem = 1024 + kQTiles * kQBytes + (size_t)kKvStages * kKvStageBytes + 512;
constexpr uint32_t kBufCols = 128, kColPV = 64, kAttTmemCols = 512;

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float y;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}
__device__ __forceinline__ float2 f2(uint32_t a, uint32_t b) { return make_float2(__uint_as_float(a), __uint_as_float(b)); }

// One key tile of one query row: S (128 fp32 in TMEM) -> running max, P (bf16 pairs written over
// the first 64 columns), row sum of P.  `valid` < 128 only in the ragged last tile.
template <bool MASKED>
__device__ __forceinline__ void softmax_tile(uint32_t t_buf, int valid, float c, float& m_run, float& alpha_out,
                                             float& sum_out) {
  // pass 1: row maximum (two independent chains, three-input max)
  float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll 1
  for (int ch = 0; ch < kKT / 32; ++ch) {
    uint32_t r[32];
    tmem_ld32(t_buf + ch * 32, r);
    tmem_ld_wait();
    if (MASKED) {
#pragma unroll
      for (int i = 0; i < 32; ++i)
        if (ch * 32 + i >= valid) r[i] = 0xFF800000u;   // -inf
    }
#pragma unroll
    for (int i = 0; i < 32; i += 4) {
      mx0 = max3(mx0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
      mx1 = max3(mx1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
    }
  }
  const float m_new = max3(m_run, mx0, mx1);
  alpha_out = ex2((m_run - m_new) * c);
  m_run = m_new;
  const float neg_mc = -m_new * c;
  const float2 c2 = make_float2(c, c), nm2 = make_float2(neg_mc, neg_mc);
  // pass 2: p = 2^(s*c - m*c); bf16 pairs go back into columns [0,64) of the same buffer
  float2 acc0 = make_float2(0.f, 0.f), acc1 = make_float2(0.f, 0.f);
#pragma unroll 1
  for (int half = 0; half < 2; ++half) {
    uint32_t packed[32];
#pragma unroll
    for (int sub = 0; sub < 2; ++sub) {
      uint32_t r[32];
      tmem_ld32(t_buf + half * 64 + sub * 32, r);
      tmem_ld_wait();
#pragma unroll
      for (int i = 0; i < 32; i += 4) {
        float2 x0 = __ffma2_rn(f2(r[i], r[i + 1]), c2, nm2);
        float2 x1 = __ffma2_rn(f2(r[i + 2], r[i + 3]), c2, nm2);
        float2 p0 = make_float2(ex2(x0.x), ex2(x0.y));
        float2 p1 = make_float2(ex2(x1.x), ex2(x1.y));
        if (MASKED) {
          const int col = half * 64 + sub * 32 + i;
          if (col >= valid) p0.x = 0.f;
          if (col + 1 >= valid) p0.y = 0.f;
          if (col + 2 >= valid) p1.x = 0.f;
          if (col + 3 >= valid) p1.y = 0.f;
        }
        acc0 = __fadd2_rn(acc0, p0);
        acc1 = __fadd2_rn(acc1, p1);
        const __nv_bfloat162 b0 = __floats2bfloat162_rn(p0.x, p0.y), b1 = __floats2bfloat162_rn(p1.x, p1.y);
        packed[sub * 16 + i / 2] = *reinterpret_cast<const uint32_t*>(&b0);
        packed[sub * 16 + i / 2 + 1] = *reinterpret_cast<const uint32_t*>(&b1);
      }
    }
    tmem_st32(t_buf + half * 32, packed);
  }
  sum_out = (acc0.x + acc0.y) + (acc1.x + acc1.y);
}

// kPerCtaStatus = false: a CTA that gave up raises the single word *status.
// kPerCtaStatus = true:  status[0] counts the CTAs that gave up and status[1 + blockIdx.x] records which.
template <bool kPerCtaStatus>
__global__ void __launch_bounds__(kAttThreads, 1)
tc_attention_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ O, int n_q, int N,
                    int heads, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s_q = smem;
  uint8_t* s_kv = smem + kQTiles * kQBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_kv + (size_t)kKvStages * kKvStageBytes);
  uint64_t* q_full = bars;
  uint64_t* kv_full = bars + 1;                    // [kKvStages]
  uint64_t* kv_empty = kv_full + kKvStages;        // [kKvStages]
  uint64_t* s_full = kv_empty + kKvStages;         // [qt][parity]  MMA -> softmax: S is ready
  uint64_t* p_full = s_full + 4;                   // [qt][parity]  softmax -> MMA: P is in TMEM
  uint64_t* pv_full = p_full + 4;                  // [qt][parity]  MMA -> softmax: P V is ready
  uint64_t* o_done = pv_full + 4;                  // [qt][parity]  softmax -> MMA: buffer may be reused
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(o_done + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q_groups = (n_q + kQT * kQTiles - 1) / (kQT * kQTiles);
  const int qg = blockIdx.x % q_groups;
  const int h = (blockIdx.x / q_groups) % heads;
  const int b = blockIdx.x / (q_groups * heads);
  const int n_kv = (N + kKT - 1) / kKT;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < kKvStages; ++i) { mbar_init(&kv_full[i], 1); mbar_init(&kv_empty[i], 1); }
    for (int i = 0; i < 4; ++i) {
      mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 4); mbar_init(&pv_full[i], 1); mbar_init(&o_done[i], 4);
    }
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 0 && lane == 0) { tma_prefetch_desc(&tm_q); tma_prefetch_desc(&tm_k); tma_prefetch_desc(&tm_v); }
  if (warp == 1) { tmem_alloc(tmem_slot, kAttTmemCols); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(q_full, kQTiles * kQBytes);
      for (int t = 0; t < kQTiles; ++t)
        tma_load_2d(s_q + t * kQBytes, &tm_q, q_full, h * kHD, b * n_q + (qg * kQTiles + t) * kQT);
      int stage = 0; uint32_t phase = 0;
      for (int j = 0; j < n_kv; ++j) {
        if (!mbar_wait(&kv_empty[stage], phase ^ 1, abort_flag)) break;
        uint8_t* sk = s_kv + (size_t)stage * kKvStageBytes;
        mbar_expect_tx(&kv_full[stage], kKvStageBytes);
        tma_load_3d(sk, &tm_k, &kv_full[stage], h * kHD, j * kKT, b);
        tma_load_3d(sk + kKBytes, &tm_v, &kv_full[stage], h * kHD, j * kKT, b);
        if (++stage == kKvStages) { stage = 0; phase ^= 1; }
      }
      for (int i = 0; i < kKvStages; ++i) {      // all armed stages consumed before the CTA retires
        if (!mbar_wait(&kv_empty[stage], phase ^ 1, abort_flag)) break;
        if (++stage == kKvStages) { stage = 0; phase ^= 1; }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc_s = idesc_bf16(kQT, kKT, 0);    // S = Q K^T : both operands K-contiguous
      constexpr uint32_t idesc_pv = idesc_bf16(kQT, kHD, 1);   // O = P V   : V is N(head_dim)-contiguous
      auto issue_s = [&](int t, int j) {
        const int st = j % kKvStages;
        const uint64_t dq = smem_desc_sw128(smem_u32(s_q + t * kQBytes), 1024);
        const uint64_t dk = smem_desc_sw128(smem_u32(s_kv + (size_t)st * kKvStageBytes), 1024);
        const uint32_t d = tmem_base + (uint32_t)(t * 2 + (j & 1)) * kBufCols;
#pragma unroll
        for (int k = 0; k < kHD / 16; ++k) mma_ss(d, dq + 2 * k, dk + 2 * k, idesc_s, k != 0);
        mma_commit(&s_full[t * 2 + (j & 1)]);
      };
      bool ok = mbar_wait(q_full, 0, abort_flag);
      if (ok) ok = mbar_wait(&kv_full[0], 0, abort_flag);
      if (ok) { tc_fence_after(); issue_s(0, 0); issue_s(1, 0); }
      for (int j = 0; j < n_kv && ok; ++j) {
        if (j + 1 < n_kv) {
          if (!(ok = mbar_wait(&kv_full[(j + 1) % kKvStages], ((j + 1) / kKvStages) & 1, abort_flag))) break;
          for (int t = 0; t < kQTiles && ok; ++t) {
            // buffer (t, (j+1)&1) last held tile j-1: its P V must have been read out
            if (j >= 1) ok = mbar_wait(&o_done[t * 2 + ((j + 1) & 1)], ((j - 1) >> 1) & 1, abort_flag);
            if (ok) { tc_fence_after(); issue_s(t, j + 1); }
          }
          if (!ok) break;
        }
        const int st = j % kKvStages;
        // V tile: rows = keys (128 bytes each), 8-key groups 1024 bytes apart; 16 keys per MMA = 2048 bytes
        const uint64_t dv = smem_desc_sw128(smem_u32(s_kv + (size_t)st * kKvStageBytes + kKBytes), 1024);
        for (int t = 0; t < kQTiles && ok; ++t) {
          const int bi = t * 2 + (j & 1);
          if (!(ok = mbar_wait(&p_full[bi], (j >> 1) & 1, abort_flag))) break;
          tc_fence_after();
          const uint32_t buf = tmem_base + (uint32_t)bi * kBufCols;
#pragma unroll
          for (int k = 0; k < kKT / 16; ++k) mma_ts(buf + kColPV, buf + 8 * k, dv + 128 * k, idesc_pv, k != 0);
          mma_commit(&pv_full[bi]);
        }
        if (ok) mma_commit(&kv_empty[st]);
      }
    }
  } else {
    // ------------------------------------------------------------ softmax + output accumulation
    const int t = (warp - 2) >> 2;                     // query tile of this softmax group
    const int quad = warp & 3;                         // TMEM lane quadrant this warp may touch
    const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(t * 2) * kBufCols;
    const float c = 0.125f * 1.4426950408889634f;      // 1/sqrt(64) * log2(e)
    float m_run = -INFINITY, l_run = 0.f, alpha_pend = 0.f;
    float2 o[kHD / 2];
#pragma unroll
    for (int i = 0; i < kHD / 2; ++i) o[i] = make_float2(0.f, 0.f);
    auto fold_pv = [&](int j) -> bool {                // O = O * alpha + (P V)_j, then release the buffer
      bool good = mbar_wait(&pv_full[t * 2 + (j & 1)], (j >> 1) & 1, abort_flag);
      good = __all_sync(0xFFFFFFFFu, good);
      if (!good) return false;
      tc_fence_after();
      const uint32_t t_pv = lane_base + (uint32_t)(j & 1) * kBufCols + kColPV;
      uint32_t r0[32], r1[32];
      tmem_ld32(t_pv, r0);
      tmem_ld32(t_pv + 32, r1);
      tmem_ld_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&o_done[t * 2 + (j & 1)]);
      const float2 a2 = make_float2(alpha_pend, alpha_pend);
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        o[i] = __ffma2_rn(o[i], a2, f2(r0[2 * i], r0[2 * i + 1]));
        o[16 + i] = __ffma2_rn(o[16 + i], a2, f2(r1[2 * i], r1[2 * i + 1]));
      }
      return true;
    };
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      ok = mbar_wait(&s_full[t * 2 + (j & 1)], (j >> 1) & 1, abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_buf = lane_base + (uint32_t)(j & 1) * kBufCols;
      const int valid = N - j * kKT;                   // keys of this tile that exist (>= 1)
      float alpha, sum;
      if (valid >= kKT) softmax_tile<false>(t_buf, valid, c, m_run, alpha, sum);
      else softmax_tile<true>(t_buf, valid, c, m_run, alpha, sum);
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[t * 2 + (j & 1)]);
      // fold in the previous tile's P V while the tensor core works on this one
      if (j > 0 && !(ok = fold_pv(j - 1))) break;
      l_run = fmaf(l_run, alpha, sum);
      alpha_pend = alpha;
    }
    if (ok && fold_pv(n_kv - 1)) {
      const int qi = (qg * kQTiles + t) * kQT + quad * 32 + lane;
      if (qi < n_q) {
        const float inv = 1.0f / l_run;
        __nv_bfloat16* dst = O + ((long long)b * n_q + qi) * ((long long)heads * kHD) + h * kHD;
#pragma unroll
        for (int v = 0; v < kHD / 8; ++v) {
          uint32_t w[4];
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const __nv_bfloat162 pk = __floats2bfloat162_rn(o[v * 4 + q].x * inv, o[v * 4 + q].y * inv);
            w[q] = *reinterpret_cast<const uint32_t*>(&pk);
          }
          *reinterpret_cast<uint4*>(dst + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) {
    if (kPerCtaStatus) { atomicAdd(status, 1); status[1 + blockIdx.x] = 2; }
    else atomicExch(status, 2);
  }
  if (warp == 1) { __syncwarp(); tc_fence_after(); tmem_dealloc(tmem_base, kAttTmemCols); }
}

}  // namespace

int launch_tc_attention(const void* q, const void* k, const void* v, void* o, int B, int n_q, int N, int heads,
                        int* d_status, cudaStream_t s) {
  if (B <= 0 || n_q <= 0) return HERO_OK;
  if (N <= 0 || heads <= 0) return HERO_ERR_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return HERO_ERR_ALIGN;
  const uint64_t D = (uint64_t)heads * kHD;
  CUtensorMap tm_q, tm_k, tm_v;
  {
    const uint64_t dims[2] = {D, (uint64_t)B * n_q};
    const uint64_t str[1] = {D * 2};
    const uint32_t box[2] = {(uint32_t)kHD, (uint32_t)kQT};
    HERO_TRY(make_tmap_bf16(&tm_q, q, 2, dims, str, box));
  }
  {
    const uint64_t dims[3] = {D, (uint64_t)N, (uint64_t)B};
    const uint64_t str[2] = {D * 2, (uint64_t)N * D * 2};
    const uint32_t box[3] = {(uint32_t)kHD, (uint32_t)kKT, 1};
    HERO_TRY(make_tmap_bf16(&tm_k, k, 3, dims, str, box));
    HERO_TRY(make_tmap_bf16(&tm_v, v, 3, dims, str, box));
  }
  static std::once_flag attr_once;
  static cudaError_t attr_err = cudaSuccess;
  std::call_once(attr_once, [] {
    attr_err = cudaFuncSetAttribute(tc_attention_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                    (int)kAttSmem);
  });
  HERO_CUDA_TRY(attr_err);
  const int q_groups = (n_q + kQT * kQTiles - 1) / (kQT * kQTiles);
  const long long grid = (long long)q_groups * heads * B;
  tc_attention_kernel<false><<<(unsigned)grid, kAttThreads, kAttSmem, s>>>(tm_q, tm_k, tm_v, (__nv_bfloat16*)o, n_q,
                                                                           N, heads, d_status);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

}  // namespace hero

// =============================================================================
// hero_attention_bf16_static: the same attention, for callers that must not allocate
// =============================================================================
// hero_attention_bf16 takes its status word from a cudaMalloc made on first use.  Some
// callers cannot afford that: a host thread inside a latency-critical serving loop (cudaMalloc
// and cudaFree synchronise the whole device), a process whose framework has already reserved all
// device memory for its own pool (the allocation would fail), or code that runs where the CUDA
// allocator must not be entered at all.  For them the scratch lives in the library image itself:
// a file-scope __device__ array that every GPU loading the library carries until the process
// exits (kStaticScratchInts * 4 bytes = 64.25 KiB per GPU).
//
// Layout: word 0 counts the CTAs of the latest call that gave up on a bounded wait, word 1 + i
// records CTA i.  The array is shared by every call and keeps the previous call's contents, so
// each call clears the words it is going to use on its stream before the kernel runs; two
// calls that overlap on the GPU (different streams, no dependency) race on it.
namespace hero {
namespace {

constexpr int kStaticMaxCtas = 16384;                 // largest grid the static scratch can serve
constexpr int kStaticScratchInts = 64 + kStaticMaxCtas;
static __device__ __align__(256) int g_att_static_scratch[kStaticScratchInts];

constexpr int kStaticMaxDevices = 64;
struct StaticSetup { bool done = false; int* scratch = nullptr; };
StaticSetup g_static_setup[kStaticMaxDevices];
std::mutex g_static_mutex;

// Once per device, with that device current: resolve the DEVICE address of the array (in host
// code the array's name is only a host-side handle, never a pointer a kernel may be given) and
// raise the kernel's dynamic shared-memory limit.
int static_setup(int** scratch) {
  int dev = -1;
  HERO_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kStaticMaxDevices) return HERO_ERR_ARG;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  StaticSetup& st = g_static_setup[dev];
  if (!st.done) {
    int* p = nullptr;
    HERO_CUDA_TRY(cudaGetSymbolAddress((void**)&p, g_att_static_scratch));
    HERO_CUDA_TRY(cudaFuncSetAttribute(tc_attention_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kAttSmem));
    st.scratch = p;
    st.done = true;
  }
  *scratch = st.scratch;
  return HERO_OK;
}

}  // namespace
}  // namespace hero

extern "C" int hero_attention_bf16_static(const void* d_q, const void* d_k, const void* d_v, void* d_o, int B,
                                          int n_q, int N, int heads, void* stream, int* h_gave_up) {
  using namespace hero;
  if (h_gave_up) *h_gave_up = 0;
  if (B < 0 || n_q < 0 || N <= 0 || heads <= 0) return HERO_ERR_ARG;
  if (B == 0 || n_q == 0) return HERO_OK;
  if (!d_q || !d_k || !d_v || !d_o) return HERO_ERR_ARG;
  if (!aligned16(d_q) || !aligned16(d_k) || !aligned16(d_v) || !aligned16(d_o)) return HERO_ERR_ALIGN;
  const long long q_groups = ((long long)n_q + kQT * kQTiles - 1) / (kQT * kQTiles);
  const long long grid = q_groups * heads * B;
  if (grid > kStaticMaxCtas) {
    set_cuda_error(cudaErrorInvalidConfiguration,
                   "hero_attention_bf16_static: ceil(n_q/256)*heads*B exceeds the 16384 CTAs its static scratch "
                   "serves; split the call or use hero_attention_bf16");
    return HERO_ERR_CAP;
  }
  cudaStream_t s = (cudaStream_t)stream;
  int* scratch = nullptr;
  HERO_TRY(static_setup(&scratch));
  const uint64_t D = (uint64_t)heads * kHD;
  CUtensorMap tm_q, tm_k, tm_v;
  {
    const uint64_t dims[2] = {D, (uint64_t)B * n_q};
    const uint64_t str[1] = {D * 2};
    const uint32_t box[2] = {(uint32_t)kHD, (uint32_t)kQT};
    HERO_TRY(make_tmap_bf16(&tm_q, d_q, 2, dims, str, box));
  }
  {
    const uint64_t dims[3] = {D, (uint64_t)N, (uint64_t)B};
    const uint64_t str[2] = {D * 2, (uint64_t)N * D * 2};
    const uint32_t box[3] = {(uint32_t)kHD, (uint32_t)kKT, 1};
    HERO_TRY(make_tmap_bf16(&tm_k, d_k, 3, dims, str, box));
    HERO_TRY(make_tmap_bf16(&tm_v, d_v, 3, dims, str, box));
  }
  // the array still holds the previous call's records: clear the words this grid will use
  HERO_CUDA_TRY(cudaMemsetAsync(scratch, 0, (size_t)(1 + grid) * sizeof(int), s));
  tc_attention_kernel<true><<<(unsigned)grid, kAttThreads, kAttSmem, s>>>(tm_q, tm_k, tm_v, (__nv_bfloat16*)d_o, n_q,
                                                                          N, heads, scratch);
  HERO_CUDA_TRY(cudaGetLastError());
  if (h_gave_up) {
    HERO_CUDA_TRY(cudaMemcpyAsync(h_gave_up, scratch, sizeof(int), cudaMemcpyDeviceToHost, s));
    HERO_CUDA_TRY(cudaStreamSynchronize(s));
    if (*h_gave_up != 0) return HERO_ERR_TIMEOUT;
  }
  return HERO_OK;
}
