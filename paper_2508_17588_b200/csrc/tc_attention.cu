// Flash-attention for the refresh path (Eq. 3 with the refreshed queries attending to the
// full cached K/V): O = softmax(Q K^T / sqrt(64)) V per (batch, head), bf16 in, fp32 softmax,
// no score matrix ever leaves the SM.
//
// One CTA = 128 query rows of one (batch, head); it streams all N cached keys in tiles of 128.
//   warp 0      TMA: Q tile once, then K/V tiles through a 4-stage ring (128-byte swizzle)
//   warp 1      tcgen05.mma issuer: S = Q K^T (M128 N128 K64) into TMEM, then O_j = P V
//               (M128 N64 K128) with P read from TMEM and V as an N-contiguous smem operand
//   warps 2..5  softmax: one thread per query row; running max / sum in registers, P written
//               back to TMEM as bf16, the running output rescaled and accumulated in registers
// S, P and the partial outputs are double-buffered in TMEM so that the MMAs of tile j+1
// overlap the softmax of tile j.
#include <cuda.h>

#include <mutex>

#include "hero_internal.h"
#include "tc_common.cuh"

namespace hero {

int make_tmap_bf16(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                   const uint32_t* box);

namespace {
using namespace tc;

constexpr int kQT = 128, kKT = 128, kHD = 64, kKvStages = 4;
constexpr int kQBytes = kQT * kHD * 2;       // 16 KB
constexpr int kKBytes = kKT * kHD * 2;       // 16 KB
constexpr int kKvStageBytes = 2 * kKBytes;   // K tile then V tile
constexpr int kAttThreads = 192;
constexpr size_t kAttSmem = 1024 + kQBytes + (size_t)kKvStages * kKvStageBytes + 256;
// TMEM columns: S0 S1 (128 each) | P0 P1 (64 each, bf16 pairs) | PV0 PV1 (64 each)
constexpr uint32_t kColS = 0, kColP = 256, kColPV = 384, kAttTmemCols = 512;

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__global__ void __launch_bounds__(kAttThreads, 1)
tc_attention_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ O, int n_q, int N,
                    int heads, int* __restrict__ status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s_q = smem;
  uint8_t* s_kv = smem + kQBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_kv + (size_t)kKvStages * kKvStageBytes);
  uint64_t* q_full = bars;
  uint64_t* kv_full = bars + 1;                    // [kKvStages]
  uint64_t* kv_empty = kv_full + kKvStages;        // [kKvStages]
  uint64_t* s_full = kv_empty + kKvStages;         // [2]
  uint64_t* p_full = s_full + 2;                   // [2]
  uint64_t* pv_full = p_full + 2;                  // [2]
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pv_full + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q_tiles = (n_q + kQT - 1) / kQT;
  const int qt = blockIdx.x % q_tiles;
  const int h = (blockIdx.x / q_tiles) % heads;
  const int b = blockIdx.x / (q_tiles * heads);
  const int n_kv = (N + kKT - 1) / kKT;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < kKvStages; ++i) { mbar_init(&kv_full[i], 1); mbar_init(&kv_empty[i], 1); }
    for (int i = 0; i < 2; ++i) { mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 4); mbar_init(&pv_full[i], 1); }
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
      mbar_expect_tx(q_full, kQBytes);
      tma_load_2d(s_q, &tm_q, q_full, h * kHD, b * n_q + qt * kQT);
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
      const uint64_t dq = smem_desc_sw128(smem_u32(s_q), 1024);
      auto issue_s = [&](int j) {
        const int st = j % kKvStages;
        const uint64_t dk = smem_desc_sw128(smem_u32(s_kv + (size_t)st * kKvStageBytes), 1024);
        const uint32_t d = tmem_base + kColS + (uint32_t)(j & 1) * kKT;
#pragma unroll
        for (int k = 0; k < kHD / 16; ++k) mma_ss(d, dq + 2 * k, dk + 2 * k, idesc_s, k != 0);
        mma_commit(&s_full[j & 1]);
      };
      bool ok = mbar_wait(q_full, 0, abort_flag);
      if (ok) ok = mbar_wait(&kv_full[0], 0, abort_flag);
      if (ok) { tc_fence_after(); issue_s(0); }
      for (int j = 0; j < n_kv && ok; ++j) {
        if (j + 1 < n_kv) {
          if (!(ok = mbar_wait(&kv_full[(j + 1) % kKvStages], ((j + 1) / kKvStages) & 1, abort_flag))) break;
          tc_fence_after();
          issue_s(j + 1);
        }
        if (!(ok = mbar_wait(&p_full[j & 1], (j >> 1) & 1, abort_flag))) break;
        tc_fence_after();
        const int st = j % kKvStages;
        // V tile: rows = keys (128 bytes each), 8-key groups 1024 bytes apart; 16 keys per MMA = 2048 bytes
        const uint64_t dv = smem_desc_sw128(smem_u32(s_kv + (size_t)st * kKvStageBytes + kKBytes), 1024);
        const uint32_t d = tmem_base + kColPV + (uint32_t)(j & 1) * kHD;
        const uint32_t a = tmem_base + kColP + (uint32_t)(j & 1) * (kKT / 2);
#pragma unroll
        for (int k = 0; k < kKT / 16; ++k) mma_ts(d, a + 8 * k, dv + 128 * k, idesc_pv, k != 0);
        mma_commit(&pv_full[j & 1]);
        mma_commit(&kv_empty[st]);
      }
    }
  } else {
    // ------------------------------------------------------------ softmax + output accumulation
    const int quad = warp & 3;
    const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16);
    const float c = 0.125f * 1.4426950408889634f;      // 1/sqrt(64) * log2(e)
    float m_run = -INFINITY, l_run = 0.f, alpha_pend = 0.f;
    float o[kHD];
#pragma unroll
    for (int i = 0; i < kHD; ++i) o[i] = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      ok = mbar_wait(&s_full[j & 1], (j >> 1) & 1, abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_s = lane_base + kColS + (uint32_t)(j & 1) * kKT;
      const int valid = N - j * kKT;                   // keys of this tile that exist (>= 1)
      // pass 1: row maximum
      float m_tile = -INFINITY;
#pragma unroll 1
      for (int ch = 0; ch < kKT / 32; ++ch) {
        uint32_t r[32];
        tmem_ld32(t_s + ch * 32, r);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float s = (ch * 32 + i < valid) ? __uint_as_float(r[i]) : -INFINITY;
          m_tile = fmaxf(m_tile, s);
        }
      }
      const float m_new = fmaxf(m_run, m_tile);
      const float alpha = ex2((m_run - m_new) * c);
      const float neg_mc = -m_new * c;
      // pass 2: probabilities, row sum, bf16 P back into TMEM (two keys per 32-bit column)
      float sum = 0.f;
      const uint32_t t_p = lane_base + kColP + (uint32_t)(j & 1) * (kKT / 2);
#pragma unroll 1
      for (int half = 0; half < 2; ++half) {
        uint32_t packed[32];
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
          uint32_t r[32];
          tmem_ld32(t_s + half * 64 + sub * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            const int col = half * 64 + sub * 32 + i;
            const float p0 = (col < valid) ? ex2(fmaf(__uint_as_float(r[i]), c, neg_mc)) : 0.f;
            const float p1 = (col + 1 < valid) ? ex2(fmaf(__uint_as_float(r[i + 1]), c, neg_mc)) : 0.f;
            sum += p0 + p1;
            const __nv_bfloat162 pk = __floats2bfloat162_rn(p0, p1);
            packed[sub * 16 + i / 2] = *reinterpret_cast<const uint32_t*>(&pk);
          }
        }
        tmem_st32(t_p + half * 32, packed);
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[j & 1]);
      // fold in the previous tile's P V while the tensor core works on this one
      if (j > 0) {
        ok = mbar_wait(&pv_full[(j - 1) & 1], ((j - 1) >> 1) & 1, abort_flag);
        ok = __all_sync(0xFFFFFFFFu, ok);
        if (!ok) break;
        tc_fence_after();
        const uint32_t t_pv = lane_base + kColPV + (uint32_t)((j - 1) & 1) * kHD;
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t r[32];
          tmem_ld32(t_pv + ch * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[ch * 32 + i] = fmaf(o[ch * 32 + i], alpha_pend, __uint_as_float(r[i]));
        }
      }
      l_run = fmaf(l_run, alpha, sum);
      alpha_pend = alpha;
      m_run = m_new;
    }
    if (ok) {
      const int jl = n_kv - 1;
      ok = mbar_wait(&pv_full[jl & 1], (jl >> 1) & 1, abort_flag);
      ok = __all_sync(0xFFFFFFFFu, ok);
      if (ok) {
        tc_fence_after();
        const uint32_t t_pv = lane_base + kColPV + (uint32_t)(jl & 1) * kHD;
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t r[32];
          tmem_ld32(t_pv + ch * 32, r);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[ch * 32 + i] = fmaf(o[ch * 32 + i], alpha_pend, __uint_as_float(r[i]));
        }
        const int qi = qt * kQT + quad * 32 + lane;
        if (qi < n_q) {
          const float inv = 1.0f / l_run;
          __nv_bfloat16* dst = O + ((long long)b * n_q + qi) * ((long long)heads * kHD) + h * kHD;
#pragma unroll
          for (int v = 0; v < kHD / 8; ++v) {
            uint32_t w[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
              const __nv_bfloat162 pk = __floats2bfloat162_rn(o[v * 8 + 2 * q] * inv, o[v * 8 + 2 * q + 1] * inv);
              w[q] = *reinterpret_cast<const uint32_t*>(&pk);
            }
            *reinterpret_cast<uint4*>(dst + v * 8) = make_uint4(w[0], w[1], w[2], w[3]);
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) atomicExch(status, 2);
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
    attr_err = cudaFuncSetAttribute(tc_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttSmem);
  });
  HERO_CUDA_TRY(attr_err);
  const int q_tiles = (n_q + kQT - 1) / kQT;
  const long long grid = (long long)q_tiles * heads * B;
  tc_attention_kernel<<<(unsigned)grid, kAttThreads, kAttSmem, s>>>(tm_q, tm_k, tm_v, (__nv_bfloat16*)o, n_q, N,
                                                                    heads, d_status);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

}  // namespace hero
