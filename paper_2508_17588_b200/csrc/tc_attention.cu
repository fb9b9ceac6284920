// Flash-attention for the refresh path (Eq. 3 with the refreshed queries attending to the
// full cached K/V): O = softmax(Q K^T / sqrt(64)) V per (batch, head), bf16 in, fp32 softmax,
// no score matrix ever leaves the SM.
//
// One CTA = 256 query rows (two tiles of 128) of one (batch, head); it streams all N cached
// keys in tiles of 96 through a 6-stage TMA ring shared by both query tiles.  TMEM (512
// columns): per query tile two score buffers of 96 columns (key tile parity) and one 64-column
// output accumulator; P (bf16) is written over the scores it was computed from and is the TMEM
// operand of O += P V.  S of tile j+2 is issued right after P V of tile j (same issuer, executed
// in issue order), so a score tile is normally ready a whole softmax iteration before it is needed.
//
// Two kernels share this layout:
//
//  * tc_attention_fast_kernel, the one that normally does all the work.  20 warps: TMA producer, one
//    tcgen05.mma issuer warp per query tile (all lanes run the loop, one elected lane issues, so that
//    the operands stay warp-uniform), and SIXTEEN softmax warps: every query row is shared by two
//    threads, each owning 48 of a key tile's 96 score columns.  A warp issues in order and stalls on
//    every ex2 while the special-function unit is busy and on every barrier, fence and TMEM round
//    trip at a tile boundary; with four softmax warps per SM sub-partition instead of two there is
//    always another warp with exponentials ready, which is what keeps that unit (the bound of this
//    kernel at head_dim 64: 16 ex2 per clock per SM against 256 tensor flops per score) busy.
//    The two threads of a row never talk in steady state: the row's scaling maximum is fixed by the
//    first key tile (one exchange through shared memory) and never moves, so a tile is ONE pass -
//    p = 2^((s - m) c), row sum, bf16 pack, store - with no running maximum, no vote and no redo.
//    That is exact as long as no later score exceeds the first tile's maximum by more than 2^100
//    (69 in natural-log units; bf16 and fp32 share their exponent range, so a large p loses no
//    precision, and the final division by the row sum makes the result independent of the maximum
//    used).  The row sum tells whether that held; a CTA in which it did not says so in its status word.
//    In the step the QKV projection hands over q already multiplied by log2(e) / sqrt(64), so a score is
//    the exponent of its weight: that instantiation (PRESCALED) takes p = 2^s as it stands - no maximum,
//    no first-tile exchange, no multiply-add per pair of scores - and is exact while a row's largest score
//    stays within about +-100; its row sum must then lie in [2^-100, 2^100), else the CTA is marked.
//  * tc_attention_safe_kernel recomputes exactly those CTAs (same grid, every other CTA returns at
//    once) with a running maximum that moves whenever a tile exceeds it by 2^8, rescaling the
//    accumulator in TMEM; it is also the whole computation when no per-CTA status words are available.
//    12 warps, one thread per row, one-pass tiles with a two-pass redo when the maximum has to move.
//
#include <cuda.h>

#include <mutex>

#include "hero_internal.h"
#include "tc_common.cuh"

#ifndef HERO_ATT_CHUNK
#define HERO_ATT_CHUNK 16
#endif

namespace hero {

int make_tmap_bf16(CUtensorMap* m, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                   const uint32_t* box);

namespace {
using namespace tc;

constexpr int kQT = 128, kQTiles = 2, kKT = 96, kHD = 64, kKvStages = 6;
constexpr int kQBytes = kQT * kHD * 2;       // 16 KB per query tile
constexpr int kKBytes = kKT * kHD * 2;       // 12 KB (a multiple of the 1024-byte swizzle atom)
constexpr int kKvStageBytes = 2 * kKBytes;   // K tile then V tile
constexpr int kFirstSoftmaxWarp = 4;
constexpr int kAttThreads = 32 * (kFirstSoftmaxWarp + 4 * kQTiles);   // 12 warps
constexpr size_t kAttSmem = 1024 + kQTiles * kQBytes + (size_t)kKvStages * kKvStageBytes + 512;
constexpr uint32_t kTileCols = 256, kColO = 2 * kKT, kAttTmemCols = 512;   // per tile: S0 | S1 | O
constexpr float kRescaleLog2 = 8.0f;           // the scaling maximum moves only when exceeded by 2^8
static_assert(2 * kKT + kHD <= (int)kTileCols && kQTiles * kTileCols <= kAttTmemCols, "TMEM layout");
static_assert(kKBytes % 1024 == 0 && kKT % 16 == 0, "tile shape");

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

// One key tile of one query row.  The kKT scores of the row are read from TMEM in one burst
// (a single wait for the whole row instead of one per chunk), reduced to their maximum, turned
// into p = 2^(s*c - m*c) and written back as bf16 pairs over columns [0, kKT/2) of the same
// buffer.  m_used is the maximum the row's P and accumulator are scaled by: it only moves when
// this tile exceeds it by more than 2^kRescaleLog2 (always at the first tile), and alpha is then
// the factor that the sum and the accumulator take.  Returns the row sum of p.
template <bool MASKED>
__device__ __forceinline__ float softmax_tile(uint32_t t_buf, int valid, float c, float& m_used, float& alpha,
                                              bool& grow) {
  uint32_t s[kKT];
#pragma unroll
  for (int ch = 0; ch < kKT / 32; ++ch) tmem_ld32(t_buf + ch * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[ch * 32]));
  tmem_ld_wait();
  if (MASKED) {
#pragma unroll
    for (int i = 0; i < kKT; ++i)
      if (i >= valid) s[i] = 0xFF800000u;   // -inf
  }
  float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
  for (int i = 0; i < kKT; i += 8) {
#pragma unroll
    for (int q = 0; q < 4; ++q) mx[q] = fmaxf(mx[q], fmaxf(__uint_as_float(s[i + 2 * q]), __uint_as_float(s[i + 2 * q + 1])));
  }
  const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3]));
  grow = (m_tile - m_used) * c > kRescaleLog2;                 // true at the first tile (m_used = -inf)
  const float m_new = grow ? m_tile : m_used;
  alpha = grow ? ex2((m_used - m_new) * c) : 1.0f;             // 0 at the first tile
  m_used = m_new;
  const float neg_mc = -m_new * c;
  const float2 c2 = make_float2(c, c), nm2 = make_float2(neg_mc, neg_mc);
  float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
  for (int ch = 0; ch < kKT / 32; ++ch) {
    uint32_t packed[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {       // pair i = columns 2i, 2i+1 of this 32-column chunk
      const int col = ch * 32 + 2 * i;
      const float2 x = __ffma2_rn(f2(s[col], s[col + 1]), c2, nm2);
      float2 p = make_float2(ex2(x.x), ex2(x.y));
      if (MASKED) {
        if (col >= valid) p.x = 0.f;
        if (col + 1 >= valid) p.y = 0.f;
      }
      acc[i & 3] = __fadd2_rn(acc[i & 3], p);
      const __nv_bfloat162 b = __floats2bfloat162_rn(p.x, p.y);
      packed[i] = *reinterpret_cast<const uint32_t*>(&b);
    }
    tmem_st16(t_buf + ch * 16, packed);
  }
  const float2 a01 = __fadd2_rn(acc[0], acc[1]), a23 = __fadd2_rn(acc[2], acc[3]);
  return (a01.x + a01.y) + (a23.x + a23.y);
}

// The common case of a key tile, in ONE pass over the row: p = 2^((s - m_used) c) with the maximum
// the row is already scaled by, the tile's own maximum tracked on the side.  The caller checks the
// maximum afterwards and falls back to softmax_tile (S is still intact: P is only kept in
// registers here) in the rare case that it has to move.  Doing without the separate maximum pass
// matters because that pass issues nothing to the exponential unit for a third of the tile.  The
// scores are read kCh columns at a time, one read ahead; short reads keep the register count low
// enough for the compiler to overlap the pairs freely (16 columns measured 4 % faster than 32).
__device__ __forceinline__ void fused_tile(uint32_t t_buf, float c, float neg_mc, uint32_t (&packed)[kKT / 2],
                                           float& sum, float& m_tile) {
  const float2 c2 = make_float2(c, c), nm2 = make_float2(neg_mc, neg_mc);
  float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
  float mx[2] = {-INFINITY, -INFINITY};
  constexpr int kCh = HERO_ATT_CHUNK;                  // score columns per TMEM read
  uint32_t ra[kCh], rb[kCh];
  if (kCh == 32) tmem_ld32(t_buf, *reinterpret_cast<uint32_t(*)[32]>(&ra[0]));
  else tmem_ld16(t_buf, *reinterpret_cast<uint32_t(*)[16]>(&ra[0]));
#pragma unroll
  for (int ch = 0; ch < kKT / kCh; ++ch) {
    uint32_t(&cur)[kCh] = (ch & 1) ? rb : ra;
    uint32_t(&nxt)[kCh] = (ch & 1) ? ra : rb;
    tmem_ld_wait();
    if (ch + 1 < kKT / kCh) {
      if (kCh == 32) tmem_ld32(t_buf + (ch + 1) * kCh, *reinterpret_cast<uint32_t(*)[32]>(&nxt[0]));
      else tmem_ld16(t_buf + (ch + 1) * kCh, *reinterpret_cast<uint32_t(*)[16]>(&nxt[0]));
    }
#pragma unroll
    for (int i = 0; i < kCh / 2; ++i) {
      const float2 x = __ffma2_rn(f2(cur[2 * i], cur[2 * i + 1]), c2, nm2);
      const float2 p = make_float2(ex2(x.x), ex2(x.y));
      acc[i & 3] = __fadd2_rn(acc[i & 3], p);
      const __nv_bfloat162 b = __floats2bfloat162_rn(p.x, p.y);
      packed[ch * (kCh / 2) + i] = *reinterpret_cast<const uint32_t*>(&b);
      mx[i & 1] = max3(mx[i & 1], __uint_as_float(cur[2 * i]), __uint_as_float(cur[2 * i + 1]));
    }
  }
  const float2 a01 = __fadd2_rn(acc[0], acc[1]), a23 = __fadd2_rn(acc[2], acc[3]);
  sum = (a01.x + a01.y) + (a23.x + a23.y);
  m_tile = fmaxf(mx[0], mx[1]);
}

// Status words: status[0] counts the CTAs that gave up on a bounded wait; cta_words (may be null) holds one
// word per CTA: 0 = done, 1 = the fast kernel's range assumption failed here (to be recomputed), 2 = gave up.
// With cta_words given, this kernel only works on the CTAs marked 1.
__global__ void __launch_bounds__(kAttThreads, 1)
tc_attention_safe_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                         const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ O, int n_q, int N,
                         int heads, const float c, int* __restrict__ status, int* __restrict__ cta_words) {
  if (cta_words != nullptr && cta_words[blockIdx.x] != 1) return;      // block-uniform
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s_q = smem;
  uint8_t* s_kv = smem + kQTiles * kQBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_kv + (size_t)kKvStages * kKvStageBytes);
  uint64_t* q_full = bars;
  uint64_t* kv_full = bars + 1;                    // [kKvStages]           TMA -> both issuers
  uint64_t* kv_empty = kv_full + kKvStages;        // [kKvStages], count 2  both issuers -> TMA
  uint64_t* s_full = kv_empty + kKvStages;         // [qt][parity]  issuer -> softmax: S is ready
  uint64_t* p_full = s_full + 4;                   // [qt][parity]  softmax -> issuer: P is in TMEM
  uint64_t* pv_full = p_full + 4;                  // [qt]          issuer -> softmax: P V of tile j done (phase j)
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pv_full + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q_groups = (n_q + kQT * kQTiles - 1) / (kQT * kQTiles);
  const int qg = blockIdx.x % q_groups;
  const int h = (blockIdx.x / q_groups) % heads;
  const int b = blockIdx.x / (q_groups * heads);
  const int n_kv = (N + kKT - 1) / kKT;
  // the last query group of a (batch, head) may reach into its second tile by no row at all: that tile's
  // issuer and softmax warps then have nothing to do and the K/V stages are released by one issuer alone
  const int n_tiles = (qg * kQTiles + 1) * kQT < n_q ? kQTiles : 1;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < kKvStages; ++i) { mbar_init(&kv_full[i], 1); mbar_init(&kv_empty[i], n_tiles); }
    for (int i = 0; i < 4; ++i) { mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 4); }
    for (int i = 0; i < kQTiles; ++i) mbar_init(&pv_full[i], 1);
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
      mbar_expect_tx(q_full, n_tiles * kQBytes);
      for (int t = 0; t < n_tiles; ++t)
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
  } else if (warp == 1 || warp == 2) {
    // ------------------------------------------------------------ MMA issuer of query tile t
    if (lane == 0 && warp - 1 < n_tiles) {
      const int t = warp - 1;
      constexpr uint32_t idesc_s = idesc_bf16(kQT, kKT, 0);    // S = Q K^T : both operands K-contiguous
      constexpr uint32_t idesc_pv = idesc_bf16(kQT, kHD, 1);   // O += P V  : V is N(head_dim)-contiguous
      const uint64_t dq = smem_desc_sw128(smem_u32(s_q + t * kQBytes), 1024);
      const uint32_t t_tile = tmem_base + (uint32_t)t * kTileCols;
      auto issue_s = [&](int j) {
        const int st = j % kKvStages;
        const uint64_t dk = smem_desc_sw128(smem_u32(s_kv + (size_t)st * kKvStageBytes), 1024);
        const uint32_t d = t_tile + (uint32_t)(j & 1) * kKT;
#pragma unroll
        for (int k = 0; k < kHD / 16; ++k) mma_ss(d, dq + 2 * k, dk + 2 * k, idesc_s, k != 0);
        mma_commit(&s_full[t * 2 + (j & 1)]);
      };
      bool ok = mbar_wait(q_full, 0, abort_flag);
      for (int j = 0; j < 2 && j < n_kv && ok; ++j) {           // two score tiles ahead of the softmax
        if ((ok = mbar_wait(&kv_full[j], 0, abort_flag))) { tc_fence_after(); issue_s(j); }
      }
      for (int j = 0; j < n_kv && ok; ++j) {
        const int st = j % kKvStages;
        // V tile: rows = keys (128 bytes each), 8-key groups 1024 bytes apart; 16 keys per MMA = 2048 bytes
        const uint64_t dv = smem_desc_sw128(smem_u32(s_kv + (size_t)st * kKvStageBytes + kKBytes), 1024);
        if (!(ok = mbar_wait(&p_full[t * 2 + (j & 1)], (j >> 1) & 1, abort_flag))) break;
        tc_fence_after();
        const uint32_t buf = t_tile + (uint32_t)(j & 1) * kKT;
#pragma unroll
        for (int k = 0; k < kKT / 16; ++k) mma_ts(t_tile + kColO, buf + 8 * k, dv + 128 * k, idesc_pv, (j | k) != 0);
        mma_commit(&pv_full[t]);
        mma_commit(&kv_empty[st]);               // second arrival comes from the other tile's issuer
        if (j + 2 < n_kv) {
          // S of tile j+2 overwrites the buffer whose P the product above reads: safe because the
          // tensor core executes this thread's MMAs in issue order
          if (!(ok = mbar_wait(&kv_full[(j + 2) % kKvStages], ((j + 2) / kKvStages) & 1, abort_flag))) break;
          tc_fence_after();
          issue_s(j + 2);
        }
      }
    }
  } else if (warp >= kFirstSoftmaxWarp && ((warp - kFirstSoftmaxWarp) >> 2) < n_tiles) {
    // ------------------------------------------------------------ softmax
    const int t = (warp - kFirstSoftmaxWarp) >> 2;     // query tile of this softmax group
    const int quad = warp & 3;                         // TMEM lane quadrant this warp may touch
    const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)t * kTileCols;
    float m_used = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      ok = mbar_wait_warp(&s_full[t * 2 + (j & 1)], (j >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_buf = lane_base + (uint32_t)(j & 1) * kKT;
      const int valid = N - j * kKT;                   // keys of this tile that exist (>= 1)
      const bool ragged = valid < kKT;
      float alpha = 1.0f, sum;
      bool grow = true;                                // first and ragged tiles take the two-pass path
      uint32_t packed[kKT / 2];
      if (j > 0 && !ragged) {
        float m_tile;
        fused_tile(t_buf, c, -m_used * c, packed, sum, m_tile);
        grow = __any_sync(0xFFFFFFFFu, (m_tile - m_used) * c > kRescaleLog2);
      }
      if (grow) {                                      // warp-uniform
        bool moved;
        sum = ragged ? softmax_tile<true>(t_buf, valid, c, m_used, alpha, moved)
                     : softmax_tile<false>(t_buf, valid, c, m_used, alpha, moved);
      } else {
#pragma unroll
        for (int ch = 0; ch < kKT / 32; ++ch)
          tmem_st16(t_buf + ch * 16, *reinterpret_cast<uint32_t(*)[16]>(&packed[ch * 16]));
      }
      l_run = fmaf(l_run, alpha, sum);
      if (j > 0 && grow) {
        // Rare (warp-uniform): the maximum moved, so the accumulator is scaled down before this tile's
        // product is added to it - once P V of tile j-1 has completed.  pv_full is only looked at here and
        // at the very end, yet the parity wait is unambiguous: S of tile j was issued after P V of tile j-2
        // (so that one is complete) and P V of tile j cannot start before this warp's arrival below, hence
        // the barrier has completed either j-1 or j phases and "phase j-1 complete" is exactly the question.
        ok = mbar_wait_warp(&pv_full[t], (j - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const float2 a2 = make_float2(alpha, alpha);     // alpha is 1 for rows that did not move
#pragma unroll
        for (int ch = 0; ch < kHD / 16; ++ch) {
          uint32_t r[16];
          tmem_ld16(lane_base + kColO + ch * 16, r);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; i += 2) {
            const float2 v = __fmul2_rn(f2(r[i], r[i + 1]), a2);
            r[i] = __float_as_uint(v.x); r[i + 1] = __float_as_uint(v.y);
          }
          tmem_st16(lane_base + kColO + ch * 16, r);
        }
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[t * 2 + (j & 1)]);
    }
    if (ok) ok = mbar_wait_warp(&pv_full[t], (n_kv - 1) & 1, abort_flag);
    if (ok) {
      tc_fence_after();
      const int qi = (qg * kQTiles + t) * kQT + quad * 32 + lane;
      const float inv = 1.0f / l_run;
      __nv_bfloat16* dst = O + ((long long)b * n_q + qi) * ((long long)heads * kHD) + h * kHD;
#pragma unroll
      for (int ch = 0; ch < kHD / 16; ++ch) {
        uint32_t r[16];
        tmem_ld16(lane_base + kColO + ch * 16, r);     // warp-collective: every lane loads
        tmem_ld_wait();
        if (qi < n_q) {
          uint32_t w[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            const __nv_bfloat162 pk = __floats2bfloat162_rn(__uint_as_float(r[2 * q]) * inv,
                                                            __uint_as_float(r[2 * q + 1]) * inv);
            w[q] = *reinterpret_cast<const uint32_t*>(&pk);
          }
          *reinterpret_cast<uint4*>(dst + ch * 16) = make_uint4(w[0], w[1], w[2], w[3]);
          *reinterpret_cast<uint4*>(dst + ch * 16 + 8) = make_uint4(w[4], w[5], w[6], w[7]);
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    if (*abort_flag) atomicAdd(status, 1);
    if (cta_words != nullptr) cta_words[blockIdx.x] = *abort_flag ? 2 : 0;
  }
  if (warp == 1) { __syncwarp(); tc_fence_after(); tmem_dealloc(tmem_base, kAttTmemCols); }
}

// =============================================================================================
// The fast kernel
// =============================================================================================
constexpr int kFastSoftmaxWarps = 16;            // 2 query tiles x 4 TMEM lane quadrants x 2 column halves
constexpr int kFastThreads = 32 * (kFirstSoftmaxWarp + kFastSoftmaxWarps);   // 20 warps
constexpr int kHalf = kKT / 2;                   // score columns of a key tile that one thread owns
constexpr int kXchgFloats = kQTiles * kQT * 2;   // one slot per (query row, column half)
constexpr size_t kFastSmem = kAttSmem + 2 * kXchgFloats * sizeof(float) + 64;
constexpr float kRowSumLimit = 1.2676506e30f;    // 2^100: a row sum at or beyond it voids the fixed-maximum assumption
constexpr float kRowSumFloor = 7.8886091e-31f;   // 2^-100: below it a row without a maximum has lost its small terms
static_assert(kHalf % 16 == 0 && (kHalf / 16) % 2 == 1, "three 16-column reads per half: the ping-pong below ends on ra");

// 2^x for two scores on the FMA pipe instead of the special-function unit (Cody-Waite reduction + a cubic).
// The unit evaluates 16 ex2 per clock per SM and is what bounds this kernel; every pair moved here frees two of
// its slots for ten FMA/ALU-pipe instructions, which the four softmax warps per sub-partition have to spare.
//   xs = sat(x / 250 + 1/2)            x clamped to [-125, 125] by the saturating FMA (x = s c - m c is formed here)
//   t  = xs * 250 + (M - 125)          M = 1.5 * 2^23: the sum rounds to M + n, n = round(x), held in t's low bits
//   f  = xs * 250 + ((M - 125) - t)    x - n, in [-1/2, 1/2]
//   2^f ~ C0 + f (C1 + f (C2 + f C3))  minimax cubic for the relative error on [-1/2, 1/2]: 7.5e-5, a fiftieth of the
//                                      bf16 rounding P goes through (coefficients from a Lawson-weighted least-squares fit)
//   result = bits(2^f) + (bits(t) << 23)   adds n to the exponent field: 127 - 125 .. 127 + 125 stays a normal number
// A score that the clamp cuts off at +125 still yields 2^125, far beyond the row-sum limit, so the row is caught.
#ifndef HERO_ATT_POLY_PAIRS
#define HERO_ATT_POLY_PAIRS 1          // of every 8 pairs of scores (1 measured best: 2.22 ms against 2.40 with none, 2.33 with 2)
#endif
#ifndef HERO_ATT_POLY_PAIRS_PRESCALED
#define HERO_ATT_POLY_PAIRS_PRESCALED 2   // with the scale folded into q a pair costs the pipes one instruction less: 2 is best
#endif
constexpr int kPolyPairs = HERO_ATT_POLY_PAIRS, kPolyPairsPrescaled = HERO_ATT_POLY_PAIRS_PRESCALED;
constexpr float kPolySpan = 250.0f, kPolyMagic = 12582912.0f - 125.0f;
__device__ __forceinline__ float fma_sat(float a, float b, float c) {
  float y;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(y) : "f"(a), "f"(b), "f"(c));
  return y;
}
__device__ __forceinline__ float2 exp2_poly_pair(float s0, float s1, float cs, float bs) {
  const float2 xs = make_float2(fma_sat(s0, cs, bs), fma_sat(s1, cs, bs));
  const float2 span = make_float2(kPolySpan, kPolySpan), mg = make_float2(kPolyMagic, kPolyMagic);
  const float2 t = __ffma2_rn(xs, span, mg);
  const float2 f = __ffma2_rn(xs, span, __ffma2_rn(t, make_float2(-1.0f, -1.0f), mg));
  float2 p = __ffma2_rn(f, make_float2(0.0551716648f, 0.0551716648f), make_float2(0.2426111251f, 0.2426111251f));
  p = __ffma2_rn(p, f, make_float2(0.6932609677f, 0.6932609677f));
  p = __ffma2_rn(p, f, make_float2(0.9999280572f, 0.9999280572f));
  return make_float2(__int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23)),
                     __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23)));
}

// One key tile of one thread's 48 columns, steady state: the scores are read 16 columns at a time (one read
// ahead), turned into p = 2^(s c - m c), summed, packed to bf16 and written back over the columns just read -
// half h keeps its P in the first 24 columns of its own 48, so neither half ever writes what the other reads.
// MASKED (the ragged last tile): columns at or beyond `valid` are keys that do not exist.
// PRESCALED: the scores are exponents already (x = s, see the kernel below), one instruction less per pair.
template <bool MASKED, bool PRESCALED>
__device__ __forceinline__ float half_tile(uint32_t t_s, int valid, const float2 c2, const float2 nm2, float cs, float bs) {
  float2 acc[4] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
  uint32_t ra[16], rb[16];
  tmem_ld16(t_s, ra);
#pragma unroll
  for (int ch = 0; ch < kHalf / 16; ++ch) {
    uint32_t(&cur)[16] = (ch & 1) ? rb : ra;
    uint32_t(&nxt)[16] = (ch & 1) ? ra : rb;
    tmem_ld_wait();
    if (ch + 1 < kHalf / 16) tmem_ld16(t_s + (ch + 1) * 16, nxt);
    uint32_t pk[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      float2 p;
      constexpr int kPoly = PRESCALED ? kPolyPairsPrescaled : kPolyPairs;
      if ((i * kPoly) % 8 < kPoly) {                    // spread evenly over the chunk (resolved at compile time)
        p = exp2_poly_pair(__uint_as_float(cur[2 * i]), __uint_as_float(cur[2 * i + 1]), cs, bs);
      } else {
        const float2 x = PRESCALED ? f2(cur[2 * i], cur[2 * i + 1]) : __ffma2_rn(f2(cur[2 * i], cur[2 * i + 1]), c2, nm2);
        p = make_float2(ex2(x.x), ex2(x.y));
      }
      if (MASKED) {
        if (ch * 16 + 2 * i >= valid) p.x = 0.f;
        if (ch * 16 + 2 * i + 1 >= valid) p.y = 0.f;
      }
      acc[i & 3] = __fadd2_rn(acc[i & 3], p);
      const __nv_bfloat162 b = __floats2bfloat162_rn(p.x, p.y);
      pk[i] = *reinterpret_cast<const uint32_t*>(&b);
    }
    tmem_st8(t_s + ch * 8, pk);
  }
  const float2 a01 = __fadd2_rn(acc[0], acc[1]), a23 = __fadd2_rn(acc[2], acc[3]);
  return (a01.x + a01.y) + (a23.x + a23.y);
}

template <bool PRESCALED>
__global__ void __launch_bounds__(kFastThreads, 1)
tc_attention_fast_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                         const __grid_constant__ CUtensorMap tm_v, __nv_bfloat16* __restrict__ O, int n_q, int N,
                         int heads, int* __restrict__ status, int* __restrict__ cta_words) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* s_q = smem;
  uint8_t* s_kv = smem + kQTiles * kQBytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(s_kv + (size_t)kKvStages * kKvStageBytes);
  uint64_t* q_full = bars;
  uint64_t* kv_full = bars + 1;                    // [kKvStages]           TMA -> both issuers
  uint64_t* kv_empty = kv_full + kKvStages;        // [kKvStages], count 2  both issuers -> TMA
  uint64_t* s_full = kv_empty + kKvStages;         // [qt][parity]  issuer -> softmax: S is ready
  uint64_t* p_full = s_full + 4;                   // [qt][parity]  softmax -> issuer: P is in TMEM (8 warps)
  uint64_t* pv_full = p_full + 4;                  // [qt]          issuer -> softmax: the last P V is done
  uint64_t* pair_bar = pv_full + 2;                // [qt][quadrant] the two warps that share 32 query rows
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(pair_bar + 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  int* cta_bad = const_cast<int*>(abort_flag) + 1;
  float* xchg_m = reinterpret_cast<float*>(smem + kAttSmem - 1024);   // behind the barrier block (512 bytes are plenty)
  float* xchg_l = xchg_m + kXchgFloats;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int q_groups = (n_q + kQT * kQTiles - 1) / (kQT * kQTiles);
  const int qg = blockIdx.x % q_groups;
  const int h = (blockIdx.x / q_groups) % heads;
  const int b = blockIdx.x / (q_groups * heads);
  const int n_kv = (N + kKT - 1) / kKT;
  // the last query group of a (batch, head) may reach into its second tile by no row at all: that tile's
  // issuer and softmax warps then have nothing to do and the K/V stages are released by one issuer alone
  const int n_tiles = (qg * kQTiles + 1) * kQT < n_q ? kQTiles : 1;

  if (threadIdx.x == 0) {
    mbar_init(q_full, 1);
    for (int i = 0; i < kKvStages; ++i) { mbar_init(&kv_full[i], 1); mbar_init(&kv_empty[i], n_tiles); }
    for (int i = 0; i < 4; ++i) { mbar_init(&s_full[i], 1); mbar_init(&p_full[i], 8); }
    for (int i = 0; i < kQTiles; ++i) mbar_init(&pv_full[i], 1);
    for (int i = 0; i < 8; ++i) mbar_init(&pair_bar[i], 2);
    *abort_flag = 0;
    *cta_bad = 0;
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
      mbar_expect_tx(q_full, n_tiles * kQBytes);
      for (int t = 0; t < n_tiles; ++t)
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
  } else if (warp == 1 || warp == 2) {
    // ------------------------------------------------------------ MMA issuer warp of query tile t
    if (warp - 1 < n_tiles) {
      const bool leader = elect_one();
      const int t = warp - 1;
      constexpr uint32_t idesc_s = idesc_bf16(kQT, kKT, 0);    // S = Q K^T : both operands K-contiguous
      constexpr uint32_t idesc_pv = idesc_bf16(kQT, kHD, 1);   // O += P V  : V is N(head_dim)-contiguous
      const uint64_t dq = smem_desc_sw128(smem_u32(s_q + t * kQBytes), 1024);
      const uint32_t t_tile = tmem_base + (uint32_t)t * kTileCols;
      auto issue_s = [&](int j) {
        const int st = j % kKvStages;
        const uint64_t dk = smem_desc_sw128(smem_u32(s_kv + (size_t)st * kKvStageBytes), 1024);
        const uint32_t d = t_tile + (uint32_t)(j & 1) * kKT;
        if (leader) {
#pragma unroll
          for (int k = 0; k < kHD / 16; ++k) mma_ss(d, dq + 2 * k, dk + 2 * k, idesc_s, k != 0);
          mma_commit(&s_full[t * 2 + (j & 1)]);
        }
      };
      bool ok = mbar_wait_warp(q_full, 0, abort_flag);
      for (int j = 0; j < 2 && j < n_kv && ok; ++j) {           // two score tiles ahead of the softmax
        if ((ok = mbar_wait_warp(&kv_full[j], 0, abort_flag))) { tc_fence_after(); issue_s(j); }
      }
      for (int j = 0; j < n_kv && ok; ++j) {
        const int st = j % kKvStages;
        // V tile: rows = keys (128 bytes each), 8-key groups 1024 bytes apart; 16 keys per MMA = 2048 bytes
        const uint64_t dv = smem_desc_sw128(smem_u32(s_kv + (size_t)st * kKvStageBytes + kKBytes), 1024);
        if (!(ok = mbar_wait_warp(&p_full[t * 2 + (j & 1)], (j >> 1) & 1, abort_flag))) break;
        tc_fence_after();
        const uint32_t buf = t_tile + (uint32_t)(j & 1) * kKT;
        if (leader) {
          // P of keys [16k, 16k+16) sits in 8 columns: the first 48 keys in columns [0, 24) of the buffer,
          // the last 48 in columns [48, 72) (each half of the softmax writes inside its own score columns)
#pragma unroll
          for (int k = 0; k < kKT / 16; ++k)
            mma_ts(t_tile + kColO, buf + (k / 3) * kHalf + (k % 3) * 8, dv + 128 * k, idesc_pv, (j | k) != 0);
          if (j == n_kv - 1) mma_commit(&pv_full[t]);
          mma_commit(&kv_empty[st]);             // second arrival comes from the other tile's issuer
        }
        if (j + 2 < n_kv) {
          // S of tile j+2 overwrites the buffer whose P the product above reads: safe because the
          // tensor core executes this thread's MMAs in issue order
          if (!(ok = mbar_wait_warp(&kv_full[(j + 2) % kKvStages], ((j + 2) / kKvStages) & 1, abort_flag))) break;
          tc_fence_after();
          issue_s(j + 2);
        }
      }
    }
  } else if (warp >= kFirstSoftmaxWarp && (((warp - kFirstSoftmaxWarp) >> 2) & 1) < n_tiles) {
    // ------------------------------------------------------------ softmax
    const int sid = warp - kFirstSoftmaxWarp;
    const int t = (sid >> 2) & 1;                      // query tile
    const int hh = sid >> 3;                           // which 48 of a tile's 96 score columns
    const int quad = warp & 3;                         // TMEM lane quadrant this warp may touch
    const int row = quad * 32 + lane;                  // query row within the tile
    const uint32_t lane_base = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)t * kTileCols;
    uint64_t* my_pair = &pair_bar[t * 4 + quad];
    const float c = PRESCALED ? 1.0f : kScoreScaleLog2;
    const float2 c2 = make_float2(c, c);
    float2 nm2 = make_float2(0.f, 0.f);
    const float cs = c / kPolySpan;
    float bs = 0.5f;
    float l_half = 0.f;
    uint32_t pair_phase = 0;
    bool ok = true;
    for (int j = 0; j < n_kv; ++j) {
      ok = mbar_wait_warp(&s_full[t * 2 + (j & 1)], (j >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const uint32_t t_s = lane_base + (uint32_t)(j & 1) * kKT + (uint32_t)hh * kHalf;
      int valid = N - j * kKT - hh * kHalf;            // columns of this half that are keys
      valid = valid < 0 ? 0 : (valid > kHalf ? kHalf : valid);
      if (!PRESCALED && j == 0) {
        // First tile: the maximum over its (existing) keys becomes the row's scaling maximum for good.
        // Both halves read their columns, trade their maxima through shared memory, and then form P
        // from the scores they still hold in registers.
        uint32_t s[kHalf];
#pragma unroll
        for (int ch = 0; ch < kHalf / 16; ++ch) tmem_ld16(t_s + ch * 16, *reinterpret_cast<uint32_t(*)[16]>(&s[ch * 16]));
        tmem_ld_wait();
        float m = -INFINITY;
#pragma unroll
        for (int i = 0; i < kHalf; ++i)
          if (i < valid) m = fmaxf(m, __uint_as_float(s[i]));
        xchg_m[(t * kQT + row) * 2 + hh] = m;
        __syncwarp();
        if (lane == 0) mbar_arrive(my_pair);
        if (!(ok = mbar_wait_warp(my_pair, pair_phase, abort_flag))) break;
        pair_phase ^= 1;
        m = fmaxf(xchg_m[(t * kQT + row) * 2], xchg_m[(t * kQT + row) * 2 + 1]);   // finite: column 0 always exists
        nm2 = make_float2(-m * c, -m * c);
        bs = fmaf(-m, cs, 0.5f);
        float2 acc = make_float2(0.f, 0.f);
#pragma unroll
        for (int ch = 0; ch < kHalf / 16; ++ch) {
          uint32_t pk[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int col = ch * 16 + 2 * i;
            const float2 x = __ffma2_rn(f2(s[col], s[col + 1]), c2, nm2);
            float2 p = make_float2(ex2(x.x), ex2(x.y));
            if (col >= valid) p.x = 0.f;
            if (col + 1 >= valid) p.y = 0.f;
            acc = __fadd2_rn(acc, p);
            const __nv_bfloat162 bb = __floats2bfloat162_rn(p.x, p.y);
            pk[i] = *reinterpret_cast<const uint32_t*>(&bb);
          }
          tmem_st8(t_s + ch * 8, pk);
        }
        l_half = acc.x + acc.y;
      } else if (valid == kHalf) {
        l_half += half_tile<false, PRESCALED>(t_s, valid, c2, nm2, cs, bs);
      } else {
        l_half += half_tile<true, PRESCALED>(t_s, valid, c2, nm2, cs, bs);
      }
      tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&p_full[t * 2 + (j & 1)]);
    }
    // The row sum is the sum of the halves'; it also tells whether the fixed maximum was good enough.
    if (ok) {
      xchg_l[(t * kQT + row) * 2 + hh] = l_half;
      __syncwarp();
      if (lane == 0) mbar_arrive(my_pair);
      ok = mbar_wait_warp(my_pair, pair_phase, abort_flag);
    }
    if (ok) {
      const float l_row = xchg_l[(t * kQT + row) * 2] + xchg_l[(t * kQT + row) * 2 + 1];
      const int qi = (qg * kQTiles + t) * kQT + row;
      // (also catches Inf and NaN; without a maximum the sum must not be vanishingly small either)
      const bool bad = qi < n_q && !(l_row < kRowSumLimit && (!PRESCALED || l_row > kRowSumFloor));
      if (__any_sync(0xFFFFFFFFu, bad) && lane == 0) atomicOr(cta_bad, 1);
      ok = mbar_wait_warp(&pv_full[t], 0, abort_flag);
      if (ok) {
        tc_fence_after();
        const float inv = 1.0f / l_row;
        // each half writes 32 of the row's 64 output features
        __nv_bfloat16* dst = O + ((long long)b * n_q + qi) * ((long long)heads * kHD) + h * kHD + hh * 32;
#pragma unroll
        for (int ch = 0; ch < 2; ++ch) {
          uint32_t r[16];
          tmem_ld16(lane_base + kColO + hh * 32 + ch * 16, r);     // warp-collective: every lane loads
          tmem_ld_wait();
          if (qi < n_q) {
            uint32_t w[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
              const __nv_bfloat162 pk = __floats2bfloat162_rn(__uint_as_float(r[2 * q]) * inv,
                                                              __uint_as_float(r[2 * q + 1]) * inv);
              w[q] = *reinterpret_cast<const uint32_t*>(&pk);
            }
            *reinterpret_cast<uint4*>(dst + ch * 16) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(dst + ch * 16 + 8) = make_uint4(w[4], w[5], w[6], w[7]);
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0) {
    if (*abort_flag) atomicAdd(status, 1);
    cta_words[blockIdx.x] = *abort_flag ? 2 : (*cta_bad ? 1 : 0);
  }
  if (warp == 1) { __syncwarp(); tc_fence_after(); tmem_dealloc(tmem_base, kAttTmemCols); }
}

}  // namespace

// Tensor maps of one attention problem: Q as [B * n_q, D] rows, K and V as [B][N][D].
static int make_attention_maps(const void* q, const void* k, const void* v, int B, int n_q, int N, int heads,
                               CUtensorMap* tm_q, CUtensorMap* tm_k, CUtensorMap* tm_v) {
  const uint64_t D = (uint64_t)heads * kHD;
  {
    const uint64_t dims[2] = {D, (uint64_t)B * n_q};
    const uint64_t str[1] = {D * 2};
    const uint32_t box[2] = {(uint32_t)kHD, (uint32_t)kQT};
    HERO_TRY(make_tmap_bf16(tm_q, q, 2, dims, str, box));
  }
  {
    const uint64_t dims[3] = {D, (uint64_t)N, (uint64_t)B};
    const uint64_t str[2] = {D * 2, (uint64_t)N * D * 2};
    const uint32_t box[3] = {(uint32_t)kHD, (uint32_t)kKT, 1};
    HERO_TRY(make_tmap_bf16(tm_k, k, 3, dims, str, box));
    HERO_TRY(make_tmap_bf16(tm_v, v, 3, dims, str, box));
  }
  return HERO_OK;
}

static int attention_kernel_attributes() {
  static PerDeviceOnce attr_once;            // the opt-in is a property of the kernel ON a device
  return per_device_once(attr_once, [](int) {
    HERO_CUDA_TRY(cudaFuncSetAttribute(tc_attention_safe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kAttSmem));
    HERO_CUDA_TRY(cudaFuncSetAttribute(tc_attention_fast_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kFastSmem));
    HERO_CUDA_TRY(cudaFuncSetAttribute(tc_attention_fast_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       (int)kFastSmem));
    return HERO_OK;
  });
}

long long tc_attention_grid(int B, int n_q, int heads) {
  const long long q_groups = ((long long)n_q + kQT * kQTiles - 1) / (kQT * kQTiles);
  return q_groups * heads * B;
}

// d_status[0] counts CTAs that gave up; d_status[1 .. 1 + status_ctas) are the per-CTA words.  When the grid
// fits in them the fast kernel runs, followed by the safe kernel on the CTAs the fast one marked; otherwise the
// safe kernel does everything.  q_prescaled: the caller has multiplied Q by log2(e) / sqrt(head_dim) already, so
// a score IS the exponent of its weight; the fast kernel then takes 2^s as it stands, with no maximum at all
// (exact while a row's largest score stays within about +-100, the row sum telling when it did not).
int launch_tc_attention(const void* q, const void* k, const void* v, void* o, int B, int n_q, int N, int heads,
                        bool q_prescaled, int* d_status, int status_ctas, cudaStream_t s) {
  if (B <= 0 || n_q <= 0) return HERO_OK;
  if (N <= 0 || heads <= 0) return HERO_ERR_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return HERO_ERR_ALIGN;
  CUtensorMap tm_q, tm_k, tm_v;
  HERO_TRY(make_attention_maps(q, k, v, B, n_q, N, heads, &tm_q, &tm_k, &tm_v));
  HERO_TRY(attention_kernel_attributes());
  const long long grid = tc_attention_grid(B, n_q, heads);
  if (grid > 0x7FFFFFFFll) return HERO_ERR_ARG;
  int* cta_words = grid <= status_ctas ? d_status + 1 : nullptr;
  if (cta_words) {
    if (q_prescaled)
      tc_attention_fast_kernel<true><<<(unsigned)grid, kFastThreads, kFastSmem, s>>>(
          tm_q, tm_k, tm_v, (__nv_bfloat16*)o, n_q, N, heads, d_status, cta_words);
    else
      tc_attention_fast_kernel<false><<<(unsigned)grid, kFastThreads, kFastSmem, s>>>(
          tm_q, tm_k, tm_v, (__nv_bfloat16*)o, n_q, N, heads, d_status, cta_words);
  }
  tc_attention_safe_kernel<<<(unsigned)grid, kAttThreads, kAttSmem, s>>>(
      tm_q, tm_k, tm_v, (__nv_bfloat16*)o, n_q, N, heads, q_prescaled ? 1.0f : kScoreScaleLog2, d_status, cta_words);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

// Test hook: the safe kernel alone on every CTA (what runs when there are no per-CTA words).
int launch_tc_attention_safe(const void* q, const void* k, const void* v, void* o, int B, int n_q, int N, int heads,
                             bool q_prescaled, int* d_status, cudaStream_t s) {
  return launch_tc_attention(q, k, v, o, B, n_q, N, heads, q_prescaled, d_status, 0, s);
}

}  // namespace hero

// =============================================================================
// hero_attention_bf16_static: the same attention, for callers that must not allocate
// =============================================================================
// hero_attention_bf16 takes its status words from a cudaMalloc made on first use.  Some
// callers cannot afford that: a host thread inside a latency-critical serving loop (cudaMalloc
// and cudaFree synchronise the whole device), a process whose framework has already reserved all
// device memory for its own pool (the allocation would fail), or code that runs where the CUDA
// allocator must not be entered at all.  For them the scratch lives in the library image itself:
// a file-scope __device__ array that every GPU loading the library carries until the process
// exits (kStaticScratchInts * 4 bytes = 64.25 KiB per GPU).
//
// Layout: word 0 counts the CTAs of the latest call that gave up on a bounded wait, word 1 + i
// is CTA i's word (0 = done, 1 = left to the safe kernel, which then clears it, 2 = gave up).  The
// array is shared by every call and keeps the previous call's contents, so each call clears the
// words it is going to use on its stream before the kernels run; two calls that overlap on the
// GPU (different streams, no dependency) race on it.
namespace hero {
namespace {

constexpr int kStaticMaxCtas = 16384;                 // largest grid the static scratch can serve
constexpr int kStaticScratchInts = 64 + kStaticMaxCtas;
static __device__ __align__(256) int g_att_static_scratch[kStaticScratchInts];

struct StaticSetup { bool done = false; int* scratch = nullptr; };
StaticSetup g_static_setup[kMaxDevices];
std::mutex g_static_mutex;

// Once per device, with that device current: resolve the DEVICE address of the array (in host
// code the array's name is only a host-side handle, never a pointer a kernel may be given) and
// raise the kernels' dynamic shared-memory limit.
int static_setup(int** scratch) {
  int dev = -1;
  HERO_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= kMaxDevices) return HERO_ERR_ARG;
  HERO_TRY(attention_kernel_attributes());
  std::lock_guard<std::mutex> lock(g_static_mutex);
  StaticSetup& st = g_static_setup[dev];
  if (!st.done) {
    int* p = nullptr;
    HERO_CUDA_TRY(cudaGetSymbolAddress((void**)&p, g_att_static_scratch));
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
  const long long grid = tc_attention_grid(B, n_q, heads);
  if (grid > kStaticMaxCtas) {
    set_cuda_error(cudaErrorInvalidConfiguration,
                   "hero_attention_bf16_static: ceil(n_q/256)*heads*B exceeds the 16384 CTAs its static scratch "
                   "serves; split the call or use hero_attention_bf16");
    return HERO_ERR_CAP;
  }
  cudaStream_t s = (cudaStream_t)stream;
  int* scratch = nullptr;
  HERO_TRY(static_setup(&scratch));
  // the array still holds the previous call's records: clear the words this grid will use
  HERO_CUDA_TRY(cudaMemsetAsync(scratch, 0, (size_t)(1 + grid) * sizeof(int), s));
  HERO_TRY(launch_tc_attention(d_q, d_k, d_v, d_o, B, n_q, N, heads, false, scratch, kStaticMaxCtas, s));
  if (h_gave_up) {
    HERO_CUDA_TRY(cudaMemcpyAsync(h_gave_up, scratch, sizeof(int), cudaMemcpyDeviceToHost, s));
    HERO_CUDA_TRY(cudaStreamSynchronize(s));
    if (*h_gave_up != 0) return HERO_ERR_TIMEOUT;
  }
  return HERO_OK;
}

// The verdict of the latest hero_attention_bf16_static call on the current device, for callers that passed
// h_gave_up == NULL to stay asynchronous: copies the counter (and, on request, the per-thread-block records)
// out of the static array behind everything queued on `stream`, and waits for that copy.  Allocates nothing.
extern "C" int hero_attention_bf16_static_status(void* stream, int* h_gave_up, int* h_records, int n_records) {
  using namespace hero;
  if (!h_gave_up || n_records < 0 || n_records > kStaticMaxCtas || (n_records > 0 && !h_records)) return HERO_ERR_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  int* scratch = nullptr;
  HERO_TRY(static_setup(&scratch));
  HERO_CUDA_TRY(cudaMemcpyAsync(h_gave_up, scratch, sizeof(int), cudaMemcpyDeviceToHost, s));
  if (n_records > 0)
    HERO_CUDA_TRY(cudaMemcpyAsync(h_records, scratch + 1, (size_t)n_records * sizeof(int), cudaMemcpyDeviceToHost, s));
  HERO_CUDA_TRY(cudaStreamSynchronize(s));
  return *h_gave_up != 0 ? HERO_ERR_TIMEOUT : HERO_OK;
}
