// Token selection S(z) = union_i Sample(P^i, R) (Eq. 4) with frequency-aware tracking
// (Sec. 4.3): integer-only, data-independent, bit-exact against the CPU oracle.
//
// One CTA per block to select (all shallow blocks of a step go in one launch).  Each thread
// owns one video token per sweep: it rebuilds the keys of its patch mates from the old ages,
// ranks itself, and the CTA compacts the winners in ascending row order with warp ballots
// and a prefix scan over the warp counts.  Ages are double-buffered (read old, write new)
// because a patch spans several grid rows and therefore several sweeps.
#include "hero_internal.h"

namespace hero {
namespace {

constexpr int kSelThreads = 1024;

__device__ __forceinline__ uint32_t mix32(uint32_t x) {
  // xor-shift / odd-multiply avalanche rounds (the published MurmurHash3 finaliser)
  x ^= x >> 16;
  x *= 0x85EBCA6Bu;
  x ^= x >> 13;
  x *= 0xC2B2AE35u;
  x ^= x >> 16;
  return x;
}

// Sampling key of a token: larger wins.  Mode 0: (age+1) * (hash+1), a uniform draw on (0, age+1] up to
// scale, so the chance of being picked grows with the time a token has gone unsampled.  Mode 1: age first,
// hash second - strict oldest-first, the draw only orders tokens of equal age.
__device__ __forceinline__ unsigned long long make_key(int track_mode, uint32_t age, uint32_t hash) {
  return track_mode == 0 ? (unsigned long long)(age + 1u) * ((unsigned long long)hash + 1ull)
                         : ((unsigned long long)age << 32) | (unsigned long long)hash;
}

__global__ void __launch_bounds__(kSelThreads) select_kernel(const SelectGeom g, const SelectBatch batch) {
  const int e = blockIdx.x;
  if (e >= batch.n) return;
  const uint16_t* __restrict__ ages_in = batch.ages_in[e];
  uint16_t* __restrict__ ages_out = batch.ages_out[e];
  int* __restrict__ idx = batch.idx[e];
  const int call = batch.call[e];
  const uint32_t h_block = mix32(mix32(g.seed_lo ^ (uint32_t)batch.block[e]) + (uint32_t)call);

  const int H = g.grid_h, W = g.grid_w;
  const int n_video = g.frames * H * W;
  const int ph = g.patch_h, pw = g.patch_w;
  const long long off = (long long)call * ph * pw;
  const long long ra = g.ratio_num, rb = g.ratio_den;

  __shared__ int warp_count[kSelThreads / 32];
  __shared__ int running;
  if (threadIdx.x == 0) running = 0;
  __syncthreads();

  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int base = 0; base < n_video; base += kSelThreads) {
    const int v = base + threadIdx.x;
    bool pick = false;
    uint32_t age_v = 0;
    if (v < n_video) {
      const int t = v / (H * W);
      const int rem = v - t * H * W;
      const int y = rem / W, x = rem - y * W;
      const int py = y / ph, px = x / pw;
      const int y0 = py * ph, x0 = px * pw;
      const int hh = min(ph, H - y0), ww = min(pw, W - x0);
      const int n_here = hh * ww;
      // tokens in patches that precede this one (patch-id order: frame, patch row, patch column)
      const long long before = (long long)t * H * W + (long long)y0 * W + (long long)hh * x0;
      int quota;
      if (g.quota_mode == 0) {
        quota = (int)(((before + n_here + off) * ra) / rb - ((before + off) * ra) / rb);
      } else {
        quota = min(n_here, (int)((2ll * n_here * ra + rb) / (2 * rb)));
      }
      age_v = ages_in[v];
      const unsigned long long key_v = make_key(g.track_mode, age_v, mix32(h_block + (uint32_t)v));
      int beaten_by = 0;
      for (int dy = 0; dy < hh; ++dy) {
        for (int dx = 0; dx < ww; ++dx) {
          const int u = (t * H + y0 + dy) * W + x0 + dx;
          if (u == v) continue;
          const unsigned long long key_u = make_key(g.track_mode, (uint32_t)ages_in[u], mix32(h_block + (uint32_t)u));
          beaten_by += (key_u > key_v || (key_u == key_v && u < v)) ? 1 : 0;
        }
      }
      pick = beaten_by < quota;
    }
    const unsigned ballot = __ballot_sync(0xFFFFFFFFu, pick);
    if (lane == 0) warp_count[warp] = __popc(ballot);
    __syncthreads();
    // exclusive prefix over the 32 warp counts (each warp recomputes it with one shuffle scan)
    int c = warp_count[lane];
    int incl = c;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const int o = __shfl_up_sync(0xFFFFFFFFu, incl, s);
      if (lane >= s) incl += o;
    }
    const int warp_base = __shfl_sync(0xFFFFFFFFu, incl - c, warp);
    const int total = __shfl_sync(0xFFFFFFFFu, incl, 31);
    const int start = running;
    if (v < n_video) {
      if (pick) idx[start + warp_base + __popc(ballot & ((1u << lane) - 1u))] = g.n_text + v;
      ages_out[v] = pick ? (uint16_t)0 : (uint16_t)min(age_v + 1u, 65535u);
    }
    __syncthreads();
    if (threadIdx.x == 0) running = start + total;
    __syncthreads();
  }
}

}  // namespace

int launch_select(const SelectGeom& g, const SelectBatch& batch, cudaStream_t s) {
  if (batch.n <= 0) return HERO_OK;
  select_kernel<<<batch.n, kSelThreads, 0, s>>>(g, batch);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

}  // namespace hero
