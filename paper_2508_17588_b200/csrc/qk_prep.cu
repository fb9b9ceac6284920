// Treatment of the fresh q and k rows between the QKV projection and attention, as in the base
// video DiT the method is applied to (Sec. 3 leaves the block's internals to the base model):
// an optional LayerNorm over every head's features with a learned gain and bias, then an optional
// 3-D rotary position embedding of the video rows.  q is the compact [B, n_sel, D] projection
// output; k is rewritten in place in the block's K cache at the rows of the index list, so the
// cache always holds keys in their final form (a row never changes position, so cached keys stay
// valid across steps).  HBM-bound: every element is read once and written once.  Generic kernel (fp32,
// any even head_dim <= 256): one warp owns one (row, head) slice, a lane the rotary pairs (2p, 2p+1)
// for p = lane, lane + 32, ...; the bf16 head_dim-64 kernel further down moves 16 bytes per access.
#include "hero_internal.h"

namespace hero {
namespace {

constexpr int kMaxPairsPerLane = 4;  // head_dim <= 256

template <typename T>
__device__ __forceinline__ float2 load_pair(const T* p);
template <>
__device__ __forceinline__ float2 load_pair<float>(const float* p) {
  return *reinterpret_cast<const float2*>(p);
}
template <>
__device__ __forceinline__ float2 load_pair<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(p));
}
template <typename T>
__device__ __forceinline__ void store_pair(T* p, float2 v);
template <>
__device__ __forceinline__ void store_pair<float>(float* p, float2 v) {
  *reinterpret_cast<float2*>(p) = v;
}
template <>
__device__ __forceinline__ void store_pair<__nv_bfloat16>(__nv_bfloat16* p, float2 v) {
  *reinterpret_cast<__nv_bfloat162*>(p) = __float22bfloat162_rn(v);
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <typename T>
__global__ void __launch_bounds__(256) qk_prep_kernel(QkPrepArgs a) {
  const int lane = threadIdx.x & 31;
  const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const long long n_items = (long long)a.B * a.n_sel * a.n_heads * 2;
  const int pairs = a.head_dim >> 1;
  const float inv_hd = 1.0f / (float)a.head_dim;
  for (long long item = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5; item < n_items; item += n_warps) {
    const int which = (int)(item & 1);                // 0: q, 1: k
    long long rest = item >> 1;
    const int head = (int)(rest % a.n_heads); rest /= a.n_heads;
    const int i = (int)(rest % a.n_sel);
    const int b = (int)(rest / a.n_sel);
    const int row = a.idx ? a.idx[i] : i;
    T* p = which ? static_cast<T*>(a.k) + ((long long)b * a.N + row) * a.D + head * a.head_dim
                 : static_cast<T*>(a.q) + ((long long)b * a.n_sel + i) * a.D + head * a.head_dim;
    float2 v[kMaxPairsPerLane];
#pragma unroll
    for (int j = 0; j < kMaxPairsPerLane; ++j) {
      const int pr = lane + 32 * j;
      v[j] = pr < pairs ? load_pair<T>(p + 2 * pr) : make_float2(0.f, 0.f);
    }
    if (a.qn_w) {
      const T* gw = static_cast<const T*>(which ? a.kn_w : a.qn_w);
      const T* gb = static_cast<const T*>(which ? a.kn_b : a.qn_b);
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < kMaxPairsPerLane; ++j) s += v[j].x + v[j].y;   // absent pairs hold zeros
      const float mu = warp_sum(s) * inv_hd;
      float q2 = 0.f;
#pragma unroll
      for (int j = 0; j < kMaxPairsPerLane; ++j)
        if (lane + 32 * j < pairs) q2 += (v[j].x - mu) * (v[j].x - mu) + (v[j].y - mu) * (v[j].y - mu);
      const float rstd = rsqrtf(warp_sum(q2) * inv_hd + a.eps);
#pragma unroll
      for (int j = 0; j < kMaxPairsPerLane; ++j) {
        const int pr = lane + 32 * j;
        if (pr < pairs) {
          const float2 w = load_pair<T>(gw + 2 * pr), bb = load_pair<T>(gb + 2 * pr);
          v[j].x = (v[j].x - mu) * rstd * w.x + bb.x;
          v[j].y = (v[j].y - mu) * rstd * w.y + bb.y;
        }
      }
    }
    if (a.rope && row >= a.n_text) {
      const int t = row - a.n_text;
      const int pos_t = t / (a.grid_h * a.grid_w), pos_h = (t / a.grid_w) % a.grid_h, pos_w = t % a.grid_w;
#pragma unroll
      for (int j = 0; j < kMaxPairsPerLane; ++j) {
        const int pr = lane + 32 * j;
        if (pr < pairs) {
          int at;                                     // entry of the (cos, sin) table
          if (pr < a.p_t) at = pos_t * a.p_t + pr;
          else if (pr < a.p_t + a.p_h) at = a.frames * a.p_t + pos_h * a.p_h + (pr - a.p_t);
          else at = a.frames * a.p_t + a.grid_h * a.p_h + pos_w * a.p_w + (pr - a.p_t - a.p_h);
          const float2 cs = a.rope[at];
          const float x = v[j].x, y = v[j].y;
          v[j].x = x * cs.x - y * cs.y;
          v[j].y = x * cs.y + y * cs.x;
        }
      }
    }
    const float out_scale = (!which && a.q_scale != 0.f) ? a.q_scale : 1.0f;
#pragma unroll
    for (int j = 0; j < kMaxPairsPerLane; ++j) {
      const int pr = lane + 32 * j;
      if (pr < pairs) store_pair<T>(p + 2 * pr, make_float2(v[j].x * out_scale, v[j].y * out_scale));
    }
  }
}

// bf16, head_dim 64: a thread owns 8 consecutive features (rotary pairs 4s..4s+3 of one head, s = its
// position in the 8-lane group that covers the head) and two such chunks half the problem apart, so
// that 32 bytes per thread are in flight; the LayerNorm sums run over the 8-lane group.
__global__ void __launch_bounds__(256) qk_prep_hd64_kernel(QkPrepArgs a, int n_chunks_half) {
  const int c0 = blockIdx.x * blockDim.x + threadIdx.x;
  const int per_row = a.D >> 3;
  const int n_chunks = (int)((long long)a.B * a.n_sel * 2 * per_row);
  __nv_bfloat16* ptr[2];
  int row[2], which[2], sub[2];
  uint4 raw[2];
  bool live[2];
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    const int c = c0 + u * n_chunks_half;
    live[u] = c0 < n_chunks_half && c < n_chunks;
    const int cc = live[u] ? c : 0;
    const int item = cc / per_row, within = cc - item * per_row;
    which[u] = item & 1;
    const int bi = item >> 1, b = bi / a.n_sel, i = bi - b * a.n_sel;
    row[u] = a.idx ? a.idx[i] : i;
    sub[u] = within & 7;
    ptr[u] = (which[u] ? static_cast<__nv_bfloat16*>(a.k) + ((long long)b * a.N + row[u]) * a.D
                       : static_cast<__nv_bfloat16*>(a.q) + ((long long)b * a.n_sel + i) * a.D) + within * 8;
    raw[u] = live[u] ? *reinterpret_cast<const uint4*>(ptr[u]) : make_uint4(0, 0, 0, 0);
  }
#pragma unroll
  for (int u = 0; u < 2; ++u) {
    float2 v[4];
    const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&raw[u]);
#pragma unroll
    for (int j = 0; j < 4; ++j) v[j] = __bfloat1622float2(h2[j]);
    if (a.qn_w) {                                   // uniform over the grid: the shuffles below are convergent
      float s = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) s += v[j].x + v[j].y;
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
      const float mu = s * (1.0f / 64.0f);
      float q2 = 0.f;
#pragma unroll
      for (int j = 0; j < 4; ++j) q2 += (v[j].x - mu) * (v[j].x - mu) + (v[j].y - mu) * (v[j].y - mu);
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) q2 += __shfl_xor_sync(0xffffffffu, q2, o);
      const float rstd = rsqrtf(q2 * (1.0f / 64.0f) + a.eps);
      const uint4 gw = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(which[u] ? a.kn_w : a.qn_w) + sub[u] * 8);
      const uint4 gb = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(which[u] ? a.kn_b : a.qn_b) + sub[u] * 8);
      const __nv_bfloat162* w2 = reinterpret_cast<const __nv_bfloat162*>(&gw);
      const __nv_bfloat162* b2 = reinterpret_cast<const __nv_bfloat162*>(&gb);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float2 w = __bfloat1622float2(w2[j]), bb = __bfloat1622float2(b2[j]);
        v[j].x = (v[j].x - mu) * rstd * w.x + bb.x;
        v[j].y = (v[j].y - mu) * rstd * w.y + bb.y;
      }
    }
    if (a.rope && row[u] >= a.n_text) {
      const int t = row[u] - a.n_text;
      const int pos_t = t / (a.grid_h * a.grid_w), pos_h = (t / a.grid_w) % a.grid_h, pos_w = t % a.grid_w;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int pr = sub[u] * 4 + j;
        int at;
        if (pr < a.p_t) at = pos_t * a.p_t + pr;
        else if (pr < a.p_t + a.p_h) at = a.frames * a.p_t + pos_h * a.p_h + (pr - a.p_t);
        else at = a.frames * a.p_t + a.grid_h * a.p_h + pos_w * a.p_w + (pr - a.p_t - a.p_h);
        const float2 cs = __ldg(a.rope + at);
        const float x = v[j].x, y = v[j].y;
        v[j].x = x * cs.x - y * cs.y;
        v[j].y = x * cs.y + y * cs.x;
      }
    }
    const float out_scale = (!which[u] && a.q_scale != 0.f) ? a.q_scale : 1.0f;
    uint4 out;
    __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(&out);
#pragma unroll
    for (int j = 0; j < 4; ++j) o2[j] = __float22bfloat162_rn(make_float2(v[j].x * out_scale, v[j].y * out_scale));
    if (live[u]) *reinterpret_cast<uint4*>(ptr[u]) = out;
  }
}

}  // namespace

int launch_qk_prep(const QkPrepArgs& a, int dtype, cudaStream_t s) {
  if (a.head_dim % 2 != 0 || a.head_dim > 64 * kMaxPairsPerLane) return HERO_ERR_ARG;
  const long long n_items = (long long)a.B * a.n_sel * a.n_heads * 2;
  if (n_items <= 0) return HERO_OK;
  const long long n_chunks = (long long)a.B * a.n_sel * 2 * (a.D / 8);
  if (dtype == HERO_DTYPE_BF16 && a.head_dim == 64 && a.D == a.n_heads * 64 && n_chunks < (1ll << 30)) {
    const int half = (int)((n_chunks + 1) / 2);
    qk_prep_hd64_kernel<<<(half + 255) / 256, 256, 0, s>>>(a, half);
    HERO_CUDA_TRY(cudaGetLastError());
    return HERO_OK;
  }
  int dev = 0, sms = 0;
  HERO_CUDA_TRY(cudaGetDevice(&dev));
  HERO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const long long want = (n_items + 7) / 8;                       // 8 warps per block
  const int grid = (int)(want < (long long)sms * 8 ? want : (long long)sms * 8);
  if (dtype == HERO_DTYPE_BF16) qk_prep_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>(a);
  else qk_prep_kernel<float><<<grid, 256, 0, s>>>(a);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

}  // namespace hero
