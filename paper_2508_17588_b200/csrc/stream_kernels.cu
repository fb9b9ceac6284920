// HBM-bound kernels of the cached step: linear extrapolation (Eq. 5), residual adds
// (Algorithm 1), row gather / scatter (Eq. 3's merge), the adaLN modulation vectors and the
// fused gather + LayerNorm + modulate prologue of Eq. 2.  All of them move each byte once
// with 128-bit accesses; grids are sized in multiples of the SM count.
#include "hero_internal.h"

namespace hero {

// SM count of the calling thread's current device (looked up once per device).
int num_sms() {
  static PerDeviceOnce once;
  static int count[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  per_device_once(once, [](int d) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, d) != cudaSuccess || n <= 0) n = 148;
    count[d] = n;
    return HERO_OK;
  });
  return count[dev] > 0 ? count[dev] : 148;
}

namespace {

// ------------------------------------------------------------------ 128-bit packets
template <typename T>
struct Vec;  // 16 bytes of T
template <>
struct Vec<float> {
  static constexpr int N = 4;
  float4 raw;
  __device__ __forceinline__ void unpack(float (&f)[4]) const {
    f[0] = raw.x; f[1] = raw.y; f[2] = raw.z; f[3] = raw.w;
  }
  __device__ __forceinline__ void pack(const float (&f)[4]) { raw = make_float4(f[0], f[1], f[2], f[3]); }
};
template <>
struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  uint4 raw;
  __device__ __forceinline__ void unpack(float (&f)[8]) const {
    const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ __forceinline__ void pack(const float (&f)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 p = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&p);
    }
    raw = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

template <typename T>
__device__ __forceinline__ float to_f(T v);
template <>
__device__ __forceinline__ float to_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ float to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T>
__device__ __forceinline__ T from_f(float v);
template <>
__device__ __forceinline__ float from_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// streaming loads/stores: these tensors are touched once per step, keep them out of L1
template <typename V>
__device__ __forceinline__ V ld_stream(const V* p) {
  V v;
  v.raw = __ldcs(&p->raw);
  return v;
}
template <typename V>
__device__ __forceinline__ void st_stream(V* p, const V& v) { __stcs(&p->raw, v.raw); }

constexpr int kStreamThreads = 256;
constexpr int kStreamUnroll = 2;

static inline int stream_grid(long long n_vec) {
  const long long per_block = (long long)kStreamThreads * kStreamUnroll;
  long long blocks = (n_vec + per_block - 1) / per_block;
  const long long cap = (long long)num_sms() * 16;   // grid-stride beyond 16 CTAs per SM
  if (blocks > cap) blocks = cap;
  if (blocks < 1) blocks = 1;
  return (int)blocks;
}

// ------------------------------------------------------------------ Eq. 5
// e = g_last + (g_last - g_prev) * (k/d), evaluated as one fp32 FMA per element.
template <typename T>
__global__ void __launch_bounds__(kStreamThreads) extrapolate_kernel(const T* __restrict__ g_prev,
                                                                     const T* __restrict__ g_last,
                                                                     T* __restrict__ out, long long n, float c) {
  using V = Vec<T>;
  const long long n_vec = n / V::N;
  const V* p = reinterpret_cast<const V*>(g_prev);
  const V* l = reinterpret_cast<const V*>(g_last);
  V* o = reinterpret_cast<V*>(out);
  const long long stride = (long long)gridDim.x * kStreamThreads * kStreamUnroll;
  for (long long i0 = (long long)blockIdx.x * kStreamThreads * kStreamUnroll + threadIdx.x; i0 < n_vec; i0 += stride) {
    V vp[kStreamUnroll], vl[kStreamUnroll];
#pragma unroll
    for (int u = 0; u < kStreamUnroll; ++u) {
      const long long i = i0 + (long long)u * kStreamThreads;
      if (i < n_vec) { vp[u] = ld_stream(p + i); vl[u] = ld_stream(l + i); }
    }
#pragma unroll
    for (int u = 0; u < kStreamUnroll; ++u) {
      const long long i = i0 + (long long)u * kStreamThreads;
      if (i < n_vec) {
        float fp[V::N], fl[V::N];
        vp[u].unpack(fp); vl[u].unpack(fl);
#pragma unroll
        for (int j = 0; j < V::N; ++j) fl[j] = fmaf(fl[j] - fp[j], c, fl[j]);
        V r; r.pack(fl);
        st_stream(o + i, r);
      }
    }
  }
  // ragged tail (fewer than one packet)
  const long long tail0 = n_vec * V::N;
  if (blockIdx.x == 0 && threadIdx.x < n - tail0) {
    const long long i = tail0 + threadIdx.x;
    const float a = to_f(g_last[i]), b = to_f(g_prev[i]);
    out[i] = from_f<T>(fmaf(a - b, c, a));
  }
}

// x += e(attn) ; x += e(ffn)  (both branches of a deep block in one pass: 5 reads, 1 write)
template <typename T>
__global__ void __launch_bounds__(kStreamThreads)
extrapolate_residual_kernel(T* __restrict__ x, const T* __restrict__ ga_prev, const T* __restrict__ ga_last,
                            const T* __restrict__ gf_prev, const T* __restrict__ gf_last, long long n, float c) {
  using V = Vec<T>;
  const long long n_vec = n / V::N;
  V* xv = reinterpret_cast<V*>(x);
  const V* ap = reinterpret_cast<const V*>(ga_prev);
  const V* al = reinterpret_cast<const V*>(ga_last);
  const V* fp_ = reinterpret_cast<const V*>(gf_prev);
  const V* fl_ = reinterpret_cast<const V*>(gf_last);
  const long long stride = (long long)gridDim.x * kStreamThreads;
  for (long long i = (long long)blockIdx.x * kStreamThreads + threadIdx.x; i < n_vec; i += stride) {
    const V vx = ld_stream(xv + i), v1 = ld_stream(ap + i), v2 = ld_stream(al + i), v3 = ld_stream(fp_ + i),
            v4 = ld_stream(fl_ + i);
    float fx[V::N], f1[V::N], f2[V::N], f3[V::N], f4[V::N];
    vx.unpack(fx); v1.unpack(f1); v2.unpack(f2); v3.unpack(f3); v4.unpack(f4);
#pragma unroll
    for (int j = 0; j < V::N; ++j) {
      const float ea = fmaf(f2[j] - f1[j], c, f2[j]);
      const float ef = fmaf(f4[j] - f3[j], c, f4[j]);
      fx[j] = (fx[j] + ea) + ef;
    }
    V r; r.pack(fx);
    st_stream(xv + i, r);
  }
  const long long tail0 = n_vec * V::N;
  if (blockIdx.x == 0 && threadIdx.x < n - tail0) {
    const long long i = tail0 + threadIdx.x;
    const float a1 = to_f(ga_prev[i]), a2 = to_f(ga_last[i]), b1 = to_f(gf_prev[i]), b2 = to_f(gf_last[i]);
    x[i] = from_f<T>((to_f(x[i]) + fmaf(a2 - a1, c, a2)) + fmaf(b2 - b1, c, b2));
  }
}

// Eq. 5 for a run of consecutive extrapolated blocks in ONE pass over x: a deep block touches nothing but
// the residual stream, so x can stay in registers while the blocks' four history tensors stream by.  Per
// element and block that is 8 bytes read instead of 12 moved (x is read and written once per launch, not
// once per block), and the sum is rounded to the storage type once.  The adds keep the order of the blocks.
template <typename T>
__global__ void __launch_bounds__(kStreamThreads) extrapolate_group_kernel(T* __restrict__ x, const DeepGroup grp,
                                                                           long long first, long long n, float c) {
  using V = Vec<T>;
  const long long n_vec = n / V::N;
  V* xv = reinterpret_cast<V*>(x + first);
  const long long stride = (long long)gridDim.x * kStreamThreads;
  for (long long i = (long long)blockIdx.x * kStreamThreads + threadIdx.x; i < n_vec; i += stride) {
    float fx[V::N];
    ld_stream(xv + i).unpack(fx);
#pragma unroll 4
    for (int e = 0; e < grp.n_entries; ++e) {
      const V vp = ld_stream(reinterpret_cast<const V*>(static_cast<const T*>(grp.prev[e]) + first) + i);
      const V vl = ld_stream(reinterpret_cast<const V*>(static_cast<const T*>(grp.last[e]) + first) + i);
      float fp_[V::N], fl_[V::N];
      vp.unpack(fp_); vl.unpack(fl_);
#pragma unroll
      for (int j = 0; j < V::N; ++j) fx[j] += fmaf(fl_[j] - fp_[j], c, fl_[j]);
    }
    V r; r.pack(fx);
    st_stream(xv + i, r);
  }
  const long long tail0 = n_vec * V::N;
  if (blockIdx.x == 0 && threadIdx.x < n - tail0) {
    const long long i = first + tail0 + threadIdx.x;
    float v = to_f(x[i]);
    for (int e = 0; e < grp.n_entries; ++e) {
      const float a = to_f(static_cast<const T*>(grp.prev[e])[i]), b = to_f(static_cast<const T*>(grp.last[e])[i]);
      v += fmaf(b - a, c, b);
    }
    x[i] = from_f<T>(v);
  }
}

// x = (x + ga) + gf  (both residual adds of a refresh block in one pass)
template <typename T>
__global__ void __launch_bounds__(kStreamThreads) residual2_kernel(T* __restrict__ x, const T* __restrict__ ga,
                                                                   const T* __restrict__ gf, long long n) {
  using V = Vec<T>;
  const long long n_vec = n / V::N;
  V* xv = reinterpret_cast<V*>(x);
  const V* a = reinterpret_cast<const V*>(ga);
  const V* f = reinterpret_cast<const V*>(gf);
  const long long stride = (long long)gridDim.x * kStreamThreads * kStreamUnroll;
  for (long long i0 = (long long)blockIdx.x * kStreamThreads * kStreamUnroll + threadIdx.x; i0 < n_vec; i0 += stride) {
    V vx[kStreamUnroll], va[kStreamUnroll], vf[kStreamUnroll];
#pragma unroll
    for (int u = 0; u < kStreamUnroll; ++u) {
      const long long i = i0 + (long long)u * kStreamThreads;
      if (i < n_vec) { vx[u] = ld_stream(xv + i); va[u] = ld_stream(a + i); vf[u] = ld_stream(f + i); }
    }
#pragma unroll
    for (int u = 0; u < kStreamUnroll; ++u) {
      const long long i = i0 + (long long)u * kStreamThreads;
      if (i < n_vec) {
        float fx[V::N], fa[V::N], ff[V::N];
        vx[u].unpack(fx); va[u].unpack(fa); vf[u].unpack(ff);
#pragma unroll
        for (int j = 0; j < V::N; ++j) fx[j] = (fx[j] + fa[j]) + ff[j];
        V r; r.pack(fx);
        st_stream(xv + i, r);
      }
    }
  }
  const long long tail0 = n_vec * V::N;
  if (blockIdx.x == 0 && threadIdx.x < n - tail0) {
    const long long i = tail0 + threadIdx.x;
    x[i] = from_f<T>((to_f(x[i]) + to_f(ga[i])) + to_f(gf[i]));
  }
}

// ------------------------------------------------------------------ deep-stack collapse
// fp32 side-band packets matching one 16-byte packet of T
template <typename T>
struct AccVec;
template <>
struct AccVec<float> {
  __device__ static void load(const float* p, long long i, float (&f)[4]) {
    const float4 v = __ldcs(reinterpret_cast<const float4*>(p) + i);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  __device__ static void store(float* p, long long i, const float (&f)[4]) {
    __stcs(reinterpret_cast<float4*>(p) + i, make_float4(f[0], f[1], f[2], f[3]));
  }
};
template <>
struct AccVec<__nv_bfloat16> {
  __device__ static void load(const float* p, long long i, float (&f)[8]) {
    const float4 a = __ldcs(reinterpret_cast<const float4*>(p) + 2 * i), b = __ldcs(reinterpret_cast<const float4*>(p) + 2 * i + 1);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
  }
  __device__ static void store(float* p, long long i, const float (&f)[8]) {
    __stcs(reinterpret_cast<float4*>(p) + 2 * i, make_float4(f[0], f[1], f[2], f[3]));
    __stcs(reinterpret_cast<float4*>(p) + 2 * i + 1, make_float4(f[4], f[5], f[6], f[7]));
  }
};

// Full step, deep block, collapse mode: x = (x + ga) + gf and acc += ga + gf (fp32 running sum of the
// deep stack's branch outputs, the quantity Eq. 5 is applied to on cached steps).
template <typename T>
__global__ void __launch_bounds__(kStreamThreads) residual2_acc_kernel(T* __restrict__ x, const T* __restrict__ ga,
                                                                       const T* __restrict__ gf,
                                                                       float* __restrict__ acc, long long n) {
  using V = Vec<T>;
  const long long n_vec = n / V::N;
  V* xv = reinterpret_cast<V*>(x);
  const V* a = reinterpret_cast<const V*>(ga);
  const V* f = reinterpret_cast<const V*>(gf);
  const long long stride = (long long)gridDim.x * kStreamThreads;
  for (long long i = (long long)blockIdx.x * kStreamThreads + threadIdx.x; i < n_vec; i += stride) {
    const V vx = ld_stream(xv + i), va = ld_stream(a + i), vf = ld_stream(f + i);
    float fx[V::N], fa[V::N], ff[V::N], fs[V::N];
    vx.unpack(fx); va.unpack(fa); vf.unpack(ff);
    AccVec<T>::load(acc, i, fs);
#pragma unroll
    for (int j = 0; j < V::N; ++j) { fx[j] = (fx[j] + fa[j]) + ff[j]; fs[j] += fa[j] + ff[j]; }
    V r; r.pack(fx);
    st_stream(xv + i, r);
    AccVec<T>::store(acc, i, fs);
  }
  const long long tail0 = n_vec * V::N;
  if (blockIdx.x == 0 && threadIdx.x < n - tail0) {
    const long long i = tail0 + threadIdx.x;
    const float va = to_f(ga[i]), vf = to_f(gf[i]);
    x[i] = from_f<T>((to_f(x[i]) + va) + vf);
    acc[i] += va + vf;
  }
}

// Cached step, whole deep stack in one pass: x += s_last + (s_last - s_prev) * c  (Eq. 5 on the sums).
template <typename T>
__global__ void __launch_bounds__(kStreamThreads) extrapolate_stack_kernel(T* __restrict__ x,
                                                                           const float* __restrict__ s_prev,
                                                                           const float* __restrict__ s_last,
                                                                           long long n, float c) {
  using V = Vec<T>;
  const long long n_vec = n / V::N;
  V* xv = reinterpret_cast<V*>(x);
  const long long stride = (long long)gridDim.x * kStreamThreads;
  for (long long i = (long long)blockIdx.x * kStreamThreads + threadIdx.x; i < n_vec; i += stride) {
    const V vx = ld_stream(xv + i);
    float fx[V::N], fp[V::N], fl[V::N];
    vx.unpack(fx);
    AccVec<T>::load(s_prev, i, fp);
    AccVec<T>::load(s_last, i, fl);
#pragma unroll
    for (int j = 0; j < V::N; ++j) fx[j] += fmaf(fl[j] - fp[j], c, fl[j]);
    V r; r.pack(fx);
    st_stream(xv + i, r);
  }
  const long long tail0 = n_vec * V::N;
  if (blockIdx.x == 0 && threadIdx.x < n - tail0) {
    const long long i = tail0 + threadIdx.x;
    x[i] = from_f<T>(to_f(x[i]) + fmaf(s_last[i] - s_prev[i], c, s_last[i]));
  }
}

// ------------------------------------------------------------------ gather / scatter of rows
// One warp moves one row in 16-byte packets, four packets per lane in flight at a time (2 KB per
// warp, 16 KB per CTA); GATHER reads row idx[i] and writes row i, SCATTER the reverse.  Rows not
// listed are never touched.
constexpr int kMoveUnroll = 4;
template <bool GATHER>
__global__ void __launch_bounds__(256) move_rows_kernel(const uint4* __restrict__ src, const int* __restrict__ idx,
                                                        uint4* __restrict__ dst, int B, int N, int n_sel,
                                                        int row_vec) {
  const long long warp_global = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long n_warps = ((long long)gridDim.x * blockDim.x) >> 5;
  const int lane = threadIdx.x & 31;
  const long long total = (long long)B * n_sel;
  for (long long m = warp_global; m < total; m += n_warps) {
    const int b = (int)(m / n_sel), i = (int)(m - (long long)b * n_sel);
    const long long far = ((long long)b * N + __ldg(idx + i)) * row_vec, near = m * row_vec;
    const uint4* s = src + (GATHER ? far : near);
    uint4* d = dst + (GATHER ? near : far);
    for (int c0 = lane; c0 < row_vec; c0 += 32 * kMoveUnroll) {
      uint4 v[kMoveUnroll];
#pragma unroll
      for (int u = 0; u < kMoveUnroll; ++u)
        if (c0 + 32 * u < row_vec) v[u] = __ldcs(s + c0 + 32 * u);
#pragma unroll
      for (int u = 0; u < kMoveUnroll; ++u)
        if (c0 + 32 * u < row_vec) __stcs(d + c0 + 32 * u, v[u]);
    }
  }
}

// ------------------------------------------------------------------ adaLN modulation vectors
// mod[b, j] = b_mod[j] + sum_e silu(temb[b, e]) * w_mod[j, e].  A warp owns kModRows consecutive output columns
// j at a time: their weight rows are read once with 16-byte loads, all kModRows loads of a step in flight
// together (a row of 512 weights is two loads per lane: one row at a time leaves the warp waiting on DRAM
// latency for most of its life), and reused for every batch item.
constexpr int kModMaxB = 8, kModRows = 4;

// silu(temb) into shared memory, laid out [B][V::N][E / V::N]: element e of a row sits at
// (e % V::N) * (E / V::N) + e / V::N, so that the lanes of a warp, which hold consecutive 16-byte packets of a
// weight row, read consecutive words
template <typename T>
__device__ __forceinline__ void modulation_stage_activations(const T* __restrict__ temb, float* s_act, int B, int E) {
  for (int i = threadIdx.x; i < B * E; i += blockDim.x) {
    const float t = to_f(temb[i]);
    const int b = i / E, e = i - b * E;
    s_act[b * E + (e % Vec<T>::N) * (E / Vec<T>::N) + e / Vec<T>::N] = t / (1.0f + expf(-t));
  }
  __syncthreads();
}

template <typename T, int MAXB>
__device__ __forceinline__ void modulation_rows(const float* s_act, const T* __restrict__ w_mod,
                                                const T* __restrict__ b_mod, float* __restrict__ mod, int B,
                                                int n_out, int E) {
  using V = Vec<T>;
  const int lane = threadIdx.x & 31;
  const int warps = gridDim.x * (blockDim.x >> 5), warp = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int packets = E / V::N;
  for (int j0 = warp * kModRows; j0 < n_out; j0 += warps * kModRows) {
    float acc[kModRows][MAXB];
#pragma unroll
    for (int r = 0; r < kModRows; ++r)
#pragma unroll
      for (int b = 0; b < MAXB; ++b) acc[r][b] = 0.f;
#pragma unroll(MAXB <= 2 ? 2 : 1)
    for (int c = lane; c < packets; c += 32) {
      V wv[kModRows];
#pragma unroll
      for (int r = 0; r < kModRows; ++r) {
        const int j = j0 + r < n_out ? j0 + r : n_out - 1;           // a row past the end repeats the last one
        wv[r].raw = __ldg(&reinterpret_cast<const V*>(w_mod + (long long)j * E)[c].raw);
      }
      float wf[kModRows][V::N];
#pragma unroll
      for (int r = 0; r < kModRows; ++r) wv[r].unpack(wf[r]);
#pragma unroll
      for (int b = 0; b < MAXB; ++b) {
        if (b < B) {
#pragma unroll
          for (int q = 0; q < V::N; ++q) {
            const float a = s_act[b * E + q * packets + c];
#pragma unroll
            for (int r = 0; r < kModRows; ++r) acc[r][b] = fmaf(a, wf[r][q], acc[r][b]);
          }
        }
      }
    }
#pragma unroll
    for (int r = 0; r < kModRows; ++r) {
#pragma unroll
      for (int b = 0; b < MAXB; ++b) {
        if (b < B) {
          float v = acc[r][b];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
          if (lane == 0 && j0 + r < n_out) mod[(long long)b * n_out + j0 + r] = v + to_f(b_mod[j0 + r]);
        }
      }
    }
  }
}

template <typename T, int MAXB>
__global__ void __launch_bounds__(256, 2) modulation_kernel(const T* __restrict__ temb, const T* __restrict__ w_mod,
                                                         const T* __restrict__ b_mod, float* __restrict__ mod,
                                                         int B, int n_out, int E) {
  extern __shared__ float s_act[];
  modulation_stage_activations<T>(temb, s_act, B, E);
  modulation_rows<T, MAXB>(s_act, w_mod, b_mod, mod, B, n_out, E);
}

// The same for several blocks at once: blockIdx.y picks the block's weights and output.
template <typename T, int MAXB>
__global__ void __launch_bounds__(256, 2) modulation_batch_kernel(const T* __restrict__ temb, const ModBatch batch, int B,
                                                               int n_out, int E) {
  extern __shared__ float s_act[];
  modulation_stage_activations<T>(temb, s_act, B, E);
  modulation_rows<T, MAXB>(s_act, static_cast<const T*>(batch.w_mod[blockIdx.y]), static_cast<const T*>(batch.b_mod[blockIdx.y]),
                     batch.mod[blockIdx.y], B, n_out, E);
}

// ------------------------------------------------------------------ gather + LayerNorm + modulate (Eq. 2 prologue)
// One CTA per refreshed row: the row (plus, for the FFN branch, the not-yet-added attention
// output of the same row) is read once into shared memory as fp32, mean and biased variance
// are reduced in two passes over that copy, and the modulated row is written compactly.
constexpr int kLnThreads = 256;
__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = (lane < kLnThreads / 32) ? red[lane] : 0.f;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xFFFFFFFFu, t, o);
  return t;
}

template <typename T>
__global__ void __launch_bounds__(kLnThreads)
gather_ln_modulate_kernel(const T* __restrict__ x, const T* __restrict__ add, const int* __restrict__ idx,
                          const float* __restrict__ shift, const float* __restrict__ scale, int mod_ld,
                          T* __restrict__ a, int N, int n_sel, int D, float eps) {
  extern __shared__ float s_row[];   // [D]
  __shared__ float red[kLnThreads / 32];
  using V = Vec<T>;
  const int m = blockIdx.x;
  const int b = m / n_sel, i = m - b * n_sel;
  const long long row = (long long)b * N + (idx ? idx[i] : i);
  const V* xr = reinterpret_cast<const V*>(x + row * D);
  const V* ar = add ? reinterpret_cast<const V*>(add + row * D) : nullptr;
  const int n_vec = D / V::N;
  float sum = 0.f;
  for (int c = threadIdx.x; c < n_vec; c += kLnThreads) {
    float f[V::N];
    V v; v.raw = __ldg(&xr[c].raw);
    v.unpack(f);
    if (ar) {
      float g[V::N];
      V w; w.raw = __ldg(&ar[c].raw);
      w.unpack(g);
#pragma unroll
      for (int q = 0; q < V::N; ++q) f[q] += g[q];
    }
#pragma unroll
    for (int q = 0; q < V::N; ++q) { s_row[c * V::N + q] = f[q]; sum += f[q]; }
  }
  const float mean = block_sum(sum, red) / (float)D;
  float sq = 0.f;
  for (int c = threadIdx.x; c < D; c += kLnThreads) { const float d = s_row[c] - mean; sq = fmaf(d, d, sq); }
  const float var = block_sum(sq, red) / (float)D;
  const float rstd = 1.0f / sqrtf(var + eps);
  const float* sh = shift + (long long)b * mod_ld;
  const float* sc = scale + (long long)b * mod_ld;
  V* out = reinterpret_cast<V*>(a + (long long)m * D);
  for (int c = threadIdx.x; c < n_vec; c += kLnThreads) {
    float f[V::N];
#pragma unroll
    for (int q = 0; q < V::N; ++q) {
      const int col = c * V::N + q;
      f[q] = fmaf((s_row[col] - mean) * rstd, 1.0f + sc[col], sh[col]);
    }
    V r; r.pack(f);
    out[c] = r;
  }
}

// bf16 rows of 256 * VPL elements: one WARP per refreshed row, the row held in registers (VPL
// 16-byte packets per lane), statistics by warp shuffles alone - no block barrier per row, 8 independent
// rows in flight per CTA.  The CTAs are persistent and each serves ONE batch item: it first puts that
// item's (1 + scale) and shift vectors into shared memory in fp32 (24 KB at D = 3072, once per CTA), so a
// row costs its own 6 KB in and 6 KB out of HBM plus shared-memory reads - not 24 KB of L1/L2 traffic for
// the vectors again.  Layout of the vectors: four planes of float4, [low/high half of a packet's (1 + scale),
// low/high half of its shift][packet], so that the lanes of a warp read consecutive 16-byte words.
template <int VPL>
__global__ void __launch_bounds__(256, (VPL > 12) ? 1 : 2)
gather_ln_modulate_warp_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ add,
                               const int* __restrict__ idx, const float* __restrict__ shift,
                               const float* __restrict__ scale, int mod_ld, __nv_bfloat16* __restrict__ a, int N,
                               int n_sel, int B, float eps) {
  using V = Vec<__nv_bfloat16>;
  constexpr int D = VPL * 256, kPackets = VPL * 32;
  extern __shared__ float4 s_mod[];                 // [4][kPackets]
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int b = blockIdx.x % B, slot = blockIdx.x / B, slots = gridDim.x / B;
  {
    const float4* sc = reinterpret_cast<const float4*>(scale + (long long)b * mod_ld);
    const float4* sh = reinterpret_cast<const float4*>(shift + (long long)b * mod_ld);
    for (int i = threadIdx.x; i < 2 * kPackets; i += 256) {        // float4 i covers columns [4i, 4i + 4)
      const float4 s4 = __ldg(sc + i), h4 = __ldg(sh + i);
      s_mod[(i & 1) * kPackets + (i >> 1)] = make_float4(1.0f + s4.x, 1.0f + s4.y, 1.0f + s4.z, 1.0f + s4.w);
      s_mod[(2 + (i & 1)) * kPackets + (i >> 1)] = h4;
    }
  }
  __syncthreads();
  for (int i = slot * 8 + warp; i < n_sel; i += slots * 8) {
    const long long row = (long long)b * N + (idx ? __ldg(idx + i) : i);
    const V* xr = reinterpret_cast<const V*>(x + row * D);
    V raw[VPL];
#pragma unroll
    for (int c = 0; c < VPL; ++c) raw[c].raw = __ldcs(&xr[c * 32 + lane].raw);
    float f[VPL][8];
#pragma unroll
    for (int c = 0; c < VPL; ++c) raw[c].unpack(f[c]);
    if (add) {
      const V* ar = reinterpret_cast<const V*>(add + row * D);
#pragma unroll
      for (int c = 0; c < VPL; ++c) raw[c].raw = __ldcs(&ar[c * 32 + lane].raw);
#pragma unroll
      for (int c = 0; c < VPL; ++c) {
        float g[8];
        raw[c].unpack(g);
#pragma unroll
        for (int q = 0; q < 8; ++q) f[c][q] += g[q];
      }
    }
    float sum = 0.f;
#pragma unroll
    for (int c = 0; c < VPL; ++c)
#pragma unroll
      for (int q = 0; q < 8; ++q) sum += f[c][q];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
    const float mean = sum / (float)D;
    float sq = 0.f;
#pragma unroll
    for (int c = 0; c < VPL; ++c)
#pragma unroll
      for (int q = 0; q < 8; ++q) { const float d = f[c][q] - mean; sq = fmaf(d, d, sq); }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xFFFFFFFFu, sq, o);
    const float rstd = 1.0f / sqrtf(sq / (float)D + eps);
    V* out = reinterpret_cast<V*>(a + ((long long)b * n_sel + i) * D);
#pragma unroll
    for (int c = 0; c < VPL; ++c) {
      const int v = c * 32 + lane;       // packet index: columns [8v, 8v + 8)
      const float4 s0 = s_mod[v], s1 = s_mod[kPackets + v], h0 = s_mod[2 * kPackets + v], h1 = s_mod[3 * kPackets + v];
      const float scl[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
      const float sft[8] = {h0.x, h0.y, h0.z, h0.w, h1.x, h1.y, h1.z, h1.w};
      float r[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) r[q] = fmaf((f[c][q] - mean) * rstd, scl[q], sft[q]);
      V o; o.pack(r);
      __stcs(&out[v].raw, o.raw);
    }
  }
}

template <int VPL>
int gather_ln_warp(const void* x, const void* add, const int* idx, const float* shift, const float* scale, int mod_ld,
                   void* a, int N, int n_sel, int B, float eps, cudaStream_t s) {
  using T = __nv_bfloat16;
  // persistent CTAs, the same number for every batch item; two per SM (one for the widest rows) is all that fits
  const int per_sm = VPL > 12 ? 1 : 2;
  int slots = (num_sms() * per_sm + B - 1) / B;
  const int need = (n_sel + 7) / 8;
  if (slots > need) slots = need;
  if (slots < 1) slots = 1;
  const size_t smem = (size_t)4 * VPL * 32 * sizeof(float4);
  gather_ln_modulate_warp_kernel<VPL><<<(unsigned)(slots * B), 256, smem, s>>>(
      (const T*)x, (const T*)add, idx, shift, scale, mod_ld, (T*)a, N, n_sel, B, eps);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

template <typename T>
int extrapolate_t(const void* p, const void* l, void* o, long long n, float c, cudaStream_t s) {
  extrapolate_kernel<T><<<stream_grid(n / Vec<T>::N), kStreamThreads, 0, s>>>((const T*)p, (const T*)l, (T*)o, n, c);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

}  // namespace

int launch_extrapolate(const void* g_prev, const void* g_last, void* out, long long n, int k, int d, int dtype,
                       cudaStream_t s) {
  const float c = (float)k / (float)d;
  return dtype == HERO_DTYPE_BF16 ? extrapolate_t<__nv_bfloat16>(g_prev, g_last, out, n, c, s)
                                  : extrapolate_t<float>(g_prev, g_last, out, n, c, s);
}

int launch_extrapolate_residual(void* x, const void* ga_prev, const void* ga_last, const void* gf_prev,
                                const void* gf_last, long long n, int k, int d, int dtype, cudaStream_t s) {
  const float c = (float)k / (float)d;
  if (dtype == HERO_DTYPE_BF16) {
    using T = __nv_bfloat16;
    const long long n_vec = n / Vec<T>::N;
    long long blocks = (n_vec + kStreamThreads - 1) / kStreamThreads;
    blocks = blocks < 1 ? 1 : (blocks > (long long)num_sms() * 32 ? (long long)num_sms() * 32 : blocks);
    extrapolate_residual_kernel<T><<<(int)blocks, kStreamThreads, 0, s>>>(
        (T*)x, (const T*)ga_prev, (const T*)ga_last, (const T*)gf_prev, (const T*)gf_last, n, c);
  } else {
    using T = float;
    const long long n_vec = n / Vec<T>::N;
    long long blocks = (n_vec + kStreamThreads - 1) / kStreamThreads;
    blocks = blocks < 1 ? 1 : (blocks > (long long)num_sms() * 32 ? (long long)num_sms() * 32 : blocks);
    extrapolate_residual_kernel<T><<<(int)blocks, kStreamThreads, 0, s>>>(
        (T*)x, (const T*)ga_prev, (const T*)ga_last, (const T*)gf_prev, (const T*)gf_last, n, c);
  }
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

int launch_extrapolate_group(void* x, const DeepGroup& grp, long long first, long long n, int k, int d, int dtype,
                             cudaStream_t s) {
  if (grp.n_entries <= 0 || n <= 0) return HERO_OK;
  const float c = (float)k / (float)d;
  const int per = dtype == HERO_DTYPE_BF16 ? 8 : 4;
  if (first % per != 0) return HERO_ERR_ALIGN;            // keeps every 16-byte access aligned
  long long blocks = (n / per + kStreamThreads - 1) / kStreamThreads;
  blocks = blocks < 1 ? 1 : (blocks > (long long)num_sms() * 16 ? (long long)num_sms() * 16 : blocks);
  if (dtype == HERO_DTYPE_BF16)
    extrapolate_group_kernel<__nv_bfloat16><<<(int)blocks, kStreamThreads, 0, s>>>((__nv_bfloat16*)x, grp, first, n, c);
  else
    extrapolate_group_kernel<float><<<(int)blocks, kStreamThreads, 0, s>>>((float*)x, grp, first, n, c);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

int launch_residual2(void* x, const void* ga, const void* gf, long long n, int dtype, cudaStream_t s) {
  if (dtype == HERO_DTYPE_BF16) {
    using T = __nv_bfloat16;
    residual2_kernel<T><<<stream_grid(n / Vec<T>::N), kStreamThreads, 0, s>>>((T*)x, (const T*)ga, (const T*)gf, n);
  } else {
    residual2_kernel<float><<<stream_grid(n / 4), kStreamThreads, 0, s>>>((float*)x, (const float*)ga,
                                                                           (const float*)gf, n);
  }
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

static int wide_grid(long long n_vec) {
  long long blocks = (n_vec + kStreamThreads - 1) / kStreamThreads;
  const long long cap = (long long)num_sms() * 32;
  return (int)(blocks < 1 ? 1 : (blocks > cap ? cap : blocks));
}

int launch_residual2_acc(void* x, const void* ga, const void* gf, float* acc, long long n, int dtype, cudaStream_t s) {
  if (dtype == HERO_DTYPE_BF16) {
    using T = __nv_bfloat16;
    residual2_acc_kernel<T><<<wide_grid(n / Vec<T>::N), kStreamThreads, 0, s>>>((T*)x, (const T*)ga, (const T*)gf, acc, n);
  } else {
    residual2_acc_kernel<float><<<wide_grid(n / 4), kStreamThreads, 0, s>>>((float*)x, (const float*)ga,
                                                                          (const float*)gf, acc, n);
  }
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

int launch_extrapolate_stack(void* x, const float* s_prev, const float* s_last, long long n, int k, int d, int dtype,
                             cudaStream_t s) {
  const float c = (float)k / (float)d;
  if (dtype == HERO_DTYPE_BF16) {
    using T = __nv_bfloat16;
    extrapolate_stack_kernel<T><<<wide_grid(n / Vec<T>::N), kStreamThreads, 0, s>>>((T*)x, s_prev, s_last, n, c);
  } else {
    extrapolate_stack_kernel<float><<<wide_grid(n / 4), kStreamThreads, 0, s>>>((float*)x, s_prev, s_last, n, c);
  }
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

static __global__ void attend_list_kernel(const int* __restrict__ idx, int n_sel, int n_text, int* __restrict__ list) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n_text) list[i] = i;
  else if (i < n_text + n_sel) list[i] = idx[i - n_text];
}
int launch_attend_list(const int* idx, int n_sel, int n_text, int* list, cudaStream_t s) {
  const int n = n_text + n_sel;
  if (n <= 0) return HERO_OK;
  attend_list_kernel<<<(n + 255) / 256, 256, 0, s>>>(idx, n_sel, n_text, list);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}
static int move_rows(bool gather, const void* src, const int* idx, void* dst, int B, int N, int n_sel, int D,
                     int dtype, cudaStream_t s) {
  const long long row_bytes = (long long)D * dtype_size(dtype);
  if (row_bytes % 16 != 0) return HERO_ERR_ALIGN;
  const long long rows = (long long)B * n_sel;
  if (rows == 0) return HERO_OK;
  long long blocks = (rows + 7) / 8;   // 8 warps per CTA, one row per warp
  const long long cap = (long long)num_sms() * 16;
  if (blocks > cap) blocks = cap;
  if (gather)
    move_rows_kernel<true><<<(int)blocks, 256, 0, s>>>((const uint4*)src, idx, (uint4*)dst, B, N, n_sel,
                                                       (int)(row_bytes / 16));
  else
    move_rows_kernel<false><<<(int)blocks, 256, 0, s>>>((const uint4*)src, idx, (uint4*)dst, B, N, n_sel,
                                                        (int)(row_bytes / 16));
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

int launch_gather_rows(const void* src, const int* idx, void* dst, int B, int N, int n_sel, int D, int dtype,
                       cudaStream_t s) {
  return move_rows(true, src, idx, dst, B, N, n_sel, D, dtype, s);
}
int launch_scatter_rows(const void* src, const int* idx, void* dst, int B, int N, int n_sel, int D, int dtype,
                        cudaStream_t s) {
  return move_rows(false, src, idx, dst, B, N, n_sel, D, dtype, s);
}

// The kernels are instantiated for 1, 2, 4 and 8 batch items so that a warp's accumulators are as many as it needs.
template <typename T, int MAXB>
static void modulation_batch_launch(const void* temb, const ModBatch& batch, int B, int n_out, int E, dim3 grid,
                                    size_t smem, cudaStream_t s) {
  modulation_batch_kernel<T, MAXB><<<grid, 256, smem, s>>>((const T*)temb, batch, B, n_out, E);
}
template <typename T, int MAXB>
static void modulation_launch(const void* temb, const void* w_mod, const void* b_mod, float* mod, int B, int n_out,
                              int E, int blocks, size_t smem, cudaStream_t s) {
  modulation_kernel<T, MAXB><<<blocks, 256, smem, s>>>((const T*)temb, (const T*)w_mod, (const T*)b_mod, mod, B, n_out, E);
}
#define HERO_MOD_DISPATCH(FN, T, ...)                      \
  do {                                                     \
    if (B <= 1) FN<T, 1>(__VA_ARGS__);                     \
    else if (B <= 2) FN<T, 2>(__VA_ARGS__);                \
    else if (B <= 4) FN<T, 4>(__VA_ARGS__);                \
    else FN<T, kModMaxB>(__VA_ARGS__);                     \
  } while (0)

int launch_modulation_batch(const void* temb, const ModBatch& batch, int B, int n_out, int E, int dtype,
                            cudaStream_t s) {
  if (B > kModMaxB || batch.n < 0 || batch.n > kMaxModBatch) return HERO_ERR_ARG;
  if (batch.n == 0) return HERO_OK;
  const size_t smem = (size_t)B * E * sizeof(float);
  int bx = (n_out + 8 * kModRows - 1) / (8 * kModRows);     // eight warps per CTA, kModRows columns per warp and turn
  const int cap = num_sms() * 2 / batch.n;     // two CTAs per SM over the whole grid (what the registers allow): one wave
  if (bx > cap) bx = cap < 1 ? 1 : cap;
  const dim3 grid(bx, batch.n);
  if (dtype == HERO_DTYPE_BF16) {
    if (E % 8) return HERO_ERR_ALIGN;
    HERO_MOD_DISPATCH(modulation_batch_launch, __nv_bfloat16, temb, batch, B, n_out, E, grid, smem, s);
  } else {
    if (E % 4) return HERO_ERR_ALIGN;
    HERO_MOD_DISPATCH(modulation_batch_launch, float, temb, batch, B, n_out, E, grid, smem, s);
  }
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

int launch_modulation(const void* temb, const void* w_mod, const void* b_mod, float* mod, int B, int n_out, int E,
                      int dtype, cudaStream_t s) {
  if (B > kModMaxB) return HERO_ERR_ARG;
  const size_t smem = (size_t)B * E * sizeof(float);
  int blocks = (n_out + 8 * kModRows - 1) / (8 * kModRows);
  const int cap = num_sms() * 2;
  if (blocks > cap) blocks = cap;
  if (dtype == HERO_DTYPE_BF16) {
    if (E % 8) return HERO_ERR_ALIGN;
    HERO_MOD_DISPATCH(modulation_launch, __nv_bfloat16, temb, w_mod, b_mod, mod, B, n_out, E, blocks, smem, s);
  } else {
    if (E % 4) return HERO_ERR_ALIGN;
    HERO_MOD_DISPATCH(modulation_launch, float, temb, w_mod, b_mod, mod, B, n_out, E, blocks, smem, s);
  }
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}
#undef HERO_MOD_DISPATCH

int launch_gather_ln_modulate(const void* x, const void* add, const int* idx, const float* shift,
                              const float* scale, int mod_ld, void* a, int B, int N, int n_sel, int D, float eps,
                              int dtype, cudaStream_t s) {
  const long long rows = (long long)B * n_sel;
  if (rows == 0) return HERO_OK;
  const size_t smem = (size_t)D * sizeof(float);
  if (dtype == HERO_DTYPE_BF16) {
    using T = __nv_bfloat16;
    if (D % 8) return HERO_ERR_ALIGN;
    // the adaLN vectors are read as float4: every block's slice starts 16-byte aligned when mod_ld % 4 == 0
    const bool vec_ok = mod_ld % 4 == 0 && ((reinterpret_cast<uintptr_t>(shift) | reinterpret_cast<uintptr_t>(scale)) & 15) == 0;
    if (vec_ok && D == 1024) return gather_ln_warp<4>(x, add, idx, shift, scale, mod_ld, a, N, n_sel, B, eps, s);
    if (vec_ok && D == 2048) return gather_ln_warp<8>(x, add, idx, shift, scale, mod_ld, a, N, n_sel, B, eps, s);
    if (vec_ok && D == 3072) return gather_ln_warp<12>(x, add, idx, shift, scale, mod_ld, a, N, n_sel, B, eps, s);
    if (vec_ok && D == 4096) return gather_ln_warp<16>(x, add, idx, shift, scale, mod_ld, a, N, n_sel, B, eps, s);
    gather_ln_modulate_kernel<T><<<(unsigned)rows, kLnThreads, smem, s>>>((const T*)x, (const T*)add, idx, shift,
                                                                           scale, mod_ld, (T*)a, N, n_sel, D, eps);
  } else {
    if (D % 4) return HERO_ERR_ALIGN;
    gather_ln_modulate_kernel<float><<<(unsigned)rows, kLnThreads, smem, s>>>(
        (const float*)x, (const float*)add, idx, shift, scale, mod_ld, (float*)a, N, n_sel, D, eps);
  }
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

}  // namespace hero
