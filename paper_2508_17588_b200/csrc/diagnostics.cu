// Diagnostics of Sec. 4.1 (hierarchical feature analysis): moments of the second-order temporal
// difference f_a - 2 f_b + f_c of one layer's features, from which the host forms the variance and
// the [0, 1] stability score, and the squared error of Eq. 5's prediction against the features that
// were actually computed.  Both are one-pass HBM-bound reductions over three tensors (three reads per
// element, nothing written but two doubles): 16-byte loads, fp32 partial sums per thread over at most
// a few hundred elements, double precision from the warp reduction on, one atomicAdd pair per block.
#include "hero_internal.h"

namespace hero {
namespace {

template <typename T>
struct Pack;
template <>
struct Pack<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&f)[4]) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  __device__ static float one(const float* p) { return *p; }
};
template <>
struct Pack<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&f)[8]) {
    const uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ static float one(const __nv_bfloat16* p) { return __bfloat162float(*p); }
};

constexpr int kThreads = 256;
constexpr int kFlushEvery = 64;   // packets a thread sums in fp32 before moving the partial sums to double

// MODE 0: u = a - 2b + c,                out += (sum u, sum u^2)
// MODE 1: u = b + (b - a) * coef - c,    out += (sum u^2, sum c^2)
template <typename T, int MODE>
__global__ void __launch_bounds__(kThreads) moments_kernel(const T* __restrict__ a, const T* __restrict__ b,
                                                          const T* __restrict__ c, long long n, float coef,
                                                          double* __restrict__ out) {
  constexpr int V = Pack<T>::N;
  const long long n_vec = n / V;
  const long long stride = (long long)gridDim.x * kThreads;
  double d0 = 0.0, d1 = 0.0;
  float s0 = 0.f, s1 = 0.f;
  int pending = 0;
  auto term = [&](float fa, float fb, float fc) {
    if (MODE == 0) {
      const float u = (fa - fb) + (fc - fb);
      s0 += u; s1 = fmaf(u, u, s1);
    } else {
      const float u = fmaf(fb - fa, coef, fb) - fc;
      s0 = fmaf(u, u, s0); s1 = fmaf(fc, fc, s1);
    }
  };
  for (long long v = (long long)blockIdx.x * kThreads + threadIdx.x; v < n_vec; v += stride) {
    float fa[V], fb[V], fc[V];
    Pack<T>::load(a + v * V, fa); Pack<T>::load(b + v * V, fb); Pack<T>::load(c + v * V, fc);
#pragma unroll
    for (int i = 0; i < V; ++i) term(fa[i], fb[i], fc[i]);
    if (++pending == kFlushEvery) { d0 += s0; d1 += s1; s0 = s1 = 0.f; pending = 0; }
  }
  // ragged tail (fewer than V elements), by the first threads of block 0
  if (blockIdx.x == 0 && threadIdx.x < (int)(n - n_vec * V)) {
    const long long i = n_vec * V + threadIdx.x;
    term(Pack<T>::one(a + i), Pack<T>::one(b + i), Pack<T>::one(c + i));
  }
  d0 += s0; d1 += s1;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    d0 += __shfl_xor_sync(0xffffffffu, d0, o);
    d1 += __shfl_xor_sync(0xffffffffu, d1, o);
  }
  __shared__ double w0[kThreads / 32], w1[kThreads / 32];
  if ((threadIdx.x & 31) == 0) { w0[threadIdx.x >> 5] = d0; w1[threadIdx.x >> 5] = d1; }
  __syncthreads();
  if (threadIdx.x == 0) {
    double t0 = 0.0, t1 = 0.0;
#pragma unroll
    for (int i = 0; i < kThreads / 32; ++i) { t0 += w0[i]; t1 += w1[i]; }
    atomicAdd(out, t0);
    atomicAdd(out + 1, t1);
  }
}

template <int MODE>
int launch(const void* a, const void* b, const void* c, long long n, float coef, int dtype, double* out,
           cudaStream_t s) {
  int dev = 0, sms = 0;
  HERO_CUDA_TRY(cudaGetDevice(&dev));
  HERO_CUDA_TRY(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  const int per = dtype == HERO_DTYPE_BF16 ? 8 : 4;
  long long blocks = (n / per + kThreads - 1) / kThreads;
  blocks = blocks < 1 ? 1 : (blocks > (long long)sms * 8 ? (long long)sms * 8 : blocks);
  if (dtype == HERO_DTYPE_BF16)
    moments_kernel<__nv_bfloat16, MODE><<<(int)blocks, kThreads, 0, s>>>(
        static_cast<const __nv_bfloat16*>(a), static_cast<const __nv_bfloat16*>(b),
        static_cast<const __nv_bfloat16*>(c), n, coef, out);
  else
    moments_kernel<float, MODE><<<(int)blocks, kThreads, 0, s>>>(static_cast<const float*>(a),
                                                                static_cast<const float*>(b),
                                                                static_cast<const float*>(c), n, coef, out);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

int check(const void* a, const void* b, const void* c, long long n, int dtype, const double* out) {
  if (n < 0) return HERO_ERR_ARG;
  if (dtype != HERO_DTYPE_FP32 && dtype != HERO_DTYPE_BF16) return HERO_ERR_ARG;
  if (!out) return HERO_ERR_ARG;
  if (n == 0) return 1;
  if (!a || !b || !c) return HERO_ERR_ARG;
  if (((uintptr_t)a | (uintptr_t)b | (uintptr_t)c) & 15) return HERO_ERR_ALIGN;
  if ((uintptr_t)out & 7) return HERO_ERR_ALIGN;
  return HERO_OK;
}

}  // namespace
}  // namespace hero

extern "C" {

int hero_second_difference_moments(const void* d_f_a, const void* d_f_b, const void* d_f_c, long long n_elem,
                                   int dtype, double* d_moments, void* stream) {
  const int r = hero::check(d_f_a, d_f_b, d_f_c, n_elem, dtype, d_moments);
  if (r != HERO_OK) return r < 0 ? r : HERO_OK;
  return hero::launch<0>(d_f_a, d_f_b, d_f_c, n_elem, 0.f, dtype, d_moments, (cudaStream_t)stream);
}

int hero_extrapolation_error(const void* d_g_prev, const void* d_g_last, const void* d_g_true, long long n_elem,
                             int k, int d, int dtype, double* d_err, void* stream) {
  if (d <= 0 || k < 0) return HERO_ERR_ARG;
  const int r = hero::check(d_g_prev, d_g_last, d_g_true, n_elem, dtype, d_err);
  if (r != HERO_OK) return r < 0 ? r : HERO_OK;
  return hero::launch<1>(d_g_prev, d_g_last, d_g_true, n_elem, (float)k / (float)d, dtype, d_err,
                         (cudaStream_t)stream);
}

}  // extern "C"
