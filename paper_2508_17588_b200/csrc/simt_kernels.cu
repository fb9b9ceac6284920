// CUDA-core GEMM and attention for the fp32 run mode (config "tiny": fp32 parity at ~1e-5
// against the float64 oracle rules out tensor-core input rounding).  Same epilogue contract
// as the tensor-core path: bias, optional GELU-tanh / gate, and the merge of Eq. 3 done by
// writing rows straight into their cache slots.
#include "hero_internal.h"

namespace hero {
namespace {

template <typename T>
__device__ __forceinline__ float ldf(const T* p);
template <>
__device__ __forceinline__ float ldf<float>(const float* p) { return __ldg(p); }
template <>
__device__ __forceinline__ float ldf<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T>
__device__ __forceinline__ void stf(T* p, float v);
template <>
__device__ __forceinline__ void stf<float>(float* p, float v) { *p = v; }
template <>
__device__ __forceinline__ void stf<__nv_bfloat16>(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float gelu_tanh(float t) {
  const float kAlpha = 0.7978845608028654f;   // sqrt(2/pi)
  return 0.5f * t * (1.0f + tanhf(kAlpha * (t + 0.044715f * t * t * t)));
}

// C tile 64x64, K step 16, 256 threads, 4x4 outputs per thread, fp32 FMA accumulation.
constexpr int BM = 64, BN = 64, BK = 16;
template <typename T>
__global__ void __launch_bounds__(256) simt_gemm_kernel(const T* __restrict__ A, const T* __restrict__ W,
                                                        const T* __restrict__ bias, int M, int Nout, int K,
                                                        const GemmOut out) {
  __shared__ float sA[BK][BM + 1];
  __shared__ float sW[BK][BN + 1];
  const int m0 = blockIdx.y * BM, n0 = blockIdx.x * BN;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += BK) {
    for (int e = threadIdx.x; e < BM * BK; e += 256) {
      const int r = e / BK, c = e - r * BK;
      const int gm = m0 + r, gk = k0 + c;
      sA[c][r] = (gm < M && gk < K) ? ldf(A + (long long)gm * K + gk) : 0.f;
      const int gn = n0 + r;
      sW[c][r] = (gn < Nout && gk < K) ? ldf(W + (long long)gn * K + gk) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = sA[kk][ty * 4 + i]; w[i] = sW[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
    const int b = m / out.n_sel, li = m - b * out.n_sel;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= Nout) continue;
      const int seg = n / out.seg_cols, col = n - seg * out.seg_cols;
      float v = acc[i][j] + ldf(bias + n);
      if (out.act == 1) v = gelu_tanh(v);
      if (out.gate) v *= out.gate[(long long)b * out.gate_ld + col];
      const long long row = out.scatter[seg] ? (long long)b * out.n_rows + (out.idx ? out.idx[li] : li) : (long long)m;
      stf(reinterpret_cast<T*>(out.ptr[seg]) + row * out.ld[seg] + col, v);
    }
  }
}

// One warp per (query row, head).  Keys are taken 32 at a time: each lane scores one key
// (full dot product over head_dim), the warp agrees on the running maximum, and the
// probability-weighted V rows are accumulated with the lanes owning head_dim/32 columns each.
// Online softmax: no score matrix is stored.
template <typename T, int HD>
__global__ void __launch_bounds__(128) simt_attention_kernel(const T* __restrict__ Q, const T* __restrict__ Kc,
                                                             const T* __restrict__ Vc, T* __restrict__ O, int B,
                                                             int n_q, int N, int heads) {
  constexpr int PER = HD / 32;
  __shared__ float s_q[4][HD];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long w = (long long)blockIdx.x * 4 + warp;
  const long long total = (long long)B * n_q * heads;
  const bool active = w < total;
  const long long wq = active ? w : 0;
  const int h = (int)(wq % heads);
  const long long mrow = wq / heads;           // b * n_q + i
  const int b = (int)(mrow / n_q);
  const int D = heads * HD;
  const T* q = Q + mrow * D + h * HD;
  for (int c = lane; c < HD; c += 32) s_q[warp][c] = ldf(q + c);
  __syncwarp();
  const float scale = rsqrtf((float)HD);
  float m_run = -INFINITY, l_run = 0.f, acc[PER];
#pragma unroll
  for (int p = 0; p < PER; ++p) acc[p] = 0.f;
  const T* kb = Kc + (long long)b * N * D + h * HD;
  const T* vb = Vc + (long long)b * N * D + h * HD;
  for (int j0 = 0; j0 < N; j0 += 32) {
    const int j = j0 + lane;
    float s = -INFINITY;
    if (j < N) {
      const T* kr = kb + (long long)j * D;
      float dot = 0.f;
#pragma unroll 8
      for (int c = 0; c < HD; ++c) dot = fmaf(s_q[warp][c], ldf(kr + c), dot);
      s = dot * scale;
    }
    float m_tile = s;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m_tile = fmaxf(m_tile, __shfl_xor_sync(0xFFFFFFFFu, m_tile, o));
    const float m_new = fmaxf(m_run, m_tile);
    const float alpha = expf(m_run - m_new);          // exp(-inf) = 0 on the first tile
    const float p = (j < N) ? expf(s - m_new) : 0.f;
    float psum = p;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) psum += __shfl_xor_sync(0xFFFFFFFFu, psum, o);
    l_run = l_run * alpha + psum;
#pragma unroll
    for (int pp = 0; pp < PER; ++pp) acc[pp] *= alpha;
    const int cnt = min(32, N - j0);
    for (int t = 0; t < cnt; ++t) {
      const float pt = __shfl_sync(0xFFFFFFFFu, p, t);
      const T* vr = vb + (long long)(j0 + t) * D;
#pragma unroll
      for (int pp = 0; pp < PER; ++pp) acc[pp] = fmaf(pt, ldf(vr + lane + 32 * pp), acc[pp]);
    }
    m_run = m_new;
  }
  if (active) {
    T* o = O + mrow * D + h * HD;
#pragma unroll
    for (int pp = 0; pp < PER; ++pp) stf(o + lane + 32 * pp, acc[pp] / l_run);
  }
}

}  // namespace

int launch_simt_gemm(const void* a, const void* w, const void* bias, int M, int Nout, int K, const GemmOut& out,
                     int dtype, cudaStream_t s) {
  if (M <= 0) return HERO_OK;
  dim3 grid((Nout + BN - 1) / BN, (M + BM - 1) / BM);
  if (dtype == HERO_DTYPE_BF16)
    simt_gemm_kernel<__nv_bfloat16><<<grid, 256, 0, s>>>((const __nv_bfloat16*)a, (const __nv_bfloat16*)w,
                                                         (const __nv_bfloat16*)bias, M, Nout, K, out);
  else
    simt_gemm_kernel<float><<<grid, 256, 0, s>>>((const float*)a, (const float*)w, (const float*)bias, M, Nout, K, out);
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

int launch_simt_attention(const void* q, const void* k, const void* v, void* o, int B, int n_q, int N, int heads,
                          int head_dim, int dtype, cudaStream_t s) {
  const long long total = (long long)B * n_q * heads;
  if (total == 0) return HERO_OK;
  const unsigned blocks = (unsigned)((total + 3) / 4);
#define HERO_ATT(T, HD)                                                                                       \
  simt_attention_kernel<T, HD><<<blocks, 128, 0, s>>>((const T*)q, (const T*)k, (const T*)v, (T*)o, B, n_q, N, heads)
  if (dtype == HERO_DTYPE_BF16) {
    if (head_dim == 64) HERO_ATT(__nv_bfloat16, 64);
    else if (head_dim == 32) HERO_ATT(__nv_bfloat16, 32);
    else if (head_dim == 128) HERO_ATT(__nv_bfloat16, 128);
    else return HERO_ERR_ARG;
  } else {
    if (head_dim == 64) HERO_ATT(float, 64);
    else if (head_dim == 32) HERO_ATT(float, 32);
    else if (head_dim == 128) HERO_ATT(float, 128);
    else return HERO_ERR_ARG;
  }
#undef HERO_ATT
  HERO_CUDA_TRY(cudaGetLastError());
  return HERO_OK;
}

}  // namespace hero
