// Internal declarations shared by the translation units of libhero.so.
// Nothing here is part of the public ABI (see include/hero.h).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "hero.h"

namespace hero {

// ---------------------------------------------------------------------------
// Error plumbing
// ---------------------------------------------------------------------------
void set_cuda_error(cudaError_t e, const char* what);
#define HERO_CUDA_TRY(expr)                                  \
  do {                                                       \
    cudaError_t e__ = (expr);                                \
    if (e__ != cudaSuccess) {                                \
      ::hero::set_cuda_error(e__, #expr);                    \
      return HERO_ERR_CUDA;                                  \
    }                                                        \
  } while (0)
#define HERO_TRY(expr)                  \
  do {                                  \
    int r__ = (expr);                   \
    if (r__ != HERO_OK) return r__;     \
  } while (0)

static inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ---------------------------------------------------------------------------
// Set-up that has to happen once PER DEVICE (a kernel's shared-memory opt-in, a status word in that
// device's memory, its SM count): a process may drive several GPUs, so nothing of this kind may be
// cached per process.  `fn` runs under the table's lock, with the calling thread's device current, the
// first time that device comes by; a failure is not remembered and is retried on the next call.
// ---------------------------------------------------------------------------
constexpr int kMaxDevices = 64;
struct PerDeviceOnce {
  std::mutex mu;
  bool done[kMaxDevices] = {};
};
template <class F>
int per_device_once(PerDeviceOnce& once, F&& fn) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return HERO_ERR_CUDA;
  std::lock_guard<std::mutex> lock(once.mu);
  if (!once.done[dev]) {
    const int rc = fn(dev);
    if (rc != HERO_OK) return rc;
    once.done[dev] = true;
  }
  return HERO_OK;
}
static inline size_t dtype_size(int dtype) { return dtype == HERO_DTYPE_BF16 ? 2 : 4; }

// ---------------------------------------------------------------------------
// Where a GEMM's output goes (Eq. 3's merge happens in the epilogue).
// The N dimension is cut into up to three segments of seg_cols columns (q | k | v for the
// QKV projection, one segment otherwise).  Row m of the compact operand belongs to batch
// b = m / n_sel and list position i = m % n_sel; a scattered segment writes it to row
// b * n_rows + (idx ? idx[i] : i) of its destination, a compact segment to row m.
// ---------------------------------------------------------------------------
struct GemmOut {
  void* ptr[3];
  long long ld[3];
  int scatter[3];
  int seg_cols;
  const int* idx;
  int n_sel;
  int n_rows;
  const float* gate;   // optional multiplier [B, gate_ld], indexed by column within the segment
  int gate_ld;
  int act;             // 0 = identity, 1 = GELU-tanh
  float seg0_scale;    // when not 0: factor on the columns of segment 0 (applied after the bias, before rounding)
};

// Geometry of the selection problem (Sec. 4.3).
struct SelectGeom {
  int frames, grid_h, grid_w, n_text;
  int patch_h, patch_w;
  int ratio_num, ratio_den, quota_mode, track_mode;
  uint32_t seed_lo;
};
constexpr int kMaxSelectBatch = 64;
struct SelectBatch {
  int n;                                  // number of blocks selected in this launch
  int block[kMaxSelectBatch];             // block id (enters the hash)
  int call[kMaxSelectBatch];              // per-block call counter value
  const uint16_t* ages_in[kMaxSelectBatch];
  uint16_t* ages_out[kMaxSelectBatch];
  int* idx[kMaxSelectBatch];
};

// ---------------------------------------------------------------------------
// Kernel launchers (each returns HERO_OK or HERO_ERR_CUDA; all asynchronous)
// ---------------------------------------------------------------------------
int launch_select(const SelectGeom& g, const SelectBatch& batch, cudaStream_t s);

int launch_extrapolate(const void* g_prev, const void* g_last, void* out, long long n, int k, int d,
                       int dtype, cudaStream_t s);
// x += e(attn history) ; x += e(ffn history)
int launch_extrapolate_residual(void* x, const void* ga_prev, const void* ga_last, const void* gf_prev,
                                const void* gf_last, long long n, int k, int d, int dtype, cudaStream_t s);
// Several extrapolated blocks in one pass: x += sum over the group's (block, branch) entries of Eq. 5,
// added in the order of the entries, for elements [first, first + n) of every tensor.
constexpr int kMaxDeepGroup = 32;           // blocks per launch (two entries each)
struct DeepGroup {
  int n_entries;
  const void* prev[2 * kMaxDeepGroup];
  const void* last[2 * kMaxDeepGroup];
};
int launch_extrapolate_group(void* x, const DeepGroup& grp, long long first, long long n, int k, int d, int dtype,
                             cudaStream_t s);
// x = (x + ga) + gf
int launch_residual2(void* x, const void* ga, const void* gf, long long n, int dtype, cudaStream_t s);
// deep-stack collapse: x = (x + ga) + gf, acc += ga + gf (fp32);  x += s_last + (s_last - s_prev) * k/d
int launch_residual2_acc(void* x, const void* ga, const void* gf, float* acc, long long n, int dtype, cudaStream_t s);
int launch_extrapolate_stack(void* x, const float* s_prev, const float* s_last, long long n, int k, int d, int dtype,
                             cudaStream_t s);
// Per-head LayerNorm and rotary embedding of fresh q (compact) and k (in the cache) rows.
struct QkPrepArgs {
  void* q;                 // [B, n_sel, D]
  void* k;                 // [B, N, D], rows idx[i] (or i when idx is null)
  const int* idx;
  const void *qn_w, *qn_b, *kn_w, *kn_b;   // [head_dim] in the run dtype, or all null
  const float2* rope;      // (cos, sin) per (axis position, pair) or null
  int B, N, n_sel, D, n_heads, head_dim;
  int n_text, frames, grid_h, grid_w;
  int p_t, p_h, p_w;       // rotary pairs per axis
  float eps;
  float q_scale;           // when not 0: factor on the finished q rows (the softmax scale, folded in here)
};
int launch_qk_prep(const QkPrepArgs& a, int dtype, cudaStream_t s);
// list[i] = i for i < n_text, list[n_text + i] = idx[i] for i < n_sel (rows a literal Eq. 3 attends to)
int launch_attend_list(const int* idx, int n_sel, int n_text, int* list, cudaStream_t s);
int launch_gather_rows(const void* src, const int* idx, void* dst, int B, int N, int n_sel, int D,
                       int dtype, cudaStream_t s);
int launch_scatter_rows(const void* src, const int* idx, void* dst, int B, int N, int n_sel, int D,
                        int dtype, cudaStream_t s);
// mod[b, j] = b_mod[j] + sum_e silu(temb[b,e]) * w_mod[j,e]   (fp32 output)
// The adaLN vectors of several blocks in one launch (they depend on the timestep embedding only).
constexpr int kMaxModBatch = 64;
struct ModBatch {
  int n;
  const void* w_mod[kMaxModBatch];
  const void* b_mod[kMaxModBatch];
  float* mod[kMaxModBatch];
};
int launch_modulation_batch(const void* temb, const ModBatch& batch, int B, int n_out, int E, int dtype, cudaStream_t s);
int launch_modulation(const void* temb, const void* w_mod, const void* b_mod, float* mod, int B,
                      int n_out, int E, int dtype, cudaStream_t s);
// a[m,:] = LN(x[row(m),:] (+ add[row(m),:])) * (1 + scale[b,:]) + shift[b,:]
int launch_gather_ln_modulate(const void* x, const void* add, const int* idx, const float* shift,
                              const float* scale, int mod_ld, void* a, int B, int N, int n_sel, int D,
                              float eps, int dtype, cudaStream_t s);

// fp32 / generic CUDA-core path (config 1 runs in fp32, where tensor cores would break parity)
int launch_simt_gemm(const void* a, const void* w, const void* bias, int M, int Nout, int K,
                     const GemmOut& out, int dtype, cudaStream_t s);
int launch_simt_attention(const void* q, const void* k, const void* v, void* o, int B, int n_q, int N,
                          int heads, int head_dim, int dtype, cudaStream_t s);

// bf16 tensor-core path (tcgen05 + TMEM + TMA)
int tc_init_driver_api();   // resolves cuTensorMapEncodeTiled once
int launch_tc_gemm(const void* a, const void* w, const void* bias, int M, int Nout, int K,
                   const GemmOut& out, int* d_status, cudaStream_t s);
// d_status: word 0 (give-up counter) followed by status_ctas per-CTA words
// The tensor-core attention serves head_dim 64: a score s enters the softmax as 2^(s * kScoreScaleLog2).
constexpr float kScoreScaleLog2 = 0.125f * 1.4426950408889634f;   // 1/sqrt(64) * log2(e)
// q_prescaled: Q holds q * kScoreScaleLog2 (the softmax scale folded into the projection)
int launch_tc_attention(const void* q, const void* k, const void* v, void* o, int B, int n_q, int N,
                        int heads, bool q_prescaled, int* d_status, int status_ctas, cudaStream_t s);
int launch_tc_attention_safe(const void* q, const void* k, const void* v, void* o, int B, int n_q, int N,
                             int heads, bool q_prescaled, int* d_status, cudaStream_t s);
long long tc_attention_grid(int B, int n_q, int heads);   // CTAs of one attention launch

// one thread block, no TMA, no TMEM: a bounded wait on a barrier nobody arms; raises *d_status and returns
int launch_wait_timeout_selftest(int* d_status, int budget_us, cudaStream_t s);

int num_sms();

}  // namespace hero
