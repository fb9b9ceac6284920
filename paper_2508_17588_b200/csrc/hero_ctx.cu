// Context, bookkeeping and the C ABI of the HERO cached step (Algorithm 1).
// All device work is enqueued on the context's stream; the host only does schedule
// arithmetic (which step is full, the selection list length, k and d of Eq. 5).
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>
#include <string>
#include <vector>

#include "hero_internal.h"

namespace hero {

static thread_local std::string g_last_error;
void set_cuda_error(cudaError_t e, const char* what) {
  g_last_error = std::string(what) + ": " + cudaGetErrorString(e);
}

struct BlockMem {
  void* k = nullptr;          // shallow: K cache [B,N,D]
  void* v = nullptr;          // shallow: V cache
  void* g[2] = {nullptr, nullptr};                       // shallow: G_attn, G_ffn
  void* hist[2][2] = {{nullptr, nullptr}, {nullptr, nullptr}};   // deep: [branch][slot]
  int last_slot = 0;          // deep: slot holding g_last
  int n_hist = 0;             // deep: full passes recorded (saturates at 2)
  uint16_t* ages[2] = {nullptr, nullptr};                // shallow: double-buffered age counters
  int ages_cur = 0;
  int calls = 0;              // selections made on this block
  unsigned filled = 0;        // shallow: which of K, V, G_attn, G_ffn hold valid rows (bits 0..3); a full pass
                              // sets all four, planting a cache through hero_state_set sets its bit
};
constexpr unsigned kAllCaches = 0xFu;

}  // namespace hero

using namespace hero;

constexpr int kHostPieces = 8;                 // pieces of x copied back while the next one is computed
constexpr long long kHostPieceAlign = 4096;    // elements; keeps every piece 16-byte aligned in both dtypes

struct hero_ctx {
  hero_config cfg;
  cudaStream_t stream = nullptr;
  int N = 0, n_video = 0, n_mod = 4, idx_cap = 0;
  size_t esz = 4;
  long long elems = 0;                   // B*N*D
  std::vector<hero_block_weights> w;
  std::vector<BlockMem> blk;
  void* kv_tmp[2] = {nullptr, nullptr};  // K/V of deep blocks during full passes (never cached)
  // deep-stack collapse: branch outputs of a deep block are transient, their fp32 sum over the stack is kept
  void* deep_g[2] = {nullptr, nullptr};
  float* stack_hist[2] = {nullptr, nullptr};
  int stack_last = 0, stack_n = 0, stack_new = 0;
  // attend_mode 1: compact K/V of the rows a cached step attends to (text + refreshed) and their list
  void* kv_cmp[2] = {nullptr, nullptr};
  int* att_list = nullptr;
  // hero_step_host: device-to-host copies of finished pieces of x run on this stream, behind the events
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t piece_done[kHostPieces] = {};
  // hero_step_host, cached step with a pinned host buffer: the first refresh block normalises its rows
  // straight out of host memory while the bulk upload of x is still under way on the copy stream
  cudaEvent_t x_uploaded = nullptr;
  const void* first_rows_src = nullptr;   // device alias of the caller's pinned x, consumed by one refresh_block
  bool wait_x_upload = false;
  // rope 1: (cos, sin) of every (axis position, rotary pair), computed on the host in double precision
  float2* rope_tab = nullptr;
  int rope_pairs[3] = {0, 0, 0};
  void *ws_a = nullptr, *ws_q = nullptr, *ws_o = nullptr, *ws_u = nullptr;
  float* mod = nullptr;                  // [n_blocks, B, n_mod*D] adaLN vectors, one slot per block
  int* idx_ws = nullptr;                 // [n_shallow, idx_cap] selection lists of the current step
  int* d_status = nullptr;                // word 0: kernels that gave up on a wait; then one word per attention CTA
  int status_ctas = 0;
  void *x_stage = nullptr, *temb_stage = nullptr;
  int n_full = 0, s_prev = 0, s_last = 0;
  int mode1_n_sel = 0;
  long long bytes = 0;
  std::vector<void*> allocs;
  // launch accounting and optional per-category event timing
  long long launches[HERO_PROF_CATEGORIES] = {0};
  bool profiling = false;
  struct ProfSpan { int cat; cudaEvent_t a, b; };
  std::vector<ProfSpan> spans;        // recorded since hero_profile_begin
  std::vector<ProfSpan> span_pool;    // reusable event pairs
};

namespace {

// Every kernel launch goes through this: counts it and, while profiling, brackets it with events.
struct LaunchScope {
  hero_ctx* c; int cat; cudaEvent_t stop = nullptr;
  LaunchScope(hero_ctx* ctx, int category) : c(ctx), cat(category) {
    c->launches[cat]++;
    if (!c->profiling) return;
    hero_ctx::ProfSpan sp;
    if (!c->span_pool.empty()) { sp = c->span_pool.back(); c->span_pool.pop_back(); }
    else if (cudaEventCreate(&sp.a) != cudaSuccess || cudaEventCreate(&sp.b) != cudaSuccess) return;
    sp.cat = cat;
    cudaEventRecord(sp.a, c->stream);
    stop = sp.b;
    c->spans.push_back(sp);
  }
  ~LaunchScope() { if (stop) cudaEventRecord(stop, c->stream); }
};
#define HERO_LAUNCH(ctx, cat, expr)        \
  do {                                     \
    LaunchScope scope__(ctx, cat);         \
    int r__ = (expr);                      \
    if (r__ != HERO_OK) return r__;        \
  } while (0)

int dev_alloc(hero_ctx* c, void** p, size_t bytes) {
  *p = nullptr;
  if (bytes == 0) bytes = 16;
  cudaError_t e = cudaMalloc(p, bytes);
  if (e != cudaSuccess) {
    set_cuda_error(e, "cudaMalloc");
    cudaGetLastError();
    return HERO_ERR_NOMEM;
  }
  c->allocs.push_back(*p);
  c->bytes += (long long)bytes;
  return HERO_OK;
}

SelectGeom geom_of(const hero_config& c) {
  SelectGeom g;
  g.frames = c.frames; g.grid_h = c.grid_h; g.grid_w = c.grid_w; g.n_text = c.n_text;
  g.patch_h = c.patch_h; g.patch_w = c.patch_w;
  g.ratio_num = c.ratio_num; g.ratio_den = c.ratio_den; g.quota_mode = c.quota_mode; g.track_mode = c.track_mode;
  g.seed_lo = (uint32_t)(c.seed & 0xFFFFFFFFull);
  return g;
}

// Length of the selection list: a closed form in mode 0 (the running-floor quotas telescope),
// a constant summed once in mode 1.
int n_sel_for_call(const hero_ctx* c, int call) {
  const hero_config& g = c->cfg;
  if (g.quota_mode == 0) {
    const long long off = (long long)call * g.patch_h * g.patch_w;
    return (int)(((c->n_video + off) * g.ratio_num) / g.ratio_den - (off * g.ratio_num) / g.ratio_den);
  }
  return c->mode1_n_sel;
}

int mode1_total(const hero_config& g) {
  long long total = 0;
  for (int y0 = 0; y0 < g.grid_h; y0 += g.patch_h)
    for (int x0 = 0; x0 < g.grid_w; x0 += g.patch_w) {
      const long long n = (long long)(g.grid_h - y0 < g.patch_h ? g.grid_h - y0 : g.patch_h) *
                          (g.grid_w - x0 < g.patch_w ? g.grid_w - x0 : g.patch_w);
      long long q = (2 * n * g.ratio_num + g.ratio_den) / (2 * g.ratio_den);
      total += q < n ? q : n;
    }
  return (int)(total * g.frames);
}

bool is_full(const hero_config& g, int step) {
  if (step < g.warmup_full_steps) return true;
  return g.full_interval > 0 && (step - (g.warmup_full_steps - 1)) % g.full_interval == 0;
}

int run_gemm(hero_ctx* c, const void* a, const void* w, const void* bias, int M, int Nout, int K, const GemmOut& out) {
  LaunchScope scope(c, HERO_PROF_GEMM);
  if (c->cfg.dtype == HERO_DTYPE_BF16) return launch_tc_gemm(a, w, bias, M, Nout, K, out, c->d_status, c->stream);
  return launch_simt_gemm(a, w, bias, M, Nout, K, out, c->cfg.dtype, c->stream);
}

int run_attention(hero_ctx* c, const void* q, const void* k, const void* v, void* o, int n_q) {
  const hero_config& g = c->cfg;
  LaunchScope scope(c, HERO_PROF_ATTENTION);
  if (g.dtype == HERO_DTYPE_BF16)
    return launch_tc_attention(q, k, v, o, g.batch, n_q, c->N, g.n_heads, true, c->d_status, c->status_ctas, c->stream);
  return launch_simt_attention(q, k, v, o, g.batch, n_q, c->N, g.n_heads, g.head_dim, g.dtype, c->stream);
}

// adaLN vectors of blocks [l0, l1) into their slots of c->mod, at most kMaxModBatch blocks per launch
int modulation_for_blocks(hero_ctx* c, int l0, int l1, const void* d_temb) {
  const hero_config& g = c->cfg;
  const int mod_ld = c->n_mod * g.hidden;
  for (int l = l0; l < l1; l += kMaxModBatch) {
    ModBatch mb;
    mb.n = 0;
    for (int b = l; b < l1 && b < l + kMaxModBatch; ++b, ++mb.n) {
      mb.w_mod[mb.n] = c->w[b].w_mod; mb.b_mod[mb.n] = c->w[b].b_mod;
      mb.mod[mb.n] = c->mod + (size_t)b * g.batch * mod_ld;
    }
    HERO_LAUNCH(c, HERO_PROF_MODULATION,
                launch_modulation_batch(d_temb, mb, g.batch, mod_ld, g.temb_dim, g.dtype, c->stream));
  }
  return HERO_OK;
}

// Eq. 2 on the listed rows + Eq. 3's merge + the residual adds of Algorithm 1.  mod_ready: the block's adaLN
// vectors are in its slot already (hero_step computes them for all blocks of the step in one launch).
int refresh_block(hero_ctx* c, int block, void* d_x, const void* d_temb, const int* d_idx, int n_sel,
                  bool mod_ready = false) {
  const hero_config& g = c->cfg;
  const int B = g.batch, N = c->N, D = g.hidden, F = g.ffn_dim;
  const bool full = d_idx == nullptr;
  const bool deep = block >= g.n_shallow;
  BlockMem& bm = c->blk[block];
  const hero_block_weights& w = c->w[block];
  const int M = B * n_sel;
  const int mod_ld = c->n_mod * D;

  void *kdst, *vdst, *ga, *gf;
  int new_slot = 0;
  const bool collapse = deep && g.deep_collapse;
  if (collapse) {
    kdst = c->kv_tmp[0]; vdst = c->kv_tmp[1];
    ga = c->deep_g[0]; gf = c->deep_g[1];
  } else if (deep) {
    new_slot = bm.n_hist == 0 ? 0 : (bm.last_slot ^ 1);
    kdst = c->kv_tmp[0]; vdst = c->kv_tmp[1];
    ga = bm.hist[0][new_slot]; gf = bm.hist[1][new_slot];
  } else {
    kdst = bm.k; vdst = bm.v; ga = bm.g[0]; gf = bm.g[1];
  }

  float* mod = c->mod + (size_t)block * B * mod_ld;       // this block's slot; hero_step fills all slots up front
  if (!mod_ready)
    HERO_LAUNCH(c, HERO_PROF_MODULATION,
                launch_modulation(d_temb, w.w_mod, w.b_mod, mod, B, mod_ld, g.temb_dim, g.dtype, c->stream));
  const float* shift1 = mod;
  const float* scale1 = mod + D;
  const float* shift2 = mod + 2 * D;
  const float* scale2 = mod + 3 * D;
  const float* gate1 = g.has_gate ? mod + 4 * D : nullptr;
  const float* gate2 = g.has_gate ? mod + 5 * D : nullptr;

  // attention branch
  const void* host_rows = c->first_rows_src;
  c->first_rows_src = nullptr;
  if (host_rows && d_idx) {
    // x is still on its way to the device (hero_step_host): fetch the listed rows from the caller's pinned
    // buffer, once, normalise them from that compact copy, and plant them in the device copy of x, where the
    // FFN branch below will look for them.  The upload under way writes the same values over them.
    HERO_LAUNCH(c, HERO_PROF_GATHER_LN, launch_gather_rows(host_rows, d_idx, c->ws_o, B, N, n_sel, D, g.dtype, c->stream));
    HERO_LAUNCH(c, HERO_PROF_GATHER_LN,
                launch_gather_ln_modulate(c->ws_o, nullptr, nullptr, shift1, scale1, mod_ld, c->ws_a, B, n_sel, n_sel, D,
                                          1e-5f, g.dtype, c->stream));
    HERO_LAUNCH(c, HERO_PROF_GATHER_LN, launch_scatter_rows(c->ws_o, d_idx, d_x, B, N, n_sel, D, g.dtype, c->stream));
  } else {
    HERO_LAUNCH(c, HERO_PROF_GATHER_LN,
                launch_gather_ln_modulate(host_rows ? host_rows : d_x, nullptr, d_idx, shift1, scale1, mod_ld, c->ws_a, B,
                                          N, n_sel, D, 1e-5f, g.dtype, c->stream));
  }
  GemmOut o_qkv = {};
  o_qkv.ptr[0] = c->ws_q; o_qkv.ld[0] = D; o_qkv.scatter[0] = 0;
  o_qkv.ptr[1] = kdst;    o_qkv.ld[1] = D; o_qkv.scatter[1] = 1;
  o_qkv.ptr[2] = vdst;    o_qkv.ld[2] = D; o_qkv.scatter[2] = 1;
  o_qkv.seg_cols = D; o_qkv.idx = d_idx; o_qkv.n_sel = n_sel; o_qkv.n_rows = N;
  // The tensor-core attention takes q with the softmax scale folded in (a score is then the exponent of its
  // weight): by the projection's epilogue, or by the q/k treatment below when that runs and has the last word on q.
  const bool fold_scale = g.dtype == HERO_DTYPE_BF16;
  const bool qk_treated = g.qk_norm || g.rope;
  if (fold_scale && !qk_treated) o_qkv.seg0_scale = kScoreScaleLog2;
  HERO_TRY(run_gemm(c, c->ws_a, w.w_qkv, w.b_qkv, M, 3 * D, D, o_qkv));
  if (qk_treated) {
    QkPrepArgs qa = {};
    if (fold_scale) qa.q_scale = kScoreScaleLog2;
    qa.q = c->ws_q; qa.k = kdst; qa.idx = d_idx;
    if (g.qk_norm) { qa.qn_w = w.qn_w; qa.qn_b = w.qn_b; qa.kn_w = w.kn_w; qa.kn_b = w.kn_b; }
    qa.rope = g.rope ? c->rope_tab : nullptr;
    qa.B = B; qa.N = N; qa.n_sel = n_sel; qa.D = D; qa.n_heads = g.n_heads; qa.head_dim = g.head_dim;
    qa.n_text = g.n_text; qa.frames = g.frames; qa.grid_h = g.grid_h; qa.grid_w = g.grid_w;
    qa.p_t = c->rope_pairs[0]; qa.p_h = c->rope_pairs[1]; qa.p_w = c->rope_pairs[2];
    qa.eps = 1e-6f;
    HERO_LAUNCH(c, HERO_PROF_GATHER_LN, launch_qk_prep(qa, g.dtype, c->stream));
  }
  if (g.attend_mode == 1 && !full) {
    // Eq. 3 read literally: the refreshed queries see the refreshed rows (just written) and the text rows
    const int n_att = g.n_text + n_sel;
    HERO_LAUNCH(c, HERO_PROF_GATHER_LN, launch_attend_list(d_idx, n_sel, g.n_text, c->att_list, c->stream));
    HERO_LAUNCH(c, HERO_PROF_GATHER_LN,
                launch_gather_rows(kdst, c->att_list, c->kv_cmp[0], B, N, n_att, D, g.dtype, c->stream));
    HERO_LAUNCH(c, HERO_PROF_GATHER_LN,
                launch_gather_rows(vdst, c->att_list, c->kv_cmp[1], B, N, n_att, D, g.dtype, c->stream));
    LaunchScope scope(c, HERO_PROF_ATTENTION);
    if (g.dtype == HERO_DTYPE_BF16)
      HERO_TRY(launch_tc_attention(c->ws_q, c->kv_cmp[0], c->kv_cmp[1], c->ws_o, B, n_sel, n_att, g.n_heads, true,
                                   c->d_status, c->status_ctas, c->stream));
    else
      HERO_TRY(launch_simt_attention(c->ws_q, c->kv_cmp[0], c->kv_cmp[1], c->ws_o, B, n_sel, n_att, g.n_heads, g.head_dim,
                                     g.dtype, c->stream));
  } else {
    HERO_TRY(run_attention(c, c->ws_q, kdst, vdst, c->ws_o, n_sel));
  }
  GemmOut o_attn = {};
  o_attn.ptr[0] = ga; o_attn.ld[0] = D; o_attn.scatter[0] = 1;
  o_attn.seg_cols = D; o_attn.idx = d_idx; o_attn.n_sel = n_sel; o_attn.n_rows = N;
  o_attn.gate = gate1; o_attn.gate_ld = mod_ld;
  HERO_TRY(run_gemm(c, c->ws_o, w.w_o, w.b_o, M, D, D, o_attn));

  // FFN branch: its input rows are x + G_attn (the residual add is applied to x once, below)
  HERO_LAUNCH(c, HERO_PROF_GATHER_LN,
              launch_gather_ln_modulate(d_x, ga, d_idx, shift2, scale2, mod_ld, c->ws_a, B, N, n_sel, D, 1e-5f,
                                        g.dtype, c->stream));
  GemmOut o_up = {};
  o_up.ptr[0] = c->ws_u; o_up.ld[0] = F; o_up.scatter[0] = 0;
  o_up.seg_cols = F; o_up.idx = d_idx; o_up.n_sel = n_sel; o_up.n_rows = N; o_up.act = 1;
  HERO_TRY(run_gemm(c, c->ws_a, w.w_1, w.b_1, M, F, D, o_up));
  GemmOut o_dn = {};
  o_dn.ptr[0] = gf; o_dn.ld[0] = D; o_dn.scatter[0] = 1;
  o_dn.seg_cols = D; o_dn.idx = d_idx; o_dn.n_sel = n_sel; o_dn.n_rows = N;
  o_dn.gate = gate2; o_dn.gate_ld = mod_ld;
  HERO_TRY(run_gemm(c, c->ws_u, w.w_2, w.b_2, M, D, F, o_dn));

  // x = (x + G_attn) + G_ffn for every row: fresh rows and cached rows alike
  if (c->wait_x_upload) {                  // every row of x is read from here on: the upload has to be complete
    c->wait_x_upload = false;
    HERO_CUDA_TRY(cudaStreamWaitEvent(c->stream, c->x_uploaded, 0));
  }
  if (collapse) {
    HERO_LAUNCH(c, HERO_PROF_RESIDUAL,
                launch_residual2_acc(d_x, ga, gf, c->stack_hist[c->stack_new], c->elems, g.dtype, c->stream));
    return HERO_OK;
  }
  HERO_LAUNCH(c, HERO_PROF_RESIDUAL, launch_residual2(d_x, ga, gf, c->elems, g.dtype, c->stream));

  if (full) {
    if (deep) {
      bm.last_slot = new_slot;
      if (bm.n_hist < 2) bm.n_hist++;
    } else {
      bm.filled = kAllCaches;
      HERO_CUDA_TRY(cudaMemsetAsync(bm.ages[bm.ages_cur], 0, (size_t)c->n_video * sizeof(uint16_t), c->stream));
    }
  }
  return HERO_OK;
}

int extrapolate_stack(hero_ctx* c, void* d_x, int k, int d) {
  if (c->stack_n == 0) return HERO_ERR_STATE;
  const int last = c->stack_last, prev = c->stack_n >= 2 ? (last ^ 1) : last;   // one slot only: Delta = 0
  HERO_LAUNCH(c, HERO_PROF_EXTRAPOLATE,
              launch_extrapolate_stack(d_x, c->stack_hist[prev], c->stack_hist[last], c->elems, k, d, c->cfg.dtype,
                                       c->stream));
  return HERO_OK;
}

int extrapolate_block(hero_ctx* c, int block, void* d_x, int k, int d) {
  BlockMem& bm = c->blk[block];
  if (bm.n_hist == 0) return HERO_ERR_STATE;
  const int last = bm.last_slot, prev = bm.n_hist >= 2 ? (last ^ 1) : last;   // one slot only: Delta = 0
  HERO_LAUNCH(c, HERO_PROF_EXTRAPOLATE,
              launch_extrapolate_residual(d_x, bm.hist[0][prev], bm.hist[0][last], bm.hist[1][prev],
                                          bm.hist[1][last], c->elems, k, d, c->cfg.dtype, c->stream));
  return HERO_OK;
}

// Blocks [l0, l1) (all extrapolated) over elements [first, first + n) of the residual stream, at most
// kMaxDeepGroup blocks per launch.
int extrapolate_blocks(hero_ctx* c, int l0, int l1, void* d_x, long long first, long long n, int k, int d) {
  for (int l = l0; l < l1; l += kMaxDeepGroup) {
    DeepGroup grp;
    grp.n_entries = 0;
    for (int b = l; b < l1 && b < l + kMaxDeepGroup; ++b) {
      const BlockMem& bm = c->blk[b];
      if (bm.n_hist == 0) return HERO_ERR_STATE;
      const int last = bm.last_slot, prev = bm.n_hist >= 2 ? (last ^ 1) : last;   // one slot only: Delta = 0
      for (int br = 0; br < 2; ++br) {
        grp.prev[grp.n_entries] = bm.hist[br][prev];
        grp.last[grp.n_entries] = bm.hist[br][last];
        grp.n_entries++;
      }
    }
    HERO_LAUNCH(c, HERO_PROF_EXTRAPOLATE, launch_extrapolate_group(d_x, grp, first, n, k, d, c->cfg.dtype, c->stream));
  }
  return HERO_OK;
}

int validate(const hero_config* g) {
  if (g->n_blocks <= 0 || g->n_shallow < 0 || g->n_shallow > g->n_blocks) return HERO_ERR_ARG;
  if (g->hidden <= 0 || g->n_heads <= 0 || g->head_dim <= 0 || g->hidden != g->n_heads * g->head_dim) return HERO_ERR_ARG;
  if (g->ffn_dim <= 0 || g->temb_dim <= 0) return HERO_ERR_ARG;
  if (g->batch <= 0 || g->batch > 8 || g->frames <= 0 || g->grid_h <= 0 || g->grid_w <= 0 || g->n_text < 0) return HERO_ERR_ARG;
  if (g->patch_h <= 0 || g->patch_w <= 0) return HERO_ERR_ARG;
  if (g->ratio_num <= 0 || g->ratio_den <= 0 || g->ratio_num > g->ratio_den) return HERO_ERR_ARG;
  if (g->quota_mode != 0 && g->quota_mode != 1) return HERO_ERR_ARG;
  if (g->warmup_full_steps < 1 || g->full_interval < 0) return HERO_ERR_ARG;
  if (g->dtype != HERO_DTYPE_FP32 && g->dtype != HERO_DTYPE_BF16) return HERO_ERR_ARG;
  if (g->n_shallow > kMaxSelectBatch) return HERO_ERR_ARG;
  if (g->deep_collapse != 0 && g->deep_collapse != 1) return HERO_ERR_ARG;
  if (g->track_mode != 0 && g->track_mode != 1) return HERO_ERR_ARG;
  if (g->share_selection != 0 && g->share_selection != 1) return HERO_ERR_ARG;
  if (g->attend_mode != 0 && g->attend_mode != 1) return HERO_ERR_ARG;
  if ((g->qk_norm != 0 && g->qk_norm != 1) || (g->rope != 0 && g->rope != 1)) return HERO_ERR_ARG;
  if ((g->qk_norm || g->rope) && (g->head_dim % 2 != 0 || g->head_dim > 256)) return HERO_ERR_ARG;
  if (g->dtype == HERO_DTYPE_BF16) {
    // the tensor-core GEMM cuts its output into 32-column pieces per destination (q | k | v, FFN width)
    if (g->head_dim != 64 || g->hidden % 32 || g->ffn_dim % 32 || g->temb_dim % 8) return HERO_ERR_ALIGN;
  } else {
    if (g->head_dim != 32 && g->head_dim != 64 && g->head_dim != 128) return HERO_ERR_ARG;
    if (g->hidden % 4 || g->ffn_dim % 4 || g->temb_dim % 4) return HERO_ERR_ALIGN;
  }
  // dynamic shared memory the streaming kernels take without an opt-in (48 KB): SiLU(temb) of the whole batch
  // in the adaLN kernels, one fp32 row in the generic LayerNorm prologue (the bf16 warp-per-row kernel, used
  // for hidden = 1024 / 2048 / 3072 / 4096, needs none)
  constexpr long long kPlainSmem = 48 * 1024;
  if ((long long)g->batch * g->temb_dim * 4 > kPlainSmem) return HERO_ERR_ARG;
  const bool warp_ln = g->dtype == HERO_DTYPE_BF16 &&
                       (g->hidden == 1024 || g->hidden == 2048 || g->hidden == 3072 || g->hidden == 4096);
  if (!warp_ln && (long long)g->hidden * 4 > kPlainSmem) return HERO_ERR_ARG;
  const long long n_video = (long long)g->frames * g->grid_h * g->grid_w;
  if (n_video + g->n_text > (1ll << 30)) return HERO_ERR_ARG;
  return HERO_OK;
}

}  // namespace

extern "C" {

const char* hero_strerror(int code) {
  switch (code) {
    case HERO_OK: return "ok";
    case HERO_ERR_ARG: return "invalid argument";
    case HERO_ERR_ALIGN: return "pointer or dimension not 16-byte aligned";
    case HERO_ERR_CAP: return "index list capacity too small";
    case HERO_ERR_STATE: return "call order violated";
    case HERO_ERR_CUDA: return "CUDA call failed";
    case HERO_ERR_TIMEOUT: return "bounded device wait ran out";
    case HERO_ERR_NOMEM: return "device allocation failed";
    default: return "unknown error";
  }
}

const char* hero_last_cuda_error(void) { return g_last_error.c_str(); }

void hero_destroy(hero_ctx* c) {
  if (!c) return;
  if (c->stream) cudaStreamSynchronize(c->stream); else cudaDeviceSynchronize();
  if (c->copy_stream) { cudaStreamSynchronize(c->copy_stream); cudaStreamDestroy(c->copy_stream); }
  for (cudaEvent_t e : c->piece_done) if (e) cudaEventDestroy(e);
  if (c->x_uploaded) cudaEventDestroy(c->x_uploaded);
  for (void* p : c->allocs) cudaFree(p);
  for (auto& sp : c->spans) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
  for (auto& sp : c->span_pool) { cudaEventDestroy(sp.a); cudaEventDestroy(sp.b); }
  delete c;
}

int hero_init(hero_ctx** out, const hero_config* cfg, const hero_block_weights* blocks, void* cuda_stream) {
  if (!out || !cfg || !blocks) return HERO_ERR_ARG;
  *out = nullptr;
  HERO_TRY(validate(cfg));
  for (int l = 0; l < cfg->n_blocks; ++l) {
    const void* ps[10] = {blocks[l].w_mod, blocks[l].b_mod, blocks[l].w_qkv, blocks[l].b_qkv, blocks[l].w_o,
                          blocks[l].b_o,   blocks[l].w_1,   blocks[l].b_1,   blocks[l].w_2,   blocks[l].b_2};
    for (const void* p : ps) {
      if (!p) return HERO_ERR_ARG;
      if (!aligned16(p)) return HERO_ERR_ALIGN;
    }
    if (cfg->qk_norm) {
      for (const void* p : {blocks[l].qn_w, blocks[l].qn_b, blocks[l].kn_w, blocks[l].kn_b}) {
        if (!p) return HERO_ERR_ARG;
        if (!aligned16(p)) return HERO_ERR_ALIGN;
      }
    }
  }
  if (cfg->dtype == HERO_DTYPE_BF16) HERO_TRY(tc_init_driver_api());
  hero_ctx* c = new (std::nothrow) hero_ctx();
  if (!c) return HERO_ERR_NOMEM;
  c->cfg = *cfg;
  c->stream = (cudaStream_t)cuda_stream;
  c->n_video = cfg->frames * cfg->grid_h * cfg->grid_w;
  c->N = cfg->n_text + c->n_video;
  c->n_mod = cfg->has_gate ? 6 : 4;
  c->esz = dtype_size(cfg->dtype);
  c->elems = (long long)cfg->batch * c->N * cfg->hidden;
  c->idx_cap = c->n_video;
  c->mode1_n_sel = mode1_total(*cfg);
  c->w.assign(blocks, blocks + cfg->n_blocks);
  c->blk.resize(cfg->n_blocks);
  const size_t tensor = (size_t)c->elems * c->esz;
  int rc = HERO_OK;
  auto A = [&](void** p, size_t bytes) { if (rc == HERO_OK) rc = dev_alloc(c, p, bytes); };
  for (int l = 0; l < cfg->n_blocks && rc == HERO_OK; ++l) {
    BlockMem& bm = c->blk[l];
    if (l < cfg->n_shallow) {
      A(&bm.k, tensor); A(&bm.v, tensor); A(&bm.g[0], tensor); A(&bm.g[1], tensor);
      A((void**)&bm.ages[0], (size_t)c->n_video * 2); A((void**)&bm.ages[1], (size_t)c->n_video * 2);
    } else if (!cfg->deep_collapse) {
      for (int br = 0; br < 2; ++br) for (int s = 0; s < 2; ++s) A(&bm.hist[br][s], tensor);
    }
  }
  if (cfg->deep_collapse && cfg->n_shallow < cfg->n_blocks) {
    A(&c->deep_g[0], tensor); A(&c->deep_g[1], tensor);
    A((void**)&c->stack_hist[0], (size_t)c->elems * sizeof(float));
    A((void**)&c->stack_hist[1], (size_t)c->elems * sizeof(float));
  }
  if (cfg->n_shallow < cfg->n_blocks) { A(&c->kv_tmp[0], tensor); A(&c->kv_tmp[1], tensor); }
  if (cfg->attend_mode == 1) {
    A(&c->kv_cmp[0], tensor); A(&c->kv_cmp[1], tensor);
    A((void**)&c->att_list, (size_t)c->N * sizeof(int));
  }
  std::vector<float2> rope_host;
  if (cfg->rope) {
    const int pairs = cfg->head_dim / 2;
    c->rope_pairs[0] = pairs / 4;
    c->rope_pairs[1] = (pairs - c->rope_pairs[0]) / 2;
    c->rope_pairs[2] = pairs - c->rope_pairs[0] - c->rope_pairs[1];
    const int extent[3] = {cfg->frames, cfg->grid_h, cfg->grid_w};
    for (int ax = 0; ax < 3; ++ax)
      for (int pos = 0; pos < extent[ax]; ++pos)
        for (int i = 0; i < c->rope_pairs[ax]; ++i) {
          const double ang = (double)pos * std::pow(10000.0, -(double)i / (double)c->rope_pairs[ax]);
          rope_host.push_back(make_float2((float)std::cos(ang), (float)std::sin(ang)));
        }
    A((void**)&c->rope_tab, (rope_host.size() + 1) * sizeof(float2));
  }
  A(&c->ws_a, tensor); A(&c->ws_q, tensor); A(&c->ws_o, tensor);
  A(&c->ws_u, (size_t)cfg->batch * c->N * cfg->ffn_dim * c->esz);
  A((void**)&c->mod, (size_t)cfg->n_blocks * cfg->batch * c->n_mod * cfg->hidden * sizeof(float));
  A((void**)&c->idx_ws, (size_t)(cfg->n_shallow > 0 ? cfg->n_shallow : 1) * c->idx_cap * sizeof(int));
  // the largest attention launch of this context is the full pass (n_q = N)
  c->status_ctas = cfg->dtype == HERO_DTYPE_BF16 ? (int)tc_attention_grid(cfg->batch, c->N, cfg->n_heads) : 0;
  A((void**)&c->d_status, (size_t)(4 + c->status_ctas) * sizeof(int));
  A(&c->x_stage, tensor);
  A(&c->temb_stage, (size_t)cfg->batch * cfg->temb_dim * c->esz);
  if (rc != HERO_OK) { hero_destroy(c); return rc; }
  if (!rope_host.empty()) {
    cudaError_t er = cudaMemcpy(c->rope_tab, rope_host.data(), rope_host.size() * sizeof(float2), cudaMemcpyHostToDevice);
    if (er != cudaSuccess) { set_cuda_error(er, "cudaMemcpy(rope table)"); hero_destroy(c); return HERO_ERR_CUDA; }
  }
  cudaError_t e = cudaMemsetAsync(c->d_status, 0, (size_t)(4 + c->status_ctas) * sizeof(int), c->stream);
  if (e != cudaSuccess) { set_cuda_error(e, "cudaMemsetAsync"); hero_destroy(c); return HERO_ERR_CUDA; }
  rc = hero_reset(c);
  if (rc != HERO_OK) { hero_destroy(c); return rc; }
  *out = c;
  return HERO_OK;
}

int hero_reset(hero_ctx* c) {
  if (!c) return HERO_ERR_ARG;
  for (int l = 0; l < c->cfg.n_blocks; ++l) {
    BlockMem& bm = c->blk[l];
    bm.calls = 0; bm.ages_cur = 0; bm.n_hist = 0; bm.last_slot = 0; bm.filled = 0;
    if (bm.ages[0]) HERO_CUDA_TRY(cudaMemsetAsync(bm.ages[0], 0, (size_t)c->n_video * 2, c->stream));
    if (bm.ages[1]) HERO_CUDA_TRY(cudaMemsetAsync(bm.ages[1], 0, (size_t)c->n_video * 2, c->stream));
  }
  c->n_full = 0; c->s_prev = 0; c->s_last = 0;
  c->stack_last = 0; c->stack_n = 0; c->stack_new = 0;
  return HERO_OK;
}

long long hero_device_bytes(const hero_ctx* c) { return c ? c->bytes : 0; }

long long hero_launch_count(const hero_ctx* c) {
  if (!c) return 0;
  long long n = 0;
  for (int i = 0; i < HERO_PROF_CATEGORIES; ++i) n += c->launches[i];
  return n;
}

int hero_profile_begin(hero_ctx* c) {
  if (!c) return HERO_ERR_ARG;
  for (auto& sp : c->spans) c->span_pool.push_back(sp);
  c->spans.clear();
  c->profiling = true;
  return HERO_OK;
}

int hero_profile_end(hero_ctx* c, double* ms, long long* launches) {
  if (!c || !ms || !launches) return HERO_ERR_ARG;
  c->profiling = false;
  HERO_CUDA_TRY(cudaStreamSynchronize(c->stream));
  for (int i = 0; i < HERO_PROF_CATEGORIES; ++i) { ms[i] = 0.0; launches[i] = 0; }
  for (auto& sp : c->spans) {
    float t = 0.f;
    HERO_CUDA_TRY(cudaEventElapsedTime(&t, sp.a, sp.b));
    ms[sp.cat] += t;
    launches[sp.cat]++;
    c->span_pool.push_back(sp);
  }
  c->spans.clear();
  return HERO_OK;
}

int hero_check_status(hero_ctx* c) {
  if (!c) return HERO_ERR_ARG;
  int st = 0;
  HERO_CUDA_TRY(cudaMemcpyAsync(&st, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  HERO_CUDA_TRY(cudaStreamSynchronize(c->stream));
  if (st != 0) {
    cudaMemsetAsync(c->d_status, 0, sizeof(int), c->stream);
    return HERO_ERR_TIMEOUT;
  }
  return HERO_OK;
}

int hero_next_n_sel(const hero_ctx* c, int block) {
  if (!c || block < 0 || block >= c->cfg.n_shallow) return HERO_ERR_ARG;
  return n_sel_for_call(c, c->blk[block].calls);
}

int hero_select_tokens(hero_ctx* c, int block, int* d_idx, int cap, int* n_sel) {
  if (!c || !d_idx) return HERO_ERR_ARG;
  if (block < 0 || block >= c->cfg.n_shallow) return HERO_ERR_ARG;
  BlockMem& bm = c->blk[block];
  const int n = n_sel_for_call(c, bm.calls);
  if (cap < n) return HERO_ERR_CAP;
  SelectBatch batch;
  batch.n = 1;
  batch.block[0] = block; batch.call[0] = bm.calls;
  batch.ages_in[0] = bm.ages[bm.ages_cur]; batch.ages_out[0] = bm.ages[bm.ages_cur ^ 1];
  batch.idx[0] = d_idx;
  HERO_LAUNCH(c, HERO_PROF_SELECT, launch_select(geom_of(c->cfg), batch, c->stream));
  bm.ages_cur ^= 1;
  bm.calls++;
  if (n_sel) *n_sel = n;
  return HERO_OK;
}

int hero_refresh_block(hero_ctx* c, int block, void* d_x, const void* d_temb, const int* d_idx, int n_sel) {
  if (!c || !d_x || !d_temb) return HERO_ERR_ARG;
  if (block < 0 || block >= c->cfg.n_blocks) return HERO_ERR_ARG;
  if (!aligned16(d_x) || !aligned16(d_temb)) return HERO_ERR_ALIGN;
  if (n_sel == 0) {                                        // empty list: nothing refreshed,
    if (block >= c->cfg.n_shallow) return HERO_ERR_ARG;    // the residual adds still happen
    BlockMem& bm = c->blk[block];
    if (bm.filled != kAllCaches) return HERO_ERR_STATE;    // nothing cached yet to add
    HERO_LAUNCH(c, HERO_PROF_RESIDUAL, launch_residual2(d_x, bm.g[0], bm.g[1], c->elems, c->cfg.dtype, c->stream));
    return HERO_OK;
  }
  if (c->cfg.deep_collapse && block >= c->cfg.n_shallow) return HERO_ERR_STATE;   // driven by hero_step only
  if (d_idx == nullptr) {
    if (n_sel != c->N) return HERO_ERR_ARG;
  } else {
    if (n_sel < 0 || n_sel > c->N) return HERO_ERR_ARG;
    if (block >= c->cfg.n_shallow) return HERO_ERR_ARG;   // deep blocks keep no K/V cache to refresh against
    // a partial refresh merges with the cache (Eq. 3): the block must have seen a full pass first
    if (c->blk[block].filled != kAllCaches) return HERO_ERR_STATE;
  }
  return refresh_block(c, block, d_x, d_temb, d_idx, n_sel);
}

int hero_extrapolate_block(hero_ctx* c, int block, void* d_x, int k, int d) {
  if (!c || !d_x) return HERO_ERR_ARG;
  if (block < c->cfg.n_shallow || block >= c->cfg.n_blocks) return HERO_ERR_ARG;
  if (k < 0 || d <= 0) return HERO_ERR_ARG;
  if (!aligned16(d_x)) return HERO_ERR_ALIGN;
  if (c->cfg.deep_collapse) return HERO_ERR_STATE;          // no per-block history in this mode
  return extrapolate_block(c, block, d_x, k, d);
}

int hero_extrapolate_deep_stack(hero_ctx* c, void* d_x, int k, int d) {
  if (!c || !d_x || k < 0 || d <= 0) return HERO_ERR_ARG;
  if (!aligned16(d_x)) return HERO_ERR_ALIGN;
  if (!c->cfg.deep_collapse || c->cfg.n_shallow >= c->cfg.n_blocks) return HERO_ERR_STATE;
  return extrapolate_stack(c, d_x, k, d);
}

int hero_is_full_step(const hero_ctx* c, int step) {
  if (!c || step < 0) return HERO_ERR_ARG;
  return is_full(c->cfg, step) ? 1 : 0;
}

// One step of Algorithm 1.  With h_out set (hero_step_host) the deep blocks of a cached step run piece by
// piece over x, and each finished piece is copied to h_out on the copy stream while the next one is
// computed; *copied_out then tells the caller that nothing is left to copy.
static int step_impl(hero_ctx* c, int step, void* d_x, const void* d_temb, void* h_out, bool* copied_out);

int hero_step(hero_ctx* c, int step, void* d_x, const void* d_temb) {
  return step_impl(c, step, d_x, d_temb, nullptr, nullptr);
}

static int step_impl(hero_ctx* c, int step, void* d_x, const void* d_temb, void* h_out, bool* copied_out) {
  if (!c || !d_x || !d_temb || step < 0) return HERO_ERR_ARG;
  if (!aligned16(d_x) || !aligned16(d_temb)) return HERO_ERR_ALIGN;
  const hero_config& g = c->cfg;
  const bool collapse = g.deep_collapse && g.n_shallow < g.n_blocks;
  if (is_full(g, step)) {
    if (collapse) {                          // the deep stack's branch outputs are summed into a fresh slot
      c->stack_new = c->stack_n == 0 ? 0 : (c->stack_last ^ 1);
      HERO_CUDA_TRY(cudaMemsetAsync(c->stack_hist[c->stack_new], 0, (size_t)c->elems * sizeof(float), c->stream));
    }
    HERO_TRY(modulation_for_blocks(c, 0, g.n_blocks, d_temb));
    for (int l = 0; l < g.n_blocks; ++l) HERO_TRY(refresh_block(c, l, d_x, d_temb, nullptr, c->N, true));
    if (collapse) { c->stack_last = c->stack_new; if (c->stack_n < 2) c->stack_n++; }
    c->s_prev = c->s_last; c->s_last = step; c->n_full++;
    return HERO_OK;
  }
  if (c->n_full == 0) return HERO_ERR_STATE;
  const int k = step - c->s_last;
  const int d = c->n_full >= 2 ? c->s_last - c->s_prev : 1;
  if (k <= 0 || d <= 0) return HERO_ERR_STATE;
  // all shallow blocks draw their lists in one launch: the draw depends on counters only
  int n_sel[kMaxSelectBatch];
  // one list for the whole step (drawn with block 0's sampler) or one per shallow block
  const int n_draws = g.share_selection ? (g.n_shallow > 0 ? 1 : 0) : g.n_shallow;
  if (g.n_shallow > 0) {
    SelectBatch batch;
    batch.n = n_draws;
    for (int l = 0; l < n_draws; ++l) {
      BlockMem& bm = c->blk[l];
      n_sel[l] = n_sel_for_call(c, bm.calls);
      batch.block[l] = l; batch.call[l] = bm.calls;
      batch.ages_in[l] = bm.ages[bm.ages_cur]; batch.ages_out[l] = bm.ages[bm.ages_cur ^ 1];
      batch.idx[l] = c->idx_ws + (size_t)l * c->idx_cap;
    }
    HERO_LAUNCH(c, HERO_PROF_SELECT, launch_select(geom_of(g), batch, c->stream));
    for (int l = 0; l < n_draws; ++l) { c->blk[l].ages_cur ^= 1; c->blk[l].calls++; }
    for (int l = n_draws; l < g.n_shallow; ++l) n_sel[l] = n_sel[0];
  }
  HERO_TRY(modulation_for_blocks(c, 0, g.n_shallow, d_temb));
  for (int l = 0; l < g.n_blocks; ++l) {
    if (l < g.n_shallow) {
      if (n_sel[l] > 0) {
        HERO_TRY(refresh_block(c, l, d_x, d_temb, c->idx_ws + (size_t)(g.share_selection ? 0 : l) * c->idx_cap, n_sel[l],
                               true));
      } else {
        HERO_LAUNCH(c, HERO_PROF_RESIDUAL,
                    launch_residual2(d_x, c->blk[l].g[0], c->blk[l].g[1], c->elems, g.dtype, c->stream));
      }
    } else if (collapse) {
      HERO_TRY(extrapolate_stack(c, d_x, k, d));   // Eq. 5 once, on the sums over all deep blocks
      break;
    } else if (h_out && c->copy_stream && c->elems >= (long long)kHostPieces * kHostPieceAlign) {
      // the rest of the stack, piece by piece, each piece on its way to the host as soon as it is final
      const long long per = ((c->elems + kHostPieces - 1) / kHostPieces + kHostPieceAlign - 1) / kHostPieceAlign *
                            kHostPieceAlign;
      for (int p = 0; p < kHostPieces; ++p) {
        const long long first = (long long)p * per;
        const long long n = first >= c->elems ? 0 : (c->elems - first < per ? c->elems - first : per);
        if (n <= 0) break;
        HERO_TRY(extrapolate_blocks(c, l, g.n_blocks, d_x, first, n, k, d));
        HERO_CUDA_TRY(cudaEventRecord(c->piece_done[p], c->stream));
        HERO_CUDA_TRY(cudaStreamWaitEvent(c->copy_stream, c->piece_done[p], 0));
        HERO_CUDA_TRY(cudaMemcpyAsync(static_cast<char*>(h_out) + first * c->esz,
                                      static_cast<const char*>(d_x) + first * c->esz, (size_t)n * c->esz,
                                      cudaMemcpyDeviceToHost, c->copy_stream));
      }
      *copied_out = true;
      break;
    } else {
      HERO_TRY(extrapolate_blocks(c, l, g.n_blocks, d_x, 0, c->elems, k, d));   // the rest of the stack in one pass
      break;
    }
  }
  return HERO_OK;
}

int hero_step_host(hero_ctx* c, int step, void* h_x, const void* h_temb) {
  if (!c || !h_x || !h_temb) return HERO_ERR_ARG;
  const size_t xb = (size_t)c->elems * c->esz, tb = (size_t)c->cfg.batch * c->cfg.temb_dim * c->esz;
  if (!c->copy_stream) {
    HERO_CUDA_TRY(cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
    for (cudaEvent_t& e : c->piece_done) HERO_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    HERO_CUDA_TRY(cudaEventCreateWithFlags(&c->x_uploaded, cudaEventDisableTiming));
  }
  // A cached step whose first block refreshes something, with x in pinned (device-visible) host memory: the
  // upload of x goes to the copy stream and the first block's LayerNorm reads its rows from the host copy, so
  // that its GEMMs and attention run while the rest of x is still on its way.
  const void* h_alias = nullptr;
  const hero_config& g = c->cfg;
  if (step >= 0 && !is_full(g, step) && g.n_shallow > 0 && c->n_full > 0 &&
      n_sel_for_call(c, c->blk[0].calls) > 0) {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, h_x) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer)
      h_alias = at.devicePointer;
    else
      cudaGetLastError();                    // pageable memory: not an error, just no shortcut
  }
  HERO_CUDA_TRY(cudaMemcpyAsync(c->temb_stage, h_temb, tb, cudaMemcpyHostToDevice, c->stream));
  if (h_alias) {
    HERO_CUDA_TRY(cudaMemcpyAsync(c->x_stage, h_x, xb, cudaMemcpyHostToDevice, c->copy_stream));
    HERO_CUDA_TRY(cudaEventRecord(c->x_uploaded, c->copy_stream));
    c->first_rows_src = h_alias;
    c->wait_x_upload = true;
  } else {
    HERO_CUDA_TRY(cudaMemcpyAsync(c->x_stage, h_x, xb, cudaMemcpyHostToDevice, c->stream));
  }
  bool copied = false;
  const int rc = step_impl(c, step, c->x_stage, c->temb_stage, h_x, &copied);
  c->first_rows_src = nullptr;
  if (rc != HERO_OK || c->wait_x_upload) {   // leave no copy in flight behind an error (or an unused upload)
    c->wait_x_upload = false;
    cudaStreamSynchronize(c->copy_stream);
    if (rc != HERO_OK) return rc;
  }
  if (!copied) HERO_CUDA_TRY(cudaMemcpyAsync(h_x, c->x_stage, xb, cudaMemcpyDeviceToHost, c->stream));
  HERO_CUDA_TRY(cudaStreamSynchronize(c->stream));
  HERO_CUDA_TRY(cudaStreamSynchronize(c->copy_stream));
  return HERO_OK;
}

// ---------------------------------------------------------------- isolated kernels
int hero_extrapolate(const void* g_prev, const void* g_last, void* out, long long n, int k, int d, int dtype,
                     void* stream) {
  if (n < 0 || d <= 0 || k < 0) return HERO_ERR_ARG;
  if (dtype != HERO_DTYPE_FP32 && dtype != HERO_DTYPE_BF16) return HERO_ERR_ARG;
  if (n == 0) return HERO_OK;
  if (!g_prev || !g_last || !out) return HERO_ERR_ARG;
  if (!aligned16(g_prev) || !aligned16(g_last) || !aligned16(out)) return HERO_ERR_ALIGN;
  return launch_extrapolate(g_prev, g_last, out, n, k, d, dtype, (cudaStream_t)stream);
}

static int check_rows(const void* src, const int* idx, void* dst, int B, int N, int n_sel, int D, int dtype) {
  if (B < 0 || N < 0 || n_sel < 0 || D <= 0 || n_sel > N) return HERO_ERR_ARG;
  if (dtype != HERO_DTYPE_FP32 && dtype != HERO_DTYPE_BF16) return HERO_ERR_ARG;
  if (B == 0 || n_sel == 0) return HERO_OK;
  if (!src || !idx || !dst) return HERO_ERR_ARG;
  if (!aligned16(src) || !aligned16(dst)) return HERO_ERR_ALIGN;
  return 1;
}
int hero_gather_rows(const void* src, const int* idx, void* dst, int B, int N, int n_sel, int D, int dtype,
                     void* stream) {
  const int r = check_rows(src, idx, dst, B, N, n_sel, D, dtype);
  if (r <= 0) return r;
  return launch_gather_rows(src, idx, dst, B, N, n_sel, D, dtype, (cudaStream_t)stream);
}
int hero_scatter_rows(const void* src, const int* idx, void* dst, int B, int N, int n_sel, int D, int dtype,
                      void* stream) {
  const int r = check_rows(src, idx, dst, B, N, n_sel, D, dtype);
  if (r <= 0) return r;
  return launch_scatter_rows(src, idx, dst, B, N, n_sel, D, dtype, (cudaStream_t)stream);
}

// Eq. 2's prologue alone: out[b, i, :] = LN(x[b, idx[i], :] (+ add[b, idx[i], :])) * (1 + scale[b, :]) + shift[b, :]
int hero_gather_ln_modulate(const void* d_x, const void* d_add, const int* d_idx, const float* d_shift,
                            const float* d_scale, int mod_ld, void* d_out, int B, int N, int n_sel, int D, int dtype,
                            void* stream) {
  if (B < 0 || N < 0 || n_sel < 0 || n_sel > N || D <= 0 || mod_ld < D) return HERO_ERR_ARG;
  if (dtype != HERO_DTYPE_FP32 && dtype != HERO_DTYPE_BF16) return HERO_ERR_ARG;
  if (B == 0 || n_sel == 0) return HERO_OK;
  if (!d_x || !d_shift || !d_scale || !d_out) return HERO_ERR_ARG;
  if (!aligned16(d_x) || !aligned16(d_out) || (d_add && !aligned16(d_add))) return HERO_ERR_ALIGN;
  if (D % (dtype == HERO_DTYPE_BF16 ? 8 : 4)) return HERO_ERR_ALIGN;
  const bool warp_ln = dtype == HERO_DTYPE_BF16 && (D == 1024 || D == 2048 || D == 3072 || D == 4096);
  if (!warp_ln && (long long)D * 4 > 48 * 1024) return HERO_ERR_ARG;      // one fp32 row of shared memory
  return launch_gather_ln_modulate(d_x, d_add, d_idx, d_shift, d_scale, mod_ld, d_out, B, N, n_sel, D, 1e-5f, dtype,
                                   (cudaStream_t)stream);
}

// The isolated tensor-core calls own a status word each; a timeout is reported on the next call.
// The words live in the memory of the device that is current at the call (one set per device, kept until exit):
// word 0 for give-ups, then one word per attention CTA (larger grids run the safe attention kernel alone).
constexpr int kIsolatedStatusCtas = 65536;
static int* isolated_status() {
  static PerDeviceOnce once;
  static int* word[kMaxDevices];
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  const int rc = per_device_once(once, [](int d) {
    int* p = nullptr;
    const size_t bytes = (size_t)(4 + kIsolatedStatusCtas) * sizeof(int);
    if (cudaMalloc((void**)&p, bytes) != cudaSuccess) { cudaGetLastError(); return HERO_ERR_NOMEM; }
    if (cudaMemset(p, 0, bytes) != cudaSuccess) { cudaFree(p); return HERO_ERR_CUDA; }
    word[d] = p;
    return HERO_OK;
  });
  return rc == HERO_OK ? word[dev] : nullptr;
}
static int poll_isolated_status(cudaStream_t s) {
  int* p = isolated_status();
  if (!p) return HERO_ERR_NOMEM;
  int st = 0;
  HERO_CUDA_TRY(cudaMemcpyAsync(&st, p, 4, cudaMemcpyDeviceToHost, s));
  HERO_CUDA_TRY(cudaStreamSynchronize(s));
  if (st) { cudaMemset(p, 0, sizeof(int)); return HERO_ERR_TIMEOUT; }
  return HERO_OK;
}

int hero_gemm_bf16(const void* a, const void* w, const void* bias, void* cmat, int M, int N, int K, int act,
                   void* stream) {
  if (M < 0 || N <= 0 || K <= 0 || (act != 0 && act != 1)) return HERO_ERR_ARG;
  if (M == 0) return HERO_OK;
  if (!a || !w || !bias || !cmat) return HERO_ERR_ARG;
  int* st = isolated_status();
  if (!st) return HERO_ERR_NOMEM;
  GemmOut o = {};
  o.ptr[0] = cmat; o.ld[0] = N; o.scatter[0] = 0;
  o.seg_cols = (N + 31) / 32 * 32; o.n_sel = M; o.n_rows = M; o.act = act;
  return launch_tc_gemm(a, w, bias, M, N, K, o, st, (cudaStream_t)stream);
}

int hero_attention_bf16(const void* q, const void* k, const void* v, void* o, int B, int n_q, int N, int heads,
                        void* stream) {
  if (B < 0 || n_q < 0 || N <= 0 || heads <= 0) return HERO_ERR_ARG;
  if (B == 0 || n_q == 0) return HERO_OK;
  if (!q || !k || !v || !o) return HERO_ERR_ARG;
  int* st = isolated_status();
  if (!st) return HERO_ERR_NOMEM;
  return launch_tc_attention(q, k, v, o, B, n_q, N, heads, false, st, kIsolatedStatusCtas, (cudaStream_t)stream);
}

int hero_attention_bf16_q_scaled(const void* q, const void* k, const void* v, void* o, int B, int n_q, int N,
                                 int heads, void* stream) {
  if (B < 0 || n_q < 0 || N <= 0 || heads <= 0) return HERO_ERR_ARG;
  if (B == 0 || n_q == 0) return HERO_OK;
  if (!q || !k || !v || !o) return HERO_ERR_ARG;
  int* st = isolated_status();
  if (!st) return HERO_ERR_NOMEM;
  return launch_tc_attention(q, k, v, o, B, n_q, N, heads, true, st, kIsolatedStatusCtas, (cudaStream_t)stream);
}

int hero_attention_bf16_safe(const void* q, const void* k, const void* v, void* o, int B, int n_q, int N, int heads,
                             void* stream) {
  if (B < 0 || n_q < 0 || N <= 0 || heads <= 0) return HERO_ERR_ARG;
  if (B == 0 || n_q == 0) return HERO_OK;
  if (!q || !k || !v || !o) return HERO_ERR_ARG;
  int* st = isolated_status();
  if (!st) return HERO_ERR_NOMEM;
  return launch_tc_attention_safe(q, k, v, o, B, n_q, N, heads, false, st, (cudaStream_t)stream);
}

// Synchronise `stream` and report whether an isolated tensor-core call gave up on a wait.
int hero_isolated_status(void* stream) { return poll_isolated_status((cudaStream_t)stream); }

// Self-test of the give-up path: one thread block waits, with a budget of `budget_us` microseconds, on a
// barrier that nobody will ever complete, through the same bounded-wait helper the tensor-core kernels use;
// the wait runs out, the block raises the status word and returns.  With a context the word is the
// context's (hero_check_status then reports HERO_ERR_TIMEOUT once), without one it is the word of the
// isolated tensor-core calls (hero_isolated_status reports it).
int hero_selftest_wait_timeout(hero_ctx* c, int budget_us, void* stream) {
  if (budget_us < 1 || budget_us > 100000) return HERO_ERR_ARG;
  int* st = c ? c->d_status : isolated_status();
  if (!st) return HERO_ERR_NOMEM;
  return launch_wait_timeout_selftest(st, budget_us, c ? c->stream : (cudaStream_t)stream);
}

// ---------------------------------------------------------------- state access
static int state_ptr(hero_ctx* c, int block, int what, void** p, size_t* bytes) {
  const hero_config& g = c->cfg;
  if (what == HERO_STATE_STEPS) { *p = nullptr; *bytes = 12; return HERO_OK; }
  if (what == HERO_STATE_STACK_LAST || what == HERO_STATE_STACK_PREV) {
    if (!g.deep_collapse || !c->stack_hist[0]) return HERO_ERR_ARG;
    *p = c->stack_hist[what == HERO_STATE_STACK_LAST ? c->stack_last : (c->stack_last ^ 1)];
    *bytes = (size_t)c->elems * sizeof(float);
    return HERO_OK;
  }
  if (block < 0 || block >= g.n_blocks) return HERO_ERR_ARG;
  BlockMem& bm = c->blk[block];
  const bool deep = block >= g.n_shallow;
  const size_t tensor = (size_t)c->elems * c->esz;
  if (deep && g.deep_collapse) return HERO_ERR_ARG;        // deep blocks keep no per-block state in this mode
  switch (what) {
    case HERO_STATE_AGES: if (deep) return HERO_ERR_ARG; *p = bm.ages[bm.ages_cur]; *bytes = (size_t)c->n_video * 2; return HERO_OK;
    case HERO_STATE_CALLS: *p = nullptr; *bytes = 4; return HERO_OK;
    case HERO_STATE_K: if (deep) return HERO_ERR_ARG; *p = bm.k; *bytes = tensor; return HERO_OK;
    case HERO_STATE_V: if (deep) return HERO_ERR_ARG; *p = bm.v; *bytes = tensor; return HERO_OK;
    case HERO_STATE_G_ATTN: *p = deep ? bm.hist[0][bm.last_slot] : bm.g[0]; *bytes = tensor; return HERO_OK;
    case HERO_STATE_G_FFN: *p = deep ? bm.hist[1][bm.last_slot] : bm.g[1]; *bytes = tensor; return HERO_OK;
    case HERO_STATE_G_ATTN_PREV: if (!deep) return HERO_ERR_ARG; *p = bm.hist[0][bm.last_slot ^ 1]; *bytes = tensor; return HERO_OK;
    case HERO_STATE_G_FFN_PREV: if (!deep) return HERO_ERR_ARG; *p = bm.hist[1][bm.last_slot ^ 1]; *bytes = tensor; return HERO_OK;
    default: return HERO_ERR_ARG;
  }
}

int hero_state_get(hero_ctx* c, int block, int what, void* h_out, long long bytes) {
  if (!c || !h_out) return HERO_ERR_ARG;
  void* p; size_t need;
  HERO_TRY(state_ptr(c, block, what, &p, &need));
  if (bytes != (long long)need) return HERO_ERR_ARG;
  if (what == HERO_STATE_STEPS) { int v[3] = {c->n_full, c->s_prev, c->s_last}; memcpy(h_out, v, 12); return HERO_OK; }
  if (what == HERO_STATE_CALLS) { memcpy(h_out, &c->blk[block].calls, 4); return HERO_OK; }
  HERO_CUDA_TRY(cudaMemcpyAsync(h_out, p, need, cudaMemcpyDeviceToHost, c->stream));
  HERO_CUDA_TRY(cudaStreamSynchronize(c->stream));
  return HERO_OK;
}

int hero_state_set(hero_ctx* c, int block, int what, const void* h_in, long long bytes) {
  if (!c || !h_in) return HERO_ERR_ARG;
  void* p; size_t need;
  HERO_TRY(state_ptr(c, block, what, &p, &need));
  if (bytes != (long long)need) return HERO_ERR_ARG;
  if (what == HERO_STATE_STEPS) {
    int v[3]; memcpy(v, h_in, 12);
    if (v[0] < 0) return HERO_ERR_ARG;
    c->n_full = v[0]; c->s_prev = v[1]; c->s_last = v[2];
    return HERO_OK;
  }
  if (what == HERO_STATE_CALLS) { int v; memcpy(&v, h_in, 4); if (v < 0) return HERO_ERR_ARG; c->blk[block].calls = v; return HERO_OK; }
  HERO_CUDA_TRY(cudaMemcpyAsync(p, h_in, need, cudaMemcpyHostToDevice, c->stream));
  HERO_CUDA_TRY(cudaStreamSynchronize(c->stream));
  if (what == HERO_STATE_STACK_LAST) { if (c->stack_n < 1) c->stack_n = 1; return HERO_OK; }
  if (what == HERO_STATE_STACK_PREV) { c->stack_n = 2; return HERO_OK; }
  if (block < c->cfg.n_shallow) {    // planting a shallow block's cache marks it as valid
    if (what == HERO_STATE_K) c->blk[block].filled |= 1u;
    if (what == HERO_STATE_V) c->blk[block].filled |= 2u;
    if (what == HERO_STATE_G_ATTN) c->blk[block].filled |= 4u;
    if (what == HERO_STATE_G_FFN) c->blk[block].filled |= 8u;
  }
  if (block >= c->cfg.n_shallow) {   // planting a deep block's history marks the slots as valid
    BlockMem& bm = c->blk[block];
    if (what == HERO_STATE_G_ATTN || what == HERO_STATE_G_FFN) { if (bm.n_hist < 1) bm.n_hist = 1; }
    if (what == HERO_STATE_G_ATTN_PREV || what == HERO_STATE_G_FFN_PREV) bm.n_hist = 2;
  }
  return HERO_OK;
}

}  // extern "C"
