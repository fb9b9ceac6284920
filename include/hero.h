/*
 * hero.h - C ABI of the HERO cached DiT denoising step for NVIDIA B200 (sm_100a).
 *
 * The library implements the hot path of "HERO: Hierarchical Extrapolation and
 * Refresh for Efficient World Models": in shallow blocks a patch-wise,
 * frequency-aware sampler picks tokens, only those rows are recomputed through
 * attention and the FFN and merged back into a per-block feature cache (Sec. 4.3,
 * Eq. 3, Eq. 4); in deep blocks attention and FFN are skipped and the branch
 * outputs are linearly extrapolated from two cached steps (Sec. 4.4, Eq. 5);
 * Algorithm 1 sequences the two.
 *
 * Conventions
 *   - Every pointer named d_* is DEVICE memory, h_* is HOST memory.  The caller
 *     owns all buffers it passes; the context owns every cache, counter and
 *     workspace it allocates in hero_init and frees them in hero_destroy.
 *   - Sequence layout: x is [batch, N, hidden] row-major, N = n_text + frames *
 *     grid_h * grid_w; the n_text text rows come first, then video tokens in
 *     (frame, y, x) order.  Run dtype (fp32 or bf16) applies to x, temb, weights
 *     and caches alike.
 *   - Weight matrices are row-major [out_features, in_features] (K contiguous).
 *     Device pointers must be 16-byte aligned; in bf16 mode hidden and ffn_dim must be
 *     multiples of 32, temb_dim a multiple of 8 and head_dim must be 64.  batch * temb_dim
 *     is at most 12288, and hidden at most 12288 unless the run is bf16 with hidden 1024,
 *     2048, 3072 or 4096 (shared-memory limits of the streaming kernels); hero_init
 *     refuses anything else with HERO_ERR_ARG / HERO_ERR_ALIGN.
 *   - All work is enqueued on the CUDA stream given to hero_init; no call
 *     synchronises the device unless stated.  Calls on one context must not
 *     overlap in time.  hero_step, hero_refresh_block and the extrapolation calls
 *     only enqueue kernels (no allocation, no host read), so they may be recorded
 *     by a stream capture into a CUDA graph; the context's host-side counters
 *     advance at capture time, once, as if the step had run, so each captured step
 *     is to be replayed exactly once.
 *   - Return value: HERO_OK (0) or a negative HERO_ERR_* code.  After an argument
 *     error nothing has been launched.  No exception crosses this boundary.
 */
#ifndef HERO_H_
#define HERO_H_

#ifdef __cplusplus
extern "C" {
#endif

#define HERO_OK            0
#define HERO_ERR_ARG      -1   /* NULL pointer, size out of range, inconsistent config */
#define HERO_ERR_ALIGN    -2   /* pointer not 16-byte aligned / dimension not vectorisable */
#define HERO_ERR_CAP      -3   /* index list capacity too small */
#define HERO_ERR_STATE    -4   /* call order violated (e.g. cached step before any full step) */
#define HERO_ERR_CUDA     -5   /* a CUDA runtime/driver call failed; see hero_last_cuda_error */
#define HERO_ERR_TIMEOUT  -6   /* a bounded device-side wait ran out (reported by hero_check_status) */
#define HERO_ERR_NOMEM    -7   /* device allocation failed */

#define HERO_DTYPE_FP32 0
#define HERO_DTYPE_BF16 1

typedef struct hero_ctx hero_ctx;   /* opaque */

/* Hyper-parameters of Algorithm 1 and the DiT block shape. */
typedef struct hero_config {
  int n_blocks;            /* L */
  int n_shallow;           /* blocks [0, n_shallow) refresh ("l < K"), the rest extrapolate */
  int hidden, n_heads, head_dim, ffn_dim, temb_dim;
  int batch, frames, grid_h, grid_w, n_text;
  int patch_h, patch_w;    /* p_h x p_w spatial patches inside each frame (Sec. 4.3) */
  int ratio_num, ratio_den;/* refresh ratio R as an exact rational, 0 < R <= 1 */
  int quota_mode;          /* 0: running-floor split of R*#P; 1: round-half-up(R*#P) */
  int warmup_full_steps;   /* leading steps that are always full ("initial caching") */
  int full_interval;       /* M: a full step every M steps after warm-up; 0 = never */
  int dtype;               /* HERO_DTYPE_* */
  int has_gate;            /* 1: adaLN also yields a gate per branch (6 chunks instead of 4) */
  unsigned long long seed; /* low 32 bits seed the sampler's counter-based hash */
  int deep_collapse;       /* 1: hero_step keeps ONE history pair for the whole deep stack (see below) */
  int track_mode;          /* frequency-aware tracking (Sec. 4.3): 0 = weighted draw, key (age+1)*(hash+1);
                              1 = strict oldest-first, key (age, hash): the longest-unsampled tokens of a
                              patch always win, the hash only breaks ties */
  int share_selection;     /* 1: hero_step draws ONE list per cached step (block 0's sampler and age
                              counters) and every shallow block refreshes those rows */
  int attend_mode;         /* which keys the refreshed queries of a cached step attend to: 0 = the full cached
                              K/V of all rows (default); 1 = only the rows refreshed in this step plus the
                              text rows (Eq. 3 read literally, F(S(z), S(tau)) with the text kept) */
  int qk_norm;             /* 1: LayerNorm (eps 1e-6) of every head's q and k features with the learned gain and
                              bias qn_w/qn_b, kn_w/kn_b of hero_block_weights, before attention (base-model
                              detail; the paper's Sec. 3 leaves the block's internals to the base model) */
  int rope;                /* 1: 3-D rotary embedding of the video rows' q and k (after qk_norm): head feature
                              pairs (2i, 2i+1); with P = head_dim/2 pairs, the first P/4 turn with the frame
                              index, the next (P - P/4)/2 with the grid row, the rest with the grid column,
                              pair i of an axis with n pairs by pos * 10000^(-i/n) radians; text rows are
                              not turned.  The K cache holds keys in this final form. */
} hero_config;

/* Device pointers to one block's parameters (borrowed for the context's lifetime).
 * w_mod [n_mod*hidden, temb_dim] with chunks (shift1, scale1, shift2, scale2[, gate1, gate2]);
 * w_qkv [3*hidden, hidden] with output chunks (q, k, v); w_o [hidden, hidden];
 * w_1 [ffn_dim, hidden]; w_2 [hidden, ffn_dim]; biases match the output size.
 * qn_w, qn_b, kn_w, kn_b [head_dim] (run dtype): gains and biases of the q/k LayerNorm, shared by the
 * heads; read only when hero_config.qk_norm is 1, NULL otherwise. */
typedef struct hero_block_weights {
  const void *w_mod, *b_mod, *w_qkv, *b_qkv, *w_o, *b_o, *w_1, *b_1, *w_2, *b_2;
  const void *qn_w, *qn_b, *kn_w, *kn_b;
} hero_block_weights;

/* ---- context ------------------------------------------------------------- */

/* Algorithm 1's state: validate cfg (the hyper-parameters of Sec. 5.1: K = n_shallow, M = full_interval,
 * R, p_h x p_w), allocate the caches Algorithm 1 writes in its "initial caching" part (K, V, G_attn, G_ffn
 * per shallow block; two history slots x two branches per deep block, which carry the same information as
 * the G and Delta G of Sec. 4.4), the age counters of Sec. 4.3's tracking, workspace and TMA descriptors
 * on the current device.  blocks[n_blocks] is copied; the weights it points to are
 * not.  cuda_stream is a cudaStream_t (NULL = legacy default stream). */
int hero_init(hero_ctx **out, const hero_config *cfg, const hero_block_weights *blocks, void *cuda_stream);
/* Back to the state before Algorithm 1's first step: forget all cached state (ages, call counters, step
 * history, which caches hold a full pass); memory is kept. */
int hero_reset(hero_ctx *ctx);
void hero_destroy(hero_ctx *ctx);
const char *hero_strerror(int code);
/* Synchronise the context's stream and return HERO_ERR_TIMEOUT if any kernel gave up on
 * a bounded wait since the last check, HERO_ERR_CUDA on a CUDA error, else HERO_OK. */
int hero_check_status(hero_ctx *ctx);
/* Text of the last failing CUDA call on this thread ("" if none). */
const char *hero_last_cuda_error(void);
/* Bytes of device memory the context allocated. */
long long hero_device_bytes(const hero_ctx *ctx);

/* Kernel launches enqueued by this context since hero_init (all categories). */
long long hero_launch_count(const hero_ctx *ctx);

/* Per-category device timing.  Between hero_profile_begin and hero_profile_end every kernel the
 * context launches is bracketed by CUDA events on its stream; hero_profile_end synchronises and
 * fills ms[HERO_PROF_CATEGORIES] (summed event time) and launches[HERO_PROF_CATEGORIES]. */
#define HERO_PROF_SELECT      0   /* token selection */
#define HERO_PROF_MODULATION  1   /* adaLN vectors from the timestep embedding */
#define HERO_PROF_GATHER_LN   2   /* gather + LayerNorm + modulate */
#define HERO_PROF_GEMM        3   /* QKV, out-proj, FFN up/down (epilogue scatters into the caches) */
#define HERO_PROF_ATTENTION   4   /* refreshed queries over the full cached K/V */
#define HERO_PROF_RESIDUAL    5   /* x += G_attn + G_ffn, all rows */
#define HERO_PROF_EXTRAPOLATE 6   /* Eq. 5 + residual add in deep blocks */
#define HERO_PROF_CATEGORIES  7
int hero_profile_begin(hero_ctx *ctx);
int hero_profile_end(hero_ctx *ctx, double *h_ms, long long *h_launches);

/* ---- the method's calls (Algorithm 1) ------------------------------------ */

/* S(z) of Eq. 4 for one shallow block: per patch take the quota's worth of tokens with the
 * largest keys (age+1)*(hash+1) (frequency-aware tracking, Sec. 4.3), reset their ages, age
 * the rest, and write the selected sequence rows in ascending order to d_idx (int32,
 * capacity cap).  *n_sel (host, may be NULL) receives the list length, which is a closed
 * form of the config and the block's call counter; the counter advances by one. */
int hero_select_tokens(hero_ctx *ctx, int block, int *d_idx, int cap, int *n_sel);
/* Length hero_select_tokens will produce on its next call for this block. */
int hero_next_n_sel(const hero_ctx *ctx, int block);

/* Eq. 2 on the rows listed in d_idx (ascending sequence rows, shared by the batch), merged
 * with the block's cache as in Eq. 3, followed by the residual add for ALL rows:
 * LN+modulate -> QKV -> K,V rows written to the cache -> attention of the refreshed queries
 * over the full cached K/V -> out-proj rows into G_attn -> x += G_attn -> LN+modulate ->
 * FFN (GELU-tanh) rows into G_ffn -> x += G_ffn.  d_idx == NULL with n_sel == N is the full
 * pass ("initial caching"): all rows, ages reset, deep blocks rotate their history slots.
 * n_sel == 0 refreshes nothing and only adds the cached branches (d_idx is not read).
 * d_x [batch,N,hidden] is updated in place; d_temb is [batch, temb_dim].
 * A partial or empty refresh merges with what the block's caches hold, so the block must have had a full
 * pass first (or all four caches planted with hero_state_set): HERO_ERR_STATE otherwise. */
int hero_refresh_block(hero_ctx *ctx, int block, void *d_x, const void *d_temb,
                       const int *d_idx, int n_sel);

/* Eq. 5 for a deep block, both branches, plus the residual add:
 * x += g_last + (g_last - g_prev) * k/d for the attention and the FFN history. */
int hero_extrapolate_block(hero_ctx *ctx, int block, void *d_x, int k, int d);

/* Deep-stack collapse (hero_config.deep_collapse = 1).  Eq. 5 is linear in the cached features and a
 * deep block touches nothing but the residual stream, so the sum over deep blocks of their
 * extrapolated branch outputs equals the extrapolation of the summed branch outputs.  With the flag
 * set, a full step accumulates sum_l (G_attn^l + G_ffn^l) over the deep blocks in fp32 (two history
 * slots for the whole stack instead of four tensors per deep block) and a cached step adds its
 * extrapolation to x in one pass.  Same result in exact arithmetic, fewer roundings in bf16, about
 * (n_deep * 4 - 2) fewer cache tensors.  In this mode the deep blocks are driven by hero_step only:
 * hero_refresh_block and hero_extrapolate_block on a deep block return HERO_ERR_STATE, and
 * hero_extrapolate_deep_stack applies the collapsed extrapolation on its own. */
int hero_extrapolate_deep_stack(hero_ctx *ctx, void *d_x, int k, int d);

/* One denoising step through all blocks with Algorithm 1's schedule: a full step when
 * step < warmup_full_steps or (step - (warmup-1)) % M == 0, else select+refresh in shallow
 * blocks and extrapolation in deep ones with k, d taken from the recorded full steps. */
int hero_step(hero_ctx *ctx, int step, void *d_x, const void *d_temb);
/* Same with HOST buffers: copies h_x and h_temb to the device, runs the step, copies x
 * back into h_x and synchronises the stream.  With pinned (page-locked, device-visible) host buffers a cached
 * step overlaps both copies with the work: the first refresh block fetches its rows from h_x itself
 * while x uploads on a second stream (the upload is awaited only by that block's residual pass), and finished pieces of x travel back while the deep blocks run on the
 * next piece.  Pageable buffers work too, without the overlap.  h_x must not be written by the caller during
 * the call. */
int hero_step_host(hero_ctx *ctx, int step, void *h_x, const void *h_temb);
/* 1 if hero_step would run `step` as a full step. */
int hero_is_full_step(const hero_ctx *ctx, int step);

/* ---- diagnostics (Sec. 4.1, hierarchical feature analysis; stateless) ------- */

/* Moments of the second-order temporal difference u = f_a - 2 f_b + f_c of one layer's features at
 * three consecutive steps: d_moments[0] += sum u, d_moments[1] += sum u^2 (device doubles, 8-byte
 * aligned, zeroed by the caller; calls accumulate, so a run over T steps adds T-2 calls per layer).
 * The variance of the paper's analysis is m1/n - (m0/n)^2 over the n elements summed; its [0, 1]
 * stability score is the min-max normalisation of these variances over the layers, inverted.
 * Tensors: n_elem elements of the given dtype, 16-byte aligned.  The sums are formed in double
 * precision from fp32 partial sums of at most 512 elements; the order of the block sums is not
 * fixed, so results repeat to about 1e-15 relative, not bit for bit. */
int hero_second_difference_moments(const void *d_f_a, const void *d_f_b, const void *d_f_c, long long n_elem,
                                   int dtype, double *d_moments, void *stream);
/* Squared error of Eq. 5 against the truth: with e = g_last + (g_last - g_prev) * k/d,
 * d_err[0] += sum (e - g_true)^2 and d_err[1] += sum g_true^2; sqrt(d_err[0] / d_err[1]) is the
 * relative L2 error of extrapolating k steps from two full steps d apart.  Same conventions. */
int hero_extrapolation_error(const void *d_g_prev, const void *d_g_last, const void *d_g_true, long long n_elem,
                             int k, int d, int dtype, double *d_err, void *stream);

/* ---- isolated kernels (stateless; stream = cudaStream_t) ------------------- */

/* Eq. 5 alone: out = g_last + (g_last - g_prev) * k/d over n_elem elements. */
int hero_extrapolate(const void *d_g_prev, const void *d_g_last, void *d_out, long long n_elem,
                     int k, int d, int dtype, void *stream);
/* The gather of the selected rows S(z) that Eq. 3's F(S(z), ...) starts from:
 * dst[b, i, :] = src[b, idx[i], :] for b < B, i < n_sel; src is [B,N,D], dst [B,n_sel,D]. */
int hero_gather_rows(const void *d_src, const int *d_idx, void *d_dst, int B, int N, int n_sel,
                     int D, int dtype, void *stream);
/* dst[b, idx[i], :] = src[b, i, :]; other rows of dst are not touched (Eq. 3's merge). */
int hero_scatter_rows(const void *d_src, const int *d_idx, void *d_dst, int B, int N, int n_sel,
                      int D, int dtype, void *stream);
/* The prologue of Eq. 2 alone (LayerNorm of Sec. 3's block with the adaLN scale and shift the paper's
 * equations leave out "for clarity"), fused with the gather of the selected rows:
 * out[b, i, :] = LN(x[b, idx[i], :] + add[b, idx[i], :]) * (1 + scale[b, :]) + shift[b, :], LN = zero mean,
 * unit (biased) variance over the D features, eps 1e-5, statistics in fp32.  d_x and d_add (may be NULL)
 * are [B,N,D] in `dtype`; d_idx int32[n_sel] (NULL = rows 0..n_sel-1); d_shift, d_scale fp32 with
 * batch stride mod_ld (>= D; float4 loads are used when mod_ld % 4 == 0 and both are 16-byte aligned);
 * d_out [B,n_sel,D] compact, in `dtype`.  HERO_ERR_ARG / HERO_ERR_ALIGN before anything is launched. */
int hero_gather_ln_modulate(const void *d_x, const void *d_add, const int *d_idx, const float *d_shift,
                            const float *d_scale, int mod_ld, void *d_out, int B, int N, int n_sel, int D,
                            int dtype, void *stream);
/* C[M,N] = A[M,K] * W[N,K]^T + bias[N] in bf16 with fp32 accumulation on the tensor cores
 * (act = 1 applies GELU-tanh).  The GEMM of the refresh path, exposed for tests and timing. */
int hero_gemm_bf16(const void *d_a, const void *d_w, const void *d_bias, void *d_c,
                   int M, int N, int K, int act, void *stream);
/* O[b,i,h,:] = softmax_j(Q[b,i,h,:] . K[b,j,h,:] / sqrt(head_dim)) V[b,j,h,:], j over all N
 * rows; Q,O are [B,n_q,heads*64] bf16, K,V are [B,N,heads*64] bf16.  No score matrix is stored
 * (Sec. 4.3: the refresh stays compatible with FlashAttention-style kernels).  Two launches: a fast
 * kernel that scales every row by the maximum of its first 96 scores for good, and a second one that
 * recomputes, with a running maximum, the thread blocks in which some later score exceeded that maximum
 * by more than 2^100 (no such block on ordinary inputs: it then returns at once). */
int hero_attention_bf16(const void *d_q, const void *d_k, const void *d_v, void *d_o,
                        int B, int n_q, int N, int heads, void *stream);
/* The same result from the second kernel alone (running maximum, accumulator rescaled in place when a
 * tile exceeds it by 2^8): what hero_attention_bf16 falls back to, exposed for tests and for inputs
 * known to have an extreme dynamic range. */
int hero_attention_bf16_safe(const void *d_q, const void *d_k, const void *d_v, void *d_o,
                             int B, int n_q, int N, int heads, void *stream);

/* hero_attention_bf16 for a caller that has folded the softmax scale into its queries: d_q holds
 * Q * log2(e) / sqrt(head_dim) (= Q * 0.18033688 at head_dim 64), so a score is the base-2 exponent of its
 * weight and O = sum_j 2^(Q'.K_j) V_j / sum_j 2^(Q'.K_j), the same softmax (Sec. 4.3).  This is the form
 * hero_step and hero_refresh_block use (their QKV projection writes q that way): the fast kernel then takes
 * 2^score as it stands, with no row maximum at all.  Exact while every row's largest score lies within
 * about +-100 (bf16 and fp32 share the exponent range); a row sum outside [2^-100, 2^100) hands its thread
 * block to the second kernel, as above.  Shapes, layouts and errors as hero_attention_bf16. */
int hero_attention_bf16_q_scaled(const void *d_q, const void *d_k, const void *d_v, void *d_o,
                                 int B, int n_q, int N, int heads, void *stream);

/* hero_attention_bf16 without any allocation (the paper has no counterpart: this entry point
 * exists for the sake of callers, not of the method).  hero_attention_bf16 obtains its status
 * word with cudaMalloc on first use; a caller that must never enter the CUDA allocator - a
 * serving loop that cannot take the device-wide synchronisation cudaMalloc/cudaFree imply, a
 * process whose framework already owns all device memory, code running where allocation is
 * forbidden - calls this instead.  Same arguments and same result (bit for bit); its scratch (the
 * give-up counter and the per-thread-block words through which the fast kernel hands blocks to the
 * fallback kernel) is a fixed 64.25 KiB array inside the library image, present on every GPU that
 * loads the library until the process exits.
 *   - Limit: ceil(n_q / 256) * heads * B <= 16384 (one scratch word per thread block); beyond
 *     that nothing is launched, HERO_ERR_CAP is returned and hero_last_cuda_error() says why.
 *   - The first call on each device resolves the array's device address and sets the kernel's
 *     shared-memory limit (no allocation either); make that call before any stream capture.
 *   - Every call reuses the one array and clears the words it needs on `stream` before the
 *     kernel; calls that overlap on the GPU race on it, so order them on one stream or with events.
 *   - h_gave_up (host, may be NULL): when given, the call synchronises `stream`, stores the number
 *     of thread blocks that gave up on a bounded device-side wait (0 in a healthy run) and
 *     returns HERO_ERR_TIMEOUT if it is not 0.  When NULL the call stays asynchronous.
 * Calls cudaMalloc, cudaFree or any allocating library routine: never. */
int hero_attention_bf16_static(const void *d_q, const void *d_k, const void *d_v, void *d_o,
                               int B, int n_q, int N, int heads, void *stream, int *h_gave_up);
/* The verdict of the latest hero_attention_bf16_static call on the current device, for a caller that
 * passed h_gave_up = NULL to keep that call asynchronous and still must not allocate (hero_isolated_status
 * watches a different word, one that comes from cudaMalloc).  Waits for everything queued on `stream`,
 * then stores in *h_gave_up (host, required) the number of thread blocks of that call which gave up on a
 * bounded wait and, when h_records is given, one word per thread block i < n_records (0 = finished, 2 = gave
 * up; n_records <= 16384).  Returns HERO_ERR_TIMEOUT if the count is not 0.  The paper has no counterpart. */
int hero_attention_bf16_static_status(void *stream, int *h_gave_up, int *h_records, int n_records);

/* Synchronise `stream` and return HERO_ERR_TIMEOUT if hero_gemm_bf16 / hero_attention_bf16 gave
 * up on a bounded device-side wait since the last poll, else HERO_OK.  The word that is polled lives
 * on the device that is current at the call (one per device). */
int hero_isolated_status(void *stream);
/* Self-test of the give-up path (no counterpart in the paper).  Every device-side wait of the tensor-core
 * kernels is bounded: when its budget runs out the kernel raises a status word and returns instead of
 * spinning.  This call runs exactly that on purpose, harmlessly: ONE thread block, no TMA, no tensor
 * memory, waits budget_us microseconds (1..100000) through the same helper on a barrier that nobody
 * completes, raises the word and returns.  With ctx given the word and the stream are the context's
 * (the next hero_check_status returns HERO_ERR_TIMEOUT once, then HERO_OK again); with ctx = NULL they
 * are the isolated calls' word and `stream` (hero_isolated_status reports it the same way). */
int hero_selftest_wait_timeout(hero_ctx *ctx, int budget_us, void *stream);

/* ---- state access for tests and checkpoints -------------------------------- */
#define HERO_STATE_AGES     0   /* u16[n_video] */
#define HERO_STATE_CALLS    1   /* int32[1] selection call counter */
#define HERO_STATE_K        2   /* [B,N,D] run dtype (shallow blocks) */
#define HERO_STATE_V        3
#define HERO_STATE_G_ATTN   4   /* shallow: feature cache; deep: g_last */
#define HERO_STATE_G_FFN    5
#define HERO_STATE_G_ATTN_PREV 6 /* deep blocks: g_prev */
#define HERO_STATE_G_FFN_PREV  7
#define HERO_STATE_STEPS    8   /* int32[3]: number of full steps seen, s_prev, s_last (block ignored) */
#define HERO_STATE_STACK_LAST 9  /* deep_collapse: fp32 [B,N,D] sum of the deep blocks' branch outputs, latest full step */
#define HERO_STATE_STACK_PREV 10 /* deep_collapse: the same for the full step before (block ignored for both) */
/* Copy a piece of per-block state to / from host memory (synchronises the stream). */
int hero_state_get(hero_ctx *ctx, int block, int what, void *h_out, long long bytes);
int hero_state_set(hero_ctx *ctx, int block, int what, const void *h_in, long long bytes);

#ifdef __cplusplus
}
#endif
#endif /* HERO_H_ */
