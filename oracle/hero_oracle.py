"""CPU oracle of the HERO cached DiT denoising step (TEST INFRASTRUCTURE ONLY).

Plain numpy in float64, written from the paper's statement of the method
(Algorithm 1; Eq. 2, Eq. 3, Eq. 4, Eq. 5; Sec. 4.3 "Patch-wise Sampling" and
the frequency-aware tracking paragraph; Sec. 4.4).  It is slow on purpose and
shares no code with the CUDA library: tests, the smoke check and the benchmark's
CPU-baseline leg are the only callers.  Nothing here is blocked, fused or
reordered beyond what the cited passage states; `numpy.matmul`, `numpy.exp`,
`numpy.tanh` and `sorted` are used as library steps.

Where the paper leaves a point open the reading taken is stated beside the
function (and collected in the design notes):
  * refreshed queries attend to the full cached K/V of all rows, after the
    refreshed rows' K/V have been written (Eq. 3 says only F(S(z), S(tau)));
  * non-selected rows reuse whatever the cache last held (in-place cache);
  * quota per patch: exact running-floor split (mode 0) or round-half-up of
    R*#P (mode 1, the rounding Table 3's equally spaced FLOPs imply);
  * frequency-aware tracking: weight age+1, integer keys, top-q per patch;
  * one draw per (step, block) shared by both sub-layers and the batch;
  * text rows are never refreshed on cached steps;
  * cached steps extrapolate with the real gap between the last two full steps.

Parity pins: every function below is pinned by tests/test_oracle_*.py against something
other than itself (values the paper prints, closed forms, invariants, library routines,
brute force).  Three of them implement a READING of a point on which the paper is silent,
so their pins fix the function to the stated reading, not the reading to the paper:
rope_sections / rope_angles (opt-in; first pair of an axis = the position in radians,
linearity in the position, geometric frequencies spanning 1/10000, one section per axis),
token_hash's keying (bijective in token, call and block, no interchangeable inputs, no
serial correlation) and stability_scores' min-max normalisation (equally spaced variances
give equally spaced scores).  PARITY UNPINNED: the quality of the approximation on real
videos (VBench, depth, pose), which needs the paper's weights and datasets.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from functools import lru_cache

import numpy as np

F64 = np.float64
_M32 = 0xFFFFFFFF
AGE_MAX = 65535


# =============================================================================
# Configuration and geometry (Sec. 4.1, Sec. 4.3)
# =============================================================================
@dataclass
class Config:
    n_blocks: int
    n_shallow: int            # blocks [0, n_shallow) refresh, the rest extrapolate ("l < K")
    hidden: int
    n_heads: int
    head_dim: int
    ffn_dim: int
    temb_dim: int
    batch: int
    frames: int
    grid_h: int
    grid_w: int
    n_text: int
    patch_h: int
    patch_w: int
    ratio_num: int            # R = ratio_num / ratio_den
    ratio_den: int
    quota_mode: int = 0
    warmup_full_steps: int = 2
    full_interval: int = 0    # M; 0 = never again after warm-up
    has_gate: int = 0
    track_mode: int = 0       # 0: weighted draw (age+1)*(hash+1); 1: strict oldest-first (age, hash)
    share_selection: int = 0  # 1: one list per cached step (block 0's sampler) for every shallow block
    attend_mode: int = 0      # 0: refreshed queries see the full cached K/V; 1: refreshed + text rows only
    qk_norm: int = 0          # 1: per-head LayerNorm (learned affine) of q and k before attention
    rope: int = 0             # 1: 3-D rotary position embedding of the video rows' q and k
    seed: int = 0
    eps: float = 1e-5
    qk_eps: float = 1e-6
    rope_theta: float = 10000.0

    @classmethod
    def from_dict(cls, d):
        names = cls.__dataclass_fields__.keys()
        return cls(**{k: v for k, v in d.items() if k in names})

    @property
    def n_video(self):
        return self.frames * self.grid_h * self.grid_w

    @property
    def n_rows(self):
        return self.n_text + self.n_video


def patch_table(cfg: Config):
    return _patch_table(cfg.frames, cfg.grid_h, cfg.grid_w, cfg.patch_h, cfg.patch_w)


@lru_cache(maxsize=8)
def _patch_table(frames, H, W, ph, pw):
    """Sec. 4.3: split the f x h' x w' token grid into non-overlapping p_h x p_w
    spatial patches inside each frame (edge patches are clipped when the grid is
    not a multiple of the patch).  Returns the list of patches in patch-id order,
    each a list of video-token indices v = (t*h' + y)*w' + x in ascending order."""
    PH, PW = -(-H // ph), -(-W // pw)
    patches = []
    for t in range(frames):
        for py in range(PH):
            for px in range(PW):
                toks = []
                for y in range(py * ph, min(H, (py + 1) * ph)):
                    for x in range(px * pw, min(W, (px + 1) * pw)):
                        toks.append((t * H + y) * W + x)
                patches.append(tuple(toks))
    return tuple(patches)


# =============================================================================
# Selection S(z) (Eq. 4) with frequency-aware tracking
# =============================================================================
def mix32(x: int) -> int:
    """32-bit avalanche mixer (xor-shift / odd-multiply rounds of the published
    MurmurHash3 finaliser)."""
    x &= _M32
    x ^= x >> 16
    x = (x * 0x85EBCA6B) & _M32
    x ^= x >> 13
    x = (x * 0xC2B2AE35) & _M32
    x ^= x >> 16
    return x


def token_hash(seed: int, block: int, call: int, v: int) -> int:
    """Counter-based draw for video token v at the `call`-th selection of `block`."""
    h = mix32((seed & _M32) ^ block)
    h = mix32((h + call) & _M32)
    h = mix32((h + v) & _M32)
    return h


def patch_quotas(cfg: Config, call: int):
    """Tokens to sample from each patch: "a fixed ratio R of representative
    tokens from each patch" (Sec. 4.3).

    mode 0: running-floor split.  With S_i tokens in patches before i and a phase
    off = call * p_h * p_w, q_i = floor((S_i + #P_i + off) R) - floor((S_i + off) R):
    the quotas telescope, so their total is fixed by the host and q_i = R #P_i
    whenever that is an integer; the phase moves the leftovers round between calls.
    mode 1: q_i = round-half-up(R #P_i), at most #P_i."""
    a, b = cfg.ratio_num, cfg.ratio_den
    off = call * cfg.patch_h * cfg.patch_w
    quotas, before = [], 0
    for toks in patch_table(cfg):
        n = len(toks)
        if cfg.quota_mode == 0:
            q = ((before + n + off) * a) // b - ((before + off) * a) // b
        else:
            q = min(n, (2 * n * a + b) // (2 * b))
        quotas.append(q)
        before += n
    return quotas


def n_selected(cfg: Config, call: int) -> int:
    """Length of the index list, known on the host before the draw."""
    if cfg.quota_mode == 0:
        a, b = cfg.ratio_num, cfg.ratio_den
        off = call * cfg.patch_h * cfg.patch_w
        return ((cfg.n_video + off) * a) // b - (off * a) // b
    return sum(patch_quotas(cfg, call))


def select_tokens(cfg: Config, ages: np.ndarray, block: int, call: int):
    """S(z) = union over patches of Sample(P^i, R) (Eq. 4), where Sample favours
    tokens that have gone unsampled longer (tracking paragraph of Sec. 4.3).

    Each token draws U = (h+1) with h a 32-bit hash and competes with key
    (age+1) * U: a uniform draw on (0, age+1] up to scale, so the chance of being
    picked grows with age and is uniform when ages are equal (track_mode 0); with
    track_mode 1 the key is (age, hash): the longest-unsampled tokens always win and the
    draw only orders tokens of equal age.  The q_i largest keys of patch i win (ties:
    lower token index first).  Ages: picked -> 0, others +1
    (saturating).  Returns (sequence rows ascending, new ages)."""
    ages = np.asarray(ages)
    assert ages.shape == (cfg.n_video,)
    picked = np.zeros(cfg.n_video, dtype=bool)
    for toks, q in zip(patch_table(cfg), patch_quotas(cfg, call)):
        keyed = []
        for v in toks:
            h = token_hash(cfg.seed, block, call, v)
            if cfg.track_mode == 0:
                key = (int(ages[v]) + 1) * (h + 1)
            else:                                   # strict oldest-first: the draw only orders equal ages
                key = (int(ages[v]) << 32) | h
            keyed.append((-key, v))
        for _, v in sorted(keyed)[:q]:
            picked[v] = True
    new_ages = np.where(picked, 0, np.minimum(ages.astype(np.int64) + 1, AGE_MAX)).astype(np.uint16)
    rows = (cfg.n_text + np.nonzero(picked)[0]).astype(np.int32)
    return rows, new_ages


# =============================================================================
# Block math F (Eq. 2; scale and shift restored)
# =============================================================================
def silu(t):
    return t / (1.0 + np.exp(-t))


def gelu_tanh(t):
    return 0.5 * t * (1.0 + np.tanh(np.sqrt(2.0 / np.pi) * (t + 0.044715 * t ** 3)))


def modulation(cfg: Config, w, temb):
    """adaLN vectors from the timestep embedding: SiLU(temb) W_mod^T + b_mod, split
    into (shift1, scale1, shift2, scale2[, gate1, gate2]), each [B, D]."""
    m = silu(np.asarray(temb, F64)) @ np.asarray(w["w_mod"], F64).T + np.asarray(w["b_mod"], F64)
    return np.split(m, 6 if cfg.has_gate else 4, axis=-1)


def layernorm_modulate(cfg: Config, x, shift, scale):
    """LayerNorm over the feature axis (biased variance, no learned affine), then
    * (1 + scale) + shift.  x: [n, D]; shift, scale: [D]."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + cfg.eps) * (1.0 + scale) + shift


def qk_layernorm(cfg: Config, t, gamma, beta):
    """LayerNorm of every head's slice of t [n, D] over its head_dim features (biased
    variance, eps = qk_eps), times gamma plus beta (both [head_dim], shared by the heads).
    The base model normalises q and k this way before attention; the paper leaves the
    block's internals to the base model (Sec. 3)."""
    n = t.shape[0]
    th = t.reshape(n, cfg.n_heads, cfg.head_dim)
    mu = th.mean(axis=-1, keepdims=True)
    var = ((th - mu) ** 2).mean(axis=-1, keepdims=True)
    return ((th - mu) / np.sqrt(var + cfg.qk_eps) * gamma + beta).reshape(n, cfg.hidden)


def rope_sections(cfg: Config):
    """Number of rotary pairs given to the (frame, height, width) axes: a quarter of the
    head's pairs to time, the rest split evenly over the two spatial axes (8, 12, 12 pairs
    = 16, 24, 24 features at head_dim 64)."""
    pairs = cfg.head_dim // 2
    p_t = pairs // 4
    p_h = (pairs - p_t) // 2
    return p_t, p_h, pairs - p_t - p_h


def rope_angles(cfg: Config, rows):
    """Rotation angle of every rotary pair for sequence rows `rows`: [len(rows), head_dim/2].
    A video token at grid position (f, y, x) turns pair i of an axis' section by
    pos * theta^(-i / pairs_of_that_axis); text rows (the first n_text) are not turned."""
    rows = np.asarray(rows)
    ang = np.zeros((len(rows), cfg.head_dim // 2), F64)
    v = rows - cfg.n_text
    is_video = v >= 0
    v = np.where(is_video, v, 0)
    pos = (v // (cfg.grid_h * cfg.grid_w), (v // cfg.grid_w) % cfg.grid_h, v % cfg.grid_w)
    at = 0
    for axis, n_pairs in enumerate(rope_sections(cfg)):
        for i in range(n_pairs):
            ang[:, at + i] = pos[axis] * cfg.rope_theta ** (-i / n_pairs)
        at += n_pairs
    return ang * is_video[:, None]


def apply_rope(cfg: Config, t, rows):
    """Rotate the feature pairs (2i, 2i+1) of every head of t [len(rows), D] by rope_angles."""
    n = t.shape[0]
    ang = rope_angles(cfg, rows)[:, None, :]                      # the same for every head
    th = t.reshape(n, cfg.n_heads, cfg.head_dim // 2, 2)
    even, odd = th[..., 0], th[..., 1]
    out = np.stack([even * np.cos(ang) - odd * np.sin(ang), even * np.sin(ang) + odd * np.cos(ang)], axis=-1)
    return out.reshape(n, cfg.hidden)


def prepare_qk(cfg: Config, w, q, k, rows):
    """The base model's treatment of q and k between the QKV projection and attention:
    optional per-head LayerNorm, then optional rotary embedding by the rows' positions.
    K is cached in this final form, which stays valid because a row never moves."""
    if cfg.qk_norm:
        q = qk_layernorm(cfg, q, w["qn_w"], w["qn_b"])
        k = qk_layernorm(cfg, k, w["kn_w"], w["kn_b"])
    if cfg.rope:
        q, k = apply_rope(cfg, q, rows), apply_rope(cfg, k, rows)
    return q, k


def attention(cfg: Config, q, k_all, v_all):
    """softmax(q K^T / sqrt(head_dim)) V per head, queries [n, D] against all rows
    of K, V [N, D]; no mask.  The score matrix of one head is formed here only
    because this is the plain definition."""
    n, hd = q.shape[0], cfg.head_dim
    out = np.empty((n, cfg.hidden), F64)
    if n == 0:                 # an empty S(z): no query, nothing to attend (numpy cannot reduce an empty axis)
        return out
    for h in range(cfg.n_heads):
        sl = slice(h * hd, (h + 1) * hd)
        s = q[:, sl] @ k_all[:, sl].T / np.sqrt(hd)
        s = s - s.max(axis=-1, keepdims=True)
        p = np.exp(s)
        p = p / p.sum(axis=-1, keepdims=True)
        out[:, sl] = p @ v_all[:, sl]
    return out


# =============================================================================
# Linear extrapolation (Eq. 5)
# =============================================================================
def extrapolate(g_prev, g_last, k: int, d: int):
    """G_{t-k} = G_t + (G_t - G_{t+M}) / M * k with M = d the gap between the two
    cached full steps and k the steps since the later one."""
    g_prev, g_last = np.asarray(g_prev, F64), np.asarray(g_last, F64)
    return g_last + (g_last - g_prev) * (F64(k) / F64(d))


def extrapolate_stack(g_prev_list, g_last_list, k: int, d: int):
    """Eq. 5 applied once to the SUM of several cached features (all branches of all deep
    blocks).  Eq. 5 is linear in G and a deep block only adds its G to the residual stream
    (Sec. 4.4), so this equals the sum of the per-block extrapolations; it is written out
    separately so that the equality can be tested."""
    s_prev = sum(np.asarray(g, F64) for g in g_prev_list)
    s_last = sum(np.asarray(g, F64) for g in g_last_list)
    return extrapolate(s_prev, s_last, k, d)


# =============================================================================
# Per-block state and the three block operations of Algorithm 1
# =============================================================================
@dataclass
class BlockState:
    # shallow blocks: in-place caches of K, V and of both branch outputs G
    k_cache: np.ndarray = None
    v_cache: np.ndarray = None
    g: list = field(default_factory=lambda: [None, None])          # [attn, ffn]
    # deep blocks: two history slots per branch
    g_prev: list = field(default_factory=lambda: [None, None])
    g_last: list = field(default_factory=lambda: [None, None])
    ages: np.ndarray = None
    calls: int = 0


class HeroOracle:
    """State machine of Algorithm 1 over a stack of blocks.

    weights: list (one per block) of dicts with row-major [out, in] matrices
    w_mod, w_qkv, w_o, w_1, w_2 and biases b_*.
    """

    def __init__(self, cfg: Config, weights):
        self.cfg = cfg
        self.w = [{k: np.asarray(v, F64) for k, v in blk.items()} for blk in weights]
        assert len(self.w) == cfg.n_blocks
        assert cfg.hidden == cfg.n_heads * cfg.head_dim
        self.reset()

    def reset(self):
        c = self.cfg
        self.blocks = [BlockState(ages=np.zeros(c.n_video, np.uint16)) for _ in range(c.n_blocks)]
        self.full_steps = []          # indices of the full steps taken so far

    # ---- schedule (Algorithm 1: every M-th step is an "initial caching" step) ----
    def is_full_step(self, s: int) -> bool:
        c = self.cfg
        if s < c.warmup_full_steps:
            return True
        return c.full_interval > 0 and (s - (c.warmup_full_steps - 1)) % c.full_interval == 0

    # ---- Eq. 2 over a set of rows, with cache write-back (Eq. 3) ----
    def block_refresh(self, block: int, x, temb, rows=None, rows_out=None):
        """Refresh rows `rows` (ascending sequence rows; None = all rows = a full
        pass of Eq. 2) of both sub-layers of `block`, merge with the cache (Eq. 3)
        and add the branch outputs to the residual stream for ALL rows (Alg. 1).

        rows_out (subset of rows, default all of them) limits for which rows the
        branch outputs are recomputed; K/V are always rewritten for every row in
        `rows`, which is the only way rows influence each other.  Rows outside
        rows_out keep their cached G, so this is only for spot checks at sizes
        where the whole block is too slow on a CPU.

        x: [B, N, D] float64, updated in place and returned."""
        c, st, w = self.cfg, self.blocks[block], self.w[block]
        B, N, D = x.shape
        full = rows is None
        rows = np.arange(N) if full else np.asarray(rows)
        rows_out = rows if rows_out is None else np.asarray(rows_out)
        if st.k_cache is None:
            assert full, "the first pass of a block must be a full step"
            st.k_cache, st.v_cache = np.zeros((B, N, D), F64), np.zeros((B, N, D), F64)
            st.g = [np.zeros((B, N, D), F64), np.zeros((B, N, D), F64)]
        mod = modulation(c, w, temb)
        shift1, scale1, shift2, scale2 = mod[:4]
        gate1, gate2 = (mod[4], mod[5]) if c.has_gate else (None, None)
        for b in range(B):
            # -- attention branch --
            a = layernorm_modulate(c, x[b, rows], shift1[b], scale1[b])
            qkv = a @ w["w_qkv"].T + w["b_qkv"]
            q, k, v = qkv[:, :D], qkv[:, D:2 * D], qkv[:, 2 * D:]
            q, k = prepare_qk(c, w, q, k, rows)
            st.k_cache[b, rows] = k
            st.v_cache[b, rows] = v
            sel = np.searchsorted(rows, rows_out)
            if c.attend_mode == 1 and not full:
                # Eq. 3 read literally, F(S(z), S(tau)), with the (never refreshed) text rows kept
                seen = np.concatenate([np.arange(c.n_text), rows])
                o = attention(c, q[sel], st.k_cache[b][seen], st.v_cache[b][seen])
            else:
                o = attention(c, q[sel], st.k_cache[b], st.v_cache[b])
            g = o @ w["w_o"].T + w["b_o"]
            if c.has_gate:
                g = g * gate1[b]
            st.g[0][b, rows_out] = g                     # merge: fresh rows over cached rest
            x[b] += st.g[0][b]                           # residual add, every row
            # -- FFN branch --
            a2 = layernorm_modulate(c, x[b, rows_out], shift2[b], scale2[b])
            u = gelu_tanh(a2 @ w["w_1"].T + w["b_1"])
            g2 = u @ w["w_2"].T + w["b_2"]
            if c.has_gate:
                g2 = g2 * gate2[b]
            st.g[1][b, rows_out] = g2
            x[b] += st.g[1][b]
        if full:
            st.ages[:] = 0
            # "Initial caching": keep this step's G and the previous full step's
            # (the paper stores G_t and Delta = G_t - G_{t+M}; same information)
            for i in range(2):
                st.g_prev[i] = st.g_last[i]
                st.g_last[i] = st.g[i].copy()
        return x

    # ---- deep block on a cached step (Eq. 5 + residual add) ----
    def block_extrapolate(self, block: int, x, k: int, d: int):
        st = self.blocks[block]
        for i in range(2):
            prev = st.g_prev[i] if st.g_prev[i] is not None else st.g_last[i]   # one slot: Delta = 0
            x += extrapolate(prev, st.g_last[i], k, d)
        return x

    def deep_stack_extrapolate(self, x, k: int, d: int):
        """All deep blocks of a cached step at once: x += Eq. 5 of the summed histories."""
        deep = self.blocks[self.cfg.n_shallow:]
        last = [st.g_last[i] for st in deep for i in range(2)]
        prev = [(st.g_prev[i] if st.g_prev[i] is not None else st.g_last[i]) for st in deep for i in range(2)]
        x += extrapolate_stack(prev, last, k, d)
        return x

    # ---- selection for one shallow block ----
    def select(self, block: int):
        st = self.blocks[block]
        rows, st.ages = select_tokens(self.cfg, st.ages, block, st.calls)
        assert len(rows) == n_selected(self.cfg, st.calls)
        st.calls += 1
        return rows

    # ---- one denoising step through the block stack (Algorithm 1) ----
    def step(self, s: int, x, temb):
        c = self.cfg
        x = np.array(x, F64)
        if self.is_full_step(s):
            for l in range(c.n_blocks):
                self.block_refresh(l, x, temb, None)
            self.full_steps.append(s)
            return x
        s_last = self.full_steps[-1]
        d = s_last - self.full_steps[-2] if len(self.full_steps) > 1 else 1
        k = s - s_last
        shared = self.select(0) if (c.share_selection and c.n_shallow > 0) else None
        for l in range(c.n_blocks):
            if l < c.n_shallow:
                rows = shared if shared is not None else self.select(l)
                self.block_refresh(l, x, temb, rows)
            else:
                self.block_extrapolate(l, x, k, d)
        return x


# =============================================================================
# Diagnostics (Sec. 4.1, hierarchical feature analysis; Fig. 4)
# =============================================================================
def second_difference_variance(features):
    """Variance, over all steps and elements, of the second-order temporal differences
    F_{t+1} - 2 F_t + F_{t-1} of one layer's features.  features: [T, ...] with T >= 3."""
    f = np.asarray(features, F64)
    d2 = f[2:] - 2.0 * f[1:-1] + f[:-2]
    return float(np.mean((d2 - d2.mean()) ** 2))


def stability_scores(per_layer_features):
    """Stability score of every layer in [0, 1], higher = more stable (Sec. 4.1): the
    variances of the second-order differences are min-max normalised over the layers and
    inverted, so the layer whose features fluctuate most gets 0 and the steadiest gets 1.
    The paper states the range and the direction only; min-max over the layers is this
    reading.  All-equal variances give 1 everywhere."""
    v = np.array([second_difference_variance(f) for f in per_layer_features], F64)
    span = v.max() - v.min()
    if span == 0.0:
        return np.ones_like(v)
    return 1.0 - (v - v.min()) / span


def extrapolation_error(g_prev, g_last, g_true, k: int, d: int):
    """Relative L2 error of Eq. 5's prediction against the features actually computed k
    steps after g_last: ||extrap - g_true|| / ||g_true||."""
    e = extrapolate(np.asarray(g_prev, F64), np.asarray(g_last, F64), k, d) - np.asarray(g_true, F64)
    return float(np.sqrt((e ** 2).sum() / (np.asarray(g_true, F64) ** 2).sum()))


# =============================================================================
# The uncached step (Eq. 2 applied to every row, nothing stored)
# =============================================================================
def uncached_forward(cfg: Config, weights, x, temb):
    """Plain DiT block stack with no cache at all; written separately from
    HeroOracle so that "refresh ratio 1 with extrapolation off" can be checked
    against it."""
    x = np.array(x, F64)
    B, N, D = x.shape
    hd = cfg.head_dim
    for w in weights:
        w = {k: np.asarray(v, F64) for k, v in w.items()}
        m = silu(np.asarray(temb, F64)) @ w["w_mod"].T + w["b_mod"]
        for b in range(B):
            sh1, sc1, sh2, sc2 = (m[b, i * D:(i + 1) * D] for i in range(4))
            xb = x[b]
            xn = (xb - xb.mean(-1, keepdims=True)) / np.sqrt(xb.var(-1, keepdims=True) + cfg.eps)
            qkv = (xn * (1 + sc1) + sh1) @ w["w_qkv"].T + w["b_qkv"]
            heads = []
            for h in range(cfg.n_heads):
                qh = qkv[:, h * hd:(h + 1) * hd]
                kh = qkv[:, D + h * hd:D + (h + 1) * hd]
                vh = qkv[:, 2 * D + h * hd:2 * D + (h + 1) * hd]
                if cfg.qk_norm:
                    qh = (qh - qh.mean(-1, keepdims=True)) / np.sqrt(qh.var(-1, keepdims=True) + cfg.qk_eps) * w["qn_w"] + w["qn_b"]
                    kh = (kh - kh.mean(-1, keepdims=True)) / np.sqrt(kh.var(-1, keepdims=True) + cfg.qk_eps) * w["kn_w"] + w["kn_b"]
                if cfg.rope:
                    # pairs as complex numbers times e^{i angle}
                    turn = np.exp(1j * rope_angles(cfg, np.arange(N)))
                    qh = np.stack([((qh[:, 0::2] + 1j * qh[:, 1::2]) * turn).real,
                                   ((qh[:, 0::2] + 1j * qh[:, 1::2]) * turn).imag], -1).reshape(N, hd)
                    kh = np.stack([((kh[:, 0::2] + 1j * kh[:, 1::2]) * turn).real,
                                   ((kh[:, 0::2] + 1j * kh[:, 1::2]) * turn).imag], -1).reshape(N, hd)
                s = np.exp(qh @ kh.T / np.sqrt(hd) - (qh @ kh.T / np.sqrt(hd)).max(-1, keepdims=True))
                heads.append((s / s.sum(-1, keepdims=True)) @ vh)
            ga = np.concatenate(heads, -1) @ w["w_o"].T + w["b_o"]
            if cfg.has_gate:
                ga = ga * m[b, 4 * D:5 * D]
            xb = xb + ga
            xn = (xb - xb.mean(-1, keepdims=True)) / np.sqrt(xb.var(-1, keepdims=True) + cfg.eps)
            gf = gelu_tanh((xn * (1 + sc2) + sh2) @ w["w_1"].T + w["b_1"]) @ w["w_2"].T + w["b_2"]
            if cfg.has_gate:
                gf = gf * m[b, 5 * D:6 * D]
            x[b] = xb + gf
    return x
