"""GPU parity, tensor-core kernels (tcgen05 + TMEM + TMA) through the C ABI against the float64
oracle: the bf16 GEMM with its epilogues, flash attention over the full K/V, and whole bf16
blocks (full pass, refresh, extrapolate) with teacher-forced caches."""
import numpy as np
import pytest
import torch

from oracle import hero_oracle as O
from workloads import synthetic as S
from tests.util import make_pair, rel_l2, to_dev, to_host

pytestmark = pytest.mark.gpu

BF16_TOL = 2e-2          # rel-L2, bf16 GEMM/attention against the float64 oracle


def H():
    import paper_2508_17588_b200 as h
    return h


# ---------------------------------------------------------------- GEMM
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (1, 8, 8), (127, 264, 72), (300, 512, 256), (129, 3072, 3072),
                                   (1000, 520, 1032), (4387, 768, 128)])
@pytest.mark.parametrize("act", [0, 1])
def test_gemm_matches_oracle(M, N, K, act):
    rng = np.random.default_rng(M + N + K)
    a = S.round_bf16(rng.standard_normal((M, K)).astype(np.float32))
    w = S.round_bf16((rng.standard_normal((N, K)) * (1.0 / np.sqrt(K))).astype(np.float32))
    bias = S.round_bf16(rng.standard_normal(N).astype(np.float32) * 0.1)
    want = a.astype(np.float64) @ w.astype(np.float64).T + bias
    if act:
        want = O.gelu_tanh(want)
    c = torch.full((M, N), float("nan"), device="cuda", dtype=torch.bfloat16)
    H().hero_gemm_bf16(to_dev(a, "bf16"), to_dev(w, "bf16"), to_dev(bias, "bf16"), c, act)
    H().hero_isolated_status()
    got = to_host(c)
    assert np.isfinite(got).all()
    assert rel_l2(got, want) <= 5e-3          # one bf16 rounding of the output dominates
    # element-wise: within one bf16 ulp of the exact value plus accumulation noise
    assert np.abs(got - want).max() <= 2 ** -7 * np.abs(want).max() + 1e-3


def test_gemm_many_tiles_per_cta():
    """More tiles than SMs: every CTA walks several tiles and both TMEM accumulators."""
    M, N, K = 2500, 3072, 192
    rng = np.random.default_rng(7)
    a = S.round_bf16(rng.standard_normal((M, K)).astype(np.float32))
    w = S.round_bf16((rng.standard_normal((N, K)) / np.sqrt(K)).astype(np.float32))
    bias = np.zeros(N, np.float32)
    c = torch.empty((M, N), device="cuda", dtype=torch.bfloat16)
    H().hero_gemm_bf16(to_dev(a, "bf16"), to_dev(w, "bf16"), to_dev(bias, "bf16"), c, 0)
    H().hero_isolated_status()
    want = a.astype(np.float64) @ w.astype(np.float64).T
    assert rel_l2(to_host(c), want) <= 5e-3


# ---------------------------------------------------------------- attention
SCORE_SCALE_LOG2 = float(np.float32(0.125) * np.float32(1.4426950408889634))   # log2(e) / sqrt(64)


def fold_softmax_scale(q):
    """(what the q-scaled entry point is given, the queries that input stands for): q * log2(e)/8 rounded to
    bf16, and that product divided by the factor again in float64."""
    q_dev = S.round_bf16((q.astype(np.float64) * SCORE_SCALE_LOG2).astype(np.float32))
    return q_dev, q_dev.astype(np.float64) / SCORE_SCALE_LOG2


@pytest.mark.parametrize("B,n_q,N,heads", [(1, 128, 128, 1), (1, 1, 1, 1), (2, 37, 200, 2), (1, 130, 513, 3),
                                           (2, 300, 1000, 2), (1, 64, 2300, 1),
                                           # query counts around the 128-row tile and 256-row group edges: the
                                           # second tile of the last group is empty, one row full, or full
                                           (1, 129, 300, 2), (2, 255, 193, 1), (1, 256, 97, 2), (1, 257, 300, 1),
                                           (2, 384, 200, 1), (1, 385, 290, 2), (1, 640, 100, 1),
                                           # key counts around the 96-key tile and the 48-column split of a row between
                                           # two threads: one half empty, one key in it, exactly one tile, one key more
                                           (1, 100, 48, 1), (2, 70, 49, 2), (1, 100, 96, 1), (3, 129, 95, 1), (1, 33, 145, 1)])
@pytest.mark.parametrize("entry", ["hero_attention_bf16", "hero_attention_bf16_safe", "hero_attention_bf16_q_scaled"])
def test_attention_matches_oracle(B, n_q, N, heads, entry):
    rng = np.random.default_rng(B * 7 + n_q + N)
    D = heads * 64
    q = S.round_bf16(rng.standard_normal((B, n_q, D)).astype(np.float32))
    if entry.endswith("q_scaled"):
        q_dev, q = fold_softmax_scale(q)
    else:
        q_dev = q
    k = S.round_bf16(rng.standard_normal((B, N, D)).astype(np.float32))
    v = S.round_bf16(rng.standard_normal((B, N, D)).astype(np.float32))
    cfg = O.Config(n_blocks=1, n_shallow=1, hidden=D, n_heads=heads, head_dim=64, ffn_dim=8, temb_dim=8, batch=B,
                   frames=1, grid_h=1, grid_w=1, n_text=0, patch_h=1, patch_w=1, ratio_num=1, ratio_den=1)
    o = torch.full((B, n_q, D), float("nan"), device="cuda", dtype=torch.bfloat16)
    getattr(H(), entry)(to_dev(q_dev, "bf16"), to_dev(k, "bf16"), to_dev(v, "bf16"), o, heads)
    H().hero_isolated_status()
    got = to_host(o)
    assert np.isfinite(got).all()
    for b in range(B):
        want = O.attention(cfg, q[b].astype(np.float64), k[b].astype(np.float64), v[b].astype(np.float64))
        assert rel_l2(got[b], want) <= 1e-2, b


def test_attention_peaked_rows():
    """Large logits: a query that matches one key must return that key's value row."""
    rng = np.random.default_rng(11)
    N, D = 700, 64
    k = S.round_bf16(rng.standard_normal((1, N, D)).astype(np.float32))
    v = S.round_bf16(rng.standard_normal((1, N, D)).astype(np.float32))
    pick = np.array([0, 5, 127, 128, 400, 699])
    q = S.round_bf16(30 * k[:, pick])
    o = torch.empty((1, len(pick), D), device="cuda", dtype=torch.bfloat16)
    H().hero_attention_bf16(to_dev(q, "bf16"), to_dev(k, "bf16"), to_dev(v, "bf16"), o, 1)
    H().hero_isolated_status()
    assert np.abs(to_host(o)[0] - v[0, pick]).max() <= 2e-2


@pytest.mark.parametrize("N", [960, 1000, 97, 193])
@pytest.mark.parametrize("entry,top", [("hero_attention_bf16", 60.0), ("hero_attention_bf16_safe", 60.0),
                                       ("hero_attention_bf16", 200.0)])
def test_attention_scores_that_keep_growing(N, entry, top):
    """Keys whose scores grow steadily along the sequence (by `top` in natural-log units from the first key to
    the last).  In the safe kernel the running maximum has to move again and again (by more than the 2^8
    slack), so the accumulator is rescaled in many key tiles, on both tile parities, including the ragged
    last tile; rows with a flat score profile sit in the same warps.  The fast kernel keeps the first tile's
    maximum: a rise of 60 stays inside its 2^100 range and is computed there, a rise of 200 is not, so the
    climbing rows' thread blocks are handed to the safe kernel and the flat and descending ones are not."""
    rng = np.random.default_rng(N)
    n_q, D = 200, 64
    base = rng.standard_normal(D).astype(np.float32)
    base /= np.linalg.norm(base)
    ramp = np.linspace(0.0, top, N, dtype=np.float32)[:, None]                     # score ~ 8 * ramp * |q.base|
    k = S.round_bf16((rng.standard_normal((1, N, D)) * 0.3 + ramp * base).astype(np.float32))
    v = S.round_bf16(rng.standard_normal((1, N, D)).astype(np.float32))
    q = rng.standard_normal((1, n_q, D)).astype(np.float32) * 0.3
    q[:, ::2] += 8.0 * base                                                        # every other row climbs the ramp
    q[:, 1::4] -= 8.0 * base                                                       # some descend it
    q = S.round_bf16(q)
    cfg = O.Config(n_blocks=1, n_shallow=1, hidden=D, n_heads=1, head_dim=64, ffn_dim=8, temb_dim=8, batch=1,
                   frames=1, grid_h=1, grid_w=1, n_text=0, patch_h=1, patch_w=1, ratio_num=1, ratio_den=1)
    o = torch.full((1, n_q, D), float("nan"), device="cuda", dtype=torch.bfloat16)
    getattr(H(), entry)(to_dev(q, "bf16"), to_dev(k, "bf16"), to_dev(v, "bf16"), o, 1)
    H().hero_isolated_status()
    got = to_host(o)[0]
    assert np.isfinite(got).all()
    want = O.attention(cfg, q[0].astype(np.float64), k[0].astype(np.float64), v[0].astype(np.float64))
    assert rel_l2(got, want) <= 1e-2
    assert np.abs(got - want).max() <= 3e-2 * np.abs(want).max()


def test_attention_one_row_out_of_range_sends_only_its_thread_block_to_the_fallback():
    """Three thread blocks of queries; one row of the middle one meets a key, late in the sequence, whose score
    beats everything in the first key tile by far more than 2^100.  The result must be right everywhere: that
    block through the fallback kernel, the other two straight from the fast one."""
    rng = np.random.default_rng(77)
    n_q, N, D = 700, 1500, 64
    q = rng.standard_normal((1, n_q, D)).astype(np.float32)
    k = rng.standard_normal((1, N, D)).astype(np.float32)
    v = rng.standard_normal((1, N, D)).astype(np.float32)
    k[0, 1234] = 16.0 * q[0, 300] / np.linalg.norm(q[0, 300])     # |k| = 16, along q
    q[0, 300] *= 16.0 / np.linalg.norm(q[0, 300])                  # |q| = 16: q.k / 8 = 32 here, a few units elsewhere
    q[0, 300] *= 8.0                                               # ... and 256 after this
    q, k, v = S.round_bf16(q), S.round_bf16(k), S.round_bf16(v)
    cfg = O.Config(n_blocks=1, n_shallow=1, hidden=D, n_heads=1, head_dim=64, ffn_dim=8, temb_dim=8, batch=1,
                   frames=1, grid_h=1, grid_w=1, n_text=0, patch_h=1, patch_w=1, ratio_num=1, ratio_den=1)
    s300 = (q[0, 300].astype(np.float64) @ k[0].astype(np.float64).T) / 8.0
    assert s300[1234] - s300[:96].max() > 150.0                    # far beyond the fast kernel's range
    o = torch.full((1, n_q, D), float("nan"), device="cuda", dtype=torch.bfloat16)
    H().hero_attention_bf16(to_dev(q, "bf16"), to_dev(k, "bf16"), to_dev(v, "bf16"), o, 1)
    H().hero_isolated_status()
    got = to_host(o)[0]
    assert np.isfinite(got).all()
    want = O.attention(cfg, q[0].astype(np.float64), k[0].astype(np.float64), v[0].astype(np.float64))
    for lo in (0, 256, 512):
        assert rel_l2(got[lo:lo + 256], want[lo:lo + 256]) <= 1e-2, lo
    assert np.abs(got[300] - v[0, 1234]).max() <= 2e-2             # that row returns the one key's value


@pytest.mark.parametrize("entry", ["hero_attention_bf16", "hero_attention_bf16_q_scaled"])
def test_fallback_serves_marked_thread_blocks_scattered_over_a_large_grid(entry):
    """310 thread blocks of queries, more than two waves on the GPU's SMs; six of them, spread over the grid
    (three of them 148 apart), hold one row that meets a key in the second key tile outscoring the rest by far
    more than either fast kernel's range.  Exactly those blocks are recomputed by the fallback kernel; all 310
    must match the oracle."""
    rng = np.random.default_rng(91)
    n_blocks, N, D = 310, 200, 64
    n_q = n_blocks * 256
    q = rng.standard_normal((1, n_q, D)).astype(np.float32)
    k = rng.standard_normal((1, N, D)).astype(np.float32)
    v = rng.standard_normal((1, N, D)).astype(np.float32)
    u = k[0, 150] / np.linalg.norm(k[0, 150])
    k[0, 150] = 16.0 * u
    marked = [5, 7, 5 + 148, 200, 5 + 296, 309]
    rows = [256 * c + 17 * (i + 1) for i, c in enumerate(marked)]
    for r in rows:
        q[0, r] = 128.0 * u                                        # q.k / 8 = 256 at key 150
    q, k, v = S.round_bf16(q), S.round_bf16(k), S.round_bf16(v)
    if entry.endswith("q_scaled"):
        q_dev, q_eff = fold_softmax_scale(q)
    else:
        q_dev, q_eff = q, q.astype(np.float64)
    cfg = O.Config(n_blocks=1, n_shallow=1, hidden=D, n_heads=1, head_dim=64, ffn_dim=8, temb_dim=8, batch=1,
                   frames=1, grid_h=1, grid_w=1, n_text=0, patch_h=1, patch_w=1, ratio_num=1, ratio_den=1)
    o = torch.full((1, n_q, D), float("nan"), device="cuda", dtype=torch.bfloat16)
    getattr(H(), entry)(to_dev(q_dev, "bf16"), to_dev(k, "bf16"), to_dev(v, "bf16"), o, 1)
    H().hero_isolated_status()
    got = to_host(o)[0]
    assert np.isfinite(got).all()
    want = O.attention(cfg, q_eff[0], k[0].astype(np.float64), v[0].astype(np.float64))
    err = np.array([rel_l2(got[256 * c:256 * (c + 1)], want[256 * c:256 * (c + 1)]) for c in range(n_blocks)])
    assert err.max() <= 1e-2, (int(err.argmax()), float(err.max()))
    for r in rows:
        assert np.abs(got[r] - v[0, 150]).max() <= 2e-2, r


def test_q_scaled_attention_rows_outside_its_range_go_to_the_fallback():
    """The q-scaled entry point takes 2^score with no row maximum, which holds while a row's largest score stays
    within about +-100 (base-2 units).  Three thread blocks of queries: in the first every row is ordinary, in
    the second one row's best key scores about +190, in the third one row's scores all lie near -220 (its sum of
    weights underflows).  Both are recognised by their row sum and recomputed by the second kernel; every row of
    every block must come out right."""
    rng = np.random.default_rng(78)
    n_q, N, D = 700, 1500, 64
    q = rng.standard_normal((1, n_q, D)).astype(np.float32)
    k = rng.standard_normal((1, N, D)).astype(np.float32)
    v = rng.standard_normal((1, N, D)).astype(np.float32)
    base = rng.standard_normal(D).astype(np.float32)
    base /= np.linalg.norm(base)
    u = q[0, 300] / np.linalg.norm(q[0, 300])
    k[0, 1234] = 16.0 * u
    k[0] += 12.0 * base                                             # every key has a common component
    q[0, 300] = 64.0 * u                                            # q.k / 8 = 128 (natural units) at key 1234
    q[0, 600] = -110.0 * base                                       # q.k / 8 ~ -150 for every key
    q, k, v = S.round_bf16(q), S.round_bf16(k), S.round_bf16(v)
    q_dev, q_eff = fold_softmax_scale(q)
    s_log2 = np.einsum("qd,kd->qk", q_dev[0].astype(np.float64), k[0].astype(np.float64))
    assert s_log2[300].max() > 150.0 and s_log2[600].max() < -150.0
    others = np.delete(np.arange(n_q), [300, 600])
    assert np.abs(s_log2[others]).max() < 60.0
    cfg = O.Config(n_blocks=1, n_shallow=1, hidden=D, n_heads=1, head_dim=64, ffn_dim=8, temb_dim=8, batch=1,
                   frames=1, grid_h=1, grid_w=1, n_text=0, patch_h=1, patch_w=1, ratio_num=1, ratio_den=1)
    o = torch.full((1, n_q, D), float("nan"), device="cuda", dtype=torch.bfloat16)
    H().hero_attention_bf16_q_scaled(to_dev(q_dev, "bf16"), to_dev(k, "bf16"), to_dev(v, "bf16"), o, 1)
    H().hero_isolated_status()
    got = to_host(o)[0]
    assert np.isfinite(got).all()
    want = O.attention(cfg, q_eff[0], k[0].astype(np.float64), v[0].astype(np.float64))
    for lo in (0, 256, 512):
        assert rel_l2(got[lo:lo + 256], want[lo:lo + 256]) <= 1e-2, lo
    assert np.abs(got[300] - v[0, 1234]).max() <= 2e-2
    assert np.abs(got[600] - want[600]).max() <= 3e-2 * np.abs(want[600]).max()


def test_q_scaled_attention_on_both_sides_of_its_range():
    """Eight thread blocks of queries, each with its own level of scores: row maxima near +70, +90, +105, +120
    and near -70, -88, -105, -118 (base-2 units; all keys of a row score between half the level and the level).
    Levels inside +-100 are computed by the fast kernel as 2^score, the others are caught by their row sums
    (beyond 2^100, below 2^-100) and recomputed by the second kernel; every block must match the oracle."""
    rng = np.random.default_rng(5)
    N, D = 300, 64
    levels = [70.0, 90.0, 105.0, 120.0, -140.0, -180.0, -215.0, -240.0]      # alpha; maximum = alpha or alpha / 2
    base = rng.standard_normal(D)
    base /= np.linalg.norm(base)
    beta = rng.uniform(0.5, 1.0, N)
    beta[rng.integers(N)] = 1.0
    k = S.round_bf16((beta[:, None] * base + 0.01 * rng.standard_normal((N, D)))[None].astype(np.float32))
    v = S.round_bf16(rng.standard_normal((1, N, D)).astype(np.float32))
    alpha = np.concatenate([lv + rng.uniform(-2.0, 2.0, 256) for lv in levels])
    q_dev = S.round_bf16((alpha[:, None] * base)[None].astype(np.float32))   # already in exponent units
    q_eff = q_dev.astype(np.float64) / SCORE_SCALE_LOG2
    s_log2 = q_dev[0].astype(np.float64) @ k[0].astype(np.float64).T
    top = s_log2.max(axis=1).reshape(len(levels), 256)
    for c, want_top in enumerate([70, 90, 105, 120, -70, -88, -105, -118]):
        assert np.abs(top[c] - want_top).max() < 5.0, (c, top[c].min(), top[c].max())
    cfg = O.Config(n_blocks=1, n_shallow=1, hidden=D, n_heads=1, head_dim=64, ffn_dim=8, temb_dim=8, batch=1,
                   frames=1, grid_h=1, grid_w=1, n_text=0, patch_h=1, patch_w=1, ratio_num=1, ratio_den=1)
    o = torch.full((1, alpha.size, D), float("nan"), device="cuda", dtype=torch.bfloat16)
    H().hero_attention_bf16_q_scaled(to_dev(q_dev, "bf16"), to_dev(k, "bf16"), to_dev(v, "bf16"), o, 1)
    H().hero_isolated_status()
    got = to_host(o)[0]
    assert np.isfinite(got).all()
    want = O.attention(cfg, q_eff[0], k[0].astype(np.float64), v[0].astype(np.float64))
    for c in range(len(levels)):
        sl = slice(256 * c, 256 * (c + 1))
        assert rel_l2(got[sl], want[sl]) <= 1e-2, (c, rel_l2(got[sl], want[sl]))


# ---------------------------------------------------------------- bf16 blocks
SMALL_BF16 = dict(n_blocks=2, n_shallow=1, hidden=256, n_heads=4, head_dim=64, ffn_dim=768, temb_dim=64, batch=2,
                  frames=3, grid_h=9, grid_w=11, n_text=10, patch_h=2, patch_w=2, ratio_num=1, ratio_den=4,
                  quota_mode=0, warmup_full_steps=2, full_interval=3, dtype="bf16", has_gate=0, seed=21, steps=6)


@pytest.mark.parametrize("gate,attend_mode,qk,batch", [(0, 0, 0, 2), (1, 0, 0, 2), (0, 1, 0, 2), (1, 1, 0, 2), (0, 0, 1, 2),
                                                       (1, 1, 1, 2), (0, 0, 0, 1), (1, 0, 1, 3), (0, 1, 0, 5)])
def test_bf16_small_model_steps_teacher_forced(gate, attend_mode, qk, batch):
    """Full, refresh and extrapolate blocks in bf16 over 6 steps (full at 0, 1, 4).  Each step both
    sides start from the same input; the oracle's caches are overwritten with the GPU's
    bf16 caches after every step (teacher forcing) so the per-step error is what is graded.
    attend_mode 1 restricts the keys of a cached step to the refreshed and text rows; qk = 1 turns on the
    per-head LayerNorm and the rotary embedding of q and k; batch sizes 1, 3 and 5 beside the workloads' 2."""
    _bf16_steps_teacher_forced(dict(SMALL_BF16, has_gate=gate, attend_mode=attend_mode, qk_norm=qk, rope=qk, batch=batch))


@pytest.mark.parametrize("over", [
    dict(n_text=0),                                                    # no text rows at all
    dict(n_text=0, attend_mode=1),                                     # ... and the refreshed rows as the only keys
    dict(patch_h=2, patch_w=3, quota_mode=1, ratio_num=1, ratio_den=5, full_interval=2),   # the paper's selection
    dict(patch_h=1, patch_w=1, ratio_num=1, ratio_den=3),              # one-token patches: quota 0 or 1 per patch
    dict(frames=1, grid_h=23, grid_w=13, n_text=1, ratio_num=1, ratio_den=2),              # one frame, odd grid
    dict(ratio_num=1, ratio_den=1),                                    # every token refreshed in cached steps
], ids=["no_text", "no_text_literal_eq3", "paper_selection", "unit_patches", "one_frame_odd_grid", "ratio_one"])
def test_bf16_small_model_steps_other_geometries(over):
    """The same graded quantities on other token geometries and selection settings."""
    _bf16_steps_teacher_forced(dict(SMALL_BF16, **over))


def _bf16_steps_teacher_forced(cfgd):
    gate = cfgd.get("has_gate", 0)
    weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    for w in weights:        # larger modulation so that scale/shift/gate matter
        w["w_mod"] = S.round_bf16(w["w_mod"] * 10)
        w["b_mod"] = S.round_bf16(w["b_mod"] + (1.0 if gate else 0.0))
    orc, hero, _ = make_pair(cfgd, weights)
    x_host = S.tokens(cfgd)
    for s in range(cfgd["steps"]):
        temb = S.temb(cfgd, s)
        want = orc.step(s, x_host, temb)
        x = to_dev(x_host, "bf16")
        hero.hero_step(s, x, to_dev(temb, "bf16"))
        hero.hero_check_status()
        err = rel_l2(to_host(x), want)
        assert err <= BF16_TOL, (s, err)
        assert np.array_equal(hero.hero_state_get(0, "ages").numpy(), orc.blocks[0].ages)
        st = orc.blocks[0]
        for name, ref in (("k", st.k_cache), ("v", st.v_cache), ("g_attn", st.g[0]), ("g_ffn", st.g[1])):
            got = to_host(hero.hero_state_get(0, name))
            assert rel_l2(got, ref) <= BF16_TOL, (s, name)
            ref[...] = got                                   # teacher forcing
        dp = orc.blocks[1]
        for i, name in enumerate(("g_attn", "g_ffn")):
            got = to_host(hero.hero_state_get(1, name))
            assert rel_l2(got, dp.g_last[i]) <= BF16_TOL, (s, name)
            dp.g_last[i][...] = got
            if dp.g_prev[i] is not None:
                gp = to_host(hero.hero_state_get(1, name + "_prev"))
                assert rel_l2(gp, dp.g_prev[i]) <= BF16_TOL
                dp.g_prev[i][...] = gp
    hero.close()


def test_bf16_host_entry_point_matches_device_entry_point():
    """hero_step_host copies x back piece by piece behind the deep blocks of a cached step; the result must be
    the device entry point's, bit for bit, on full and cached steps (the last piece is ragged here)."""
    cfgd = dict(SMALL_BF16, n_blocks=4, n_shallow=2)
    weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    _, hero_a, _ = make_pair(cfgd, weights)
    _, hero_b, _ = make_pair(cfgd, weights)
    x0 = to_dev(S.tokens(cfgd), "bf16")
    for s in range(cfgd["steps"]):
        temb = to_dev(S.temb(cfgd, s), "bf16")
        xd = x0.clone()
        hero_a.hero_step(s, xd, temb)
        xh = x0.cpu().pin_memory()
        hero_b.hero_step_host(s, xh, temb.cpu().pin_memory())
        assert torch.equal(xd.cpu(), xh), s
    hero_a.hero_check_status(); hero_b.hero_check_status()
    hero_a.close(); hero_b.close()


def test_bf16_refresh_keeps_unselected_rows_bit_identical():
    cfgd = dict(SMALL_BF16, n_blocks=1, n_shallow=1)
    _, hero, _ = make_pair(cfgd)
    cfg = O.Config.from_dict(cfgd)
    x = to_dev(S.tokens(cfgd), "bf16")
    hero.hero_refresh_block(0, x, to_dev(S.temb(cfgd, 0), "bf16"))
    before = {n: hero.hero_state_get(0, n).clone() for n in ("k", "v", "g_attn", "g_ffn")}
    idx = torch.empty(cfg.n_video, dtype=torch.int32, device="cuda")
    n = hero.hero_select_tokens(0, idx)
    rows = idx[:n].cpu().numpy()
    keep = np.setdiff1d(np.arange(cfg.n_rows), rows)
    hero.hero_refresh_block(0, x, to_dev(S.temb(cfgd, 1), "bf16"), idx[:n])
    hero.hero_check_status()
    for name, b4 in before.items():
        after = hero.hero_state_get(0, name)
        assert torch.equal(after[:, keep], b4[:, keep]), name
        assert not torch.equal(after[:, rows], b4[:, rows]), name
    hero.close()


def test_free_running_drift_over_the_42_block_50_step_schedule_in_miniature(capsys):
    """No teacher forcing: a 42-block model (14 refresh + 28 extrapolated, full step every 5, 50 steps) at
    a small width runs freely on both sides, bf16 caches on the GPU against float64 in the oracle, and the
    per-step distance of the outputs is reported.  Selection is integer work, so lists and ages stay
    bit-identical however far the values drift.  Only a loose bound is asserted: the number is a report."""
    cfgd = dict(SMALL_BF16, n_blocks=42, n_shallow=14, full_interval=5, steps=50, seed=31)
    weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    orc, hero, _ = make_pair(cfgd, weights)
    x_host = S.tokens(cfgd)
    errs = []
    for s in range(cfgd["steps"]):
        temb = S.temb(cfgd, s)
        want = orc.step(s, x_host, temb)
        x = to_dev(x_host, "bf16")
        hero.hero_step(s, x, to_dev(temb, "bf16"))
        errs.append(rel_l2(to_host(x), want))
        for l in (0, 13):
            assert np.array_equal(hero.hero_state_get(l, "ages").numpy(), orc.blocks[l].ages), (s, l)
    hero.hero_check_status()
    hero.close()
    full = [e for s, e in enumerate(errs) if orc.is_full_step(s)]
    cached = [e for s, e in enumerate(errs) if not orc.is_full_step(s)]
    with capsys.disabled():
        print(f"\nfree-running drift, 42 blocks x 50 steps (bf16 vs float64): full steps max {max(full):.2e}, "
              f"cached steps max {max(cached):.2e}, last step {errs[-1]:.2e}")
    assert np.isfinite(errs).all() and max(errs) <= 5e-2
