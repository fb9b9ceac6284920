"""Pins for the oracle's block math (Eq. 2 with scale/shift), the cache merge (Eq. 3),
linear extrapolation (Eq. 5) and the step schedule (Algorithm 1).  CPU only.

The block's pieces reduce to library routines (layer_norm, scaled-dot-product
attention, GELU-tanh, SiLU, linear); each is checked against torch's float64
implementation, and the cached step is checked against the uncached forward in the
case where the paper says they coincide (refresh ratio 1, no extrapolation)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as TF

from oracle import hero_oracle as O
from workloads import synthetic as S


def small_cfg(**kw):
    base = dict(n_blocks=2, n_shallow=2, hidden=32, n_heads=2, head_dim=16, ffn_dim=64, temb_dim=12,
                batch=2, frames=2, grid_h=4, grid_w=5, n_text=3, patch_h=2, patch_w=2,
                ratio_num=1, ratio_den=4, quota_mode=0, seed=11, warmup_full_steps=2, full_interval=0)
    base.update(kw)
    return O.Config(**base)


def rand_weights(cfg, scale=0.2, seed=0):
    rng = np.random.default_rng(seed)
    d = dict(cfg.__dict__, dtype="fp32")
    return [{k: rng.standard_normal(shp) * scale + (1.0 if k in ("qn_w", "kn_w") else 0.0)
             for k, shp in S.weight_shapes(d).items()} for _ in range(cfg.n_blocks)]


def t64(a):
    return torch.from_numpy(np.asarray(a, np.float64))


# ---------------------------------------------------------------- elementary routines
def test_layernorm_modulate_vs_torch():
    cfg = small_cfg()
    rng = np.random.default_rng(0)
    x, sh, sc = rng.standard_normal((7, 32)) * 3 + 1, rng.standard_normal(32), rng.standard_normal(32)
    want = TF.layer_norm(t64(x), (32,), eps=1e-5) * (1 + t64(sc)) + t64(sh)
    np.testing.assert_allclose(O.layernorm_modulate(cfg, x, sh, sc), want.numpy(), rtol=1e-12, atol=1e-12)


def test_gelu_and_silu_vs_torch():
    t = np.linspace(-6, 6, 1001)
    np.testing.assert_allclose(O.gelu_tanh(t), TF.gelu(t64(t), approximate="tanh").numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(O.silu(t), TF.silu(t64(t)).numpy(), rtol=1e-12, atol=1e-13)


def test_attention_vs_torch_sdpa_and_rows_sum_to_one():
    cfg = small_cfg(hidden=48, n_heads=3, head_dim=16)
    rng = np.random.default_rng(1)
    n, N = 5, 23
    q, k, v = rng.standard_normal((n, 48)), rng.standard_normal((N, 48)), rng.standard_normal((N, 48))
    got = O.attention(cfg, q, k, v)
    th = lambda a, m: t64(a).reshape(m, 3, 16).transpose(0, 1)      # [heads, m, hd]
    want = TF.scaled_dot_product_attention(th(q, n), th(k, N), th(v, N)).transpose(0, 1).reshape(n, 48)
    np.testing.assert_allclose(got, want.numpy(), rtol=1e-11, atol=1e-12)
    # with V = all ones the output is exactly the sum of the probabilities
    np.testing.assert_allclose(O.attention(cfg, q, k, np.ones_like(v)), 1.0, rtol=1e-12)
    # a query is dominated by the key it matches when scaled up
    big = O.attention(cfg, 200 * k[[4]], k, v)
    assert np.abs(big - v[4]).max() < 1e-6


def test_modulation_split_order():
    cfg = small_cfg(has_gate=1)
    w = rand_weights(cfg)[0]
    temb = np.random.default_rng(2).standard_normal((2, 12))
    m = (TF.silu(t64(temb)) @ t64(w["w_mod"]).T + t64(w["b_mod"])).numpy()
    parts = O.modulation(cfg, w, temb)
    assert len(parts) == 6
    for i, p in enumerate(parts):                  # shift1, scale1, shift2, scale2, gate1, gate2
        np.testing.assert_allclose(p, m[:, i * 32:(i + 1) * 32], rtol=1e-12)


# ---------------------------------------------------------------- the whole block vs a torch block
def torch_block(cfg, w, x, temb):
    D, hd, nh = cfg.hidden, cfg.head_dim, cfg.n_heads
    w = {k: t64(v) for k, v in w.items()}
    x, temb = t64(x), t64(temb)
    m = TF.linear(TF.silu(temb), w["w_mod"], w["b_mod"])
    ch = m.chunk(6 if cfg.has_gate else 4, dim=-1)
    B, N, _ = x.shape
    a = TF.layer_norm(x, (D,), eps=cfg.eps) * (1 + ch[1][:, None]) + ch[0][:, None]
    q, k, v = TF.linear(a, w["w_qkv"], w["b_qkv"]).chunk(3, dim=-1)
    sp = lambda t: t.reshape(B, N, nh, hd).transpose(1, 2)
    o = TF.scaled_dot_product_attention(sp(q), sp(k), sp(v)).transpose(1, 2).reshape(B, N, D)
    g = TF.linear(o, w["w_o"], w["b_o"])
    if cfg.has_gate:
        g = g * ch[4][:, None]
    x = x + g
    a = TF.layer_norm(x, (D,), eps=cfg.eps) * (1 + ch[3][:, None]) + ch[2][:, None]
    g2 = TF.linear(TF.gelu(TF.linear(a, w["w_1"], w["b_1"]), approximate="tanh"), w["w_2"], w["b_2"])
    if cfg.has_gate:
        g2 = g2 * ch[5][:, None]
    return (x + g2).numpy(), g.numpy(), g2.numpy(), k.numpy(), v.numpy()


@pytest.mark.parametrize("gate", [0, 1])
def test_full_block_vs_torch_library_block(gate):
    cfg = small_cfg(n_blocks=1, n_shallow=1, has_gate=gate)
    w = rand_weights(cfg, seed=3)
    rng = np.random.default_rng(4)
    x, temb = rng.standard_normal((2, cfg.n_rows, 32)), rng.standard_normal((2, 12))
    orc = O.HeroOracle(cfg, w)
    got = orc.block_refresh(0, x.copy(), temb, None)
    want, g, g2, k, v = torch_block(cfg, w[0], x, temb)
    np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-11)
    st = orc.blocks[0]
    np.testing.assert_allclose(st.g[0], g, rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(st.g[1], g2, rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(st.k_cache, k, rtol=1e-10, atol=1e-11)
    np.testing.assert_allclose(st.v_cache, v, rtol=1e-10, atol=1e-11)


# ---------------------------------------------------------------- q/k LayerNorm and rotary embedding
def test_qk_layernorm_vs_torch_layer_norm_per_head():
    cfg = small_cfg(qk_norm=1)
    rng = np.random.default_rng(30)
    t = rng.standard_normal((7, cfg.hidden)) * 3 + 1
    gamma, beta = rng.standard_normal(cfg.head_dim), rng.standard_normal(cfg.head_dim)
    got = O.qk_layernorm(cfg, t, gamma, beta)
    want = TF.layer_norm(t64(t).reshape(7, cfg.n_heads, cfg.head_dim), (cfg.head_dim,), t64(gamma), t64(beta),
                         eps=1e-6).reshape(7, cfg.hidden).numpy()
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)


def test_rope_fixed_points_known_angles_and_shift_invariance():
    cfg = small_cfg(rope=1, head_dim=16, n_heads=2, frames=4, grid_h=6, grid_w=8)     # 8 pairs: 2 + 3 + 3
    assert O.rope_sections(cfg) == (2, 3, 3)
    assert O.rope_sections(small_cfg(head_dim=64, hidden=128)) == (8, 12, 12)          # 16 + 24 + 24 features
    row = lambda f, y, x: cfg.n_text + (f * cfg.grid_h + y) * cfg.grid_w + x
    rng = np.random.default_rng(31)
    t = rng.standard_normal((4, cfg.hidden))
    rows = np.array([1, row(0, 0, 0), row(2, 3, 4), row(3, 5, 7)])
    got = O.apply_rope(cfg, t, rows)
    assert np.array_equal(got[0], t[0])                         # a text row is not turned
    np.testing.assert_allclose(got[1], t[1], atol=1e-15)        # nor is the video token at the origin
    pairs = lambda a: a.reshape(-1, cfg.n_heads, 8, 2)
    np.testing.assert_allclose(np.linalg.norm(pairs(got), axis=-1), np.linalg.norm(pairs(t), axis=-1), rtol=1e-12)
    # unit vectors along the even feature of a pair come out as (cos, sin) of that pair's angle
    e = np.zeros((1, cfg.hidden)); e[0, 0::2] = 1.0
    turned = pairs(O.apply_rope(cfg, e, np.array([row(2, 3, 4)])))[0]
    want_angle = np.array([2.0, 2.0 * 10000 ** (-1 / 2),                          # frame axis, 2 pairs
                           3.0, 3.0 * 10000 ** (-1 / 3), 3.0 * 10000 ** (-2 / 3),  # grid row, 3 pairs
                           4.0, 4.0 * 10000 ** (-1 / 3), 4.0 * 10000 ** (-2 / 3)])
    for h in range(cfg.n_heads):
        np.testing.assert_allclose(turned[h, :, 0], np.cos(want_angle), rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(turned[h, :, 1], np.sin(want_angle), rtol=1e-12, atol=1e-15)
    # scores depend on the displacement between query and key, not on where the pair sits
    q, k = rng.standard_normal((1, cfg.hidden)), rng.standard_normal((1, cfg.hidden))
    dot = lambda a, b: (O.apply_rope(cfg, q, np.array([a])) @ O.apply_rope(cfg, k, np.array([b])).T).item()
    base = dot(row(1, 2, 3), row(0, 1, 5))
    assert abs(dot(row(3, 4, 4), row(2, 3, 6)) - base) < 1e-12
    assert abs(dot(row(1, 2, 3), row(0, 1, 6)) - base) > 1e-3


def test_rope_angles_closed_forms():
    """What fixes the rotary angles without typing their formula again: every axis' first pair turns by
    exactly `position` radians; angles are linear in the position; inside an axis the frequencies form a
    geometric sequence whose ratio, taken to the power of the axis' pair count, is 1 / 10000; an axis' pairs
    move with that axis' coordinate and no other; text rows have no angle.  A wrong split, base, index or
    axis order fails one of these."""
    cfg = small_cfg(rope=1, head_dim=64, n_heads=1, hidden=64, frames=5, grid_h=7, grid_w=9, n_text=4)
    p_t, p_h, p_w = O.rope_sections(cfg)
    assert (p_t, p_h, p_w) == (8, 12, 12) and p_t + p_h + p_w == cfg.head_dim // 2
    row = lambda f, y, x: cfg.n_text + (f * cfg.grid_h + y) * cfg.grid_w + x
    ang = lambda f, y, x: O.rope_angles(cfg, [row(f, y, x)])[0]
    first = {0: 0, 1: p_t, 2: p_t + p_h}                        # first pair of each axis' section
    a = ang(3, 5, 7)
    assert a[first[0]] == 3.0 and a[first[1]] == 5.0 and a[first[2]] == 7.0
    np.testing.assert_allclose(ang(4, 6, 8), 2.0 * ang(2, 3, 4), rtol=1e-14)              # linear in the position
    np.testing.assert_allclose(ang(1, 2, 3) + ang(3, 4, 5), ang(4, 6, 8), rtol=1e-14)
    one = ang(1, 1, 1)                                           # the frequencies themselves
    for start, n in ((0, p_t), (p_t, p_h), (p_t + p_h, p_w)):
        freq = one[start:start + n]
        ratio = freq[1:] / freq[:-1]
        np.testing.assert_allclose(ratio, ratio[0], rtol=1e-13)                           # geometric
        assert 0.0 < ratio[0] < 1.0                                                       # falling with the pair index
        np.testing.assert_allclose(ratio[0] ** n, 1.0e-4, rtol=1e-12)                     # n steps span the base
    base = ang(2, 3, 4)
    moved = [ang(3, 3, 4) != base, ang(2, 4, 4) != base, ang(2, 3, 5) != base]
    sections = [slice(0, p_t), slice(p_t, p_t + p_h), slice(p_t + p_h, None)]
    for axis in range(3):                                        # an axis' coordinate moves its own section only
        for sec in range(3):
            assert moved[axis][sections[sec]].all() == (axis == sec) and moved[axis][sections[sec]].any() == (axis == sec)
    assert not O.rope_angles(cfg, np.arange(cfg.n_text)).any()   # text rows


@pytest.mark.parametrize("extras", [dict(), dict(qk_norm=1, rope=1)])
def test_ratio_one_without_extrapolation_equals_uncached_step(extras):
    """R = 1 makes S(z) = z; with text rows included and every block shallow, a cached
    step is Eq. 2 on all rows, i.e. the uncached forward, on every step.  With q/k LayerNorm and
    rotary embedding on, the uncached forward normalises with numpy's var and turns the pairs as
    complex numbers, the block path by the plain real formulas."""
    cfg = small_cfg(n_blocks=3, n_shallow=3, ratio_num=1, ratio_den=1, **extras)
    w = rand_weights(cfg, seed=5)
    rng = np.random.default_rng(6)
    orc = O.HeroOracle(cfg, w)
    for s in range(4):
        x, temb = rng.standard_normal((2, cfg.n_rows, 32)), rng.standard_normal((2, 12))
        want = O.uncached_forward(cfg, w, x, temb)
        if orc.is_full_step(s):
            got = orc.step(s, x, temb)
        else:       # refresh every row (text included) through the refresh path
            got = np.array(x)
            for l in range(cfg.n_blocks):
                vid = orc.select(l)
                assert len(vid) == cfg.n_video
                orc.block_refresh(l, got, temb, np.arange(cfg.n_rows))
        np.testing.assert_allclose(got, want, rtol=1e-10, atol=1e-11)


def test_uncached_forward_vs_torch_block_stack():
    cfg = small_cfg(n_blocks=2, n_shallow=2)
    w = rand_weights(cfg, seed=8)
    rng = np.random.default_rng(9)
    x, temb = rng.standard_normal((2, cfg.n_rows, 32)), rng.standard_normal((2, 12))
    want = x
    for blk in w:
        want = torch_block(cfg, blk, want, temb)[0]
    np.testing.assert_allclose(O.uncached_forward(cfg, w, x, temb), want, rtol=1e-10, atol=1e-11)


# ---------------------------------------------------------------- merge (Eq. 3)
def test_refresh_touches_only_selected_rows_and_reads_the_full_kv_cache():
    cfg = small_cfg(n_blocks=1, n_shallow=1)
    w = rand_weights(cfg, seed=10)
    rng = np.random.default_rng(12)
    x0, temb0 = rng.standard_normal((2, cfg.n_rows, 32)), rng.standard_normal((2, 12))
    orc = O.HeroOracle(cfg, w)
    orc.block_refresh(0, x0.copy(), temb0, None)
    st = orc.blocks[0]
    before = [st.k_cache.copy(), st.v_cache.copy(), st.g[0].copy(), st.g[1].copy()]
    x1, temb1 = rng.standard_normal((2, cfg.n_rows, 32)), rng.standard_normal((2, 12))
    rows = orc.select(0)
    keep = np.setdiff1d(np.arange(cfg.n_rows), rows)
    x_in = x1.copy()
    out = orc.block_refresh(0, x1, temb1, rows)
    after = [st.k_cache, st.v_cache, st.g[0], st.g[1]]
    for b4, af in zip(before, after):
        assert np.array_equal(b4[:, keep], af[:, keep])            # bit-identical reuse
        assert not np.array_equal(b4[:, rows], af[:, rows])
    # residual: every row received both cached-or-fresh branch outputs
    np.testing.assert_allclose(out, x_in + st.g[0] + st.g[1], rtol=1e-12, atol=1e-12)
    # selected rows: recompute by hand against the merged K/V cache
    b, r = 1, rows[2]
    mod = O.modulation(cfg, orc.w[0], temb1)
    a = O.layernorm_modulate(cfg, x_in[b, [r]], mod[0][b], mod[1][b])
    q = (a @ orc.w[0]["w_qkv"].T + orc.w[0]["b_qkv"])[:, :32]
    g = O.attention(cfg, q, st.k_cache[b], st.v_cache[b]) @ orc.w[0]["w_o"].T + orc.w[0]["b_o"]
    np.testing.assert_allclose(st.g[0][b, r], g[0], rtol=1e-11, atol=1e-12)
    # rows_out spot-check mode gives the same values for the rows it computes
    orc2 = O.HeroOracle(cfg, w)
    orc2.block_refresh(0, x0.copy(), temb0, None)
    rows2 = orc2.select(0)
    assert np.array_equal(rows, rows2)
    orc2.block_refresh(0, x_in.copy(), temb1, rows, rows_out=rows[1:4])
    np.testing.assert_allclose(orc2.blocks[0].g[0][:, rows[1:4]], st.g[0][:, rows[1:4]], rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(orc2.blocks[0].g[1][:, rows[1:4]], st.g[1][:, rows[1:4]], rtol=1e-11, atol=1e-12)
    assert np.array_equal(orc2.blocks[0].k_cache, st.k_cache)


def _one_cached_refresh(cfg, w, poke=None):
    """One full refresh, an optional change of cached K/V rows, then one cached refresh: (oracle, rows, x_out)."""
    rng = np.random.default_rng(12)
    x0, temb0 = rng.standard_normal((2, cfg.n_rows, 32)), rng.standard_normal((2, 12))
    x1, temb1 = rng.standard_normal((2, cfg.n_rows, 32)), rng.standard_normal((2, 12))
    orc = O.HeroOracle(cfg, w)
    orc.block_refresh(0, x0, temb0, None)
    rows = orc.select(0)
    if poke is not None:
        for r in poke(rows):
            orc.blocks[0].k_cache[:, r] += 0.7
            orc.blocks[0].v_cache[:, r] -= 0.4
    return orc, rows, orc.block_refresh(0, x1, temb1, rows)


def test_literal_eq3_attention_sees_only_refreshed_and_text_rows():
    """attend_mode 1: the branch outputs of a cached step do not depend on the cached K/V of video rows that are
    not refreshed, do depend on the text rows' K/V, and with every video row refreshed equal the default mode
    (softmax attention does not depend on the order of the keys)."""
    w = rand_weights(small_cfg(n_blocks=1, n_shallow=1), seed=10)
    lit = small_cfg(n_blocks=1, n_shallow=1, attend_mode=1)
    dflt = small_cfg(n_blocks=1, n_shallow=1)
    stale = lambda rows: np.setdiff1d(np.arange(lit.n_text, lit.n_rows), rows)[:5]
    text = lambda rows: [1]
    base = _one_cached_refresh(lit, w)
    rows = base[1]
    assert 0 < len(rows) < lit.n_video
    got = _one_cached_refresh(lit, w, stale)
    assert np.array_equal(got[2][:, rows], base[2][:, rows])                  # stale video rows are never read
    got = _one_cached_refresh(lit, w, text)
    assert np.abs(got[2][:, rows] - base[2][:, rows]).max() > 1e-3            # the text rows are
    d0, d1 = _one_cached_refresh(dflt, w), _one_cached_refresh(dflt, w, stale)
    assert np.abs(d1[2][:, rows] - d0[2][:, rows]).max() > 1e-3               # the default mode reads them
    assert np.abs(d0[2][:, rows] - base[2][:, rows]).max() > 1e-3             # so the two modes differ ...
    # ... except when nothing is left out
    w1 = rand_weights(small_cfg(n_blocks=1, n_shallow=1), seed=3)
    a = _one_cached_refresh(small_cfg(n_blocks=1, n_shallow=1, ratio_den=1, attend_mode=1), w1)
    b = _one_cached_refresh(small_cfg(n_blocks=1, n_shallow=1, ratio_den=1), w1)
    assert len(a[1]) == lit.n_video
    np.testing.assert_allclose(a[2], b[2], rtol=1e-11, atol=1e-12)
    # one refreshed row by hand: softmax over [text rows, refreshed rows] of the merged cache only
    orc, rows, _ = base
    st = orc.blocks[0]
    rng = np.random.default_rng(12)
    rng.standard_normal((2, lit.n_rows, 32)); rng.standard_normal((2, 12))
    x1, temb1 = rng.standard_normal((2, lit.n_rows, 32)), rng.standard_normal((2, 12))
    bi, r = 0, rows[1]
    mod = O.modulation(lit, orc.w[0], temb1)
    q = (O.layernorm_modulate(lit, x1[bi, [r]], mod[0][bi], mod[1][bi]) @ orc.w[0]["w_qkv"].T + orc.w[0]["b_qkv"])[0, :32]
    seen = list(range(lit.n_text)) + list(rows)
    out = np.zeros(32)
    for hd in range(lit.n_heads):
        sl = slice(hd * lit.head_dim, (hd + 1) * lit.head_dim)
        sc = np.array([q[sl] @ st.k_cache[bi, j, sl] for j in seen]) / np.sqrt(lit.head_dim)
        p = np.exp(sc - sc.max()); p /= p.sum()
        out[sl] = sum(pj * st.v_cache[bi, j, sl] for pj, j in zip(p, seen))
    np.testing.assert_allclose(st.g[0][bi, r], out @ orc.w[0]["w_o"].T + orc.w[0]["b_o"], rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("attend_mode,n_text", [(0, 4), (1, 4), (1, 0)])
def test_an_empty_selection_refreshes_nothing_and_adds_the_cached_outputs(attend_mode, n_text):
    """S(z) empty (a quota of zero in every patch): Eq. 3 then keeps every cached row, no cache changes, and the
    residual stream receives the cached branch outputs - also when the literal reading of Eq. 3 leaves the
    refreshed queries no key at all (no text rows, no refreshed rows)."""
    cfg = small_cfg(n_blocks=1, n_shallow=1, attend_mode=attend_mode, n_text=n_text)
    w = rand_weights(cfg, seed=21)
    rng = np.random.default_rng(22)
    x0, temb0 = rng.standard_normal((2, cfg.n_rows, 32)), rng.standard_normal((2, 12))
    x1, temb1 = rng.standard_normal((2, cfg.n_rows, 32)), rng.standard_normal((2, 12))
    orc = O.HeroOracle(cfg, w)
    orc.block_refresh(0, x0, temb0, None)
    st = orc.blocks[0]
    before = [a.copy() for a in (st.k_cache, st.v_cache, st.g[0], st.g[1])]
    out = orc.block_refresh(0, x1.copy(), temb1, np.zeros(0, dtype=np.int64))
    for a, b in zip((st.k_cache, st.v_cache, st.g[0], st.g[1]), before):
        assert np.array_equal(a, b)
    np.testing.assert_allclose(out, x1 + before[2] + before[3], rtol=1e-13, atol=1e-13)


# ---------------------------------------------------------------- extrapolation (Eq. 5)
def test_extrapolation_is_exact_on_features_linear_in_step():
    rng = np.random.default_rng(13)
    A, Bm = rng.standard_normal((3, 17, 8)), rng.standard_normal((3, 17, 8))
    for s_prev, s_last, s in [(0, 1, 2), (0, 1, 5), (1, 6, 7), (1, 6, 10), (6, 11, 13)]:
        got = O.extrapolate(A + s_prev * Bm, A + s_last * Bm, s - s_last, s_last - s_prev)
        np.testing.assert_allclose(got, A + s * Bm, rtol=1e-12, atol=1e-12)


def test_extrapolation_special_cases():
    rng = np.random.default_rng(14)
    g0, g1 = rng.standard_normal((4, 9)), rng.standard_normal((4, 9))
    assert np.array_equal(O.extrapolate(g0, g1, 0, 3), g1)              # k = 0: plain reuse
    assert np.array_equal(O.extrapolate(g1, g1, 2, 3), g1)              # Delta = 0: plain reuse
    np.testing.assert_allclose(O.extrapolate(g0, g1, 1, 1), 2 * g1 - g0)
    np.testing.assert_allclose(O.extrapolate(g0, g1, 2, 4), 1.5 * g1 - 0.5 * g0)


# ---------------------------------------------------------------- schedule and step bookkeeping (Alg. 1)
def test_schedule():
    cfg = small_cfg(warmup_full_steps=2, full_interval=5)
    orc = O.HeroOracle(cfg, rand_weights(cfg))
    full = [s for s in range(50) if orc.is_full_step(s)]
    assert full == [0, 1, 6, 11, 16, 21, 26, 31, 36, 41, 46]
    cfg0 = small_cfg(warmup_full_steps=2, full_interval=0)
    orc0 = O.HeroOracle(cfg0, rand_weights(cfg0))
    assert [s for s in range(10) if orc0.is_full_step(s)] == [0, 1]
    cfg2 = small_cfg(warmup_full_steps=2, full_interval=2)
    orc2 = O.HeroOracle(cfg2, rand_weights(cfg2))
    assert [s for s in range(8) if orc2.is_full_step(s)] == [0, 1, 3, 5, 7]


def test_cached_step_extrapolates_with_the_real_gap():
    """Plant histories that are linear in the step index in the deep blocks; a cached
    step must then add exactly their value at the current step (pins k and d)."""
    cfg = small_cfg(n_blocks=3, n_shallow=1, warmup_full_steps=2, full_interval=4)
    w = rand_weights(cfg, seed=15)
    rng = np.random.default_rng(16)
    orc = O.HeroOracle(cfg, w)
    x = rng.standard_normal((2, cfg.n_rows, 32))
    temb = rng.standard_normal((2, 12))
    for s in range(6):                       # full steps: 0, 1, 5
        orc.step(s, x, temb)
    assert orc.full_steps == [0, 1, 5]
    shape = (2, cfg.n_rows, 32)
    A = [[rng.standard_normal(shape) for _ in range(2)] for _ in range(3)]
    Bm = [[rng.standard_normal(shape) for _ in range(2)] for _ in range(3)]
    for l in (1, 2):
        for i in range(2):
            orc.blocks[l].g_prev[i] = A[l][i] + 1 * Bm[l][i]
            orc.blocks[l].g_last[i] = A[l][i] + 5 * Bm[l][i]
    for s in (6, 7, 8):
        # shallow block 0 runs first; take its output as the deep blocks' input
        ref = O.HeroOracle(cfg, w)
        ref.blocks[0] = orc.blocks[0]
        calls, ages = orc.blocks[0].calls, orc.blocks[0].ages.copy()
        snapshot = [a.copy() for a in (orc.blocks[0].k_cache, orc.blocks[0].v_cache, *orc.blocks[0].g)]
        xin = np.array(x)
        rows = ref.select(0)
        ref.block_refresh(0, xin, temb, rows)
        # rewind block 0 and run the real step
        st = orc.blocks[0]
        st.calls, st.ages = calls, ages
        st.k_cache, st.v_cache, st.g[0], st.g[1] = snapshot
        got = orc.step(s, x, temb)
        want = xin + sum(A[l][i] + s * Bm[l][i] for l in (1, 2) for i in range(2))
        np.testing.assert_allclose(got, want, rtol=1e-11, atol=1e-11)


def test_history_rotation_and_age_reset_on_full_steps():
    cfg = small_cfg(n_blocks=2, n_shallow=1, warmup_full_steps=2, full_interval=3)
    w = rand_weights(cfg, seed=17)
    rng = np.random.default_rng(18)
    orc = O.HeroOracle(cfg, w)
    xs = [rng.standard_normal((2, cfg.n_rows, 32)) for _ in range(5)]
    te = [rng.standard_normal((2, 12)) for _ in range(5)]
    orc.step(0, xs[0], te[0])
    g_step0 = orc.blocks[1].g_last[0].copy()
    assert orc.blocks[1].g_prev[0] is None
    orc.step(1, xs[1], te[1])
    assert np.array_equal(orc.blocks[1].g_prev[0], g_step0)
    g_step1 = orc.blocks[1].g_last[1].copy()
    orc.step(2, xs[2], te[2])              # cached
    assert orc.blocks[0].calls == 1 and orc.blocks[0].ages.max() == 1
    assert np.array_equal(orc.blocks[1].g_last[1], g_step1)          # untouched by cached steps
    orc.step(3, xs[3], te[3])              # cached
    assert orc.blocks[0].calls == 2
    orc.step(4, xs[4], te[4])              # full (1 + 3)
    assert orc.full_steps == [0, 1, 4]
    assert orc.blocks[0].ages.max() == 0 and orc.blocks[0].calls == 2
    assert np.array_equal(orc.blocks[1].g_prev[1], g_step1)


def test_tiny_config_ten_steps_runs_and_follows_schedule():
    cfgd = S.CONFIGS["tiny"]
    cfg = O.Config.from_dict(cfgd)
    w = [S.block_weights(cfgd, l) for l in range(cfg.n_blocks)]
    orc = O.HeroOracle(cfg, w)
    x = S.tokens(cfgd)
    n_sel = []
    for s in range(cfgd["steps"]):
        out = orc.step(s, x, S.temb(cfgd, s))
        assert np.isfinite(out).all()
    assert orc.full_steps == [0, 1]
    assert orc.blocks[0].calls == 8 and orc.blocks[1].calls == 8
    assert orc.blocks[2].calls == 0
    assert O.n_selected(cfg, 0) == 32           # 25 % of 128 video tokens


# ---------------------------------------------------------------- deep-stack collapse (linearity of Eq. 5)
def test_extrapolating_the_sum_equals_summing_the_extrapolations():
    rng = np.random.default_rng(5)
    prev = [rng.standard_normal((2, 7, 16)) for _ in range(6)]
    last = [p + 0.1 * rng.standard_normal(p.shape) for p in prev]
    for k, d in ((1, 1), (2, 5), (4, 5), (0, 3)):
        one_by_one = sum(O.extrapolate(p, l, k, d) for p, l in zip(prev, last))
        assert np.allclose(O.extrapolate_stack(prev, last, k, d), one_by_one, rtol=0, atol=1e-12)
    # not a tautology: a non-linear rule (e.g. clipping each block's step) would break it
    clipped = sum(np.clip(O.extrapolate(p, l, 4, 5), -0.5, 0.5) for p, l in zip(prev, last))
    assert not np.allclose(np.clip(O.extrapolate_stack(prev, last, 4, 5), -0.5, 0.5), clipped)


def test_deep_stack_extrapolate_matches_block_by_block_step():
    cfgd = dict(S.CONFIGS["tiny"], n_blocks=5, n_shallow=1, full_interval=3)
    weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    a = O.HeroOracle(O.Config.from_dict(cfgd), weights)
    x0 = S.tokens(cfgd)
    for s in range(3):                                    # full at 0, 1; cached at 2
        xa = a.step(s, x0, S.temb(cfgd, s))
    # redo the cached step's deep part with the collapsed form on a copy of the state before it
    b = O.HeroOracle(O.Config.from_dict(cfgd), weights)
    for s in range(2):
        b.step(s, x0, S.temb(cfgd, s))
    xb = np.array(x0, np.float64)
    rows = b.select(0)
    b.block_refresh(0, xb, S.temb(cfgd, 2), rows)
    b.deep_stack_extrapolate(xb, 1, 1)
    assert np.allclose(xa, xb, rtol=0, atol=1e-11)


# ---------------------------------------------------------------- diagnostics (Sec. 4.1)
def test_second_difference_variance_closed_forms():
    rng = np.random.default_rng(40)
    a, b, c = rng.standard_normal((3, 5, 7))
    t = np.arange(6.0)[:, None, None]
    assert O.second_difference_variance(a + b * t) < 1e-24                      # linear in the step: no curvature
    # quadratic in the step: the second difference is 2c at every step, so its variance is that of 2c over elements
    np.testing.assert_allclose(O.second_difference_variance(a + b * t + c * t * t), np.var(2 * c), rtol=1e-10)
    # white noise of variance s^2 per step: coefficients (1, -2, 1) give 6 s^2
    f = rng.standard_normal((400, 2000)) * 0.5
    np.testing.assert_allclose(O.second_difference_variance(f), 6 * 0.25, rtol=2e-2)
    # brute force on a tiny input
    g = rng.standard_normal((4, 3))
    d2 = [g[t + 1][j] - 2 * g[t][j] + g[t - 1][j] for t in (1, 2) for j in range(3)]
    np.testing.assert_allclose(O.second_difference_variance(g), np.var(d2), rtol=1e-12)


def test_stability_scores_order_range_and_invariances():
    rng = np.random.default_rng(41)
    noise = rng.standard_normal((3, 8, 50))
    layers = [noise[0] * 2.0, noise[1] * 0.5, noise[2] * 1.0]                   # most, least, middling fluctuation
    sc = O.stability_scores(layers)
    assert sc[0] == 0.0 and sc[1] == 1.0 and 0.0 < sc[2] < 1.0
    v = [O.second_difference_variance(f) for f in layers]
    np.testing.assert_allclose(sc[2], 1.0 - (v[2] - v[1]) / (v[0] - v[1]), rtol=1e-12)
    # a drift that is linear in the step changes nothing; a common rescaling of all layers neither
    t = np.arange(8.0)[:, None]
    np.testing.assert_allclose(O.stability_scores([f + 3.0 * t + 1.0 for f in layers]), sc, atol=1e-12)
    np.testing.assert_allclose(O.stability_scores([7.0 * f for f in layers]), sc, atol=1e-12)
    assert np.array_equal(O.stability_scores([layers[0], layers[0]]), np.ones(2))
    # closed form of the normalisation: white noise of standard deviation s has second-difference variance
    # 6 s^2, so layers with s^2 in arithmetic progression land on equally spaced scores 1, 1/2, 0 (up to
    # sampling noise), and one more layer between two others moves none of theirs
    big = rng.standard_normal((3, 300, 4000))
    sc3 = O.stability_scores([big[0] * np.sqrt(1.0), big[1] * np.sqrt(2.0), big[2] * np.sqrt(3.0)])
    np.testing.assert_allclose(sc3, [1.0, 0.5, 0.0], atol=2e-2)
    sc4 = O.stability_scores([big[0], big[1] * np.sqrt(2.0), big[2] * np.sqrt(3.0), big[1] * np.sqrt(1.5)])
    np.testing.assert_allclose(sc4[:3], sc3, atol=1e-12)
    np.testing.assert_allclose(sc4[3], 0.75, atol=2e-2)


def test_extrapolation_error_is_zero_on_linear_features_and_known_on_a_quadratic():
    rng = np.random.default_rng(42)
    a, b, c = rng.standard_normal((3, 4, 6))
    f = lambda t: a + b * t + c * t * t
    lin = lambda t: a + b * t
    assert O.extrapolation_error(lin(0.0), lin(5.0), lin(7.0), 2, 5) < 1e-14
    # features quadratic in the step, sampled at 0 and d, predicted at d + k: the line through the two samples
    # misses by c k (d + k), whatever a and b are
    d, k = 5, 2
    want = np.linalg.norm(c * k * (d + k)) / np.linalg.norm(f(d + k))
    np.testing.assert_allclose(O.extrapolation_error(f(0.0), f(float(d)), f(float(d + k)), k, d), want, rtol=1e-12)
