"""GPU parity, HBM-bound kernels: extrapolation (Eq. 5), row gather/scatter (Eq. 3's merge)
and token selection (Eq. 4 + tracking), each through the C ABI against the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import hero_oracle as O
from workloads import synthetic as S
from tests.util import rel_l2, rel_max, to_dev, to_host

pytestmark = pytest.mark.gpu

EXTRAP_TOL = {"fp32": 1e-6, "bf16": 1e-2}     # max-abs error / max-abs value


def H():
    import paper_2508_17588_b200 as h
    return h


# ---------------------------------------------------------------- extrapolation
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("n", [0, 1, 7, 8, 1000, 4096 + 3, 2 * 1777 * 3072 + 5])
@pytest.mark.parametrize("k,d", [(1, 1), (1, 5), (4, 5), (0, 3)])
def test_extrapolate_matches_oracle(dtype, n, k, d):
    cfg = dict(S.CONFIGS["kernels"], dtype=dtype)
    g_prev, g_last = S.feature_history(cfg, shape=(n,))
    want = O.extrapolate(g_prev, g_last, k, d)
    dp, dl = to_dev(g_prev, dtype), to_dev(g_last, dtype)
    out = torch.full_like(dl, float("nan"))
    H().hero_extrapolate(dp, dl, out, k, d)
    torch.cuda.synchronize()
    if n == 0:
        return
    got = to_host(out)
    assert np.isfinite(got).all()
    assert rel_max(got, want) <= EXTRAP_TOL[dtype]
    if k == 0:
        assert np.array_equal(got, g_last.astype(np.float64))          # plain reuse, bit for bit


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_extrapolate_exact_on_linear_features(dtype):
    """Features A + s*B at steps 1 and 6 -> step 8 is A + 8B up to one rounding."""
    rng = np.random.default_rng(3)
    A, Bm = rng.standard_normal(50000).astype(np.float32), rng.standard_normal(50000).astype(np.float32)
    g_prev, g_last = A + 1 * Bm, A + 6 * Bm
    if dtype == "bf16":
        g_prev, g_last = S.round_bf16(g_prev), S.round_bf16(g_last)
    out = torch.empty(50000, device="cuda", dtype=torch.bfloat16 if dtype == "bf16" else torch.float32)
    H().hero_extrapolate(to_dev(g_prev, dtype), to_dev(g_last, dtype), out, 2, 5)
    want = g_last.astype(np.float64) + (g_last.astype(np.float64) - g_prev) * 0.4
    assert rel_max(to_host(out), want) <= EXTRAP_TOL[dtype]


def test_extrapolate_full_size_sampled():
    """Config 2 shape [2, 17776, 3072] bf16 in the launch configuration the bench times;
    a random sample of elements is checked one by one against the oracle."""
    n = 2 * 17776 * 3072
    g = torch.Generator(device="cuda").manual_seed(5)
    a = torch.randn(n, device="cuda", generator=g).bfloat16()
    b = (a.float() + 0.1 * torch.randn(n, device="cuda", generator=g)).bfloat16()
    out = torch.empty_like(a)
    H().hero_extrapolate(a, b, out, 4, 5)
    pick = torch.from_numpy(np.random.default_rng(0).integers(0, n, 20000)).cuda()
    pick = torch.cat([pick, torch.tensor([0, 1, n - 2, n - 1], device="cuda")])
    want = O.extrapolate(to_host(a[pick]), to_host(b[pick]), 4, 5)
    assert rel_max(to_host(out[pick]), want) <= EXTRAP_TOL["bf16"]
    # property that holds at any size: out - g_last has the sign of g_last - g_prev or is zero
    delta, step = (b.float() - a.float()), (out.float() - b.float())
    assert bool(((delta * step) >= 0).all())


# ---------------------------------------------------------------- gather / scatter
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("B,N,D,n_sel", [(1, 9, 8, 0), (1, 9, 8, 9), (2, 50, 64, 13), (2, 300, 3072, 77), (3, 41, 136, 40)])
def test_gather_scatter_bit_exact(dtype, B, N, D, n_sel):
    rng = np.random.default_rng(B * 1000 + N)
    src = S.round_bf16(rng.standard_normal((B, N, D)).astype(np.float32))
    idx = np.sort(rng.choice(N, n_sel, replace=False)).astype(np.int32)
    d_src, d_idx = to_dev(src, dtype), torch.from_numpy(idx).cuda()
    comp = torch.full((B, n_sel, D), 7.0, device="cuda", dtype=d_src.dtype)
    H().hero_gather_rows(d_src, d_idx, comp)
    assert np.array_equal(to_host(comp), src[:, idx].astype(np.float64))
    # scatter into a cache full of sentinels: listed rows replaced, every other row untouched
    cache0 = S.round_bf16(rng.standard_normal((B, N, D)).astype(np.float32))
    cache = to_dev(cache0, dtype)
    H().hero_scatter_rows(comp * 2, d_idx, cache)
    want = cache0.astype(np.float64).copy()
    want[:, idx] = 2 * src[:, idx]
    assert np.array_equal(to_host(cache), want)


def test_gather_scatter_full_size_lists():
    """Config 2: [2,17776,3072] bf16 with index lists drawn by the oracle's sampler at 10/25/50 %."""
    B, N, D = 2, 17776, 3072
    src = torch.randn(B, N, D, device="cuda", generator=torch.Generator(device="cuda").manual_seed(1)).bfloat16()
    for num, den, n_expect in [(1, 10, 1755), (1, 4, 4387), (1, 2, 8775)]:
        cfg = O.Config.from_dict(dict(S.CONFIGS["kernels"], ratio_num=num, ratio_den=den))
        rows, _ = O.select_tokens(cfg, np.zeros(cfg.n_video, np.uint16), 0, 0)
        assert len(rows) == n_expect
        d_idx = torch.from_numpy(rows).cuda()
        comp = torch.empty(B, len(rows), D, device="cuda", dtype=torch.bfloat16)
        H().hero_gather_rows(src, d_idx, comp)
        assert torch.equal(comp, src[:, d_idx.long()])
        cache = torch.zeros_like(src)
        H().hero_scatter_rows(comp, d_idx, cache)
        mask = torch.zeros(N, dtype=torch.bool, device="cuda")
        mask[d_idx.long()] = True
        assert torch.equal(cache[:, mask], src[:, mask])
        assert int(cache[:, ~mask].abs().max()) == 0


# ---------------------------------------------------------------- selection
SEL_CASES = {
    "tiny": dict(S.CONFIGS["tiny"]),
    "ragged_2x3_mode1": dict(S.CONFIGS["tiny"], frames=3, grid_h=5, grid_w=7, patch_h=2, patch_w=3, ratio_num=1,
                             ratio_den=5, quota_mode=1, n_text=5, seed=123456789012),
    "tenth": dict(S.CONFIGS["tiny"], frames=2, grid_h=9, grid_w=11, ratio_num=1, ratio_den=10, seed=9),
    "cogvideo_25": dict(S.CONFIGS["kernels"], dtype="fp32", hidden=64, n_heads=1, ffn_dim=64, temb_dim=8),
    "aether_10": dict(S.CONFIGS["aether"], dtype="fp32", hidden=64, n_heads=1, ffn_dim=64, temb_dim=8,
                      n_blocks=2, n_shallow=2, ratio_num=1, ratio_den=10),
    "oldest_first": dict(S.CONFIGS["tiny"], frames=3, grid_h=7, grid_w=9, patch_h=2, patch_w=3, ratio_num=1,
                         ratio_den=3, track_mode=1, seed=4),
    "paper_2x3_r02": dict(S.CONFIGS["kernels"], dtype="fp32", hidden=64, n_heads=1, ffn_dim=64, temb_dim=8,
                          frames=11, patch_h=2, patch_w=3, ratio_num=1, ratio_den=5, quota_mode=1),
}


@pytest.mark.parametrize("name", list(SEL_CASES))
def test_select_bit_exact(name):
    cfgd = dict(SEL_CASES[name], n_blocks=max(2, SEL_CASES[name]["n_shallow"]))
    cfgd["n_shallow"] = 2
    cfgd["n_blocks"] = 2
    cfg = O.Config.from_dict(cfgd)
    rng = np.random.default_rng(0)
    w = [{k: rng.standard_normal(s).astype(np.float32) * 0.02 for k, s in S.weight_shapes(cfgd).items()}
         for _ in range(2)]
    h = H()
    hero = h.Hero(cfgd, [h.device_weights(x, cfgd["dtype"]) for x in w])
    n_calls = 6 if cfg.n_video > 5000 else 25
    for block in (0, 1):
        ages = np.zeros(cfg.n_video, np.uint16)
        for call in range(n_calls):
            want_rows, ages = O.select_tokens(cfg, ages, block, call)
            assert hero.hero_next_n_sel(block) == len(want_rows) == O.n_selected(cfg, call)
            idx = torch.full((cfg.n_video,), -1, dtype=torch.int32, device="cuda")
            n = hero.hero_select_tokens(block, idx)
            assert n == len(want_rows)
            got = idx.cpu().numpy()
            assert np.array_equal(got[:n], want_rows)
            assert (got[n:] == -1).all()                                   # nothing written past the list
            assert np.array_equal(hero.hero_state_get(block, "ages").numpy(), ages)
            assert int(hero.hero_state_get(block, "calls")[0]) == call + 1
    # capacity is checked before anything is launched
    small = torch.empty(1, dtype=torch.int32, device="cuda")
    with pytest.raises(h.HeroError) as e:
        hero.hero_select_tokens(0, small)
    assert e.value.code == -3
    hero.close()


@pytest.mark.parametrize("case", range(24))
def test_select_bit_exact_on_random_geometries(case):
    """A seeded sweep over grids, patch shapes (also larger than the grid, also 1x1), ratios, quota and
    tracking modes, with and without text rows: lists, ages and counters bit for bit over 12 calls."""
    rng = np.random.default_rng(1000 + case)
    den = int(rng.integers(1, 12))
    cfgd = dict(S.CONFIGS["tiny"], hidden=64, n_heads=1, head_dim=64, ffn_dim=64, temb_dim=8, n_blocks=1, n_shallow=1,
                frames=int(rng.integers(1, 5)), grid_h=int(rng.integers(1, 14)), grid_w=int(rng.integers(1, 14)),
                patch_h=int(rng.integers(1, 5)), patch_w=int(rng.integers(1, 5)), n_text=int(rng.integers(0, 6)),
                ratio_num=int(rng.integers(1, den + 1)), ratio_den=den, quota_mode=int(rng.integers(0, 2)),
                track_mode=int(rng.integers(0, 2)), seed=int(rng.integers(0, 2 ** 40)))
    cfg = O.Config.from_dict(cfgd)
    w = [{k: np.zeros(s, np.float32) for k, s in S.weight_shapes(cfgd).items()}]
    h = H()
    hero = h.Hero(cfgd, [h.device_weights(x, "fp32") for x in w])
    ages = np.zeros(cfg.n_video, np.uint16)
    for call in range(12):
        want_rows, ages = O.select_tokens(cfg, ages, 0, call)
        assert hero.hero_next_n_sel(0) == len(want_rows), (cfgd, call)
        idx = torch.full((max(cfg.n_video, 1),), -1, dtype=torch.int32, device="cuda")
        n = hero.hero_select_tokens(0, idx)
        got = idx.cpu().numpy()
        assert n == len(want_rows) and np.array_equal(got[:n], want_rows), (cfgd, call)
        assert (got[n:] == -1).all()
        assert np.array_equal(hero.hero_state_get(0, "ages").numpy(), ages), (cfgd, call)
    hero.close()


# ---------------------------------------------------------------- gather + LayerNorm + modulate (Eq. 2's prologue)
@pytest.mark.parametrize("dtype,B,N,D,n_sel,with_add", [
    ("fp32", 1, 40, 128, 9, False), ("fp32", 2, 33, 260, 33, True),        # generic kernel (row through shared memory)
    ("bf16", 2, 50, 256, 17, True), ("bf16", 1, 20, 1000, 20, False),      # generic kernel, bf16
    ("bf16", 2, 300, 1024, 77, False), ("bf16", 2, 123, 2048, 50, True),   # one warp per row, 4 / 8 packets per lane
    ("bf16", 2, 500, 3072, 259, True), ("bf16", 3, 64, 3072, 64, False),   # the CogVideoX width, ragged last CTA
    ("bf16", 1, 40, 4096, 13, True)])
def test_gather_ln_modulate_matches_oracle(dtype, B, N, D, n_sel, with_add):
    rng = np.random.default_rng(N * 7 + D + n_sel)
    rnd = (lambda a: S.round_bf16(a.astype(np.float32))) if dtype == "bf16" else (lambda a: a.astype(np.float32))
    x = rnd(rng.standard_normal((B, N, D)) * 2.0 + 0.5)
    add = rnd(rng.standard_normal((B, N, D)) * 0.3) if with_add else None
    idx = np.sort(rng.choice(N, n_sel, replace=False)).astype(np.int32)
    mod = rng.standard_normal((B, 4 * D)).astype(np.float32) * 0.5          # shift | scale | two unused chunks
    cfg = O.Config(n_blocks=1, n_shallow=1, hidden=D, n_heads=1, head_dim=D, ffn_dim=8, temb_dim=8, batch=B,
                   frames=1, grid_h=1, grid_w=1, n_text=0, patch_h=1, patch_w=1, ratio_num=1, ratio_den=1)
    mod_d = torch.from_numpy(mod).cuda()
    out = torch.full((B, n_sel, D), float("nan"), device="cuda", dtype=torch.bfloat16 if dtype == "bf16" else torch.float32)
    H().hero_gather_ln_modulate(to_dev(x, dtype), None if add is None else to_dev(add, dtype),
                                torch.from_numpy(idx).cuda(), mod_d[:, :D], mod_d[:, D:2 * D], out)
    torch.cuda.synchronize()
    got = to_host(out)
    for b in range(B):
        rows = x[b, idx].astype(np.float64) + (0.0 if add is None else add[b, idx].astype(np.float64))
        want = O.layernorm_modulate(cfg, rows, mod[b, :D].astype(np.float64), mod[b, D:2 * D].astype(np.float64))
        if dtype == "bf16":        # fp32 statistics, one bf16 rounding of the result
            assert np.abs(got[b] - want).max() <= 2 ** -8 * np.abs(want).max() + 1e-6, b
            assert rel_l2(got[b], want) <= 3e-3
        else:
            assert np.abs(got[b] - want).max() <= 2e-5 * np.abs(want).max(), b
