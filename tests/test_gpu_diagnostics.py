"""GPU parity of the Sec. 4.1 diagnostics (moments of the second-order temporal differences, from which the
stability score follows, and the error of Eq. 5 against recomputed features) with the float64 oracle."""
import numpy as np
import pytest
import torch

from oracle import hero_oracle as O
from workloads import synthetic as S
from tests.util import to_dev, to_host

pytestmark = pytest.mark.gpu

MOMENT_TOL = 2e-6        # relative, fp32 partial sums of <= 512 terms then double


def H():
    import paper_2508_17588_b200 as h
    return h


def gpu_variance(frames, dtype):
    """Variance of the second differences of frames [T, ...] through the device moments."""
    m = torch.zeros(2, dtype=torch.float64, device="cuda")
    dev = [to_dev(f, dtype) for f in frames]
    for t in range(1, len(frames) - 1):
        H().hero_second_difference_moments(dev[t - 1], dev[t], dev[t + 1], m)
    n = (len(frames) - 2) * frames[0].size
    m0, m1 = m.cpu().numpy()
    return m1 / n - (m0 / n) ** 2, (m0, m1, n)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("shape", [(1, 7), (3, 1000, 129), (2, 4099, 257)])      # ragged tails, several blocks
def test_second_difference_moments_match_oracle(dtype, shape):
    cfg = dict(seed=5, dtype=dtype)
    frames = [S.normal(5, "diag", shape, std=1.0 + 0.3 * t, index=t, dtype=dtype) + np.float32(0.25 * t * t) for t in range(5)]
    if dtype == "bf16":
        frames = [S.round_bf16(f) for f in frames]
    var, (m0, m1, n) = gpu_variance(frames, dtype)
    f64 = np.stack(frames).astype(np.float64)
    d2 = f64[2:] - 2 * f64[1:-1] + f64[:-2]
    assert abs(m1 - (d2 ** 2).sum()) <= MOMENT_TOL * (d2 ** 2).sum()
    assert abs(m0 - d2.sum()) <= MOMENT_TOL * np.abs(d2).sum()
    np.testing.assert_allclose(var, O.second_difference_variance(f64), rtol=1e-5)


def test_stability_scores_of_a_tiny_uncached_run_match_oracle():
    """Eight full steps of the tiny fp32 model on both sides; the attention-branch outputs of every block are
    the 'temporal features'.  The device forms the moments, the host the min-max score."""
    cfgd = dict(S.CONFIGS["tiny"], warmup_full_steps=8, full_interval=0, steps=8)
    cfg = O.Config.from_dict(cfgd)
    weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    orc = O.HeroOracle(cfg, weights)
    h = H()
    hero = h.Hero(cfgd, [h.device_weights(w, "fp32") for w in weights])
    x_host = S.tokens(cfgd)
    feats_o = [[] for _ in range(cfg.n_blocks)]
    feats_g = [[] for _ in range(cfg.n_blocks)]
    for s in range(8):
        temb = S.temb(cfgd, s)
        orc.step(s, x_host, temb)
        x = to_dev(x_host, "fp32")
        hero.hero_step(s, x, to_dev(temb, "fp32"))
        for l in range(cfg.n_blocks):
            st = orc.blocks[l]
            feats_o[l].append(np.array(st.g[0] if l < cfg.n_shallow else st.g_last[0]))
            feats_g[l].append(hero.hero_state_get(l, "g_attn").cuda())
    want = O.stability_scores([np.stack(f) for f in feats_o])
    var = []
    for l in range(cfg.n_blocks):
        m = torch.zeros(2, dtype=torch.float64, device="cuda")
        for t in range(1, 7):
            h.hero_second_difference_moments(feats_g[l][t - 1], feats_g[l][t], feats_g[l][t + 1], m)
        n = 6 * feats_g[l][0].numel()
        m0, m1 = m.cpu().numpy()
        var.append(m1 / n - (m0 / n) ** 2)
    var = np.array(var)
    got = 1.0 - (var - var.min()) / (var.max() - var.min())
    np.testing.assert_allclose(got, want, atol=1e-4)
    assert got.min() == 0.0 and got.max() == 1.0
    hero.close()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("k,d", [(1, 1), (2, 5), (4, 5)])
def test_extrapolation_error_matches_oracle(dtype, k, d):
    cfg = dict(S.CONFIGS["tiny"], dtype=dtype, seed=9)
    shape = (2, 1031, 193)
    g_prev, g_last = S.feature_history(cfg, shape=shape, drift=0.1)
    g_true = (g_last + (g_last - g_prev) * np.float32(k / d) + S.normal(9, "truth", shape, std=0.05)).astype(np.float32)
    if dtype == "bf16":
        g_true = S.round_bf16(g_true)
    err = torch.zeros(2, dtype=torch.float64, device="cuda")
    H().hero_extrapolation_error(to_dev(g_prev, dtype), to_dev(g_last, dtype), to_dev(g_true, dtype), k, d, err)
    e0, e1 = err.cpu().numpy()
    want = O.extrapolation_error(g_prev, g_last, g_true, k, d)
    np.testing.assert_allclose(np.sqrt(e0 / e1), want, rtol=1e-4)
    np.testing.assert_allclose(e1, (g_true.astype(np.float64) ** 2).sum(), rtol=MOMENT_TOL)


def test_diagnostics_accumulate_and_reject_bad_arguments():
    h = H()
    a = torch.ones(1000, device="cuda")
    m = torch.zeros(2, dtype=torch.float64, device="cuda")
    h.hero_second_difference_moments(a, a * 0, a, m)             # u = 2 everywhere
    h.hero_second_difference_moments(a, a * 0, a, m)
    assert m.cpu().tolist() == [4000.0, 8000.0]
    h.hero_second_difference_moments(a[:0], a[:0], a[:0], m)     # empty input: nothing added
    assert m.cpu().tolist() == [4000.0, 8000.0]
    with pytest.raises(h.HeroError):
        h.hero_second_difference_moments(a[1:], a[1:], a[1:], m)     # not 16-byte aligned
    with pytest.raises(h.HeroError):
        h.hero_extrapolation_error(a, a, a, 1, 0, m)                 # d = 0
