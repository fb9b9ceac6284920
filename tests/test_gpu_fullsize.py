"""GPU parity at the full sizes of the one-block and Aether-shaped workloads (bf16, B = 2,
N = 17776 or 23176 rows, hidden 3072, 48 heads, FFN 12288), in the launch configuration the
benchmark times.  The oracle cannot run a whole block at this size in seconds, so the caches are
teacher-forced with seeded values, the K/V rewrite of every selected row is checked in full, and
the branch outputs and the residual stream are checked on sampled rows that the oracle computes
one by one; the merge of Eq. 3 is checked by bit-identity of sampled untouched rows."""
import numpy as np
import pytest
import torch

from oracle import hero_oracle as O
from workloads import synthetic as S
from tests.util import rel_l2, to_dev, to_host

pytestmark = pytest.mark.gpu

BF16_TOL = 2e-2          # rel-L2, bf16 GEMM/attention against the float64 oracle


def H():
    import paper_2508_17588_b200 as h
    return h


CASES = {
    "cogvideox_block_25": dict(S.CONFIGS["block"], ratio_num=1, ratio_den=4),
    "cogvideox_block_25_qk_norm_rope": dict(S.CONFIGS["block"], ratio_num=1, ratio_den=4, qk_norm=1, rope=1),
    "cogvideox_block_25_attend_refreshed": dict(S.CONFIGS["block"], ratio_num=1, ratio_den=4, attend_mode=1),
    "aether_block_10": dict(S.CONFIGS["aether"], n_blocks=1, n_shallow=1, ratio_num=1, ratio_den=10, full_interval=0),
}


@pytest.mark.parametrize("name", list(CASES))
def test_refresh_block_full_size_sampled(name):
    cfgd = CASES[name]
    cfg = O.Config.from_dict(cfgd)
    B, N, D = cfg.batch, cfg.n_rows, cfg.hidden
    weights = [S.block_weights(cfgd, 0)]
    orc = O.HeroOracle(cfg, weights)
    h = H()
    hero = h.Hero(cfgd, [h.device_weights(weights[0], "bf16")])

    # teacher-forced caches: the same bf16-exact values on both sides
    st = orc.blocks[0]
    fills = {"k": S.cache_fill(cfgd, "k", 0), "v": S.cache_fill(cfgd, "v", 0),
             "g_attn": S.cache_fill(cfgd, "ga", 0, std=0.1), "g_ffn": S.cache_fill(cfgd, "gf", 0, std=0.1)}
    for key, val in fills.items():
        hero.hero_state_set(0, key, torch.from_numpy(val))
    st.k_cache, st.v_cache = fills["k"].astype(np.float64), fills["v"].astype(np.float64)
    st.g = [fills["g_attn"].astype(np.float64), fills["g_ffn"].astype(np.float64)]

    # selection: bit-exact list and ages
    rows = orc.select(0)
    idx = torch.full((cfg.n_video,), -1, dtype=torch.int32, device="cuda")
    n = hero.hero_select_tokens(0, idx)
    assert n == len(rows) == O.n_selected(cfg, 0)
    assert np.array_equal(idx[:n].cpu().numpy(), rows)
    assert np.array_equal(hero.hero_state_get(0, "ages").numpy(), st.ages)

    rng = np.random.default_rng(17)
    sample = np.sort(rng.choice(rows, 24, replace=False))                 # refreshed rows checked end to end
    sample = np.unique(np.concatenate([sample, rows[:1], rows[-1:]]))     # first and last list entries too
    others = np.setdiff1d(np.arange(N), rows)
    keep = np.sort(rng.choice(others, 64, replace=False))                 # untouched rows
    keep = np.setdiff1d(np.unique(np.concatenate([keep, [0, cfg.n_text - 1, N - 1]])), rows)   # text rows, last row

    x_host = S.tokens(cfgd)
    temb = S.temb(cfgd, 2)
    x_dev = to_dev(x_host, "bf16")
    hero.hero_refresh_block(0, x_dev, to_dev(temb, "bf16"), idx[:n], n)
    hero.hero_check_status()
    want_x = orc.block_refresh(0, x_host.astype(np.float64), temb, rows, rows_out=sample)

    got = {key: to_host(hero.hero_state_get(0, key)) for key in ("k", "v", "g_attn", "g_ffn")}
    got_x = to_host(x_dev)
    # K/V of every refreshed row, both batch items
    assert rel_l2(got["k"][:, rows], st.k_cache[:, rows]) <= BF16_TOL
    assert rel_l2(got["v"][:, rows], st.v_cache[:, rows]) <= BF16_TOL
    # branch outputs and residual stream on the sampled refreshed rows
    assert rel_l2(got["g_attn"][:, sample], st.g[0][:, sample]) <= BF16_TOL
    assert rel_l2(got["g_ffn"][:, sample], st.g[1][:, sample]) <= BF16_TOL
    assert rel_l2(got_x[:, sample], want_x[:, sample]) <= BF16_TOL
    for r in sample[:4]:                                                   # row by row as well
        assert rel_l2(got["g_attn"][:, r], st.g[0][:, r]) <= BF16_TOL, r
        assert rel_l2(got["g_ffn"][:, r], st.g[1][:, r]) <= BF16_TOL, r
    # Eq. 3's merge: untouched rows of every cache are bit-identical, their residual is x + G + G
    for key, val in fills.items():
        assert np.array_equal(got[key][:, keep], val[:, keep].astype(np.float64)), key
    assert rel_l2(got_x[:, keep], want_x[:, keep]) <= 2 ** -8              # one bf16 rounding of the sum
    assert np.isfinite(got_x).all()
    hero.close()
