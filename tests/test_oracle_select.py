"""Pins for the oracle's selection function S(z) (Eq. 4 and the tracking paragraph
of Sec. 4.3): invariants the paper fixes, closed forms, brute force on tiny grids
and the quota rounding that Table 3 implies.  CPU only."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import hero_oracle as O
from workloads import synthetic as S

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def make_cfg(**kw):
    base = dict(n_blocks=1, n_shallow=1, hidden=8, n_heads=1, head_dim=8, ffn_dim=16, temb_dim=4,
                batch=1, frames=2, grid_h=8, grid_w=8, n_text=3, patch_h=2, patch_w=2,
                ratio_num=1, ratio_den=4, quota_mode=0, seed=7)
    base.update(kw)
    return O.Config(**base)


# ---------------------------------------------------------------- mixer
def _unxorshift(x, s):
    y = x
    for _ in range(32 // s + 1):
        y = x ^ (y >> s)
    return y & 0xFFFFFFFF


def test_mix32_is_a_bijection_with_explicit_inverse():
    inv1 = pow(0x85EBCA6B, -1, 1 << 32)
    inv2 = pow(0xC2B2AE35, -1, 1 << 32)
    rng = np.random.default_rng(0)
    for x in [0, 1, 0xFFFFFFFF, 0x80000000] + [int(v) for v in rng.integers(0, 1 << 32, 200)]:
        y = O.mix32(x)
        z = _unxorshift(y, 16)
        z = (z * inv2) & 0xFFFFFFFF
        z = _unxorshift(z, 13)
        z = (z * inv1) & 0xFFFFFFFF
        z = _unxorshift(z, 16)
        assert z == x
    assert O.mix32(0) == 0


def test_mix32_avalanche():
    rng = np.random.default_rng(1)
    flips = []
    for x in rng.integers(0, 1 << 32, 300):
        x = int(x)
        for bit in (0, 7, 19, 31):
            flips.append(bin(O.mix32(x) ^ O.mix32(x ^ (1 << bit))).count("1"))
    assert 14.5 < np.mean(flips) < 17.5


# ---------------------------------------------------------------- geometry
@pytest.mark.parametrize("f,h,w,ph,pw", [(1, 4, 5, 2, 2), (2, 8, 8, 2, 2), (3, 5, 7, 2, 3), (13, 30, 45, 2, 2)])
def test_patch_table_is_a_partition_with_formula_ids(f, h, w, ph, pw):
    cfg = make_cfg(frames=f, grid_h=h, grid_w=w, patch_h=ph, patch_w=pw)
    table = O.patch_table(cfg)
    PH, PW = -(-h // ph), -(-w // pw)
    assert len(table) == f * PH * PW
    seen = np.full(cfg.n_video, -1)
    for i, toks in enumerate(table):
        assert list(toks) == sorted(toks) and 1 <= len(toks) <= ph * pw
        for v in toks:
            assert seen[v] == -1
            seen[v] = i
    # independent restatement: patch id from the token's coordinates
    for v in range(cfg.n_video):
        t, rem = divmod(v, h * w)
        y, x = divmod(rem, w)
        assert seen[v] == (t * PH + y // ph) * PW + x // pw
    # closed form for the number of tokens in earlier patches
    before = 0
    for i, toks in enumerate(table):
        t, rem = divmod(i, PH * PW)
        py, px = divmod(rem, PW)
        rows_here = min(ph, h - py * ph)
        assert before == t * h * w + py * ph * w + rows_here * px * pw
        before += len(toks)


# ---------------------------------------------------------------- quotas
@pytest.mark.parametrize("num,den", [(1, 10), (1, 4), (1, 2), (1, 1), (1, 5), (3, 7)])
@pytest.mark.parametrize("grid", [(1, 4, 5), (2, 8, 8), (13, 30, 45)])
def test_quota_mode0_invariants(num, den, grid):
    cfg = make_cfg(frames=grid[0], grid_h=grid[1], grid_w=grid[2], ratio_num=num, ratio_den=den)
    R = Fraction(num, den)
    table = O.patch_table(cfg)
    for call in (0, 1, 2, 5, 1000):
        q = O.patch_quotas(cfg, call)
        off = call * cfg.patch_h * cfg.patch_w
        assert sum(q) == O.n_selected(cfg, call)
        assert sum(q) == int((cfg.n_video + off) * R) - int(off * R)       # floor via Fraction
        assert abs(sum(q) - cfg.n_video * R) < 1
        for qi, toks in zip(q, table):
            assert 0 <= qi <= len(toks)
            exact = R * len(toks)
            if exact.denominator == 1:
                assert qi == exact                      # "a fixed ratio R ... from each patch"
            else:
                assert abs(qi - exact) < 1


def test_quota_ratio_one_selects_everything():
    cfg = make_cfg(ratio_num=1, ratio_den=1, frames=2, grid_h=5, grid_w=7, patch_w=3)
    rows, ages = O.select_tokens(cfg, np.full(cfg.n_video, 3, np.uint16), 0, 4)
    assert rows.tolist() == list(range(cfg.n_text, cfg.n_rows))
    assert (ages == 0).all()


def test_quota_mode1_matches_table3_golden():
    """Table 3 lists FLOPs that fall in equal steps for R = 0.8, 0.7, 0.5, 0.3, 0.2 with
    2x3 patches: only integer per-patch quotas 5, 4, 3, 2, 1 produce that."""
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table3_quota.txt")) if l[0] != "#"]
    flops = []
    for r_txt, flop_txt, q_txt in rows:
        R = Fraction(r_txt)
        cfg = make_cfg(frames=1, grid_h=4, grid_w=6, patch_h=2, patch_w=3, quota_mode=1,
                       ratio_num=R.numerator, ratio_den=R.denominator)
        q = O.patch_quotas(cfg, 0)
        assert set(q) == {int(q_txt)}
        flops.append((int(q_txt), float(flop_txt)))
    # the printed FLOPs are affine in the quota (same increment per extra token per patch)
    (q0, f0), (q1, f1) = flops[0], flops[-1]
    slope = (f0 - f1) / (q0 - q1)
    for q, f in flops:
        assert abs(f - (f1 + slope * (q - q1))) < 0.5


def test_quota_mode0_brute_force_tiny_grid():
    cfg = make_cfg(frames=1, grid_h=4, grid_w=5, ratio_num=1, ratio_den=4)
    # 1x4x5 grid, 2x2 patches -> patch sizes 4,4,2,4,4,2 ; running floor of cumulative R*count
    sizes = [4, 4, 2, 4, 4, 2]
    assert [len(t) for t in O.patch_table(cfg)] == sizes
    for call in range(6):
        cum, expect = call * 4, []
        for n in sizes:
            expect.append((cum + n) // 4 - cum // 4)
            cum += n
        assert O.patch_quotas(cfg, call) == expect


# ---------------------------------------------------------------- sampler
def _brute_select(cfg, ages, block, call):
    """Independent restatement: rank of a token = number of patch mates that beat it."""
    picked = []
    table = O.patch_table(cfg)
    quotas = O.patch_quotas(cfg, call)
    key = lambda v: (int(ages[v]) + 1) * (O.token_hash(cfg.seed, block, call, v) + 1)
    for toks, q in zip(table, quotas):
        for v in toks:
            beaten_by = sum(1 for u in toks if key(u) > key(v) or (key(u) == key(v) and u < v))
            if beaten_by < q:
                picked.append(v)
    return sorted(picked)


@pytest.mark.parametrize("grid,patch,ratio", [((1, 4, 5), (2, 2), (1, 4)), ((2, 8, 8), (2, 2), (1, 4)),
                                              ((2, 5, 7), (2, 3), (1, 5)), ((2, 6, 6), (2, 3), (1, 2))])
def test_select_matches_rank_definition_and_replays_ages(grid, patch, ratio):
    cfg = make_cfg(frames=grid[0], grid_h=grid[1], grid_w=grid[2], patch_h=patch[0], patch_w=patch[1],
                   ratio_num=ratio[0], ratio_den=ratio[1])
    ages = np.zeros(cfg.n_video, np.uint16)
    for call in range(12):
        rows, new_ages = O.select_tokens(cfg, ages, 1, call)
        want = _brute_select(cfg, ages, 1, call)
        assert (rows - cfg.n_text).tolist() == want
        assert len(rows) == O.n_selected(cfg, call)
        assert (np.diff(rows) > 0).all()                        # strictly ascending, no duplicates
        assert rows.min() >= cfg.n_text and rows.max() < cfg.n_rows   # text rows never picked
        replay = ages.astype(np.int64) + 1
        replay[np.array(want, dtype=int)] = 0
        assert (new_ages == replay).all()
        for toks, q in zip(O.patch_table(cfg), O.patch_quotas(cfg, call)):
            assert sum(1 for v in toks if v in set(want)) == q   # every patch gets exactly its quota
        ages = new_ages


def test_age_saturates():
    cfg = make_cfg(frames=1, grid_h=2, grid_w=2, ratio_num=1, ratio_den=4)
    ages = np.array([65535, 65534, 0, 0], np.uint16)
    _, new = O.select_tokens(cfg, ages, 0, 0)
    assert new.max() <= 65535 and set(new.tolist()) <= {0, 1, 65535}


def test_equal_ages_give_uniform_sampling():
    """Equal ages: every token of a patch is equally likely (chi-square over many draws)."""
    cfg = make_cfg(frames=1, grid_h=2, grid_w=3, patch_h=2, patch_w=3, ratio_num=1, ratio_den=3)  # q = 2 of 6
    counts = np.zeros(6)
    n_draws = 6000
    for call in range(n_draws):
        cfg.seed = 1000 + call
        rows, _ = O.select_tokens(cfg, np.zeros(6, np.uint16), 0, 0)
        assert len(rows) == 2
        counts[rows - cfg.n_text] += 1
    expected = n_draws * 2 / 6
    chi2 = ((counts - expected) ** 2 / expected).sum()
    assert chi2 < 25.0          # 5 dof, p ~ 1e-4


@pytest.mark.parametrize("age_a,age_b", [(0, 0), (1, 0), (3, 1), (9, 0), (4, 4)])
def test_two_token_closed_form_probability(age_a, age_b):
    """Two tokens, one slot, weights w = age+1 with w_a >= w_b: the older one wins with
    probability 1 - w_b / (2 w_a) (area of {U_a*w_a > U_b*w_b} for independent uniforms)."""
    cfg = make_cfg(frames=1, grid_h=1, grid_w=2, patch_h=1, patch_w=2, ratio_num=1, ratio_den=2)
    wa, wb = age_a + 1, age_b + 1
    p = 1 - wb / (2 * wa)
    n, wins = 8000, 0
    for s in range(n):
        cfg.seed = 77 + s
        rows, _ = O.select_tokens(cfg, np.array([age_a, age_b], np.uint16), 2, 5)
        wins += int(rows[0] - cfg.n_text == 0)
    sigma = np.sqrt(p * (1 - p) / n) + 1e-9
    assert abs(wins / n - p) < 4.5 * sigma + 1e-3


def test_selection_probability_grows_with_age():
    cfg = make_cfg(frames=1, grid_h=2, grid_w=2, ratio_num=1, ratio_den=4)
    rate = []
    for age0 in (0, 2, 8, 40):
        hit = 0
        for s in range(3000):
            cfg.seed = s
            rows, _ = O.select_tokens(cfg, np.array([age0, 1, 1, 1], np.uint16), 0, 3)
            hit += int(rows[0] == cfg.n_text)
        rate.append(hit / 3000)
    assert rate == sorted(rate) and rate[0] < 0.2 and rate[-1] > 0.9


def test_no_token_is_starved():
    """With tracking, the longest wait stays bounded (here: well under 8x the mean period)."""
    cfg = make_cfg(frames=2, grid_h=8, grid_w=8, ratio_num=1, ratio_den=4)
    ages = np.zeros(cfg.n_video, np.uint16)
    worst = 0
    for call in range(200):
        _, ages = O.select_tokens(cfg, ages, 0, call)
        worst = max(worst, int(ages.max()))
    assert worst < 32


def test_draws_differ_between_blocks_and_calls():
    cfg = make_cfg()
    z = np.zeros(cfg.n_video, np.uint16)
    a, _ = O.select_tokens(cfg, z, 0, 0)
    b, _ = O.select_tokens(cfg, z, 1, 0)
    c, _ = O.select_tokens(cfg, z, 0, 1)
    assert not np.array_equal(a, b) and not np.array_equal(a, c)
    a2, _ = O.select_tokens(cfg, z, 0, 0)
    assert np.array_equal(a, a2)


# ---------------------------------------------------------------- strict oldest-first tracking (track_mode 1)
def test_oldest_first_never_leaves_a_token_unsampled_longer_than_one_round():
    """With the key (age, hash) a patch of #P tokens and quota q samples every token once per
    ceil(#P / q) calls: ages never exceed that bound (the guarantee the tracking paragraph asks for)."""
    cfgd = dict(S.CONFIGS["tiny"], frames=2, grid_h=6, grid_w=6, patch_h=2, patch_w=3, ratio_num=1, ratio_den=3,
                quota_mode=1, track_mode=1, seed=3)
    cfg = O.Config.from_dict(cfgd)
    assert set(O.patch_quotas(cfg, 0)) == {2}                      # 6-token patches, two per call
    ages = np.zeros(cfg.n_video, np.uint16)
    seen = np.zeros(cfg.n_video, int)
    for call in range(12):
        rows, ages = O.select_tokens(cfg, ages, 0, call)
        seen[rows - cfg.n_text] += 1
        assert ages.max() <= 2                                     # ceil(6/2) - 1
        if (call + 1) % 3 == 0:
            assert (seen == (call + 1) // 3).all()                 # exact round robin, order decided by the hash
    # the weighted mode has no such bound: some token waits longer over the same calls
    cfg0 = O.Config.from_dict(dict(cfgd, track_mode=0))
    ages, worst = np.zeros(cfg0.n_video, np.uint16), 0
    for call in range(12):
        _, ages = O.select_tokens(cfg0, ages, 0, call)
        worst = max(worst, int(ages.max()))
    assert worst > 2


def test_oldest_first_prefers_age_over_any_draw_and_uses_the_draw_among_equals():
    cfgd = dict(S.CONFIGS["tiny"], frames=1, grid_h=2, grid_w=2, patch_h=2, patch_w=2, ratio_num=1, ratio_den=4,
                track_mode=1, n_text=0)
    cfg = O.Config.from_dict(cfgd)
    for seed in range(40):
        c = O.Config.from_dict(dict(cfgd, seed=seed))
        ages = np.array([0, 3, 1, 2], np.uint16)
        rows, new = O.select_tokens(c, ages, 0, 0)
        assert list(rows) == [1]                                   # the oldest token, whatever the draw
        assert list(new) == [1, 0, 2, 3]
    winners = set()
    for seed in range(40):                                         # equal ages: the draw decides
        rows, _ = O.select_tokens(O.Config.from_dict(dict(cfgd, seed=seed)), np.zeros(4, np.uint16), 0, 0)
        winners.add(int(rows[0]))
    assert winners == {0, 1, 2, 3}


def test_every_input_of_the_draw_enters_it_and_none_collides():
    """How the draw is keyed, without typing the composition again: for fixed other inputs the draw is a
    bijection of the token index, of the call counter and of the block index (each passes through an invertible
    mixer round after it is added), so no two tokens, calls or blocks share a draw; only the low 32 bits of the
    seed matter; and the four inputs are not interchangeable (the draw of (block, call, token) = (a, b, c) is
    not that of any permutation), which a transposed argument would break."""
    seed = 0x1234ABCD
    n = 1 << 12
    assert len({O.token_hash(seed, 3, 5, v) for v in range(n)}) == n
    assert len({O.token_hash(seed, 3, c, 77) for c in range(n)}) == n
    assert len({O.token_hash(seed, b, 5, 77) for b in range(n)}) == n
    assert O.token_hash(seed + (7 << 32), 3, 5, 77) == O.token_hash(seed, 3, 5, 77)
    assert O.token_hash(seed ^ 1, 3, 5, 77) != O.token_hash(seed, 3, 5, 77)
    import itertools
    a, b, c = 2, 11, 301
    draws = {perm: O.token_hash(seed, *perm) for perm in itertools.permutations((a, b, c))}
    assert len(set(draws.values())) == 6
    # consecutive tokens, calls and blocks give unrelated draws: the low bit of the draw is balanced and shows
    # no correlation along any of the three axes (a dropped mixer round would leave a counter's pattern in it)
    import numpy as np
    for axis in range(3):
        args = [[3, 5, 77] for _ in range(4096)]
        for i, arg in enumerate(args):
            arg[axis] = i
        bits = np.array([O.token_hash(seed, *arg) & 1 for arg in args], dtype=np.float64)
        assert abs(bits.mean() - 0.5) < 0.04
        assert abs(np.corrcoef(bits[:-1], bits[1:])[0, 1]) < 0.06
