"""GPU parity, config 1: the tiny fp32 DiT (2 refresh + 2 extrapolate blocks) over all 10
denoising steps through hero_step, against the float64 oracle; plus the cases where the paper
fixes the answer (ratio 1 == uncached step, untouched cache rows)."""
import numpy as np
import pytest
import torch

from oracle import hero_oracle as O
from workloads import synthetic as S
from tests.util import make_pair, rel_l2, to_dev, to_host

pytestmark = pytest.mark.gpu

FP32_TOL = 2e-5          # rel-L2 of fp32 CUDA-core kernels against float64


def test_tiny_ten_steps_match_oracle():
    cfgd = S.CONFIGS["tiny"]
    orc, hero, _ = make_pair(cfgd)
    x_host = S.tokens(cfgd)
    worst = 0.0
    for s in range(cfgd["steps"]):
        temb = S.temb(cfgd, s)
        want = orc.step(s, x_host, temb)
        x = to_dev(x_host, "fp32")
        assert hero.hero_is_full_step(s) == orc.is_full_step(s)
        hero.hero_step(s, x, to_dev(temb, "fp32"))
        hero.hero_check_status()
        err = rel_l2(to_host(x), want)
        worst = max(worst, err)
        assert err <= FP32_TOL, (s, err)
        # bookkeeping is bit-exact: ages, call counters, recorded full steps
        for l in range(cfgd["n_shallow"]):
            assert np.array_equal(hero.hero_state_get(l, "ages").numpy(), orc.blocks[l].ages)
            assert int(hero.hero_state_get(l, "calls")[0]) == orc.blocks[l].calls
        steps = hero.hero_state_get(0, "steps").numpy()
        assert steps[0] == len(orc.full_steps) and steps[2] == orc.full_steps[-1]
        # caches track the oracle's
        for l in range(cfgd["n_shallow"]):
            for name, ref in (("k", orc.blocks[l].k_cache), ("v", orc.blocks[l].v_cache),
                              ("g_attn", orc.blocks[l].g[0]), ("g_ffn", orc.blocks[l].g[1])):
                assert rel_l2(to_host(hero.hero_state_get(l, name)), ref) <= FP32_TOL, (s, l, name)
        for l in range(cfgd["n_shallow"], cfgd["n_blocks"]):
            assert rel_l2(to_host(hero.hero_state_get(l, "g_attn")), orc.blocks[l].g_last[0]) <= FP32_TOL
            assert rel_l2(to_host(hero.hero_state_get(l, "g_ffn")), orc.blocks[l].g_last[1]) <= FP32_TOL
            if len(orc.full_steps) > 1:
                assert rel_l2(to_host(hero.hero_state_get(l, "g_attn_prev")), orc.blocks[l].g_prev[0]) <= FP32_TOL
        # next step starts from the oracle's input on both sides (same x every step, as in the recipe)
    hero.close()
    print("worst rel-L2 over 10 steps:", worst)


@pytest.mark.parametrize("pinned", [True, False])
def test_tiny_host_entry_point_matches_device_entry_point(pinned):
    """Pinned host buffers take the overlapped route (first block's rows read from the host copy while x uploads,
    finished pieces copied back behind the deep pass); pageable ones the plain copy-in, step, copy-out."""
    cfgd = S.CONFIGS["tiny"]
    _, hero_a, w = make_pair(cfgd)
    _, hero_b, _ = make_pair(cfgd, w)
    x0 = torch.from_numpy(S.tokens(cfgd))
    for s in range(5):
        temb = torch.from_numpy(S.temb(cfgd, s))
        xd = x0.cuda()
        hero_a.hero_step(s, xd, temb.cuda())
        xh = x0.clone().pin_memory() if pinned else x0.clone()
        assert xh.is_pinned() == pinned
        hero_b.hero_step_host(s, xh, temb.pin_memory() if pinned else temb.clone())
        assert torch.equal(xd.cpu(), xh), s
    hero_a.hero_check_status(); hero_b.hero_check_status()
    hero_a.close(); hero_b.close()


def test_ratio_one_all_shallow_equals_uncached_forward():
    """Refresh ratio 100 % with extrapolation off: the cached step is the uncached step."""
    cfgd = dict(S.CONFIGS["tiny"], n_shallow=4, ratio_num=1, ratio_den=1)
    orc, hero, w = make_pair(cfgd)
    cfg = O.Config.from_dict(cfgd)
    x_host = S.tokens(cfgd)
    all_rows = torch.arange(cfg.n_rows, dtype=torch.int32, device="cuda")
    for s in range(4):
        temb = S.temb(cfgd, s)
        want = O.uncached_forward(cfg, w, x_host, temb)
        x, t = to_dev(x_host, "fp32"), to_dev(temb, "fp32")
        if s < 2:
            hero.hero_step(s, x, t)
        else:   # explicit refresh of every row, text included, through the refresh path
            idx = torch.empty(cfg.n_video, dtype=torch.int32, device="cuda")
            for l in range(4):
                assert hero.hero_select_tokens(l, idx) == cfg.n_video
                hero.hero_refresh_block(l, x, t, all_rows)
        assert rel_l2(to_host(x), want) <= FP32_TOL
    hero.close()


def test_refresh_leaves_unselected_cache_rows_untouched():
    cfgd = dict(S.CONFIGS["tiny"], n_blocks=1, n_shallow=1)
    orc, hero, _ = make_pair(cfgd)
    cfg = O.Config.from_dict(cfgd)
    x_host = S.tokens(cfgd)
    t0, t1 = S.temb(cfgd, 0), S.temb(cfgd, 1)
    x = to_dev(x_host, "fp32")
    hero.hero_refresh_block(0, x, to_dev(t0, "fp32"))
    before = {n: hero.hero_state_get(0, n).clone() for n in ("k", "v", "g_attn", "g_ffn")}
    idx = torch.empty(cfg.n_video, dtype=torch.int32, device="cuda")
    n = hero.hero_select_tokens(0, idx)
    rows = idx[:n].cpu().numpy()
    keep = np.setdiff1d(np.arange(cfg.n_rows), rows)
    x2 = to_dev(x_host * 0.5, "fp32")
    hero.hero_refresh_block(0, x2, to_dev(t1, "fp32"), idx[:n])
    for name, b4 in before.items():
        after = hero.hero_state_get(0, name)
        assert torch.equal(after[:, keep], b4[:, keep]), name             # byte-identical reuse
        assert not torch.equal(after[:, rows], b4[:, rows]), name
    # and the refreshed values are the oracle's
    orc.block_refresh(0, np.array(x_host, np.float64), t0, None)
    want_rows = orc.select(0)
    assert np.array_equal(want_rows, rows)
    want = orc.block_refresh(0, np.array(x_host * 0.5, np.float64), t1, want_rows)
    assert rel_l2(to_host(x2), want) <= FP32_TOL
    hero.close()


def test_empty_refresh_list_still_adds_cached_branches():
    cfgd = dict(S.CONFIGS["tiny"], n_blocks=1, n_shallow=1)
    orc, hero, _ = make_pair(cfgd)
    x_host = S.tokens(cfgd)
    x = to_dev(x_host, "fp32")
    hero.hero_refresh_block(0, x, to_dev(S.temb(cfgd, 0), "fp32"))
    g = to_host(hero.hero_state_get(0, "g_attn")) + to_host(hero.hero_state_get(0, "g_ffn"))
    x2 = to_dev(x_host, "fp32")
    empty = torch.empty(0, dtype=torch.int32, device="cuda")
    hero.hero_refresh_block(0, x2, to_dev(S.temb(cfgd, 1), "fp32"), empty, 0)
    assert rel_l2(to_host(x2), x_host + g) <= 1e-6
    hero.close()


def test_call_order_and_argument_errors():
    import paper_2508_17588_b200 as H
    cfgd = S.CONFIGS["tiny"]
    _, hero, _ = make_pair(cfgd)
    x, t = to_dev(S.tokens(cfgd), "fp32"), to_dev(S.temb(cfgd, 0), "fp32")
    with pytest.raises(H.HeroError) as e:
        hero.hero_extrapolate_block(2, x, 1, 1)       # no history yet
    assert e.value.code == -4
    with pytest.raises(H.HeroError) as e:
        hero.hero_extrapolate_block(0, x, 1, 1)       # block 0 is shallow
    assert e.value.code == -1
    idx = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(H.HeroError) as e:
        hero.hero_refresh_block(3, x, t, idx)         # deep block cannot be partially refreshed
    assert e.value.code == -1
    with pytest.raises(H.HeroError) as e:
        hero.hero_refresh_block(0, x[:, :, 1:], t)    # misaligned view
    assert e.value.code == -2
    hero.close()


@pytest.mark.parametrize("name,M,batch,steps,full_at", [
    ("planning_M2", 2, 2, 9, [0, 1, 3, 5, 7]),          # visual planning: the guidance pair, M = 2
    ("planning_M3", 3, 2, 11, [0, 1, 4, 7, 10]),        # M = 3: cached steps with k = 1 and k = 2, gap d = 3
    ("reconstruction_M2", 2, 1, 9, [0, 1, 3, 5, 7]),    # reconstruction: one sequence, no guidance pair
    ("reconstruction_M3", 3, 1, 11, [0, 1, 4, 7, 10])])
def test_paper_hyperparameters_small_model(name, M, batch, steps, full_at):
    """The paper's own settings (Sec. 5.1) in miniature: 2x3 patches, R = 0.2 with round-half-up quotas (one
    token per full patch), three of four blocks refreshed, a full step every M = 2 or 3 steps, with and
    without the guidance pair; through hero_step, every step against the oracle, with the schedule (which
    steps are full, and the k and d the extrapolation therefore uses) checked against the expected list."""
    cfgd = dict(S.CONFIGS["tiny"], frames=2, grid_h=6, grid_w=9, patch_h=2, patch_w=3, ratio_num=1, ratio_den=5,
                quota_mode=1, n_shallow=3, full_interval=M, batch=batch, steps=steps, seed=77)
    orc, hero, _ = make_pair(cfgd)
    cfg = O.Config.from_dict(cfgd)
    assert O.n_selected(cfg, 0) == cfg.n_video // 6
    x_host = S.tokens(cfgd)
    seen_full, seen_kd = [], set()
    for s in range(cfgd["steps"]):
        temb = S.temb(cfgd, s)
        want = orc.step(s, x_host, temb)
        x = to_dev(x_host, "fp32")
        assert hero.hero_is_full_step(s) == orc.is_full_step(s)
        if orc.is_full_step(s):
            seen_full.append(s)
        hero.hero_step(s, x, to_dev(temb, "fp32"))
        assert rel_l2(to_host(x), want) <= FP32_TOL, s
        n_full, s_prev, s_last = (int(v) for v in hero.hero_state_get(0, "steps"))
        assert (n_full, s_last) == (len(seen_full), seen_full[-1])
        if not orc.is_full_step(s):
            seen_kd.add((s - s_last, s_last - s_prev))
        for l in range(cfgd["n_shallow"]):
            assert np.array_equal(hero.hero_state_get(l, "ages").numpy(), orc.blocks[l].ages)
            assert int(hero.hero_state_get(l, "calls")[0]) == orc.blocks[l].calls
    assert seen_full == full_at
    assert seen_kd == ({(1, 1), (1, 2)} if M == 2 else {(1, 1), (2, 1), (1, 3), (2, 3)})
    hero.close()


@pytest.mark.parametrize("variant", [dict(track_mode=1), dict(share_selection=1), dict(track_mode=1, share_selection=1, deep_collapse=1),
                                     dict(attend_mode=1), dict(attend_mode=1, share_selection=1, quota_mode=1),
                                     dict(qk_norm=1), dict(rope=1), dict(qk_norm=1, rope=1, attend_mode=1, has_gate=1)])
def test_tracking_and_selection_variants(variant):
    """Strict oldest-first tracking, one selection list shared by all refresh blocks of a step, both together
    with the collapsed deep stack, attention restricted to the refreshed and text rows, and the base model's
    q/k LayerNorm and rotary embedding: 8 steps through hero_step against the oracle."""
    cfgd = dict(S.CONFIGS["tiny"], n_blocks=5, n_shallow=3, full_interval=3, steps=8, seed=21, **variant)
    orc, hero, _ = make_pair(cfgd)
    x_host = S.tokens(cfgd)
    for s in range(cfgd["steps"]):
        temb = S.temb(cfgd, s)
        want = orc.step(s, x_host, temb)
        x = to_dev(x_host, "fp32")
        hero.hero_step(s, x, to_dev(temb, "fp32"))
        assert rel_l2(to_host(x), want) <= FP32_TOL, s
        for l in range(cfgd["n_shallow"]):
            assert np.array_equal(hero.hero_state_get(l, "ages").numpy(), orc.blocks[l].ages), (s, l)
            assert int(hero.hero_state_get(l, "calls")[0]) == orc.blocks[l].calls
    if variant.get("share_selection"):
        assert orc.blocks[1].calls == 0 and orc.blocks[0].calls > 0       # only block 0's sampler is used
    hero.close()
