"""GPU parity of the deep-stack collapse (hero_config.deep_collapse = 1): the whole deep stack keeps
one fp32 history pair, a cached step applies Eq. 5 to the sums in one pass.  Eq. 5 is linear, so
the plain block-by-block oracle is the reference; tolerances are those of the block-wise path."""
import numpy as np
import pytest
import torch

from oracle import hero_oracle as O
from workloads import synthetic as S
from tests.util import make_pair, rel_l2, to_dev, to_host

pytestmark = pytest.mark.gpu


def H():
    import paper_2508_17588_b200 as h
    return h


def test_tiny_fp32_collapsed_steps_match_oracle():
    cfgd = dict(S.CONFIGS["tiny"], deep_collapse=1, full_interval=4)       # full at 0, 1, 5, 9
    orc, hero, _ = make_pair(cfgd)
    plain = dict(cfgd, deep_collapse=0)
    _, hero_plain, _ = make_pair(plain)
    assert hero.hero_device_bytes() < hero_plain.hero_device_bytes()
    x_host = S.tokens(cfgd)
    for s in range(cfgd["steps"]):
        temb = S.temb(cfgd, s)
        want = orc.step(s, x_host, temb)
        x, xp, t = to_dev(x_host, "fp32"), to_dev(x_host, "fp32"), to_dev(temb, "fp32")
        hero.hero_step(s, x, t)
        hero_plain.hero_step(s, xp, t)
        assert rel_l2(to_host(x), want) <= 2e-5, s
        assert rel_l2(to_host(x), to_host(xp)) <= 2e-6, s                    # the two modes agree to fp32 rounding
        deep = orc.blocks[cfgd["n_shallow"]:]
        want_last = sum(st.g_last[i] for st in deep for i in range(2))
        assert rel_l2(to_host(hero.hero_state_get(0, "stack_last")), want_last) <= 2e-5, s
        if len(orc.full_steps) > 1:
            want_prev = sum(st.g_prev[i] for st in deep for i in range(2))
            assert rel_l2(to_host(hero.hero_state_get(0, "stack_prev")), want_prev) <= 2e-5, s
    hero.close(); hero_plain.close()


SMALL = dict(n_blocks=4, n_shallow=1, hidden=256, n_heads=4, head_dim=64, ffn_dim=768, temb_dim=64, batch=2,
             frames=3, grid_h=9, grid_w=11, n_text=10, patch_h=2, patch_w=2, ratio_num=1, ratio_den=4,
             quota_mode=0, warmup_full_steps=2, full_interval=3, dtype="bf16", has_gate=0, seed=31, steps=7,
             deep_collapse=1)


def test_bf16_collapsed_steps_match_oracle():
    orc, hero, _ = make_pair(SMALL)
    x_host = S.tokens(SMALL)
    for s in range(SMALL["steps"]):                     # full at 0, 1, 4; cached at 2, 3, 5, 6 (k = 1, 2)
        temb = S.temb(SMALL, s)
        want = orc.step(s, x_host, temb)
        x = to_dev(x_host, "bf16")
        hero.hero_step(s, x, to_dev(temb, "bf16"))
        hero.hero_check_status()
        assert rel_l2(to_host(x), want) <= 2e-2, s
        st = orc.blocks[0]                               # teacher-force the shallow block's caches
        for name, ref in (("k", st.k_cache), ("v", st.v_cache), ("g_attn", st.g[0]), ("g_ffn", st.g[1])):
            got = to_host(hero.hero_state_get(0, name))
            assert rel_l2(got, ref) <= 2e-2, (s, name)
            ref[...] = got
    hero.close()


def test_collapsed_extrapolation_alone_and_call_order():
    h = H()
    orc, hero, _ = make_pair(SMALL)
    cfg = O.Config.from_dict(SMALL)
    x = to_dev(S.tokens(SMALL), "bf16")
    t = to_dev(S.temb(SMALL, 0), "bf16")
    for call in (lambda: hero.hero_extrapolate_deep_stack(x, 1, 1),      # no full step yet
                 lambda: hero.hero_extrapolate_block(2, x, 1, 1),        # no per-block history in this mode
                 lambda: hero.hero_refresh_block(2, x, t)):              # deep blocks are driven by hero_step
        with pytest.raises(h.HeroError) as e:
            call()
        assert e.value.code == -4
    # planted histories: Eq. 5 on them, against the oracle's formula
    rng = np.random.default_rng(2)
    prev = rng.standard_normal((cfg.batch, cfg.n_rows, cfg.hidden)).astype(np.float32)
    last = (prev + 0.1 * rng.standard_normal(prev.shape)).astype(np.float32)
    hero.hero_state_set(0, "stack_last", torch.from_numpy(last))
    x0 = to_host(x)
    hero.hero_extrapolate_deep_stack(x, 2, 5)                            # one slot only: Delta = 0 -> reuse
    assert rel_l2(to_host(x), x0 + last) <= 2 ** -8
    # the slot that is not "last" becomes "prev"
    hero.hero_state_set(0, "stack_prev", torch.from_numpy(prev))
    x = to_dev(S.tokens(SMALL), "bf16")
    hero.hero_extrapolate_deep_stack(x, 2, 5)
    assert rel_l2(to_host(x), x0 + O.extrapolate(prev, last, 2, 5)) <= 2 ** -8
    hero.close()
    # a context without the flag refuses the collapsed call
    _, plain, _ = make_pair(dict(SMALL, deep_collapse=0))
    with pytest.raises(h.HeroError) as e:
        plain.hero_extrapolate_deep_stack(x, 1, 1)
    assert e.value.code == -4
    plain.close()
