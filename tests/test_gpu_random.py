"""Seeded random shapes and configurations through the C ABI against the oracle: the tensor-core kernels on shapes
nobody picked by hand, whole steps on small random geometries with random option settings, and the host entry
point against the device entry point."""
import math
import random

import numpy as np
import pytest
import torch

from oracle import hero_oracle as O
from workloads import synthetic as S
from tests.util import make_pair, rel_l2, to_dev, to_host

pytestmark = pytest.mark.gpu

SCORE_SCALE_LOG2 = float(np.float32(0.125) * np.float32(1.4426950408889634))   # log2(e) / sqrt(64)


def H():
    import paper_2508_17588_b200 as h
    return h


def _gelu_tanh(t):
    return 0.5 * t * (1.0 + np.tanh(math.sqrt(2.0 / math.pi) * (t + 0.044715 * t ** 3)))


@pytest.mark.parametrize("seed", range(4))
def test_gemm_random_shapes(seed):
    rnd = random.Random(100 + seed)
    rng = np.random.default_rng(100 + seed)
    for _ in range(10):
        M = rnd.choice([1, 7, 127, 128, 129, 255, 257, rnd.randint(1, 1500)])
        N, K, act = 8 * rnd.randint(1, 160), 8 * rnd.randint(1, 96), rnd.randint(0, 1)
        a = S.round_bf16(rng.standard_normal((M, K)).astype(np.float32))
        w = S.round_bf16((rng.standard_normal((N, K)) / math.sqrt(K)).astype(np.float32))
        b = S.round_bf16(rng.standard_normal(N).astype(np.float32))
        c = torch.full((M, N), float("nan"), device="cuda", dtype=torch.bfloat16)
        H().hero_gemm_bf16(to_dev(a, "bf16"), to_dev(w, "bf16"), to_dev(b, "bf16"), c, act)
        H().hero_isolated_status()
        want = a.astype(np.float64) @ w.astype(np.float64).T + b.astype(np.float64)
        if act:
            want = _gelu_tanh(want)
        got = to_host(c)
        assert np.isfinite(got).all(), (M, N, K, act)
        assert rel_l2(got, want) <= 6e-3, (M, N, K, act)


@pytest.mark.parametrize("seed", range(4))
def test_attention_random_shapes(seed):
    rnd = random.Random(200 + seed)
    rng = np.random.default_rng(200 + seed)
    for _ in range(6):
        B, heads = rnd.randint(1, 3), rnd.randint(1, 3)
        D = heads * 64
        n_q = rnd.choice([1, 31, 128, 129, 256, 257, rnd.randint(1, 600)])
        N = rnd.choice([1, 47, 48, 49, 95, 96, 97, 191, 192, 193, rnd.randint(1, 1500)])
        q = S.round_bf16(rng.standard_normal((B, n_q, D)).astype(np.float32))
        k = S.round_bf16(rng.standard_normal((B, N, D)).astype(np.float32))
        v = S.round_bf16(rng.standard_normal((B, N, D)).astype(np.float32))
        q_scaled = S.round_bf16((q.astype(np.float64) * SCORE_SCALE_LOG2).astype(np.float32))
        cfg = O.Config(n_blocks=1, n_shallow=1, hidden=D, n_heads=heads, head_dim=64, ffn_dim=8, temb_dim=8, batch=B,
                       frames=1, grid_h=1, grid_w=1, n_text=0, patch_h=1, patch_w=1, ratio_num=1, ratio_den=1)
        for entry, q_dev, q_eff in (("hero_attention_bf16", q, q.astype(np.float64)),
                                    ("hero_attention_bf16_safe", q, q.astype(np.float64)),
                                    ("hero_attention_bf16_static", q, q.astype(np.float64)),
                                    ("hero_attention_bf16_q_scaled", q_scaled, q_scaled.astype(np.float64) / SCORE_SCALE_LOG2)):
            o = torch.full((B, n_q, D), float("nan"), device="cuda", dtype=torch.bfloat16)
            getattr(H(), entry)(to_dev(q_dev, "bf16"), to_dev(k, "bf16"), to_dev(v, "bf16"), o, heads)
            H().hero_isolated_status()
            got = to_host(o)
            assert np.isfinite(got).all(), (entry, B, n_q, N, heads)
            for b in range(B):
                want = O.attention(cfg, q_eff[b], k[b].astype(np.float64), v[b].astype(np.float64))
                assert rel_l2(got[b], want) <= 1e-2, (entry, B, n_q, N, heads, b)


def _random_config(rnd, dtype):
    heads = rnd.choice([1, 2, 4])
    n_blocks = rnd.randint(1, 5)
    return dict(n_blocks=n_blocks, n_shallow=rnd.randint(0, n_blocks), hidden=heads * 64, n_heads=heads, head_dim=64,
                ffn_dim=rnd.choice([128, 256, 416]), temb_dim=rnd.choice([32, 64, 128]), batch=rnd.randint(1, 4),
                frames=rnd.randint(1, 4), grid_h=rnd.randint(1, 9), grid_w=rnd.randint(1, 11), n_text=rnd.choice([0, 1, 5, 17]),
                patch_h=rnd.randint(1, 3), patch_w=rnd.randint(1, 3), ratio_num=rnd.randint(1, 4), ratio_den=rnd.randint(4, 9),
                quota_mode=rnd.randint(0, 1), warmup_full_steps=rnd.randint(1, 2), full_interval=rnd.choice([0, 2, 3, 4]),
                dtype=dtype, has_gate=rnd.randint(0, 1), seed=rnd.randint(0, 999), steps=7, track_mode=rnd.randint(0, 1),
                share_selection=rnd.randint(0, 1), attend_mode=rnd.randint(0, 1), qk_norm=rnd.randint(0, 1),
                rope=rnd.randint(0, 1), deep_collapse=rnd.randint(0, 1))


@pytest.mark.parametrize("dtype,tol", [("fp32", 2e-5), ("bf16", 3e-2)])
@pytest.mark.parametrize("seed", range(6))
def test_whole_steps_on_random_small_configurations(seed, dtype, tol):
    """Seven steps of a random small model with random option settings; in fp32 the run is free (each step starts
    from the oracle's previous output), in bf16 every step starts from the same tokens while the caches evolve on
    their own on both sides.  The age counters must agree bit for bit after every step."""
    rnd = random.Random(300 + seed * 2 + (dtype == "bf16"))
    cfgd = _random_config(rnd, dtype)
    orc, hero, _ = make_pair(cfgd)
    x_host = S.tokens(cfgd)
    for s in range(cfgd["steps"]):
        temb = S.temb(cfgd, s)
        want = orc.step(s, x_host, temb)
        x = to_dev(x_host, dtype)
        hero.hero_step(s, x, to_dev(temb, dtype))
        hero.hero_check_status()
        assert rel_l2(to_host(x), want) <= tol, (s, cfgd)
        for l in range(cfgd["n_shallow"]):
            assert np.array_equal(hero.hero_state_get(l, "ages").numpy(), orc.blocks[l].ages), (s, l, cfgd)
        if dtype == "fp32":
            x_host = want.astype(np.float32)
    hero.close()


@pytest.mark.parametrize("seed", range(6))
def test_host_entry_point_equals_device_entry_point_on_random_configurations(seed):
    """hero_step_host (pinned or pageable buffers) against hero_step, bit for bit, six steps."""
    rnd = random.Random(400 + seed)
    dtype = rnd.choice(["fp32", "bf16"])
    cfgd = _random_config(rnd, dtype)
    cfgd.update(hidden=rnd.choice([2, 4, 8]) * 64, grid_h=rnd.randint(2, 12), grid_w=rnd.randint(2, 14), frames=rnd.randint(1, 5))
    cfgd["n_heads"] = cfgd["hidden"] // 64
    weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    _, hero_a, _ = make_pair(cfgd, weights)
    _, hero_b, _ = make_pair(cfgd, weights)
    td = torch.float32 if dtype == "fp32" else torch.bfloat16
    x0 = torch.from_numpy(S.tokens(cfgd)).to(td)
    for s in range(6):
        temb = torch.from_numpy(S.temb(cfgd, s)).to(td)
        xa = x0.cuda()
        hero_a.hero_step(s, xa, temb.cuda())
        hero_a.hero_check_status()
        pinned = rnd.random() < 0.7
        xh = x0.clone().pin_memory() if pinned else x0.clone()
        hero_b.hero_step_host(s, xh, temb.pin_memory() if pinned else temb.clone())
        hero_b.hero_check_status()
        assert torch.equal(xa.cpu(), xh), (s, pinned, cfgd)
    hero_a.close()
    hero_b.close()
