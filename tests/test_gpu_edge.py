"""GPU edge cases of the cached step through the C ABI: empty and full selections, ragged grids,
no text rows, gates, context reuse, call-order and argument errors with a live context."""
import numpy as np
import pytest
import torch

from oracle import hero_oracle as O
from workloads import synthetic as S
from tests.util import make_pair, rel_l2, to_dev, to_host

pytestmark = pytest.mark.gpu

FP32_TOL = 2e-5


def H():
    import paper_2508_17588_b200 as h
    return h


def _run_steps(cfgd, steps, dtype_tol):
    orc, hero, _ = make_pair(cfgd)
    x_host = S.tokens(cfgd)
    outs = []
    for s in range(steps):
        temb = S.temb(cfgd, s)
        want = orc.step(s, x_host, temb)
        x = to_dev(x_host, cfgd["dtype"])
        hero.hero_step(s, x, to_dev(temb, cfgd["dtype"]))
        hero.hero_check_status()
        assert rel_l2(to_host(x), want) <= dtype_tol, s
        for l in range(cfgd["n_shallow"]):
            assert np.array_equal(hero.hero_state_get(l, "ages").numpy(), orc.blocks[l].ages)
        outs.append(x.clone())
    return orc, hero, outs


def test_selection_lists_that_are_sometimes_empty():
    """R = 1/50 on a 2x3x3 grid with 2x2 patches: most calls select nothing, some one token."""
    cfgd = dict(S.CONFIGS["tiny"], frames=2, grid_h=3, grid_w=3, n_text=3, ratio_num=1, ratio_den=50, steps=12, seed=5)
    cfg = O.Config.from_dict(cfgd)
    lens = [O.n_selected(cfg, c) for c in range(10)]
    assert 0 in lens and max(lens) >= 1
    _, hero, _ = _run_steps(cfgd, 12, FP32_TOL)
    hero.close()


@pytest.mark.parametrize("dtype,tol", [("fp32", FP32_TOL), ("bf16", 3e-2)])
def test_no_text_rows_literal_eq3_and_selections_that_are_mostly_empty(dtype, tol):
    """Two video tokens, no text rows, the refreshed rows as the only keys (attend_mode 1) and a ratio that
    selects one token on some calls and none on most: cached steps whose refresh has neither queries nor keys."""
    cfgd = dict(n_blocks=3, n_shallow=2, hidden=256, n_heads=4, head_dim=64, ffn_dim=128, temb_dim=64, batch=4,
                frames=1, grid_h=1, grid_w=2, n_text=0, patch_h=3, patch_w=1, ratio_num=1, ratio_den=5, quota_mode=0,
                warmup_full_steps=1, full_interval=0, dtype=dtype, has_gate=0, seed=1, steps=7, attend_mode=1)
    cfg = O.Config.from_dict(cfgd)
    lens = [O.n_selected(cfg, c) for c in range(6)]
    assert 0 in lens and 1 in lens
    _, hero, _ = _run_steps(cfgd, 7, tol)
    hero.close()


def test_ratio_one_refreshes_every_video_row_bf16():
    cfgd = dict(n_blocks=2, n_shallow=1, hidden=128, n_heads=2, head_dim=64, ffn_dim=256, temb_dim=64, batch=1,
                frames=2, grid_h=5, grid_w=7, n_text=0, patch_h=2, patch_w=3, ratio_num=1, ratio_den=1,
                quota_mode=1, warmup_full_steps=2, full_interval=0, dtype="bf16", has_gate=1, seed=8, steps=4)
    cfg = O.Config.from_dict(cfgd)
    assert O.n_selected(cfg, 0) == cfg.n_video == cfg.n_rows          # no text rows, clipped edge patches
    weights = [S.block_weights(cfgd, l) for l in range(2)]
    orc, hero, _ = make_pair(cfgd, weights)
    x_host = S.tokens(cfgd)
    for s in range(4):
        temb = S.temb(cfgd, s)
        want = orc.step(s, x_host, temb)
        x = to_dev(x_host, "bf16")
        hero.hero_step(s, x, to_dev(temb, "bf16"))
        hero.hero_check_status()
        assert rel_l2(to_host(x), want) <= 2e-2, s
        st = orc.blocks[0]
        for name, ref in (("k", st.k_cache), ("v", st.v_cache), ("g_attn", st.g[0]), ("g_ffn", st.g[1])):
            ref[...] = to_host(hero.hero_state_get(0, name))             # teacher forcing
    hero.close()


def test_batch_three_with_gates_fp32():
    cfgd = dict(S.CONFIGS["tiny"], batch=3, has_gate=1, frames=1, grid_h=7, grid_w=5, n_text=1, steps=5, seed=13)
    _, hero, _ = _run_steps(cfgd, 5, FP32_TOL)
    hero.close()


@pytest.mark.parametrize("batch", [5, 8])
def test_larger_batches_fp32(batch):
    """Batch sizes beyond the workloads' 1 and 2: the adaLN kernel is instantiated for up to 1, 2, 4 and 8 items
    (8 is the most the library takes), and every other kernel derives its row and batch indices from B."""
    cfgd = dict(S.CONFIGS["tiny"], batch=batch, frames=1, grid_h=6, grid_w=5, n_text=3, steps=4, seed=29 + batch)
    _, hero, _ = _run_steps(cfgd, 4, FP32_TOL)
    hero.close()


def test_reset_reproduces_the_run_bit_for_bit_and_contexts_are_independent():
    cfgd = dict(S.CONFIGS["tiny"], steps=5)
    _, hero, first = _run_steps(cfgd, 5, FP32_TOL)
    _, other, _ = make_pair(cfgd)                                      # a second live context on the same weights' values
    hero.hero_reset()
    x_host = S.tokens(cfgd)
    for s in range(5):
        t = to_dev(S.temb(cfgd, s), "fp32")
        x, y = to_dev(x_host, "fp32"), to_dev(x_host, "fp32")
        hero.hero_step(s, x, t)
        other.hero_step(s, y, t)
        assert torch.equal(x, first[s]) and torch.equal(y, first[s]), s
    hero.close(); other.close()


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_cached_step_can_be_captured_in_a_cuda_graph(dtype):
    """A cached step enqueues kernels only (no allocation, no synchronisation, no host read), so a stream
    capture of hero_step yields a graph whose replay does the step's device work: the replayed result equals
    the plainly launched one bit for bit, in the residual stream, the caches and the age counters."""
    cfgd = dict(S.CONFIGS["tiny"], dtype=dtype, hidden=128, n_heads=2)
    weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):                       # the context takes the current stream; capture needs a non-default one
        _, plain, _ = make_pair(cfgd, weights)
        _, graphed, _ = make_pair(cfgd, weights)
        x0 = to_dev(S.tokens(cfgd), dtype)
        for s in range(2):                              # the two full steps, launched plainly on both
            t = to_dev(S.temb(cfgd, s), dtype)
            a, b = x0.clone(), x0.clone()
            plain.hero_step(s, a, t); graphed.hero_step(s, b, t)
        t2 = to_dev(S.temb(cfgd, 2), dtype)
        a, b = x0.clone(), x0.clone()
        plain.hero_step(2, a, t2)
        side.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=side):
            graphed.hero_step(2, b, t2)                 # recorded, not run
        assert torch.equal(b, x0)
        g.replay()
        side.synchronize()
        assert torch.equal(a, b)
        for l in range(cfgd["n_shallow"]):
            assert torch.equal(plain.hero_state_get(l, "ages"), graphed.hero_state_get(l, "ages"))
            for name in ("k", "v", "g_attn", "g_ffn"):
                assert torch.equal(plain.hero_state_get(l, name), graphed.hero_state_get(l, name)), (l, name)
        plain.hero_check_status(); graphed.hero_check_status()
        plain.close(); graphed.close()


@pytest.mark.parametrize("name", ["tiny_fp32", "small_bf16"])
def test_batch_items_in_separate_contexts_reproduce_the_joint_batch(name):
    """The split of a problem's batch over GPUs (one item per rank, no exchange) emulated on one GPU: two
    contexts of batch 1 run one after the other on the two items give the joint context's result bit for
    bit, with the same selection lists."""
    import bench
    if name == "tiny_fp32":
        cfgd = dict(S.CONFIGS["tiny"], batch=2, full_interval=3, steps=6)
    else:
        cfgd = dict(n_blocks=3, n_shallow=2, hidden=256, n_heads=4, head_dim=64, ffn_dim=768, temb_dim=64, batch=2,
                    frames=3, grid_h=9, grid_w=11, n_text=10, patch_h=2, patch_w=2, ratio_num=1, ratio_den=4,
                    quota_mode=0, warmup_full_steps=2, full_interval=3, dtype="bf16", has_gate=0, seed=23, steps=6)
    dt = cfgd["dtype"]
    weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    _, joint, _ = make_pair(cfgd, weights)
    parts = [bench.shard_cfg_pair(cfgd, r, 2) for r in range(2)]
    ranks = [make_pair(c, weights)[1] for c, _ in parts]
    x_host = S.tokens(cfgd)
    for s in range(cfgd["steps"]):
        temb = S.temb(cfgd, s)
        x = to_dev(x_host, dt)
        joint.hero_step(s, x, to_dev(temb, dt))
        for (c, sl), h in zip(parts, ranks):
            y = to_dev(x_host[sl], dt)
            h.hero_step(s, y, to_dev(temb[sl], dt))
            assert torch.equal(y, x[sl]), (s, sl)
            assert torch.equal(h.hero_state_get(0, "ages"), joint.hero_state_get(0, "ages"))
    for h in ranks + [joint]:
        h.hero_check_status(); h.close()


def test_call_order_and_argument_errors_with_a_live_context():
    h = H()
    cfgd = dict(S.CONFIGS["tiny"])
    _, hero, _ = make_pair(cfgd)
    cfg = O.Config.from_dict(cfgd)
    x = to_dev(S.tokens(cfgd), "fp32")
    t = to_dev(S.temb(cfgd, 0), "fp32")
    idx = torch.zeros(cfg.n_video, dtype=torch.int32, device="cuda")

    def code(fn):
        with pytest.raises(h.HeroError) as e:
            fn()
        return e.value.code

    assert code(lambda: hero.hero_step(2, x, t)) == -4                                  # cached step before any full step
    assert code(lambda: hero.hero_refresh_block(0, x, t, idx, 4)) == -4                 # partial refresh before any full pass
    assert code(lambda: hero.hero_refresh_block(0, x, t, idx, 0)) == -4                 # nothing cached yet to add either
    assert code(lambda: hero.hero_extrapolate_block(2, x, 1, 1)) == -4                  # no history yet
    assert code(lambda: hero.hero_extrapolate_block(0, x, 1, 1)) == -1                  # block 0 is a refresh block
    assert code(lambda: hero.hero_extrapolate_block(2, x, 1, 0)) == -1                  # d = 0
    assert code(lambda: hero.hero_refresh_block(9, x, t)) == -1                         # no such block
    assert code(lambda: hero.hero_refresh_block(0, x, t, idx, cfg.n_rows + 1)) == -1    # list longer than the sequence
    assert code(lambda: hero.hero_refresh_block(3, x, t, idx, 4)) == -1                 # partial refresh of a deep block
    assert code(lambda: hero.hero_select_tokens(2, idx)) == -1                          # selection on a deep block
    assert code(lambda: hero.hero_select_tokens(0, idx[:3])) == -3                      # capacity
    misaligned = torch.zeros(x.numel() + 1, device="cuda")[1:].view_as(x)
    assert code(lambda: hero.hero_step(0, misaligned, t)) == -2
    # none of the refused calls changed any state: the run still matches a fresh context
    _, fresh, _ = make_pair(cfgd)
    for s in range(3):
        ts = to_dev(S.temb(cfgd, s), "fp32")
        a, b = to_dev(S.tokens(cfgd), "fp32"), to_dev(S.tokens(cfgd), "fp32")
        hero.hero_step(s, a, ts)
        fresh.hero_step(s, b, ts)
        assert torch.equal(a, b)
    assert int(hero.hero_state_get(0, "calls")[0]) == 1
    hero.close(); fresh.close()


def test_many_contexts_do_not_leak_device_memory():
    cfgd = dict(S.CONFIGS["tiny"])
    _, hero, w = make_pair(cfgd)
    hero.close()
    torch.cuda.synchronize()
    free0 = torch.cuda.mem_get_info()[0]
    for _ in range(20):
        _, hero, _ = make_pair(cfgd, w)
        x = to_dev(S.tokens(cfgd), "fp32")
        hero.hero_step(0, x, to_dev(S.temb(cfgd, 0), "fp32"))
        hero.close()
        del x
    torch.cuda.synchronize()
    torch.cuda.empty_cache()
    assert torch.cuda.mem_get_info()[0] >= free0 - (8 << 20)


def test_partial_refresh_needs_a_full_pass_or_planted_caches():
    """Eq. 3 merges fresh rows with the block's cache: until the block has had a full pass (or all four
    caches were planted) a partial refresh is a call-order error, and hero_reset brings that state back."""
    h = H()
    cfgd = dict(S.CONFIGS["tiny"])
    _, hero, _ = make_pair(cfgd)
    cfg = O.Config.from_dict(cfgd)
    x = to_dev(S.tokens(cfgd), "fp32")
    t = to_dev(S.temb(cfgd, 0), "fp32")
    idx = torch.arange(cfg.n_text, cfg.n_text + 8, dtype=torch.int32, device="cuda")

    def code(fn):
        with pytest.raises(h.HeroError) as e:
            fn()
        return e.value.code

    assert code(lambda: hero.hero_refresh_block(0, x, t, idx)) == -4
    zeros = torch.zeros(cfg.batch, cfg.n_rows, cfg.hidden)
    for name in ("k", "v", "g_attn"):
        hero.hero_state_set(0, name, zeros)
    assert code(lambda: hero.hero_refresh_block(0, x, t, idx)) == -4                    # G_ffn still missing
    hero.hero_state_set(0, "g_ffn", zeros)
    hero.hero_refresh_block(0, x, t, idx)                                               # all four planted: fine
    hero.hero_reset()
    assert code(lambda: hero.hero_refresh_block(0, x, t, idx)) == -4
    hero.hero_refresh_block(0, x, t)                                                    # full pass
    hero.hero_refresh_block(0, x, t, idx)
    hero.hero_refresh_block(0, x, t, idx, 0)
    hero.hero_check_status()
    hero.close()


def test_a_wait_that_runs_out_is_reported_once_and_the_next_calls_are_healthy():
    """The give-up path, made to happen harmlessly: one thread block waits 50 microseconds on a barrier
    nobody completes, through the helper the tensor-core kernels use; it must raise the status word and
    RETURN.  The host then reports HERO_ERR_TIMEOUT exactly once, and the kernels that share the word run
    normally afterwards."""
    h = H()
    # the isolated calls' word
    h.hero_isolated_status()
    h.hero_selftest_wait_timeout(50)
    with pytest.raises(h.HeroError) as e:
        h.hero_isolated_status()
    assert e.value.code == -6
    h.hero_isolated_status()                                          # the word was cleared by the report
    g = torch.Generator(device="cuda").manual_seed(3)
    q, k, v = (torch.randn(1, n, 64, device="cuda", generator=g).bfloat16() for n in (70, 200, 200))
    o = torch.full_like(q, float("nan"))
    h.hero_attention_bf16(q, k, v, o, 1)
    h.hero_isolated_status()
    want = torch.softmax(q.float()[0] @ k.float()[0].T / 8.0, -1) @ v.float()[0]
    assert float((o.float()[0] - want).norm() / want.norm()) <= 1e-2
    # a context's word
    cfgd = dict(n_blocks=1, n_shallow=1, hidden=128, n_heads=2, head_dim=64, ffn_dim=256, temb_dim=64, batch=1,
                frames=1, grid_h=4, grid_w=4, n_text=2, patch_h=2, patch_w=2, ratio_num=1, ratio_den=4,
                quota_mode=0, warmup_full_steps=2, full_interval=0, dtype="bf16", has_gate=0, seed=2, steps=3)
    orc, hero, _ = make_pair(cfgd)
    hero.hero_check_status()
    hero.hero_selftest_wait_timeout(50)
    with pytest.raises(h.HeroError) as e:
        hero.hero_check_status()
    assert e.value.code == -6
    hero.hero_check_status()
    x_host = S.tokens(cfgd)
    for s in range(3):
        temb = S.temb(cfgd, s)
        want = orc.step(s, x_host, temb)
        x = to_dev(x_host, "bf16")
        hero.hero_step(s, x, to_dev(temb, "bf16"))
        hero.hero_check_status()
        assert rel_l2(to_host(x), want) <= 3e-2, s
    hero.close()
