#!/usr/bin/env python
"""Benchmark of the HERO cached DiT step on B200.

One "step" is one cached denoising step of the 42-block CogVideoX-5B-shaped DiT (config
"dit42": 14 refresh blocks at 25 % + 28 extrapolated blocks, B=2 x N=17776 tokens, bf16):
token selection, gather+LN, QKV/attention/out-proj/FFN on the refreshed rows with the merge
into the caches, residual adds, and linear extrapolation in the deep blocks.  The two warm-up
full steps that fill the caches are set-up, not timed; a full step is timed once and reported
in `config` together with the 50-step schedule average.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl hero|reference] [--workload dit42|aether|paper_hp|paper_hp_m3|paper_recon|paper_recon_m3|block|tiny|kernels [--only LIST] [--small]]

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs its own sequence on its
own GPU (independent problems, no data-path collective): "scaling": "weak".  `--cfg-split` instead
gives each rank batch/N items of one problem (the guidance pair, one item per GPU at N = 2; the ranks draw
the same selection lists on their own, nothing is exchanged): "scaling": "strong".
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from workloads import synthetic as S  # noqa: E402

METRIC = "hero_cached_step_tokens_per_s"
ATTENTION_TRAFFIC_RATIO = 1.002   # dram__bytes_read+write / algorithmic bytes of tc_attention_fast_kernel<1> (ncu, small case: 0.998-1.006)
UNIT = "tokens/s"
NOMINAL_BF16_TFLOPS = 2250.0      # dense bf16, the figure the 60 % target is stated against
NOMINAL_HBM_GBS = 8000.0          # the figure the 70 % target is stated against


# --------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons during the timed region (read-only queries)."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
            t0 = time.time()
            while not self.lines and time.time() - t0 < 2.0:      # the first sample marks the loop as running
                time.sleep(0.01)
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def refresh_flops(cfg, n_sel):
    """Algorithmic flops of one refresh block on n = B*n_sel rows."""
    B, D, F = cfg["batch"], cfg["hidden"], cfg["ffn_dim"]
    N = S.n_rows(cfg)
    n = B * n_sel
    return dict(gemm=2 * n * D * 3 * D + 2 * n * D * D + 4 * n * D * F, attention=4 * n * N * D)


# --------------------------------------------------------------------------- CPU baseline (oracle)
class OracleSample:
    """The CPU oracle, as it stands, on a bounded sample of one cached step, scaled to a whole
    step.  Sample: one shallow block refreshed on its real selection with the K/V rewrite of every
    selected row and the branch outputs of `sample_rows` of them, and one deep block's
    extrapolation over the full tensor; a cached step is n_shallow times the first (outputs
    scaled to all selected rows) plus n_deep times the second.  Caches hold synthetic values."""

    def __init__(self, cfg):
        from oracle import hero_oracle as O
        self.cfg = cfg
        one = dict(cfg, n_blocks=2, n_shallow=1)
        w = [S.block_weights(one, 0)]
        w.append(w[0])
        self.orc = O.HeroOracle(O.Config.from_dict(one), w)
        B, N, D = cfg["batch"], S.n_rows(cfg), cfg["hidden"]
        rng = np.random.default_rng(0)
        st = self.orc.blocks[0]
        st.k_cache, st.v_cache = rng.standard_normal((B, N, D)), rng.standard_normal((B, N, D))
        st.g = [rng.standard_normal((B, N, D)), rng.standard_normal((B, N, D))]
        dp = self.orc.blocks[1]
        dp.g_prev = [st.k_cache, st.v_cache]          # any full-size tensors do for timing
        dp.g_last = [st.g[0], st.g[1]]
        self.x = rng.standard_normal((B, N, D))
        self.temb = S.temb(one, 2)

    def step_seconds(self, sample_rows=256):
        orc, cfg = self.orc, self.cfg
        t0 = time.perf_counter()
        rows = orc.select(0)
        t_sel = time.perf_counter() - t0
        sample_rows = min(sample_rows, len(rows))
        small = max(sample_rows // 4, 1)
        t0 = time.perf_counter()
        orc.block_refresh(0, self.x, self.temb, rows, rows_out=rows[:sample_rows])
        t_a = time.perf_counter() - t0
        # the same with a quarter of the sample separates the fixed part from the per-row part
        t0 = time.perf_counter()
        orc.block_refresh(0, self.x, self.temb, rows, rows_out=rows[:small])
        t_b = time.perf_counter() - t0
        per_row = max(t_a - t_b, 0.0) / max(sample_rows - small, 1)
        fixed = max(t_a - per_row * sample_rows, 0.0)
        t_refresh = t_sel + fixed + per_row * len(rows)
        t0 = time.perf_counter()
        orc.block_extrapolate(1, self.x, 1, 5)
        t_ext = time.perf_counter() - t0
        n_sh, n_dp = cfg["n_shallow"], cfg["n_blocks"] - cfg["n_shallow"]
        total = n_sh * t_refresh + n_dp * t_ext
        detail = dict(select_s=t_sel, refresh_fixed_s=fixed, refresh_per_row_s=per_row, n_sel=int(len(rows)),
                      extrapolate_block_s=t_ext, cpu_work_s=t_sel + t_a + t_b + t_ext)
        return total, detail


ORACLE_SAMPLE_ROWS = 128      # rows whose branch outputs the oracle computes per sampled step (both arms)
ORACLE_SAMPLE_TEXT = ("one shallow block refreshed on its real selection (K/V of every selected row, branch outputs of "
                      "%d rows, scaled to all) + one deep block extrapolated, scaled by block counts" % ORACLE_SAMPLE_ROWS)


def cpu_cores_used():
    try:
        from threadpoolctl import threadpool_info
        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
        return int(n)
    except Exception:
        return os.cpu_count() or 1


def workload_config(args, cfg) -> dict:
    """The part of `config` that names the workload; both arms print the same keys."""
    return {"workload": args.workload, "blocks": cfg["n_blocks"], "refresh_blocks": cfg["n_shallow"],
            "refresh_ratio": cfg["ratio_num"] / cfg["ratio_den"], "batch": cfg["batch"],
            "tokens_per_seq": S.n_rows(cfg), "hidden": cfg["hidden"]}


def run_reference(args, cfg, rank, world):
    """Reference arm: the oracle on this machine's host cores, on bounded samples of the same workload."""
    if rank != 0:
        return
    tokens = cfg["batch"] * S.n_rows(cfg)
    vals = []
    sample_obj = OracleSample(cfg)
    for i in range(args.warmup + args.steps):
        sec, detail = sample_obj.step_seconds(sample_rows=ORACLE_SAMPLE_ROWS)
        if i >= args.warmup:
            vals.append(sec)
    sec = statistics.mean(vals)
    sample = "per step: " + ORACLE_SAMPLE_TEXT
    line = {"impl": "reference", "metric": METRIC, "value": tokens / sec, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": dict(workload_config(args, cfg), note="oracle (numpy float64) timed on host cores"),
            "cpu_baseline": {"value": tokens / sec, "unit": UNIT, "cores": cpu_cores_used(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": tokens / sec, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# --------------------------------------------------------------------------- multi-rank plumbing
def max_over_ranks(value: float, dist, device) -> float:
    """A timing is the slowest rank's (works on any backend: the tensor lives where `device` says)."""
    if dist is None:
        return float(value)
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_throughput(tokens_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Independent sequences, one per rank (weak scaling): units of all ranks over the slowest rank's time."""
    return world * tokens_per_rank_step / (ms_per_step * 1e-3)


def shard_cfg_pair(cfg: dict, rank: int, world: int):
    """The items of one problem's batch (the classifier-free-guidance pair) split over the ranks: every rank
    keeps the seed, hence the same selection lists, and runs batch/world sequences; nothing is exchanged.
    Returns the rank's config and its slice of the batch axis."""
    if world < 1 or not 0 <= rank < world or cfg["batch"] % world:
        raise ValueError(f"batch {cfg['batch']} does not split over {world} ranks")
    per = cfg["batch"] // world
    return dict(cfg, batch=per), slice(rank * per, (rank + 1) * per)


def rank_seed(base_seed: int, rank: int) -> int:
    """Each rank draws its own problem."""
    return base_seed + rank


# --------------------------------------------------------------------------- CUDA arm
def build_device_weights(cfg, device):
    dt = torch.bfloat16 if cfg["dtype"] == "bf16" else torch.float32
    weights = []
    for l in range(cfg["n_blocks"]):
        blk = {}
        for name, shape in S.weight_shapes(cfg).items():
            t = S.device_normal(cfg["seed"], name, shape, 0.02, l, None, device)
            if name in ("qn_w", "kn_w"):
                t = t + 1.0                       # LayerNorm gains sit around one
            blk[name] = t.to(dt).contiguous()
        weights.append(blk)
    return weights


def run_hero(args, cfg, rank, world, local_rank):
    import paper_2508_17588_b200 as H
    H.load()                                     # fails loudly if the CUDA library is missing
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path for the product arm")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=device)
    dt = torch.bfloat16 if cfg["dtype"] == "bf16" else torch.float32
    run_cfg = dict(cfg, full_interval=0)         # after the two warm-up full steps every step is cached
    B_all, N, D = cfg["batch"], S.n_rows(cfg), cfg["hidden"]
    if args.cfg_split:
        # one problem, its batch items split over the ranks (strong scaling, no exchange)
        run_cfg, part = shard_cfg_pair(run_cfg, rank, world)
    else:
        run_cfg["seed"] = rank_seed(cfg["seed"], rank)   # each rank its own sequence (independent problems)
        part = slice(0, B_all)
    weights = build_device_weights(run_cfg, device)
    hero = H.Hero(run_cfg, weights)
    B = run_cfg["batch"]
    tokens = B * N
    x = S.device_normal(run_cfg["seed"], "x0", (B_all, N, D), 1.0, 0, None, device).to(dt)[part].contiguous()
    tembs = [S.device_normal(run_cfg["seed"], "temb", (B_all, cfg["temb_dim"]), 1.0, s, None, device).to(dt)[part].contiguous()
             for s in range(8)]

    def ev():
        return torch.cuda.Event(enable_timing=True)

    # set-up: the two "initial caching" full steps; the second one is timed for the record
    hero.hero_step(0, x, tembs[0])
    e0, e1 = ev(), ev()
    torch.cuda.synchronize()
    e0.record()
    hero.hero_step(1, x, tembs[1])
    e1.record()
    torch.cuda.synchronize()
    full_ms = e0.elapsed_time(e1)
    hero.hero_check_status()

    step = 2
    for _ in range(args.warmup):
        hero.hero_step(step, x, tembs[step % 8]); step += 1
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    sampler = ClockSampler(torch.cuda.current_device() if "CUDA_VISIBLE_DEVICES" not in os.environ else local_rank)
    sampler.start()
    launches0 = hero.hero_launch_count()
    torch.cuda.synchronize()
    e0, e1 = ev(), ev()
    e0.record()
    for _ in range(args.steps):
        hero.hero_step(step, x, tembs[step % 8]); step += 1
    e1.record()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    total_ms = e0.elapsed_time(e1)
    launches = hero.hero_launch_count() - launches0
    clocks = sampler.stop()
    hero.hero_check_status()
    total_ms = max_over_ranks(total_ms, dist, device)
    ms_per_step = total_ms / args.steps
    value = whole_job_throughput(tokens, world, ms_per_step)

    # per-category device time over two more cached steps (events around every launch)
    n_prof = 2
    hero.hero_profile_begin()
    n_sel_seen = []
    for _ in range(n_prof):
        n_sel_seen.append(hero.hero_next_n_sel(0) if cfg["n_shallow"] else 0)
        hero.hero_step(step, x, tembs[step % 8]); step += 1
    prof = hero.hero_profile_end()
    breakdown = {k: {"ms_per_step": v[0] / n_prof, "launches_per_step": v[1] / n_prof} for k, v in prof.items()}
    peaks = measured_peaks()
    roofline = None
    if cfg["n_shallow"] and prof["attention"][1]:
        n_sel = statistics.mean(n_sel_seen)
        fl = refresh_flops(run_cfg, n_sel)
        att_ms = prof["attention"][0] / prof["attention"][1]
        gemm_ms_blk = prof["gemm"][0] / prof["attention"][1]          # four GEMMs per attention launch
        achieved = fl["attention"] / (att_ms * 1e-3) / 1e12
        peak = peaks["bf16_tflops_sustained"]
        # DRAM bytes per launch: an ncu capture of a smaller launch of this kernel read and wrote 1.005 x its
        # algorithmic bytes (K and V once, Q in, O out); the traffic grows in proportion with those, so the
        # full launch is that ratio times its own algorithmic bytes
        alg_bytes = 2 * B * N * D * 2 + 2 * B * n_sel * D * 2
        gemm_tf = fl["gemm"] / (gemm_ms_blk * 1e-3) / 1e12
        roofline = {"kernel": "tc_attention_fast_kernel", "bound": "tensor", "achieved": achieved, "peak": peak,
                    "unit": "TFLOP/s", "frac": achieved / peak, "frac_of_burst": achieved / peaks["bf16_tflops"],
                    "frac_of_2250": achieved / NOMINAL_BF16_TFLOPS, "traffic": ATTENTION_TRAFFIC_RATIO * alg_bytes,
                    "traffic_source": "ncu small case (profiles/tc_attention_small_q768.md) scaled by algorithmic bytes",
                    "peak_source": peaks["source"] + " (sustained cuBLAS bf16)",
                    "flops_per_launch": fl["attention"], "ms_per_launch": att_ms,
                    "gemm": {"achieved": gemm_tf, "unit": "TFLOP/s", "frac": gemm_tf / peak,
                             "frac_of_burst": gemm_tf / peaks["bf16_tflops"], "frac_of_2250": gemm_tf / NOMINAL_BF16_TFLOPS,
                             "flops_per_block": fl["gemm"], "ms_per_block": gemm_ms_blk},
                    "refresh_block": {"achieved": (fl["gemm"] + fl["attention"]) / ((gemm_ms_blk + att_ms) * 1e-3) / 1e12,
                                      "unit": "TFLOP/s",
                                      "frac": (fl["gemm"] + fl["attention"]) / ((gemm_ms_blk + att_ms) * 1e-3) / 1e12 / peak,
                                      "frac_of_2250": (fl["gemm"] + fl["attention"]) / ((gemm_ms_blk + att_ms) * 1e-3) / 1e12
                                                      / NOMINAL_BF16_TFLOPS,
                                      "note": "the four GEMMs and the attention of one refresh block together"}}
        if breakdown["extrapolate"]["launches_per_step"]:
            # all deep blocks in one pass per launch: four history tensors read per block, x read and written
            # once per launch
            n_deep = cfg["n_blocks"] - cfg["n_shallow"]
            ext_ms = prof["extrapolate"][0] / n_prof
            ext_bytes = B * N * D * 2 * (4 * n_deep + 2 * breakdown["extrapolate"]["launches_per_step"])
            gbs = ext_bytes / (ext_ms * 1e-3) / 1e9
            roofline["extrapolate"] = {"achieved": gbs, "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                                       "frac_of_8tbs": gbs / NOMINAL_HBM_GBS,
                                       "ms_per_step": ext_ms, "bytes_per_step": ext_bytes, "blocks": n_deep}

    # end to end through the host entry point: pinned host buffers, H2D + step + D2H per call
    h_x = x.detach().cpu().pin_memory()
    h_t = tembs[0].detach().cpu().pin_memory()
    n_e2e = max(2, min(args.steps, 5))
    hero.hero_step_host(step, h_x, h_t); step += 1
    torch.cuda.synchronize()
    first_rows = []                      # rows the first refresh block reads straight from the pinned buffer
    t0 = time.perf_counter()
    for _ in range(n_e2e):
        first_rows.append(hero.hero_next_n_sel(0) if cfg["n_shallow"] else 0)
        hero.hero_step_host(step, h_x, h_t); step += 1
    e2e_s = (time.perf_counter() - t0) / n_e2e
    e2e_s = max_over_ranks(e2e_s, dist, device)
    xb = h_x.numel() * h_x.element_size()
    tb = h_t.numel() * h_t.element_size()
    zero_copy = int(statistics.mean(first_rows) * B * D * h_x.element_size())
    e2e = {"value": whole_job_throughput(tokens, world, e2e_s * 1e3), "unit": UNIT, "ms_per_step": e2e_s * 1e3,
           "h2d_bytes_per_step": xb + tb + zero_copy, "d2h_bytes_per_step": xb,
           "h2d_copy_bytes_per_step": xb + tb, "h2d_zero_copy_bytes_per_step": zero_copy,
           "note": "h2d = the upload of x and temb plus the rows of x that the first refresh block's LayerNorm reads "
                   "directly from the pinned host buffer over PCIe while the upload is under way"}
    hero.hero_check_status()
    mem = hero.hero_device_bytes()
    hero.close()

    # the same cached step under two opt-in variants (reported beside the headline, never as it)
    def time_variant(extra, w=None):
        hv = H.Hero(dict(run_cfg, **extra), w or weights)
        for s_ in range(2):
            hv.hero_step(s_, x, tembs[s_])
        st = 2
        for _ in range(args.warmup):
            hv.hero_step(st, x, tembs[st % 8]); st += 1
        n_c = max(2, min(args.steps, 5))
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(n_c):
            hv.hero_step(st, x, tembs[st % 8]); st += 1
        e1.record()
        torch.cuda.synchronize()
        hv.hero_check_status()
        v_ms = max_over_ranks(e0.elapsed_time(e1) / n_c, dist, device)
        out = {"ms_per_step": v_ms, "value": whole_job_throughput(tokens, world, v_ms), "unit": UNIT,
               "device_bytes": hv.hero_device_bytes()}
        hv.close()
        return out

    collapsed = attend_refreshed = base_qk = None
    if not args.no_collapse:
        if cfg["n_shallow"] < cfg["n_blocks"]:
            collapsed = time_variant(dict(deep_collapse=1))
            collapsed["note"] = "deep_collapse=1: Eq. 5 applied once to the fp32 sum of the deep blocks' branch outputs"
        if cfg["n_shallow"] > 0:
            attend_refreshed = time_variant(dict(attend_mode=1))
            attend_refreshed["note"] = ("attend_mode=1: the refreshed queries of a cached step attend to the refreshed "
                                        "and text rows only (Eq. 3 read literally) instead of the full cached K/V")
            hd = cfg["head_dim"]
            w_qk = [dict(blk, qn_w=torch.ones(hd, device=device, dtype=dt), qn_b=torch.zeros(hd, device=device, dtype=dt),
                         kn_w=torch.ones(hd, device=device, dtype=dt), kn_b=torch.zeros(hd, device=device, dtype=dt))
                    for blk in weights]
            base_qk = time_variant(dict(qk_norm=1, rope=1), w_qk)
            base_qk["note"] = ("qk_norm=1, rope=1: the base model's per-head LayerNorm and 3-D rotary embedding of the "
                               "fresh q and k rows (one extra HBM-bound pass per refresh block)")

    kernels_record = None
    if rank == 0 and world == 1 and not args.no_kernels:
        recs, k_clocks = config2_kernels(H, device, measured_peaks(), iters=20, warm=3)
        kernels_record = {"workload": "isolated kernels on [2, 17776, 3072] bf16, index lists at 10/25/50 % of a 13x30x45 "
                                      "grid (2x2 patches)",
                          "timing": "each kernel alone, CUDA events, median of 20 calls, L2 flushed before every call",
                          "clocks": k_clocks, "kernels": recs}

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        del weights
        torch.cuda.empty_cache()
        # the same sample and estimator as `--impl reference`: one untimed pass (BLAS threads, page faults), then
        # the mean of two
        smp = OracleSample(cfg)
        smp.step_seconds(sample_rows=ORACLE_SAMPLE_ROWS)
        runs = [smp.step_seconds(sample_rows=ORACLE_SAMPLE_ROWS) for _ in range(2)]
        sec = statistics.mean(r[0] for r in runs)
        cpu_baseline = {"value": tokens / sec, "unit": UNIT, "cores": cpu_cores_used(), "kind": "oracle",
                        "sample": ORACLE_SAMPLE_TEXT + "; mean of 2 samples after 1 untimed, "
                                  f"{sum(r[1]['cpu_work_s'] for r in runs):.1f} s of timed CPU work",
                        "ms_per_step": sec * 1e3}

    if rank == 0:
        n_full = sum(1 for s in range(cfg["steps"])
                     if s < cfg["warmup_full_steps"] or
                     (cfg["full_interval"] > 0 and (s - (cfg["warmup_full_steps"] - 1)) % cfg["full_interval"] == 0))
        sched_ms = (n_full * full_ms + (cfg["steps"] - n_full) * ms_per_step) / cfg["steps"]
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "strong" if args.cfg_split and world > 1 else "weak",
                "vs_baseline": None, "dtype": cfg["dtype"], "data": "synthetic",
                "config": dict(workload_config(args, cfg),
                               l2="inputs larger than L2 (each step streams > 30 GB of caches)",
                               full_step_ms=full_ms, schedule_avg_ms_per_step=sched_ms,
                               schedule="%d full + %d cached of %d steps" % (n_full, cfg["steps"] - n_full, cfg["steps"]),
                               device_bytes=mem,
                               parallelism=("cfg_split" if args.cfg_split else "replicas") if world > 1 else "single"),
                "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "breakdown_ms": breakdown}
        if collapsed:
            line["deep_collapse_variant"] = collapsed
        if attend_refreshed:
            line["attend_refreshed_variant"] = attend_refreshed
        if base_qk:
            line["qk_norm_rope_variant"] = base_qk
        if roofline:
            # the same launch against the exponential unit: one ex2 per score, 16 per clock per SM (measured on
            # this chip), at the SM clock sampled during the timed region
            if clocks.get("sm_mhz") and cfg["head_dim"] == 64:
                sms = torch.cuda.get_device_properties(device).multi_processor_count
                exps = roofline["flops_per_launch"] / (4.0 * cfg["head_dim"])      # 4 * head_dim flop per score
                peak_exp = 16.0 * sms * clocks["sm_mhz"] * 1e6
                ach_exp = exps / (roofline["ms_per_launch"] * 1e-3)
                roofline["exp_unit"] = {"achieved": ach_exp / 1e12, "peak": peak_exp / 1e12, "unit": "Texp/s",
                                        "frac": ach_exp / peak_exp,
                                        "note": "secondary bound of the attention kernel at head_dim 64"}
            line["roofline"] = roofline
        if kernels_record:
            line["kernels"] = kernels_record
        if cpu_baseline:
            line["cpu_baseline"] = cpu_baseline
        print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


# --------------------------------------------------------------------------- isolated kernels
def _time_flushed(fn, iters, warmup, flush):
    """Median device time (ms) of fn() with L2 flushed before each call: a write larger than L2, then a
    read of the same buffer so that what L2 is left holding is clean (evicting it costs no write-back)."""
    ts = []
    for i in range(warmup + iters):
        flush.zero_()
        flush.max()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        e1.synchronize()
        if i >= warmup:
            ts.append(e0.elapsed_time(e1))
    return statistics.median(ts)



def config2_kernels(H, dev, peaks, iters=20, warm=3, want=None):
    """The isolated-kernel workload (feature cache [2, 17776, 3072] bf16, index lists at 10 / 25 / 50 % drawn by
    the library's own sampler on the 13x30x45 grid with 2x2 patches): Eq. 5 alone, row gather and scatter, and
    the gather + LayerNorm + modulate prologue, each timed alone with CUDA events, L2 flushed before every call,
    median of `iters` calls, clocks sampled over the whole group.  Returns (records, clocks)."""
    want = want or (lambda name: True)
    cfg = dict(S.CONFIGS["kernels"])
    B, N, D = cfg["batch"], S.n_rows(cfg), cfg["hidden"]
    bf = torch.bfloat16
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    out = {}

    def rnd(*shape, std=1.0):
        return (torch.randn(*shape, device=dev) * std).to(bf)

    def hbm(name, ms, nbytes, **extra):
        gbs = nbytes / (ms * 1e-3) / 1e9
        out[name] = dict(ms=ms, bytes=nbytes, achieved=gbs, unit="GB/s", frac=gbs / peaks["hbm_gbs"],
                         frac_of_8tbs=gbs / NOMINAL_HBM_GBS, bound="hbm", **extra)

    # index lists from the library's own sampler (a context with a one-head block: only geometry matters)
    lists = {}
    small_cfg = dict(cfg, hidden=64, n_heads=1, ffn_dim=64, temb_dim=64, n_blocks=1, n_shallow=1)
    w = [{k: torch.zeros(s_, device=dev, dtype=bf) for k, s_ in S.weight_shapes(small_cfg).items()}]
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    for num, den in ((1, 10), (1, 4), (1, 2)):
        hero = H.Hero(dict(small_cfg, ratio_num=num, ratio_den=den), w)
        idx = torch.empty(S.n_video(cfg), dtype=torch.int32, device=dev)
        n = hero.hero_select_tokens(0, idx)
        lists[f"{num}/{den}"] = idx[:n].clone()
        if want("select") and (num, den) == (1, 4):
            ms = _time_flushed(lambda: hero.hero_select_tokens(0, idx), iters, warm, flush)
            out["select_25"] = dict(ms=ms, tokens=S.n_video(cfg), bound="latency",
                                    note="integer work on 35 KB of counters; no bandwidth figure applies")
        hero.close()
    if want("extrapolate"):
        a, b_, o = rnd(B, N, D), rnd(B, N, D), torch.empty(B, N, D, device=dev, dtype=bf)
        hbm("extrapolate", _time_flushed(lambda: H.hero_extrapolate(a, b_, o, 4, 5), iters, warm, flush), 3 * a.numel() * 2)
        del a, b_, o
    if want("gather") or want("scatter") or want("gather_ln"):
        src = rnd(B, N, D)
        add = rnd(B, N, D, std=0.3)
        mod = torch.randn(B, 4 * D, device=dev) * 0.5
        for key, idx in lists.items():
            comp = torch.empty(B, idx.numel(), D, device=dev, dtype=bf)
            nbytes = 2 * B * idx.numel() * D * 2 + 4 * idx.numel()
            if want("gather"):
                hbm(f"gather_{key}", _time_flushed(lambda: H.hero_gather_rows(src, idx, comp), iters, warm, flush),
                    nbytes, rows=idx.numel())
            if want("scatter"):
                hbm(f"scatter_{key}", _time_flushed(lambda: H.hero_scatter_rows(comp, idx, src), iters, warm, flush),
                    nbytes, rows=idx.numel())
            if want("gather_ln"):
                # the prologue of the attention branch (rows in, rows out) and of the FFN branch (two rows in)
                hbm(f"gather_ln_{key}", _time_flushed(
                    lambda: H.hero_gather_ln_modulate(src, None, idx, mod[:, :D], mod[:, D:2 * D], comp), iters, warm, flush),
                    nbytes, rows=idx.numel())
                hbm(f"gather_ln_add_{key}", _time_flushed(
                    lambda: H.hero_gather_ln_modulate(src, add, idx, mod[:, :D], mod[:, D:2 * D], comp), iters, warm, flush),
                    nbytes + B * idx.numel() * D * 2, rows=idx.numel())
        del src, add
    torch.cuda.synchronize()
    clocks = sampler.stop()
    return out, clocks

def run_kernels(args):
    """Each kernel of the cached step alone, at the shapes of the isolated-kernel and one-block
    workloads ([2, 17776, 3072] bf16, index lists at 10/25/50 %), against its own roofline.
    `--small` shrinks the tensor-core cases to what a profiler capture handles in seconds."""
    import paper_2508_17588_b200 as H
    H.load()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU path for the product arm")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks = measured_peaks()
    cfg = dict(S.CONFIGS["kernels"])
    B, N, D, F = cfg["batch"], S.n_rows(cfg), cfg["hidden"], cfg["ffn_dim"]
    heads = cfg["n_heads"]
    only = set(args.only.split(",")) if args.only else None
    want = lambda name: only is None or name in only
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    iters, warm = max(args.steps, 5), max(args.warmup, 3)        # default 20 calls per kernel, median
    bf = torch.bfloat16
    out = {}

    def rnd(*shape, std=1.0):
        return (torch.randn(*shape, device=dev) * std).to(bf)

    def hbm(name, ms, nbytes, **extra):
        gbs = nbytes / (ms * 1e-3) / 1e9
        out[name] = dict(ms=ms, bytes=nbytes, achieved=gbs, unit="GB/s", frac=gbs / peaks["hbm_gbs"],
                         frac_of_8tbs=gbs / 8000.0, bound="hbm", **extra)

    def tensor(name, ms, flops, **extra):
        tf = flops / (ms * 1e-3) / 1e12
        out[name] = dict(ms=ms, flops=flops, achieved=tf, unit="TFLOP/s", frac=tf / peaks["bf16_tflops"],
                         frac_of_sustained=tf / peaks["bf16_tflops_sustained"], frac_of_2250=tf / 2250.0,
                         bound="tensor", **extra)

    sampler = ClockSampler(torch.cuda.current_device())
    c2, c2_clocks = config2_kernels(H, dev, peaks, iters, warm, want)
    out.update(c2)
    sampler.start()
    if want("diagnostics"):
        a, b_, c_ = rnd(B, N, D), rnd(B, N, D), rnd(B, N, D)
        mom = torch.zeros(2, dtype=torch.float64, device=dev)
        ms = _time_flushed(lambda: H.hero_second_difference_moments(a, b_, c_, mom), iters, warm, flush)
        hbm("second_difference_moments", ms, 3 * a.numel() * 2)
        ms = _time_flushed(lambda: H.hero_extrapolation_error(a, b_, c_, 2, 5, mom), iters, warm, flush)
        hbm("extrapolation_error", ms, 3 * a.numel() * 2)
        del a, b_, c_
    if want("attention"):
        cases = [(1, 768)] if args.small else [(B, 1755), (B, 4387), (B, 8775)]
        for bb, nq in cases:
            # the form the step runs: q carries the softmax scale log2(e)/sqrt(64) from the projection's epilogue
            q, k, v = rnd(bb, nq, D, std=0.125 * 1.4426950408889634), rnd(bb, N, D), rnd(bb, N, D)
            o = torch.empty_like(q)
            ms = _time_flushed(lambda: H.hero_attention_bf16_q_scaled(q, k, v, o, heads), iters, warm, flush)
            H.hero_isolated_status()
            tensor(f"attention_b{bb}_q{nq}", ms, 4 * bb * nq * N * D)
            if nq == 4387:      # the entry point for unscaled queries (first-tile maximum, scale applied per score)
                ms = _time_flushed(lambda: H.hero_attention_bf16(q, k, v, o, heads), iters, warm, flush)
                H.hero_isolated_status()
                tensor(f"attention_unscaled_q_b{bb}_q{nq}", ms, 4 * bb * nq * N * D)
            del q, k, v, o
    if want("gemm"):
        M = 2048 if args.small else B * 4387
        shapes = [("qkv", 3 * D, D, 0)] if args.small else [("qkv", 3 * D, D, 0), ("out", D, D, 0),
                                                             ("ffn_up", F, D, 1), ("ffn_down", D, F, 0)]
        for name, n_out, kk, act in shapes:
            a, w_, bias = rnd(M, kk), rnd(n_out, kk, std=0.02), rnd(n_out, std=0.02)
            c = torch.empty(M, n_out, device=dev, dtype=bf)
            ms = _time_flushed(lambda: H.hero_gemm_bf16(a, w_, bias, c, act), iters, warm, flush)
            H.hero_isolated_status()
            tensor(f"gemm_{name}_m{M}", ms, 2 * M * n_out * kk)
            del a, w_, bias, c
    if want("deep") and not args.small:
        # the fused passes that only exist inside a context: Eq. 5 + residual of a deep block (12 B per
        # element: 5 reads + 1 write) and the double residual add of a refresh block (8 B per element)
        dcfg = dict(S.CONFIGS["block"], n_blocks=2, n_shallow=1)
        weights = build_device_weights(dcfg, dev)
        hero = H.Hero(dcfg, weights)
        x = S.device_normal(dcfg["seed"], "x0", (B, N, D), 1.0, 0, None, dev).to(bf)
        temb = S.device_normal(dcfg["seed"], "temb", (B, dcfg["temb_dim"]), 1.0, 0, None, dev).to(bf)
        for s_ in range(2):
            hero.hero_step(s_, x, temb)
        n_el = B * N * D
        hbm("extrapolate_residual_block", _time_flushed(lambda: hero.hero_extrapolate_block(1, x, 1, 1), iters, warm, flush),
            12 * n_el)
        idx0 = torch.zeros(1, dtype=torch.int32, device=dev)
        hbm("residual2_block", _time_flushed(lambda: hero.hero_refresh_block(0, x, temb, idx0, 0), iters, warm, flush),
            8 * n_el)
        hero.hero_check_status()
        hero.close()
        del weights, x
    if want("deep_group") and not args.small:
        # a stack of four extrapolated blocks and nothing else: its cached step is exactly one launch of the
        # grouped pass (16 history tensors read, x read and written once: 36 B per element)
        gcfg = dict(S.CONFIGS["block"], n_blocks=4, n_shallow=0)
        weights = build_device_weights(gcfg, dev)
        hero = H.Hero(gcfg, weights)
        x = S.device_normal(gcfg["seed"], "x0", (B, N, D), 1.0, 0, None, dev).to(bf)
        temb = S.device_normal(gcfg["seed"], "temb", (B, gcfg["temb_dim"]), 1.0, 0, None, dev).to(bf)
        for s_ in range(2):
            hero.hero_step(s_, x, temb)
        state = {"s": 2}

        def one_group():
            hero.hero_step(state["s"], x, temb); state["s"] += 1
        hbm("extrapolate_group_4_blocks", _time_flushed(one_group, iters, warm, flush), (8 * 4 + 4) * B * N * D)
        hero.hero_check_status()
        hero.close()
        del weights, x
    if want("block") and not args.small:
        bcfg = dict(S.CONFIGS["block"])
        weights = build_device_weights(bcfg, dev)
        x = S.device_normal(bcfg["seed"], "x0", (B, N, D), 1.0, 0, None, dev).to(bf)
        temb = S.device_normal(bcfg["seed"], "temb", (B, bcfg["temb_dim"]), 1.0, 0, None, dev).to(bf)
        for num, den in ((1, 10), (1, 4), (1, 2), (1, 1)):
            hero = H.Hero(dict(bcfg, ratio_num=num, ratio_den=den), weights)
            hero.hero_refresh_block(0, x, temb)                 # fill the caches (full pass)
            idx = torch.empty(S.n_video(bcfg), dtype=torch.int32, device=dev)
            state = {}

            def one():
                if (num, den) == (1, 1):
                    state["n"] = N
                    hero.hero_refresh_block(0, x, temb)
                else:
                    state["n"] = hero.hero_select_tokens(0, idx)
                    hero.hero_refresh_block(0, x, temb, idx, state["n"])
            ms = _time_flushed(one, iters, warm, flush)
            hero.hero_check_status()
            fl = refresh_flops(bcfg, state["n"])
            tensor(f"refresh_block_{num}/{den}", ms, fl["gemm"] + fl["attention"], n_sel=state["n"])
            hero.close()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    print(json.dumps({"workload": "kernels", "small": bool(args.small), "iters": iters, "timing":
                      "CUDA events, median, L2 flushed by a 256 MiB write + read before every call",
                      "peaks": peaks, "clocks": {"isolated_hbm_kernels": c2_clocks, "tensor_and_block_kernels": clocks},
                      "kernels": out}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed steps (default 10; kernels workload: timed calls per kernel, default 20)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="hero", choices=["hero", "reference"])
    ap.add_argument("--workload", default="dit42", choices=["dit42", "aether", "paper_hp", "paper_hp_m3", "paper_recon", "paper_recon_m3", "block", "tiny", "kernels"])
    ap.add_argument("--only", default="", help="kernels workload: comma list of select,extrapolate,gather,scatter,gather_ln,"
                                               "attention,gemm,deep,deep_group,block,diagnostics")
    ap.add_argument("--small", action="store_true", help="kernels workload: profiler-sized tensor-core cases")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernels", action="store_true", help="skip the isolated-kernel record of the default line")
    ap.add_argument("--cfg-split", action="store_true",
                    help="with --gpus N: split the batch items of ONE problem over the ranks instead of running N problems")
    ap.add_argument("--no-collapse", action="store_true", help="skip the variant runs (collapsed deep stack, refreshed-rows-only attention)")
    args = ap.parse_args()
    if args.steps is None:
        args.steps = 20 if args.workload == "kernels" else 10
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.workload == "kernels" and args.impl == "hero":
        if rank == 0:
            run_kernels(args)
        return
    cfg = dict(S.CONFIGS[args.workload])
    if args.impl == "reference":
        run_reference(args, cfg, rank, world)
    else:
        run_hero(args, cfg, rank, world, local_rank)


if __name__ == "__main__":
    main()
