"""Helpers shared by the GPU parity tests: build the oracle and the CUDA context from the
same seeded workload, and the error measures the tolerances are stated in."""
import numpy as np
import torch

from oracle import hero_oracle as O
from workloads import synthetic as S


def rel_l2(got, want) -> float:
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    return float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-300))


def rel_max(got, want) -> float:
    """max-abs error over max-abs value."""
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    return float(np.abs(got - want).max() / max(np.abs(want).max(), 1e-300))


def to_dev(a: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32))
    return t.to(device="cuda", dtype=torch.bfloat16 if dtype == "bf16" else torch.float32).contiguous()


def to_host(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def make_pair(cfgd: dict, weights=None):
    """(oracle, cuda context, host weights) for one workload dict."""
    import paper_2508_17588_b200 as H
    if weights is None:
        weights = [S.block_weights(cfgd, l) for l in range(cfgd["n_blocks"])]
    orc = O.HeroOracle(O.Config.from_dict(cfgd), weights)
    dev_w = [H.device_weights(w, cfgd["dtype"]) for w in weights]
    hero = H.Hero(cfgd, dev_w)
    return orc, hero, weights
