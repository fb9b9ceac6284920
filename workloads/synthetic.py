"""Seeded synthetic inputs for the HERO cached DiT step.

This module holds shapes and random-number recipes only: no LayerNorm, no
attention, no selection, no extrapolation.  Both the CPU oracle's tests and the
CUDA path's tests/bench draw their inputs from here so that the two sides see
the same numbers; neither side's arithmetic lives here.

Recipe (stands in for the paper's world-model workloads, Sec. 5.1: Aether /
CogVideoX-5B latents; trained weights and video clips are not available and
the cost and bookkeeping of the cached step do not depend on values):
  weights  ~ N(0, 0.02^2), biases ~ N(0, 0.02^2)
  latents, text embeddings, timestep embeddings ~ N(0, 1)
  feature histories (isolated extrapolation): g_prev = A, g_last = A + 0.1*Bd
  every tensor comes from its own Philox stream keyed by (seed, tag, index)
  bf16 workloads: each tensor is rounded once to bf16 (round-to-nearest-even)
  and handed to both sides as exactly representable fp32 values.
"""
from __future__ import annotations

import zlib

import numpy as np

# ----------------------------------------------------------------------------
# Workload shapes.  Keys are plain integers so that each side can build its own
# configuration object from them.
# ----------------------------------------------------------------------------
_COGVIDEO = dict(hidden=3072, n_heads=48, head_dim=64, ffn_dim=12288, temb_dim=512,
                 batch=2, grid_h=30, grid_w=45, n_text=226, patch_h=2, patch_w=2,
                 quota_mode=0, warmup_full_steps=2, dtype="bf16", has_gate=0)

CONFIGS = {
    # config 1: tiny fp32 DiT, 2 refresh + 2 extrapolate blocks, 10 steps
    "tiny": dict(n_blocks=4, n_shallow=2, hidden=128, n_heads=2, head_dim=64, ffn_dim=512,
                 temb_dim=128, batch=1, frames=2, grid_h=8, grid_w=8, n_text=16,
                 patch_h=2, patch_w=2, ratio_num=1, ratio_den=4, quota_mode=0,
                 warmup_full_steps=2, full_interval=0, dtype="fp32", has_gate=0,
                 seed=0, steps=10),
    # config 2: isolated extrapolation / gather / scatter kernels on [2,17776,3072] bf16
    "kernels": dict(_COGVIDEO, n_blocks=1, n_shallow=1, frames=13, ratio_num=1, ratio_den=4,
                    full_interval=0, seed=1, steps=1),
    # config 3: one block at CogVideoX-5B shape, refresh ratio swept
    "block": dict(_COGVIDEO, n_blocks=1, n_shallow=1, frames=13, ratio_num=1, ratio_den=4,
                  full_interval=0, seed=2, steps=1),
    # config 4: 42 blocks, 14 refresh at 25 % + 28 extrapolate, full step every 5
    "dit42": dict(_COGVIDEO, n_blocks=42, n_shallow=14, frames=13, ratio_num=1, ratio_den=4,
                  full_interval=5, seed=3, steps=50),
    # config 5: Aether-shaped sequence, 17 latent frames (the 48 latent channels enter through the patch
    # embedding, which is outside the block stack this library covers: the stack sees [B, N, hidden] tokens)
    "aether": dict(_COGVIDEO, n_blocks=42, n_shallow=14, frames=17, ratio_num=1, ratio_den=4,
                   full_interval=5, seed=4, steps=50),
    # the paper's own hyper-parameters (Sec. 5.1): 2x3 patches, R = 0.2 rounded per patch (Table 3 implies
    # round(6R) tokens), the first 20 blocks refreshed, a full step every M = 2 steps, 11 latent frames
    "paper_hp": dict(_COGVIDEO, n_blocks=42, n_shallow=20, frames=11, patch_h=2, patch_w=3, ratio_num=1,
                     ratio_den=5, quota_mode=1, full_interval=2, seed=5, steps=50),
    # the same with the paper's other interval, M = 3 (visual planning: T = 50 steps, guidance pair)
    "paper_hp_m3": dict(_COGVIDEO, n_blocks=42, n_shallow=20, frames=11, patch_h=2, patch_w=3, ratio_num=1,
                        ratio_den=5, quota_mode=1, full_interval=3, seed=5, steps=50),
    # reconstruction-shaped runs of the same model: one sequence (no guidance pair), T = 30 steps, M = 2 and 3
    "paper_recon": dict(_COGVIDEO, n_blocks=42, n_shallow=20, frames=11, patch_h=2, patch_w=3, ratio_num=1,
                        ratio_den=5, quota_mode=1, full_interval=2, seed=6, steps=30, batch=1),
    "paper_recon_m3": dict(_COGVIDEO, n_blocks=42, n_shallow=20, frames=11, patch_h=2, patch_w=3, ratio_num=1,
                           ratio_den=5, quota_mode=1, full_interval=3, seed=6, steps=30, batch=1),
}


def n_video(cfg) -> int:
    return cfg["frames"] * cfg["grid_h"] * cfg["grid_w"]


def n_rows(cfg) -> int:
    """Sequence length: text rows first, then the video-token grid."""
    return cfg["n_text"] + n_video(cfg)


# ----------------------------------------------------------------------------
# Random streams
# ----------------------------------------------------------------------------
def _rng(seed: int, tag: str, index: int = 0) -> np.random.Generator:
    key = (int(seed) & 0xFFFFFFFF) | (zlib.crc32(tag.encode()) << 32)
    return np.random.Generator(np.random.Philox(key=key, counter=[int(index), 0, 0, 0]))


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round fp32 values to the nearest bf16 (ties to even); result stays fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """uint16 storage of values that are already bf16-representable."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16).reshape(a.shape)


def from_bf16_bits(b: np.ndarray) -> np.ndarray:
    b = np.ascontiguousarray(b, dtype=np.uint16)
    return (b.astype(np.uint32) << 16).view(np.float32).reshape(b.shape)


def normal(seed: int, tag: str, shape, std: float = 1.0, index: int = 0,
           dtype: str = "fp32") -> np.ndarray:
    a = _rng(seed, tag, index).standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return round_bf16(a) if dtype == "bf16" else a


# ----------------------------------------------------------------------------
# Tensors of the DiT workloads
# ----------------------------------------------------------------------------
WEIGHT_NAMES = ("w_mod", "b_mod", "w_qkv", "b_qkv", "w_o", "b_o", "w_1", "b_1", "w_2", "b_2")


def weight_shapes(cfg) -> dict:
    """All weight matrices are row-major [out_features, in_features]."""
    D, F, E = cfg["hidden"], cfg["ffn_dim"], cfg["temb_dim"]
    n_mod = 6 if cfg.get("has_gate", 0) else 4
    shapes = {"w_mod": (n_mod * D, E), "b_mod": (n_mod * D,),
              "w_qkv": (3 * D, D), "b_qkv": (3 * D,),
              "w_o": (D, D), "b_o": (D,),
              "w_1": (F, D), "b_1": (F,),
              "w_2": (D, F), "b_2": (D,)}
    if cfg.get("qk_norm", 0):
        hd = cfg["head_dim"]
        shapes.update({"qn_w": (hd,), "qn_b": (hd,), "kn_w": (hd,), "kn_b": (hd,)})
    return shapes


def block_weights(cfg, block: int) -> dict:
    """Weights of one block, N(0, 0.02), as fp32 arrays (bf16-exact if cfg is bf16)."""
    out = {}
    for name, shape in weight_shapes(cfg).items():
        if name in ("qn_w", "kn_w"):       # LayerNorm gains: around one
            out[name] = 1.0 + normal(cfg["seed"], name, shape, std=0.1, index=block)
        elif name in ("qn_b", "kn_b"):
            out[name] = normal(cfg["seed"], name, shape, std=0.1, index=block)
        else:
            out[name] = normal(cfg["seed"], name, shape, std=0.02, index=block, dtype=cfg["dtype"])
        if cfg["dtype"] == "bf16":
            out[name] = round_bf16(out[name])
    return out


def tokens(cfg, tag: str = "x0") -> np.ndarray:
    """Input sequence [B, N, D] ~ N(0,1): text rows first, then video tokens."""
    return normal(cfg["seed"], tag, (cfg["batch"], n_rows(cfg), cfg["hidden"]), dtype=cfg["dtype"])


def temb(cfg, step: int) -> np.ndarray:
    """Timestep embedding [B, temb_dim] ~ N(0,1), one stream per step."""
    return normal(cfg["seed"], "temb", (cfg["batch"], cfg["temb_dim"]), index=step, dtype=cfg["dtype"])


def feature_history(cfg, shape=None, drift: float = 0.1, index: int = 0):
    """(g_prev, g_last) = (A, A + drift*Bd): N(0,1) features plus a linear drift term."""
    if shape is None:
        shape = (cfg["batch"], n_rows(cfg), cfg["hidden"])
    a = normal(cfg["seed"], "hist_a", shape, index=index)
    bd = normal(cfg["seed"], "hist_b", shape, index=index)
    g_prev, g_last = a, a + np.float32(drift) * bd
    if cfg["dtype"] == "bf16":
        g_prev, g_last = round_bf16(g_prev), round_bf16(g_last)
    return g_prev, g_last


def cache_fill(cfg, tag: str, block: int, shape=None, std: float = 1.0) -> np.ndarray:
    """Synthetic contents for a feature / K / V cache (teacher-forced tests)."""
    if shape is None:
        shape = (cfg["batch"], n_rows(cfg), cfg["hidden"])
    return normal(cfg["seed"], "cache_" + tag, shape, std=std, index=block, dtype=cfg["dtype"])


# ----------------------------------------------------------------------------
# Device-side generation for benchmarks (no oracle comparison on these)
# ----------------------------------------------------------------------------
def device_normal(seed: int, tag: str, shape, std, index, torch_dtype, device):
    """Seeded N(0, std) tensor created directly in device memory (benchmarks only)."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(((int(seed) & 0xFFFF) << 40) ^ (zlib.crc32(tag.encode()) << 8) ^ int(index))
    t = torch.empty(shape, dtype=torch.float32 if torch_dtype is None else torch_dtype, device=device)
    t.normal_(0.0, std, generator=g)
    return t
