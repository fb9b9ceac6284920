"""The C-ABI library loads on a machine without a GPU and exports every symbol that
include/hero.h declares; argument errors are reported before any CUDA work."""
import ctypes as C
import os
import re

import paper_2508_17588_b200 as H
from paper_2508_17588_b200 import binding as Bd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "hero.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hero_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = H.load()
    names = declared_symbols()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(H.EXPORTS) == names


def test_strerror_and_codes():
    lib = H.load()
    assert lib.hero_strerror(0) == b"ok"
    for code in range(-7, 0):
        assert lib.hero_strerror(code) not in (b"ok", b"unknown error")
    assert lib.hero_strerror(-99) == b"unknown error"


def test_config_struct_matches_header_field_order():
    text = open(os.path.join(ROOT, "include", "hero.h")).read()
    body = re.search(r"typedef struct hero_config \{(.*?)\} hero_config;", text, flags=re.S).group(1)
    body = re.sub(r"/\*.*?\*/", "", body, flags=re.S)
    fields = []
    for stmt in body.split(";"):
        stmt = stmt.strip()
        if not stmt:
            continue
        names = re.sub(r"^(unsigned long long|int)\b", "", stmt)
        fields += [n.strip() for n in names.split(",") if n.strip()]
    assert fields == [n for n, _ in Bd.HeroConfig._fields_]


def test_argument_errors_need_no_gpu():
    lib = H.load()
    ctx = C.c_void_p()
    cfg = Bd.HeroConfig()               # all zeros: invalid
    w = (Bd.HeroBlockWeights * 1)()
    assert lib.hero_init(C.byref(ctx), C.byref(cfg), w, None) == Bd.ERR_ARG
    assert lib.hero_init(None, C.byref(cfg), w, None) == Bd.ERR_ARG
    assert lib.hero_step(None, 0, None, None) == Bd.ERR_ARG
    assert lib.hero_extrapolate(None, None, None, 16, 1, 0, 0, None) == Bd.ERR_ARG     # d = 0
    assert lib.hero_extrapolate(None, None, None, 0, 1, 1, 0, None) == Bd.OK           # empty input
    assert lib.hero_extrapolate(8, 16, 32, 64, 1, 1, 1, None) == Bd.ERR_ALIGN          # misaligned pointer
    assert lib.hero_gather_rows(None, None, None, 2, 8, 0, 64, 1, None) == Bd.OK       # empty list
    assert lib.hero_gather_rows(None, None, None, 2, 8, 9, 64, 1, None) == Bd.ERR_ARG  # n_sel > N
    assert lib.hero_gemm_bf16(None, None, None, None, 4, 0, 8, 0, None) == Bd.ERR_ARG


def _valid_bf16_config():
    cfg = Bd.HeroConfig()
    for name, val in dict(n_blocks=1, n_shallow=1, hidden=128, n_heads=2, head_dim=64, ffn_dim=256, temb_dim=64, batch=1,
                          frames=1, grid_h=2, grid_w=2, n_text=0, patch_h=2, patch_w=2, ratio_num=1, ratio_den=4,
                          warmup_full_steps=2, dtype=Bd.DTYPE_BF16).items():
        setattr(cfg, name, val)
    return cfg


def test_shapes_the_kernels_cannot_run_are_refused_at_init_not_in_the_middle_of_a_step():
    """Every size limit of a kernel is checked by hero_init before anything is allocated or launched.  The
    weight pointers given here are non-NULL and aligned but point nowhere: hero_init never reads through them,
    so a config that passes ends in OK (with a GPU) or in a CUDA / allocation error (without one), and a
    config that does not pass ends in the argument error named beside it, GPU or not."""
    lib = H.load()
    ctx = C.c_void_p()
    w = (Bd.HeroBlockWeights * 1)()
    for name, _ in Bd.HeroBlockWeights._fields_:
        setattr(w[0], name, 4096)

    def init(cfg):
        rc = lib.hero_init(C.byref(ctx), C.byref(cfg), w, None)
        if rc == Bd.OK:
            lib.hero_destroy(ctx)
        return rc

    passes = (Bd.OK, Bd.ERR_CUDA, Bd.ERR_NOMEM)
    assert init(_valid_bf16_config()) in passes
    for field, bad, want in (("ffn_dim", 264, Bd.ERR_ALIGN),      # bf16 GEMM output pieces are 32 columns wide
                             ("temb_dim", 60, Bd.ERR_ALIGN),      # 16-byte packets of bf16
                             ("temb_dim", 12296, Bd.ERR_ARG),     # SiLU(temb) of the batch: more than 48 KB of shared memory
                             ("head_dim", 32, Bd.ERR_ARG)):       # hidden != heads * head_dim
        cfg = _valid_bf16_config()
        setattr(cfg, field, bad)
        assert init(cfg) == want, field
    cfg = _valid_bf16_config()                # 12800 columns: not a warp-per-row width, and wider than the
    cfg.hidden, cfg.n_heads = 64 * 200, 200   # 12288 floats the generic LayerNorm keeps in shared memory
    assert init(cfg) == Bd.ERR_ARG
    cfg = _valid_bf16_config()
    cfg.dtype, cfg.hidden, cfg.n_heads, cfg.head_dim = Bd.DTYPE_FP32, 12288 + 128, 97, 128
    assert init(cfg) == Bd.ERR_ARG            # fp32 rows always go through shared memory
    cfg.hidden, cfg.n_heads = 12288, 96
    assert init(cfg) in passes
    assert lib.hero_gather_ln_modulate(None, None, None, None, None, 64, None, 1, 8, 0, 64, 1, None) == Bd.OK   # empty
    assert lib.hero_gather_ln_modulate(None, None, None, None, None, 32, None, 1, 8, 4, 64, 1, None) == Bd.ERR_ARG  # mod_ld < D
    assert lib.hero_selftest_wait_timeout(None, 0, None) == Bd.ERR_ARG
    gave_up = C.c_int(0)
    assert lib.hero_attention_bf16_static_status(None, None, None, 0) == Bd.ERR_ARG
    assert lib.hero_attention_bf16_static_status(None, C.byref(gave_up), None, 5) == Bd.ERR_ARG
