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
