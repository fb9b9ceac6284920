"""Thin ctypes binding of libhero.so: argument marshalling only.

Every step of the cached DiT step runs inside the library's CUDA kernels; torch is used
here for device memory and the current stream, nothing else.  Function names match
include/hero.h.  There is no fallback: a missing library or a missing GPU raises.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libhero.so")

OK, ERR_ARG, ERR_ALIGN, ERR_CAP, ERR_STATE, ERR_CUDA, ERR_TIMEOUT, ERR_NOMEM = 0, -1, -2, -3, -4, -5, -6, -7
DTYPE_FP32, DTYPE_BF16 = 0, 1
STATE = dict(ages=0, calls=1, k=2, v=3, g_attn=4, g_ffn=5, g_attn_prev=6, g_ffn_prev=7, steps=8, stack_last=9,
             stack_prev=10)

PROF_CATEGORIES = ("select", "modulation", "gather_ln", "gemm", "attention", "residual", "extrapolate")

EXPORTS = [
    "hero_init", "hero_reset", "hero_destroy", "hero_strerror", "hero_check_status", "hero_last_cuda_error",
    "hero_device_bytes", "hero_launch_count", "hero_profile_begin", "hero_profile_end", "hero_select_tokens", "hero_next_n_sel", "hero_refresh_block",
    "hero_extrapolate_block", "hero_extrapolate_deep_stack", "hero_step", "hero_step_host", "hero_is_full_step", "hero_extrapolate",
    "hero_gather_rows", "hero_scatter_rows", "hero_gemm_bf16", "hero_attention_bf16", "hero_attention_bf16_safe", "hero_attention_bf16_q_scaled", "hero_attention_bf16_static", "hero_attention_bf16_static_status",
    "hero_isolated_status", "hero_selftest_wait_timeout", "hero_gather_ln_modulate",
    "hero_state_get", "hero_state_set", "hero_second_difference_moments", "hero_extrapolation_error",
]


class HeroConfig(C.Structure):
    _fields_ = [(n, C.c_int) for n in (
        "n_blocks", "n_shallow", "hidden", "n_heads", "head_dim", "ffn_dim", "temb_dim",
        "batch", "frames", "grid_h", "grid_w", "n_text", "patch_h", "patch_w",
        "ratio_num", "ratio_den", "quota_mode", "warmup_full_steps", "full_interval", "dtype", "has_gate")
    ] + [("seed", C.c_ulonglong), ("deep_collapse", C.c_int), ("track_mode", C.c_int), ("share_selection", C.c_int), ("attend_mode", C.c_int), ("qk_norm", C.c_int), ("rope", C.c_int)]


class HeroBlockWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("w_mod", "b_mod", "w_qkv", "b_qkv", "w_o", "b_o", "w_1", "b_1", "w_2", "b_2",
                 "qn_w", "qn_b", "kn_w", "kn_b")]
    OPTIONAL = ("qn_w", "qn_b", "kn_w", "kn_b")      # read only with hero_config.qk_norm


class HeroError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        msg = load().hero_strerror(code).decode()
        extra = load().hero_last_cuda_error().decode() if code == ERR_CUDA else ""
        super().__init__(f"{where}: {msg} ({code}) {extra}".strip())


_lib = None


def load() -> C.CDLL:
    """Load libhero.so (built in-tree by paper_2508_17588_b200.build); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError(
            f"{LIB_PATH} not found: run `python -m paper_2508_17588_b200.build` (nvcc, sm_100a). "
            "There is no CPU or PyTorch fallback for this library.")
    lib = C.CDLL(LIB_PATH)
    vp, ip, i, ll = C.c_void_p, C.POINTER(C.c_int), C.c_int, C.c_longlong
    sig = {
        "hero_init": (i, [C.POINTER(vp), C.POINTER(HeroConfig), C.POINTER(HeroBlockWeights), vp]),
        "hero_reset": (i, [vp]),
        "hero_destroy": (None, [vp]),
        "hero_strerror": (C.c_char_p, [i]),
        "hero_check_status": (i, [vp]),
        "hero_last_cuda_error": (C.c_char_p, []),
        "hero_device_bytes": (ll, [vp]),
        "hero_launch_count": (ll, [vp]),
        "hero_profile_begin": (i, [vp]),
        "hero_profile_end": (i, [vp, C.POINTER(C.c_double), C.POINTER(ll)]),
        "hero_select_tokens": (i, [vp, i, vp, i, ip]),
        "hero_next_n_sel": (i, [vp, i]),
        "hero_refresh_block": (i, [vp, i, vp, vp, vp, i]),
        "hero_extrapolate_block": (i, [vp, i, vp, i, i]),
        "hero_extrapolate_deep_stack": (i, [vp, vp, i, i]),
        "hero_step": (i, [vp, i, vp, vp]),
        "hero_step_host": (i, [vp, i, vp, vp]),
        "hero_is_full_step": (i, [vp, i]),
        "hero_extrapolate": (i, [vp, vp, vp, ll, i, i, i, vp]),
        "hero_gather_rows": (i, [vp, vp, vp, i, i, i, i, i, vp]),
        "hero_scatter_rows": (i, [vp, vp, vp, i, i, i, i, i, vp]),
        "hero_gemm_bf16": (i, [vp, vp, vp, vp, i, i, i, i, vp]),
        "hero_attention_bf16": (i, [vp, vp, vp, vp, i, i, i, i, vp]),
        "hero_attention_bf16_safe": (i, [vp, vp, vp, vp, i, i, i, i, vp]),
        "hero_attention_bf16_q_scaled": (i, [vp, vp, vp, vp, i, i, i, i, vp]),
        "hero_attention_bf16_static": (i, [vp, vp, vp, vp, i, i, i, i, vp, ip]),
        "hero_attention_bf16_static_status": (i, [vp, ip, ip, i]),
        "hero_isolated_status": (i, [vp]),
        "hero_selftest_wait_timeout": (i, [vp, i, vp]),
        "hero_gather_ln_modulate": (i, [vp, vp, vp, vp, vp, i, vp, i, i, i, i, i, vp]),
        "hero_second_difference_moments": (i, [vp, vp, vp, ll, i, vp, vp]),
        "hero_extrapolation_error": (i, [vp, vp, vp, ll, i, i, i, vp, vp]),
        "hero_state_get": (i, [vp, i, i, vp, ll]),
        "hero_state_set": (i, [vp, i, i, vp, ll]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _check(code: int, where: str) -> int:
    if code < 0:
        raise HeroError(code, where)
    return code


def _require_cuda():
    if not torch.cuda.is_available():
        raise RuntimeError("paper_2508_17588_b200 needs a CUDA device (B200, sm_100a); there is no CPU path")


def _ptr(t) -> int:
    return 0 if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def torch_dtype(dtype) -> torch.dtype:
    return torch.bfloat16 if dtype in (DTYPE_BF16, "bf16") else torch.float32


def dtype_code(dtype) -> int:
    if dtype in (DTYPE_BF16, "bf16", torch.bfloat16):
        return DTYPE_BF16
    if dtype in (DTYPE_FP32, "fp32", torch.float32):
        return DTYPE_FP32
    raise ValueError(f"unsupported dtype {dtype}")


def make_config(d: dict) -> HeroConfig:
    cfg = HeroConfig()
    for name, _ in HeroConfig._fields_:
        if name == "dtype":
            cfg.dtype = dtype_code(d["dtype"])
        elif name in d:
            setattr(cfg, name, int(d[name]))
    return cfg


class Hero:
    """Owner of one hero_ctx.  `weights` is a list (one per block) of dicts of CUDA tensors
    named as in hero_block_weights, row-major [out, in], in the run dtype."""

    def __init__(self, cfg: dict, weights):
        _require_cuda()
        self.lib = load()
        self.cfg = dict(cfg)
        self.c_cfg = make_config(cfg)
        self.dt = torch_dtype(self.c_cfg.dtype)
        self.N = cfg["n_text"] + cfg["frames"] * cfg["grid_h"] * cfg["grid_w"]
        self.n_video = self.N - cfg["n_text"]
        assert len(weights) == cfg["n_blocks"]
        self._weights = weights      # keep the tensors alive: the library borrows the pointers
        arr = (HeroBlockWeights * cfg["n_blocks"])()
        for l, w in enumerate(weights):
            for name, _ in HeroBlockWeights._fields_:
                if name in HeroBlockWeights.OPTIONAL and not cfg.get("qk_norm", 0):
                    continue
                t = w[name]
                assert t.is_cuda and t.is_contiguous() and t.dtype == self.dt, name
                setattr(arr[l], name, t.data_ptr())
        self.ctx = C.c_void_p()
        _check(self.lib.hero_init(C.byref(self.ctx), C.byref(self.c_cfg), arr, _stream()), "hero_init")
        self._stream = _stream()

    def close(self):
        if getattr(self, "ctx", None) is not None and self.ctx:
            self.lib.hero_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- the method's calls -------------------------------------------------
    def hero_select_tokens(self, block: int, idx: torch.Tensor) -> int:
        n = C.c_int(0)
        _check(self.lib.hero_select_tokens(self.ctx, block, _ptr(idx), idx.numel(), C.byref(n)), "hero_select_tokens")
        return n.value

    def hero_next_n_sel(self, block: int) -> int:
        return _check(self.lib.hero_next_n_sel(self.ctx, block), "hero_next_n_sel")

    def hero_refresh_block(self, block: int, x, temb, idx=None, n_sel=None):
        n = self.N if idx is None else (idx.numel() if n_sel is None else n_sel)
        _check(self.lib.hero_refresh_block(self.ctx, block, _ptr(x), _ptr(temb), _ptr(idx), n), "hero_refresh_block")

    def hero_extrapolate_block(self, block: int, x, k: int, d: int):
        _check(self.lib.hero_extrapolate_block(self.ctx, block, _ptr(x), k, d), "hero_extrapolate_block")

    def hero_extrapolate_deep_stack(self, x, k: int, d: int):
        _check(self.lib.hero_extrapolate_deep_stack(self.ctx, _ptr(x), k, d), "hero_extrapolate_deep_stack")

    def hero_step(self, step: int, x, temb):
        _check(self.lib.hero_step(self.ctx, step, _ptr(x), _ptr(temb)), "hero_step")

    def hero_step_host(self, step: int, h_x, h_temb):
        assert not h_x.is_cuda and not h_temb.is_cuda
        _check(self.lib.hero_step_host(self.ctx, step, _ptr(h_x), _ptr(h_temb)), "hero_step_host")

    def hero_is_full_step(self, step: int) -> bool:
        return bool(_check(self.lib.hero_is_full_step(self.ctx, step), "hero_is_full_step"))

    def hero_reset(self):
        _check(self.lib.hero_reset(self.ctx), "hero_reset")

    def hero_check_status(self):
        _check(self.lib.hero_check_status(self.ctx), "hero_check_status")

    def hero_selftest_wait_timeout(self, budget_us: int = 50):
        """Make one bounded device-side wait run out on purpose (it raises this context's status word)."""
        _check(self.lib.hero_selftest_wait_timeout(self.ctx, budget_us, None), "hero_selftest_wait_timeout")

    def hero_device_bytes(self) -> int:
        return self.lib.hero_device_bytes(self.ctx)

    def hero_launch_count(self) -> int:
        return self.lib.hero_launch_count(self.ctx)

    def hero_profile_begin(self):
        _check(self.lib.hero_profile_begin(self.ctx), "hero_profile_begin")

    def hero_profile_end(self) -> dict:
        """{category: (summed device ms, launches)} since hero_profile_begin."""
        ms = (C.c_double * len(PROF_CATEGORIES))()
        n = (C.c_longlong * len(PROF_CATEGORIES))()
        _check(self.lib.hero_profile_end(self.ctx, ms, n), "hero_profile_end")
        return {name: (ms[i], n[i]) for i, name in enumerate(PROF_CATEGORIES)}

    # ---- state access ---------------------------------------------------------
    def _state_tensor(self, what: str) -> torch.Tensor:
        if what == "ages":
            return torch.empty(self.n_video, dtype=torch.uint16)
        if what == "calls":
            return torch.empty(1, dtype=torch.int32)
        if what == "steps":
            return torch.empty(3, dtype=torch.int32)
        if what in ("stack_last", "stack_prev"):
            return torch.empty(self.cfg["batch"], self.N, self.cfg["hidden"], dtype=torch.float32)
        return torch.empty(self.cfg["batch"], self.N, self.cfg["hidden"], dtype=self.dt)

    def hero_state_get(self, block: int, what: str) -> torch.Tensor:
        t = self._state_tensor(what)
        _check(self.lib.hero_state_get(self.ctx, block, STATE[what], t.data_ptr(), t.numel() * t.element_size()),
               "hero_state_get")
        return t

    def hero_state_set(self, block: int, what: str, t: torch.Tensor):
        ref = self._state_tensor(what)
        t = t.detach().cpu().to(ref.dtype).contiguous()
        assert t.numel() == ref.numel(), what
        _check(self.lib.hero_state_set(self.ctx, block, STATE[what], t.data_ptr(), t.numel() * t.element_size()),
               "hero_state_set")


# ---- isolated kernels ---------------------------------------------------------
def hero_extrapolate(g_prev, g_last, out, k: int, d: int):
    _require_cuda()
    _check(load().hero_extrapolate(_ptr(g_prev), _ptr(g_last), _ptr(out), g_last.numel(), k, d,
                                   dtype_code(g_last.dtype), _stream()), "hero_extrapolate")
    return out


# ---- diagnostics (Sec. 4.1) ------------------------------------------------------
def hero_second_difference_moments(f_a, f_b, f_c, moments):
    """moments (CUDA float64[2]) += (sum u, sum u^2) of u = f_a - 2 f_b + f_c."""
    _require_cuda()
    assert moments.is_cuda and moments.dtype == torch.float64 and moments.numel() == 2
    _check(load().hero_second_difference_moments(_ptr(f_a), _ptr(f_b), _ptr(f_c), f_b.numel(), dtype_code(f_b.dtype),
                                                 _ptr(moments), _stream()), "hero_second_difference_moments")
    return moments


def hero_extrapolation_error(g_prev, g_last, g_true, k: int, d: int, err):
    """err (CUDA float64[2]) += (sum (Eq. 5 prediction - g_true)^2, sum g_true^2)."""
    _require_cuda()
    assert err.is_cuda and err.dtype == torch.float64 and err.numel() == 2
    _check(load().hero_extrapolation_error(_ptr(g_prev), _ptr(g_last), _ptr(g_true), g_last.numel(), k, d,
                                           dtype_code(g_last.dtype), _ptr(err), _stream()), "hero_extrapolation_error")
    return err


def hero_gather_rows(src, idx, dst):
    _require_cuda()
    B, N, D = src.shape
    _check(load().hero_gather_rows(_ptr(src), _ptr(idx), _ptr(dst), B, N, idx.numel(), D, dtype_code(src.dtype),
                                   _stream()), "hero_gather_rows")
    return dst


def hero_scatter_rows(src, idx, dst):
    _require_cuda()
    B, N, D = dst.shape
    _check(load().hero_scatter_rows(_ptr(src), _ptr(idx), _ptr(dst), B, N, idx.numel(), D, dtype_code(dst.dtype),
                                    _stream()), "hero_scatter_rows")
    return dst


def hero_gemm_bf16(a, w, bias, c, act: int = 0):
    _require_cuda()
    M, K = a.shape
    N = w.shape[0]
    _check(load().hero_gemm_bf16(_ptr(a), _ptr(w), _ptr(bias), _ptr(c), M, N, K, act, _stream()), "hero_gemm_bf16")
    return c


def hero_attention_bf16(q, k, v, o, heads: int):
    _require_cuda()
    B, n_q, _ = q.shape
    N = k.shape[1]
    _check(load().hero_attention_bf16(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, n_q, N, heads, _stream()),
           "hero_attention_bf16")
    return o


def hero_attention_bf16_safe(q, k, v, o, heads: int):
    """The fallback attention kernel alone (running maximum with in-place rescaling)."""
    _require_cuda()
    B, n_q, _ = q.shape
    N = k.shape[1]
    _check(load().hero_attention_bf16_safe(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, n_q, N, heads, _stream()),
           "hero_attention_bf16_safe")
    return o


def hero_attention_bf16_q_scaled(q, k, v, o, heads: int):
    """hero_attention_bf16 for queries that already carry the factor log2(e) / sqrt(head_dim)."""
    _require_cuda()
    B, n_q, _ = q.shape
    N = k.shape[1]
    _check(load().hero_attention_bf16_q_scaled(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, n_q, N, heads, _stream()),
           "hero_attention_bf16_q_scaled")
    return o


def hero_attention_bf16_static(q, k, v, o, heads: int, check: bool = True):
    """hero_attention_bf16 for callers that must not allocate device memory: the kernel's scratch is a
    fixed array inside the library.  With check=True the call waits for the result and raises if any
    thread block gave up on a bounded wait; with check=False it only enqueues the work."""
    _require_cuda()
    B, n_q, _ = q.shape
    N = k.shape[1]
    gave_up = C.c_int(0)
    _check(load().hero_attention_bf16_static(_ptr(q), _ptr(k), _ptr(v), _ptr(o), B, n_q, N, heads, _stream(),
                                             C.byref(gave_up) if check else None), "hero_attention_bf16_static")
    return o


def hero_attention_bf16_static_status(n_records: int = 0):
    """(thread blocks that gave up, their per-block records) of the latest hero_attention_bf16_static call."""
    _require_cuda()
    gave_up = C.c_int(-1)
    rec = (C.c_int * max(n_records, 1))()
    _check(load().hero_attention_bf16_static_status(_stream(), C.byref(gave_up), rec if n_records else None, n_records),
           "hero_attention_bf16_static_status")
    return gave_up.value, list(rec)[:n_records]


def hero_isolated_status():
    _check(load().hero_isolated_status(_stream()), "hero_isolated_status")


def hero_selftest_wait_timeout(budget_us: int = 50):
    """Make one bounded device-side wait run out on purpose (raises the isolated calls' status word)."""
    _require_cuda()
    _check(load().hero_selftest_wait_timeout(None, budget_us, _stream()), "hero_selftest_wait_timeout")


def hero_gather_ln_modulate(x, add, idx, shift, scale, out):
    """out[b, i] = LN(x[b, idx[i]] (+ add[b, idx[i]])) * (1 + scale[b]) + shift[b]; shift/scale fp32 [B, D]."""
    _require_cuda()
    B, N, D = x.shape
    n_sel = out.shape[1]
    assert shift.dtype == torch.float32 and scale.dtype == torch.float32 and shift.stride(0) == scale.stride(0)
    _check(load().hero_gather_ln_modulate(_ptr(x), _ptr(add), _ptr(idx), _ptr(shift), _ptr(scale), shift.stride(0),
                                          _ptr(out), B, N, n_sel, D, dtype_code(x.dtype), _stream()),
           "hero_gather_ln_modulate")
    return out


def device_weights(host_weights: dict, dtype, device="cuda") -> dict:
    """Upload one block's host weights (numpy fp32, bf16-exact when dtype is bf16)."""
    dt = torch_dtype(dtype_code(dtype))
    return {k: torch.from_numpy(v).to(device=device, dtype=dt).contiguous() for k, v in host_weights.items()}
