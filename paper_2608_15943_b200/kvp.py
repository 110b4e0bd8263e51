"""ctypes binding of the C-ABI library (``include/kvp.h``): argument marshalling only.

Every function takes torch tensors (device memory, streams) and passes raw pointers and sizes to
the entry point of the same name; all computation happens in the library's CUDA kernels.  Importing
this module loads ``libkvp.so`` and raises if it has not been built -- there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkvp.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2608_15943_b200.build` (nvcc, sm_100a)")
lib = C.CDLL(LIB_PATH)

OK, ERR_INVALID_ARG, ERR_BAD_DONOR, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT = range(7)
PLAN_STOP_ON_NO_IMPROVE, PLAN_STAGE_LOCAL_DONOR = 1, 2
STOP_TOLERANCE, STOP_BUDGET, STOP_EXHAUSTED, STOP_NO_IMPROVE = range(4)
PLACE_ARCH_BALANCED, PLACE_UNIFORM, PLACE_BIPOLAR = range(3)
OP_PROJ_FWD, OP_PROJ_BWD, OP_ATTN_FWD, OP_ATTN_BWD, OP_DECODE = range(5)
BF16, F32 = 0, 1   # dtype of the activations / weights in the caller's memory (kvp_shape.dtype, kvp_decode_desc.dtype)

EXPORTS = ["kvp_status_string", "kvp_device_status", "kvp_launch_count", "kvp_set_timing_events", "kvp_set_gemm_pair_mode", "kvp_selftest_bounded_wait_pair",
           "kvp_timing_events_used", "kvp_plan", "kvp_layer_flops", "kvp_sim_1f1b", "kvp_workspace_bytes",
           "kvp_proj_fwd", "kvp_proj_bwd", "kvp_proj_bwd_range", "kvp_out_proj_fwd", "kvp_out_proj_bwd", "kvp_attn_fwd", "kvp_attn_bwd",
           "kvp_gemm", "kvp_rmsnorm", "kvp_rope", "kvp_swiglu", "kvp_add", "kvp_decode_workspace_bytes", "kvp_cache_append",
           "kvp_decode", "kvp_decode_static", "kvp_selftest_bounded_wait"]


class KvpError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


lib.kvp_status_string.restype = C.c_char_p
lib.kvp_status_string.argtypes = [C.c_int]


def status_string(status: int) -> str:
    return lib.kvp_status_string(int(status)).decode()


def _check(status: int, where: str) -> None:
    if status != OK:
        raise KvpError(status, where)


def device_status() -> int:
    """Synchronises and returns the library's device status (OK or ERR_TIMEOUT / ERR_CUDA)."""
    lib.kvp_device_status.restype = C.c_int
    return int(lib.kvp_device_status())


def _stream() -> C.c_void_p:
    # Without a device the entry points still validate their arguments (and fail before any launch).
    if not torch.cuda.is_available():
        return C.c_void_p(0)
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t: Optional[torch.Tensor]) -> int:
    return 0 if t is None else t.data_ptr()


def _ptr_array(ts: Sequence[Optional[torch.Tensor]]):
    arr = (C.c_void_p * len(ts))()
    for i, t in enumerate(ts):
        arr[i] = _ptr(t)
    return arr


def _i32_array(xs: Sequence[int]):
    return (C.c_int32 * len(xs))(*[int(x) for x in xs])


def _u64_array(xs: Sequence[int]):
    return (C.c_uint64 * len(xs))(*[int(x) for x in xs])


# ------------------------------------------------------------------------------------------
# gemm
# ------------------------------------------------------------------------------------------
lib.kvp_gemm.restype = C.c_int
lib.kvp_gemm.argtypes = [C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int64, C.c_int, C.c_void_p, C.c_int64, C.c_int,
                         C.c_void_p, C.c_int64, C.c_int, C.c_void_p]


def gemm(a: torch.Tensor, b: torch.Tensor, c: torch.Tensor, a_mn: bool = False, b_mn: bool = False) -> torch.Tensor:
    """c[M,N] = A B.  a is stored [M,K] (a_mn False) or [K,M]; b is stored [N,K] (b_mn False) or
    [K,N]; c is bf16 or fp32, row-major."""
    M, N = c.shape
    K = a.shape[0] if a_mn else a.shape[1]
    _check(lib.kvp_gemm(M, N, K, a.data_ptr(), a.stride(0), int(a_mn), b.data_ptr(), b.stride(0), int(b_mn),
                        c.data_ptr(), c.stride(0), int(c.dtype == torch.float32), _stream()), "kvp_gemm")
    return c


# ------------------------------------------------------------------------------------------
# element-wise stage operators
# ------------------------------------------------------------------------------------------
lib.kvp_rmsnorm.restype = C.c_int
lib.kvp_rmsnorm.argtypes = [C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_float, C.c_void_p, C.c_void_p]
lib.kvp_rope.restype = C.c_int
lib.kvp_rope.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_int32, C.c_void_p, C.c_void_p]
lib.kvp_swiglu.restype = C.c_int
lib.kvp_swiglu.argtypes = [C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
lib.kvp_add.restype = C.c_int
lib.kvp_add.argtypes = [C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]


def rmsnorm(x: torch.Tensor, w: torch.Tensor, eps: float, y: torch.Tensor) -> torch.Tensor:
    """kvp_rmsnorm: y[T,D] = x / sqrt(mean(x^2) + eps) * w (bf16)."""
    T, D = x.shape
    _check(lib.kvp_rmsnorm(T, D, x.data_ptr(), w.data_ptr(), float(eps), y.data_ptr(), _stream()), "kvp_rmsnorm")
    return y


def rope(x: torch.Tensor, theta: float = 10000.0, pos0: int = 0) -> torch.Tensor:
    """kvp_rope: in place on x [B,S,H,dh] (bf16)."""
    B, S, H, dh = x.shape
    _check(lib.kvp_rope(B, S, H, dh, float(theta), int(pos0), x.data_ptr(), _stream()), "kvp_rope")
    return x


def swiglu(gate: torch.Tensor, up: torch.Tensor, out: torch.Tensor) -> torch.Tensor:
    """kvp_swiglu: out = silu(gate) * up (bf16, same shapes)."""
    _check(lib.kvp_swiglu(gate.numel(), gate.data_ptr(), up.data_ptr(), out.data_ptr(), _stream()), "kvp_swiglu")
    return out


def add(a: torch.Tensor, b: torch.Tensor, out: torch.Tensor) -> torch.Tensor:
    """kvp_add: out = a + b (bf16, same shapes)."""
    _check(lib.kvp_add(a.numel(), a.data_ptr(), b.data_ptr(), out.data_ptr(), _stream()), "kvp_add")
    return out


# ------------------------------------------------------------------------------------------
# planner (host)
# ------------------------------------------------------------------------------------------
class _PlanIn(C.Structure):
    _fields_ = [("L", C.c_int32), ("P", C.c_int32), ("stage_begin", C.POINTER(C.c_int32)),
                ("f_full", C.POINTER(C.c_uint64)), ("f_share", C.POINTER(C.c_uint64)),
                ("stage_extra", C.POINTER(C.c_uint64)), ("eps_num", C.c_uint32), ("eps_den", C.c_uint32),
                ("max_conv", C.c_int32), ("flags", C.c_uint32), ("alpha_num", C.c_uint32), ("alpha_den", C.c_uint32),
                ("placement", C.c_int32)]


class _PlanOut(C.Structure):
    _fields_ = [("z", C.POINTER(C.c_uint8)), ("donor", C.POINTER(C.c_int32)), ("stage_flops", C.POINTER(C.c_uint64)),
                ("stage_ratio", C.POINTER(C.c_double)), ("fir_num", C.c_uint64), ("fir_den", C.c_uint64),
                ("fir", C.c_double), ("n_conv", C.c_int32), ("stop_reason", C.c_int32)]


class _ModelDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("h", "f", "a", "g", "dh", "s", "vocab", "causal_half")]


lib.kvp_plan.restype = C.c_int
lib.kvp_plan.argtypes = [C.POINTER(_PlanIn), C.POINTER(_PlanOut)]
lib.kvp_layer_flops.restype = C.c_int
lib.kvp_layer_flops.argtypes = [C.POINTER(_ModelDesc), C.POINTER(C.c_uint64), C.POINTER(C.c_uint64),
                                C.POINTER(C.c_uint64)]


def plan(stage_begin, f_full, f_share, stage_extra, eps=(0, 1), max_conv=0, stop_on_no_improve=False,
         stage_local_donor=False, alpha=None, placement=PLACE_ARCH_BALANCED) -> dict:
    """kvp_plan (Algorithm 1).  Returns dict(z, donor, stage, stage_ratio, fir_num, fir_den, fir,
    n_conv, stop_reason)."""
    P = len(stage_begin) - 1
    L = len(f_full)
    sb, ff, fs, ex = _i32_array(stage_begin), _u64_array(f_full), _u64_array(f_share), _u64_array(stage_extra)
    z = (C.c_uint8 * L)()
    donor = (C.c_int32 * L)()
    st = (C.c_uint64 * P)()
    ratio = (C.c_double * P)()
    flags = (PLAN_STOP_ON_NO_IMPROVE if stop_on_no_improve else 0) | (PLAN_STAGE_LOCAL_DONOR if stage_local_donor else 0)
    an, ad = alpha if alpha else (0, 1)
    pin = _PlanIn(L, P, sb, ff, fs, ex, eps[0], eps[1], max_conv, flags, an, ad, placement)
    pout = _PlanOut(z, donor, st, ratio, 0, 0, 0.0, 0, 0)
    _check(lib.kvp_plan(C.byref(pin), C.byref(pout)), "kvp_plan")
    return dict(z=list(z), donor=list(donor), stage=list(st), stage_ratio=list(ratio), fir_num=pout.fir_num,
                fir_den=pout.fir_den, fir=pout.fir, n_conv=pout.n_conv, stop_reason=pout.stop_reason)


def layer_flops(h, f, a, g, dh, s, vocab, causal_half=True):
    """kvp_layer_flops -> (f_full, f_share, f_lm_head), per token, forward."""
    m = _ModelDesc(h, f, a, g, dh, s, vocab, int(causal_half))
    o = [C.c_uint64() for _ in range(3)]
    _check(lib.kvp_layer_flops(C.byref(m), *[C.byref(x) for x in o]), "kvp_layer_flops")
    return tuple(int(x.value) for x in o)


class _SimOut(C.Structure):
    _fields_ = [("makespan", C.c_int64), ("idle", C.POINTER(C.c_int64))]


lib.kvp_sim_1f1b.restype = C.c_int
lib.kvp_sim_1f1b.argtypes = [C.c_int32, C.c_int32, C.POINTER(C.c_int64), C.POINTER(C.c_int64), C.POINTER(_SimOut)]


def sim_1f1b(t_fwd, t_bwd, M):
    """kvp_sim_1f1b -> (makespan, idle[P]) for per-stage forward / backward times (integers) and M micro-batches."""
    P = len(t_fwd)
    tf = (C.c_int64 * P)(*[int(x) for x in t_fwd])
    tb = (C.c_int64 * len(t_bwd))(*[int(x) for x in t_bwd])
    idle = (C.c_int64 * max(P, 1))()
    out = _SimOut(0, idle)
    _check(lib.kvp_sim_1f1b(P if len(t_bwd) == P else -1, int(M), tf, tb, C.byref(out)), "kvp_sim_1f1b")
    return int(out.makespan), [int(x) for x in idle[:P]]


# ------------------------------------------------------------------------------------------
# training / prefill path
# ------------------------------------------------------------------------------------------
class Shape(C.Structure):
    """kvp_shape."""
    _fields_ = [(n, C.c_int32) for n in ("L", "B", "S", "D", "Hq", "Hkv", "dh", "dtype")]

    def __init__(self, L, B, S, D, Hq, Hkv, dh, dtype=0):
        super().__init__(L, B, S, D, Hq, Hkv, dh, dtype)


_PP = C.POINTER(C.c_void_p)
lib.kvp_workspace_bytes.restype = C.c_size_t
lib.kvp_workspace_bytes.argtypes = [C.c_int, C.POINTER(Shape), C.POINTER(C.c_int32)]
lib.kvp_proj_fwd.restype = C.c_int
lib.kvp_proj_fwd.argtypes = [C.POINTER(Shape), C.POINTER(C.c_int32)] + [_PP] * 7 + [C.c_void_p, C.c_size_t, C.c_void_p]
lib.kvp_proj_bwd.restype = C.c_int
lib.kvp_proj_bwd.argtypes = [C.POINTER(Shape), C.POINTER(C.c_int32)] + [_PP] * 11 + [C.c_void_p, C.c_size_t, C.c_void_p]
lib.kvp_proj_bwd_range.restype = C.c_int
lib.kvp_proj_bwd_range.argtypes = [C.POINTER(Shape), C.POINTER(C.c_int32)] + [_PP] * 11 + [C.c_int, C.c_int, C.c_void_p, C.c_size_t,
                                                                                          C.c_void_p]
lib.kvp_out_proj_fwd.restype = C.c_int
lib.kvp_out_proj_fwd.argtypes = [C.POINTER(Shape)] + [_PP] * 3 + [C.c_void_p]
lib.kvp_out_proj_bwd.restype = C.c_int
lib.kvp_out_proj_bwd.argtypes = [C.POINTER(Shape)] + [_PP] * 5 + [C.c_void_p]
lib.kvp_attn_fwd.restype = C.c_int
lib.kvp_attn_fwd.argtypes = [C.POINTER(Shape), C.POINTER(C.c_int32), C.c_int, C.c_float] + [_PP] * 5 + \
    [C.c_void_p, C.c_size_t, C.c_void_p]
lib.kvp_attn_bwd.restype = C.c_int
lib.kvp_attn_bwd.argtypes = [C.POINTER(Shape), C.POINTER(C.c_int32), C.c_int, C.c_float] + [_PP] * 9 + \
    [C.c_void_p, C.c_size_t, C.c_void_p]


def workspace_bytes(op: int, shape: Shape, donor) -> int:
    return int(lib.kvp_workspace_bytes(op, C.byref(shape), _i32_array(donor)))


def _ws(ws: Optional[torch.Tensor]):
    return (C.c_void_p(_ptr(ws)), 0 if ws is None else ws.numel() * ws.element_size())


def proj_fwd(shape, donor, x, wq, wk, wv, q, k, v, ws=None):
    p, n = _ws(ws)
    _check(lib.kvp_proj_fwd(C.byref(shape), _i32_array(donor), _ptr_array(x), _ptr_array(wq), _ptr_array(wk),
                            _ptr_array(wv), _ptr_array(q), _ptr_array(k), _ptr_array(v), p, n, _stream()),
           "kvp_proj_fwd")


def proj_bwd(shape, donor, x, wq, wk, wv, dq, dk_sum, dv_sum, dwq, dwk, dwv, dx, ws, layer_begin=None, layer_end=None):
    """kvp_proj_bwd, or kvp_proj_bwd_range when a layer range is given."""
    p, n = _ws(ws)
    args = (C.byref(shape), _i32_array(donor), _ptr_array(x), _ptr_array(wq), _ptr_array(wk), _ptr_array(wv),
            _ptr_array(dq), _ptr_array(dk_sum), _ptr_array(dv_sum), _ptr_array(dwq), _ptr_array(dwk), _ptr_array(dwv),
            _ptr_array(dx))
    if layer_begin is None and layer_end is None:
        _check(lib.kvp_proj_bwd(*args, p, n, _stream()), "kvp_proj_bwd")
    else:
        _check(lib.kvp_proj_bwd_range(*args, int(layer_begin or 0), shape.L if layer_end is None else int(layer_end), p, n,
                                      _stream()), "kvp_proj_bwd_range")


def out_proj_fwd(shape, o, wo, y):
    _check(lib.kvp_out_proj_fwd(C.byref(shape), _ptr_array(o), _ptr_array(wo), _ptr_array(y), _stream()),
           "kvp_out_proj_fwd")


def out_proj_bwd(shape, o, wo, dy, d_o, dwo):
    _check(lib.kvp_out_proj_bwd(C.byref(shape), _ptr_array(o), _ptr_array(wo), _ptr_array(dy), _ptr_array(d_o),
                                _ptr_array(dwo), _stream()), "kvp_out_proj_bwd")


def attn_fwd(shape, donor, q, k, v, o, lse, causal=True, scale=0.0, ws=None):
    p, n = _ws(ws)
    _check(lib.kvp_attn_fwd(C.byref(shape), _i32_array(donor), int(causal), float(scale), _ptr_array(q),
                            _ptr_array(k), _ptr_array(v), _ptr_array(o), _ptr_array(lse), p, n, _stream()),
           "kvp_attn_fwd")


def attn_bwd(shape, donor, q, k, v, o, d_o, lse, dq, dk_sum, dv_sum, ws, causal=True, scale=0.0):
    p, n = _ws(ws)
    _check(lib.kvp_attn_bwd(C.byref(shape), _i32_array(donor), int(causal), float(scale), _ptr_array(q),
                            _ptr_array(k), _ptr_array(v), _ptr_array(o), _ptr_array(d_o), _ptr_array(lse),
                            _ptr_array(dq), _ptr_array(dk_sum), _ptr_array(dv_sum), p, n, _stream()), "kvp_attn_bwd")


# ------------------------------------------------------------------------------------------
# decode over the shared paged cache
# ------------------------------------------------------------------------------------------
class DecodeDesc(C.Structure):
    """kvp_decode_desc."""
    _fields_ = [(n, C.c_int32) for n in ("L", "B", "Hq", "Hkv", "dh", "page_size", "max_pages", "n_pages",
                                         "num_splits", "dtype")]

    def __init__(self, L, B, Hq, Hkv, dh, page_size, max_pages, n_pages, num_splits=0, dtype=0):
        super().__init__(L, B, Hq, Hkv, dh, page_size, max_pages, n_pages, num_splits, dtype)


lib.kvp_decode_workspace_bytes.restype = C.c_size_t
lib.kvp_decode_workspace_bytes.argtypes = [C.POINTER(DecodeDesc), C.POINTER(C.c_int32)]
lib.kvp_cache_append.restype = C.c_int
lib.kvp_cache_append.argtypes = [C.POINTER(DecodeDesc), C.POINTER(C.c_int32)] + [_PP] * 4 + \
    [C.c_void_p, C.c_void_p, C.c_void_p]
lib.kvp_decode.restype = C.c_int
lib.kvp_decode.argtypes = [C.POINTER(DecodeDesc), C.POINTER(C.c_int32), C.c_float] + [_PP] * 3 + \
    [C.c_void_p, C.c_void_p] + [_PP] * 2 + [C.c_int, C.c_int, C.c_void_p, C.c_size_t, C.c_void_p]


def decode_workspace_bytes(desc: DecodeDesc, donor) -> int:
    return int(lib.kvp_decode_workspace_bytes(C.byref(desc), _i32_array(donor)))


def cache_append(desc, donor, k_new, v_new, k_cache, v_cache, block_table, lengths):
    _check(lib.kvp_cache_append(C.byref(desc), _i32_array(donor), _ptr_array(k_new), _ptr_array(v_new),
                                _ptr_array(k_cache), _ptr_array(v_cache), block_table.data_ptr(),
                                lengths.data_ptr(), _stream()), "kvp_cache_append")


def decode(desc, donor, q, k_cache, v_cache, block_table, lengths, o, lse, ws, scale=0.0, layer_begin=0,
           layer_end=None):
    p, n = _ws(ws)
    _check(lib.kvp_decode(C.byref(desc), _i32_array(donor), float(scale), _ptr_array(q), _ptr_array(k_cache),
                          _ptr_array(v_cache), block_table.data_ptr(), lengths.data_ptr(), _ptr_array(o),
                          _ptr_array(lse), layer_begin, desc.L if layer_end is None else layer_end, p, n, _stream()),
           "kvp_decode")


# ------------------------------------------------------------------------------------------
# benchmark bookkeeping
# ------------------------------------------------------------------------------------------
KERNEL_GEMM, KERNEL_ATTN_FWD, KERNEL_ATTN_BWD, KERNEL_DECODE, KERNEL_ATTN_BWD_AUX = range(5)
lib.kvp_launch_count.restype = C.c_ulonglong
lib.kvp_set_timing_events.restype = C.c_int
lib.kvp_set_timing_events.argtypes = [C.c_int, _PP, _PP, C.c_int]
lib.kvp_timing_events_used.restype = C.c_int
lib.kvp_timing_events_used.argtypes = [C.c_int]


def launch_count() -> int:
    return int(lib.kvp_launch_count())


lib.kvp_set_gemm_pair_mode.restype = None
lib.kvp_set_gemm_pair_mode.argtypes = [C.c_int]


def set_gemm_pair_mode(mode: int) -> None:
    """kvp_set_gemm_pair_mode: 1 = CTA-pair tiles for the forward GEMMs (default), 0 = single-CTA tiles everywhere,
    2 = CTA pairs everywhere."""
    lib.kvp_set_gemm_pair_mode(int(mode))


class KernelTimer:
    """Records CUDA events around up to n launches of one of the library's kernels and returns the
    per-launch durations in milliseconds."""

    def __init__(self, kernel: int, n: int):
        self.kernel, self.n = kernel, n
        self.starts = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        self.stops = [torch.cuda.Event(enable_timing=True) for _ in range(n)]
        for e in self.starts + self.stops:
            e.record()            # torch creates the underlying event lazily, on first record
        torch.cuda.synchronize()
        self._a = (C.c_void_p * n)(*[e.cuda_event for e in self.starts])
        self._b = (C.c_void_p * n)(*[e.cuda_event for e in self.stops])

    def __enter__(self):
        _check(lib.kvp_set_timing_events(self.kernel, self._a, self._b, self.n), "kvp_set_timing_events")
        return self

    def __exit__(self, *exc):
        self.used = int(lib.kvp_timing_events_used(self.kernel))
        lib.kvp_set_timing_events(self.kernel, None, None, 0)

    def durations_ms(self):
        torch.cuda.synchronize()
        return [self.starts[i].elapsed_time(self.stops[i]) for i in range(self.used)]


lib.kvp_selftest_bounded_wait.restype = C.c_int
lib.kvp_selftest_bounded_wait.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]


lib.kvp_selftest_bounded_wait_pair.restype = C.c_int
lib.kvp_selftest_bounded_wait_pair.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]


def selftest_bounded_wait_pair(scratch: torch.Tensor):
    """kvp_selftest_bounded_wait_pair: the same self-test on the CTA-pair GEMM kernel (scratch of at least 768 KiB)."""
    _check(lib.kvp_selftest_bounded_wait_pair(scratch.data_ptr(), scratch.numel() * scratch.element_size(), _stream()),
           "kvp_selftest_bounded_wait_pair")


def selftest_bounded_wait(scratch: torch.Tensor):
    """kvp_selftest_bounded_wait: enqueue the GEMM whose ring-stage arrival is withheld once; afterwards
    device_status() returns ERR_TIMEOUT once and the library stays usable."""
    _check(lib.kvp_selftest_bounded_wait(scratch.data_ptr(), scratch.numel() * scratch.element_size(), _stream()),
           "kvp_selftest_bounded_wait")


# ------------------------------------------------------------------------------------------
# decode without a workspace: scratch lives in a fixed array inside the library
# ------------------------------------------------------------------------------------------
ERR_STATIC_SCRATCH = 7
DECODE_STATIC_SCRATCH_BYTES = 16 << 20
lib.kvp_decode_static.restype = C.c_int
lib.kvp_decode_static.argtypes = [C.POINTER(DecodeDesc), C.POINTER(C.c_int32), C.c_float] + [_PP] * 3 + \
    [C.c_void_p, C.c_void_p] + [_PP] * 2 + [C.c_int, C.c_int, C.c_void_p]


def decode_static(desc, donor, q, k_cache, v_cache, block_table, lengths, o, lse, scale=0.0, layer_begin=0,
                  layer_end=None):
    """kvp_decode_static: same results as `decode`, for callers that cannot allocate device memory
    (no workspace tensor is passed and the library allocates nothing).  Raises KvpError with
    ERR_STATIC_SCRATCH when the request does not fit the built-in DECODE_STATIC_SCRATCH_BYTES array.
    Calls share that array, so do not let two of them overlap on the GPU."""
    _check(lib.kvp_decode_static(C.byref(desc), _i32_array(donor), float(scale), _ptr_array(q), _ptr_array(k_cache),
                                 _ptr_array(v_cache), block_table.data_ptr(), lengths.data_ptr(), _ptr_array(o),
                                 _ptr_array(lse), layer_begin, desc.L if layer_end is None else layer_end, _stream()),
           "kvp_decode_static")
