"""ctypes binding of libb200gemm.so: argument marshalling only.

Every function here has the name and meaning of the C entry point it calls
(see include/b200gemm.h); tensors are torch CUDA tensors used purely as device
memory, `stream` is a torch.cuda.Stream (default: the current stream).  There
is no fallback: if the shared library is missing or an entry point fails, an
exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

from . import build as _build

GEMM_OK = 0
PREC_FP16, PREC_S8, PREC_S4 = 0, 1, 2
PRECISION_ID = {"fp16": PREC_FP16, "s8": PREC_S8, "s4": PREC_S4}

EXPORTS = (
    "gemm_fp16", "gemm_s8", "gemm_s4", "gemm_s4_workspace_bytes", "gemm_s4_ws",
    "gemm_fp16_f16out", "gemm_s8_dequant", "gemm_s4_dequant", "gemm_host", "gemm_host_release",
    "gemm_s4_static", "gemm_s4_static_capacity", "gemm_release_workspaces", "gemm_unpack_s4", "gemm_mma_peak_probe", "gemm_query_config",
    "gemm_set_config_override", "gemm_set_kernel_family", "gemm_set_s4_scheme", "gemm_set_swap_ab", "gemm_set_l2_policy", "gemm_trace_enable", "gemm_trace_read", "gemm_set_stages_override", "gemm_debug_counters", "gemm_debug_host_cost", "gemm_debug_read_probe", "gemm_debug_reset_l2",
    "gemm_last_device_status", "gemm_read_device_status", "gemm_last_cuda_error",
    "gemm_status_string", "gemm_version",
)

_lib = None


class GemmError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        text = lib().gemm_status_string(code).decode()
        extra = ""
        if code == -5:
            extra = " (cudaError %d)" % lib().gemm_last_cuda_error()
        super().__init__("%s failed: %s [%d]%s" % (where, text, code, extra))


def library_path() -> str:
    return _build.LIB


def lib() -> ctypes.CDLL:
    """Loads the shared library (never builds it implicitly)."""
    global _lib
    if _lib is None:
        path = library_path()
        if not os.path.exists(path):
            raise ImportError(
                "%s not found: build it with `python -m paper_2608_10103_b200.build`" % path)
        L = ctypes.CDLL(path)
        vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.gemm_fp16.argtypes = [i, i, i, vp, vp, vp, vp]
        L.gemm_s8.argtypes = [i, i, i, vp, vp, vp, vp]
        L.gemm_s4.argtypes = [i, i, i, vp, vp, vp, vp]
        L.gemm_s4_ws.argtypes = [i, i, i, vp, vp, vp, vp, sz, vp]
        L.gemm_fp16_f16out.argtypes = [i, i, i, vp, vp, vp, vp]
        L.gemm_host.argtypes = [i, i, i, i, vp, vp, vp, vp]
        L.gemm_s8_dequant.argtypes = [i, i, i, vp, vp, vp, vp, vp, i, vp]
        L.gemm_s4_dequant.argtypes = [i, i, i, vp, vp, vp, vp, vp, i, vp]
        L.gemm_s4_workspace_bytes.argtypes = [i, i, i]
        L.gemm_s4_workspace_bytes.restype = sz
        L.gemm_s4_static.argtypes = [i, i, i, vp, vp, vp, vp]
        L.gemm_s4_static_capacity.argtypes = []
        L.gemm_s4_static_capacity.restype = sz
        L.gemm_unpack_s4.argtypes = [i, i, vp, vp, sz, vp]
        L.gemm_mma_peak_probe.argtypes = [i, i, i, i, ctypes.POINTER(ctypes.c_double), vp]
        L.gemm_query_config.argtypes = [i, i, i, i, ctypes.c_char_p, i]
        L.gemm_set_config_override.argtypes = [i, i, i, i]
        L.gemm_set_s4_scheme.argtypes = [i]
        L.gemm_set_kernel_family.argtypes = [i]
        L.gemm_set_stages_override.argtypes = [i]
        L.gemm_debug_counters.argtypes = [ctypes.POINTER(ctypes.c_longlong), i]
        L.gemm_debug_host_cost.argtypes = [i, i, i, i, vp, vp, vp, vp, i, ctypes.POINTER(ctypes.c_double)]
        L.gemm_debug_read_probe.argtypes = [vp, sz, vp]
        L.gemm_read_device_status.argtypes = [vp, vp]
        L.gemm_set_swap_ab.argtypes = [i]
        L.gemm_set_l2_policy.argtypes = [i]
        L.gemm_trace_enable.argtypes = [i]
        L.gemm_trace_read.argtypes = [ctypes.POINTER(ctypes.c_ulonglong), i]
        L.gemm_status_string.argtypes = [i]
        L.gemm_status_string.restype = ctypes.c_char_p
        for name in EXPORTS:
            fn = getattr(L, name)
            if name not in ("gemm_s4_workspace_bytes", "gemm_s4_static_capacity",
                            "gemm_status_string"):
                fn.restype = i
        _lib = L
    return _lib


def _stream_handle(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _check(rc: int, where: str):
    if rc != GEMM_OK:
        raise GemmError(rc, where)


def _dev_ptr(t: torch.Tensor, dtype, what: str) -> int:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError("%s must be a CUDA tensor" % what)
    if t.dtype != dtype:
        raise TypeError("%s must have dtype %s, got %s" % (what, dtype, t.dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % what)
    return t.data_ptr()


def _out(C, M, N, dtype, device):
    if C is None:
        C = torch.empty((M, N), dtype=dtype, device=device)
    elif tuple(C.shape) != (M, N):
        raise ValueError("C must have shape (%d, %d)" % (M, N))
    return C


def gemm_fp16(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor | None = None, stream=None):
    """C[M,N] (float32) = A[M,K] (float16) @ B[N,K]^T (float16)."""
    M, K = A.shape
    N, Kb = B.shape
    if K != Kb:
        raise ValueError("A and B disagree on K")
    C = _out(C, M, N, torch.float32, A.device)
    _check(lib().gemm_fp16(M, N, K, _dev_ptr(A, torch.float16, "A"), _dev_ptr(B, torch.float16, "B"),
                           _dev_ptr(C, torch.float32, "C"), _stream_handle(stream)), "gemm_fp16")
    return C


def gemm_s8(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor | None = None, stream=None):
    """C[M,N] (int32) = A[M,K] (int8) @ B[N,K]^T (int8), exact."""
    M, K = A.shape
    N, Kb = B.shape
    if K != Kb:
        raise ValueError("A and B disagree on K")
    C = _out(C, M, N, torch.int32, A.device)
    _check(lib().gemm_s8(M, N, K, _dev_ptr(A, torch.int8, "A"), _dev_ptr(B, torch.int8, "B"),
                         _dev_ptr(C, torch.int32, "C"), _stream_handle(stream)), "gemm_s8")
    return C


def gemm_s4(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor | None = None, stream=None):
    """C[M,N] (int32) = A @ B^T for packed signed 4-bit operands: A is (M, K/2)
    uint8, B is (N, K/2) uint8, low nibble first."""
    M, Kh = A.shape
    N, Khb = B.shape
    if Kh != Khb:
        raise ValueError("A and B disagree on K")
    C = _out(C, M, N, torch.int32, A.device)
    _check(lib().gemm_s4(M, N, 2 * Kh, _dev_ptr(A, torch.uint8, "A"), _dev_ptr(B, torch.uint8, "B"),
                         _dev_ptr(C, torch.int32, "C"), _stream_handle(stream)), "gemm_s4")
    return C


_HOST_DTYPES = {"fp16": (torch.float16, torch.float32), "s8": (torch.int8, torch.int32),
                "s4": (torch.uint8, torch.int32)}


def gemm_host(precision: str, A: torch.Tensor, B: torch.Tensor, C: torch.Tensor | None = None,
              stream=None):
    """C = A @ B^T for HOST tensors (pinned memory recommended).  Returns C (host); it is
    complete once `stream` (default: the current stream) has been synchronised."""
    in_dtype, out_dtype = _HOST_DTYPES[precision]
    for t, what in ((A, "A"), (B, "B")):
        if not isinstance(t, torch.Tensor) or t.is_cuda or t.dtype != in_dtype or not t.is_contiguous():
            raise TypeError("%s must be a contiguous CPU tensor of dtype %s" % (what, in_dtype))
    M, N = A.shape[0], B.shape[0]
    if A.shape[1] != B.shape[1]:
        raise ValueError("A and B disagree on K")
    K = A.shape[1] * (2 if precision == "s4" else 1)
    if C is None:
        C = torch.empty((M, N), dtype=out_dtype, pin_memory=True)
    elif C.is_cuda or C.dtype != out_dtype or tuple(C.shape) != (M, N) or not C.is_contiguous():
        raise TypeError("C must be a contiguous CPU tensor (%d, %d) of dtype %s" % (M, N, out_dtype))
    _check(lib().gemm_host(PRECISION_ID[precision], M, N, K, A.data_ptr(), B.data_ptr(),
                           C.data_ptr(), _stream_handle(stream)), "gemm_host")
    return C


def gemm_host_release():
    _check(lib().gemm_host_release(), "gemm_host_release")


def gemm_fp16_f16out(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor | None = None, stream=None):
    """C[M,N] (float16) = A[M,K] (float16) @ B[N,K]^T, FP32 accumulate, one rounding to half."""
    M, K = A.shape
    N, Kb = B.shape
    if K != Kb:
        raise ValueError("A and B disagree on K")
    C = _out(C, M, N, torch.float16, A.device)
    _check(lib().gemm_fp16_f16out(M, N, K, _dev_ptr(A, torch.float16, "A"),
                                  _dev_ptr(B, torch.float16, "B"), _dev_ptr(C, torch.float16, "C"),
                                  _stream_handle(stream)), "gemm_fp16_f16out")
    return C


def _dequant(fn_name, A, B, K, row_scale, col_scale, C, out_dtype, a_dtype, stream):
    M, N = A.shape[0], B.shape[0]
    if out_dtype not in (torch.float32, torch.float16):
        raise TypeError("out_dtype must be float32 or float16")
    C = _out(C, M, N, out_dtype, A.device)
    if row_scale.numel() != M or col_scale.numel() != N:
        raise ValueError("row_scale needs M entries, col_scale N")
    _check(getattr(lib(), fn_name)(M, N, K, _dev_ptr(A, a_dtype, "A"), _dev_ptr(B, a_dtype, "B"),
                                   _dev_ptr(row_scale, torch.float32, "row_scale"),
                                   _dev_ptr(col_scale, torch.float32, "col_scale"),
                                   _dev_ptr(C, out_dtype, "C"), 1 if out_dtype == torch.float16 else 0,
                                   _stream_handle(stream)), fn_name)
    return C


def gemm_s8_dequant(A, B, row_scale, col_scale, C=None, out_dtype=torch.float32, stream=None):
    """C[i,j] = float(int32 sum) * row_scale[i] * col_scale[j], as float32 or float16."""
    if A.shape[1] != B.shape[1]:
        raise ValueError("A and B disagree on K")
    return _dequant("gemm_s8_dequant", A, B, A.shape[1], row_scale, col_scale, C, out_dtype,
                    torch.int8, stream)


def gemm_s4_dequant(A, B, row_scale, col_scale, C=None, out_dtype=torch.float32, stream=None):
    """gemm_s8_dequant for packed signed 4-bit operands ((rows, K/2) uint8)."""
    if A.shape[1] != B.shape[1]:
        raise ValueError("A and B disagree on K")
    return _dequant("gemm_s4_dequant", A, B, 2 * A.shape[1], row_scale, col_scale, C, out_dtype,
                    torch.uint8, stream)


def gemm_s4_workspace_bytes(M: int, N: int, K: int) -> int:
    return int(lib().gemm_s4_workspace_bytes(M, N, K))


def gemm_s4_ws(A: torch.Tensor, B: torch.Tensor, workspace: torch.Tensor,
               C: torch.Tensor | None = None, stream=None):
    """gemm_s4 with caller-owned scratch (a uint8 CUDA tensor)."""
    M, Kh = A.shape
    N, Khb = B.shape
    if Kh != Khb:
        raise ValueError("A and B disagree on K")
    C = _out(C, M, N, torch.int32, A.device)
    _check(lib().gemm_s4_ws(M, N, 2 * Kh, _dev_ptr(A, torch.uint8, "A"),
                            _dev_ptr(B, torch.uint8, "B"), _dev_ptr(C, torch.int32, "C"),
                            _dev_ptr(workspace, torch.uint8, "workspace"), workspace.numel(),
                            _stream_handle(stream)), "gemm_s4_ws")
    return C


def gemm_s4_static(A: torch.Tensor, B: torch.Tensor, C: torch.Tensor | None = None, stream=None):
    """gemm_s4 without any device allocation inside the library: the unpacked
    operands go to a fixed 32 MiB array in the library's device image.  Pass C
    (preallocated) if the caller itself must not allocate either.  Problems
    whose workspace exceeds gemm_s4_static_capacity() raise GemmError(-7)."""
    M, Kh = A.shape
    N, Khb = B.shape
    if Kh != Khb:
        raise ValueError("A and B disagree on K")
    C = _out(C, M, N, torch.int32, A.device)
    _check(lib().gemm_s4_static(M, N, 2 * Kh, _dev_ptr(A, torch.uint8, "A"),
                                _dev_ptr(B, torch.uint8, "B"), _dev_ptr(C, torch.int32, "C"),
                                _stream_handle(stream)), "gemm_s4_static")
    return C


def gemm_s4_static_capacity() -> int:
    return int(lib().gemm_s4_static_capacity())


def gemm_unpack_s4(packed: torch.Tensor, out: torch.Tensor | None = None, stream=None):
    """(rows, K/2) uint8 packed nibbles -> (rows, K) int8."""
    rows, Kh = packed.shape
    K = 2 * Kh
    if out is None:
        out = torch.empty((rows, K), dtype=torch.int8, device=packed.device)
    _check(lib().gemm_unpack_s4(rows, K, _dev_ptr(packed, torch.uint8, "packed"),
                                _dev_ptr(out, torch.int8, "out"), out.stride(0),
                                _stream_handle(stream)), "gemm_unpack_s4")
    return out


def gemm_release_workspaces():
    _check(lib().gemm_release_workspaces(), "gemm_release_workspaces")


def gemm_mma_peak_probe(precision: str, iters: int, n_cols: int = 256, commit_every: int = 0,
                        stream=None) -> float:
    """Launches the MMA-only probe; returns the operation count it performs."""
    ops = ctypes.c_double(0.0)
    _check(lib().gemm_mma_peak_probe(PRECISION_ID[precision], iters, n_cols, commit_every,
                                     ctypes.byref(ops), _stream_handle(stream)),
           "gemm_mma_peak_probe")
    return ops.value


def gemm_query_config(precision: str, M: int, N: int, K: int) -> str:
    buf = ctypes.create_string_buffer(256)
    _check(lib().gemm_query_config(PRECISION_ID[precision], M, N, K, buf, 256), "gemm_query_config")
    return buf.value.decode()


def gemm_set_config_override(bn: int = 0, group_m: int = 0, cta_group: int = 0, split_k: int = 0):
    _check(lib().gemm_set_config_override(bn, group_m, cta_group, split_k),
           "gemm_set_config_override")


def gemm_set_kernel_family(family: int = 0):
    """Kernel family: 0 = automatic, 1 = 256 x 256 tile per CTA pair, 2 = 512 x 256 (large
    problems); 3 = the integer kernel for a few rows wherever it exists (a short side of up to
    32 rows; 1 and 2 never take it)."""
    _check(lib().gemm_set_kernel_family(int(family)), "gemm_set_kernel_family")


def gemm_set_stages_override(stages: int = 0):
    """Ring depth of the 256 x 256 CTA-pair kernel (raw outputs): 0 = shipped (6), or 3..6."""
    _check(lib().gemm_set_stages_override(int(stages)), "gemm_set_stages_override")


def gemm_debug_counters() -> dict:
    """Host-side counters: tensor maps encoded so far, scratch buffers pooled on the current
    device, whether this thread's last INT4 call ran the overlapped pre-pass."""
    buf = (ctypes.c_longlong * 3)()
    _check(lib().gemm_debug_counters(buf, 3), "gemm_debug_counters")
    return {"map_encodes": int(buf[0]), "pool_buffers": int(buf[1]), "s4_overlapped": int(buf[2])}


def gemm_debug_host_cost(precision: str, A: torch.Tensor, B: torch.Tensor, C: torch.Tensor,
                         stream=None, calls: int = 200) -> float:
    """Host nanoseconds per call of gemm_fp16 / gemm_s8 / gemm_s4 on these device tensors,
    timed inside the library over `calls` (<= 512) back-to-back calls after a stream sync."""
    M, N = A.shape[0], B.shape[0]
    K = A.shape[1] * (2 if precision == "s4" else 1)
    out = ctypes.c_double(0.0)
    _check(lib().gemm_debug_host_cost(PRECISION_ID[precision], M, N, K, A.data_ptr(), B.data_ptr(),
                                      C.data_ptr(), _stream_handle(stream), int(calls),
                                      ctypes.byref(out)), "gemm_debug_host_cost")
    return float(out.value)


def gemm_debug_read_probe(data: torch.Tensor, stream=None):
    """Enqueues a kernel that reads `data` (device tensor, a multiple of 16 bytes) once and
    keeps nothing: the time a call bound by reading that operand could at best take."""
    if not data.is_cuda or not data.is_contiguous():
        raise ValueError("data must be a contiguous CUDA tensor")
    _check(lib().gemm_debug_read_probe(data.data_ptr(), data.numel() * data.element_size(),
                                       _stream_handle(stream)), "gemm_debug_read_probe")


def gemm_debug_reset_l2():
    """Waits for the device and returns L2 lines held with raised priority ("evict last") to
    normal status, so that a following measurement starts from an L2 an ordinary flush can clear."""
    _check(lib().gemm_debug_reset_l2(), "gemm_debug_reset_l2")


def gemm_read_device_status(host_out: torch.Tensor, stream=None):
    """Enqueues a copy of the device status word into `host_out` (a pinned int32 CPU tensor of
    one element) on `stream`; the value is there once the stream has passed the copy."""
    if host_out.is_cuda or host_out.dtype != torch.int32 or host_out.numel() < 1:
        raise TypeError("host_out must be an int32 CPU tensor")
    _check(lib().gemm_read_device_status(host_out.data_ptr(), _stream_handle(stream)),
           "gemm_read_device_status")


def gemm_set_s4_scheme(scheme: int = 0):
    """Route of gemm_s4 / gemm_s4_dequant: 0 = automatic (nibbles expanded inside the GEMM
    kernel for problems with few rows on one side, else a pre-pass to int8 + the INT8 GEMM);
    1 = always the pre-pass; 2 = inside the GEMM kernel wherever such a variant is built;
    4 = the pre-pass done by extra warps of the INT8 GEMM kernel where that applies;
    5 / 6 = as 2, never / always with A as an int8 image made beforehand on the CTA-pair tiles
    (the automatic rule takes that form for large N x K against a short M)."""
    _check(lib().gemm_set_s4_scheme(int(scheme)), "gemm_set_s4_scheme")


def gemm_set_swap_ab(mode: int = 0):
    """Run the kernel on exchanged operands (long operand on the 128-row tile side, C stored
    along N by plain stores): 0 = automatic (N >= 1024 and M <= 32, M <= 64 for INT8 / INT4 / FP16 output), 1 = never, 2 = always."""
    _check(lib().gemm_set_swap_ab(int(mode)), "gemm_set_swap_ab")


def gemm_set_l2_policy(policy: int = 11):
    """Bit set: bits 0-1 operand eviction priority (0 normal, 1 keep A / stream B, 2 keep
    both, 3 keep A), +4 serpentine K order off, +8 C stores evict-first, +16 128-byte L2
    promotion, +32 plain stream order (no programmatic dependent launch).  Default 11."""
    _check(lib().gemm_set_l2_policy(int(policy)), "gemm_set_l2_policy")


TRACE_FIELDS = ("cycles", "nanos", "producer_wait", "mma_wait_operands", "mma_wait_accumulator",
                "epilogue_wait", "epilogue_busy", "tiles", "mma_issue", "mma_commit", "setup",
                "producer_issue", "unpack_wait_packed", "unpack_wait_slot", "unpack_busy", "mma_wait_accumulator1")
TRACE_SLOTS = len(TRACE_FIELDS)


def gemm_trace_enable(flags: int = 1):
    """1 = record cycles; +2 = issue no MMAs; +4 = issue no operand loads; +8 = epilogue
    waits back off with nanosleep; +16 = failure drill (a slot is never filled: the bounded
    waits expire and the kernel reports it); +32 = epilogue stores C straight from registers;
    +64 = epilogue reads TMEM in the 16x256b shape and stores whole 32-byte sectors; 0 = off."""
    _check(lib().gemm_trace_enable(int(flags)), "gemm_trace_enable")


def gemm_trace_read(max_ctas: int = 160):
    """Per-CTA cycle accounting of the last traced launch: list of dicts."""
    buf = (ctypes.c_ulonglong * (TRACE_SLOTS * max_ctas))()
    n = lib().gemm_trace_read(buf, max_ctas)
    if n < 0:
        raise GemmError(n, "gemm_trace_read")
    return [dict(zip(TRACE_FIELDS, buf[TRACE_SLOTS * c: TRACE_SLOTS * (c + 1)])) for c in range(n)]


def gemm_last_device_status() -> int:
    return int(lib().gemm_last_device_status())


def gemm_status_string(code: int) -> str:
    return lib().gemm_status_string(code).decode()


def gemm_last_cuda_error() -> int:
    return int(lib().gemm_last_cuda_error())


def gemm_version() -> int:
    return int(lib().gemm_version())


def gemm(precision: str, A, B, C=None, stream=None):
    """Dispatch by precision name ("fp16", "s8", "s4")."""
    return {"fp16": gemm_fp16, "s8": gemm_s8, "s4": gemm_s4}[precision](A, B, C, stream)
