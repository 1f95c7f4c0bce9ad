"""Thin ctypes binding over libswizzleperf.so: argument marshalling only.

Function names follow the C header (``include/swizzleperf.h``) without the ``sp_`` prefix.
Device buffers are torch CUDA tensors (PyTorch is used for device memory and streams
only); every step of the computation runs in the library's own kernels.  There is no
CPU fallback: if the shared library cannot be loaded the import of any entry point
raises.
"""

from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libswizzleperf.so")

# sp_status
OK, ERR_INVALID_ARG, ERR_NOT_BIJECTIVE, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_CUDA, ERR_TIMEOUT, ERR_DEVICE = range(8)
# sp_scheme
ROW_MAJOR, COL_MAJOR, GROUP_M, GROUP_N, MORTON, HILBERT, XCD, DIE_SPLIT, CUSTOM, HILBERT_RECT = range(10)
SCHEME_NAMES = ["row_major", "col_major", "group_m", "group_n", "morton", "hilbert", "xcd", "die_split", "custom", "hilbert_rect"]


class SpParams(ctypes.Structure):
    _fields_ = [
        ("struct_size", ctypes.c_uint32),
        ("group", ctypes.c_int32),
        ("num_xcds", ctypes.c_int32),
        ("wave", ctypes.c_int32),
        ("xcd_balanced", ctypes.c_int32),
        ("split_axis", ctypes.c_int32),
        ("inner_scheme", ctypes.c_int32),
        ("inner_group", ctypes.c_int32),
        ("interleave", ctypes.c_int32),
        ("custom_perm", ctypes.POINTER(ctypes.c_int32)),
        ("tile_m", ctypes.c_int32),
        ("tile_n", ctypes.c_int32),
        ("out_dtype", ctypes.c_int32),
        ("b_layout", ctypes.c_int32),
        ("flags", ctypes.c_uint32),
    ]


class SpTraceRec(ctypes.Structure):
    _fields_ = [("slot", ctypes.c_int32), ("tile", ctypes.c_int32), ("smid", ctypes.c_int32), ("unit", ctypes.c_int32),
                ("t_begin", ctypes.c_uint64), ("t_end", ctypes.c_uint64), ("t_mma_begin", ctypes.c_uint64),
                ("t_mma_issued", ctypes.c_uint64), ("mma_wait_data", ctypes.c_uint32), ("mma_wait_acc", ctypes.c_uint32),
                ("load_wait_stage", ctypes.c_uint32), ("epi_wait_acc", ctypes.c_uint32)]


TRACE_DTYPE = np.dtype([("slot", "<i4"), ("tile", "<i4"), ("smid", "<i4"), ("unit", "<i4"), ("t_begin", "<u8"),
                        ("t_end", "<u8"), ("t_mma_begin", "<u8"), ("t_mma_issued", "<u8"), ("mma_wait_data", "<u4"),
                        ("mma_wait_acc", "<u4"), ("load_wait_stage", "<u4"), ("epi_wait_acc", "<u4")])

EXPORTS = ["sp_tile_count", "sp_tile_map", "sp_tile_map_device", "sp_gemm", "sp_gemm_trace", "sp_gemm_host",
           "sp_gemm_noalloc", "sp_transpose", "sp_stencil2d", "sp_softmax", "sp_gemm_units", "sp_streamk_plan", "sp_recommend",
           "sp_probe_dispatch", "sp_probe_topology", "sp_probe_l2_capacity", "sp_selftest_timeout", "sp_selftest_pinned_tickets", "sp_get_status", "sp_last_error", "sp_shutdown"]


class SpError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"sp_status {status}: {message}")
        self.status = status


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2508_20258_b200.build` (needs nvcc)")
        L = ctypes.CDLL(LIB_PATH)
        i64, i32, vp = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p
        pp = ctypes.POINTER(SpParams)
        L.sp_tile_count.restype = i64
        L.sp_tile_count.argtypes = [i64, i64, i32, i32]
        L.sp_tile_map.restype = ctypes.c_int
        L.sp_tile_map.argtypes = [i64, i64, i32, i32, ctypes.c_int, pp, vp]
        L.sp_tile_map_device.restype = ctypes.c_int
        L.sp_tile_map_device.argtypes = [i64, i64, i32, i32, ctypes.c_int, pp, vp, vp]
        L.sp_gemm.restype = ctypes.c_int
        L.sp_gemm.argtypes = [vp, vp, vp, i64, i64, i64, ctypes.c_int, pp, vp]
        L.sp_gemm_trace.restype = ctypes.c_int
        L.sp_gemm_trace.argtypes = [vp, vp, vp, i64, i64, i64, ctypes.c_int, pp, vp, vp]
        L.sp_gemm_host.restype = ctypes.c_int
        L.sp_gemm_host.argtypes = [vp, vp, vp, i64, i64, i64, ctypes.c_int, pp, vp]
        L.sp_gemm_noalloc.restype = ctypes.c_int
        L.sp_gemm_noalloc.argtypes = [vp, vp, vp, i64, i64, i64, ctypes.c_int, pp, vp, ctypes.POINTER(ctypes.c_int32)]
        L.sp_transpose.restype = ctypes.c_int
        L.sp_transpose.argtypes = [vp, vp, i64, i64, ctypes.c_int, pp, vp]
        L.sp_stencil2d.restype = ctypes.c_int
        L.sp_stencil2d.argtypes = [vp, vp, i64, i64, ctypes.c_float, ctypes.c_float, ctypes.c_int, pp, vp]
        L.sp_softmax.restype = ctypes.c_int
        L.sp_softmax.argtypes = [vp, vp, i64, i64, i32, ctypes.c_int, pp, vp]
        L.sp_gemm_units.restype = ctypes.c_int
        L.sp_gemm_units.argtypes = [i32, i32, i64]
        L.sp_recommend.restype = ctypes.c_int
        L.sp_recommend.argtypes = [i64, i64, i64, i32, i32, pp, ctypes.POINTER(ctypes.c_int)]
        L.sp_streamk_plan.restype = ctypes.c_int
        L.sp_streamk_plan.argtypes = [i64, i32, i32, ctypes.POINTER(ctypes.c_int32), vp]
        L.sp_probe_dispatch.restype = ctypes.c_int
        L.sp_probe_dispatch.argtypes = [i32, i32, vp, vp]
        L.sp_probe_topology.restype = ctypes.c_int
        L.sp_probe_topology.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_float), vp]
        L.sp_probe_l2_capacity.restype = ctypes.c_int
        L.sp_probe_l2_capacity.argtypes = [i32, vp, i32, vp]
        L.sp_selftest_pinned_tickets.restype = ctypes.c_int
        L.sp_selftest_pinned_tickets.argtypes = [i32, i32, i32]
        L.sp_selftest_timeout.restype = ctypes.c_int
        L.sp_selftest_timeout.argtypes = [i32, ctypes.POINTER(ctypes.c_int32), ctypes.POINTER(ctypes.c_int64)]
        L.sp_get_status.restype = ctypes.c_int
        L.sp_get_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32)]
        L.sp_last_error.restype = ctypes.c_char_p
        L.sp_last_error.argtypes = []
        L.sp_shutdown.restype = None
        L.sp_shutdown.argtypes = []
        _lib = L
    return _lib


def last_error() -> str:
    return lib().sp_last_error().decode()


def _check(rc: int) -> None:
    if rc != OK:
        raise SpError(rc, last_error())


def make_params(group: int = 1, num_xcds: int = 1, wave: int = 0, xcd_balanced: int = 0, split_axis: int = 0,
                inner_scheme: int = ROW_MAJOR, inner_group: int = 1, interleave: int = 0,
                custom_perm: Optional[Sequence[int]] = None, tile_m: int = 0, tile_n: int = 0, out_dtype: int = 0,
                b_layout: int = 0, flags: int = 0) -> SpParams:
    p = SpParams()
    p.struct_size = ctypes.sizeof(SpParams)
    p.group, p.num_xcds, p.wave, p.xcd_balanced = group, num_xcds, wave, xcd_balanced
    p.split_axis, p.inner_scheme, p.inner_group, p.interleave = split_axis, inner_scheme, inner_group, interleave
    p.tile_m, p.tile_n, p.out_dtype, p.b_layout, p.flags = tile_m, tile_n, out_dtype, b_layout, flags
    if custom_perm is not None:
        arr = np.ascontiguousarray(np.asarray(custom_perm, dtype=np.int32))
        p._keepalive = arr  # the struct only holds a raw pointer
        p.custom_perm = arr.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    return p


def _pp(params: Optional[SpParams]):
    return ctypes.byref(params) if params is not None else None


def _stream_handle(stream) -> int:
    if stream is None:
        import torch
        return int(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def tile_count(M: int, N: int, tile_m: int, tile_n: int) -> int:
    return int(lib().sp_tile_count(M, N, tile_m, tile_n))


def tile_map(M: int, N: int, tile_m: int, tile_n: int, scheme: int, params: Optional[SpParams] = None) -> np.ndarray:
    """perm[s] = tile executed at slot s (host evaluation)."""
    T = tile_count(M, N, tile_m, tile_n)
    out = np.full(max(T, 1), -1, dtype=np.int32)
    _check(lib().sp_tile_map(M, N, tile_m, tile_n, scheme, _pp(params), out.ctypes.data))
    return out[:T]


def tile_map_device(M: int, N: int, tile_m: int, tile_n: int, scheme: int, params: Optional[SpParams] = None,
                    stream=None):
    """The same remap evaluated by the device code; returns an int32 CUDA tensor."""
    import torch
    T = tile_count(M, N, tile_m, tile_n)
    if T <= 0:
        raise SpError(ERR_INVALID_ARG, "sizes must be positive")
    out = torch.full((T,), -1, dtype=torch.int32, device="cuda")
    _check(lib().sp_tile_map_device(M, N, tile_m, tile_n, scheme, _pp(params), out.data_ptr(), _stream_handle(stream)))
    return out


def _dims(A, B, C, params: Optional[SpParams]):
    M, K = A.shape
    b_nk = bool(params.b_layout) if params is not None else False
    if b_nk:
        N, K2 = B.shape
    else:
        K2, N = B.shape
    if K2 != K or tuple(C.shape) != (M, N):
        raise ValueError("shape mismatch")
    for t in (A, B, C):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("A, B, C must be contiguous CUDA tensors")
    return M, N, K


def gemm(A, B, C, scheme: int = ROW_MAJOR, params: Optional[SpParams] = None, stream=None) -> None:
    """C = A . B on the current CUDA device under the given tile order (asynchronous)."""
    M, N, K = _dims(A, B, C, params)
    _check(lib().sp_gemm(A.data_ptr(), B.data_ptr(), C.data_ptr(), M, N, K, scheme, _pp(params), _stream_handle(stream)))


def gemm_noalloc(A, B, C, scheme: int = ROW_MAJOR, params: Optional[SpParams] = None, stream=None,
                 check_status: bool = False) -> None:
    """gemm() that performs no device allocation: its scratch is a fixed array inside the library
    (at most 65536 tiles; calls on one device must not overlap).  For callers whose device memory is
    entirely owned by their own pool, or that cannot afford an allocation's hidden synchronisation.
    With ``check_status`` the call synchronises the stream and raises if a device-side wait expired."""
    M, N, K = _dims(A, B, C, params)
    word = ctypes.c_int32(0)
    _check(lib().sp_gemm_noalloc(A.data_ptr(), B.data_ptr(), C.data_ptr(), M, N, K, scheme, _pp(params),
                                 _stream_handle(stream), ctypes.byref(word) if check_status else None))


def gemm_trace(A, B, C, scheme: int = ROW_MAJOR, params: Optional[SpParams] = None, stream=None) -> np.ndarray:
    """gemm() that also returns one record per slot (numpy structured array, TRACE_DTYPE)."""
    import torch
    M, N, K = _dims(A, B, C, params)
    tm = params.tile_m if params is not None and params.tile_m else 256
    tn = params.tile_n if params is not None and params.tile_n else 256
    T = tile_count(M, N, tm, tn)
    buf = torch.zeros((T * ctypes.sizeof(SpTraceRec),), dtype=torch.uint8, device="cuda")
    _check(lib().sp_gemm_trace(A.data_ptr(), B.data_ptr(), C.data_ptr(), M, N, K, scheme, _pp(params),
                               _stream_handle(stream), buf.data_ptr()))
    torch.cuda.synchronize()
    return np.frombuffer(buf.cpu().numpy().tobytes(), dtype=TRACE_DTYPE)


def _host_ptr(x) -> int:
    """Address of a host buffer: numpy array or CPU torch tensor (pinned or not)."""
    if isinstance(x, np.ndarray):
        if not x.flags["C_CONTIGUOUS"]:
            raise ValueError("host arrays must be C-contiguous")
        return int(x.ctypes.data)
    if x.is_cuda or not x.is_contiguous():
        raise ValueError("host tensors must be contiguous CPU tensors")
    return int(x.data_ptr())


def gemm_host(A, B, C, scheme: int = ROW_MAJOR, params: Optional[SpParams] = None, stream=None) -> None:
    """C = A . B for HOST matrices (bf16 bit patterns as uint16/bfloat16; C bf16 or fp32 per params).
    Copies in, computes on the GPU, copies out; C is valid on return."""
    M, K = A.shape
    b_nk = bool(params.b_layout) if params is not None else False
    N = B.shape[0] if b_nk else B.shape[1]
    if (B.shape[1] if b_nk else B.shape[0]) != K or tuple(C.shape) != (M, N):
        raise ValueError("shape mismatch")
    _check(lib().sp_gemm_host(_host_ptr(A), _host_ptr(B), _host_ptr(C), M, N, K, scheme, _pp(params),
                              _stream_handle(stream)))


TRANSPOSE_TILE = 64


def transpose(x, out, scheme: int = ROW_MAJOR, params: Optional[SpParams] = None, stream=None) -> None:
    """out [N, M] = x [M, N] transposed, 2-byte elements, tiles visited in the given order (asynchronous)."""
    M, N = x.shape
    if tuple(out.shape) != (N, M) or x.element_size() != 2 or out.element_size() != 2:
        raise ValueError("need a [M, N] input and a [N, M] output of 2-byte elements")
    for t in (x, out):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("x and out must be contiguous CUDA tensors")
    _check(lib().sp_transpose(x.data_ptr(), out.data_ptr(), M, N, scheme, _pp(params), _stream_handle(stream)))


STENCIL_TILE = (64, 128)


def stencil2d(x, out, c_center: float, c_neighbor: float, scheme: int = ROW_MAJOR, params: Optional[SpParams] = None,
              stream=None) -> None:
    """out = one five-point sweep over x (fp32 [M, N]; the rim is copied), tiles visited in the given order (asynchronous)."""
    import torch
    M, N = x.shape
    if tuple(out.shape) != (M, N) or x.dtype != torch.float32 or out.dtype != torch.float32:
        raise ValueError("need fp32 input and output of the same [M, N] shape")
    for t in (x, out):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("x and out must be contiguous CUDA tensors")
    _check(lib().sp_stencil2d(x.data_ptr(), out.data_ptr(), M, N, c_center, c_neighbor, scheme, _pp(params),
                              _stream_handle(stream)))


SOFTMAX_TILE = (32, 512)
SOFTMAX_SINGLE_PASS, SOFTMAX_TWO_PHASE, SOFTMAX_TWO_PHASE_REVERSED = 0, 1, 2


def softmax(x, out, mode: int = SOFTMAX_SINGLE_PASS, scheme: int = ROW_MAJOR, params: Optional[SpParams] = None,
            stream=None) -> None:
    """out = row softmax of x (fp32 [M, N]); single pass through shared memory, or the two-phase tiled form whose tiles
    are visited in the given order (asynchronous)."""
    import torch
    M, N = x.shape
    if tuple(out.shape) != (M, N) or x.dtype != torch.float32 or out.dtype != torch.float32:
        raise ValueError("need fp32 input and output of the same [M, N] shape")
    for t in (x, out):
        if not t.is_cuda or not t.is_contiguous():
            raise ValueError("x and out must be contiguous CUDA tensors")
    _check(lib().sp_softmax(x.data_ptr(), out.data_ptr(), M, N, mode, scheme, _pp(params), _stream_handle(stream)))


def gemm_units(tile_m: int, tile_n: int, T: int) -> int:
    return int(lib().sp_gemm_units(tile_m, tile_n, T))


FLAG_DIE_PINNED, FLAG_SERPENTINE, FLAG_STREAM_K, FLAG_OVERLAP, FLAG_CLC, FLAG_K_ALTERNATE = 2, 4, 8, 16, 32, 64
FLAG_STEAL = 4096
FLAG_TRACE = 1      # reserved (tracing is its own entry point)
FLAG_HINT_C_EVICT_FIRST, FLAG_HINT_A_EVICT_FIRST, FLAG_HINT_B_EVICT_FIRST, FLAG_HINT_A_EVICT_LAST, FLAG_HINT_B_EVICT_LAST = 128, 256, 512, 1024, 2048
STREAMK_MAX_SEGMENTS = 8
WORK_FULL, WORK_CONTRIB, WORK_OWNER = 0, 1, 2


def recommend(M: int, N: int, K: int, out_dtype: int = 0, b_layout: int = 0):
    """(scheme, params) the library suggests for this problem on B200: a table distilled from its own sweeps."""
    p = SpParams()
    scheme = ctypes.c_int(0)
    _check(lib().sp_recommend(M, N, K, out_dtype, b_layout, ctypes.byref(p), ctypes.byref(scheme)))
    return int(scheme.value), p


def streamk_plan(T: int, units: int, kblocks: int):
    """The k-split of SP_FLAG_STREAM_K: (first_slot, segments) with segments[u] = list of (slot, k0, k1, kind)
    in the order unit u walks them.  Host only."""
    first = ctypes.c_int32(0)
    out = np.zeros((units, STREAMK_MAX_SEGMENTS, 4), dtype=np.int32)
    _check(lib().sp_streamk_plan(T, units, kblocks, ctypes.byref(first), out.ctypes.data))
    segs = [[tuple(int(v) for v in out[u, j]) for j in range(STREAMK_MAX_SEGMENTS) if out[u, j, 0] >= 0]
            for u in range(units)]
    return int(first.value), segs


def probe_dispatch(n_blocks: int, cluster: int = 1):
    smid = np.zeros(n_blocks, dtype=np.int32)
    start = np.zeros(n_blocks, dtype=np.uint64)
    _check(lib().sp_probe_dispatch(n_blocks, cluster, smid.ctypes.data, start.ctypes.data))
    return smid, start


PROBE_LINES = 128


def probe_topology():
    """(sm_to_die[n_sm], confidence, latencies[n_sm, PROBE_LINES]) from the L2-latency probe."""
    die = np.full(1024, -1, dtype=np.int32)
    lat = np.zeros(1024 * PROBE_LINES, dtype=np.uint32)
    n = ctypes.c_int32(0)
    conf = ctypes.c_float(0)
    _check(lib().sp_probe_topology(die.ctypes.data, ctypes.byref(n), ctypes.byref(conf), lat.ctypes.data))
    return die[:n.value].copy(), float(conf.value), lat[:n.value * PROBE_LINES].reshape(n.value, PROBE_LINES).copy()


def probe_l2_capacity(sizes_bytes, half: int = -1) -> np.ndarray:
    """Aggregate re-read rate (GB/s) per working-set size; half = -1 all SMs, 0 / 1 one L2 half's SMs only."""
    sizes = np.ascontiguousarray(np.asarray(sizes_bytes, dtype=np.int64))
    out = np.zeros(len(sizes), dtype=np.float32)
    _check(lib().sp_probe_l2_capacity(len(sizes), sizes.ctypes.data, half, out.ctypes.data))
    return out


def selftest_timeout(timeout_us: int):
    """(status code recorded, microseconds waited) of a device-side wait that is made to expire."""
    code = ctypes.c_int32(0)
    waited = ctypes.c_int64(0)
    _check(lib().sp_selftest_timeout(timeout_us, ctypes.byref(code), ctypes.byref(waited)))
    return int(code.value), int(waited.value)


def get_status(stream=None) -> int:
    """Synchronises the stream; raises SpError(ERR_TIMEOUT) if a device-side wait expired."""
    detail = ctypes.c_int32(0)
    rc = lib().sp_get_status(_stream_handle(stream), ctypes.byref(detail))
    _check(rc)
    return int(detail.value)


def shutdown() -> None:
    lib().sp_shutdown()
