"""ctypes binding of libcompass.so: same names as the C ABI, argument
marshalling only.  torch provides device memory and streams; every step of the
path runs inside the library.  There is no fallback: if the library is missing
the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libcompass.so")

OK, ERR_INVALID_ARG, ERR_SHAPE, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_BUFFER_TOO_SMALL, ERR_CUDA, ERR_TIMEOUT = range(8)
ERR_SCRATCH_LIMIT = 8
NOALLOC_SCRATCH_BYTES = 32 * 1024 * 1024
OP_AG_GEMM, OP_GEMM_RS = 0, 1
DTYPE_BF16 = 0
RS_SEGMENTED_K, RS_RING_RMW, RS_RING_RMW_F32 = 0, 1, 2
STRATEGY_INTRAFUSION, STRATEGY_INTERDECOM = 0, 1
ORDER_RANK_MAJOR, ORDER_STEP_MAJOR = 0, 1
COPY_KERNEL, COPY_ENGINES = 0, 1
WS_FUSED, WS_DECOMP, WS_PUSH = 0, 1, 2
ACT_NONE, ACT_GELU_TANH, ACT_SWIGLU = 0, 1, 2
B_NK, B_KN = 0, 1
MAX_P = 16
STATUS_BYTES = 256

# every symbol include/compass.h declares
EXPORTS = (
    "compass_schedule", "compass_ag_gemm", "compass_gemm_rs", "compass_decomp", "compass_select",
    "compass_model_decomp_time", "compass_model_optimal_degree", "compass_model_fusion_time",
    "compass_calib_fit_decomp", "compass_calib_fit_fusion", "compass_workspace_bytes", "compass_workspace_init",
    "compass_read_status", "compass_launch_plan", "compass_fused_host", "compass_status_string",
    "compass_last_cuda_error", "compass_kernel_launch_count", "compass_gemm_rs_sequential_noalloc",
    "compass_set_wait_limit_us", "compass_calib_fit_line", "compass_ag_gemm_push", "compass_read_kernel_clock",
    "compass_mlp_workspace_bytes", "compass_mlp_block", "compass_noalloc_read_status", "compass_select_ex", "compass_test_drop_flag_writes", "compass_tensor_map_cache_stats", "compass_decomp_comm", "compass_tile_plan",
)


class CompassError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status}, cuda error {last_cuda_error()})")


class Problem(C.Structure):
    _fields_ = [("op", C.c_int32), ("P", C.c_int32), ("rings", C.c_int32), ("d", C.c_int32),
                ("M", C.c_int64), ("N", C.c_int64), ("K", C.c_int64),
                ("dtype", C.c_int32), ("rs_variant", C.c_int32), ("order", C.c_int32), ("copy_mode", C.c_int32),
                ("b_layout", C.c_int32), ("ring_group", C.c_int32)]


class Mlp(C.Structure):
    _fields_ = [("P", C.c_int32), ("rings", C.c_int32), ("M", C.c_int64), ("hidden", C.c_int64), ("ffn", C.c_int64),
                ("activation", C.c_int32), ("rs_variant", C.c_int32), ("order", C.c_int32), ("b_layout", C.c_int32)]


class SchedEntry(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("rank", "step", "ring", "part", "chunk", "peer", "row_begin", "row_count")]


class Calib(C.Structure):
    _fields_ = [(n, C.c_double) for n in ("comp_a", "comp_b", "comm_a", "comm_b",
                                           "alpha_decomp", "beta_decomp", "alpha_fusion", "beta_fusion")]


class Choice(C.Structure):
    _fields_ = [("strategy", C.c_int32), ("d_star", C.c_int32), ("t_fusion", C.c_double), ("t_decomp", C.c_double),
                ("t_comp", C.c_double), ("t_comm", C.c_double), ("lam", C.c_double), ("t_star", C.c_double)]


class TileCounts(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("cta_pairs", "blocks", "rows_per_block", "blocks_per_group", "tiles_512x256",
                                          "tiles_256x256", "tiles_256x128", "tiles_128x256", "total_tiles")]


class PlanBlock(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("rank", "step", "ring", "part", "a_tensor", "a_row_begin", "out_tensor",
                                          "out_row_begin", "rows", "first_tile", "tile_count")]


_lib: Optional[C.CDLL] = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_10549_b200.build` "
                               "(there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        pp = C.POINTER(C.c_void_p)
        L.compass_schedule.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int64, C.POINTER(SchedEntry), C.c_size_t,
                                       C.POINTER(C.c_size_t)]
        for name in ("compass_ag_gemm", "compass_gemm_rs"):
            getattr(L, name).argtypes = [C.POINTER(Problem), pp, pp, pp, C.c_void_p, C.c_size_t, C.c_void_p]
        L.compass_decomp.argtypes = [C.POINTER(Problem), pp, pp, pp, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.compass_decomp_comm.argtypes = [C.POINTER(Problem), pp, pp, pp, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.compass_ag_gemm_push.argtypes = [C.POINTER(Problem), pp, pp, pp, C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
        L.compass_mlp_workspace_bytes.argtypes = [C.POINTER(Mlp), C.POINTER(C.c_size_t)]
        L.compass_mlp_block.argtypes = [C.POINTER(Mlp), pp, pp, pp, pp, pp, C.c_void_p, C.c_size_t, C.c_void_p]
        L.compass_select.argtypes = [C.POINTER(Problem), C.POINTER(Calib), C.POINTER(Choice)]
        L.compass_select_ex.argtypes = [C.POINTER(Problem), C.POINTER(Calib), C.c_int, C.POINTER(Choice)]
        L.compass_model_decomp_time.argtypes = [C.c_double] * 4 + [C.c_int, C.POINTER(C.c_double)]
        L.compass_model_optimal_degree.argtypes = [C.c_double] * 4 + [C.c_int, C.c_int, C.POINTER(C.c_int),
                                                                       C.POINTER(C.c_double)]
        L.compass_model_fusion_time.argtypes = [C.c_double, C.c_double, C.c_int, C.c_double, C.c_double, C.c_double,
                                                C.POINTER(C.c_double)]
        dp, ip = C.POINTER(C.c_double), C.POINTER(C.c_int)
        L.compass_calib_fit_decomp.argtypes = [dp, dp, ip, dp, C.c_size_t, dp, dp]
        L.compass_calib_fit_fusion.argtypes = [dp, dp, ip, dp, dp, C.c_size_t, dp, dp]
        L.compass_calib_fit_line.argtypes = [dp, dp, C.c_size_t, dp, dp]
        L.compass_workspace_bytes.argtypes = [C.POINTER(Problem), C.c_int, C.POINTER(C.c_size_t)]
        L.compass_workspace_init.argtypes = [C.c_void_p, C.c_size_t, C.c_void_p]
        L.compass_read_status.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_int)]
        L.compass_read_kernel_clock.argtypes = [C.c_void_p, C.c_void_p, C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
        L.compass_launch_plan.argtypes = [C.POINTER(Problem), C.POINTER(PlanBlock), C.c_size_t, C.POINTER(C.c_size_t)]
        L.compass_tile_plan.argtypes = [C.POINTER(Problem), C.c_int, C.c_int, C.POINTER(TileCounts)]
        L.compass_fused_host.argtypes = [C.POINTER(Problem), pp, pp, pp, C.c_void_p, C.c_size_t, C.POINTER(C.c_size_t),
                                         C.c_void_p, C.c_size_t, C.c_void_p]
        L.compass_gemm_rs_sequential_noalloc.argtypes = [C.POINTER(Problem), pp, pp, pp, C.c_void_p]
        L.compass_noalloc_read_status.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
        L.compass_set_wait_limit_us.argtypes = [C.c_uint32]
        L.compass_test_drop_flag_writes.argtypes = [C.c_int]
        L.compass_tensor_map_cache_stats.argtypes = [C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
        L.compass_status_string.argtypes = [C.c_int]
        L.compass_status_string.restype = C.c_char_p
        L.compass_last_cuda_error.restype = C.c_int
        L.compass_kernel_launch_count.restype = C.c_uint64
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().compass_status_string(int(status)).decode()


def last_cuda_error() -> int:
    return int(lib().compass_last_cuda_error())


def compass_set_wait_limit_us(microseconds: int) -> None:
    _check(lib().compass_set_wait_limit_us(int(microseconds)), "compass_set_wait_limit_us")


def compass_test_drop_flag_writes(count: int) -> None:
    _check(lib().compass_test_drop_flag_writes(int(count)), "compass_test_drop_flag_writes")


def tensor_map_cache_stats():
    """(hits, misses) of the library's table of encoded TMA tensor maps since it was loaded."""
    hits, misses = C.c_uint64(0), C.c_uint64(0)
    _check(lib().compass_tensor_map_cache_stats(C.byref(hits), C.byref(misses)), "compass_tensor_map_cache_stats")
    return int(hits.value), int(misses.value)


def kernel_launch_count() -> int:
    return int(lib().compass_kernel_launch_count())


def _check(status: int, where: str) -> None:
    if status != OK:
        raise CompassError(status, where)


def make_problem(op: int, P: int, M: int, N: int, K: int, rings: int = 2, d: int = 1,
                 rs_variant: int = RS_SEGMENTED_K, dtype: int = DTYPE_BF16, order: int = ORDER_RANK_MAJOR,
                 copy_mode: int = COPY_KERNEL, b_layout: int = B_NK, ring_group: int = 0) -> Problem:
    return Problem(op=op, P=P, rings=rings, d=d, M=M, N=N, K=K, dtype=dtype, rs_variant=rs_variant, order=order,
                   copy_mode=copy_mode, b_layout=b_layout, ring_group=ring_group)


# ---- host-only calls -------------------------------------------------------------

def compass_schedule(op: int, P: int, rings: int, M: int) -> np.ndarray:
    """Returns the schedule as an int32 array [count, 8] (columns as in compass_sched_entry)."""
    n = C.c_size_t(0)
    _check(lib().compass_schedule(op, P, rings, M, None, 0, C.byref(n)), "compass_schedule")
    buf = (SchedEntry * n.value)()
    _check(lib().compass_schedule(op, P, rings, M, buf, n.value, C.byref(n)), "compass_schedule")
    return np.frombuffer(buf, dtype=np.int32).reshape(n.value, 8).copy()


def compass_select(problem: Problem, calib: Calib, eq5_as_printed: bool = False) -> Choice:
    out = Choice()
    if eq5_as_printed:
        _check(lib().compass_select_ex(C.byref(problem), C.byref(calib), 1, C.byref(out)), "compass_select_ex")
    else:
        _check(lib().compass_select(C.byref(problem), C.byref(calib), C.byref(out)), "compass_select")
    return out


def compass_model_decomp_time(t_comp: float, t_comm: float, alpha: float, beta: float, d: int) -> float:
    out = C.c_double()
    _check(lib().compass_model_decomp_time(t_comp, t_comm, alpha, beta, d, C.byref(out)), "compass_model_decomp_time")
    return out.value


def compass_model_optimal_degree(t_comp: float, t_comm: float, alpha: float, beta: float, d_max: int = 16,
                                 as_printed: bool = False):
    d, x = C.c_int(), C.c_double()
    _check(lib().compass_model_optimal_degree(t_comp, t_comm, alpha, beta, d_max, int(as_printed), C.byref(d),
                                              C.byref(x)), "compass_model_optimal_degree")
    return d.value, (x.value if x.value >= 0 else None)


def compass_model_fusion_time(t_comp: float, t_comm: float, n_chunks: int, alpha_f: float, beta_f: float,
                              m_volume: float) -> float:
    out = C.c_double()
    _check(lib().compass_model_fusion_time(t_comp, t_comm, n_chunks, alpha_f, beta_f, m_volume, C.byref(out)),
           "compass_model_fusion_time")
    return out.value


def _darr(xs):
    return (C.c_double * len(xs))(*[float(x) for x in xs])


def _iarr(xs):
    return (C.c_int * len(xs))(*[int(x) for x in xs])


def compass_calib_fit_decomp(t_comp, t_comm, d, t_measured):
    a, b = C.c_double(), C.c_double()
    _check(lib().compass_calib_fit_decomp(_darr(t_comp), _darr(t_comm), _iarr(d), _darr(t_measured), len(d),
                                          C.byref(a), C.byref(b)), "compass_calib_fit_decomp")
    return a.value, b.value


def compass_calib_fit_line(x, y):
    a, b = C.c_double(), C.c_double()
    _check(lib().compass_calib_fit_line(_darr(x), _darr(y), len(x), C.byref(a), C.byref(b)), "compass_calib_fit_line")
    return a.value, b.value


def compass_calib_fit_fusion(t_comp, t_comm, n_chunks, m_volume, t_measured):
    a, b = C.c_double(), C.c_double()
    _check(lib().compass_calib_fit_fusion(_darr(t_comp), _darr(t_comm), _iarr(n_chunks), _darr(m_volume),
                                          _darr(t_measured), len(n_chunks), C.byref(a), C.byref(b)),
           "compass_calib_fit_fusion")
    return a.value, b.value


def compass_workspace_bytes(problem: Problem, which: int = WS_FUSED) -> int:
    n = C.c_size_t(0)
    _check(lib().compass_workspace_bytes(C.byref(problem), which, C.byref(n)), "compass_workspace_bytes")
    return int(n.value)


def compass_tile_plan(problem: Problem, decomposed: bool = False, cta_pairs: int = 74) -> TileCounts:
    out = TileCounts()
    _check(lib().compass_tile_plan(C.byref(problem), int(decomposed), int(cta_pairs), C.byref(out)), "compass_tile_plan")
    return out


def compass_launch_plan(problem: Problem) -> List[PlanBlock]:
    n = C.c_size_t(0)
    _check(lib().compass_launch_plan(C.byref(problem), None, 0, C.byref(n)), "compass_launch_plan")
    buf = (PlanBlock * n.value)()
    _check(lib().compass_launch_plan(C.byref(problem), buf, n.value, C.byref(n)), "compass_launch_plan")
    return list(buf)


# ---- device calls (torch tensors supply the memory) ------------------------------

def _ptr_array(tensors: Sequence) -> C.Array:
    return (C.c_void_p * len(tensors))(*[int(t.data_ptr()) for t in tensors])


def _stream_handle(stream) -> C.c_void_p:
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return C.c_void_p(int(stream.cuda_stream))


def _ws(workspace):
    return C.c_void_p(int(workspace.data_ptr())), int(workspace.numel() * workspace.element_size())


def compass_workspace_init(workspace, stream=None) -> None:
    p, n = _ws(workspace)
    _check(lib().compass_workspace_init(p, n, _stream_handle(stream)), "compass_workspace_init")


def compass_read_status(workspace, stream=None):
    detail = C.c_int(0)
    p, _ = _ws(workspace)
    st = lib().compass_read_status(p, _stream_handle(stream), C.byref(detail))
    return int(st), int(detail.value)


def compass_read_kernel_clock(workspace, stream=None):
    """(SM cycles, nanoseconds) of CTA 0 of the last GEMM kernel that used this workspace."""
    cycles, ns = C.c_uint64(0), C.c_uint64(0)
    p, _ = _ws(workspace)
    _check(lib().compass_read_kernel_clock(p, _stream_handle(stream), C.byref(cycles), C.byref(ns)),
           "compass_read_kernel_clock")
    return int(cycles.value), int(ns.value)


def compass_ag_gemm(problem: Problem, A: Sequence, B: Sequence, Cout: Sequence, workspace, stream=None) -> None:
    p, n = _ws(workspace)
    _check(lib().compass_ag_gemm(C.byref(problem), _ptr_array(A), _ptr_array(B), _ptr_array(Cout), p, n,
                                 _stream_handle(stream)), "compass_ag_gemm")


def compass_gemm_rs(problem: Problem, A: Sequence, B: Sequence, Out: Sequence, workspace, stream=None) -> None:
    p, n = _ws(workspace)
    _check(lib().compass_gemm_rs(C.byref(problem), _ptr_array(A), _ptr_array(B), _ptr_array(Out), p, n,
                                 _stream_handle(stream)), "compass_gemm_rs")


def compass_ag_gemm_push(problem: Problem, A: Sequence, B: Sequence, Cout: Sequence, workspace, stream_compute,
                         stream_copy) -> None:
    p, n = _ws(workspace)
    _check(lib().compass_ag_gemm_push(C.byref(problem), _ptr_array(A), _ptr_array(B), _ptr_array(Cout), p, n,
                                      _stream_handle(stream_compute), _stream_handle(stream_copy)), "compass_ag_gemm_push")


def make_mlp(P: int, M: int, hidden: int, ffn: int, activation: int = 0, rings: int = 2,
             rs_variant: int = RS_SEGMENTED_K, order: int = ORDER_RANK_MAJOR, b_layout: int = B_NK) -> Mlp:
    return Mlp(P=P, rings=rings, M=M, hidden=hidden, ffn=ffn, activation=activation, rs_variant=rs_variant,
               order=order, b_layout=b_layout)


def compass_mlp_workspace_bytes(mlp: Mlp) -> int:
    n = C.c_size_t(0)
    _check(lib().compass_mlp_workspace_bytes(C.byref(mlp), C.byref(n)), "compass_mlp_workspace_bytes")
    return int(n.value)


def alloc_mlp_workspace(mlp: Mlp, device="cuda"):
    import torch
    ws = torch.empty(compass_mlp_workspace_bytes(mlp), dtype=torch.uint8, device=device)
    compass_workspace_init(ws)
    return ws


def compass_mlp_block(mlp: Mlp, X: Sequence, W0: Sequence, H: Sequence, W1: Sequence, Out: Sequence, workspace,
                      stream=None) -> None:
    p, n = _ws(workspace)
    _check(lib().compass_mlp_block(C.byref(mlp), _ptr_array(X), _ptr_array(W0), _ptr_array(H), _ptr_array(W1),
                                   _ptr_array(Out), p, n, _stream_handle(stream)), "compass_mlp_block")


def compass_decomp(problem: Problem, A: Sequence, B: Sequence, out: Sequence, workspace, stream_compute=None,
                   stream_copy=None) -> None:
    p, n = _ws(workspace)
    sc = _stream_handle(stream_compute)
    sp = _stream_handle(stream_copy) if stream_copy is not None else sc
    _check(lib().compass_decomp(C.byref(problem), _ptr_array(A), _ptr_array(B), _ptr_array(out), p, n, sc, sp),
           "compass_decomp")


def compass_decomp_comm(problem: Problem, A: Sequence, B: Sequence, out: Sequence, workspace, stream_compute=None,
                        stream_copy=None) -> None:
    """The d sub-collectives of compass_decomp alone (no sub-GEMMs): T_comm, measurable on its own."""
    p, n = _ws(workspace)
    sc = _stream_handle(stream_compute)
    sp = _stream_handle(stream_copy) if stream_copy is not None else sc
    _check(lib().compass_decomp_comm(C.byref(problem), _ptr_array(A), _ptr_array(B), _ptr_array(out), p, n, sc, sp),
           "compass_decomp_comm")


def compass_gemm_rs_sequential_noalloc(problem: Problem, A: Sequence, B: Sequence, Out: Sequence, stream=None) -> None:
    """GEMM+ReduceScatter (sequential form) whose scratch is the library's built-in
    device array: for callers that cannot allocate or pass a workspace (all device
    memory already handed out, or no tolerance for cudaMalloc's device-wide sync).
    Refuses problems needing more than NOALLOC_SCRATCH_BYTES."""
    _check(lib().compass_gemm_rs_sequential_noalloc(C.byref(problem), _ptr_array(A), _ptr_array(B), _ptr_array(Out),
                                                    _stream_handle(stream)), "compass_gemm_rs_sequential_noalloc")


def compass_noalloc_read_status(stream=None):
    """(status, detail) the last compass_gemm_rs_sequential_noalloc on the current device left in the
    built-in array; synchronises the stream, allocates nothing."""
    detail = C.c_int(0)
    st = lib().compass_noalloc_read_status(_stream_handle(stream), C.byref(detail))
    return int(st), int(detail.value)


def compass_fused_host_bytes(problem: Problem) -> int:
    n = C.c_size_t(0)
    _check(lib().compass_fused_host(C.byref(problem), None, None, None, None, 0, C.byref(n), None, 0, None),
           "compass_fused_host")
    return int(n.value)


def compass_fused_host(problem: Problem, A_host: Sequence, B_host: Sequence, out_host: Sequence, staging, workspace,
                       stream=None) -> None:
    """A_host/B_host/out_host: CPU tensors (pinned recommended)."""
    p, n = _ws(workspace)
    sp, sn = _ws(staging)
    need = C.c_size_t(0)
    _check(lib().compass_fused_host(C.byref(problem), _ptr_array(A_host), _ptr_array(B_host), _ptr_array(out_host),
                                    sp, sn, C.byref(need), p, n, _stream_handle(stream)), "compass_fused_host")


# ---- small conveniences (no arithmetic) ------------------------------------------

@dataclass
class DeviceWorkload:
    problem: Problem
    A: list
    B: list
    out: list
    workspace: object


def to_device(bits: np.ndarray, device="cuda"):
    """uint16 BF16 bit patterns -> torch.bfloat16 tensor on the device."""
    import torch
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


def to_bits(t) -> np.ndarray:
    """torch.bfloat16 tensor -> uint16 BF16 bit patterns on the host."""
    import torch
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16)


def alloc_workspace(problem: Problem, which: int = WS_FUSED, device="cuda"):
    import torch
    n = compass_workspace_bytes(problem, which)
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    compass_workspace_init(ws)
    return ws
