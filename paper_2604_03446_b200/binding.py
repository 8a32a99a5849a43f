"""ctypes binding of libmmee.so: the same entry points as include/mmee.h, argument marshalling only.

PyTorch supplies device memory (uint8 CUDA tensors hold the result records) and the stream.
Every step of the search runs in the library's CUDA kernels; if the shared object cannot be
loaded this module raises -- there is no other implementation to fall back to.
"""
from __future__ import annotations

import ctypes as C
import os

from . import build as _build

OBJ_ENERGY, OBJ_LATENCY, OBJ_EDP, OBJ_ENERGY_LCAP, OBJ_LATENCY_ECAP = 0, 1, 2, 3, 4
TILE_POW2, TILE_ALL_DIVISORS = 0, 1
ORD_NORECOMP2, ORD_ALL6 = 0, 1
FUSE_FUSED, FUSE_SOFTMAX_IN_OP1, FUSE_SEPARATE = 1, 2, 4
MAX_TOPK = 16
NO_INDEX = 2 ** 64 - 1
OK, ERR_ARG, ERR_OVERFLOW, ERR_QUANTUM, ERR_NO_FEASIBLE, ERR_CUDA, ERR_TIMEOUT, ERR_RANGE, ERR_CHECK = range(9)

EXPORTS = ("mmee_create", "mmee_search", "mmee_search_host", "mmee_destroy", "mmee_search_static", "mmee_num_candidates", "mmee_num_tilings",
           "mmee_num_rows", "mmee_strerror", "mmee_last_cuda_error", "mmee_eval", "mmee_decode", "mmee_dump_keys", "mmee_filter_flags", "mmee_solve_host", "mmee_pareto_front", "mmee_pareto_front_bs_da", "mmee_search_shapes",
           "mmee_query_vector", "mmee_recompute_flag", "mmee_row_pruning_keep", "mmee_last_search_stats", "mmee_kernel_timing",
           "mmee_alu_peak")


class Workload(C.Structure):
    _fields_ = [(n, C.c_uint32) for n in
                ("batch", "q_heads", "kv_heads", "seq_q", "seq_kv", "d_qk", "d_v", "word_bytes")]


class Arch(C.Structure):
    _fields_ = [("pe_rows", C.c_uint32), ("pe_cols", C.c_uint32), ("n_arrays", C.c_uint32),
                ("gb_bytes", C.c_uint64), ("rf_bytes", C.c_uint64),
                ("dram_words_per_cycle", C.c_uint32),
                ("e_dram_pj", C.c_double), ("e_gb_pj", C.c_double), ("e_rf_pj", C.c_double),
                ("e_mac_pj", C.c_double), ("c_softmax", C.c_double),
                ("energy_quantum_pj", C.c_double)]


class Objective(C.Structure):
    _fields_ = [("objective", C.c_uint32), ("topk", C.c_uint32), ("tiling_set", C.c_uint32),
                ("order_set", C.c_uint32), ("fuse_mask", C.c_uint32), ("row_pruning", C.c_uint32),
                ("t_begin", C.c_uint64), ("t_end", C.c_uint64), ("key_cap", C.c_int64),
                ("stationary_mask", C.c_uint32), ("rf_tiling", C.c_uint32)]


class Result(C.Structure):
    _fields_ = [("idx", C.c_uint64), ("t", C.c_uint64), ("row", C.c_uint32),
                ("bound", C.c_uint32 * 8),
                ("phi", C.c_uint8), ("pi", C.c_uint8), ("beta", C.c_uint8 * 5), ("sm", C.c_uint8 * 2),
                ("recompute", C.c_uint8), ("feasible", C.c_uint8), ("reserved", C.c_uint8 * 5),
                ("status", C.c_int32),
                ("bs_x", C.c_int64 * 5), ("bs_op1", C.c_int64), ("bs_op2", C.c_int64), ("bs", C.c_int64),
                ("da_x", C.c_int64 * 5), ("da_sm", C.c_int64),
                ("br", C.c_int64), ("cyc1", C.c_int64), ("cyc2", C.c_int64),
                ("n", C.c_int64 * 5), ("e_key", C.c_int64), ("l_key", C.c_int64),
                ("edp_key", C.c_double), ("energy_pj", C.c_double), ("latency_cycles", C.c_double),
                ("n_total", C.c_uint64), ("n_feasible", C.c_uint64),
                ("rf_block", C.c_uint32 * 6), ("reserved2", C.c_uint32 * 2)]


class LaunchStats(C.Structure):
    _fields_ = [("kernels_launched", C.c_uint32), ("grid", C.c_uint32), ("block", C.c_uint32),
                ("smem_bytes", C.c_uint32), ("tasks", C.c_uint64),
                ("search_ms", C.c_float), ("finalize_ms", C.c_float),
                ("rows_per_tiling", C.c_uint32), ("rows_evaluated_per_tiling", C.c_uint32),
                ("exact_path_visits", C.c_uint64), ("create_ms", C.c_float), ("reserved", C.c_uint32),
                ("rows_tested", C.c_uint64)]


RESULT_BYTES = C.sizeof(Result)


class MmeeError(RuntimeError):
    def __init__(self, code: int, where: str):
        msg = library().mmee_strerror(code).decode() if _lib is not None else "status %d" % code
        if code == ERR_CUDA and _lib is not None:
            msg += ": " + library().mmee_last_cuda_error().decode()
        super().__init__("%s: %s (status %d)" % (where, msg, code))
        self.code = code


_lib = None


def library():
    """Load libmmee.so (building it first when its sources are newer and nvcc is present)."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    try:
        if _build.is_stale():
            _build.build_library()
    except Exception:
        if not os.path.exists(path):
            raise
    L = C.CDLL(path)
    H = C.c_void_p
    L.mmee_create.argtypes = [C.POINTER(Workload), C.POINTER(Arch), C.POINTER(Objective), C.POINTER(H)]
    L.mmee_search.argtypes = [H, C.c_void_p, C.c_void_p, C.c_void_p]
    L.mmee_search_host.argtypes = [H, C.POINTER(Result), C.POINTER(Result)]
    L.mmee_destroy.argtypes = [H]
    L.mmee_search_static.argtypes = [C.POINTER(Workload), C.POINTER(Arch), C.POINTER(Objective),
                                     C.c_void_p, C.c_void_p, C.c_void_p]
    for name in ("mmee_num_candidates", "mmee_num_tilings", "mmee_num_rows"):
        getattr(L, name).argtypes = [H]
        getattr(L, name).restype = C.c_uint64
    L.mmee_strerror.argtypes = [C.c_int]
    L.mmee_strerror.restype = C.c_char_p
    L.mmee_last_cuda_error.argtypes = []
    L.mmee_last_cuda_error.restype = C.c_char_p
    L.mmee_eval.argtypes = [H, C.c_void_p, C.c_uint64, C.c_uint64, C.c_void_p]
    L.mmee_decode.argtypes = [H, C.c_uint64, C.POINTER(Result)]
    L.mmee_dump_keys.argtypes = [H, C.c_void_p, C.c_void_p]
    L.mmee_filter_flags.argtypes = [H, C.c_void_p, C.c_int64, C.c_void_p]
    L.mmee_solve_host.argtypes = [C.POINTER(Workload), C.POINTER(Arch), C.POINTER(Objective),
                                  C.POINTER(Result), C.POINTER(Result),
                                  C.POINTER(C.c_uint64), C.POINTER(C.c_uint64)]
    L.mmee_pareto_front.argtypes = [C.POINTER(Workload), C.POINTER(Arch), C.POINTER(Objective),
                                    C.POINTER(Result), C.c_uint32, C.POINTER(C.c_uint32)]
    L.mmee_pareto_front_bs_da.argtypes = L.mmee_pareto_front.argtypes
    L.mmee_search_shapes.argtypes = [C.POINTER(Workload), C.POINTER(Arch), C.POINTER(Objective),
                                     C.POINTER(C.c_uint32), C.c_uint32, C.POINTER(Result), C.POINTER(C.c_uint32)]
    L.mmee_query_vector.argtypes = [C.c_uint32] * 6 + [C.POINTER(C.c_uint8)]
    L.mmee_recompute_flag.argtypes = [C.c_uint32, C.c_uint32, C.POINTER(C.c_uint32)]
    L.mmee_row_pruning_keep.argtypes = [C.POINTER(Objective), C.POINTER(C.c_uint8), C.c_uint32,
                                        C.POINTER(C.c_uint32)]
    L.mmee_last_search_stats.argtypes = [H, C.POINTER(LaunchStats)]
    L.mmee_kernel_timing.argtypes = [H, C.c_int]
    L.mmee_alu_peak.argtypes = [C.POINTER(C.c_double)]
    _lib = L
    return L


def _fill(struct, values: dict):
    for k, v in values.items():
        setattr(struct, k, v)
    return struct


def _check(code: int, where: str):
    if code != OK:
        raise MmeeError(code, where)


def _stream_ptr(stream):
    import torch
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def mmee_create(workload: dict, arch: dict, objective: dict) -> C.c_void_p:
    h = C.c_void_p()
    _check(library().mmee_create(_fill(Workload(), workload), _fill(Arch(), arch),
                                 _fill(Objective(), objective), C.byref(h)), "mmee_create")
    return h


def mmee_destroy(handle) -> None:
    _check(library().mmee_destroy(handle), "mmee_destroy")


def mmee_num_candidates(handle) -> int:
    return library().mmee_num_candidates(handle)


def mmee_num_tilings(handle) -> int:
    return library().mmee_num_tilings(handle)


def mmee_num_rows(handle) -> int:
    return library().mmee_num_rows(handle)


def result_buffer(n: int, device="cuda"):
    """Uninitialised device buffer for n result records."""
    import torch
    return torch.empty(n * RESULT_BYTES, dtype=torch.uint8, device=device)


def mmee_search(handle, out_best, out_topk=None, stream=None) -> None:
    """Asynchronous: out_best / out_topk are uint8 CUDA tensors from result_buffer()."""
    _check(library().mmee_search(handle, _stream_ptr(stream), C.c_void_p(out_best.data_ptr()),
                                 C.c_void_p(out_topk.data_ptr()) if out_topk is not None else None),
           "mmee_search")


def mmee_search_host(handle, want_topk: bool = False, topk: int = 0):
    """Search through a planned handle with the records copied to host structs: (best, list of top-k or None)."""
    best = Result()
    arr = (Result * topk)() if want_topk else None
    _check(library().mmee_search_host(handle, C.byref(best), arr), "mmee_search_host")
    return best, (list(arr) if want_topk else None)


def mmee_search_static(workload: dict, arch: dict, objective: dict, out_best, out_topk=None, stream=None) -> None:
    """Search without device allocation: plans on the host, uses the library's fixed scratch.
    Asynchronous; out_best / out_topk are caller-owned uint8 CUDA tensors (result_buffer())."""
    _check(library().mmee_search_static(_fill(Workload(), workload), _fill(Arch(), arch),
                                        _fill(Objective(), objective), _stream_ptr(stream),
                                        C.c_void_p(out_best.data_ptr()),
                                        C.c_void_p(out_topk.data_ptr()) if out_topk is not None else None),
           "mmee_search_static")


def mmee_eval(handle, idx_begin: int, count: int, out, stream=None) -> None:
    _check(library().mmee_eval(handle, _stream_ptr(stream), idx_begin, count, C.c_void_p(out.data_ptr())),
           "mmee_eval")


def mmee_decode(handle, idx: int) -> Result:
    """The mapping behind one candidate index with its full evaluation, as a host record (synchronous)."""
    r = Result()
    _check(library().mmee_decode(handle, idx, C.byref(r)), "mmee_decode")
    return r


def mmee_dump_keys(handle, out_keys, stream=None) -> None:
    """out_keys: int64 CUDA tensor with one entry per candidate of the handle's tiling range."""
    _check(library().mmee_dump_keys(handle, _stream_ptr(stream), C.c_void_p(out_keys.data_ptr())),
           "mmee_dump_keys")


def mmee_filter_flags(handle, threshold_key: int, out_flags, stream=None) -> None:
    """out_flags: uint8 CUDA tensor with 25 entries per task of the handle's tiling range (1 = group flagged)."""
    _check(library().mmee_filter_flags(handle, _stream_ptr(stream), threshold_key, C.c_void_p(out_flags.data_ptr())),
           "mmee_filter_flags")


def mmee_solve_host(workload: dict, arch: dict, objective: dict):
    """(best, topk list, h2d bytes, d2h bytes) with host buffers."""
    k = objective["topk"]
    best, topk = Result(), (Result * k)()
    h2d, d2h = C.c_uint64(), C.c_uint64()
    _check(library().mmee_solve_host(_fill(Workload(), workload), _fill(Arch(), arch),
                                     _fill(Objective(), objective), C.byref(best), topk,
                                     C.byref(h2d), C.byref(d2h)), "mmee_solve_host")
    return best, list(topk), h2d.value, d2h.value


def mmee_pareto_front(workload: dict, arch: dict, objective: dict, capacity: int = 256):
    """Energy-latency Pareto front of the whole mapping space: list of Result, by increasing energy."""
    pts = (Result * capacity)()
    n = C.c_uint32()
    _check(library().mmee_pareto_front(_fill(Workload(), workload), _fill(Arch(), arch),
                                       _fill(Objective(), objective), pts, capacity, C.byref(n)),
           "mmee_pareto_front")
    return list(pts[:n.value])


def mmee_pareto_front_bs_da(workload: dict, arch: dict, objective: dict, capacity: int = 1024):
    """Buffer-size / DRAM-traffic Pareto front of the whole mapping space: list of Result, by decreasing buffer size."""
    pts = (Result * capacity)()
    n = C.c_uint32()
    _check(library().mmee_pareto_front_bs_da(_fill(Workload(), workload), _fill(Arch(), arch),
                                             _fill(Objective(), objective), pts, capacity, C.byref(n)),
           "mmee_pareto_front_bs_da")
    return list(pts[:n.value])


def mmee_search_shapes(workload: dict, arch: dict, objective: dict, shapes):
    """One search per logical array shape (rows, cols): (list of Result per shape, index of the best shape or None)."""
    n = len(shapes)
    flat = (C.c_uint32 * (2 * n))(*[v for rc in shapes for v in rc])
    out = (Result * n)()
    best = C.c_uint32()
    _check(library().mmee_search_shapes(_fill(Workload(), workload), _fill(Arch(), arch), _fill(Objective(), objective),
                                        flat, n, out, C.byref(best)), "mmee_search_shapes")
    return list(out), (None if best.value == 2 ** 32 - 1 else best.value)


def mmee_query_vector(metric: int, phi: int, pi: int, operand: int, beta: int, recompute: int = 0):
    q = (C.c_uint8 * 8)()
    _check(library().mmee_query_vector(metric, phi, pi, operand, beta, recompute, q), "mmee_query_vector")
    return list(q)


def mmee_row_pruning_keep(objective: dict):
    """List of 0/1 per row of a tiling: the rows evaluated under objective.row_pruning = 1."""
    rows = C.c_uint32()
    buf = (C.c_uint8 * 26250)()
    _check(library().mmee_row_pruning_keep(_fill(Objective(), objective), buf, 26250, C.byref(rows)),
           "mmee_row_pruning_keep")
    return list(buf[:rows.value])


def mmee_recompute_flag(pi: int, beta_c: int) -> int:
    f = C.c_uint32()
    _check(library().mmee_recompute_flag(pi, beta_c, C.byref(f)), "mmee_recompute_flag")
    return f.value


def mmee_last_search_stats(handle) -> LaunchStats:
    s = LaunchStats()
    _check(library().mmee_last_search_stats(handle, C.byref(s)), "mmee_last_search_stats")
    return s


def mmee_kernel_timing(handle, enable: bool) -> None:
    _check(library().mmee_kernel_timing(handle, int(enable)), "mmee_kernel_timing")


def mmee_alu_peak():
    out = (C.c_double * 4)()
    _check(library().mmee_alu_peak(out), "mmee_alu_peak")
    return list(out)


def read_results(buf, n: int):
    """Copy n records from a device buffer to host Result structs (synchronises)."""
    raw = bytes(buf.cpu().numpy().tobytes())
    return [Result.from_buffer_copy(raw[i * RESULT_BYTES:(i + 1) * RESULT_BYTES]) for i in range(n)]
