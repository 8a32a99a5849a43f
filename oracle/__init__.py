"""CPU oracle for the MMEE search path -- TEST INFRASTRUCTURE ONLY.

Thin ctypes view of ``mmee_oracle.c`` (plain C, one candidate at a time, written from the
paper's model definitions).  Nothing in the CUDA library or its Python binding imports this
package; only tests, the smoke entry and the benchmark's CPU-baseline leg do.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mmee_oracle.c")
_HDR = os.path.join(_HERE, "mmee_oracle.h")
_LIB = os.path.join(_HERE, "libmmee_oracle.so")

OBJ_ENERGY, OBJ_LATENCY, OBJ_EDP = 0, 1, 2
TILE_POW2, TILE_ALL_DIVISORS = 0, 1
ORD_NORECOMP2, ORD_ALL6 = 0, 1
OK, ERR_ARG, ERR_OVERFLOW, ERR_QUANTUM = 0, 1, 2, 3
MAX_DIVISORS = 256
NO_INDEX = 2**64 - 1


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
                ("order_set", C.c_uint32), ("fuse_mask", C.c_uint32), ("stationary_mask", C.c_uint32),
                ("t_begin", C.c_uint64), ("t_end", C.c_uint64), ("rf_tiling", C.c_uint32), ("pad", C.c_uint32)]


class Problem(C.Structure):
    _fields_ = [("dim", C.c_uint64 * 4), ("instances", C.c_uint32), ("ndiv", C.c_uint32 * 4),
                ("divs", (C.c_uint32 * MAX_DIVISORS) * 4), ("T", C.c_uint64),
                ("n_orders", C.c_uint32), ("order_id", C.c_uint32 * 6),
                ("n_phi", C.c_uint32), ("phi_id", C.c_uint32 * 3),
                ("R", C.c_uint64), ("N", C.c_uint64), ("t_begin", C.c_uint64), ("t_end", C.c_uint64),
                ("cq_dram", C.c_int64), ("cq_gb", C.c_int64), ("cq_rf", C.c_int64),
                ("cq_mac", C.c_int64), ("cq_sfu", C.c_int64), ("quantum_pj", C.c_double),
                ("has_rf", C.c_int), ("cap_words", C.c_uint64),
                ("pe_rows", C.c_uint32), ("pe_cols", C.c_uint32), ("n_arrays", C.c_uint32),
                ("bw", C.c_uint32), ("objective", C.c_uint32), ("topk", C.c_uint32),
                ("stationary_mask", C.c_uint32), ("rf_tiling", C.c_uint32), ("rf_words", C.c_uint64)]


class Record(C.Structure):
    _fields_ = [("idx", C.c_uint64), ("t", C.c_uint64), ("row", C.c_uint32),
                ("bound", C.c_uint32 * 8), ("phi", C.c_uint32), ("pi", C.c_uint32),
                ("beta", C.c_uint32 * 5), ("sm", C.c_uint32 * 2),
                ("recompute", C.c_uint32), ("feasible", C.c_uint32),
                ("bs_x", C.c_int64 * 5), ("bs_op1", C.c_int64), ("bs_op2", C.c_int64),
                ("bs", C.c_int64), ("da_x", C.c_int64 * 5), ("da_sm", C.c_int64),
                ("da1", C.c_int64), ("da2", C.c_int64),
                ("br", C.c_int64), ("cyc1", C.c_int64), ("cyc2", C.c_int64),
                ("n", C.c_int64 * 5), ("e_key", C.c_int64), ("l_key", C.c_int64),
                ("edp_key", C.c_double), ("energy_pj", C.c_double), ("latency_cycles", C.c_double),
                ("rf_block", C.c_uint32 * 6)]


class SimOut(C.Structure):
    _fields_ = [("loads", C.c_int64 * 5), ("c_productions", C.c_int64),
                ("op1_stages", C.c_int64), ("op2_stages", C.c_int64),
                ("peak_op1", C.c_int64), ("peak_op2", C.c_int64), ("peak", C.c_int64),
                ("n_trace", C.c_int32), ("trace", C.c_int64 * 64), ("trace_kind", C.c_int32 * 64)]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its sources."""
    stale = force or not os.path.exists(_LIB) or \
        os.path.getmtime(_LIB) < max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if stale:
        tmp = _LIB + ".tmp%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared",
                               "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        L.mo_problem_init.argtypes = [C.POINTER(Workload), C.POINTER(Arch), C.POINTER(Objective),
                                      C.POINTER(Problem)]
        L.mo_eval.argtypes = [C.POINTER(Problem), C.c_uint64, C.POINTER(Record)]
        L.mo_eval_range.argtypes = [C.POINTER(Problem), C.c_uint64, C.c_uint64, C.POINTER(Record)]
        L.mo_keys_range.argtypes = [C.POINTER(Problem), C.c_uint64, C.c_uint64,
                                    C.POINTER(C.c_int64), C.POINTER(C.c_uint8)]
        L.mo_search.argtypes = [C.POINTER(Problem), C.POINTER(Record), C.POINTER(C.c_uint64),
                                C.POINTER(C.c_uint64), C.POINTER(C.c_uint32), C.c_int]
        L.mo_simulate.argtypes = [C.POINTER(C.c_uint32), C.c_uint32, C.POINTER(C.c_uint32),
                                  C.POINTER(SimOut)]
        L.mo_threads_used.restype = C.c_int
        _lib = L
    return _lib


class OracleError(RuntimeError):
    def __init__(self, code: int):
        super().__init__("oracle error %d" % code)
        self.code = code


def _fill(struct, values: dict):
    names = {f[0] for f in struct._fields_}
    for k, v in values.items():
        if k in names:            # (the three input dicts also serve the CUDA binding, whose structs have more fields)
            setattr(struct, k, v)
    return struct


def make_problem(workload: dict, arch: dict, objective: dict) -> Problem:
    """Build the oracle's problem from three plain dicts (field names of the paper's inputs)."""
    p = Problem()
    rc = lib().mo_problem_init(_fill(Workload(), workload), _fill(Arch(), arch),
                               _fill(Objective(), objective), p)
    if rc:
        raise OracleError(rc)
    return p


def evaluate(p: Problem, idx: int) -> Record:
    r = Record()
    rc = lib().mo_eval(p, idx, r)
    if rc:
        raise OracleError(rc)
    return r


def evaluate_range(p: Problem, begin: int, count: int):
    arr = (Record * count)()
    rc = lib().mo_eval_range(p, begin, count, arr)
    if rc:
        raise OracleError(rc)
    return arr


def keys_range(p: Problem, begin: int, count: int):
    """(keys int64[count], feasible uint8[count]) as numpy arrays."""
    import numpy as np
    keys = np.empty(count, dtype=np.int64)
    feas = np.empty(count, dtype=np.uint8)
    rc = lib().mo_keys_range(p, begin, count, keys.ctypes.data_as(C.POINTER(C.c_int64)),
                             feas.ctypes.data_as(C.POINTER(C.c_uint8)))
    if rc:
        raise OracleError(rc)
    return keys, feas


@dataclass
class SearchResult:
    topk: list            # list of Record, best first (only the found ones)
    n_total: int
    n_feasible: int


def search(p: Problem, threads: int = 0) -> SearchResult:
    arr = (Record * p.topk)()
    nt, nf, nfound = C.c_uint64(), C.c_uint64(), C.c_uint32()
    rc = lib().mo_search(p, arr, nt, nf, nfound, threads)
    if rc:
        raise OracleError(rc)
    return SearchResult([arr[i] for i in range(nfound.value)], nt.value, nf.value)


def simulate(bound, pi: int, beta) -> SimOut:
    out = SimOut()
    rc = lib().mo_simulate((C.c_uint32 * 8)(*bound), pi, (C.c_uint32 * 5)(*beta), out)
    if rc:
        raise OracleError(rc)
    return out


class RowSymbols(C.Structure):
    _fields_ = [("bs_q", C.c_uint8 * 5), ("da_q", C.c_uint8 * 5), ("tau", C.c_uint8 * 5),
                ("recompute", C.c_uint8)]


def row_symbolic(pi: int, beta) -> RowSymbols:
    out = RowSymbols()
    L = lib()
    L.mo_row_symbolic.argtypes = [C.c_uint32, C.POINTER(C.c_uint32), C.POINTER(RowSymbols)]
    rc = L.mo_row_symbolic(pi, (C.c_uint32 * 5)(*beta), out)
    if rc:
        raise OracleError(rc)
    return out


def symbolic_prune():
    """(keep uint8[18750], kept per recompute group, rows per recompute group) -- Eq. (12) of Section VI-B."""
    import numpy as np
    keep = np.zeros(18750, dtype=np.uint8)
    kept, total = (C.c_uint32 * 2)(), (C.c_uint32 * 2)()
    L = lib()
    L.mo_symbolic_prune.argtypes = [C.POINTER(C.c_uint8), C.POINTER(C.c_uint32), C.POINTER(C.c_uint32)]
    rc = L.mo_symbolic_prune(keep.ctypes.data_as(C.POINTER(C.c_uint8)), kept, total)
    if rc:
        raise OracleError(rc)
    return keep, list(kept), list(total)


class SimUnfusedOut(C.Structure):
    _fields_ = [("loads", C.c_int64 * 5), ("c_stores", C.c_int64), ("softmax_words", C.c_int64),
                ("op1_stages", C.c_int64), ("op2_stages", C.c_int64),
                ("peak_op1", C.c_int64), ("peak_op2", C.c_int64)]


def simulate_unfused(bound, pi: int, beta, phi: int) -> SimUnfusedOut:
    """Tile-granular execution of the producer nest, the softmax pass and the consumer nest of an unfused mapping."""
    out = SimUnfusedOut()
    L = lib()
    L.mo_simulate_unfused.argtypes = [C.POINTER(C.c_uint32), C.c_uint32, C.POINTER(C.c_uint32), C.c_uint32,
                                      C.POINTER(SimUnfusedOut)]
    rc = L.mo_simulate_unfused((C.c_uint32 * 8)(*bound), pi, (C.c_uint32 * 5)(*beta), phi, out)
    if rc:
        raise OracleError(rc)
    return out


class ArrayCounts(C.Structure):
    _fields_ = [("cycles", C.c_int64), ("words", C.c_int64), ("macs", C.c_int64), ("rf", C.c_int64)]


def array_tile(sm: int, m: int, r: int, n: int, rows: int, cols: int, resume: bool = False) -> ArrayCounts:
    """Element-level execution of one (m x r) * (r x n) tile on a rows x cols PE array."""
    out = ArrayCounts()
    L = lib()
    L.mo_array_tile.argtypes = [C.c_uint32] * 6 + [C.c_int, C.POINTER(ArrayCounts)]
    rc = L.mo_array_tile(sm, m, r, n, rows, cols, int(resume), out)
    if rc:
        raise OracleError(rc)
    return out


def array_chain(bound, productions: int, sm1: int, sm2: int, rows: int, cols: int):
    """Element-level execution of every tile invocation of both operators: (Op1 counts, Op2 counts)."""
    out = (ArrayCounts * 2)()
    L = lib()
    L.mo_array_chain.argtypes = [C.POINTER(C.c_uint32)] + [C.c_uint32] * 5 + [C.POINTER(ArrayCounts)]
    rc = L.mo_array_chain((C.c_uint32 * 8)(*bound), productions, sm1, sm2, rows, cols, out)
    if rc:
        raise OracleError(rc)
    return out[0], out[1]


def array_tile_blocked(sm: int, m: int, r: int, n: int, rows: int, cols: int, a: int, b: int,
                       resume: bool = False) -> ArrayCounts:
    """Element-level execution of one tile whose stationary operand is processed in register-file blocks of a x b."""
    out = ArrayCounts()
    L = lib()
    L.mo_array_tile_blocked.argtypes = [C.c_uint32] * 8 + [C.c_int, C.POINTER(ArrayCounts)]
    rc = L.mo_array_tile_blocked(sm, m, r, n, rows, cols, a, b, int(resume), out)
    if rc:
        raise OracleError(rc)
    return out


def rf_block(objective: int, sm: int, m: int, r: int, n: int, rows: int, cols: int, rf_words: int):
    """The register-file block the model picks for one tile: ((m, r, n) block, words, cycles)."""
    blk = (C.c_uint32 * 3)()
    w, c = C.c_int64(), C.c_int64()
    L = lib()
    L.mo_rf_block.argtypes = [C.c_uint32] * 7 + [C.c_uint64, C.POINTER(C.c_uint32), C.POINTER(C.c_int64),
                                                 C.POINTER(C.c_int64)]
    rc = L.mo_rf_block(objective, sm, m, r, n, rows, cols, rf_words, blk, C.byref(w), C.byref(c))
    if rc:
        raise OracleError(rc)
    return tuple(blk), w.value, c.value


def threads_used() -> int:
    return lib().mo_threads_used()
