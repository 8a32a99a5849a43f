"""CPU-only checks of the CUDA library's host side: the shared object loads and exports what the
header declares, the planner's query vectors match the paper's printed vector and the oracle's
monomials, and argument errors are reported before any device work."""
import ctypes as C
import os
import re

import pytest

import mmee_inputs as mi
import oracle
import paper_2604_03446_b200.binding as mm
from helpers import candidate_index
from test_oracle_pins import PRIME_BOUNDS, _prime_problem, _read_golden

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "mmee.h")).read()
    declared = set(re.findall(r"^(?:int|uint64_t|const char\*)\s+(mmee_\w+)\s*\(", header, flags=re.M))
    assert declared == set(mm.EXPORTS)
    lib = mm.library()
    for name in declared:
        assert getattr(lib, name) is not None
    assert lib.mmee_strerror(mm.ERR_QUANTUM).decode().startswith("an energy")


def test_result_record_layout():
    assert C.sizeof(mm.Result) == 72 + 8 * 24 + 8 * 3 + 16 + 32 == 336
    assert mm.Result.status.offset == 68 and mm.Result.bs_x.offset == 72


def test_query_vector_of_the_worked_example():
    """Section V-E prints q = [0,1,0,0,1,1,0,0] for BS_A in the setting of Section V-A/B."""
    want = {row[0]: [int(v) for v in row[1:]] for row in _read_golden("worked_example.txt")}
    assert mm.mmee_query_vector(0, 0, 0, 0, 4) == want["BS_A"]
    assert mm.mmee_query_vector(1, 0, 0, 0, 4) == want["DA_A"]
    assert mm.mmee_query_vector(1, 0, 0, 3, 3) == want["DA_D"]


def test_query_vectors_reproduce_the_oracle_monomials():
    """For every order, operand, level (and recompute flag where it matters) the product of the
    bounds the planner's query vector selects equals the oracle's BS_X / DA_X."""
    def product(q):
        v = 1
        for sel, b in zip(q, PRIME_BOUNDS):
            if sel:
                v *= b
        return v

    for fuse, phi in ((mi.FUSE_FUSED, 0), (mi.FUSE_SOFTMAX_IN_OP1, 1), (mi.FUSE_SEPARATE, 2)):
        p = _prime_problem(fuse_mask=fuse)
        I, L = int(p.dim[0]), int(p.dim[2])
        for pi in range(6):
            for x in range(5):
                for beta in range(3, 8):
                    if phi and x == 2 and beta != 3:
                        continue
                    levels = [3, 3, 3, 3, 3]
                    levels[x] = beta
                    # vary C's level as well so that both recompute settings are visited
                    for beta_c in ((3, 5, 7) if (phi == 0 and x != 2) else (levels[2],)):
                        levels[2] = beta_c
                        r = oracle.evaluate(p, candidate_index(p, PRIME_BOUNDS[4:], phi, pi, levels))
                        assert product(mm.mmee_query_vector(0, phi, pi, x, beta)) == r.bs_x[x]
                        if phi == 0:
                            assert mm.mmee_recompute_flag(pi, beta_c) == r.recompute
                            if x != 2:
                                q = mm.mmee_query_vector(1, 0, pi, x, beta, r.recompute)
                                assert product(q) == r.da_x[x]
                        elif x == 2:
                            assert product(mm.mmee_query_vector(1, phi, pi, 2, 3)) + I * L == r.da_x[2]
                        else:
                            assert product(mm.mmee_query_vector(1, phi, pi, x, beta)) == r.da_x[x]


def test_argument_errors_come_before_any_device_call():
    w, a, o = mi.workload(1, 1, 1, 8, 8, 4, 4), mi.arch_tiny(), mi.objective()
    for bad_w in (dict(w, seq_kv=0), dict(w, q_heads=3, kv_heads=2), dict(w, word_bytes=0)):
        with pytest.raises(mm.MmeeError) as e:
            mm.mmee_create(bad_w, a, o)
        assert e.value.code == mm.ERR_ARG
    for bad_o, code in ((dict(o, fuse_mask=0), mm.ERR_ARG), (dict(o, topk=0), mm.ERR_ARG),
                        (dict(o, topk=17), mm.ERR_RANGE), (dict(o, objective=5), mm.ERR_ARG), (dict(o, objective=3, key_cap=-1), mm.ERR_ARG),
                        (dict(o, t_begin=5, t_end=2), mm.ERR_ARG), (dict(o, stationary_mask=0x200), mm.ERR_ARG),
                        (dict(o, rf_tiling=2), mm.ERR_ARG), (dict(o, rf_tiling=1, objective=2), mm.ERR_ARG)):
        with pytest.raises(mm.MmeeError) as e:
            mm.mmee_create(w, a, bad_o)
        assert e.value.code == code
    with pytest.raises(mm.MmeeError) as e:
        mm.mmee_create(w, dict(a, e_gb_pj=6.3), o)
    assert e.value.code == mm.ERR_QUANTUM
    # 2^5 * 3^3 * 5 * 7 * 11 = 332640 has 192 divisors: above the per-dimension maximum
    with pytest.raises(mm.MmeeError) as e:
        mm.mmee_create(dict(w, seq_q=332640), a, o)
    assert e.value.code == mm.ERR_RANGE
    # a problem whose worst-case key cannot be held in 62 bits
    with pytest.raises(mm.MmeeError) as e:
        mm.mmee_create(mi.workload(1, 1, 1, 2 ** 20, 2 ** 20, 4096, 4096), mi.arch_cloud(), o)
    assert e.value.code == mm.ERR_OVERFLOW
    lib = mm.library()
    assert lib.mmee_destroy(None) == mm.ERR_ARG
    assert lib.mmee_search(None, None, None, None) == mm.ERR_ARG
    assert lib.mmee_search_host(None, None, None) == mm.ERR_ARG
    assert lib.mmee_decode(None, 0, None) == mm.ERR_ARG
    assert lib.mmee_filter_flags(None, None, 0, None) == mm.ERR_ARG
    n = C.c_uint32(7)
    assert lib.mmee_pareto_front_bs_da(None, None, None, None, 0, C.byref(n)) == mm.ERR_ARG
    assert lib.mmee_pareto_front_bs_da(None, None, None, None, 0, None) == mm.ERR_ARG
    assert lib.mmee_query_vector(0, 0, 9, 0, 3, 0, (C.c_uint8 * 8)()) == mm.ERR_ARG
    assert lib.mmee_query_vector(1, 0, 0, 2, 3, 0, (C.c_uint8 * 8)()) == mm.ERR_ARG


def test_without_a_gpu_create_fails_loudly():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(mm.MmeeError) as e:
        mm.mmee_create(mi.workload(1, 1, 1, 8, 8, 4, 4), mi.arch_tiny(), mi.objective())
    assert e.value.code == mm.ERR_CUDA


def test_tie_safe_row_pruning_never_drops_a_lowest_index_optimum():
    """The planner's symbolic row pruning (Section VI-B, Eq. 12 with a lower-index dominator): for
    every tiling and objective of small problems, the (key, idx)-smallest feasible mapping over the
    kept rows is the (key, idx)-smallest over all rows."""
    import numpy as np
    full = np.array(mm.mmee_row_pruning_keep(mi.objective()), dtype=bool)
    assert (full.size, int(full.sum()), int(full[:18750].sum())) == (26250, 204, 100)
    assert int(np.array(mm.mmee_row_pruning_keep(mi.config1()["searches"][0])).sum()) == 56
    for seed in (1, 2, 3, 5, 8, 11):
        cfg = mi.random_tiny_problem(seed)
        for objective in (mi.OBJ_ENERGY, mi.OBJ_LATENCY, mi.OBJ_EDP):
            obj = dict(cfg["searches"][0], objective=objective, topk=1)
            keep = np.array(mm.mmee_row_pruning_keep(obj), dtype=bool)
            p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
            assert keep.size == p.R
            n_t = min(p.T, max(1, 1_500_000 // (p.R * 9)))
            keys, feas = oracle.keys_range(p, 0, n_t * p.R * 9)
            keys = np.where(feas.astype(bool), keys, np.iinfo(np.int64).max).reshape(n_t, p.R, 9)
            flat_all = keys.reshape(n_t, -1)
            masked = np.where(keep[None, :, None], keys, np.iinfo(np.int64).max).reshape(n_t, -1)
            # argmin returns the first (lowest-index) minimum
            assert np.array_equal(flat_all.argmin(axis=1), masked.argmin(axis=1))
            assert np.array_equal(flat_all.min(axis=1), masked.min(axis=1))
