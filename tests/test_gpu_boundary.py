"""GPU tests of the C-ABI boundary's helpers: decoding one index, launch counters, device checks."""
import ctypes as C

import numpy as np
import pytest
import torch

import mmee_inputs as mi
import oracle
import paper_2604_03446_b200.binding as mm
from test_gpu_parity import Handle, assert_same_record

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [1, 4, 9])
def test_decode_returns_the_mapping_and_its_evaluation(seed):
    """mmee_decode against the oracle's evaluation of the same index: sampled indices of the whole space,
    its first and its last index; an index outside the space is an argument error."""
    cfg = mi.random_tiny_problem(seed)
    obj = cfg["searches"][0]
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    rng = np.random.default_rng(seed)
    picks = [0, p.N - 1] + [int(i) for i in rng.integers(0, p.N, size=40)]
    with Handle(cfg, obj) as h:
        assert mm.mmee_num_candidates(h) == p.N
        for idx in picks:
            got = mm.mmee_decode(h, idx)
            want = oracle.evaluate(p, idx)
            assert_same_record(got, want, "idx %d" % idx)
            assert got.status == mm.OK
        assert mm.library().mmee_decode(h, p.N, C.byref(mm.Result())) == mm.ERR_ARG
        assert mm.library().mmee_decode(h, 0, None) == mm.ERR_ARG


def test_decode_at_full_size():
    cfg = mi.config4()
    obj = cfg["searches"][1]
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    with Handle(cfg, obj) as h:
        for idx in (0, p.N // 3 + 7, p.N - 1):
            assert_same_record(mm.mmee_decode(h, idx), oracle.evaluate(p, idx), "idx %d" % idx)


def test_search_with_host_records_equals_the_device_path():
    cfg = mi.random_tiny_problem(3)
    obj = dict(cfg["searches"][0], topk=5)
    want = oracle.search(oracle.make_problem(cfg["workload"], cfg["arch"], obj))
    with Handle(cfg, obj) as h:
        for _ in range(2):
            best, topk = mm.mmee_search_host(h, True, 5)
            assert [r.idx for r in topk if r.idx != mm.NO_INDEX] == [r.idx for r in want.topk]
            assert best.n_feasible == want.n_feasible and best.n_total == want.n_total
            if want.topk:
                assert_same_record(best, want.topk[0])
        best_only, none = mm.mmee_search_host(h)
        assert none is None and bytes(best_only) == bytes(best)


def test_launch_counters_of_a_search():
    """Create time, launches, persistent CTAs and the number of groups that went to the exact path are reported;
    a search cannot find an optimum without at least one visit of the exact path."""
    cfg = mi.config1()
    obj = cfg["searches"][0]
    best = mm.result_buffer(1)
    with Handle(cfg, obj) as h:
        assert mm.mmee_last_search_stats(h).exact_path_visits == 0
        mm.mmee_search(h, best)
        torch.cuda.synchronize()
        st = mm.mmee_last_search_stats(h)
        assert st.kernels_launched == 1 and st.grid >= 1 and st.block == 256
        assert st.create_ms > 0.0
        assert 1 <= st.exact_path_visits <= st.tasks * 25
        first = st.exact_path_visits
        mm.mmee_search(h, best)
        torch.cuda.synchronize()
        assert mm.mmee_last_search_stats(h).exact_path_visits > 0
        assert first > 0
    assert mm.read_results(best, 1)[0].status == mm.OK


def test_a_handle_is_refused_on_another_device():
    """A handle lives on the device that was current at mmee_create; calls with another device current are
    argument errors and launch nothing."""
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two devices")
    cfg = mi.config1()
    obj = dict(cfg["searches"][0], t_begin=0, t_end=50)
    with torch.cuda.device(0):
        h = mm.mmee_create(cfg["workload"], cfg["arch"], obj)
    try:
        with torch.cuda.device(1):
            best = mm.result_buffer(1, device="cuda:1")
            lib = mm.library()
            assert lib.mmee_search(h, None, C.c_void_p(best.data_ptr()), None) == mm.ERR_ARG
            assert lib.mmee_decode(h, 0, C.byref(mm.Result())) == mm.ERR_ARG
            assert lib.mmee_eval(h, None, 0, 1, C.c_void_p(best.data_ptr())) == mm.ERR_ARG
    finally:
        with torch.cuda.device(0):
            mm.mmee_destroy(h)
