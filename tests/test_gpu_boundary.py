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


def _bs_da_of_every_candidate(cfg, obj, limit):
    """(buffer words, DRAM words, idx) of every candidate of the range-limited problem, from the oracle's records."""
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    if p.N > limit:
        obj = dict(obj, t_begin=0, t_end=max(1, limit // (p.R * 9)))
        p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    begin, count = p.t_begin * p.R * 9, (p.t_end - p.t_begin) * p.R * 9
    recs = oracle.evaluate_range(p, begin, count)
    raw = np.frombuffer(recs, dtype=np.uint8).reshape(count, C.sizeof(oracle.Record))
    field = lambda off: raw[:, off:off + 8].copy().view(np.int64).ravel()
    bs = field(oracle.Record.bs.offset)
    da = field(oracle.Record.n.offset)
    return obj, p, bs, da, np.arange(begin, begin + count, dtype=np.int64)


@pytest.mark.parametrize("seed", [2, 3, 6, 8, 11])
def test_buffer_size_dram_traffic_pareto_front(seed):
    """The buffer-size / DRAM-traffic front (Section VI-A, Section VII-C) by device searches under a shrinking buffer,
    against a brute-force front over the oracle's (BS, N_DRAM) pair of every candidate: by increasing traffic,
    each point the least buffer that reaches that traffic, with the lowest index that attains the pair."""
    cfg = mi.random_tiny_problem(seed)
    obj, p, bs, da, idx = _bs_da_of_every_candidate(cfg, dict(cfg["searches"][0], objective=mi.OBJ_ENERGY, topk=1), 250_000)
    fits = bs <= p.cap_words
    want, best_bs = [], None
    for d in np.unique(da[fits]):
        sel = fits & (da == d)
        b = int(bs[sel].min())
        if best_bs is None or b < best_bs:
            want.append((b, int(d), int(idx[sel & (bs == b)].min())))
            best_bs = b
    got = mm.mmee_pareto_front_bs_da(cfg["workload"], cfg["arch"], obj)
    assert [(r.bs, r.n[0], r.idx) for r in got] == want
    assert len(want) >= 2
    for r in got:
        assert r.e_key == r.n[0]                # the search's key was the DRAM word count


def test_buffer_size_dram_traffic_front_of_the_ffn_task():
    """On the fused feed-forward GEMMs of the paper's buffer-size study the front is a staircase: strictly less
    buffer and strictly more traffic from point to point, no point above the buffer, the last one at the
    smallest buffer any mapping needs; a plain search at a point's buffer size finds that point's traffic."""
    cfg = [c for c in mi.ffn_dram_sweep_configs() if c["name"] == "ffn_gpt3_dram_1024KB"][0]
    obj = dict(cfg["searches"][0], t_begin=0, t_end=4000)
    got = mm.mmee_pareto_front_bs_da(cfg["workload"], cfg["arch"], obj)
    cap = cfg["arch"]["gb_bytes"] // cfg["workload"]["word_bytes"]
    assert len(got) >= 3 and got[0].bs <= cap
    for a, b in zip(got, got[1:]):
        assert b.bs < a.bs and b.n[0] > a.n[0]
    mid = got[len(got) // 2]
    arch = dict(cfg["arch"], gb_bytes=mid.bs * cfg["workload"]["word_bytes"])
    best = mm.mmee_solve_host(cfg["workload"], arch, obj)[0]
    assert (best.n[0], best.bs, best.idx) == (mid.n[0], mid.bs, mid.idx)
    below = dict(cfg["arch"], gb_bytes=(got[-1].bs - 1) * cfg["workload"]["word_bytes"])
    assert mm.mmee_solve_host(cfg["workload"], below, obj)[0].idx == mm.NO_INDEX


def _group_minima(cfg, obj):
    """Least key of the feasible mappings of every group of 45 consecutive candidates (INT64_MAX: none), from the
    oracle's keys."""
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    begin, count = p.t_begin * p.R * 9, (p.t_end - p.t_begin) * p.R * 9
    keys, feas = oracle.keys_range(p, begin, count)
    masked = np.where(feas.astype(bool), keys, np.iinfo(np.int64).max)
    return masked.reshape(-1, 45).min(axis=1), keys[feas.astype(bool)]


def _filter_flags(cfg, obj, thr, n_groups):
    flags = torch.empty(n_groups, dtype=torch.uint8, device="cuda")
    with Handle(cfg, obj) as h:
        mm.mmee_filter_flags(h, int(thr), flags)
        torch.cuda.synchronize()
    return flags.cpu().numpy().astype(bool)


@pytest.mark.parametrize("objective", [mi.OBJ_ENERGY, mi.OBJ_LATENCY, mi.OBJ_EDP])
@pytest.mark.parametrize("seed", [1, 2, 5, 7, 10, 12])
def test_the_filter_flags_every_group_that_holds_a_passing_mapping(seed, objective):
    """The search kernel's filter against fixed thresholds (the 1st, 50th and 99th percentile of the oracle's feasible
    keys, just above the optimum, the optimum itself and the largest key): every group of five rows that holds a
    feasible mapping with a key below the threshold is flagged.  In these small problems the energy and latency
    filters work in units of one quantum / one word, where they are exact: nothing else is flagged either; the
    energy-delay filter also flags groups whose least key equals the threshold or lies within its rounding margin."""
    cfg = mi.random_tiny_problem(seed)
    obj = shrink_to(cfg, dict(cfg["searches"][0], objective=objective, topk=1), 1_200_000)
    gmin, fkeys = _group_minima(cfg, obj)
    if fkeys.size == 0:
        pytest.skip("nothing fits")
    ranked = np.sort(fkeys)
    thresholds = [ranked[(ranked.size - 1) * q // 100] for q in (1, 50, 99)] + [ranked[0] + 1, ranked[0], ranked[-1] + 1]
    for thr in thresholds:
        flags = _filter_flags(cfg, obj, thr, gmin.size)
        must = gmin < int(thr)
        assert not (must & ~flags).any(), "a group with a passing mapping was not flagged (threshold %d)" % thr
        extra = flags & ~must
        if objective == mi.OBJ_EDP:
            # (keys are bit patterns of positive doubles; the filter compares products rounded in floating point
            # with "<=" against the threshold widened by 1e-14: a group is flagged beyond need only if its least key
            # is within that margin of the threshold)
            as_double = lambda a: np.asarray(a, dtype=np.int64).view(np.float64)
            assert (as_double(gmin[extra]) <= as_double([int(thr)])[0] * (1.0 + 1e-13)).all()
        else:
            assert not extra.any()


@pytest.mark.parametrize("log2_quantum", [-12, -24])
@pytest.mark.parametrize("seed", [3, 4, 8])
def test_the_filter_in_coarse_units_never_misses(seed, log2_quantum):
    """The same with a tiny energy quantum: keys are then large, the 32-bit filter works in units of many quanta with
    every term rounded down (and the largest ones capped), so it may flag more groups than pass, never fewer."""
    cfg = mi.random_tiny_problem(seed)
    arch = dict(cfg["arch"], energy_quantum_pj=cfg["arch"]["energy_quantum_pj"] * 2.0 ** log2_quantum)
    cfg = dict(cfg, arch=arch)
    obj = shrink_to(cfg, dict(cfg["searches"][0], objective=mi.OBJ_ENERGY, topk=1), 1_200_000)
    gmin, fkeys = _group_minima(cfg, obj)
    if fkeys.size == 0:
        pytest.skip("nothing fits")
    ranked = np.sort(fkeys)
    for q in (1, 50, 99):
        thr = ranked[(ranked.size - 1) * q // 100]
        flags = _filter_flags(cfg, obj, thr, gmin.size)
        must = gmin < int(thr)
        assert not (must & ~flags).any()
        assert (flags & ~must).sum() <= max(16, gmin.size // 4)


def shrink_to(cfg, obj, limit):
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    if p.N <= limit:
        return dict(obj)
    return dict(obj, t_begin=0, t_end=max(1, limit // (p.R * 9)))


# ---- register-file-level tiling ------------------------------------------------------------------------------------

def _with_register_file_tiling(cfg, objective, rf_words, topk=1):
    arch = dict(cfg["arch"], rf_bytes=rf_words * cfg["workload"]["word_bytes"])
    if arch["e_rf_pj"] == 0:
        arch["e_rf_pj"] = arch["energy_quantum_pj"]
    obj = dict(cfg["searches"][0], objective=objective, topk=topk, rf_tiling=1, row_pruning=0)
    return dict(cfg, arch=arch), obj


@pytest.mark.parametrize("objective", [mi.OBJ_ENERGY, mi.OBJ_LATENCY])
@pytest.mark.parametrize("seed,rf_words", [(1, 6), (2, 7), (4, 8), (6, 16), (9, 64)])
def test_register_file_tiling_keys_records_and_search(seed, rf_words, objective):
    """The third tiling level on small problems: every candidate's key, sampled full records (with the register-file
    block of each operator) and the top-5 of the search equal the oracle's, from a register file that holds a single
    stationary element per PE to one that holds whole tiles."""
    cfg, obj = _with_register_file_tiling(mi.random_tiny_problem(seed), objective, rf_words, topk=5)
    obj = shrink_to(cfg, obj, 600_000)
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    begin, count = p.t_begin * p.R * 9, (p.t_end - p.t_begin) * p.R * 9
    want_keys, want_feas = oracle.keys_range(p, begin, count)
    want_keys = np.where(want_feas.astype(bool), want_keys, np.iinfo(np.int64).max)
    keys = torch.empty(count, dtype=torch.int64, device="cuda")
    with Handle(cfg, obj) as h:
        mm.mmee_dump_keys(h, keys)
        torch.cuda.synchronize()
        rng = np.random.default_rng(seed)
        for idx in [begin, begin + count - 1] + [int(i) for i in rng.integers(begin, begin + count, size=60)]:
            assert_same_record(mm.mmee_decode(h, idx), oracle.evaluate(p, idx), "idx %d" % idx)
        best, topk = mm.mmee_search_host(h, True, 5)
    assert np.array_equal(keys.cpu().numpy(), want_keys)
    want = oracle.search(p)
    assert [r.idx for r in topk if r.idx != mm.NO_INDEX] == [r.idx for r in want.topk]
    assert best.n_feasible == want.n_feasible
    for g, o in zip(topk, want.topk):
        assert_same_record(g, o)
        assert any(g.rf_block)


def test_register_file_tiling_at_full_size_sampled():
    """BERT-base on the edge accelerator with the third tiling level: sampled candidates against the oracle, and the
    search's optimum is a mapping whose record the oracle reproduces and whose key no sampled candidate beats; a
    larger register file never makes the optimum worse."""
    cfg = mi.config2()
    rng = np.random.default_rng(17)
    best_keys = []
    for rf_words in (8, 512):
        cfgr, obj = _with_register_file_tiling(cfg, mi.OBJ_ENERGY, rf_words)
        p = oracle.make_problem(cfgr["workload"], cfgr["arch"], obj)
        with Handle(cfgr, obj) as h:
            best, _ = mm.mmee_search_host(h)
            assert best.status == mm.OK
            assert_same_record(best, oracle.evaluate(p, best.idx), "optimum")
            for idx in rng.integers(0, p.N, size=300):
                o = oracle.evaluate(p, int(idx))
                assert_same_record(mm.mmee_decode(h, int(idx)), o, "idx %d" % idx)
                assert not o.feasible or (o.e_key, o.idx) >= (best.e_key, best.idx)
        best_keys.append(best.e_key)
    assert best_keys[1] <= best_keys[0]
    plain, _, _ = __import__("test_gpu_parity").gpu_search(cfg, cfg["searches"][0])
    assert plain.rf_block[0] == 0


def test_fronts_and_flags_on_a_problem_in_which_nothing_fits():
    """A buffer smaller than any tile set: both Pareto fronts are empty, no group is flagged, and the plain search
    reports that nothing fits."""
    cfg = mi.random_tiny_problem(3)
    arch = dict(cfg["arch"], gb_bytes=2 * cfg["workload"]["word_bytes"])
    obj = dict(cfg["searches"][0], objective=mi.OBJ_ENERGY, topk=1)
    assert mm.mmee_pareto_front_bs_da(cfg["workload"], arch, obj) == []
    assert mm.mmee_pareto_front(cfg["workload"], arch, obj) == []
    small = dict(cfg, arch=arch)
    obj = shrink_to(small, obj, 400_000)
    p = oracle.make_problem(small["workload"], small["arch"], obj)
    n_groups = (p.t_end - p.t_begin) * p.R // 5
    assert not _filter_flags(small, obj, 2 ** 62, n_groups).any()
    with Handle(small, obj) as h:
        best, _ = mm.mmee_search_host(h)
    assert best.idx == mm.NO_INDEX and best.status == mm.ERR_NO_FEASIBLE and best.n_feasible == 0
