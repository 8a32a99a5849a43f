"""GPU parity: the CUDA library against the CPU oracle, through the C ABI.

Integer fields (access counts, buffer sizes, keys, indices, counters) must be bit-identical;
floating-point outputs within 1e-12 relative.
"""
import glob
import json
import os

import numpy as np
import pytest
import torch

import mmee_inputs as mi
import oracle
import paper_2604_03446_b200.binding as mm

pytestmark = pytest.mark.gpu

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
REL_TOL = 1e-12
INT_FIELDS = ("idx", "t", "row", "phi", "pi", "recompute", "feasible", "bs_op1", "bs_op2", "bs",
              "da_sm", "br", "cyc1", "cyc2", "e_key", "l_key")
ARRAY_FIELDS = ("bound", "beta", "sm", "bs_x", "da_x", "n", "rf_block")
FLOAT_FIELDS = ("edp_key", "energy_pj", "latency_cycles")


def assert_same_record(g, o, where=""):
    for f in INT_FIELDS:
        assert int(getattr(g, f)) == int(getattr(o, f)), "%s field %s" % (where, f)
    for f in ARRAY_FIELDS:
        assert list(getattr(g, f)) == list(getattr(o, f)), "%s field %s" % (where, f)
    for f in FLOAT_FIELDS:
        a, b = float(getattr(g, f)), float(getattr(o, f))
        assert abs(a - b) <= REL_TOL * abs(b), "%s field %s: %r vs %r" % (where, f, a, b)


class Handle:
    def __init__(self, cfg, obj):
        self.args = (cfg["workload"], cfg["arch"], obj)
        self.h = None

    def __enter__(self):
        self.h = mm.mmee_create(*self.args)
        return self.h

    def __exit__(self, *exc):
        mm.mmee_destroy(self.h)


def gpu_search(cfg, obj):
    k = obj["topk"]
    best, topk = mm.result_buffer(1), mm.result_buffer(k)
    with Handle(cfg, obj) as h:
        mm.mmee_search(h, best, topk)
        torch.cuda.synchronize()
        stats = mm.mmee_last_search_stats(h)
    return mm.read_results(best, 1)[0], mm.read_results(topk, k), stats


def check_search(cfg, obj, threads=0):
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    want = oracle.search(p, threads)
    best, topk, _ = gpu_search(cfg, obj)
    assert best.n_total == want.n_total
    assert best.n_feasible == want.n_feasible
    found = [r for r in topk if r.idx != mm.NO_INDEX]
    assert [r.idx for r in found] == [r.idx for r in want.topk]
    for g, o in zip(found, want.topk):
        assert_same_record(g, o, cfg["name"])
    if want.topk:
        assert best.status == mm.OK and best.idx == want.topk[0].idx
        assert_same_record(best, want.topk[0], cfg["name"])
    else:
        assert best.status == mm.ERR_NO_FEASIBLE and best.idx == mm.NO_INDEX
    return best, found


def shrink(cfg, obj, limit):
    """Restrict the tiling range so that at most `limit` candidates are enumerated."""
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    if p.N <= limit:
        return dict(obj)
    return dict(obj, t_begin=0, t_end=max(1, limit // (p.R * 9)))


TINY_SEEDS = list(range(1, 13))


@pytest.mark.parametrize("seed", TINY_SEEDS)
def test_every_candidate_key_matches_the_oracle(seed):
    """The search kernel's own evaluation path, element by element: one key per candidate,
    INT64_MAX where the mapping does not fit the buffer."""
    cfg = mi.random_tiny_problem(seed)
    obj = shrink(cfg, cfg["searches"][0], 4_000_000)
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    begin, count = p.t_begin * p.R * 9, (p.t_end - p.t_begin) * p.R * 9
    keys, feas = oracle.keys_range(p, begin, count)
    want = np.where(feas.astype(bool), keys, np.iinfo(np.int64).max)
    out = torch.full((count,), -7, dtype=torch.int64, device="cuda")
    with Handle(cfg, obj) as h:
        assert mm.mmee_num_candidates(h) == p.N
        mm.mmee_dump_keys(h, out)
        torch.cuda.synchronize()
    got = out.cpu().numpy()
    bad = np.nonzero(got != want)[0]
    assert bad.size == 0, "first mismatch at candidate %d: %d vs %d" % (begin + bad[0], got[bad[0]], want[bad[0]])


@pytest.mark.parametrize("seed", TINY_SEEDS[:8])
def test_every_candidate_record_matches_the_oracle(seed):
    """The query-vector evaluation (mmee_eval): every field of every candidate."""
    cfg = mi.random_tiny_problem(seed)
    obj = cfg["searches"][0]
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    count = min(p.N, 150_000)
    begin = (p.N - count) // 2
    want = oracle.evaluate_range(p, begin, count)
    buf = mm.result_buffer(count)
    with Handle(cfg, obj) as h:
        mm.mmee_eval(h, begin, count, buf)
        torch.cuda.synchronize()
    got = mm.read_results(buf, count)
    for g, o in zip(got, want):
        assert_same_record(g, o, "seed %d idx %d" % (seed, o.idx))


@pytest.mark.parametrize("seed", TINY_SEEDS)
@pytest.mark.parametrize("k", [1, 16])
def test_search_matches_the_oracle_on_tiny_problems(seed, k):
    cfg = mi.random_tiny_problem(seed)
    for objective in (mi.OBJ_ENERGY, mi.OBJ_LATENCY, mi.OBJ_EDP):
        obj = shrink(cfg, dict(cfg["searches"][0], objective=objective, topk=k), 6_000_000)
        check_search(cfg, obj)


@pytest.mark.parametrize("seed", TINY_SEEDS[:6])
@pytest.mark.parametrize("log2_quantum", [-12, -24])
def test_energy_search_in_coarse_relative_units(seed, log2_quantum):
    """The energy walk keeps threshold-relative keys in units of 2^rel_shift quanta once the largest DRAM term
    leaves 28 bits.  A small energy quantum (a power of two, so that every energy stays an integer multiple)
    drives small problems into that regime and, at 2^-24 pJ, into saturated stationary-pair terms; the top-16,
    the optimum and the feasible count must still be the oracle's."""
    cfg = mi.random_tiny_problem(seed)
    arch = dict(cfg["arch"], energy_quantum_pj=2.0 ** log2_quantum)
    cfg = dict(cfg, arch=arch)
    for k in (1, 16):
        obj = shrink(cfg, dict(cfg["searches"][0], objective=mi.OBJ_ENERGY, topk=k), 6_000_000)
        check_search(cfg, obj)


@pytest.mark.parametrize("seed", TINY_SEEDS[:6])
def test_search_with_the_largest_admissible_buffer(seed):
    """Capacities just below 2^30 words (the documented maximum): no size saturates below the capacity, every
    mapping fits, and the 32-bit capacity arithmetic of the walk must not overflow."""
    cfg = mi.random_tiny_problem(seed)
    wb = cfg["workload"]["word_bytes"]
    cfg = dict(cfg, arch=dict(cfg["arch"], gb_bytes=((1 << 30) - 2) * wb))
    for objective in (mi.OBJ_ENERGY, mi.OBJ_LATENCY):
        obj = shrink(cfg, dict(cfg["searches"][0], objective=objective, topk=4), 4_000_000)
        best, _ = check_search(cfg, obj)
        assert best.n_feasible == best.n_total


@pytest.mark.parametrize("seed", TINY_SEEDS[:8])
def test_search_over_a_subset_of_stationary_pairs(seed):
    """Arrays that offer only some stationary pairs (Section VII-K): every objective, k = 1 and 16, masks from a
    single pair to eight of nine; optimum, top-k, records and the feasible count against the oracle."""
    cfg = mi.random_tiny_problem(seed)
    masks = [1 << (seed % 9), 0x1ff ^ (1 << ((3 * seed) % 9)), (0x0a5 << (seed % 2)) & 0x1ff, 0x007, 0x049]
    for i, mask in enumerate(masks):
        objective = (mi.OBJ_ENERGY, mi.OBJ_LATENCY, mi.OBJ_EDP)[(seed + i) % 3]
        for k in (1, 16):
            obj = shrink(cfg, dict(cfg["searches"][0], objective=objective, topk=k, stationary_mask=mask), 4_000_000)
            _, found = check_search(cfg, obj)
            assert all((mask >> (3 * r.sm[0] + r.sm[1])) & 1 for r in found)


def test_every_key_with_a_stationary_mask():
    """The key dump under a mask: INT64_MAX for the pairs the array does not offer, the oracle's key elsewhere."""
    cfg = mi.random_tiny_problem(4)
    for objective, mask in ((mi.OBJ_ENERGY, 0x124), (mi.OBJ_LATENCY, 0x00f), (mi.OBJ_EDP, 0x180)):
        obj = shrink(cfg, dict(cfg["searches"][0], objective=objective, stationary_mask=mask), 2_000_000)
        p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
        begin, count = p.t_begin * p.R * 9, (p.t_end - p.t_begin) * p.R * 9
        keys, feas = oracle.keys_range(p, begin, count)
        want = np.where(feas.astype(bool), keys, np.iinfo(np.int64).max)
        got = torch.empty(count, dtype=torch.int64, device="cuda")
        with Handle(cfg, obj) as h:
            mm.mmee_dump_keys(h, got)
            torch.cuda.synchronize()
        assert np.array_equal(got.cpu().numpy(), want)


def test_search_shapes_picks_the_best_logical_array():
    """Reconfigurable array shapes (Section VII-K): one search per shape, each equal to the oracle's search on that
    shape, and the index of the shape with the least key; for the four designs of the paper's comparison
    (fixed pair on one shape, free pairs, free shape, both) more freedom is never worse."""
    cfg = mi.random_tiny_problem(6)
    shapes = [(4, 4), (2, 8), (8, 2), (1, 16), (16, 1)]
    best_key = {}
    for name, mask, shp in (("fixed", 0x001, shapes[:1]), ("flow", 0x1ff, shapes[:1]),
                            ("shape", 0x001, shapes), ("shape_flow", 0x1ff, shapes)):
        obj = shrink(cfg, dict(cfg["searches"][0], objective=mi.OBJ_EDP, topk=1, stationary_mask=mask), 3_000_000)
        per_shape, best = mm.mmee_search_shapes(cfg["workload"], cfg["arch"], obj, shp)
        want = []
        for (r, c), got in zip(shp, per_shape):
            arch = dict(cfg["arch"], pe_rows=r, pe_cols=c)
            res = oracle.search(oracle.make_problem(cfg["workload"], arch, obj))
            assert got.n_feasible == res.n_feasible
            if res.topk:
                assert_same_record(got, res.topk[0], name)
                want.append(res.topk[0].edp_key)
            else:
                assert got.idx == mm.NO_INDEX
                want.append(float("inf"))
        assert best == (None if min(want) == float("inf") else want.index(min(want)))
        best_key[name] = min(want)
    assert best_key["shape_flow"] <= best_key["shape"] <= best_key["fixed"]
    assert best_key["shape_flow"] <= best_key["flow"] <= best_key["fixed"]


def test_config1_full_search():
    cfg = mi.config1()
    best, _ = check_search(cfg, cfg["searches"][0])
    assert best.n_total == 162067500
    check_search(cfg, dict(cfg["searches"][0], topk=16, objective=mi.OBJ_LATENCY))
    check_search(cfg, dict(cfg["searches"][0], topk=16, objective=mi.OBJ_EDP))


def _golden_files():
    return sorted(glob.glob(os.path.join(GOLDEN, "search_*.json")))


@pytest.mark.parametrize("path", _golden_files(), ids=lambda p: os.path.basename(p)[7:-5])
def test_full_size_search_matches_stored_oracle_answers(path):
    """Benchmark configurations at full size, in the launch configuration the benchmark times.
    Expected values were written by tests/golden/make_search_goldens.py from the oracle alone."""
    with open(path) as f:
        gold = json.load(f)
    cfg = dict(name=gold["name"], workload=gold["workload"], arch=gold["arch"])
    for s in gold["searches"]:
        best, topk, stats = gpu_search(cfg, s["objective"])
        assert stats.kernels_launched == 1 and stats.grid >= 1
        assert best.n_total == s["n_total"] and best.n_feasible == s["n_feasible"]
        found = [r for r in topk if r.idx != mm.NO_INDEX]
        assert [r.idx for r in found] == [r["idx"] for r in s["topk"]]
        for g, o in zip(found, s["topk"]):
            for f in ("t", "row", "phi", "pi", "recompute", "bs", "bs_op1", "bs_op2", "br", "cyc1", "cyc2",
                      "e_key", "l_key"):
                assert int(getattr(g, f)) == o[f], f
            for f in ("bound", "beta", "sm", "n"):
                assert list(getattr(g, f)) == o[f], f
            for f in ("edp_key", "energy_pj", "latency_cycles"):
                b = float.fromhex(o[f + "_hex"])
                assert abs(float(getattr(g, f)) - b) <= REL_TOL * abs(b), f


@pytest.mark.parametrize("maker", [mi.config2, mi.config3, mi.config4])
def test_sampled_candidates_at_full_size(maker):
    """Candidates drawn over the whole index space of the large configurations, each compared
    field by field with the oracle's one-at-a-time evaluation."""
    cfg = maker()
    rng = np.random.default_rng(11)
    for obj in cfg["searches"]:
        p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
        starts = [0, p.N - 64] + [int(v) for v in rng.integers(0, p.N - 64, size=30)]
        with Handle(cfg, obj) as h:
            for s in starts:
                buf = mm.result_buffer(64)
                mm.mmee_eval(h, s, 64, buf)
                torch.cuda.synchronize()
                for g, o in zip(mm.read_results(buf, 64), oracle.evaluate_range(p, s, 64)):
                    assert_same_record(g, o, "%s idx %d" % (cfg["name"], o.idx))


def test_sub_ranges_partition_the_search():
    """Tiling sub-ranges: each range agrees with the oracle; the best over the ranges is the best
    of the whole; feasible counts add up."""
    cfg = mi.random_tiny_problem(5)
    obj = dict(cfg["searches"][0], objective=mi.OBJ_ENERGY, topk=4)
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    T = p.T
    cuts = [0, T // 3, T // 3 + 1, T]
    total_feasible, bests = 0, []
    for lo, hi in zip(cuts[:-1], cuts[1:]):
        best, found = check_search(cfg, dict(obj, t_begin=lo, t_end=hi))
        total_feasible += best.n_feasible
        bests += [(r.e_key, r.idx) for r in found]
    whole, found = check_search(cfg, obj)
    assert total_feasible == whole.n_feasible
    assert sorted(bests)[:len(found)] == [(r.e_key, r.idx) for r in found]


@pytest.mark.parametrize("n_tilings", [1, 2, 3, 5, 7, 9, 12, 23, 64])
def test_interval_lengths_around_the_range_order_cases(n_tilings):
    """The kernel's CTAs pull ranges of the task interval in a two-part order (some spread evenly, the others
    ascending, a tail).  Intervals of 1 to 64 tilings give 1 to about 30 ranges (odd and even counts, with and
    without a tail): every range must be walked exactly once, which the feasible count and the top-k show."""
    cfg = mi.config2()
    obj = dict(cfg["searches"][1], topk=3, t_begin=1000, t_end=1000 + n_tilings)
    check_search(cfg, obj)


def test_interval_with_more_ranges_than_ctas_but_fewer_than_twice_as_many():
    """About 420 ranges on a grid of at most 296 CTAs: the spread part is half the ranges, not one per CTA."""
    cfg = mi.config2()
    check_search(cfg, dict(cfg["searches"][0], topk=2, t_begin=300, t_end=1200))


def test_whole_tiling_ranges_with_odd_interval_ends():
    """An interval long enough for ranges of whole tilings with a tail of short ranges, with ends that are not
    multiples of the range length: the two small end pieces are checked against the oracle directly, and the three
    pieces together must give the stored whole-problem answer (feasible count; the best of the pieces)."""
    with open(os.path.join(GOLDEN, "search_gqa_b4_s8192.json")) as f:
        gold = json.load(f)
    cfg = dict(name=gold["name"], workload=gold["workload"], arch=gold["arch"])
    s = gold["searches"][0]
    obj = dict(s["objective"], topk=1)
    T = oracle.make_problem(cfg["workload"], cfg["arch"], obj).T
    lo, hi = 3, T - 5
    pieces = [check_search(cfg, dict(obj, t_begin=0, t_end=lo))[0], check_search(cfg, dict(obj, t_begin=hi, t_end=T))[0]]
    big, _, stats = gpu_search(cfg, dict(obj, t_begin=lo, t_end=hi))
    assert stats.tasks == (hi - lo) * 210
    pieces.append(big)
    assert sum(p.n_feasible for p in pieces) == s["n_feasible"]
    key = {mi.OBJ_ENERGY: "e_key", mi.OBJ_LATENCY: "l_key"}.get(obj["objective"])
    best = min((p for p in pieces if p.idx != mm.NO_INDEX),
               key=lambda p: ((getattr(p, key) if key else p.edp_key), p.idx))
    assert best.idx == s["topk"][0]["idx"]


def test_nothing_fits():
    cfg = mi.random_tiny_problem(3)
    arch = dict(cfg["arch"], gb_bytes=cfg["workload"]["word_bytes"] * 2)
    best, found = check_search(dict(cfg, arch=arch), dict(cfg["searches"][0], topk=3))
    assert best.n_feasible == 0 and not found and best.status == mm.ERR_NO_FEASIBLE


def test_fewer_feasible_mappings_than_k():
    """A capacity that admits only a handful of mappings leaves the tail of the top-k empty."""
    cfg = dict(name="scarce", workload=mi.workload(1, 1, 1, 4, 4, 2, 2, 1),
               arch=mi.arch(2, 2, 1, 3, 0, 1, 10.0, 2.0, 0.0, 1.0))
    obj = mi.objective(mi.OBJ_ENERGY, 16, mi.TILE_ALL_DIVISORS, mi.ORD_NORECOMP2, mi.FUSE_FUSED)
    best, found = check_search(cfg, obj)
    assert 0 < best.n_feasible // 9 and len(found) <= 16


def test_massive_ties_keep_the_lowest_indices():
    """Latency on a compute-bound problem: a large share of the mappings tie at the optimum and the
    top-k must be exactly the k lowest indices among them."""
    cfg = dict(name="ties", workload=mi.workload(1, 1, 1, 64, 64, 16, 16, 2),
               arch=mi.arch(4, 4, 1, 64 * 1024, 64, 4096, 100.0, 5.0, 1.0, 1.0))
    obj = mi.objective(mi.OBJ_LATENCY, 16, mi.TILE_POW2, mi.ORD_ALL6, mi.FUSE_ALL)
    best, found = check_search(cfg, obj)
    assert len({r.l_key for r in found}) == 1


def test_repeated_searches_on_one_handle_are_identical():
    cfg = mi.config1()
    obj = dict(cfg["searches"][0], topk=16)
    bufs = [(mm.result_buffer(1), mm.result_buffer(16)) for _ in range(3)]
    with Handle(cfg, obj) as h:
        for b, t in bufs:
            mm.mmee_search(h, b, t)
        torch.cuda.synchronize()
    raws = [(bytes(b.cpu().numpy().tobytes()), bytes(t.cpu().numpy().tobytes())) for b, t in bufs]
    assert raws[0] == raws[1] == raws[2]


def test_host_buffer_entry_point_equals_device_path():
    cfg = mi.config1()
    obj = dict(cfg["searches"][0], topk=4)
    best, topk, h2d, d2h = mm.mmee_solve_host(cfg["workload"], cfg["arch"], obj)
    dbest, dtopk, _ = gpu_search(cfg, obj)
    assert bytes(best) == bytes(dbest)
    assert [bytes(r) for r in topk] == [bytes(r) for r in dtopk]
    assert h2d > 0 and d2h == 5 * mm.RESULT_BYTES


def test_search_on_a_side_stream():
    cfg = mi.random_tiny_problem(2)
    obj = shrink(cfg, dict(cfg["searches"][0], topk=2), 2_000_000)
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    want = oracle.search(p)
    st = torch.cuda.Stream()
    best = mm.result_buffer(1)
    with Handle(cfg, obj) as h:
        with torch.cuda.stream(st):
            mm.mmee_search(h, best, None, stream=st)
        st.synchronize()
    got = mm.read_results(best, 1)[0]
    assert got.idx == (want.topk[0].idx if want.topk else mm.NO_INDEX)


@pytest.mark.parametrize("seed", TINY_SEEDS)
def test_row_pruning_keeps_the_optimum(seed):
    """Offline symbolic row pruning (Section VI-B) in its tie-safe form: the optimum record of the
    pruned search is the oracle's optimum of the full space, index included, for every objective."""
    cfg = mi.random_tiny_problem(seed)
    for objective in (mi.OBJ_ENERGY, mi.OBJ_LATENCY, mi.OBJ_EDP):
        obj = shrink(cfg, dict(cfg["searches"][0], objective=objective, topk=1), 6_000_000)
        p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
        want = oracle.search(p)
        best = mm.result_buffer(1)
        with Handle(cfg, dict(obj, row_pruning=1)) as h:
            mm.mmee_search(h, best, None)
            torch.cuda.synchronize()
            stats = mm.mmee_last_search_stats(h)
        got = mm.read_results(best, 1)[0]
        assert stats.rows_evaluated_per_tiling < stats.rows_per_tiling
        if want.topk:
            assert_same_record(got, want.topk[0], "seed %d objective %d" % (seed, objective))
        else:
            assert got.idx == mm.NO_INDEX and got.status == mm.ERR_NO_FEASIBLE


def test_row_pruning_on_the_benchmark_workloads():
    for path in _golden_files():
        with open(path) as f:
            gold = json.load(f)
        if "sweep" in gold["name"] and not gold["name"].endswith("s1024"):
            continue
        cfg = dict(name=gold["name"], workload=gold["workload"], arch=gold["arch"])
        for s in gold["searches"]:
            obj = dict(s["objective"], topk=1, row_pruning=1)
            best = mm.result_buffer(1)
            with Handle(cfg, obj) as h:
                mm.mmee_search(h, best, None)
                torch.cuda.synchronize()
            got = mm.read_results(best, 1)[0]
            o = s["topk"][0]
            assert got.idx == o["idx"] and got.e_key == o["e_key"] and got.l_key == o["l_key"] and list(got.n) == o["n"]


def test_row_pruning_needs_a_single_optimum():
    cfg = mi.config1()
    with pytest.raises(mm.MmeeError) as e:
        mm.mmee_create(cfg["workload"], cfg["arch"], dict(cfg["searches"][0], topk=2, row_pruning=1))
    assert e.value.code == mm.ERR_ARG


def test_two_gemm_and_conv_chain_shapes_sampled():
    """Non-attention chains with ragged divisor lists (Section VII-J): sampled mappings field by field."""
    rng = np.random.default_rng(23)
    for cfg in mi.beyond_attention_configs():
        obj = cfg["searches"][0]
        p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
        with Handle(cfg, obj) as h:
            assert mm.mmee_num_candidates(h) == p.N
            for s in [0, p.N - 32] + [int(v) for v in rng.integers(0, p.N - 32, size=12)]:
                buf = mm.result_buffer(32)
                mm.mmee_eval(h, s, 32, buf)
                torch.cuda.synchronize()
                for g, o in zip(mm.read_results(buf, 32), oracle.evaluate_range(p, s, 32)):
                    assert_same_record(g, o, "%s idx %d" % (cfg["name"], o.idx))


def test_dram_traffic_against_buffer_size_is_a_staircase():
    """Fused feed-forward GEMMs, least DRAM traffic per buffer size (Section VII-C): 7.605e8 x 9
    mappings per search; traffic never rises with a larger buffer, never falls below the compulsory
    |A| + |B| + |D| + |E|, and the optimum is a real mapping that fits (re-evaluated by the oracle)."""
    pts = mi.ffn_dram_sweep_configs()
    last = None
    for cfg in pts[::3]:
        obj = cfg["searches"][0]
        best, _, _ = gpu_search(cfg, obj)
        assert best.n_total == 760500000 * 9 and best.status == mm.OK
        p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
        o = oracle.evaluate(p, best.idx)
        assert_same_record(best, o, cfg["name"])
        assert o.feasible and o.e_key == o.n[0]
        I, K, L, J = [int(v) for v in p.dim]
        assert o.n[0] >= I * K + K * L + L * J + I * J
        if last is not None:
            assert o.n[0] <= last
        last = o.n[0]


def _all_keys(cfg, base_obj, limit):
    """(e_key, l_key, feasible, idx) of every candidate of the (possibly range-limited) problem."""
    oe = shrink(cfg, dict(base_obj, objective=mi.OBJ_ENERGY, topk=1), limit)
    ol = dict(oe, objective=mi.OBJ_LATENCY)
    pe = oracle.make_problem(cfg["workload"], cfg["arch"], oe)
    pl = oracle.make_problem(cfg["workload"], cfg["arch"], ol)
    begin, count = pe.t_begin * pe.R * 9, (pe.t_end - pe.t_begin) * pe.R * 9
    ek, feas = oracle.keys_range(pe, begin, count)
    lk, _ = oracle.keys_range(pl, begin, count)
    return oe, ek, lk, feas.astype(bool), np.arange(begin, begin + count, dtype=np.int64)


def _brute_force_front(ek, lk, feas, idx):
    order = np.lexsort((idx[feas], lk[feas], ek[feas]))
    e, l, i = ek[feas][order], lk[feas][order], idx[feas][order]
    front, best_l = [], None
    for a, b, c in zip(e, l, i):
        if best_l is None or b < best_l:
            front.append((int(a), int(b), int(c)))
            best_l = b
    return front


@pytest.mark.parametrize("seed", [1, 2, 3, 5, 7, 9])
def test_energy_latency_pareto_front(seed):
    """The front of Section VII-E by alternating capped searches, against a brute-force sweep over
    every candidate's (energy, latency) pair from the oracle; each point with its lowest index."""
    cfg = mi.random_tiny_problem(seed)
    base = dict(cfg["searches"][0], row_pruning=0)
    obj, ek, lk, feas, idx = _all_keys(cfg, base, 3_000_000)
    want = _brute_force_front(ek, lk, feas, idx)
    got = mm.mmee_pareto_front(cfg["workload"], cfg["arch"], obj)
    assert [(r.e_key, r.l_key, r.idx) for r in got] == want
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    for r in got:
        assert_same_record(r, oracle.evaluate(p, r.idx), "front point %d" % r.idx)


def test_capped_searches_match_brute_force():
    cfg = mi.random_tiny_problem(4)
    obj, ek, lk, feas, idx = _all_keys(cfg, cfg["searches"][0], 3_000_000)
    for cap_q in (0.1, 0.5, 0.9):
        lcap = int(np.quantile(lk[feas], cap_q))
        ok = feas & (lk <= lcap)
        order = np.lexsort((idx[ok], ek[ok]))
        best, _, _ = gpu_search(cfg, dict(obj, objective=mi.OBJ_ENERGY_LCAP, key_cap=lcap))
        assert (best.e_key, best.idx) == (int(ek[ok][order[0]]), int(idx[ok][order[0]])) and best.l_key <= lcap
        ecap = int(np.quantile(ek[feas], cap_q))
        ok = feas & (ek <= ecap)
        order = np.lexsort((idx[ok], lk[ok]))
        best, _, _ = gpu_search(cfg, dict(obj, objective=mi.OBJ_LATENCY_ECAP, key_cap=ecap))
        assert (best.l_key, best.idx) == (int(lk[ok][order[0]]), int(idx[ok][order[0]])) and best.e_key <= ecap
    best, _, _ = gpu_search(cfg, dict(obj, objective=mi.OBJ_ENERGY_LCAP, key_cap=int(lk[feas].min()) - 1))
    assert best.idx == mm.NO_INDEX and best.status == mm.ERR_NO_FEASIBLE


def test_largest_divisor_list_and_ragged_dims():
    """A dimension with exactly the maximum number of divisors (7560 = 2^3 3^3 5 7 has 64), others
    ragged: sub-range searches at both ends of the tiling space, all three objectives."""
    cfg = dict(name="divisors64", workload=mi.workload(1, 1, 1, 7560, 30, 6, 6, 2),
               arch=mi.arch(4, 8, 2, 8192, 64, 6, 120.0, 4.0, 1.0, 0.5, c_softmax=3.0, energy_quantum_pj=0.5))
    base = mi.objective(mi.OBJ_ENERGY, 5)
    p = oracle.make_problem(cfg["workload"], cfg["arch"], base)
    assert list(p.ndiv) == [64, 4, 8, 4] and p.T == 8192
    for objective, (lo, hi) in ((mi.OBJ_ENERGY, (0, 9)), (mi.OBJ_LATENCY, (4000, 4007)), (mi.OBJ_EDP, (8185, 8192))):
        check_search(cfg, dict(base, objective=objective, t_begin=lo, t_end=hi))


@pytest.mark.parametrize("seed", range(13, 41))
def test_more_random_problems_keys_and_optimum(seed):
    """Wider seed range: every candidate key through the search kernel's own path, and the top-5."""
    cfg = mi.random_tiny_problem(seed)
    obj = shrink(cfg, dict(cfg["searches"][0], topk=5), 1_500_000)
    p = oracle.make_problem(cfg["workload"], cfg["arch"], obj)
    begin, count = p.t_begin * p.R * 9, (p.t_end - p.t_begin) * p.R * 9
    keys, feas = oracle.keys_range(p, begin, count)
    want = np.where(feas.astype(bool), keys, np.iinfo(np.int64).max)
    out = torch.full((count,), -7, dtype=torch.int64, device="cuda")
    with Handle(cfg, obj) as h:
        mm.mmee_dump_keys(h, out)
        torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy(), want)
    check_search(cfg, obj)


@pytest.mark.parametrize("topk", [1, 16])
def test_repeated_searches_after_a_cache_flush_agree(topk):
    """The same search launched many times, each time directly after a kernel that fills the L2 with written
    lines (what the benchmark does between steps): every launch returns the oracle's list.  (A search kernel
    that read the list length k from the shared-memory copy of its plan before the barrier that completes the
    copy passed every single-launch test and failed this one in about one launch in a hundred: after the
    writing kernel the copy is slower, and a warp that ran ahead took k from what the previous kernel had left
    in shared memory.)"""
    cfg = mi.config1()
    obj = dict(cfg["searches"][0], topk=topk)
    want = oracle.search(oracle.make_problem(cfg["workload"], cfg["arch"], obj))
    expected = (want.n_feasible, tuple((w.idx, w.e_key) for w in want.topk))
    flush = torch.empty(64 * 1024 * 1024, dtype=torch.uint8, device="cuda")
    best, top = mm.result_buffer(1), mm.result_buffer(topk)
    with Handle(cfg, obj) as h:
        for it in range(1200):
            if it < 1000:
                flush.fill_(it & 255)
            mm.mmee_search(h, best, top)
            torch.cuda.synchronize()
            r = mm.read_results(best, 1)[0]
            got = (r.n_feasible, tuple((x.idx, x.e_key) for x in mm.read_results(top, topk)))
            assert r.status == mm.OK and got == expected, (it, r.status, got[1][:2], expected[1][:2])
