"""Pins of the oracle's array-level terms and of its unfused rows (no GPU needed).

The closed forms of the oracle (compute cycles and buffer<->array words per stationary mode, carried
partial sums, MAC and register-file counts, DRAM words and buffer need of the two separate loop nests
of an unfused mapping) are compared with executions that count events one by one and contain none of
those formulas: `mo_array_tile` / `mo_array_chain` run every tile on the PE array fold by fold,
`mo_simulate_unfused` runs the producer nest, the softmax pass and the consumer nest tile by tile.
"""
import itertools

import numpy as np
import pytest

import mmee_inputs as mi
import oracle
from helpers import candidate_index, tiling_index

WS, IS, OS = 0, 1, 2


def _single_tile_problem(m, r, n, j, rows, cols):
    """Dims equal to one tile: with x_G = X every inter-tile bound is 1, each operator runs one tile."""
    return oracle.make_problem(mi.workload(1, 1, 1, m, n, r, j, 1),
                               mi.arch(rows, cols, 1, 10 ** 9, 64, 1, 1.0, 1.0, 1.0, 1.0),
                               mi.objective(fuse_mask=mi.FUSE_FUSED))


@pytest.mark.parametrize("rows,cols", [(1, 1), (2, 3), (3, 2), (4, 4), (5, 3), (3, 7)])
def test_tile_cycles_and_traffic_against_fold_by_fold_execution(rows, cols):
    """Section V-D (compute latency from the array size and its utilisation; buffer<->register traffic by
    stationary mode).  One tile per operator, every extent from 1 to 7 where the array is smaller, equal
    and larger, including extents that are no multiple of the array: the oracle's cycles and words equal
    what the fold-by-fold execution counts.  Rows and columns differ, so a formula with the two array
    dimensions (or two tile extents) exchanged fails here."""
    checked = 0
    for m, r, n, j in itertools.product((1, 2, 3, 5, 7), (1, 2, 4, 7), (1, 3, 4, 6), (2, 5)):
        p = _single_tile_problem(m, r, n, j, rows, cols)
        for sm1, sm2 in itertools.product((WS, IS, OS), repeat=2):
            rec = oracle.evaluate(p, candidate_index(p, (m, r, n, j), 0, 0, (3, 3, 3, 3, 3), (sm1, sm2)))
            assert list(rec.bound[:4]) == [1, 1, 1, 1]
            t1 = oracle.array_tile(sm1, m, r, n, rows, cols)
            t2 = oracle.array_tile(sm2, m, n, j, rows, cols)
            assert rec.cyc1 == t1.cycles and rec.cyc2 == t2.cycles
            assert rec.br == t1.words + t2.words
            assert rec.n[3] == t1.macs + t2.macs == m * r * n + m * n * j
            assert rec.n[2] == t1.rf + t2.rf
            checked += 1
    assert checked == 5 * 4 * 4 * 2 * 9


def test_a_fully_used_array_needs_macs_over_pes_cycles():
    """When every tile extent is a multiple of the array extent it is folded over, no PE idles: the executed
    cycle count is MACs / PEs for every stationary mode (the 100 % utilisation case behind the paper's Table I
    latencies), and it is larger as soon as one extent is not a multiple."""
    for sm in (WS, IS, OS):
        full = oracle.array_tile(sm, 8, 12, 6, 2, 3)
        assert full.macs == 8 * 12 * 6
        assert full.cycles * 6 == full.macs
        ragged = oracle.array_tile(sm, 7, 11, 5, 2, 3)
        assert ragged.macs == 7 * 11 * 5 and ragged.cycles * 6 > ragged.macs


def _rho_by_simulation(rec):
    """How often the whole of C is produced, from the tile-level execution of the fused nest."""
    sim = oracle.simulate(list(rec.bound), rec.pi, list(rec.beta))
    tiles = rec.bound[0] * rec.bound[2]
    assert sim.c_productions % tiles == 0
    return sim.c_productions // tiles


@pytest.mark.parametrize("dims,tile,array", [((4, 6, 6, 4), (2, 3, 2, 2), (2, 2)), ((6, 4, 9, 6), (2, 2, 3, 2), (3, 2)),
                                             ((8, 3, 4, 6), (2, 1, 2, 3), (1, 4)), ((6, 6, 4, 9), (3, 2, 1, 3), (2, 5))])
def test_array_terms_of_whole_mappings_against_element_level_execution(dims, tile, array):
    """BR, compute cycles, MACs and register-file accesses of whole mappings: every tile invocation of both
    operators is executed on the array in loop order.  A reduction step after the first of an output tile has
    to take that tile's partial sums in again (the carried partial sums); C is produced once, or j_D times
    when the fused nest regenerates it (the factor is taken from the tile-level execution of the nest, not
    from the oracle's flag).  Fused rows with and without recomputation and unfused rows, all nine stationary
    pairs."""
    I, K, L, J = dims
    rows, cols = array
    p = oracle.make_problem(mi.workload(1, 1, 1, I, L, K, J, 1),
                            mi.arch(rows, cols, 1, 10 ** 9, 64, 3, 7.0, 5.0, 3.0, 2.0),
                            mi.objective())
    t = tiling_index(p, tile)
    rng = np.random.default_rng(11)
    picked = list(rng.integers(0, 18750, size=24)) + list(rng.integers(18750, 26250, size=8))
    # one row that certainly recomputes: order (j, i, l), C at L3
    picked.append(4 * 3125)
    seen_rho = set()
    for r in picked:
        for s in range(9):
            rec = oracle.evaluate(p, (t * p.R + int(r)) * 9 + s)
            rho = _rho_by_simulation(rec) if rec.phi == 0 else 1
            seen_rho.add(rho)
            op1, op2 = oracle.array_chain(list(rec.bound), rho, s // 3, s % 3, rows, cols)
            assert rec.cyc1 == op1.cycles and rec.cyc2 == op2.cycles
            assert rec.br == op1.words + op2.words
            assert rec.n[3] == op1.macs + op2.macs
            assert rec.n[2] == op1.rf + op2.rf == rec.br + 3 * rec.n[3]
            assert rec.n[1] == rec.n[0] + rec.br
    assert len(seen_rho) == 2


def test_no_register_file_level_means_no_register_file_accesses():
    p = oracle.make_problem(mi.workload(1, 1, 1, 4, 4, 4, 4, 1), mi.arch(2, 2, 1, 10 ** 9, 0, 1, 1, 1, 0, 1),
                            mi.objective())
    for idx in range(0, p.N, 997):
        assert oracle.evaluate(p, idx).n[2] == 0


def _unfused_levels(q):
    return (3 + q // 125, 3 + (q // 25) % 5, 3, 3 + (q // 5) % 5, 3 + q % 5)


@pytest.mark.parametrize("phi", [1, 2])
@pytest.mark.parametrize("dims,tile", [((4, 6, 6, 4), (2, 3, 2, 2)), ((6, 4, 9, 6), (2, 2, 3, 2))])
def test_unfused_rows_against_execution_of_the_two_nests(phi, dims, tile):
    """All 3 750 rows (6 orders x 5^4 levels of A, B, D, E) of an unfused mode on a tiling whose inter-tile
    bounds are all >= 2: DRAM words of every operand, the C round trip (stored once by the producer nest, read
    back by the consumer nest), the separate softmax pass, the per-operator DRAM sums and both operators'
    buffer needs equal what a tile-by-tile execution of the two nests counts."""
    I, K, L, J = dims
    bw = 3
    rows, cols = 2, 3
    p = oracle.make_problem(mi.workload(1, 1, 1, I, L, K, J, 1),
                            mi.arch(rows, cols, 1, 10 ** 9, 64, bw, 7.0, 5.0, 3.0, 2.0, c_softmax=4.0),
                            mi.objective(fuse_mask=1 << phi))
    assert p.R == 3750
    t = tiling_index(p, tile)
    for r in range(3750):
        pi, q = divmod(r, 625)
        beta = _unfused_levels(q)
        rec = oracle.evaluate(p, (t * p.R + r) * 9 + (r % 9))
        assert rec.phi == phi and rec.pi == pi and tuple(rec.beta) == beta and rec.recompute == 0
        assert min(rec.bound[:4]) >= 2
        sim = oracle.simulate_unfused(list(rec.bound), pi, beta, phi)
        assert sim.op1_stages == rec.bound[0] * rec.bound[1] * rec.bound[2]
        assert sim.op2_stages == rec.bound[0] * rec.bound[2] * rec.bound[3]
        for x in (0, 1, 3, 4):
            assert rec.da_x[x] == sim.loads[x], (r, x)
        assert sim.c_stores == I * L                                  # every element of C written once
        assert rec.da_x[2] == sim.c_stores + sim.loads[2]
        assert rec.da_sm == sim.softmax_words == (2 * I * L if phi == 2 else 0)
        assert rec.da1 == sim.loads[0] + sim.loads[1] + sim.c_stores
        assert rec.da2 == sim.loads[2] + sim.loads[3] + sim.loads[4]
        assert rec.n[0] == rec.da1 + rec.da2 + rec.da_sm
        assert rec.bs_op1 == sim.peak_op1 and rec.bs_op2 == sim.peak_op2
        assert rec.bs == max(sim.peak_op1, sim.peak_op2)
        if r % 37 == 0:
            # Latency and energy from counted events only (Section V-D): the two operators and the softmax
            # pass run one after the other, inside each the DRAM transfers and the computation overlap;
            # energy is linear in the per-level access counts.
            s = r % 9
            op1, op2 = oracle.array_chain(list(rec.bound), 1, s // 3, s % 3, rows, cols)
            assert rec.l_key == max(rec.da1, op1.cycles * bw) + sim.softmax_words + max(rec.da2, op2.cycles * bw)
            n_dram = sum(sim.loads) + sim.c_stores + sim.softmax_words
            words = op1.words + op2.words
            assert rec.e_key == 7 * n_dram + 5 * (n_dram + words) + 3 * (op1.rf + op2.rf) \
                + 2 * (op1.macs + op2.macs) + 4 * 2 * I * L


def test_fused_keys_from_counted_events():
    """The energy and latency keys of fused mappings recomputed from counted events alone: tile loads of the
    fused nest (rows on which the closed forms are exact: orders 0 and 1), array words, MACs and register-file
    accesses of the element-level execution, one softmax element per produced score."""
    I, K, L, J = 4, 6, 6, 4
    bw, rows, cols = 3, 2, 3
    p = oracle.make_problem(mi.workload(1, 1, 1, I, L, K, J, 1),
                            mi.arch(rows, cols, 1, 10 ** 9, 64, bw, 7.0, 5.0, 3.0, 2.0, c_softmax=4.0),
                            mi.objective(fuse_mask=mi.FUSE_FUSED))
    t = tiling_index(p, (2, 3, 2, 2))
    rng = np.random.default_rng(5)
    for r in rng.integers(0, 6250, size=60):
        s = int(r) % 9
        rec = oracle.evaluate(p, (t * p.R + int(r)) * 9 + s)
        sim = oracle.simulate(list(rec.bound), rec.pi, list(rec.beta))
        op1, op2 = oracle.array_chain(list(rec.bound), 1, s // 3, s % 3, rows, cols)
        n_dram = sum(sim.loads)
        assert rec.n[0] == n_dram
        assert rec.l_key == max(n_dram, (op1.cycles + op2.cycles) * bw)
        assert rec.e_key == 7 * n_dram + 5 * (n_dram + op1.words + op2.words) + 3 * (op1.rf + op2.rf) \
            + 2 * (op1.macs + op2.macs) + 4 * 2 * I * L


# ---- register-file-level tiling -----------------------------------------------------------------------------------

def _divisors(x):
    return [d for d in range(1, x + 1) if x % d == 0]


def _stationary_extents(sm, m, r, n):
    return {WS: (r, n), IS: (m, r), OS: (m, n)}[sm]


def _best_block_by_execution(objective, sm, m, r, n, rows, cols, rf_words):
    """Every admissible block executed element by element; the choice rule applied to the counted figures."""
    ea, eb = _stationary_extents(sm, m, r, n)
    best = None
    for a in _divisors(ea):
        for b in _divisors(eb):
            per_pe = max(sum(1 for x in range(a) for y in range(b) if (x % rows, y % cols) == pe)
                         for pe in {(x % rows, y % cols) for x in range(a) for y in range(b)})
            if per_pe + 2 > rf_words:
                continue
            c = oracle.array_tile_blocked(sm, m, r, n, rows, cols, a, b)
            key = (c.cycles, c.words) if objective == mi.OBJ_LATENCY else (c.words, c.cycles)
            if best is None or key < best[0]:
                best = (key, (a, b), c.words, c.cycles)
    return best


@pytest.mark.parametrize("rows,cols,rf_words", [(2, 3, 3), (2, 3, 6), (3, 2, 12), (4, 4, 4), (1, 5, 40)])
def test_register_file_block_choice_against_element_level_execution(rows, cols, rf_words):
    """Register-file-level tiling: for every stationary mode and several tile shapes, the block the oracle picks and
    the words and cycles it reports equal what an element-by-element execution of every admissible block gives
    under the same choice rule (fewest words, then cycles, for energy; fewest cycles, then words, for latency;
    the first such block in ascending order)."""
    for m, r, n in [(4, 6, 6), (6, 4, 9), (8, 12, 6), (5, 7, 3), (12, 2, 8)]:
        for sm in (WS, IS, OS):
            for objective in (mi.OBJ_ENERGY, mi.OBJ_LATENCY):
                blk, words, cycles = oracle.rf_block(objective, sm, m, r, n, rows, cols, rf_words)
                _, (a, b), w_sim, c_sim = _best_block_by_execution(objective, sm, m, r, n, rows, cols, rf_words)
                want_blk = {WS: (1, a, b), IS: (a, b, 1), OS: (a, 1, b)}[sm]
                assert (blk, words, cycles) == (want_blk, w_sim, c_sim), (sm, objective, m, r, n)
                # a resumed tile takes its partial outputs in first: m * n words more, same cycles
                res = oracle.array_tile_blocked(sm, m, r, n, rows, cols, a, b, resume=True)
                assert res.words == w_sim + m * n and res.cycles == c_sim and res.macs == m * r * n


def test_mappings_under_register_file_tiling_from_counted_events():
    """Whole mappings with the third tiling level: BR, cycles, N_RF and both keys of sampled fused and unfused rows
    equal the sums over all tile invocations of the element-level execution with the picked blocks (a reduction
    step after the first of an output tile resumes it); the level changes nothing above the array: buffer need,
    DRAM words and MACs are those of the same mapping without it."""
    I, K, L, J = 8, 6, 6, 4
    rows, cols, bw = 2, 3, 3
    w = mi.workload(1, 1, 1, I, L, K, J, 1)
    a = mi.arch(rows, cols, 1, 10 ** 9, 6, bw, 7.0, 5.0, 3.0, 2.0, c_softmax=4.0)
    rng = np.random.default_rng(3)
    for objective in (mi.OBJ_ENERGY, mi.OBJ_LATENCY):
        p = oracle.make_problem(w, a, dict(mi.objective(objective), rf_tiling=1))
        plain = oracle.make_problem(w, a, mi.objective(objective))
        t = tiling_index(p, (4, 3, 2, 2))
        for r in list(rng.integers(0, 6250, size=20)) + list(rng.integers(18750, 26250, size=10)):
            s = int(r) % 9
            idx = (t * p.R + int(r)) * 9 + s
            rec, ref = oracle.evaluate(p, idx), oracle.evaluate(plain, idx)
            assert list(rec.bs_x) == list(ref.bs_x) and list(rec.da_x) == list(ref.da_x) and rec.n[3] == ref.n[3]
            iD, kD, lD, jD, iG, kG, lG, jG = rec.bound
            rho = jD if rec.recompute else 1
            blocks = (tuple(rec.rf_block[:3]), tuple(rec.rf_block[3:]))
            tiles = ((s // 3, iG, kG, lG, rho * iD * lD, kD), (s % 3, iG, lG, jG, iD * jD, lD))
            words, cyc = [], []
            for (sm, m, rr, n, outputs, steps), blk in zip(tiles, blocks):
                ab = {WS: (blk[1], blk[2]), IS: (blk[0], blk[1]), OS: (blk[0], blk[2])}[sm]
                first = oracle.array_tile_blocked(sm, m, rr, n, rows, cols, *ab)
                again = oracle.array_tile_blocked(sm, m, rr, n, rows, cols, *ab, resume=True)
                words.append(outputs * (first.words + (steps - 1) * again.words))
                cyc.append(outputs * steps * first.cycles)
            assert (rec.cyc1, rec.cyc2) == tuple(cyc) and rec.br == sum(words)
            assert rec.n[2] == rec.br + 3 * rec.n[3] and rec.n[1] == rec.n[0] + rec.br
            assert rec.e_key == 7 * rec.n[0] + 5 * rec.n[1] + 3 * rec.n[2] + 2 * rec.n[3] + 8 * rec.n[4]
            if rec.phi == 0:
                assert rec.l_key == max(rec.n[0], (rec.cyc1 + rec.cyc2) * bw)
            # the level is a refinement: the energy objective never moves more words between buffer and array than
            # the best single block shape of the plain model's kind could, and every block respects the capacity
            for sm, blk in zip((s // 3, s % 3), blocks):
                held = {WS: (blk[1], blk[2]), IS: (blk[0], blk[1]), OS: (blk[0], blk[2])}[sm]
                assert -(-held[0] // rows) * -(-held[1] // cols) + 2 <= 6


def test_register_file_tiling_is_refused_where_it_is_not_defined():
    w, a = mi.workload(1, 1, 1, 8, 8, 4, 4), mi.arch(2, 2, 1, 4096, 0, 1, 1, 1, 0, 1)
    for obj in (dict(mi.objective(mi.OBJ_ENERGY), rf_tiling=1),                      # no register-file level
                ):
        with pytest.raises(oracle.OracleError):
            oracle.make_problem(w, a, obj)
    with pytest.raises(oracle.OracleError):                                           # product objective
        oracle.make_problem(w, dict(a, rf_bytes=64, e_rf_pj=1), dict(mi.objective(mi.OBJ_EDP), rf_tiling=1))
