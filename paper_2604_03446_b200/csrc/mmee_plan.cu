// Host planner: input validation, tiling enumeration by integer factorisation (Section VI-A),
// the query vectors of every (order, operand, level) -- the paper's offline enumeration of loop
// orders and buffering levels, kept as 8-bit selector rows of the query matrices (Section V-E,
// Section VI-A) -- energy quantisation and the worst-case key bound.
#include "mmee_plan.h"

#include <cmath>
#include <cstring>

namespace mmee {

namespace {

// Orders of the three outer inter-tile loops, outer -> inner.  k2 is always the innermost
// inter-tile loop (level 4): an intermediate tile must be fully accumulated before the consumer
// may read it (constraint "No Psum Propagation", Section III-C).
const int kOrders[6][3] = {
    {LOOP_I, LOOP_L, LOOP_J}, {LOOP_L, LOOP_I, LOOP_J}, {LOOP_I, LOOP_J, LOOP_L},
    {LOOP_L, LOOP_J, LOOP_I}, {LOOP_J, LOOP_I, LOOP_L}, {LOOP_J, LOOP_L, LOOP_I}};

// Own inter-tile dimensions of A(i,k) B(k,l) C(i,l) D(l,j) E(i,j)  (Section V-A).
const int kOwn[5][2] = {{LOOP_I, LOOP_K}, {LOOP_K, LOOP_L}, {LOOP_I, LOOP_L},
                        {LOOP_L, LOOP_J}, {LOOP_I, LOOP_J}};

inline uint8_t bit_d(int loop) { return (uint8_t)(1u << loop); }        // x_D of a loop
inline uint8_t bit_g(int loop) { return (uint8_t)(1u << (4 + loop)); }  // x_G of a loop

struct Nest {
    int level_of[4];      // loop -> level 4..7
    uint8_t absent;       // loops (as x_D bits) that do not exist in this nest
};

Nest nest_of(int order, uint8_t absent) {
    Nest n;
    n.level_of[LOOP_K] = 4;
    n.level_of[kOrders[order][2]] = 5;
    n.level_of[kOrders[order][1]] = 6;
    n.level_of[kOrders[order][0]] = 7;
    n.absent = absent;
    return n;
}

// Query row of BS_X (Section V-B): the two x_G bits of the operand's tile plus the x_D bit of every own loop
// that sits at or below the buffering level.
uint8_t buffer_query(const Nest& n, int x, int beta) {
    uint8_t q = (uint8_t)(bit_g(kOwn[x][0]) | bit_g(kOwn[x][1]));
    for (int s = 0; s < 2; ++s) {
        int a = kOwn[x][s];
        if (!(n.absent & bit_d(a)) && n.level_of[a] <= beta) q |= bit_d(a);
    }
    return q;
}

// DA_X, Scenario 1 (Section V-C): BS_X times the blocker's bound times the bounds of the
// effective dimensions above the blocker.  The blocker is the lowest own loop above beta.
uint8_t dram_query_own_blocker(const Nest& n, int x, int beta, uint8_t effective) {
    uint8_t q = buffer_query(n, x, beta);
    int blocker = -1;
    for (int s = 0; s < 2; ++s) {
        int a = kOwn[x][s];
        if ((n.absent & bit_d(a)) || n.level_of[a] <= beta) continue;
        if (blocker < 0 || n.level_of[a] < n.level_of[blocker]) blocker = a;
    }
    if (blocker < 0) return q;                       // operand fully resident: fetched once
    q |= bit_d(blocker);
    for (int u = 0; u < 4; ++u)
        if (!(n.absent & bit_d(u)) && (effective & bit_d(u)) && n.level_of[u] > n.level_of[blocker])
            q |= bit_d(u);
    return q;
}

// C is regenerated for every j2 iteration when j2 runs outside the loop that replaces the
// buffered part of C (Section III-C, "Recomputation").
bool regenerates_c(const Nest& n, int beta_c) {
    int lowest = 99;
    if (n.level_of[LOOP_I] > beta_c && n.level_of[LOOP_I] < lowest) lowest = n.level_of[LOOP_I];
    if (n.level_of[LOOP_L] > beta_c && n.level_of[LOOP_L] < lowest) lowest = n.level_of[LOOP_L];
    return lowest != 99 && n.level_of[LOOP_J] > lowest;
}

int quantise(double e_pj, double quantum, int64_t* out) {
    if (!(e_pj >= 0.0) || !(quantum > 0.0) || !std::isfinite(e_pj)) return MMEE_ERR_ARG;
    double ratio = e_pj / quantum;
    double nearest = std::nearbyint(ratio);
    double tol = 1e-6 * (nearest > 1.0 ? nearest : 1.0);
    if (std::fabs(ratio - nearest) > tol) return MMEE_ERR_QUANTUM;
    if (nearest > 1e15) return MMEE_ERR_OVERFLOW;
    *out = (int64_t)nearest;
    return MMEE_OK;
}

}  // namespace

void build_query_tables(QueryTables* q) {
    std::memset(q, 0, sizeof(*q));
    const uint8_t producer_dims = (uint8_t)(bit_d(LOOP_I) | bit_d(LOOP_K) | bit_d(LOOP_L));
    const uint8_t consumer_dims = (uint8_t)(bit_d(LOOP_I) | bit_d(LOOP_L) | bit_d(LOOP_J));
    for (int o = 0; o < 6; ++o) {
        const Nest fused = nest_of(o, 0);
        const Nest op1 = nest_of(o, bit_d(LOOP_J));       // unfused producer nest: no j2
        const Nest op2 = nest_of(o, bit_d(LOOP_K));       // unfused consumer nest: no k2
        for (int b = 3; b <= 7; ++b) {
            q->recompute[o][b - 3] = regenerates_c(fused, b) ? 1 : 0;
            for (int x = 0; x < 5; ++x) {
                const bool consumer = (x == OP_D || x == OP_E);
                q->bs[o][x][b - 3] = buffer_query(fused, x, b);
                for (int rc = 0; rc < 2; ++rc) {
                    uint8_t v;
                    if (x == OP_C) {
                        v = 0;                               // DA_C = 0 when fused
                    } else if (consumer && b == 3) {
                        // Scenario 2: the blocker is the producer's reduction loop k2; its bound
                        // is excluded and every loop above it is effective for the consumer.
                        v = (uint8_t)(buffer_query(fused, x, b) | consumer_dims);
                    } else {
                        // Effective dims (Section V-A): producer operands see j2 only under
                        // recomputation; consumer operands see the whole fused nest.
                        uint8_t eff = consumer ? consumer_dims
                                               : (uint8_t)(producer_dims | (rc ? bit_d(LOOP_J) : 0));
                        v = dram_query_own_blocker(fused, x, b, eff);
                    }
                    q->da[o][x][b - 3][rc] = v;
                }
                if (x == OP_A || x == OP_B)
                    q->da_unfused[o][x][b - 3] = dram_query_own_blocker(op1, x, b, producer_dims);
                else if (x == OP_D || x == OP_E)
                    q->da_unfused[o][x][b - 3] = dram_query_own_blocker(op2, x, b, consumer_dims);
                else
                    q->da_unfused[o][x][b - 3] = dram_query_own_blocker(op2, OP_C, 3, consumer_dims);
            }
        }
    }
}

int build_plan(const mmee_workload_t* w, const mmee_arch_t* a, const mmee_objective_t* o, Plan* p) {
    if (!w || !a || !o || !p) return MMEE_ERR_ARG;
    std::memset(p, 0, sizeof(*p));
    if (!w->batch || !w->q_heads || !w->kv_heads || (w->q_heads % w->kv_heads)) return MMEE_ERR_ARG;
    if (!w->seq_q || !w->seq_kv || !w->d_qk || !w->d_v || !w->word_bytes) return MMEE_ERR_ARG;
    if (!a->pe_rows || !a->pe_cols || !a->n_arrays || !a->dram_words_per_cycle) return MMEE_ERR_ARG;
    if (o->objective > MMEE_OBJ_LATENCY_ECAP) return MMEE_ERR_ARG;
    if (o->objective >= MMEE_OBJ_ENERGY_LCAP && o->key_cap < 0) return MMEE_ERR_ARG;
    if (o->topk < 1) return MMEE_ERR_ARG;
    if (o->topk > MMEE_MAX_TOPK) return MMEE_ERR_RANGE;
    if (o->row_pruning > 1 || (o->row_pruning && o->topk != 1)) return MMEE_ERR_ARG;
    if (o->tiling_set > MMEE_TILE_ALL_DIVISORS || o->order_set > MMEE_ORD_ALL6) return MMEE_ERR_ARG;
    if (!(o->fuse_mask & 7u) || (o->fuse_mask & ~7u)) return MMEE_ERR_ARG;
    if ((o->stationary_mask & ~0x1ffu) || o->rf_tiling > 1) return MMEE_ERR_ARG;
    if (o->rf_tiling && (o->objective > MMEE_OBJ_LATENCY || !a->rf_bytes)) return MMEE_ERR_ARG;

    // The g = q_heads/kv_heads query heads of one K/V head are stacked along I, so that K and V
    // are fetched once per group; each (batch, kv head) pair is one independent instance.
    const uint64_t dims[4] = {(uint64_t)(w->q_heads / w->kv_heads) * w->seq_q, w->d_qk, w->seq_kv, w->d_v};
    const uint64_t inst = (uint64_t)w->batch * w->kv_heads;
    if (inst > 0xffffffffull) return MMEE_ERR_ARG;
    p->instances = (uint32_t)inst;
    p->n_arrays = a->n_arrays;

    p->n_tilings = 1;
    for (int d = 0; d < 4; ++d) {
        if (dims[d] > 0xffffffffull) return MMEE_ERR_ARG;
        p->dim[d] = (uint32_t)dims[d];
        // divisors in ascending order: small ones up, cofactors down
        uint32_t lo[MMEE_MAX_DIVISORS], hi[MMEE_MAX_DIVISORS];
        uint32_t nlo = 0, nhi = 0;
        for (uint64_t x = 1; x * x <= dims[d]; ++x) {
            if (dims[d] % x) continue;
            const uint64_t y = dims[d] / x;
            const bool keep_x = o->tiling_set == MMEE_TILE_ALL_DIVISORS || !(x & (x - 1));
            const bool keep_y = (y != x) && (o->tiling_set == MMEE_TILE_ALL_DIVISORS || !(y & (y - 1)));
            if (keep_x) { if (nlo == MMEE_MAX_DIVISORS) return MMEE_ERR_RANGE; lo[nlo++] = (uint32_t)x; }
            if (keep_y) { if (nhi == MMEE_MAX_DIVISORS) return MMEE_ERR_RANGE; hi[nhi++] = (uint32_t)y; }
        }
        if (nlo + nhi > MMEE_MAX_DIVISORS) return MMEE_ERR_RANGE;
        uint32_t n = 0;
        for (uint32_t i = 0; i < nlo; ++i) p->divs[d][n++] = lo[i];
        for (uint32_t i = nhi; i-- > 0;) p->divs[d][n++] = hi[i];
        p->ndiv[d] = n;
        p->n_tilings *= n;
    }

    if (o->order_set == MMEE_ORD_NORECOMP2) { p->n_orders = 2; p->order_id[0] = 0; p->order_id[1] = 1; }
    else { p->n_orders = 6; for (uint32_t i = 0; i < 6; ++i) p->order_id[i] = i; }

    // Row blocks: the fused block of every order first, then one block per order and unfused mode.
    for (uint32_t phi = 0; phi < 3; ++phi) {
        if (!(o->fuse_mask & (1u << phi))) continue;
        for (uint32_t s = 0; s < p->n_orders; ++s) {
            p->block_phi[p->n_blocks] = (uint8_t)phi;
            p->block_order_slot[p->n_blocks] = (uint8_t)s;
            ++p->n_blocks;
            if (phi == 0) ++p->n_fused_blocks;
        }
    }
    p->fused_tasks = p->n_fused_blocks * 25u;
    p->tasks_per_tiling = p->fused_tasks + (p->n_blocks - p->n_fused_blocks) * 5u;
    p->rows_per_tiling = p->tasks_per_tiling * (uint32_t)kRowsPerTask;
    if (p->n_tilings > UINT64_MAX / ((uint64_t)p->rows_per_tiling * 9u)) return MMEE_ERR_OVERFLOW;

    p->t_begin = o->t_begin;
    p->t_end = o->t_end;
    if (p->t_begin == 0 && p->t_end == 0) p->t_end = p->n_tilings;
    if (p->t_begin > p->t_end || p->t_end > p->n_tilings) return MMEE_ERR_ARG;

    int rc;
    if ((rc = quantise(a->e_dram_pj, a->energy_quantum_pj, &p->cq[0]))) return rc;
    if ((rc = quantise(a->e_gb_pj, a->energy_quantum_pj, &p->cq[1]))) return rc;
    if ((rc = quantise(a->e_rf_pj, a->energy_quantum_pj, &p->cq[2]))) return rc;
    if ((rc = quantise(a->e_mac_pj, a->energy_quantum_pj, &p->cq[3]))) return rc;
    if ((rc = quantise(a->c_softmax * a->e_mac_pj, a->energy_quantum_pj, &p->cq[4]))) return rc;
    p->quantum_pj = a->energy_quantum_pj;
    p->has_rf = a->rf_bytes > 0 ? 1u : 0u;
    if (p->has_rf && a->rf_bytes < 6ull * w->word_bytes) return MMEE_ERR_ARG;

    // Energy is linear in the access counts, so the per-level coefficients are regrouped per count:
    //   E = cq_dram*N_DRAM + cq_gb*(N_DRAM + BR) + cq_rf*(BR + 3*N_MAC) + cq_mac*N_MAC + cq_sfu*N_SFU
    p->c_dram_gb = p->cq[0] + p->cq[1];
    p->c_br = p->cq[1] + (p->has_rf ? p->cq[2] : 0);
    p->c_mac = p->cq[3] + (p->has_rf ? 3 * p->cq[2] : 0);
    p->c_sfu = p->cq[4];

    // The row loop compares buffer sizes in 32 bits, saturated at 2^30 - 1 words.
    if (a->gb_bytes / w->word_bytes >= (1ull << 30) - 1) return MMEE_ERR_RANGE;
    p->cap_words = (int64_t)(a->gb_bytes / w->word_bytes);
    p->bw = a->dram_words_per_cycle;
    p->pe_rows = a->pe_rows;
    p->pe_cols = a->pe_cols;
    p->objective = o->objective;
    p->topk = o->topk;
    p->row_pruning = o->row_pruning;
    p->sm_mask = o->stationary_mask ? o->stationary_mask : 0x1ffu;
    for (uint32_t b = 0; b < 9; ++b) p->n_sm += (p->sm_mask >> b) & 1u;
    p->key_cap = o->key_cap;
    p->rf_tiling = o->rf_tiling;
    {
        const uint64_t rfw = a->rf_bytes / w->word_bytes;
        p->rf_words = rfw > 0xffffffffull ? 0xffffffffu : (uint32_t)rfw;
    }

    // Largest key any mapping of this problem can have.  M bounds the MAC count with the largest
    // recomputation factor (j_D <= J); each of at most seven DRAM terms is <= I*K*L*J <= M, the
    // array moves at most 5 words per MAC, a tile takes at most one cycle per MAC.
    const long double M = (long double)dims[0] * dims[2] * dims[3] * ((long double)dims[1] + 1.0L);
    const long double emax = M * (7.0L * p->cq[0] + 12.0L * p->cq[1] + 8.0L * p->cq[2] + p->cq[3] + p->cq[4]);
    const long double lmax = M * (7.0L + (long double)p->bw);
    const long double limit = 4611686018427387904.0L;     // 2^62
    if (emax >= limit || lmax >= limit) return MMEE_ERR_OVERFLOW;

    // Scale of the 32-bit threshold-relative keys of the energy and latency walks: the largest DRAM term of any
    // mapping, I*K*L*J words (times c_dram_gb quanta for energy), must fit below 2^28 after the shift.
    p->rel_shift = 0;
    p->unit = 1;
    if (p->objective == MMEE_OBJ_ENERGY || p->objective == MMEE_OBJ_LATENCY) {
        long double biggest = (long double)dims[0] * dims[1] * dims[2] * dims[3] *
                              (p->objective == MMEE_OBJ_ENERGY ? (long double)p->c_dram_gb : 1.0L);
        while (biggest >= 268435456.0L) { biggest /= 2.0L; ++p->rel_shift; }
    }

    build_query_tables(&p->q);
    return MMEE_OK;
}

}  // namespace mmee
