// Device-side model arithmetic shared by the kernels: exact monomials from query vectors
// (Section V-E), array-level terms per stationary mode, and the full evaluation of one mapping.
#pragma once

#include "mmee_plan.h"

namespace mmee {

// exp(q . ln b) taken exactly: the product of the bounds the query vector selects (Eq. 8).
__device__ __forceinline__ int64_t monomial(uint32_t q, const uint32_t b[8]) {
    int64_t v = 1;
#pragma unroll
    for (int d = 0; d < 8; ++d)
        if (q & (1u << d)) v *= (int64_t)b[d];
    return v;
}

// Ceiling of a / b for 32-bit operands (tile extents and array sizes), widened for the products.
__device__ __forceinline__ int64_t ceil_div(uint32_t a, uint32_t b) { return (int64_t)((a + b - 1u) / b); }

// Compute cycles of one (m x r) * (r x n) tile on a rows x cols array.
// 0 weight stationary: r x n weights folded onto the array, m inputs streamed per fold;
// 1 input stationary:  m x r inputs folded, n weight columns streamed;
// 2 output stationary: m x n outputs folded, r reduction steps streamed.
__device__ __forceinline__ int64_t tile_cycles(int sm, uint32_t m, uint32_t r, uint32_t n, uint32_t rows, uint32_t cols) {
    if (sm == 0) return ceil_div(r, rows) * ceil_div(n, cols) * (int64_t)m;
    if (sm == 1) return ceil_div(m, rows) * ceil_div(r, cols) * (int64_t)n;
    return ceil_div(m, rows) * ceil_div(n, cols) * (int64_t)r;
}

// Words moved between the global buffer and the array for one tile: the stationary operand
// once, the streamed operand once per fold of the other dimension, partial sums read and
// written between reduction folds (2*folds - 1 transfers per output element).
__device__ __forceinline__ int64_t tile_traffic(int sm, uint32_t m, uint32_t r, uint32_t n, uint32_t rows, uint32_t cols) {
    const int64_t M = m, R = r, N = n;
    if (sm == 0) return R * N + M * R * ceil_div(n, cols) + M * N * (2 * ceil_div(r, rows) - 1);
    if (sm == 1) return M * R + R * N * ceil_div(m, rows) + M * N * (2 * ceil_div(r, cols) - 1);
    return M * R * ceil_div(n, cols) + R * N * ceil_div(m, rows) + M * N;
}

// Register-file-level tiling (objective.rf_tiling): buffer<->array words and compute cycles of one tile when
// its stationary operand is processed in blocks of a x b elements; the block is searched over the divisors of the
// operand's two extents (dimension ids da, db: the extents are tile extents of those dimensions, so their
// divisors are among the plan's divisor lists), in ascending (a, b) order, keeping the admissible block with
// the least (words, cycles) for the energy objective and the least (cycles, words) for the latency objective.
// blk receives the block as (m, r, n) extents, 1 for the streamed extent.
__device__ __forceinline__ void rf_block_terms(const Plan& p, int sm, uint32_t m, uint32_t r, uint32_t n, int da, int db,
                                               int64_t& words, int64_t& cycles, uint32_t blk[3]) {
    const uint32_t ea = sm == 0 ? r : m, eb = sm == 0 ? n : (sm == 1 ? r : n);
    const int64_t M = m, R = r, N = n;
    bool have = false;
    int64_t bw = 0, bc = 0;
    uint32_t ba = 0, bb = 0;
    for (uint32_t ia = 0; ia < p.ndiv[da]; ++ia) {
        const uint32_t a = p.divs[da][ia];
        if (a > ea) break;
        if (ea % a) continue;
        const int64_t ha = ceil_div(a, p.pe_rows);
        for (uint32_t ib = 0; ib < p.ndiv[db]; ++ib) {
            const uint32_t b = p.divs[db][ib];
            if (b > eb) break;
            if (eb % b) continue;
            const int64_t held = ha * ceil_div(b, p.pe_cols);       // stationary elements per PE
            if (held + 2 > (int64_t)p.rf_words) continue;
            int64_t w, c;
            if (sm == 0) {
                w = R * N + M * R * (int64_t)(n / b) + M * N * (2 * (int64_t)(r / a) - 1);
                c = (int64_t)(r / a) * (int64_t)(n / b) * M * held;
            } else if (sm == 1) {
                w = M * R + R * N * (int64_t)(m / a) + M * N * (2 * (int64_t)(r / b) - 1);
                c = (int64_t)(m / a) * (int64_t)(r / b) * N * held;
            } else {
                w = M * R * (int64_t)(n / b) + R * N * (int64_t)(m / a) + M * N;
                c = (int64_t)(m / a) * (int64_t)(n / b) * R * held;
            }
            const bool better = !have || (p.objective == MMEE_OBJ_LATENCY ? (c < bc || (c == bc && w < bw))
                                                                          : (w < bw || (w == bw && c < bc)));
            if (better) { have = true; bw = w; bc = c; ba = a; bb = b; }
        }
    }
    // (a block of one element needs three registers, which the planner requires: some block is always admissible)
    words = bw;
    cycles = bc;
    blk[0] = sm == 0 ? 1u : ba;
    blk[1] = sm == 0 ? ba : (sm == 1 ? bb : 1u);
    blk[2] = sm == 1 ? 1u : bb;
}

// Words and cycles of one tile of operator `op` (0: (i_G x k_G)(k_G x l_G), 1: (i_G x l_G)(l_G x j_G)) under
// stationary mode sm: one array fold per pass, or the register-file block search.
__device__ __forceinline__ void tile_array_terms(const Plan& p, const uint32_t b[8], int op, int sm, int64_t& words,
                                                 int64_t& cycles, uint32_t blk[3]) {
    const uint32_t m = b[4], r = op == 0 ? b[5] : b[6], n = op == 0 ? b[6] : b[7];
    if (p.rf_tiling) {
        // dimensions of the stationary operand's two extents
        const int dm = LOOP_I, dr = op == 0 ? LOOP_K : LOOP_L, dn = op == 0 ? LOOP_L : LOOP_J;
        rf_block_terms(p, sm, m, r, n, sm == 0 ? dr : dm, sm == 0 ? dn : (sm == 1 ? dr : dn), words, cycles, blk);
    } else {
        words = tile_traffic(sm, m, r, n, p.pe_rows, p.pe_cols);
        cycles = tile_cycles(sm, m, r, n, p.pe_rows, p.pe_cols);
        blk[0] = blk[1] = blk[2] = 0;
    }
}

// Tile invocations and carried partial sums of one tiling (no recomputation).
struct TilingCounts {
    int64_t t1, t2;             // tile invocations of Op1 and Op2
    int64_t carry1, carry2;     // partial sums carried between consecutive reduction steps
    int64_t ikl, ilj, il;       // I*K*L, I*L*J, I*L
};

__device__ __forceinline__ TilingCounts tiling_counts(const Plan& p, const uint32_t b[8]) {
    const int64_t iD = b[0], kD = b[1], lD = b[2], jD = b[3], iG = b[4], lG = b[6], jG = b[7];
    TilingCounts c;
    c.t1 = iD * kD * lD;
    c.t2 = iD * lD * jD;
    c.carry1 = (c.t1 - iD * lD) * iG * lG;      // every reduction step but the first of each C tile
    c.carry2 = (c.t2 - iD * jD) * iG * jG;
    c.ikl = (int64_t)p.dim[0] * p.dim[1] * p.dim[2];
    c.ilj = (int64_t)p.dim[0] * p.dim[2] * p.dim[3];
    c.il = (int64_t)p.dim[0] * p.dim[2];
    return c;
}

// Tiling index -> boundary vector b (one column of the boundary matrix, Section VI-A).
__device__ __forceinline__ void tiling_bounds(const Plan& p, uint64_t t64, uint32_t b[8]) {
    uint32_t t = (uint32_t)t64;                 // at most MMEE_MAX_DIVISORS^4 = 2^24 tilings
#pragma unroll
    for (int d = 3; d >= 0; --d) {
        const uint32_t q = t / p.ndiv[d];
        const uint32_t a = t - q * p.ndiv[d];
        t = q;
        const uint32_t g = p.divs[d][a];
        b[4 + d] = g;
        b[d] = p.dim[d] / g;
    }
}

// Task index inside a tiling -> (block, outer levels).  A task is 125 consecutive rows: a fused
// task fixes the levels of A and B and walks those of C, D, E; an unfused task (C always at L3)
// fixes the level of A and walks those of B, D, E.
struct TaskChoice {
    uint32_t block, phi, order_slot, order;
    uint32_t la, lb;            // beta - 3; lb is not used by an unfused task
};

__device__ __forceinline__ TaskChoice decode_task(const Plan& p, uint32_t w) {
    TaskChoice c;
    if (w < p.fused_tasks) {
        c.block = w / 25u;
        const uint32_t rem = w - c.block * 25u;
        c.la = rem / 5u;
        c.lb = rem % 5u;
    } else {
        const uint32_t u = w - p.fused_tasks;
        c.block = p.n_fused_blocks + u / 5u;
        c.la = u % 5u;
        c.lb = 0;
    }
    c.phi = p.block_phi[c.block];
    c.order_slot = p.block_order_slot[c.block];
    c.order = p.order_id[c.order_slot];
    return c;
}

// One candidate index taken apart (index layout: include/mmee.h).
struct CandidateChoice {
    uint64_t t;
    uint32_t row, s;
    TaskChoice c;
    uint32_t lv[5];             // beta - 3 of A, B, C, D, E
    int sm1, sm2;
    bool fused;
    uint32_t rc;                // C is regenerated (Section III-C)
};

__device__ __forceinline__ CandidateChoice decode_candidate(const Plan& p, uint64_t idx) {
    CandidateChoice d;
    const uint64_t per_t = (uint64_t)p.rows_per_tiling * 9u;
    d.t = idx / per_t;
    const uint32_t rem = (uint32_t)(idx - d.t * per_t);
    d.row = rem / 9u;
    d.s = rem % 9u;
    const uint32_t w = d.row / 125u, mid = (d.row % 125u) / 25u, de = d.row % 25u;
    d.c = decode_task(p, w);
    d.fused = d.c.phi == 0;
    d.lv[OP_A] = d.c.la;
    d.lv[OP_B] = d.fused ? d.c.lb : mid;
    d.lv[OP_C] = d.fused ? mid : 0u;
    d.lv[OP_D] = de / 5u;
    d.lv[OP_E] = de % 5u;
    d.sm1 = (int)(d.s / 3u);
    d.sm2 = (int)(d.s % 3u);
    d.rc = d.fused ? p.q.recompute[d.c.order][d.lv[OP_C]] : 0u;
    return d;
}

// Buffer words and DRAM words of one operand (Section V-B, V-C) from its two query vectors.  For the
// intermediate C of an unfused mapping `da` is the read-back by the consumer nest only.
__device__ __forceinline__ void operand_terms(const Plan& p, const CandidateChoice& d, const uint32_t b[8], int x,
                                              int64_t& bs, int64_t& da) {
    const QueryTables& q = p.q;
    bs = monomial(q.bs[d.c.order][x][d.lv[x]], b);
    if (d.fused) da = (x == OP_C) ? 0 : monomial(q.da[d.c.order][x][d.lv[x]][d.rc], b);
    else da = monomial(q.da_unfused[d.c.order][x][d.lv[x]], b);
}

// Array-level terms of one operator (0: C = A*B, 1: E = C*D) under one stationary mode: buffer<->PE words
// including the carried partial sums, and compute cycles.
__device__ __forceinline__ void operator_array_terms(const Plan& p, const uint32_t b[8], const TilingCounts& c, int op,
                                                     int sm, bool recompute, int64_t& words, int64_t& cycles,
                                                     uint32_t blk[3]) {
    int64_t w, cy;
    tile_array_terms(p, b, op, sm, w, cy, blk);
    if (op == 0) {
        const int64_t rho = recompute ? (int64_t)b[3] : 1;
        const int64_t t1 = rho * c.t1;
        words = t1 * w + rho * c.carry1;
        cycles = t1 * cy;
    } else {
        words = c.t2 * w + c.carry2;
        cycles = c.t2 * cy;
    }
}

// The record of one mapping from its parts: all five metric groups of Section VI-A (buffer sizes of
// producer and consumer, DRAM access, compute latency of both operators, buffer<->register
// traffic), then energy and latency (Section V-D).
__device__ __forceinline__ void assemble_record(const Plan& p, uint64_t idx, const CandidateChoice& d, const uint32_t b[8],
                                                const TilingCounts& tt, const int64_t bs[5], const int64_t da_in[5],
                                                int64_t words1, int64_t cyc1, int64_t words2, int64_t cyc2,
                                                const uint32_t blk1[3], const uint32_t blk2[3], mmee_result_t& o) {
    const uint32_t* lv = d.lv;
    o.idx = idx; o.t = d.t; o.row = d.row;
    for (int i = 0; i < 8; ++i) o.bound[i] = b[i];
    o.phi = (uint8_t)d.c.phi; o.pi = (uint8_t)d.c.order;
    for (int x = 0; x < 5; ++x) o.beta[x] = (uint8_t)(lv[x] + 3);
    o.sm[0] = (uint8_t)d.sm1; o.sm[1] = (uint8_t)d.sm2;
    for (int i = 0; i < 5; ++i) o.reserved[i] = 0;
    o.status = MMEE_OK;

    int64_t da[5];
    for (int x = 0; x < 5; ++x) da[x] = da_in[x];
    int64_t bs1, bs2, da_sm = 0, da1 = 0, da2 = 0;
    if (d.fused) {
        // Eq. (1)/(2): operands of the other operator count only when retained (tau = 1).
        bs1 = bs[OP_A] + bs[OP_B] + bs[OP_C] + (lv[OP_D] ? bs[OP_D] : 0) + (lv[OP_E] ? bs[OP_E] : 0);
        bs2 = bs[OP_C] + bs[OP_D] + bs[OP_E] + (lv[OP_A] ? bs[OP_A] : 0) + (lv[OP_B] ? bs[OP_B] : 0);
    } else {
        bs1 = bs[OP_A] + bs[OP_B] + bs[OP_C];
        bs2 = bs[OP_C] + bs[OP_D] + bs[OP_E];
        const int64_t c_write = tt.il;                 // Op1 stores C, Op2 reads it back
        da1 = da[OP_A] + da[OP_B] + c_write;
        da2 = da[OP_C] + da[OP_D] + da[OP_E];
        da[OP_C] += c_write;
        if (d.c.phi == 2) da_sm = 2 * tt.il;           // separate softmax pass: read S, write P
    }
    const int64_t n_dram = da[0] + da[1] + da[2] + da[3] + da[4] + da_sm;
    const int64_t rho = d.rc ? (int64_t)b[3] : 1;
    const int64_t n_mac = rho * tt.ikl + tt.ilj, n_sfu = rho * tt.il, br = words1 + words2;
    const int64_t n_gb = n_dram + br;
    const int64_t n_rf = p.has_rf ? br + 3 * n_mac : 0;

    const int64_t e_key = p.cq[0] * n_dram + p.cq[1] * n_gb + p.cq[2] * n_rf + p.cq[3] * n_mac + p.cq[4] * n_sfu;
    int64_t l_key;
    if (d.fused) {
        const int64_t comp = (cyc1 + cyc2) * (int64_t)p.bw;
        l_key = n_dram > comp ? n_dram : comp;
    } else {
        const int64_t c1 = cyc1 * (int64_t)p.bw, c2 = cyc2 * (int64_t)p.bw;
        l_key = (da1 > c1 ? da1 : c1) + da_sm + (da2 > c2 ? da2 : c2);
    }

    for (int x = 0; x < 5; ++x) { o.bs_x[x] = bs[x]; o.da_x[x] = da[x]; }
    o.bs_op1 = bs1; o.bs_op2 = bs2; o.bs = bs1 > bs2 ? bs1 : bs2;
    o.da_sm = da_sm;
    o.br = br; o.cyc1 = cyc1; o.cyc2 = cyc2;
    o.n[0] = n_dram; o.n[1] = n_gb; o.n[2] = n_rf; o.n[3] = n_mac; o.n[4] = n_sfu;
    o.e_key = e_key; o.l_key = l_key;
    o.recompute = (uint8_t)d.rc;
    o.feasible = (uint8_t)(o.bs <= p.cap_words && ((p.sm_mask >> d.s) & 1u));
    o.edp_key = __dmul_rn((double)e_key, (double)l_key);
    o.energy_pj = __dmul_rn(__dmul_rn((double)e_key, p.quantum_pj), (double)p.instances);
    const uint32_t waves = (p.instances + p.n_arrays - 1) / p.n_arrays;
    o.latency_cycles = __dmul_rn(__ddiv_rn((double)l_key, (double)p.bw), (double)waves);
    o.n_total = 0; o.n_feasible = 0;
    for (int i = 0; i < 3; ++i) { o.rf_block[i] = blk1[i]; o.rf_block[3 + i] = blk2[i]; }
    o.reserved2[0] = o.reserved2[1] = 0;
}

// Full evaluation of one mapping by one thread.
__device__ inline void evaluate_candidate(const Plan& p, uint64_t idx, mmee_result_t& o) {
    const CandidateChoice d = decode_candidate(p, idx);
    uint32_t b[8];
    tiling_bounds(p, d.t, b);
    const TilingCounts tt = tiling_counts(p, b);
    int64_t bs[5], da[5];
    for (int x = 0; x < 5; ++x) operand_terms(p, d, b, x, bs[x], da[x]);
    int64_t w1, c1, w2, c2;
    uint32_t blk1[3], blk2[3];
    operator_array_terms(p, b, tt, 0, d.sm1, d.rc != 0, w1, c1, blk1);
    operator_array_terms(p, b, tt, 1, d.sm2, d.rc != 0, w2, c2, blk2);
    assemble_record(p, idx, d, b, tt, bs, da, w1, c1, w2, c2, blk1, blk2, o);
}

// The same by one warp (all 32 lanes call it converged): lanes 0..4 take one operand each, lanes 5 and 6 one
// operator's array-level terms each; lane 0 gathers the parts and holds the record on return.
__device__ inline void evaluate_candidate_warp(const Plan& p, uint64_t idx, int lane, mmee_result_t& o) {
    const CandidateChoice d = decode_candidate(p, idx);
    uint32_t b[8];
    tiling_bounds(p, d.t, b);
    const TilingCounts tt = tiling_counts(p, b);
    int64_t v0 = 0, v1 = 0;
    uint32_t blk[3] = {0, 0, 0};
    if (lane < 5) operand_terms(p, d, b, lane, v0, v1);
    else if (lane < 7) operator_array_terms(p, b, tt, lane - 5, lane == 5 ? d.sm1 : d.sm2, d.rc != 0, v0, v1, blk);
    int64_t part0[7], part1[7];
#pragma unroll
    for (int i = 0; i < 7; ++i) {
        part0[i] = __shfl_sync(0xffffffffu, v0, i);
        part1[i] = __shfl_sync(0xffffffffu, v1, i);
    }
    uint32_t blk1[3], blk2[3];
#pragma unroll
    for (int i = 0; i < 3; ++i) {
        blk1[i] = __shfl_sync(0xffffffffu, blk[i], 5);
        blk2[i] = __shfl_sync(0xffffffffu, blk[i], 6);
    }
    if (lane == 0) assemble_record(p, idx, d, b, tt, part0, part1, part0[5], part1[5], part0[6], part1[6], blk1, blk2, o);
}

}  // namespace mmee
