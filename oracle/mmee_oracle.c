/*
 * CPU oracle for the MMEE search path -- TEST INFRASTRUCTURE ONLY (see mmee_oracle.h).
 *
 * Plain restatement of the analytical model of "Fast Cross-Operator Optimization of
 * Attention Dataflow" (Sections III-VI).  One candidate at a time, ordinary branches,
 * 128-bit intermediates with "fits in int64" checks.  Nothing here is blocked, fused,
 * tabulated or reordered.
 *
 * Notation (Section V-E): loop bounds b = [i_D,k_D,l_D,j_D,i_G,k_G,l_G,j_G], x_D*x_G = X.
 * Operands A(i,k) B(k,l) C(i,l) D(l,j) E(i,j); Op1: C = A*B, Op2: E = C*D.
 * Loop levels: L3 = one tile, L4 = k2 (No Psum Propagation, Section III-C: the producer's
 * reduction loop is the innermost inter-tile loop), L5..L7 = the order of (i2,l2,j2),
 * inner to outer.
 */
#include "mmee_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef __int128 i128;

enum { LP_I = 0, LP_K = 1, LP_L = 2, LP_J = 3 };
enum { OPD_A = 0, OPD_B = 1, OPD_C = 2, OPD_D = 3, OPD_E = 4 };
enum { SM_WS = 0, SM_IS = 1, SM_OS = 2 };

/* Inter-tile orders of (i2, l2, j2), written outer -> inner. */
static const int ORDERS[6][3] = {
    {LP_I, LP_L, LP_J}, {LP_L, LP_I, LP_J}, {LP_I, LP_J, LP_L},
    {LP_L, LP_J, LP_I}, {LP_J, LP_I, LP_L}, {LP_J, LP_L, LP_I},
};

/* Operand's (inter-tile) dimensions, Section V-A. */
static const int OWN[5][2] = {
    {LP_I, LP_K}, {LP_K, LP_L}, {LP_I, LP_L}, {LP_L, LP_J}, {LP_I, LP_J},
};

static int is_own(int x, int loop) { return OWN[x][0] == loop || OWN[x][1] == loop; }

static int fits64(i128 v) { return v >= 0 && v <= (i128)INT64_MAX; }

static uint64_t ceil_div(uint64_t a, uint64_t b) { return (a + b - 1) / b; }

/* ------------------------------------------------------------------------------------------ */
/* problem set-up                                                                              */
/* ------------------------------------------------------------------------------------------ */

static int quantise(double e_pj, double quantum, int64_t* out)
{
    if (!(e_pj >= 0.0) || !(quantum > 0.0)) return MO_ERR_ARG;
    double q = e_pj / quantum;
    double r = nearbyint(q);
    if (fabs(q - r) > 1e-6 * (r > 1.0 ? r : 1.0)) return MO_ERR_QUANTUM;
    if (r > 1e15) return MO_ERR_OVERFLOW;
    *out = (int64_t)r;
    return MO_OK;
}

int mo_problem_init(const mo_workload* w, const mo_arch* a, const mo_objective* o, mo_problem* p)
{
    if (!w || !a || !o || !p) return MO_ERR_ARG;
    memset(p, 0, sizeof(*p));
    if (!w->batch || !w->q_heads || !w->kv_heads || w->q_heads % w->kv_heads) return MO_ERR_ARG;
    if (!w->seq_q || !w->seq_kv || !w->d_qk || !w->d_v || !w->word_bytes) return MO_ERR_ARG;
    if (!a->pe_rows || !a->pe_cols || !a->n_arrays || !a->dram_words_per_cycle) return MO_ERR_ARG;
    if (o->objective > MO_OBJ_EDP || o->topk < 1 || o->topk > MO_MAX_TOPK) return MO_ERR_ARG;
    if (o->tiling_set > MO_TILE_ALL_DIVISORS || o->order_set > MO_ORD_ALL6) return MO_ERR_ARG;
    if ((o->fuse_mask & 7u) == 0 || (o->fuse_mask & ~7u)) return MO_ERR_ARG;
    if (o->stationary_mask & ~0x1ffu) return MO_ERR_ARG;
    if (o->rf_tiling > 1 || o->pad) return MO_ERR_ARG;
    if (o->rf_tiling && (o->objective > MO_OBJ_LATENCY || !a->rf_bytes)) return MO_ERR_ARG;

    /* Heads are independent instances (Section V, opening paragraph: the model is stated per head); the g query
     * heads that share one K/V head are stacked along I, so K and V are loaded once per group. */
    uint64_t g = w->q_heads / w->kv_heads;
    p->dim[LP_I] = g * (uint64_t)w->seq_q;
    p->dim[LP_K] = w->d_qk;
    p->dim[LP_L] = w->seq_kv;
    p->dim[LP_J] = w->d_v;
    p->instances = w->batch * w->kv_heads;
    for (int d = 0; d < 4; ++d)
        if (p->dim[d] > 0xffffffffull) return MO_ERR_ARG;

    /* Tilings: every integer factorisation x_D * x_G = X (Section VI-A). */
    p->T = 1;
    for (int d = 0; d < 4; ++d) {
        uint32_t n = 0;
        for (uint64_t x = 1; x <= p->dim[d]; ++x) {
            if (p->dim[d] % x) continue;
            if (o->tiling_set == MO_TILE_POW2 && (x & (x - 1))) continue;
            if (n == MO_MAX_DIVISORS) return MO_ERR_ARG;
            p->divs[d][n++] = (uint32_t)x;
        }
        p->ndiv[d] = n;
        p->T *= n;
    }

    if (o->order_set == MO_ORD_NORECOMP2) { p->n_orders = 2; p->order_id[0] = 0; p->order_id[1] = 1; }
    else { p->n_orders = 6; for (int i = 0; i < 6; ++i) p->order_id[i] = (uint32_t)i; }
    p->n_phi = 0;
    for (uint32_t phi = 0; phi < 3; ++phi)
        if (o->fuse_mask & (1u << phi)) p->phi_id[p->n_phi++] = phi;
    p->R = 0;
    for (uint32_t i = 0; i < p->n_phi; ++i)
        p->R += (uint64_t)p->n_orders * (p->phi_id[i] == 0 ? 3125u : 625u);
    if (p->T > UINT64_MAX / (p->R * 9)) return MO_ERR_OVERFLOW;
    p->N = p->T * p->R * 9;

    p->t_begin = o->t_begin; p->t_end = o->t_end;
    if (p->t_begin == 0 && p->t_end == 0) p->t_end = p->T;
    if (p->t_begin > p->t_end || p->t_end > p->T) return MO_ERR_ARG;

    int rc;
    p->quantum_pj = a->energy_quantum_pj;
    if ((rc = quantise(a->e_dram_pj, a->energy_quantum_pj, &p->cq_dram))) return rc;
    if ((rc = quantise(a->e_gb_pj, a->energy_quantum_pj, &p->cq_gb))) return rc;
    if ((rc = quantise(a->e_rf_pj, a->energy_quantum_pj, &p->cq_rf))) return rc;
    if ((rc = quantise(a->e_mac_pj, a->energy_quantum_pj, &p->cq_mac))) return rc;
    /* softmax: c_softmax MAC-energies per element of S (Section V-D). */
    if ((rc = quantise(a->c_softmax * a->e_mac_pj, a->energy_quantum_pj, &p->cq_sfu))) return rc;
    p->has_rf = a->rf_bytes > 0;
    if (p->has_rf && a->rf_bytes < 6ull * w->word_bytes) return MO_ERR_ARG;
    p->cap_words = a->gb_bytes / w->word_bytes;
    p->pe_rows = a->pe_rows; p->pe_cols = a->pe_cols; p->n_arrays = a->n_arrays;
    p->bw = a->dram_words_per_cycle;
    p->objective = o->objective; p->topk = o->topk;
    p->stationary_mask = o->stationary_mask ? o->stationary_mask : 0x1ffu;
    p->rf_tiling = o->rf_tiling;
    p->rf_words = a->rf_bytes / w->word_bytes;

    /* Worst-case key bound.  With M = I*L*J*(K+1) >= the largest MAC count (recomputation factor
     * at most J): every DRAM term is at most I*K*L*J <= M and there are at most 7 of them; array
     * traffic is at most 4 words per MAC plus the carried partial sums, BR <= 5M; cycles <= M. */
    i128 M = (i128)p->dim[LP_I] * p->dim[LP_L] * p->dim[LP_J] * (p->dim[LP_K] + 1);
    i128 emax = M * (7 * (i128)p->cq_dram + 12 * (i128)p->cq_gb + 8 * (i128)p->cq_rf
                     + (i128)p->cq_mac + (i128)p->cq_sfu);
    i128 lmax = M * (7 + (i128)p->bw);
    if (emax >= ((i128)1 << 62) || lmax >= ((i128)1 << 62)) return MO_ERR_OVERFLOW;
    return MO_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* per-candidate evaluation                                                                    */
/* ------------------------------------------------------------------------------------------ */

typedef struct {
    int lev[8];          /* lev[v] = loop at level v, v = 4..7                               */
    int present[8];      /* level takes part in the nest the operand is evaluated in         */
} nest_t;

/* Operand buffer words: tile footprint times the bounds of the operand's own loops at and
 * below its buffering level (Section V-B, first definition). */
static i128 buffer_words(int x, int beta, const nest_t* n, const uint64_t* dD, i128 tile)
{
    i128 bs = tile;
    for (int v = 4; v <= beta; ++v)
        if (n->present[v] && is_own(x, n->lev[v])) bs *= dD[n->lev[v]];
    return bs;
}

/* Scenario 1 (Section V-C): blocker = innermost loop above the buffering level that is one of
 * the operand's own dimensions; DA = BS * bound(blocker) * bounds of effective dims above it. */
static i128 dram_words_own_blocker(int x, int beta, i128 bs, const nest_t* n, const uint64_t* dD,
                                   const int eff[4])
{
    int blocker = 0;
    for (int v = beta + 1; v <= 7; ++v) {
        if (!n->present[v]) continue;
        if (is_own(x, n->lev[v])) { blocker = v; break; }
    }
    if (!blocker) return bs;                     /* whole operand resident: fetched once */
    i128 da = bs * dD[n->lev[blocker]];
    for (int u = blocker + 1; u <= 7; ++u)
        if (n->present[u] && eff[n->lev[u]]) da *= dD[n->lev[u]];
    return da;
}

/* Array-level terms for one tile (m x r) * (r x n) on a rows x cols array. */
static i128 tile_cycles(int sm, uint64_t m, uint64_t r, uint64_t n, uint64_t rows, uint64_t cols)
{
    switch (sm) {
    case SM_WS: return (i128)ceil_div(r, rows) * ceil_div(n, cols) * m;
    case SM_IS: return (i128)ceil_div(m, rows) * ceil_div(r, cols) * n;
    default:    return (i128)ceil_div(m, rows) * ceil_div(n, cols) * r;
    }
}

static i128 tile_buffer_traffic(int sm, uint64_t m, uint64_t r, uint64_t n, uint64_t rows, uint64_t cols)
{
    switch (sm) {
    case SM_WS:   /* weights once; inputs per column fold; outputs read+written per row fold */
        return (i128)r * n + (i128)m * r * ceil_div(n, cols) + (i128)m * n * (2 * ceil_div(r, rows) - 1);
    case SM_IS:
        return (i128)m * r + (i128)r * n * ceil_div(m, rows) + (i128)m * n * (2 * ceil_div(r, cols) - 1);
    default:      /* outputs stay in the array; both inputs re-streamed per fold */
        return (i128)m * r * ceil_div(n, cols) + (i128)r * n * ceil_div(m, rows) + (i128)m * n;
    }
}

/* Register-file-level tiling: a tile whose stationary operand is processed in blocks of a x b elements.
 * The block is pinned once (a*b words); every streamed vector passes once per block; partial sums leave the
 * array after every block of the reduction dimension and are read back by the next one. */
static void blocked_tile_terms(int sm, uint64_t m, uint64_t r, uint64_t n, uint64_t rows, uint64_t cols,
                               uint64_t a, uint64_t b, i128* words, i128* cycles)
{
    i128 held = (i128)ceil_div(a, rows) * ceil_div(b, cols);      /* stationary elements per PE */
    switch (sm) {
    case SM_WS:   /* block = a reduction indices x b output columns; the m input rows stream */
        *words = (i128)r * n + (i128)m * r * (n / b) + (i128)m * n * (2 * (r / a) - 1);
        *cycles = (i128)(r / a) * (n / b) * m * held;
        break;
    case SM_IS:   /* block = a output rows x b reduction indices; the n weight columns stream */
        *words = (i128)m * r + (i128)r * n * (m / a) + (i128)m * n * (2 * (r / b) - 1);
        *cycles = (i128)(m / a) * (r / b) * n * held;
        break;
    default:      /* block = a output rows x b output columns; the r reduction steps stream */
        *words = (i128)m * r * (n / b) + (i128)r * n * (m / a) + (i128)m * n;
        *cycles = (i128)(m / a) * (n / b) * r * held;
        break;
    }
}

int mo_rf_block(uint32_t objective, uint32_t sm, uint32_t m, uint32_t r, uint32_t n, uint32_t rows, uint32_t cols,
                uint64_t rf_words, uint32_t block_mrn[3], int64_t* words, int64_t* cycles)
{
    if (sm > 2 || !m || !r || !n || !rows || !cols || !block_mrn || !words || !cycles) return MO_ERR_ARG;
    uint64_t ea = sm == SM_WS ? r : m;                   /* extents of the stationary operand */
    uint64_t eb = sm == SM_WS ? n : (sm == SM_IS ? r : n);
    int have = 0;
    i128 best_w = 0, best_c = 0;
    uint64_t best_a = 0, best_b = 0;
    for (uint64_t a = 1; a <= ea; ++a) {
        if (ea % a) continue;
        for (uint64_t b = 1; b <= eb; ++b) {
            if (eb % b) continue;
            if ((i128)ceil_div(a, rows) * ceil_div(b, cols) + 2 > (i128)rf_words) continue;
            i128 w, c;
            blocked_tile_terms((int)sm, m, r, n, rows, cols, a, b, &w, &c);
            int better;
            if (!have) better = 1;
            else if (objective == MO_OBJ_LATENCY) better = c < best_c || (c == best_c && w < best_w);
            else better = w < best_w || (w == best_w && c < best_c);
            if (better) { have = 1; best_w = w; best_c = c; best_a = a; best_b = b; }
        }
    }
    if (!have || !fits64(best_w) || !fits64(best_c)) return MO_ERR_ARG;
    block_mrn[0] = sm == SM_WS ? 1u : (uint32_t)best_a;
    block_mrn[1] = sm == SM_WS ? (uint32_t)best_a : (sm == SM_IS ? (uint32_t)best_b : 1u);
    block_mrn[2] = sm == SM_IS ? 1u : (uint32_t)best_b;
    *words = (int64_t)best_w;
    *cycles = (int64_t)best_c;
    return MO_OK;
}

static int decode(const mo_problem* p, uint64_t idx, mo_record* o)
{
    if (idx >= p->N) return MO_ERR_ARG;
    memset(o, 0, sizeof(*o));
    o->idx = idx;
    uint64_t per_t = p->R * 9;
    uint64_t t = idx / per_t, rem = idx % per_t;
    uint32_t r = (uint32_t)(rem / 9), s = (uint32_t)(rem % 9);
    o->t = t; o->row = r;
    o->sm[0] = s / 3; o->sm[1] = s % 3;

    /* tiling: mixed radix over the ascending divisor lists, j fastest */
    uint32_t a[4];
    uint64_t tt = t;
    for (int d = 3; d >= 0; --d) { a[d] = (uint32_t)(tt % p->ndiv[d]); tt /= p->ndiv[d]; }
    for (int d = 0; d < 4; ++d) {
        uint32_t xg = p->divs[d][a[d]];
        o->bound[4 + d] = xg;
        o->bound[d] = (uint32_t)(p->dim[d] / xg);
    }

    /* row: the fused block first (if present), then one block per unfused mode */
    uint64_t fused_rows = (p->n_phi && p->phi_id[0] == 0) ? (uint64_t)p->n_orders * 3125u : 0;
    if (r < fused_rows) {
        uint32_t q = r % 3125u;
        o->phi = 0;
        o->pi = p->order_id[r / 3125u];
        o->beta[OPD_A] = 3 + q / 625u;
        o->beta[OPD_B] = 3 + (q / 125u) % 5u;
        o->beta[OPD_C] = 3 + (q / 25u) % 5u;
        o->beta[OPD_D] = 3 + (q / 5u) % 5u;
        o->beta[OPD_E] = 3 + q % 5u;
    } else {
        uint32_t r2 = (uint32_t)(r - fused_rows);
        uint32_t blk = p->n_orders * 625u;
        uint32_t which = r2 / blk + (fused_rows ? 1u : 0u);
        uint32_t q = r2 % blk;
        o->phi = p->phi_id[which];
        o->pi = p->order_id[q / 625u];
        q %= 625u;
        o->beta[OPD_A] = 3 + q / 125u;
        o->beta[OPD_B] = 3 + (q / 25u) % 5u;
        o->beta[OPD_C] = 3;
        o->beta[OPD_D] = 3 + (q / 5u) % 5u;
        o->beta[OPD_E] = 3 + q % 5u;
    }
    return MO_OK;
}

int mo_eval(const mo_problem* p, uint64_t idx, mo_record* o)
{
    int rc = decode(p, idx, o);
    if (rc) return rc;

    uint64_t dD[4], g[4];
    for (int d = 0; d < 4; ++d) { dD[d] = o->bound[d]; g[d] = o->bound[4 + d]; }
    const uint64_t I = p->dim[LP_I], K = p->dim[LP_K], L = p->dim[LP_L], J = p->dim[LP_J];

    i128 tile[5];
    for (int x = 0; x < 5; ++x) tile[x] = (i128)g[OWN[x][0]] * g[OWN[x][1]];

    nest_t fused;
    memset(&fused, 0, sizeof(fused));
    fused.lev[4] = LP_K;
    fused.lev[5] = ORDERS[o->pi][2];
    fused.lev[6] = ORDERS[o->pi][1];
    fused.lev[7] = ORDERS[o->pi][0];
    for (int v = 4; v <= 7; ++v) fused.present[v] = 1;

    i128 bs[5], da[5] = {0, 0, 0, 0, 0};
    i128 da_sm = 0, da1 = 0, da2 = 0, bs1, bs2;
    uint64_t rho = 1;
    int rc_flag = 0;

    if (o->phi == 0) {
        for (int x = 0; x < 5; ++x) bs[x] = buffer_words(x, (int)o->beta[x], &fused, dD, tile[x]);

        /* Recomputation (Section III-C): the intermediate tile is evicted and regenerated when
         * the consumer-only loop j2 iterates outside the loop that replaces C's buffered data. */
        int c_blocker = 0;
        for (int v = (int)o->beta[OPD_C] + 1; v <= 7; ++v)
            if (fused.lev[v] == LP_I || fused.lev[v] == LP_L) { c_blocker = v; break; }
        if (c_blocker)
            for (int u = c_blocker + 1; u <= 7; ++u)
                if (fused.lev[u] == LP_J) rc_flag = 1;
        if (rc_flag) rho = dD[LP_J];

        /* Effective dimensions (Section V-A): producer operands see the consumer's j2 only
         * under recomputation; consumer operands see every loop of the fused nest. */
        int eff_p[4] = {1, 1, 1, rc_flag};
        int eff_c[4] = {1, 0, 1, 1};

        for (int x = 0; x < 5; ++x) {
            if (x == OPD_C) { da[x] = 0; continue; }          /* DA_C = 0 when fused */
            int consumer = (x == OPD_D || x == OPD_E);
            if (consumer && o->beta[x] == 3) {
                /* Scenario 2: blocker is the producer's reduction loop k2 (L4); its bound is
                 * excluded; L5..L7 are all effective for a consumer operand. */
                da[x] = bs[x] * dD[LP_I] * dD[LP_L] * dD[LP_J];
            } else {
                da[x] = dram_words_own_blocker(x, (int)o->beta[x], bs[x], &fused, dD,
                                               consumer ? eff_c : eff_p);
            }
        }
        int tau[5];
        for (int x = 0; x < 5; ++x) tau[x] = o->beta[x] >= 4;
        /* Eq. (1), (2), (4) */
        bs1 = bs[OPD_A] + bs[OPD_B] + bs[OPD_C] + tau[OPD_D] * bs[OPD_D] + tau[OPD_E] * bs[OPD_E];
        bs2 = bs[OPD_C] + bs[OPD_D] + bs[OPD_E] + tau[OPD_A] * bs[OPD_A] + tau[OPD_B] * bs[OPD_B];
    } else {
        /* Unfused: each operator runs its own nest; C is written by Op1 and read back by Op2.
         * Nest 1 = k2 innermost, then i2 and l2 in the order's relative order; nest 2 = the
         * order's three loops.  Levels keep their fused numbers; absent levels are skipped. */
        nest_t n1 = fused, n2 = fused;
        for (int v = 4; v <= 7; ++v) n1.present[v] = (fused.lev[v] != LP_J);
        n2.present[4] = 0;
        int eff1[4] = {1, 1, 1, 0};
        int eff2[4] = {1, 0, 1, 1};
        for (int x = 0; x < 5; ++x) {
            const nest_t* n = (x == OPD_A || x == OPD_B) ? &n1 : &n2;
            bs[x] = buffer_words(x, (int)o->beta[x], n, dD, tile[x]);
        }
        da[OPD_A] = dram_words_own_blocker(OPD_A, (int)o->beta[OPD_A], bs[OPD_A], &n1, dD, eff1);
        da[OPD_B] = dram_words_own_blocker(OPD_B, (int)o->beta[OPD_B], bs[OPD_B], &n1, dD, eff1);
        da[OPD_D] = dram_words_own_blocker(OPD_D, (int)o->beta[OPD_D], bs[OPD_D], &n2, dD, eff2);
        da[OPD_E] = dram_words_own_blocker(OPD_E, (int)o->beta[OPD_E], bs[OPD_E], &n2, dD, eff2);
        i128 da_cw = (i128)I * L;
        i128 da_cr = dram_words_own_blocker(OPD_C, 3, bs[OPD_C], &n2, dD, eff2);
        da[OPD_C] = da_cw + da_cr;
        if (o->phi == 2) da_sm = 2 * (i128)I * L;          /* softmax pass: read S, write P */
        bs1 = bs[OPD_A] + bs[OPD_B] + bs[OPD_C];
        bs2 = bs[OPD_C] + bs[OPD_D] + bs[OPD_E];
        da1 = da[OPD_A] + da[OPD_B] + da_cw;
        da2 = da_cr + da[OPD_D] + da[OPD_E];
    }
    i128 bsmax = bs1 > bs2 ? bs1 : bs2;
    i128 n_dram = da[0] + da[1] + da[2] + da[3] + da[4] + da_sm;

    /* MACs and softmax elements (Section V-D) */
    i128 n_mac = (i128)rho * I * K * L + (i128)I * L * J;
    i128 n_sfu = (i128)rho * I * L;

    /* Array-level traffic and cycles: tile invocations times per-tile terms, plus the partial
     * sums carried between consecutive reduction steps of the same output tile. */
    i128 t1 = (i128)rho * dD[LP_I] * dD[LP_K] * dD[LP_L];
    i128 t2 = (i128)dD[LP_I] * dD[LP_L] * dD[LP_J];
    i128 carry1 = (t1 - t1 / dD[LP_K]) * g[LP_I] * g[LP_L];
    i128 carry2 = (t2 - t2 / dD[LP_L]) * g[LP_I] * g[LP_J];
    i128 w1, w2, c1t, c2t;                  /* buffer<->array words and cycles of one tile of each operator */
    if (p->rf_tiling) {
        /* third tiling level: the register-file block of each operator's tile, picked by the objective */
        int64_t bw_, bc_;
        if (mo_rf_block(p->objective, o->sm[0], (uint32_t)g[LP_I], (uint32_t)g[LP_K], (uint32_t)g[LP_L],
                        p->pe_rows, p->pe_cols, p->rf_words, &o->rf_block[0], &bw_, &bc_)) return MO_ERR_ARG;
        w1 = bw_; c1t = bc_;
        if (mo_rf_block(p->objective, o->sm[1], (uint32_t)g[LP_I], (uint32_t)g[LP_L], (uint32_t)g[LP_J],
                        p->pe_rows, p->pe_cols, p->rf_words, &o->rf_block[3], &bw_, &bc_)) return MO_ERR_ARG;
        w2 = bw_; c2t = bc_;
    } else {
        w1 = tile_buffer_traffic((int)o->sm[0], g[LP_I], g[LP_K], g[LP_L], p->pe_rows, p->pe_cols);
        w2 = tile_buffer_traffic((int)o->sm[1], g[LP_I], g[LP_L], g[LP_J], p->pe_rows, p->pe_cols);
        c1t = tile_cycles((int)o->sm[0], g[LP_I], g[LP_K], g[LP_L], p->pe_rows, p->pe_cols);
        c2t = tile_cycles((int)o->sm[1], g[LP_I], g[LP_L], g[LP_J], p->pe_rows, p->pe_cols);
    }
    i128 br = t1 * w1 + carry1 + t2 * w2 + carry2;
    i128 cyc1 = t1 * c1t;
    i128 cyc2 = t2 * c2t;

    i128 n_gb = n_dram + br;
    i128 n_rf = p->has_rf ? br + 3 * n_mac : 0;

    i128 e_key = (i128)p->cq_dram * n_dram + (i128)p->cq_gb * n_gb + (i128)p->cq_rf * n_rf
               + (i128)p->cq_mac * n_mac + (i128)p->cq_sfu * n_sfu;

    /* Latency (Section V-D): loads, compute and stores fully pipelined => max of DRAM time and
     * compute time; kept in words (= cycles * words-per-cycle) so that it stays an integer. */
    i128 l_key;
    if (o->phi == 0) {
        i128 comp = (cyc1 + cyc2) * p->bw;
        l_key = n_dram > comp ? n_dram : comp;
    } else {
        i128 c1 = cyc1 * p->bw, c2 = cyc2 * p->bw;
        l_key = (da1 > c1 ? da1 : c1) + da_sm + (da2 > c2 ? da2 : c2);
    }

    i128 all[] = {bs[0], bs[1], bs[2], bs[3], bs[4], bs1, bs2, da[0], da[1], da[2], da[3], da[4],
                  da_sm, n_dram, br, cyc1, cyc2, n_gb, n_rf, n_mac, n_sfu, e_key, l_key};
    for (unsigned i = 0; i < sizeof(all) / sizeof(all[0]); ++i)
        if (!fits64(all[i])) return MO_ERR_OVERFLOW;

    for (int x = 0; x < 5; ++x) { o->bs_x[x] = (int64_t)bs[x]; o->da_x[x] = (int64_t)da[x]; }
    o->bs_op1 = (int64_t)bs1; o->bs_op2 = (int64_t)bs2; o->bs = (int64_t)bsmax;
    o->da_sm = (int64_t)da_sm; o->da1 = (int64_t)da1; o->da2 = (int64_t)da2;
    o->br = (int64_t)br; o->cyc1 = (int64_t)cyc1; o->cyc2 = (int64_t)cyc2;
    o->n[0] = (int64_t)n_dram; o->n[1] = (int64_t)n_gb; o->n[2] = (int64_t)n_rf;
    o->n[3] = (int64_t)n_mac;  o->n[4] = (int64_t)n_sfu;
    o->e_key = (int64_t)e_key; o->l_key = (int64_t)l_key;
    o->recompute = (uint32_t)rc_flag;
    /* in the space iff it fits the buffer (Eq. 4) and the array offers its stationary pair (Section VII-K) */
    o->feasible = bsmax <= (i128)p->cap_words && ((p->stationary_mask >> (3u * o->sm[0] + o->sm[1])) & 1u);

    volatile double ek = (double)o->e_key, lk = (double)o->l_key;   /* one IEEE multiply, no FMA */
    o->edp_key = ek * lk;
    o->energy_pj = (double)o->e_key * p->quantum_pj * (double)p->instances;
    o->latency_cycles = (double)o->l_key / (double)p->bw
                      * (double)ceil_div(p->instances, p->n_arrays);
    return MO_OK;
}

int mo_eval_range(const mo_problem* p, uint64_t begin, uint64_t count, mo_record* out)
{
    for (uint64_t i = 0; i < count; ++i) {
        int rc = mo_eval(p, begin + i, &out[i]);
        if (rc) return rc;
    }
    return MO_OK;
}

static int64_t order_key(const mo_problem* p, const mo_record* r)
{
    if (p->objective == MO_OBJ_ENERGY) return r->e_key;
    if (p->objective == MO_OBJ_LATENCY) return r->l_key;
    int64_t bits;                       /* positive doubles order like their bit patterns */
    memcpy(&bits, &r->edp_key, sizeof(bits));
    return bits;
}

int mo_keys_range(const mo_problem* p, uint64_t begin, uint64_t count, int64_t* keys, uint8_t* feasible)
{
    int err = MO_OK;
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < (int64_t)count; ++i) {
        mo_record r;
        int rc = mo_eval(p, begin + (uint64_t)i, &r);
        if (rc) { err = rc; continue; }
        keys[i] = order_key(p, &r);
        feasible[i] = (uint8_t)r.feasible;
    }
    return err;
}

/* ------------------------------------------------------------------------------------------ */
/* exhaustive search: k smallest (key, idx) among feasible candidates                          */
/* ------------------------------------------------------------------------------------------ */

typedef struct { int64_t key; uint64_t idx; } pair_t;

static int pair_less(pair_t a, pair_t b) { return a.key < b.key || (a.key == b.key && a.idx < b.idx); }

static void topk_insert(pair_t* list, uint32_t* n, uint32_t k, pair_t c)
{
    if (*n == k && !pair_less(c, list[k - 1])) return;
    uint32_t pos = (*n < k) ? (*n)++ : k - 1;
    while (pos > 0 && pair_less(c, list[pos - 1])) { list[pos] = list[pos - 1]; --pos; }
    list[pos] = c;
}

int mo_threads_used(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

int mo_search(const mo_problem* p, mo_record* out_topk, uint64_t* n_total, uint64_t* n_feasible,
              uint32_t* n_found, int n_threads)
{
    const uint32_t k = p->topk;
    const uint64_t begin = p->t_begin * p->R * 9, end = p->t_end * p->R * 9;
    int nt = n_threads > 0 ? n_threads : mo_threads_used();
    pair_t* lists = (pair_t*)calloc((size_t)nt * k, sizeof(pair_t));
    uint32_t* counts = (uint32_t*)calloc((size_t)nt, sizeof(uint32_t));
    uint64_t* feas = (uint64_t*)calloc((size_t)nt, sizeof(uint64_t));
    int err = MO_OK;
    if (!lists || !counts || !feas) { free(lists); free(counts); free(feas); return MO_ERR_ARG; }

#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        int me = omp_get_thread_num(), team = omp_get_num_threads();
#else
        int me = 0, team = 1;
#endif
        uint64_t span = end - begin;
        uint64_t lo = begin + span / (uint64_t)team * (uint64_t)me;
        uint64_t hi = (me == team - 1) ? end : begin + span / (uint64_t)team * (uint64_t)(me + 1);
        pair_t* mine = lists + (size_t)me * k;
        uint32_t cnt = 0; uint64_t nf = 0;
        for (uint64_t idx = lo; idx < hi; ++idx) {
            mo_record r;
            int rc = mo_eval(p, idx, &r);
            if (rc) { err = rc; break; }
            if (!r.feasible) continue;
            ++nf;
            pair_t c = {order_key(p, &r), idx};
            topk_insert(mine, &cnt, k, c);
        }
        counts[me] = cnt; feas[me] = nf;
    }

    pair_t best[MO_MAX_TOPK]; uint32_t nb = 0; uint64_t nf = 0;
    for (int t = 0; t < nt; ++t) {
        nf += feas[t];
        for (uint32_t i = 0; i < counts[t]; ++i) topk_insert(best, &nb, k, lists[(size_t)t * k + i]);
    }
    for (uint32_t i = 0; i < k; ++i) {
        if (i < nb) { int rc = mo_eval(p, best[i].idx, &out_topk[i]); if (rc) err = rc; }
        else { memset(&out_topk[i], 0, sizeof(mo_record)); out_topk[i].idx = UINT64_MAX; }
    }
    if (n_total) *n_total = end - begin;
    if (n_feasible) *n_feasible = nf;
    if (n_found) *n_found = nb;
    free(lists); free(counts); free(feas);
    return err;
}

/* ------------------------------------------------------------------------------------------ */
/* symbolic rows and offline pruning (Section VI-B)                                            */
/* ------------------------------------------------------------------------------------------ */
/*
 * The same rules as in mo_eval, with "multiply by a bound" replaced by "add the bound to a set":
 * a monomial in the loop bounds with exponents 0/1 is the set of bounds it contains (the query
 * vector of Section V-E).
 */
static uint8_t sym_buffer(int x, int beta, const nest_t* n)
{
    uint8_t q = (uint8_t)((1u << (4 + OWN[x][0])) | (1u << (4 + OWN[x][1])));   /* the tile: both x_G */
    for (int v = 4; v <= beta; ++v)
        if (n->present[v] && is_own(x, n->lev[v])) q |= (uint8_t)(1u << n->lev[v]);
    return q;
}

static uint8_t sym_dram_own_blocker(int x, int beta, uint8_t bs, const nest_t* n, const int eff[4])
{
    int blocker = 0;
    for (int v = beta + 1; v <= 7; ++v) {
        if (!n->present[v]) continue;
        if (is_own(x, n->lev[v])) { blocker = v; break; }
    }
    if (!blocker) return bs;
    uint8_t q = (uint8_t)(bs | (1u << n->lev[blocker]));
    for (int u = blocker + 1; u <= 7; ++u)
        if (n->present[u] && eff[n->lev[u]]) q |= (uint8_t)(1u << n->lev[u]);
    return q;
}

int mo_row_symbolic(uint32_t pi, const uint32_t beta[5], mo_row_symbols* o)
{
    if (pi > 5 || !beta || !o) return MO_ERR_ARG;
    for (int x = 0; x < 5; ++x) if (beta[x] < 3 || beta[x] > 7) return MO_ERR_ARG;
    memset(o, 0, sizeof(*o));
    nest_t fused;
    memset(&fused, 0, sizeof(fused));
    fused.lev[4] = LP_K;
    fused.lev[5] = ORDERS[pi][2];
    fused.lev[6] = ORDERS[pi][1];
    fused.lev[7] = ORDERS[pi][0];
    for (int v = 4; v <= 7; ++v) fused.present[v] = 1;
    for (int x = 0; x < 5; ++x) {
        o->bs_q[x] = sym_buffer(x, (int)beta[x], &fused);
        o->tau[x] = beta[x] >= 4;
    }
    int c_blocker = 0, rc = 0;
    for (int v = (int)beta[OPD_C] + 1; v <= 7; ++v)
        if (fused.lev[v] == LP_I || fused.lev[v] == LP_L) { c_blocker = v; break; }
    if (c_blocker)
        for (int u = c_blocker + 1; u <= 7; ++u)
            if (fused.lev[u] == LP_J) rc = 1;
    o->recompute = (uint8_t)rc;
    int eff_p[4] = {1, 1, 1, rc};
    int eff_c[4] = {1, 0, 1, 1};
    for (int x = 0; x < 5; ++x) {
        if (x == OPD_C) continue;
        int consumer = (x == OPD_D || x == OPD_E);
        if (consumer && beta[x] == 3)
            o->da_q[x] = (uint8_t)(o->bs_q[x] | (1u << LP_I) | (1u << LP_L) | (1u << LP_J));
        else
            o->da_q[x] = sym_dram_own_blocker(x, (int)beta[x], o->bs_q[x], &fused, consumer ? eff_c : eff_p);
    }
    return MO_OK;
}

/* A sum of monomials, each a set of bounds (all bounds are integers >= 1). */
typedef struct { int n; uint8_t term[6]; } sym_sum;

/* P >= Q for every assignment of the bounds if the terms of Q can be matched one-to-one into
 * terms of P with term_Q a subset of term_P (a product over a superset of bounds >= 1 is not
 * smaller).  This is the tiling-independent comparison of Section VI-B. */
static int match_terms(const sym_sum* p, const sym_sum* q, int qi, unsigned used)
{
    if (qi == q->n) return 1;
    for (int i = 0; i < p->n; ++i) {
        if (used & (1u << i)) continue;
        if ((q->term[qi] & p->term[i]) != q->term[qi]) continue;
        if (match_terms(p, q, qi + 1, used | (1u << i))) return 1;
    }
    return 0;
}
static int sum_ge(const sym_sum* p, const sym_sum* q) { return q->n <= p->n && match_terms(p, q, 0, 0); }
/* "greater" in the paper's symbolic sense (i_G k_G < i_G k_G i_D): >= and not also <=. */
static int sum_gt(const sym_sum* p, const sym_sum* q) { return sum_ge(p, q) && !sum_ge(q, p); }

typedef struct { sym_sum bs1, bs2, da; int rc; } sym_row;

static void sym_row_build(uint32_t pi, const uint32_t beta[5], sym_row* r)
{
    mo_row_symbols s;
    mo_row_symbolic(pi, beta, &s);
    r->rc = s.recompute;
    /* Eq. (1), (2): retained operands of the other operator count */
    r->bs1.n = 0; r->bs2.n = 0; r->da.n = 0;
    r->bs1.term[r->bs1.n++] = s.bs_q[OPD_A]; r->bs1.term[r->bs1.n++] = s.bs_q[OPD_B];
    r->bs1.term[r->bs1.n++] = s.bs_q[OPD_C];
    if (s.tau[OPD_D]) r->bs1.term[r->bs1.n++] = s.bs_q[OPD_D];
    if (s.tau[OPD_E]) r->bs1.term[r->bs1.n++] = s.bs_q[OPD_E];
    r->bs2.term[r->bs2.n++] = s.bs_q[OPD_C]; r->bs2.term[r->bs2.n++] = s.bs_q[OPD_D];
    r->bs2.term[r->bs2.n++] = s.bs_q[OPD_E];
    if (s.tau[OPD_A]) r->bs2.term[r->bs2.n++] = s.bs_q[OPD_A];
    if (s.tau[OPD_B]) r->bs2.term[r->bs2.n++] = s.bs_q[OPD_B];
    r->da.term[r->da.n++] = s.da_q[OPD_A]; r->da.term[r->da.n++] = s.da_q[OPD_B];
    r->da.term[r->da.n++] = s.da_q[OPD_D]; r->da.term[r->da.n++] = s.da_q[OPD_E];
}

/* BS = max(BS1, BS2) (Eq. 4): BS_v >= BS_u when both operator sums are >=; > when, in addition,
 * one of them is >. */
static int bs_ge(const sym_row* v, const sym_row* u) { return sum_ge(&v->bs1, &u->bs1) && sum_ge(&v->bs2, &u->bs2); }
static int bs_gt(const sym_row* v, const sym_row* u)
{
    return bs_ge(v, u) && (sum_gt(&v->bs1, &u->bs1) || sum_gt(&v->bs2, &u->bs2));
}

int mo_symbolic_prune(uint8_t* keep, uint32_t kept_per_group[2], uint32_t rows_per_group[2])
{
    enum { NROWS = 18750 };
    if (!keep || !kept_per_group || !rows_per_group) return MO_ERR_ARG;
    sym_row* rows = (sym_row*)malloc(sizeof(sym_row) * NROWS);
    if (!rows) return MO_ERR_ARG;
    for (uint32_t r = 0; r < NROWS; ++r) {
        uint32_t q = r % 3125u;
        uint32_t beta[5] = {3 + q / 625u, 3 + (q / 125u) % 5u, 3 + (q / 25u) % 5u, 3 + (q / 5u) % 5u, 3 + q % 5u};
        sym_row_build(r / 3125u, beta, &rows[r]);
    }
    kept_per_group[0] = kept_per_group[1] = rows_per_group[0] = rows_per_group[1] = 0;
#pragma omp parallel for schedule(dynamic, 64)
    for (int v = 0; v < NROWS; ++v) {
        int pruned = 0;
        for (int u = 0; u < NROWS && !pruned; ++u) {
            if (u == v || rows[u].rc != rows[v].rc) continue;
            /* Eq. (12): s_v is inferior to s_u */
            if (bs_ge(&rows[v], &rows[u]) && sum_gt(&rows[v].da, &rows[u].da)) pruned = 1;
            else if (bs_gt(&rows[v], &rows[u]) && sum_ge(&rows[v].da, &rows[u].da)) pruned = 1;
        }
        keep[v] = (uint8_t)!pruned;
    }
    for (int v = 0; v < NROWS; ++v) {
        rows_per_group[rows[v].rc]++;
        kept_per_group[rows[v].rc] += keep[v];
    }
    free(rows);
    return MO_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* tile-granular simulator of the fused pseudo nested loop (Section IV)                        */
/* ------------------------------------------------------------------------------------------ */
/*
 * Executes the inter-tile loops in the given order.  For every (i2, l2, j2) point the producer
 * first sweeps k2 to build tile C(i2,l2) unless that tile is still buffered, then (after the
 * softmax stage) the consumer multiplies it into E(i2,j2).  Each operand X keeps one block in
 * the buffer: the tiles indexed by its own loops at levels <= beta_X, for the current values of
 * its own loops above beta_X.  A tile is fetched when it is used and not present; the block is
 * dropped when those outer loop values change.  Operands buffered at L3 (no retention) are also
 * dropped as soon as the other operator runs.  Loads and occupancy are counted at tile
 * granularity; nothing here uses the closed forms above.
 */
typedef struct {
    int valid;
    int64_t ident[2];          /* values of the own loops above the buffering level, else -1 */
    uint8_t* present;          /* bitmap over own0 x own1 tiles                              */
    int64_t count;             /* tiles present                                              */
    int64_t n0, n1;
} sim_block;

static void block_clear(sim_block* b)
{
    memset(b->present, 0, (size_t)(b->n0 * b->n1));
    b->count = 0; b->valid = 0;
}

/* returns 1 if the tile had to be brought in (or produced) */
static int block_touch(sim_block* b, int x, int beta, const int level_of[4], const int64_t val[4])
{
    int64_t id[2];
    for (int q = 0; q < 2; ++q) id[q] = (level_of[OWN[x][q]] > beta) ? val[OWN[x][q]] : -1;
    if (!b->valid || id[0] != b->ident[0] || id[1] != b->ident[1]) {
        block_clear(b);
        b->valid = 1; b->ident[0] = id[0]; b->ident[1] = id[1];
    }
    size_t pos = (size_t)(val[OWN[x][0]] * b->n1 + val[OWN[x][1]]);
    if (b->present[pos]) return 0;
    b->present[pos] = 1; b->count++;
    return 1;
}

static int block_has(const sim_block* b, int x, int beta, const int level_of[4], const int64_t val[4])
{
    if (!b->valid) return 0;
    for (int q = 0; q < 2; ++q) {
        int64_t id = (level_of[OWN[x][q]] > beta) ? val[OWN[x][q]] : -1;
        if (id != b->ident[q]) return 0;
    }
    return b->present[(size_t)(val[OWN[x][0]] * b->n1 + val[OWN[x][1]])];
}

int mo_simulate(const uint32_t bound[8], uint32_t pi, const uint32_t beta[5], mo_sim_out* out)
{
    if (!bound || !beta || !out || pi > 5) return MO_ERR_ARG;
    memset(out, 0, sizeof(*out));
    int64_t dD[4], g[4];
    for (int d = 0; d < 4; ++d) {
        dD[d] = bound[d]; g[d] = bound[4 + d];
        if (dD[d] < 1 || g[d] < 1 || dD[d] > 64) return MO_ERR_ARG;
    }
    for (int x = 0; x < 5; ++x) if (beta[x] < 3 || beta[x] > 7) return MO_ERR_ARG;

    int level_of[4];
    level_of[LP_K] = 4;
    level_of[ORDERS[pi][2]] = 5; level_of[ORDERS[pi][1]] = 6; level_of[ORDERS[pi][0]] = 7;

    sim_block blk[5]; int64_t tile[5];
    for (int x = 0; x < 5; ++x) {
        blk[x].n0 = dD[OWN[x][0]]; blk[x].n1 = dD[OWN[x][1]];
        blk[x].present = (uint8_t*)calloc((size_t)(blk[x].n0 * blk[x].n1), 1);
        blk[x].count = 0; blk[x].valid = 0; blk[x].ident[0] = blk[x].ident[1] = -1;
        tile[x] = g[OWN[x][0]] * g[OWN[x][1]];
    }

#define OCCUPANCY() (blk[0].count * tile[0] + blk[1].count * tile[1] + blk[2].count * tile[2] \
                   + blk[3].count * tile[3] + blk[4].count * tile[4])
#define RECORD(kind, occ) do { if (out->n_trace < 64) { out->trace[out->n_trace] = (occ); \
                                out->trace_kind[out->n_trace++] = (kind); } } while (0)
#define DROP_IF_L3(x) do { if (beta[x] == 3) block_clear(&blk[x]); } while (0)

    int64_t val[4] = {0, 0, 0, 0};
    const int o7 = ORDERS[pi][0], o6 = ORDERS[pi][1], o5 = ORDERS[pi][2];
    for (int64_t a7 = 0; a7 < dD[o7]; ++a7)
    for (int64_t a6 = 0; a6 < dD[o6]; ++a6)
    for (int64_t a5 = 0; a5 < dD[o5]; ++a5) {
        val[o7] = a7; val[o6] = a6; val[o5] = a5;
        if (!block_has(&blk[OPD_C], OPD_C, (int)beta[OPD_C], level_of, val)) {
            out->c_productions++;
            for (int64_t k2 = 0; k2 < dD[LP_K]; ++k2) {             /* producer stage */
                val[LP_K] = k2;
                DROP_IF_L3(OPD_D); DROP_IF_L3(OPD_E);
                out->loads[OPD_A] += block_touch(&blk[OPD_A], OPD_A, (int)beta[OPD_A], level_of, val);
                out->loads[OPD_B] += block_touch(&blk[OPD_B], OPD_B, (int)beta[OPD_B], level_of, val);
                (void)block_touch(&blk[OPD_C], OPD_C, (int)beta[OPD_C], level_of, val);
                int64_t occ = OCCUPANCY();
                if (occ > out->peak_op1) out->peak_op1 = occ;
                out->op1_stages++;
                RECORD(1, occ);
            }
            DROP_IF_L3(OPD_A); DROP_IF_L3(OPD_B);                   /* softmax stage */
            RECORD(2, OCCUPANCY());
        }
        DROP_IF_L3(OPD_A); DROP_IF_L3(OPD_B);                       /* consumer stage */
        out->loads[OPD_D] += block_touch(&blk[OPD_D], OPD_D, (int)beta[OPD_D], level_of, val);
        out->loads[OPD_E] += block_touch(&blk[OPD_E], OPD_E, (int)beta[OPD_E], level_of, val);
        int64_t occ = OCCUPANCY();
        if (occ > out->peak_op2) out->peak_op2 = occ;
        out->op2_stages++;
        RECORD(3, occ);
    }
    out->peak = out->peak_op1 > out->peak_op2 ? out->peak_op1 : out->peak_op2;
    for (int x = 0; x < 5; ++x) { out->loads[x] *= tile[x]; free(blk[x].present); }
    return MO_OK;
#undef OCCUPANCY
#undef RECORD
#undef DROP_IF_L3
}

/* ------------------------------------------------------------------------------------------ */
/* element-level execution of tiles on the PE array (Section V-D: compute latency from the     */
/* array size and its utilisation, buffer<->register traffic by stationary mode)               */
/* ------------------------------------------------------------------------------------------ */
/*
 * The array is rows x cols PEs.  A tile multiplies an (m x r) input block by an (r x n) weight
 * block into an (m x n) output block.  One operand is pinned to the PEs ("stationary"), fold by
 * fold when it is larger than the array; the other two move:
 *   weight stationary : PE(p, q) holds weight (reduction index p, output column q); the m input
 *                       rows stream through, one per cycle; every cycle each active column emits
 *                       one partial sum;
 *   input stationary  : PE(p, q) holds input (output row p, reduction index q); the n weight
 *                       columns stream through; every cycle each active row emits one partial sum;
 *   output stationary : PE(p, q) accumulates output (row p, column q); the r reduction steps
 *                       stream through, each bringing one input per active row and one weight per
 *                       active column; the outputs leave once per fold.
 * Partial sums that leave the array before the reduction is complete are written to the buffer
 * and read back by the fold that continues them.  Every word that crosses the buffer<->array
 * boundary is one register-file access at the PE that takes or gives it; every MAC reads two
 * operand registers and updates one accumulator register.
 */
static uint32_t active(uint32_t total, uint32_t fold, uint32_t width)
{
    uint32_t left = total - fold * width;
    return left < width ? left : width;
}

int mo_array_tile(uint32_t sm, uint32_t m, uint32_t r, uint32_t n, uint32_t rows, uint32_t cols,
                  int resume, mo_array_counts* acc)
{
    if (!acc || sm > 2 || !m || !r || !n || !rows || !cols) return MO_ERR_ARG;
    int64_t cycles = 0, words = 0, macs = 0;
    if (sm == SM_WS) {
        for (uint32_t fr = 0; fr * rows < r; ++fr)            /* folds of the reduction dim over the rows */
        for (uint32_t fc = 0; fc * cols < n; ++fc) {          /* folds of the output columns over the cols */
            uint32_t ar = active(r, fr, rows), ac = active(n, fc, cols);
            for (uint32_t pe = 0; pe < ar * ac; ++pe) ++words;             /* pin this fold's weights */
            for (uint32_t v = 0; v < m; ++v) {                             /* stream the input rows   */
                ++cycles;
                for (uint32_t p = 0; p < ar; ++p) ++words;                 /* one input per active row */
                for (uint32_t pe = 0; pe < ar * ac; ++pe) ++macs;
                for (uint32_t q = 0; q < ac; ++q) {
                    if (fr > 0 || resume) ++words;                         /* partial sum so far, read */
                    ++words;                                               /* partial sum, written     */
                }
            }
        }
    } else if (sm == SM_IS) {
        for (uint32_t fr = 0; fr * rows < m; ++fr)            /* folds of the output rows over the rows   */
        for (uint32_t fc = 0; fc * cols < r; ++fc) {          /* folds of the reduction dim over the cols */
            uint32_t ar = active(m, fr, rows), ac = active(r, fc, cols);
            for (uint32_t pe = 0; pe < ar * ac; ++pe) ++words;             /* pin this fold's inputs */
            for (uint32_t v = 0; v < n; ++v) {                             /* stream the weight columns */
                ++cycles;
                for (uint32_t q = 0; q < ac; ++q) ++words;                 /* one weight per active col */
                for (uint32_t pe = 0; pe < ar * ac; ++pe) ++macs;
                for (uint32_t p = 0; p < ar; ++p) {
                    if (fc > 0 || resume) ++words;
                    ++words;
                }
            }
        }
    } else {
        for (uint32_t fr = 0; fr * rows < m; ++fr)            /* folds of the output rows over the rows    */
        for (uint32_t fc = 0; fc * cols < n; ++fc) {          /* folds of the output columns over the cols */
            uint32_t ar = active(m, fr, rows), ac = active(n, fc, cols);
            if (resume)
                for (uint32_t pe = 0; pe < ar * ac; ++pe) ++words;         /* take the partial outputs in */
            for (uint32_t v = 0; v < r; ++v) {                             /* stream the reduction steps */
                ++cycles;
                for (uint32_t p = 0; p < ar; ++p) ++words;
                for (uint32_t q = 0; q < ac; ++q) ++words;
                for (uint32_t pe = 0; pe < ar * ac; ++pe) ++macs;
            }
            for (uint32_t pe = 0; pe < ar * ac; ++pe) ++words;             /* outputs leave the array */
        }
    }
    acc->cycles += cycles;
    acc->words += words;
    acc->macs += macs;
    acc->rf += words + 3 * macs;
    return MO_OK;
}

int mo_array_chain(const uint32_t bound[8], uint32_t productions, uint32_t sm1, uint32_t sm2,
                   uint32_t rows, uint32_t cols, mo_array_counts out[2])
{
    if (!bound || !out || !productions) return MO_ERR_ARG;
    memset(out, 0, 2 * sizeof(mo_array_counts));
    const uint32_t iD = bound[0], kD = bound[1], lD = bound[2], jD = bound[3];
    const uint32_t iG = bound[4], kG = bound[5], lG = bound[6], jG = bound[7];
    int rc = MO_OK;
    /* Op1: every C tile is accumulated over the k2 steps; the whole of C `productions` times */
    for (uint32_t rep = 0; rep < productions; ++rep)
        for (uint32_t i2 = 0; i2 < iD; ++i2)
            for (uint32_t l2 = 0; l2 < lD; ++l2)
                for (uint32_t k2 = 0; k2 < kD; ++k2)
                    if ((rc = mo_array_tile(sm1, iG, kG, lG, rows, cols, k2 > 0, &out[0]))) return rc;
    /* Op2: every E tile is accumulated over the l2 steps */
    for (uint32_t i2 = 0; i2 < iD; ++i2)
        for (uint32_t j2 = 0; j2 < jD; ++j2)
            for (uint32_t l2 = 0; l2 < lD; ++l2)
                if ((rc = mo_array_tile(sm2, iG, lG, jG, rows, cols, l2 > 0, &out[1]))) return rc;
    return MO_OK;
}

/* ------------------------------------------------------------------------------------------ */
/* tile-granular simulator of the two unfused loop nests                                       */
/* ------------------------------------------------------------------------------------------ */
/*
 * Without fusion each operator is mapped on its own (the "no fusion" baseline of Section VII-C):
 * the producer runs its whole nest and stores every finished C tile, an optional separate pass
 * applies the softmax to C in DRAM, then the consumer runs its nest and reads C back.  Buffer
 * blocks behave as in mo_simulate: an operand keeps the tiles of its own loops at levels <= beta
 * for the current values of its own loops above beta.
 */
int mo_simulate_unfused(const uint32_t bound[8], uint32_t pi, const uint32_t beta[5], uint32_t phi,
                        mo_sim_unfused_out* out)
{
    if (!bound || !beta || !out || pi > 5 || phi < 1 || phi > 2) return MO_ERR_ARG;
    memset(out, 0, sizeof(*out));
    int64_t dD[4], g[4];
    for (int d = 0; d < 4; ++d) {
        dD[d] = bound[d]; g[d] = bound[4 + d];
        if (dD[d] < 1 || g[d] < 1 || dD[d] > 64) return MO_ERR_ARG;
    }
    for (int x = 0; x < 5; ++x) if (beta[x] < 3 || beta[x] > 7) return MO_ERR_ARG;
    if (beta[OPD_C] != 3) return MO_ERR_ARG;      /* the intermediate is not retained across the two nests */

    int level_of[4];
    level_of[LP_K] = 4;
    level_of[ORDERS[pi][2]] = 5; level_of[ORDERS[pi][1]] = 6; level_of[ORDERS[pi][0]] = 7;

    sim_block blk[5]; int64_t tile[5];
    for (int x = 0; x < 5; ++x) {
        blk[x].n0 = dD[OWN[x][0]]; blk[x].n1 = dD[OWN[x][1]];
        blk[x].present = (uint8_t*)calloc((size_t)(blk[x].n0 * blk[x].n1), 1);
        blk[x].count = 0; blk[x].valid = 0; blk[x].ident[0] = blk[x].ident[1] = -1;
        tile[x] = g[OWN[x][0]] * g[OWN[x][1]];
    }
    int64_t val[4] = {0, 0, 0, 0};

    /* producer nest: i2 and l2 in the order's relative order, k2 innermost */
    int outer1 = -1, inner1 = -1;
    for (int q = 0; q < 3; ++q) {
        int lp = ORDERS[pi][q];
        if (lp == LP_J) continue;
        if (outer1 < 0) outer1 = lp; else inner1 = lp;
    }
    for (int64_t a = 0; a < dD[outer1]; ++a)
    for (int64_t b = 0; b < dD[inner1]; ++b) {
        val[outer1] = a; val[inner1] = b;
        for (int64_t k2 = 0; k2 < dD[LP_K]; ++k2) {
            val[LP_K] = k2;
            out->loads[OPD_A] += block_touch(&blk[OPD_A], OPD_A, (int)beta[OPD_A], level_of, val);
            out->loads[OPD_B] += block_touch(&blk[OPD_B], OPD_B, (int)beta[OPD_B], level_of, val);
            (void)block_touch(&blk[OPD_C], OPD_C, 3, level_of, val);
            int64_t occ = blk[OPD_A].count * tile[OPD_A] + blk[OPD_B].count * tile[OPD_B]
                        + blk[OPD_C].count * tile[OPD_C];
            if (occ > out->peak_op1) out->peak_op1 = occ;
            out->op1_stages++;
        }
        out->c_stores += tile[OPD_C];              /* the finished tile goes to DRAM */
    }
    block_clear(&blk[OPD_C]);

    /* separate softmax pass: every C tile is read and written once more */
    if (phi == 2)
        for (int64_t a = 0; a < dD[LP_I]; ++a)
            for (int64_t b = 0; b < dD[LP_L]; ++b)
                out->softmax_words += 2 * tile[OPD_C];

    /* consumer nest: the order's three loops */
    const int o7 = ORDERS[pi][0], o6 = ORDERS[pi][1], o5 = ORDERS[pi][2];
    val[LP_K] = 0;
    for (int64_t a7 = 0; a7 < dD[o7]; ++a7)
    for (int64_t a6 = 0; a6 < dD[o6]; ++a6)
    for (int64_t a5 = 0; a5 < dD[o5]; ++a5) {
        val[o7] = a7; val[o6] = a6; val[o5] = a5;
        out->loads[OPD_C] += block_touch(&blk[OPD_C], OPD_C, 3, level_of, val);
        out->loads[OPD_D] += block_touch(&blk[OPD_D], OPD_D, (int)beta[OPD_D], level_of, val);
        out->loads[OPD_E] += block_touch(&blk[OPD_E], OPD_E, (int)beta[OPD_E], level_of, val);
        int64_t occ = blk[OPD_C].count * tile[OPD_C] + blk[OPD_D].count * tile[OPD_D]
                    + blk[OPD_E].count * tile[OPD_E];
        if (occ > out->peak_op2) out->peak_op2 = occ;
        out->op2_stages++;
    }
    for (int x = 0; x < 5; ++x) { out->loads[x] *= tile[x]; free(blk[x].present); }
    return MO_OK;
}

/* One tile with register-file-level blocks (see mmee_oracle.h), executed block by block, element by element. */
int mo_array_tile_blocked(uint32_t sm, uint32_t m, uint32_t r, uint32_t n, uint32_t rows, uint32_t cols,
                          uint32_t a, uint32_t b, int resume, mo_array_counts* acc)
{
    if (!acc || sm > 2 || !m || !r || !n || !rows || !cols || !a || !b) return MO_ERR_ARG;
    const uint32_t ea = sm == SM_WS ? r : m;                   /* extents of the stationary operand */
    const uint32_t eb = sm == SM_WS ? n : (sm == SM_IS ? r : n);
    const uint32_t stream = sm == SM_WS ? m : (sm == SM_IS ? n : r);
    if (ea % a || eb % b) return MO_ERR_ARG;
    /* how many elements of a block each PE holds: element (x, y) lives in PE (x mod rows, y mod cols) */
    uint32_t* held = (uint32_t*)calloc((size_t)rows * cols, sizeof(uint32_t));
    if (!held) return MO_ERR_ARG;
    uint32_t busiest = 0;
    for (uint32_t x = 0; x < a; ++x)
        for (uint32_t y = 0; y < b; ++y) {
            uint32_t c = ++held[(size_t)(x % rows) * cols + (y % cols)];
            if (c > busiest) busiest = c;
        }
    free(held);
    int64_t cycles = 0, words = 0, macs = 0;
    for (uint32_t ba = 0; ba * a < ea; ++ba)
    for (uint32_t bb = 0; bb * b < eb; ++bb) {
        /* the reduction dimension is the first block index under weight stationary, the second under input
         * stationary; output stationary keeps the whole reduction inside one block */
        const int continues = sm == SM_WS ? (ba > 0) : (sm == SM_IS ? (bb > 0) : 0);
        if (sm != SM_OS)
            for (uint32_t e = 0; e < a * b; ++e) ++words;                      /* pin the block */
        else if (resume)
            for (uint32_t e = 0; e < a * b; ++e) ++words;                      /* take the partial outputs in */
        for (uint32_t v = 0; v < stream; ++v) {
            for (uint32_t c = 0; c < busiest; ++c) ++cycles;                   /* one cycle per element of the busiest PE */
            for (uint32_t e = 0; e < a * b; ++e) ++macs;
            if (sm == SM_WS) {
                for (uint32_t x = 0; x < a; ++x) ++words;                      /* the input row's a elements */
                for (uint32_t y = 0; y < b; ++y) { if (continues || resume) ++words; ++words; }
            } else if (sm == SM_IS) {
                for (uint32_t y = 0; y < b; ++y) ++words;                      /* the weight column's b elements */
                for (uint32_t x = 0; x < a; ++x) { if (continues || resume) ++words; ++words; }
            } else {
                for (uint32_t x = 0; x < a; ++x) ++words;
                for (uint32_t y = 0; y < b; ++y) ++words;
            }
        }
        if (sm == SM_OS)
            for (uint32_t e = 0; e < a * b; ++e) ++words;                      /* outputs leave the array */
    }
    acc->cycles += cycles;
    acc->words += words;
    acc->macs += macs;
    acc->rf += words + 3 * macs;
    return MO_OK;
}
