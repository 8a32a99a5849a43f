// The search kernels: exhaustive evaluation of every mapping, capacity pruning, top-k.
//
// Work decomposition.  A "task" is one (tiling, fusion mode, order, levels of A and B) choice: 1125
// consecutive candidate indices, idx = task*1125 + mid*225 + row*9 + s, where mid is the level of C
// (of B for an unfused task), the 25 rows are the levels of D and E and s is the stationary pair.
// One thread owns one task at a time and walks it in ascending index order.
//
// The cost of a mapping is separable over operands (Section V-B/V-C: BS and DA are sums of
// per-operand monomials; Section V-D: energy is linear in the access counts), so the query-matrix
// product exp(Q . ln B) (Eq. 11) is evaluated once per (tiling, order, operand, level) into small
// shared-memory tables -- each entry an exact integer monomial already multiplied by its energy
// coefficient -- and a candidate's key is a short sum of table entries.  The least key of the nine
// mappings of a row (one per stationary pair) is the row's sum plus the least stationary-pair term,
// which is taken once per tiling: the row loop tests one key per row, relative to the current top-k
// threshold in saturated 32-bit arithmetic (a single-precision product bound for the energy-delay
// objective); exact 64-bit keys of single mappings are formed only for groups of rows that can enter
// the list.  Nothing per candidate ever touches global memory.
//
// CTAs are persistent and pull ranges of tasks from a global counter.  All warps build the tables
// of a CTA's first range together; after that seven warps walk tasks while the eighth builds the
// tables of the next range into a second buffer and then joins them.  The CTA that finishes last
// (a ticket counter, no wait) merges the CTAs' partial lists and evaluates the winners in full.
#include <cuda_runtime.h>

#include <climits>
#include <cstddef>
#include <mutex>
#include <type_traits>

#include "mmee_eval.cuh"
#include "mmee_search.h"

namespace mmee {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kModeSearch = 0, kModeDump = 1, kModePrune = 2, kModeFlags = 3;
constexpr size_t kPlanBytes = (sizeof(Plan) + 15) / 16 * 16;
static_assert(sizeof(Plan) % 4 == 0, "the plan is copied word by word");
constexpr int kTermCap = (1 << 28) - 1;    // cap of each non-negative addend of such a sum (at most six of them)
constexpr int kSizeCap = (1 << 30) - 1;    // buffer sizes saturate here; the capacity is smaller
constexpr int kUnfit = 1 << 30;            // added to the keys of a row that does not fit; also the lower clamp of a row sum
constexpr int kRowCap = (1 << 29) - 1;     // upper cap of a row sum: kRowCap + 2 * kTermCap + kUnfit < 2^31

// ------------------------------------------------------------------------------------------------
// shared-memory tables
// ------------------------------------------------------------------------------------------------

// Row-side terms (levels of D and E) of one (tiling, order).  One instance for fused rows, one for unfused rows,
// so that the loops need no selects.  Per level: g = DRAM words times the objective's scale (energy: quanta per
// DRAM word; latency / EDP: 1), exact; and the 32-bit forms x1 = buffer words counted while Op1 runs (the
// operand's size if it is retained, else 0), x2 = buffer words while Op2 runs, both saturated to kSizeCap (which
// is above every admissible capacity, so "fits" has the same truth value as with the exact size), then g in
// relative units saturated to kTermCap and an unused word (EDP: single-precision lower bounds of the DRAM words
// and of their energy).  The energy of the DRAM words, where an objective needs both sides, is g times the cost
// of a DRAM word: it is formed where it is needed, not stored.
struct alignas(16) RowTab {
    int64_t Dg[5], Eg[5];
    int32_t Dc[5][4];
    int32_t Ec[5][4];
};

// Per (tiling, order): task-side terms (levels of A, B, C) and the two row tables.
struct alignas(16) OrderTab {
    int64_t gA[5][2], gB[5][2];                   // [level][recompute]: DRAM term, exact
    int64_t gCr;                                  // unfused: C read back by Op2
    int32_t gXc[2];                               // energy: C round trip (+ softmax pass) of an unfused task, phi = 1, 2
                                                  // (EDP: [0] = single-precision lower bound of gCr)
    // 32-bit forms: per level x1 = size, x2 = size if retained (from L4 upwards), both saturated to kSizeCap;
    // g[recompute] = DRAM term in relative units saturated to kTermCap (EDP: single-precision lower bounds)
    int32_t Ac[5][4];
    int32_t Bc[5][4];
    int32_t Cc[5][2];                             // size, recompute flag
    int32_t pad[2];
    RowTab rt[2];                                 // 0 fused, 1 unfused
};
static_assert(offsetof(OrderTab, Ac) % 16 == 0 && offsetof(OrderTab, Bc) % 16 == 0 && offsetof(OrderTab, Cc) % 8 == 0,
              "Ac / Bc rows are read as int4, Cc rows as int2");
// 26 items per order: 5 levels each of A, B, C, D, E and the unfused C read-back

// Per tiling: array-level terms by stationary pair and recompute flag.
struct alignas(16) TilingTab {
    uint32_t b[8];
    int64_t half[2][16];    // products of every subset of the four x_D bounds / of the four x_G bounds
    int64_t W[9][2];        // energy of buffer<->PE traffic, MACs and softmax, in quanta
    int64_t CB[9][2];       // fused compute time in words (cycles * words per cycle)
    int64_t QU[9][2];       // unfused Op2 compute time in words, by s (sm2 = s % 3)
    int64_t opw[2][3];      // buffer<->array words of one tile of each operator, by stationary mode
    int64_t opc[2][3];      // compute cycles of one tile of each operator, by stationary mode
    int64_t C1w[3];         // unfused Op1 compute time in words, by sm1
    int64_t cw, smx;        // C write-back words (I*L); separate softmax pass words (2*I*L)
    int64_t wmin[2];        // min over the stationary pairs of W[.][rc]
    int64_t qmin[3];        // min over the stationary pairs of CB[.][0], CB[.][1], QU[.][0]
    int32_t Qrel[3][12];    // CB[s][0], CB[s][1], QU[s][0] minus that minimum, saturated to kTermCap (kUnfit: pair not offered);
                            // entries 9..11: the least of the three entries of each sm1
    int64_t c1min;          // least C1w over the sm1 that have an offered pair
    int32_t live;           // smallest possible buffer need of this tiling fits
    int32_t pad[1];
    // energy-delay search: single-precision lower bounds (rounded down) of wmin[0], wmin[1], qmin[0], qmin[1],
    // qmin[2], the least of C1w[0..2], cw and smx
    float fl[8];
};
static_assert(offsetof(TilingTab, Qrel) % 16 == 0 && sizeof(int32_t[12]) % 16 == 0, "Qrel rows are read as int4");
static_assert(offsetof(TilingTab, fl) % 16 == 0, "fl is read as two float4");
static_assert(offsetof(RowTab, Ec) % 16 == 0 && offsetof(OrderTab, rt) % 16 == 0 && sizeof(RowTab) % 16 == 0,
              "Ec rows are read as int4");
// 21 items per tiling: 9 stationary pairs x 2 recompute flags, 3 unfused Op1 terms

// One warp's k best (key, idx) pairs, best first.  A pair is one 16-byte word, read and written whole.
struct alignas(16) WarpTop {
    longlong2 e[MMEE_MAX_TOPK];      // x = key, y = idx
    int32_t count;
    int32_t pad[3];
};
__device__ __forceinline__ int64_t top_key(const WarpTop* w, int j) { return w->e[j].x; }
__device__ __forceinline__ uint64_t top_idx(const WarpTop* w, int j) { return (uint64_t)w->e[j].y; }
__device__ __forceinline__ void top_set(WarpTop* w, int j, int64_t key, uint64_t idx) {
    w->e[j] = make_longlong2((long long)key, (long long)idx);
}

struct alignas(16) CtaShared {
    long long G;             // upper bound on the final k-th smallest key (any full list's last key)
    unsigned long long feasible_rows;
    unsigned long long exact_visits;         // groups that some warp of this CTA took to the exact path
    unsigned long long tested_rows;          // rows whose capacity test and bound were evaluated
    unsigned long long range_begin[2];       // first task of the range whose tables sit in buffer 0 / 1
    unsigned long long range_end[2];         // one past its last task
    unsigned int cursor[2];                  // next unassigned task of that range, relative to its begin
    unsigned int last_cta;                   // this CTA drew the last ticket: it runs the finalize step
    unsigned int check_failed;               // finalize step: a winner's key is not the key of its evaluation
};

__device__ __forceinline__ bool pair_less(int64_t ka, uint64_t ia, int64_t kb, uint64_t ib) {
    return ka < kb || (ka == kb && ia < ib);
}

// All 32 lanes call this converged.  Lane j holds list entry j.
__device__ __forceinline__ bool warp_insert(WarpTop* wt, int k, int64_t nk, uint64_t ni, int lane) {
    const int count = wt->count;
    const bool have = lane < count;
    const longlong2 mine = have ? wt->e[lane] : make_longlong2(kInfKey, -1ll);
    const int64_t ek = mine.x;
    const uint64_t ei = (uint64_t)mine.y;
    const unsigned smaller = __ballot_sync(kFull, have && pair_less(ek, ei, nk, ni));
    const int pos = __popc(smaller);
    if (pos >= k) return false;
    __syncwarp();
    if (have && lane >= pos && lane + 1 < k) top_set(wt, lane + 1, ek, ei);
    if (lane == pos) top_set(wt, pos, nk, ni);
    if (lane == 0 && count < k) wt->count = count + 1;
    __syncwarp();
    return true;
}

// A sorted list held by a warp in registers: lane j holds entry j, best first; an empty slot, and every lane
// from k on, holds (kInfKey, UINT64_MAX), which follows every mapping in the (key, idx) order.  All 32 lanes call
// this converged.
__device__ __forceinline__ bool reg_insert(int64_t& ek, uint64_t& ei, int k, int64_t nk, uint64_t ni, int lane) {
    const unsigned smaller = __ballot_sync(kFull, pair_less(ek, ei, nk, ni));
    const int pos = __popc(smaller);
    if (pos >= k) return false;
    const int64_t uk = __shfl_up_sync(kFull, ek, 1);
    const uint64_t ui = __shfl_up_sync(kFull, ei, 1);
    if (lane == pos) { ek = nk; ei = ni; }
    else if (lane > pos && lane < k) { ek = uk; ei = ui; }
    return true;
}

// Merge of two such lists (both sorted, (kInfKey, UINT64_MAX) in every unused lane): the k smallest pairs of
// both, sorted, stay in (ek, ei).  The other list reversed and the lane-wise minimum of the two give the 16
// smallest of the 32 pairs as a bitonic sequence, which four compare-exchange stages sort.  All 32 lanes call
// this converged.  Cheaper than insertion one by one when the other list is long.
__device__ __forceinline__ void reg_merge(int64_t& ek, uint64_t& ei, int k, int64_t ok, uint64_t oi, int lane) {
    const int rev = (MMEE_MAX_TOPK - 1 - lane) & 31;
    const int64_t rk = __shfl_sync(kFull, ok, rev);
    const uint64_t ri = __shfl_sync(kFull, oi, rev);
    if (lane < (int)MMEE_MAX_TOPK && pair_less(rk, ri, ek, ei)) { ek = rk; ei = ri; }
#pragma unroll
    for (int stride = MMEE_MAX_TOPK / 2; stride >= 1; stride >>= 1) {
        const int64_t pk = __shfl_xor_sync(kFull, ek, stride);
        const uint64_t pi = __shfl_xor_sync(kFull, ei, stride);
        const bool keep_smaller = (lane & stride) == 0;
        if (pair_less(pk, pi, ek, ei) == keep_smaller) { ek = pk; ei = pi; }
    }
    if (lane >= k) { ek = kInfKey; ei = UINT64_MAX; }
}

// Ascending sort of 32 (key, idx) pairs, one per lane (a bitonic network of 15 compare-exchange stages).  All 32
// lanes call this converged.
__device__ __forceinline__ void warp_sort_pairs(int64_t& ck, uint64_t& ci, int lane) {
#pragma unroll
    for (int size = 2; size <= 32; size <<= 1) {
#pragma unroll
        for (int stride = size >> 1; stride >= 1; stride >>= 1) {
            const int64_t pk = __shfl_xor_sync(kFull, ck, stride);
            const uint64_t pi = __shfl_xor_sync(kFull, ci, stride);
            const bool keep_smaller = ((lane & size) == 0) == ((lane & stride) == 0);
            if (pair_less(pk, pi, ck, ci) == keep_smaller) { ck = pk; ci = pi; }
        }
    }
}

// The other list has n entries, lane j holding entry j: by insertion when it is short, else by the merge above.
__device__ __forceinline__ void reg_absorb(int64_t& ek, uint64_t& ei, int k, int n, int64_t ok, uint64_t oi, int lane) {
    if (n > 3) {
        if (lane >= n) { ok = kInfKey; oi = UINT64_MAX; }
        reg_merge(ek, ei, k, ok, oi, lane);
        return;
    }
    for (int j = 0; j < n; ++j) {
        const long long sk = __shfl_sync(kFull, ok, j);
        const uint64_t si = __shfl_sync(kFull, oi, j);
        if (!reg_insert(ek, ei, k, sk, si, lane)) break;   // sorted: the rest is larger
    }
}

// Threshold for candidates whose indices are all >= first_idx: a key passes iff it can still enter
// the warp's list and is not above the CTA-wide bound G.  Strict against the list's last key
// when first_idx lies above that entry's index (a tie could then not displace it).
__device__ __forceinline__ int64_t lane_threshold(const WarpTop* wt, const CtaShared* cs, int k, uint64_t task_first_idx) {
    int64_t thr = cs->G + 1;                       // G <= INT64_MAX - 1 always
    if (wt->count == k) {
        const longlong2 last = wt->e[k - 1];
        const int64_t tk = last.x;
        const int64_t loc = (task_first_idx > (uint64_t)last.y) ? tk : tk + 1;
        thr = loc < thr ? loc : thr;
    }
    return thr;
}

__device__ __forceinline__ int64_t dbits(double v) { return __double_as_longlong(v); }

// x: row sum of the objective's primary side (energy-scaled for the energy objective, DRAM words for
// the others); xe: energy-scaled row sum (objectives that need both sides); w, p, q: stationary-pair
// terms; cap: bound on the other key for the capped objectives (a violating mapping gets kInfKey,
// which never passes a threshold).
template <int OBJ>
__device__ __forceinline__ int64_t candidate_key(int64_t x, int64_t xe, int64_t w, int64_t p, int64_t q, int64_t cap) {
    if constexpr (OBJ == MMEE_OBJ_ENERGY) {
        return x + w;
    } else if constexpr (OBJ == MMEE_OBJ_LATENCY) {
        return p + (x > q ? x : q);
    } else {
        const int64_t e = xe + w;
        const int64_t l = p + (x > q ? x : q);
        if constexpr (OBJ == MMEE_OBJ_EDP) return dbits(__dmul_rn((double)e, (double)l));
        else if constexpr (OBJ == MMEE_OBJ_ENERGY_LCAP) return l <= cap ? e : kInfKey;
        else return e <= cap ? l : kInfKey;
    }
}

// One row: the capacity test of Eq. (4) (e1 <= s1 and e2 <= s2: the two operator buffer sizes
// against their slacks) and one compare per candidate key, OR-ed into one predicate.  Written as
// PTX so that the nine compares against the common threshold stay nine compares: the compiler
// otherwise rewrites (a < t) | (b < t) into min(a, b) < t, and a 64-bit min costs more than the
// compare it saves.  Results as integers: fit = the row fits; hit = it fits and some key < thr.
__device__ __forceinline__ void row_test(const int64_t (&k)[9], int64_t thr, int64_t e1, int64_t s1,
                                         int64_t e2, int64_t s2, unsigned& fit, unsigned& hit) {
    asm("{\n\t"
        ".reg .pred p, q;\n\t"
        "setp.le.s64 q, %12, %13;\n\t"
        "setp.le.and.s64 q, %14, %15, q;\n\t"
        "setp.lt.s64 p, %2, %11;\n\t"
        "setp.lt.or.s64 p, %3, %11, p;\n\t"
        "setp.lt.or.s64 p, %4, %11, p;\n\t"
        "setp.lt.or.s64 p, %5, %11, p;\n\t"
        "setp.lt.or.s64 p, %6, %11, p;\n\t"
        "setp.lt.or.s64 p, %7, %11, p;\n\t"
        "setp.lt.or.s64 p, %8, %11, p;\n\t"
        "setp.lt.or.s64 p, %9, %11, p;\n\t"
        "setp.lt.or.s64 p, %10, %11, p;\n\t"
        "and.pred p, p, q;\n\t"
        "selp.u32 %0, 1, 0, q;\n\t"
        "selp.u32 %1, 1, 0, p;\n\t"
        "}"
        : "=r"(fit), "=r"(hit)
        : "l"(k[0]), "l"(k[1]), "l"(k[2]), "l"(k[3]), "l"(k[4]), "l"(k[5]), "l"(k[6]), "l"(k[7]), "l"(k[8]), "l"(thr),
          "l"(e1), "l"(s1), "l"(e2), "l"(s2));
}

// ------------------------------------------------------------------------------------------------
// 32-bit differential keys
// ------------------------------------------------------------------------------------------------
// Whether a candidate enters the top-k depends only on the sign of key - thr.  The row loops
// therefore evaluate the least key of every row (nine mappings) RELATIVE to the lane's current
// threshold, in saturated 32-bit arithmetic, and keep the minimum over a group of five rows; a
// negative minimum sends the warp to the exact 64-bit path, which re-evaluates the group's 45
// mappings in full.  The filter may flag a group needlessly; it must never miss a candidate that
// passes.
//
// Energy: key = x + W[s], so the row's least key is x + wmin with wmin = min_s W[s] over the offered
// pairs.  With B = thr - wmin:  x + wmin < thr  <=>  (gA + gX - B) + gB + vD + vE < 0, the g / v terms
// being the DRAM energies of the operands at their levels (gX: the C round trip of an unfused task).
// All terms are kept in units of 2^rel_shift quanta (the plan picks the shift from the largest possible
// DRAM term): every addend is rounded down and capped at kTermCap, B is rounded up, so that the 32-bit
// sum is never above the true one.  The task-level part (gA + gX - ceil(B / unit)) is clamped to
// [-kUnfit, kRowCap]; at most three addends of at most kTermCap follow, 3 * kTermCap < kUnfit, so a sum
// that was clamped from below stays negative (the group is flagged, which is the safe side), and no
// 32-bit sum overflows: kRowCap + kTermCap + kUnfit < 2^31.  Most terms are multiples of the unit, so
// that a tie with the list's last entry is still told from a better key: when every index still to be
// walked in a task lies above that entry's, the threshold is thr - 1 (decided at the start of the task
// and after each visit of the exact path).
// Latency: key = P + max(x, Q[s]) (P: the Op1 stage of an unfused task, else 0), and
// max(a, b) < thr  <=>  a - thr < 0 and b - thr < 0.  The row's least key over s has b = qmin (the
// least compute words over the offered pairs; with the least Op1 stage for an unfused task): when
// qmin + P - thr >= 0 no row of the middle level can pass, otherwise only a = (x0 + P - thr) + vD + vE
// decides, with the same units, rounding and clamping (the unit is chosen from the largest DRAM term
// in words).
// Capacity (Eq. 4): sizes are saturated to kSizeCap, which is above every admissible capacity, so
// "size <= slack" keeps its truth value in 32 bits.  A row that does not fit has kUnfit OR-ed into
// its term, which makes its key non-negative whatever the threshold.
// Integer multiply-add and arithmetic shift as single PTX instructions, opaque to the optimiser: the row
// loops use them to keep additions on the FMA pipe and sign masks out of compare-and-select form.
__device__ __forceinline__ int imad(int a, int b, int c) {
    int r;
    asm("mad.lo.s32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
    return r;
}
__device__ __forceinline__ int sign_mask(int a) {       // -1 if a < 0, else 0
    int r;
    asm("shr.s32 %0, %1, 31;" : "=r"(r) : "r"(a));
    return r;
}

__device__ __forceinline__ int sat_s32(int64_t v) {
    int r;
    asm("cvt.sat.s32.s64 %0, %1;" : "=r"(r) : "l"(v));
    return r;
}

// EDP filter for one row on the FP64 pipe: for each of the nine mappings energy = de + dW[s],
// key ~ energy * max(dl[s/3], dQP[s]); max(a, b) * e <= t  <=>  a * e <= t and b * e <= t for e >= 0, so
// each mapping is two multiplies and two compares combined in predicates (a double-precision max or
// min would cost a compare and two selects each).  Returns 1 if the row fits and some product <= thr.
__device__ __forceinline__ unsigned edp_row_test(double de, const double (&dl)[3], const double (&dW)[9],
                                                 const double (&dQP)[9], double thr, unsigned fit) {
    unsigned hit;
#define MMEE_EDP_CAND(w, l, q)                                        \
    "add.f64 e, %2, " w ";\n\t"                                       \
    "mul.f64 a, e, " l ";\n\t"                                        \
    "mul.f64 b, e, " q ";\n\t"                                        \
    "setp.le.f64 r, a, %24;\n\t"                                      \
    "setp.le.and.f64 r, b, %24, r;\n\t"                               \
    "or.pred p, p, r;\n\t"
    asm("{\n\t"
        ".reg .pred p, r, f;\n\t"
        ".reg .f64 e, a, b;\n\t"
        "setp.ne.u32 p, 0, 0;\n\t"
        MMEE_EDP_CAND("%6", "%3", "%15")
        MMEE_EDP_CAND("%7", "%3", "%16")
        MMEE_EDP_CAND("%8", "%3", "%17")
        MMEE_EDP_CAND("%9", "%4", "%18")
        MMEE_EDP_CAND("%10", "%4", "%19")
        MMEE_EDP_CAND("%11", "%4", "%20")
        MMEE_EDP_CAND("%12", "%5", "%21")
        MMEE_EDP_CAND("%13", "%5", "%22")
        MMEE_EDP_CAND("%14", "%5", "%23")
        "setp.ne.u32 f, %1, 0;\n\t"
        "and.pred p, p, f;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t"
        "}"
        : "=r"(hit)
        : "r"(fit), "d"(de), "d"(dl[0]), "d"(dl[1]), "d"(dl[2]),
          "d"(dW[0]), "d"(dW[1]), "d"(dW[2]), "d"(dW[3]), "d"(dW[4]), "d"(dW[5]), "d"(dW[6]), "d"(dW[7]), "d"(dW[8]),
          "d"(dQP[0]), "d"(dQP[1]), "d"(dQP[2]), "d"(dQP[3]), "d"(dQP[4]), "d"(dQP[5]), "d"(dQP[6]), "d"(dQP[7]), "d"(dQP[8]),
          "d"(thr));
#undef MMEE_EDP_CAND
    return hit;
}

// More pending candidates of one position than this are merged into the list in one sorted step (measured with 3, 7,
// 15 and never: 3 is fastest on the top-16 searches).
constexpr int kBulkMin = 3;

// Rare path: some lane of the warp has a key below its threshold in this row.  Every lane
// re-evaluates its nine candidates of the row from the shared tables and the warp inserts the
// passing ones, one at a time, into its sorted list.
template <int OBJ>
__device__ __noinline__ int64_t slow_row(WarpTop* wt, CtaShared* cs, long long* global_g, int k, int lane, bool f,
                                         int64_t x, int64_t xe, const int64_t* wptr, const int64_t* qptr,
                                         int64_t p0, int64_t p1, int64_t p2, int64_t cap, uint32_t sm_mask,
                                         uint64_t row_first_idx) {
    int64_t thr = lane_threshold(wt, cs, k, row_first_idx);
    for (int s = 0; s < 9; ++s) {
        const int64_t pp = s < 3 ? p0 : (s < 6 ? p1 : p2);
        const int64_t key = candidate_key<OBJ>(x, xe, wptr[2 * s], pp, qptr[2 * s], cap);
        bool pend = f && ((sm_mask >> s) & 1u) && key < thr;
        while (true) {
            const unsigned m = __ballot_sync(kFull, pend);
            if (!m) break;
            if (__popc(m) > kBulkMin) {
                // Many lanes at once (an empty list at the start of a search, or mappings tied at the threshold):
                // the pending candidates are sorted across the lanes and merged into the list in one step.
                int64_t ck = pend ? key : kInfKey;
                uint64_t ci = pend ? row_first_idx + (uint64_t)s : UINT64_MAX;
                warp_sort_pairs(ck, ci, lane);
                const int count = wt->count;
                int64_t ek = kInfKey;
                uint64_t ei = UINT64_MAX;
                if (lane < count) {
                    const longlong2 own = wt->e[lane];
                    ek = own.x; ei = (uint64_t)own.y;
                }
                reg_merge(ek, ei, k, ck, ci, lane);
                const int n_new = min(k, count + __popc(m));
                __syncwarp();
                if (lane < n_new) wt->e[lane] = make_longlong2((long long)ek, (long long)ei);
                if (lane == 0) wt->count = n_new;
                __syncwarp();
                thr = lane_threshold(wt, cs, k, row_first_idx);
                break;          // every pending candidate has been considered
            }
            const int leader = __ffs(m) - 1;
            const int64_t lk = __shfl_sync(kFull, key, leader);
            const uint64_t li = __shfl_sync(kFull, row_first_idx + (uint64_t)s, leader);
            warp_insert(wt, k, lk, li, lane);
            thr = lane_threshold(wt, cs, k, row_first_idx);
            pend = (lane == leader) ? false : (pend && key < thr);
        }
    }
    if (lane == 0 && wt->count == k) {
        const long long last = top_key(wt, k - 1);
        if (last < cs->G) {
            atomicMin(&cs->G, last);
            atomicMin(global_g, last);       // other CTAs pick it up at their next task
        }
    }
    __syncwarp();
    return thr;
}

// ------------------------------------------------------------------------------------------------
// table construction
// ------------------------------------------------------------------------------------------------

// Tables of a tiling that cannot fit at all are filled with constants under which no row fits,
// so that lanes whose task lies in such a tiling (they keep step with their warp) read defined data.
__device__ __forceinline__ void fill_dead_order_item(OrderTab* ot, int item) {
    const int l = item % 5;
    if (item < 10) {
        int64_t (*g)[2] = item < 5 ? ot->gA : ot->gB;
        g[l][0] = g[l][1] = 0;
        int32_t* c = item < 5 ? ot->Ac[l] : ot->Bc[l];
        c[0] = c[1] = kSizeCap; c[2] = c[3] = 0;
    } else if (item < 15) {
        ot->Cc[l][0] = kSizeCap; ot->Cc[l][1] = 0;
    } else if (item < 25) {
        for (int v = 0; v < 2; ++v) {
            (item < 20 ? ot->rt[v].Dg : ot->rt[v].Eg)[l] = 0;
            int32_t* c = item < 20 ? ot->rt[v].Dc[l] : ot->rt[v].Ec[l];
            c[0] = c[1] = kSizeCap; c[2] = c[3] = 0;
        }
    } else {
        ot->gCr = 0;
        ot->gXc[0] = ot->gXc[1] = 0;
        ot->pad[0] = ot->pad[1] = 0;
    }
}

__device__ __forceinline__ void fill_dead_tiling_item(struct TilingTab* tb, int item);

// One thread per (tiling slot, order, item): the monomials of one operand at one level.
template <int OBJ>
__device__ __forceinline__ void build_order_item(const Plan& p, const TilingTab* tb, uint32_t order, OrderTab* ot, int item) {
    const QueryTables& q = p.q;
    // exp(q . ln b) (Eq. 8) as the product of two subset products: bits 0-3 of a query vector select
    // x_D bounds, bits 4-7 x_G bounds
    auto monomial = [tb](uint32_t qv) { return tb->half[0][qv & 15u] * tb->half[1][qv >> 4]; };
    const int64_t scale = (OBJ == MMEE_OBJ_ENERGY) ? p.c_dram_gb : 1;
    const int64_t escale = p.c_dram_gb;
    const int l = item % 5;
    // 32-bit forms: a size saturates at kSizeCap (above every admissible capacity); a DRAM term is kept in
    // units of 2^rel_shift, rounded down, and saturates at kTermCap
    auto size32 = [](int64_t v) { return (int32_t)(v < (int64_t)kSizeCap ? v : (int64_t)kSizeCap); };
    auto term32 = [&p](int64_t v) { const int64_t u = v >> p.rel_shift; return (int32_t)(u < (int64_t)kTermCap ? u : (int64_t)kTermCap); };
    if (item < 10) {                                   // A, B
        const int x = item < 5 ? OP_A : OP_B;
        const int64_t bs = monomial(q.bs[order][x][l]);
        const int64_t v0 = monomial(q.da[order][x][l][0]), v1 = monomial(q.da[order][x][l][1]);
        int64_t (*g)[2] = x == OP_A ? ot->gA : ot->gB;
        g[l][0] = scale * v0;
        g[l][1] = scale * v1;
        int32_t* c = x == OP_A ? ot->Ac[l] : ot->Bc[l];
        c[0] = size32(bs);
        c[1] = l ? size32(bs) : 0;                     // retained (tau = 1) from L4 upwards
        c[2] = term32(scale * v0);
        c[3] = term32(scale * v1);
        if constexpr (OBJ == MMEE_OBJ_EDP) {
            // the energy-delay filter's first level: DRAM words as single-precision lower bounds (their energy is
            // the same words times the cost of a DRAM word)
            c[2] = __float_as_int(__ll2float_rd(v0));
            c[3] = __float_as_int(__ll2float_rd(v1));
        }
    } else if (item < 15) {                            // C
        ot->Cc[l][0] = size32(monomial(q.bs[order][OP_C][l]));
        ot->Cc[l][1] = (int32_t)q.recompute[order][l];
    } else if (item < 25) {                            // D, E
        const int x = item < 20 ? OP_D : OP_E;
        const int64_t bs = monomial(q.bs[order][x][l]);
        const int64_t vf = monomial(q.da[order][x][l][0]);
        const int64_t vu = monomial(q.da_unfused[order][x][l]);
        RowTab* f = &ot->rt[0];
        RowTab* u = &ot->rt[1];
        (x == OP_D ? f->Dg : f->Eg)[l] = scale * vf;
        (x == OP_D ? u->Dg : u->Eg)[l] = scale * vu;
        int32_t* fc = x == OP_D ? f->Dc[l] : f->Ec[l];
        int32_t* uc = x == OP_D ? u->Dc[l] : u->Ec[l];
        // fused rows: retained from L4 upwards while Op1 runs; unfused rows take no space while Op1 runs
        fc[0] = l ? size32(bs) : 0; fc[1] = size32(bs); fc[2] = term32(scale * vf); fc[3] = 0;
        uc[0] = 0;                  uc[1] = size32(bs); uc[2] = term32(scale * vu); uc[3] = 0;
        if constexpr (OBJ == MMEE_OBJ_EDP) {
            // the energy-delay filter's first level works on single-precision lower bounds: DRAM words and their
            // energy, each rounded down
            fc[2] = __float_as_int(__ll2float_rd(vf)); fc[3] = __float_as_int(__ll2float_rd(escale * vf));
            uc[2] = __float_as_int(__ll2float_rd(vu)); uc[3] = __float_as_int(__ll2float_rd(escale * vu));
        }
    } else {
        const int64_t v = monomial(q.da_unfused[order][OP_C][0]);
        ot->gCr = scale * v;
        ot->pad[0] = ot->pad[1] = 0;
        // energy of an unfused task's C round trip: read-back, write, and the separate softmax pass of phi = 2
        ot->gXc[0] = term32(p.c_dram_gb * (v + tb->cw));
        ot->gXc[1] = term32(p.c_dram_gb * (v + tb->cw + tb->smx));
        if constexpr (OBJ == MMEE_OBJ_EDP) ot->gXc[0] = __float_as_int(__ll2float_rd(v));
    }
}

// One thread per tiling slot: bounds, liveness, the terms that need no division.
__device__ __forceinline__ void build_tiling_head(const Plan& p, uint64_t t, TilingTab* tb) {
    uint32_t b[8];
    tiling_bounds(p, t, b);
#pragma unroll
    for (int d = 0; d < 8; ++d) tb->b[d] = b[d];
    const int64_t il = (int64_t)p.dim[0] * p.dim[2];
    tb->cw = il;
    tb->smx = 2 * il;
    // With every operand at L3 the buffer need is smallest: max(A+B+C, C+D+E) tiles (Eq. 1-4).
    const int64_t ta = (int64_t)b[4] * b[5], tbb = (int64_t)b[5] * b[6], tc = (int64_t)b[4] * b[6];
    const int64_t td = (int64_t)b[6] * b[7], te = (int64_t)b[4] * b[7];
    const int64_t need1 = ta + tbb + tc, need2 = tc + td + te;
    tb->live = ((need1 > need2 ? need1 : need2) <= p.cap_words) ? 1 : 0;
    tb->pad[0] = 0;
}

// One thread per (tiling slot, operator, stationary mode): words and cycles of one tile (the only part of the
// array-level terms that needs divisions, or the register-file block search).
__device__ __forceinline__ void build_tile_terms(const Plan& p, TilingTab* tb, int item) {
    const int op = item / 3, sm = item % 3;
    uint32_t blk[3];
    tile_array_terms(p, tb->b, op, sm, tb->opw[op][sm], tb->opc[op][sm], blk);
}

// One thread per (tiling slot, item): stationary-pair terms with the cost coefficients applied.
__device__ __forceinline__ void build_tiling_item(const Plan& p, TilingTab* tb, int item) {
    const TilingCounts c = tiling_counts(p, tb->b);
    const int64_t bw = p.bw;
    if (item < 18) {
        const int s = item >> 1, rc = item & 1;
        const int sm1 = s / 3, sm2 = s % 3;
        const int64_t rho = rc ? (int64_t)tb->b[3] : 1;
        const int64_t t1 = rho * c.t1;
        const int64_t br = t1 * tb->opw[0][sm1] + rho * c.carry1 + c.t2 * tb->opw[1][sm2] + c.carry2;
        const int64_t cyc1 = t1 * tb->opc[0][sm1], cyc2 = c.t2 * tb->opc[1][sm2];
        tb->W[s][rc] = p.c_br * br + p.c_mac * (rho * c.ikl + c.ilj) + p.c_sfu * (rho * c.il);
        tb->CB[s][rc] = (cyc1 + cyc2) * bw;
        tb->QU[s][rc] = cyc2 * bw;
    } else {
        const int sm1 = item - 18;
        tb->C1w[sm1] = c.t1 * tb->opc[0][sm1] * bw;
    }
}

__device__ __forceinline__ void fill_dead_tiling_item(TilingTab* tb, int item) {
    if (item < 18) {
        const int s = item >> 1, rc = item & 1;
        tb->W[s][rc] = tb->CB[s][rc] = tb->QU[s][rc] = 0;
    } else {
        tb->C1w[item - 18] = 0;
    }
}

// ------------------------------------------------------------------------------------------------
// walking one task
// ------------------------------------------------------------------------------------------------

// Threshold of one lane: a key passes iff key < T1; for candidates whose index lies above `ti`,
// the index of the list's last entry, the threshold is T1 - delta (a tie could not displace it).
struct LaneThreshold {
    int64_t T1;
    uint64_t ti;
    int delta;
};

__device__ __forceinline__ LaneThreshold load_threshold(const WarpTop* wt, const CtaShared* cs, int k) {
    LaneThreshold t;
    const int64_t g1 = cs->G + 1;                 // G <= INT64_MAX - 1 always
    t.T1 = g1; t.ti = UINT64_MAX; t.delta = 0;
    if (wt->count == k) {
        const longlong2 last = wt->e[k - 1];
        const int64_t tk1 = last.x + 1;
        if (tk1 <= g1) { t.T1 = tk1; t.delta = 1; t.ti = (uint64_t)last.y; }
    }
    return t;
}

// Exact 64-bit terms of one (task, middle level): the middle level m is the level of C for a fused
// task and of B for an unfused one.
struct MidExact {
    int64_t slack1, slack2;     // capacity left for the D and E terms in Op1's / Op2's buffer need (Eq. 1, 2)
    int64_t x0, xe0;            // task-level part of the row sum: the objective's primary side / the energy side
    int64_t P[3];               // unfused latency: Op1 stage and softmax pass, by sm1
    const int64_t* wptr;        // W[s][rc], stride 2
    const int64_t* qptr;        // compute words by s, stride 2
    uint32_t rc;                // C is regenerated (fused tasks)
};

template <int OBJ>
__device__ __forceinline__ MidExact mid_exact(const Plan& p, const TilingTab* tb, const OrderTab* ot, uint32_t phi,
                                              uint32_t la, uint32_t lb_task, int m, bool live) {
    MidExact r;
    const bool fused = phi == 0;
    const uint32_t lb = fused ? lb_task : (uint32_t)m;
    const uint32_t lc = fused ? (uint32_t)m : 0u;
    // Tables of a tiling that cannot fit are filled with constants: a lane whose task lies in such
    // a tiling must not index with what it reads from them.
    const uint32_t rc = (fused && live) ? ((uint32_t)ot->Cc[lc][1] & 1u) : 0u;
    // (sizes saturated to kSizeCap, which is above the capacity: every comparison with a slack keeps its result)
    const int64_t a1 = ot->Ac[la][0], b1 = ot->Bc[lb][0], c1 = ot->Cc[lc][0];
    const int64_t a2 = fused ? ot->Ac[la][1] : 0, b2 = fused ? ot->Bc[lb][1] : 0;
    // Eq. (1)/(2): a retained operand (level >= L4) of the other operator keeps its space.
    // A lane without a live task gets a negative slack, so that none of its rows fits.
    r.slack1 = live ? p.cap_words - (a1 + b1 + c1) : -1;
    r.slack2 = live ? p.cap_words - (c1 + a2 + b2) : -1;
    const int64_t gab = ot->gA[la][rc] + ot->gB[lb][rc];
    r.wptr = &tb->W[0][rc];
    r.rc = rc;
    r.xe0 = 0;
    if constexpr (OBJ == MMEE_OBJ_ENERGY) {
        const int64_t extra = p.c_dram_gb * (tb->cw + (phi == 2 ? tb->smx : 0));
        r.x0 = fused ? gab : gab + ot->gCr + extra;
        r.P[0] = r.P[1] = r.P[2] = 0;
        r.qptr = r.wptr;
    } else {
        const int64_t pass = (phi == 2) ? tb->smx : 0;
        if (fused) {
            r.x0 = gab;
            r.P[0] = r.P[1] = r.P[2] = 0;
            r.qptr = &tb->CB[0][rc];
        } else {
            // unfused latency: max(DA1, C1) + softmax pass + max(DA2, C2)
            r.x0 = ot->gCr;
            const int64_t da1 = gab + tb->cw;
#pragma unroll
            for (int j = 0; j < 3; ++j) r.P[j] = (da1 > tb->C1w[j] ? da1 : tb->C1w[j]) + pass;
            r.qptr = &tb->QU[0][0];
        }
        if constexpr (OBJ >= MMEE_OBJ_EDP) {
            // (for these objectives the g terms are DRAM words; their energy is the words times the cost of one)
            r.xe0 = p.c_dram_gb * (fused ? gab : gab + ot->gCr + tb->cw + pass);
        }
    }
    return r;
}

// Rare path: the filter flagged group d (five rows, the levels of E) of middle level m for some lane.
// Every lane finds its rows that hold a passing candidate, exactly, and the warp inserts them.
template <int OBJ>
__device__ __noinline__ void exact_group(const Plan& p, const TilingTab* tb, const OrderTab* ot, uint32_t phi, uint32_t la,
                                         uint32_t lb_task, int m, int d, uint32_t rows, bool live, uint32_t kept,
                                         uint64_t task_first_idx, WarpTop* wt, CtaShared* cs, long long* global_g, int k,
                                         int lane) {
    // The other CTAs' bound, read afresh: a lane that visits this path with a stale threshold would come back for
    // every group.  The load is consumed at the end of the visit, before the caller renews its threshold.
    const long long g_now = (lane == 0) ? *reinterpret_cast<volatile long long*>(global_g) : 0;
    const MidExact me = mid_exact<OBJ>(p, tb, ot, phi, la, lb_task, m, live);
    const RowTab* rt = &ot->rt[phi == 0 ? 0 : 1];
    const int64_t s1 = me.slack1 - rt->Dc[d][0];
    const int64_t s2 = me.slack2 - rt->Dc[d][1];
    const int64_t xd = me.x0 + rt->Dg[d];
    const int64_t xed = (OBJ >= MMEE_OBJ_EDP) ? me.xe0 + p.c_dram_gb * rt->Dg[d] : 0;
#pragma unroll 1
    for (int e = 0; e < 5; ++e) {
        if (!((rows >> e) & 1u)) continue;      // the filter flagged this row in no lane
        const bool fit = (rt->Ec[e][0] <= s1) && (rt->Ec[e][1] <= s2) && ((kept >> (d * 5 + e)) & 1u);
        const int64_t x = xd + rt->Eg[e];
        const int64_t xe = (OBJ >= MMEE_OBJ_EDP) ? xed + p.c_dram_gb * rt->Eg[e] : 0;
        const uint64_t row_first_idx = task_first_idx + (uint64_t)(m * 225 + (d * 5 + e) * 9);
        const int64_t thr_row = lane_threshold(wt, cs, k, row_first_idx);
        bool below = false;
#pragma unroll
        for (int s = 0; s < 9; ++s)
            below |= ((p.sm_mask >> s) & 1u) &&
                     candidate_key<OBJ>(x, xe, me.wptr[2 * s], me.P[s / 3], me.qptr[2 * s], p.key_cap) < thr_row;
        if (__any_sync(kFull, fit && below))
            slow_row<OBJ>(wt, cs, global_g, k, lane, fit, x, xe, me.wptr, me.qptr, me.P[0], me.P[1], me.P[2], p.key_cap,
                          p.sm_mask, row_first_idx);
    }
    if (lane == 0 && g_now < cs->G) atomicMin(&cs->G, g_now);
    __syncwarp();
}

// The same for a single optimum (k = 1), without the insertion loop: every lane finds the best of its 45
// candidates (ascending index, so the first of equal keys stays), the warp reduces those to the smallest
// (key, idx) pair, and one lane replaces the list's entry if that pair precedes it.
template <int OBJ>
__device__ __noinline__ void exact_group_single(const Plan& p, const TilingTab* tb, const OrderTab* ot, uint32_t phi,
                                                uint32_t la, uint32_t lb_task, int m, int d, uint32_t rows, bool live,
                                                uint32_t kept, uint64_t task_first_idx, WarpTop* wt, CtaShared* cs,
                                                long long* global_g, int lane) {
    // The other CTAs' bound, read afresh: a lane that visits this path with a stale threshold would come back for
    // every group.  The load is consumed at the end of the visit, before the caller renews its threshold.
    const long long g_now = (lane == 0) ? *reinterpret_cast<volatile long long*>(global_g) : 0;
    const MidExact me = mid_exact<OBJ>(p, tb, ot, phi, la, lb_task, m, live);
    const RowTab* rt = &ot->rt[phi == 0 ? 0 : 1];
    const int64_t s1 = me.slack1 - rt->Dc[d][0];
    const int64_t s2 = me.slack2 - rt->Dc[d][1];
    const int64_t xd = me.x0 + rt->Dg[d];
    const int64_t xed = (OBJ >= MMEE_OBJ_EDP) ? me.xe0 + p.c_dram_gb * rt->Dg[d] : 0;
    int64_t best = kInfKey;
    uint32_t best_pos = 0;
#pragma unroll 1
    for (int e = 0; e < 5; ++e) {
        if (!((rows >> e) & 1u)) continue;      // the filter flagged this row in no lane
        const bool fit = (rt->Ec[e][0] <= s1) && (rt->Ec[e][1] <= s2) && ((kept >> (d * 5 + e)) & 1u);
        const int64_t x = xd + rt->Eg[e];
        const int64_t xe = (OBJ >= MMEE_OBJ_EDP) ? xed + p.c_dram_gb * rt->Eg[e] : 0;
#pragma unroll
        for (int s = 0; s < 9; ++s) {
            const int64_t key = candidate_key<OBJ>(x, xe, me.wptr[2 * s], me.P[s / 3], me.qptr[2 * s], p.key_cap);
            if (fit && ((p.sm_mask >> s) & 1u) && key < best) { best = key; best_pos = (uint32_t)(e * 9 + s); }
        }
    }
    uint64_t best_idx = task_first_idx + (uint64_t)(m * 225 + d * 45) + best_pos;
    // a key above the CTA-wide bound cannot be the optimum; an infeasible or capped-out lane holds kInfKey > G
    if (best > cs->G) { best = kInfKey; best_idx = UINT64_MAX; }
    // The smallest (key, idx) pair of the warp by four 32-bit warp minima: the key's high and low words (keys are
    // non-negative), then the index's among the lanes that hold that key.  Every lane ends up with the pair.
    {
        const uint32_t kh = __reduce_min_sync(kFull, (uint32_t)((uint64_t)best >> 32));
        const bool m1 = (uint32_t)((uint64_t)best >> 32) == kh;
        const uint32_t kl = __reduce_min_sync(kFull, m1 ? (uint32_t)best : 0xffffffffu);
        const bool m2 = m1 && (uint32_t)best == kl;
        const uint32_t ih = __reduce_min_sync(kFull, m2 ? (uint32_t)(best_idx >> 32) : 0xffffffffu);
        const bool m3 = m2 && (uint32_t)(best_idx >> 32) == ih;
        const uint32_t il = __reduce_min_sync(kFull, m3 ? (uint32_t)best_idx : 0xffffffffu);
        best = (int64_t)(((uint64_t)kh << 32) | kl);
        best_idx = ((uint64_t)ih << 32) | il;
    }
    if (lane == 0 && best != kInfKey && (wt->count == 0 || pair_less(best, best_idx, top_key(wt, 0), top_idx(wt, 0)))) {
        top_set(wt, 0, best, best_idx);
        wt->count = 1;
        if (best < cs->G) {
            atomicMin(&cs->G, (long long)best);
            atomicMin(global_g, (long long)best);       // other CTAs pick it up at their next task
        }
    }
    if (lane == 0 && g_now < cs->G) atomicMin(&cs->G, g_now);
    __syncwarp();
}

// Second level of the energy-delay filter, for a group whose single-precision bound passed in some lane: every
// mapping of the group's five rows in double precision on the FP64 pipe (energy and latency sums converted once per
// row, then an add, two multiplies and two compares per mapping).  Each approximate product is within a few 2^-53
// of the exact key, so comparing against the threshold widened by 1e-14 relative can flag a row needlessly but never
// miss one; the exact path decides.  Returns the mask of the rows that fit and hold such a product.
__device__ __noinline__ unsigned edp_group_test(const Plan& p, const TilingTab* tb, const OrderTab* ot, uint32_t phi,
                                                uint32_t la, uint32_t lb_task, int m, bool live, int d, int s1c, int s2c,
                                                uint32_t kept_rows, double dthr) {
    // (the 64-bit terms of the middle level are formed again here, so that the caller's row loop need not keep
    // them, in registers or in local memory, for this rare path)
    const MidExact me = mid_exact<MMEE_OBJ_EDP>(p, tb, ot, phi, la, lb_task, m, live);
    const RowTab* rt = &ot->rt[phi == 0 ? 0 : 1];
    const uint32_t sm_mask = p.sm_mask;
    double dW[9], dQP[9];
#pragma unroll
    for (int s = 0; s < 9; ++s) {
        // (a pair the array does not offer: infinite energy, flagged at most while no bound exists yet)
        dW[s] = ((sm_mask >> s) & 1u) ? (double)me.wptr[2 * s] : __longlong_as_double(0x7ff0000000000000ll);
        dQP[s] = (double)(me.qptr[2 * s] + me.P[s / 3]);
    }
    const int64_t xd = me.x0 + rt->Dg[d];
    const int64_t xed = me.xe0 + p.c_dram_gb * rt->Dg[d];
    unsigned hit_any = 0;
#pragma unroll 1
    for (int e = 0; e < 5; ++e) {
        const unsigned fit = (unsigned)(rt->Ec[e][0] <= s1c) & (unsigned)(rt->Ec[e][1] <= s2c) & (kept_rows >> e);   // Eq. (4)
        const int64_t x = xd + rt->Eg[e];
        const double de = (double)(xed + p.c_dram_gb * rt->Eg[e]);
        double dl[3];
#pragma unroll
        for (int j = 0; j < 3; ++j) dl[j] = (double)(x + me.P[j]);
        hit_any |= edp_row_test(de, dl, dW, dQP, dthr, fit & 1u) << e;
    }
    return hit_any;
}

// The walk in 64-bit keys: the energy-delay product (double-precision filter, see edp_row_test),
// the capped objectives and the key dump.  Returns the number of rows that fit.
template <int OBJ, bool DUMP, bool PRUNE, bool FLAGS>
__device__ __forceinline__ uint32_t walk_task_exact(const Plan& p, const TilingTab* tb, const OrderTab* ot,
                                                    const TaskChoice& c, bool live, bool valid, uint32_t kept,
                                                    uint32_t kept_mid, uint64_t task_first_idx, WarpTop* wt,
                                                    CtaShared* cs, long long* global_g, int k, int lane,
                                                    int64_t* __restrict__ dump, uint64_t dump_origin, uint32_t& visits,
                                                    uint32_t& tested, unsigned char* flags) {
    // The energy-delay search sets a middle level up from the 32-bit tables alone (saturated sizes as in the
    // threshold-relative walk, single-precision lower bounds of the DRAM words); the other walks need the exact terms.
    constexpr bool FAST = !DUMP && OBJ == MMEE_OBJ_EDP;
    const bool fused = c.phi == 0;
    const RowTab* rt = &ot->rt[fused ? 0 : 1];
    LaneThreshold th = load_threshold(wt, cs, k);
    if constexpr (FLAGS) { th.T1 = p.key_cap; th.ti = UINT64_MAX; th.delta = 0; }
    uint32_t rows = 0;
    const int4 av = FAST ? *reinterpret_cast<const int4*>(ot->Ac[c.la]) : make_int4(0, 0, 0, 0);
    const int a1c = av.x, a2c = fused ? av.y : 0;
    const int capc = (int)p.cap_words;
    const float cdf = FAST ? __ll2float_rd(p.c_dram_gb) : 0.f;        // cost of a DRAM word, rounded down
    int E1c[5], E2c[5];
    float Egf[5], Eef[5];       // EDP: lower bounds of E's DRAM words and of their energy
#pragma unroll
    for (int e = 0; e < 5; ++e) {
        const int4 v = *reinterpret_cast<const int4*>(rt->Ec[e]);
        E1c[e] = v.x; E2c[e] = v.y;
        Egf[e] = __int_as_float(v.z); Eef[e] = __int_as_float(v.w);
    }
#pragma unroll 1
    for (int mi = 0; mi < (PRUNE ? 1 : 5); ++mi) {
        const int m = PRUNE ? (int)kept_mid : mi;
        const uint64_t mid_first_idx = task_first_idx + (uint64_t)(m * 225);
        MidExact me{};
        int64_t W[9] = {}, Q[9] = {};
        if constexpr (!FAST) {
            me = mid_exact<OBJ>(p, tb, ot, c.phi, c.la, c.lb, m, live);
#pragma unroll
            for (int s = 0; s < 9; ++s) {
                W[s] = me.wptr[2 * s];
                Q[s] = me.qptr[2 * s];
            }
        }
        // Energy-delay product: the first filter level is one single-precision lower bound per row,
        // (row energy + least stationary-pair energy) * max(row DRAM words + least Op1 stage, least compute
        // words + least Op1 stage), every conversion, sum and product rounded down, against the threshold
        // rounded up: no mapping of a row is below its row's bound.
        // All terms are non-negative, so a sum or product of rounded-down terms, itself rounded down, stays a
        // lower bound.  The energy of the task's DRAM words is their number times the cost of a word.
        double dthr = 0.0;
        float fthr = 0.f, fe0 = 0.f, fx0 = 0.f, fq = 0.f;
        int slack1c, slack2c;
        if constexpr (FAST) {
            const int4 bv = *reinterpret_cast<const int4*>(ot->Bc[fused ? c.lb : (uint32_t)m]);
            const int2 cv = *reinterpret_cast<const int2*>(ot->Cc[fused ? m : 0]);
            // (a lane without a live task may read the constant tables of a tiling that cannot fit)
            const uint32_t rc = (fused && live) ? ((uint32_t)cv.y & 1u) : 0u;
            // Eq. (1)/(2) in saturated 32-bit sizes: a retained operand of the other operator keeps its space
            int y1 = __viaddmin_s32(a1c, bv.x, kSizeCap);
            y1 = __viaddmin_s32(y1, cv.x, kSizeCap);
            int y2 = __viaddmin_s32(a2c, fused ? bv.y : 0, kSizeCap);
            y2 = __viaddmin_s32(y2, cv.x, kSizeCap);
            slack1c = live ? max(capc - y1, -1) : -1;       // (a lane without a live task: none of its rows fits)
            slack2c = live ? max(capc - y2, -1) : -1;
            const float4 t0 = *reinterpret_cast<const float4*>(&tb->fl[0]);
            const float4 t1 = *reinterpret_cast<const float4*>(&tb->fl[4]);
            const float fgab = __fadd_rd(__int_as_float(rc ? av.w : av.z), __int_as_float(rc ? bv.w : bv.z));
            if (fused) {
                fx0 = fgab;
                fe0 = __fadd_rd(__fmul_rd(cdf, fgab), rc ? t0.y : t0.x);
                fq = rc ? t0.w : t0.z;
            } else {
                // unfused: least Op1 stage max(DRAM words of A and B + C write-back, least Op1 compute words) plus the
                // softmax pass; the row's DRAM words start from the C read-back
                const float fgcr = __int_as_float(ot->gXc[0]);
                const float fpass = c.phi == 2 ? t1.w : 0.f;
                const float fp = __fadd_rd(fmaxf(__fadd_rd(fgab, t1.z), t1.y), fpass);
                fx0 = __fadd_rd(fgcr, fp);
                fq = __fadd_rd(t1.x, fp);
                fe0 = __fadd_rd(__fmul_rd(cdf, __fadd_rd(__fadd_rd(fgab, fgcr), __fadd_rd(t1.z, fpass))), t0.x);
            }
        } else {
            slack1c = me.slack1 < 0 ? -1 : (int)me.slack1;      // slack <= capacity < 2^30
            slack2c = me.slack2 < 0 ? -1 : (int)me.slack2;
        }
        auto refresh = [&]() {
            if constexpr (OBJ == MMEE_OBJ_EDP) {
                // EDP keys are bit patterns of positive doubles; anything from +inf up means "no bound yet"
                dthr = th.T1 >= 0x7ff0000000000000ll ? __longlong_as_double(0x7ff0000000000000ll)
                                                    : __longlong_as_double(th.T1) * (1.0 + 1e-14);
                fthr = __double2float_ru(dthr);
            }
        };
        refresh();
        if constexpr (FAST) {
            // no lane has room left for D and E at this middle level: none of its 25 rows fits
            if (!__any_sync(kFull, (slack1c | slack2c) >= 0)) continue;
        }
        uint32_t groups_walked = 0;

        // (the energy-delay search's group loop is unrolled: its body is short; the 64-bit walks' is not)
        constexpr int kUnrollGroups = (!DUMP && !PRUNE && OBJ == MMEE_OBJ_EDP) ? 5 : 1;
#pragma unroll kUnrollGroups
        for (int d = 0; d < 5; ++d) {
            if constexpr (PRUNE) {
                if (!__any_sync(kFull, live && ((kept >> (d * 5)) & 31u))) continue;
            }
            unsigned hit_any = 0, fits = 0;
            if constexpr (!DUMP && OBJ == MMEE_OBJ_EDP) {
                const int4 dc = *reinterpret_cast<const int4*>(rt->Dc[d]);
                const int s1c = slack1c - dc.x;
                const int s2c = slack2c - dc.y;
                if (!__any_sync(kFull, (s1c | s2c) >= 0)) continue;     // D leaves no room in any lane
                ++groups_walked;
                const float fxd = __fadd_rd(fx0, __int_as_float(dc.z));
                const float fed = __fadd_rd(fe0, __int_as_float(dc.w));
                const uint32_t kd = PRUNE ? (kept >> (d * 5)) : 31u;
                unsigned hit1 = 0;
#pragma unroll
                for (int e = 0; e < 5; ++e) {
                    unsigned fit = (unsigned)(E1c[e] <= s1c) & (unsigned)(E2c[e] <= s2c);             // Eq. (4)
                    if constexpr (PRUNE) fit &= kd >> e;
                    fits += fit;
                    const float fl = fmaxf(__fadd_rd(fxd, Egf[e]), fq);
                    const float lb = __fmul_rd(__fadd_rd(fed, Eef[e]), fl);
                    hit1 |= fit & (unsigned)(lb <= fthr);
                }
                if (__any_sync(kFull, hit1 != 0u))
                    hit_any = edp_group_test(p, tb, ot, c.phi, c.la, c.lb, m, live, d, s1c, s2c, kd, dthr);
            } else {
                ++groups_walked;
                const int64_t s1 = me.slack1 - rt->Dc[d][0];
                const int64_t s2 = me.slack2 - rt->Dc[d][1];
                const int64_t xd = me.x0 + rt->Dg[d];
                const int64_t xed = (OBJ >= MMEE_OBJ_EDP) ? me.xe0 + p.c_dram_gb * rt->Dg[d] : 0;
                const uint64_t group_first_idx = mid_first_idx + (uint64_t)(d * 45);
                const int64_t thr = th.T1 - (group_first_idx > th.ti ? th.delta : 0);
#pragma unroll
                for (int e = 0; e < 5; ++e) {
                    const int64_t x = xd + rt->Eg[e];
                    const int64_t xe = (OBJ >= MMEE_OBJ_EDP) ? xed + p.c_dram_gb * rt->Eg[e] : 0;
                    int64_t key[9];
#pragma unroll
                    for (int s = 0; s < 9; ++s)
                        key[s] = ((p.sm_mask >> s) & 1u) ? candidate_key<OBJ>(x, xe, W[s], me.P[s / 3], Q[s], p.key_cap) : kInfKey;
                    unsigned fit, hit;
                    row_test(key, thr, (int64_t)rt->Ec[e][0], s1, (int64_t)rt->Ec[e][1], s2, fit, hit);
                    if constexpr (PRUNE) { fit &= kept >> (d * 5 + e); hit &= fit; }
                    fits += fit;
                    hit_any |= hit << e;
                    if (DUMP) {
                        if (valid) {
#pragma unroll
                            for (int s = 0; s < 9; ++s)
                                dump[mid_first_idx - dump_origin + (d * 5 + e) * 9 + s] = fit ? key[s] : kInfKey;
                        }
                    }
                }
            }
            rows += fits;
            if constexpr (FLAGS) {
                if (hit_any && flags) flags[m * 5 + d] = 1;
            } else if (__any_sync(kFull, hit_any != 0u)) {
                ++visits;
                const uint32_t rows = __reduce_or_sync(kFull, hit_any);     // the rows that some lane's filter flags
                if (k == 1) exact_group_single<OBJ>(p, tb, ot, c.phi, c.la, c.lb, m, d, rows, live, kept, task_first_idx, wt, cs, global_g, lane);
                else exact_group<OBJ>(p, tb, ot, c.phi, c.la, c.lb, m, d, rows, live, kept, task_first_idx, wt, cs, global_g, k, lane);
                th = load_threshold(wt, cs, k);
                refresh();
            }
        }
        if (live) tested += groups_walked * 5u;
    }
    return rows;
}

// The walk in 32-bit threshold-relative keys (see "32-bit differential keys"): energy and latency
// objectives.  Everything a middle level, a group or a row needs is a 32-bit table entry or a
// register; 64-bit arithmetic is left to the places where the threshold enters (once per task and
// after each visit of the exact path).  Returns the number of rows that fit.
// FLAGS (a test mode): the threshold is the fixed key p.key_cap, nothing is inserted, and flags[mid * 5 + group]
// is set for every group the filter would send to the exact path.
template <int OBJ, bool PRUNE, bool FLAGS>
__device__ __forceinline__ uint32_t walk_task_relative(const Plan& p, const TilingTab* tb, const OrderTab* ot,
                                                       const TaskChoice& c, bool live, uint32_t kept, uint32_t kept_mid,
                                                       uint64_t task_first_idx, WarpTop* wt, CtaShared* cs,
                                                       long long* global_g, int k, int lane, uint32_t& visits,
                                                       uint32_t& tested, unsigned char* flags) {
    const bool fused = c.phi == 0;
    const RowTab* rt = &ot->rt[fused ? 0 : 1];
    // Row-side terms of E.  Its buffer need while Op1 runs is its size when retained (level >= L4 of a
    // fused task) and 0 otherwise, so that only the size itself has to be kept.
    int E2c[5], Gc[5];
#pragma unroll
    for (int e = 0; e < 5; ++e) {
        const int4 v = *reinterpret_cast<const int4*>(rt->Ec[e]);
        E2c[e] = v.y; Gc[e] = v.z;
    }
    const int4 av = *reinterpret_cast<const int4*>(ot->Ac[c.la]);
    const int a1c = av.x, a2c = fused ? av.y : 0;
    const int capc = (int)p.cap_words;
    // Differences and counts that need no saturation are written x * (-1) + y with a run-time -1: an integer
    // multiply-add runs on the FMA pipe, which is otherwise idle, instead of the integer ALU pipe.
    const int minus_one = -p.unit;
    const int gxc = (OBJ == MMEE_OBJ_ENERGY && !fused) ? ot->gXc[c.phi == 2 ? 1 : 0] : 0;
    // task-level part of key - thr, clamped to [-kUnfit, kRowCap]: clamping from below keeps the sign of every
    // sum that follows (at most 4 * kTermCap < kUnfit is added), clamping from above only lowers
    auto rel32 = [](int64_t v) { const int r = sat_s32(v); return max(min(r, kRowCap), -kUnfit); };

    // Threshold state, set at the start of the task and after each visit of the exact path.  `next_pos` is the
    // position in the task of the first candidate still to be walked: if its index lies above the list's last
    // entry, so do all that follow, a tie cannot displace that entry, and the threshold is T1 - delta.  (Most
    // terms are multiples of the unit, so that a tie is told from a better key even in coarse units.)
    // Energy: base[rc] = (terms of A and of the C round trip) - ceil((thr - wmin[rc]) / 2^rel_shift).
    // Latency, fused task: ua2[rc] = DRAM words of A and B - thr, qo2[rc] = least compute words - thr, in units
    // of 2^rel_shift words rounded down.
    int base[2] = {0, 0}, ua2[2] = {0, 0}, qo2[2] = {0, 0};
    int64_t thr = 0;
    auto rebase = [&](int next_pos) {
        if constexpr (FLAGS) {
            thr = p.key_cap;
        } else {
            const LaneThreshold th = load_threshold(wt, cs, k);
            thr = th.T1 - ((task_first_idx + (uint64_t)next_pos > th.ti) ? th.delta : 0);
        }
        if constexpr (OBJ == MMEE_OBJ_ENERGY) {
#pragma unroll
            for (int rc = 0; rc < 2; ++rc) {
                const int64_t b64 = thr - tb->wmin[rc];
                const int64_t bs = ((b64 - 1) >> p.rel_shift) + 1;                // ceiling of the quotient
                const int64_t bl = bs > (int64_t)INT_MAX ? (int64_t)INT_MAX : (bs < -(int64_t)kTermCap ? -(int64_t)kTermCap : bs);
                const int t = (rc ? av.w : av.z) + gxc - (int)bl;
                base[rc] = max(min(t, kRowCap), -kUnfit);
            }
        } else {
            if (fused) {
#pragma unroll
                for (int rc = 0; rc < 2; ++rc) {
                    ua2[rc] = rel32((ot->gA[c.la][rc] + ot->gB[c.lb][rc] - thr) >> p.rel_shift);
                    qo2[rc] = rel32((tb->qmin[rc] - thr) >> p.rel_shift);
                }
            }
        }
    };
    rebase(0);

    // low half: the number of rows that do not fit; high half: how many of them lay in middle levels and groups
    // that no lane of the warp had room for (their rows were not tested one by one)
    int unfit = 0;
    uint32_t groups = 0;
#pragma unroll 1
    for (int mi = 0; mi < (PRUNE ? 1 : 5); ++mi) {
        const int m = PRUNE ? (int)kept_mid : mi;
        const int4 bv = *reinterpret_cast<const int4*>(ot->Bc[fused ? c.lb : (uint32_t)m]);
        const int2 cv = *reinterpret_cast<const int2*>(ot->Cc[fused ? m : 0]);
        // (a lane without a live task may read the constant tables of a tiling that cannot fit)
        const uint32_t rc = (fused && live) ? ((uint32_t)cv.y & 1u) : 0u;
        // Eq. (1)/(2) in saturated 32-bit sizes: a retained operand of the other operator keeps its space
        int y1 = __viaddmin_s32(a1c, bv.x, kSizeCap);
        y1 = __viaddmin_s32(y1, cv.x, kSizeCap);
        int y2 = __viaddmin_s32(a2c, fused ? bv.y : 0, kSizeCap);
        y2 = __viaddmin_s32(y2, cv.x, kSizeCap);
        // (a lane without a live task: none of its rows fits.)  D and E of an unfused task take no space while
        // Op1 runs: its first slack only has to be non-negative, and is made large so that min(s1, s2) = s2 below.
        const int room1 = capc - y1;
        const int slack1c = live ? (fused ? max(room1, -1) : (room1 >= 0 ? kSizeCap : -1)) : -1;
        const int slack2c = live ? max(capc - y2, -1) : -1;

        // No lane has room left for D and E at this middle level: none of its 25 rows fits.
        if (!__any_sync(kFull, (slack1c | slack2c) >= 0)) {
            if constexpr (!PRUNE) unfit += 25 + (25 << 16);
            continue;
        }

        // u: the part of key - thr that is fixed by (task, middle level), with the least stationary-pair term
        // already inside.  The minimum of a row's nine keys is its row sum plus the least stationary-pair
        // term (energy), or the larger of its DRAM words and the least compute words (latency), so the
        // nine mappings of a row need one test, not nine.  (Redone after a visit of the exact path.)
        int u = 0;
        auto mid_setup = [&]() {
            if constexpr (OBJ == MMEE_OBJ_ENERGY) {
                u = __viaddmin_s32(rc ? base[1] : base[0], rc ? bv.w : bv.z, kRowCap);
            } else {
                // max(x, Q) < thr  <=>  x < thr and Q < thr: when even the least compute words reach the
                // threshold, no row of this middle level passes
                if (fused) {
                    u = (rc ? qo2[1] : qo2[0]) < 0 ? (rc ? ua2[1] : ua2[0]) : kRowCap;
                } else {
                    // unfused latency: max(DA1, C1) + softmax pass + max(DA2, C2); the first two terms are
                    // fixed by (level of A, level of B = m, sm1).  Least Op1 stage over the sm1 the array
                    // offers, least (Op1 stage + Op2 compute words) over the offered pairs.
                    const int64_t da1 = ot->gA[c.la][0] + ot->gB[m][0] + tb->cw;
                    const int64_t pass = c.phi == 2 ? tb->smx : 0;
                    // With the least stage over the offered sm1 (all 32-bit forms are monotone in the stage): the
                    // DRAM-side bound is the least over the sm1, and the compute-side gate a lower bound of every
                    // sm1's.  Only when that gate lets the middle level through are the three sm1 looked at.
                    const int64_t c1m = tb->c1min;
                    const int64_t pm = (da1 > c1m ? da1 : c1m) + pass - thr;
                    u = kRowCap;
                    if (rel32((tb->qmin[2] + pm) >> p.rel_shift) < 0) {
                        const int um = rel32((ot->gCr + pm) >> p.rel_shift);
                        const int4 qr = *reinterpret_cast<const int4*>(&tb->Qrel[2][8]);     // [9..11]: least term by sm1
                        int qm = INT_MAX;
#pragma unroll
                        for (int j = 0; j < 3; ++j) {
                            const int64_t c1w = tb->C1w[j];
                            const int64_t pj = (da1 > c1w ? da1 : c1w) + pass - thr;
                            const int qoj = rel32((tb->qmin[2] + pj) >> p.rel_shift);
                            const int qrj = j == 0 ? qr.y : (j == 1 ? qr.z : qr.w);
                            qm = min(qm, qoj + qrj);
                        }
                        u = qm < 0 ? um : kRowCap;
                    }
                }
            }
        };
        mid_setup();
        // (u is a value from here on: the compiler must not form it again from its inputs in every group)
        asm volatile("" : "+r"(u));

        // The D terms of the five groups are loaded ahead of the group loop: inside it a load could not move above
        // the (rare) calls of the exact path, and each group would wait for its own.
        int4 dcs[5];
#pragma unroll
        for (int d = 0; d < 5; ++d) dcs[d] = *reinterpret_cast<const int4*>(rt->Dc[d]);
#pragma unroll
        for (int d = 0; d < 5; ++d) {
            if constexpr (PRUNE) {
                if (!__any_sync(kFull, live && ((kept >> (d * 5)) & 31u))) continue;
            }
            // Five rows (levels of E) are evaluated branch-free; one vote decides whether any lane of the
            // warp has to enter the exact path for this group.
            const int4 dc = dcs[d];
            const int s1c = imad(dc.x, minus_one, slack1c);
            const int s2c = imad(dc.y, minus_one, slack2c);
            // Eq. (4) for the five levels of E: at L3, and in an unfused task, E takes no space while Op1
            // runs (size <= s2c, given s1c >= 0); retained, it must fit beside both operators' operands
            const int lim_l3 = s1c >= 0 ? s2c : -1;
            const int lim_retained = min(s1c, s2c);
            // D leaves no room in any lane: none of the group's five rows fits
            if (!__any_sync(kFull, lim_l3 >= 0)) {
                if constexpr (!PRUNE) unfit += 5 + (5 << 16);
                continue;
            }
            if constexpr (PRUNE) ++groups;
            const uint32_t kd = kept >> (d * 5);
            const int uc = __viaddmin_s32(u, dc.z, kRowCap);
            int g[5];
#pragma unroll
            for (int e = 0; e < 5; ++e) {
                // t = -1 if the row does not fit (Eq. 4), else 0; such a row's term is moved up by kUnfit,
                // which makes its keys non-negative whatever the threshold
                int t = sign_mask(imad(E2c[e], minus_one, e == 0 ? lim_l3 : lim_retained));
                if constexpr (PRUNE) t |= (int)((kd >> e) & 1u) - 1;
                unfit = imad(t, minus_one, unfit);
                g[e] = Gc[e] | (t & kUnfit);             // (Gc <= kTermCap < kUnfit, a single bit)
            }
            // least key of the group's 45 mappings, relative to the threshold
            const bool hit = uc + __vimin3_s32(__vimin3_s32(g[0], g[1], g[2]), g[3], g[4]) < 0;
            if constexpr (FLAGS) {
                if (hit && flags) flags[m * 5 + d] = 1;
            } else if (__any_sync(kFull, hit)) {
                ++visits;
                // the rows that some lane's bound flags: the exact path looks at no other
                // (the row terms are formed again, through an opaque instruction, so that the five of the common
                // path need not stay in registers for this rare one)
                uint32_t rows = 0;
#pragma unroll
                for (int e = 0; e < 5; ++e) {
                    int t;
                    asm volatile("shr.s32 %0, %1, 31;" : "=r"(t) : "r"(imad(E2c[e], minus_one, e == 0 ? lim_l3 : lim_retained)));
                    if constexpr (PRUNE) t |= (int)((kd >> e) & 1u) - 1;
                    rows |= (uc + (Gc[e] | (t & kUnfit)) < 0) ? (1u << e) : 0u;
                }
                rows = __reduce_or_sync(kFull, rows);
                if (k == 1) exact_group_single<OBJ>(p, tb, ot, c.phi, c.la, c.lb, m, d, rows, live, kept, task_first_idx, wt, cs, global_g, lane);
                else exact_group<OBJ>(p, tb, ot, c.phi, c.la, c.lb, m, d, rows, live, kept, task_first_idx, wt, cs, global_g, k, lane);
                rebase(m * 225 + d * 45 + 45);
                mid_setup();
                asm volatile("" : "+r"(u));
            }
        }
    }
    if constexpr (!PRUNE) groups = 25;
    if (live) tested += groups * 5u - ((uint32_t)unfit >> 16);
    return groups * 5u - ((uint32_t)unfit & 0xffffu);
}

// ------------------------------------------------------------------------------------------------
// finalize: merge the CTAs' partial lists, evaluate the winners in full, reset the scratch header
// ------------------------------------------------------------------------------------------------
// Run by every thread of ONE CTA (the last one to finish its search) after all CTAs have published their
// partial lists.  `tops` is shared memory for one list per warp, `check_failed` a shared flag (zero on entry).
__device__ __noinline__ void finalize_step(const Plan& p, Scratch* __restrict__ scratch, int n_partials,
                                              mmee_result_t* __restrict__ out_best, mmee_result_t* __restrict__ out_topk,
                                              longlong2 (*tops)[MMEE_MAX_TOPK], unsigned int* check_failed) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int kWarps = kSearchThreads / 32;
    const int k = (int)p.topk;
    int64_t ek = kInfKey;
    uint64_t ei = UINT64_MAX;
    // Thread i looks at the length of partial list i (+ a multiple of the CTA size): one round trip to the L2
    // for all lengths.  Most lists are empty, because a CTA publishes only the entries that are not above the
    // bound G it knew at its end.  Each warp then merges the non-empty lists among its 32, eight at a time
    // (lane j takes entry j of each; the loads bypass the L1 cache).
    constexpr int kBatch = 8;
    if (k == 1) {
        // A single optimum: every thread reads the only entry of its lists (all loads in flight at once), and the
        // warp's smallest pair is found by four 32-bit warp minima (key high / low word, index high / low word).
        for (int c = tid; c < n_partials; c += kSearchThreads) {
            if (__ldcg(&scratch->partial[c].count) > 0) {
                const longlong2 head = __ldcg(&scratch->partial[c].e[0]);
                if (pair_less(head.x, (uint64_t)head.y, ek, ei)) { ek = head.x; ei = (uint64_t)head.y; }
            }
        }
        const uint32_t kh = __reduce_min_sync(kFull, (uint32_t)((uint64_t)ek >> 32));
        const bool m1 = (uint32_t)((uint64_t)ek >> 32) == kh;
        const uint32_t kl = __reduce_min_sync(kFull, m1 ? (uint32_t)ek : 0xffffffffu);
        const bool m2 = m1 && (uint32_t)ek == kl;
        const uint32_t ih = __reduce_min_sync(kFull, m2 ? (uint32_t)(ei >> 32) : 0xffffffffu);
        const bool m3 = m2 && (uint32_t)(ei >> 32) == ih;
        const uint32_t il = __reduce_min_sync(kFull, m3 ? (uint32_t)ei : 0xffffffffu);
        // (lane 0 holds the warp's entry, the other lanes the empty pair)
        ek = lane == 0 ? (int64_t)(((uint64_t)kh << 32) | kl) : kInfKey;
        ei = lane == 0 ? (((uint64_t)ih << 32) | il) : UINT64_MAX;
    } else {
        for (int c0 = 0; c0 < n_partials; c0 += kSearchThreads) {
            const int c = c0 + tid;
            const int len = c < n_partials ? __ldcg(&scratch->partial[c].count) : 0;
            unsigned todo = __ballot_sync(kFull, len > 0);
            while (todo) {
                int n[kBatch];
                longlong2 mine[kBatch];
#pragma unroll
                for (int i = 0; i < kBatch; ++i) {
                    n[i] = 0;
                    mine[i] = make_longlong2(kInfKey, -1ll);
                    if (todo) {
                        const int src_lane = __ffs(todo) - 1;
                        todo &= todo - 1;
                        n[i] = __shfl_sync(kFull, len, src_lane);
                        if (lane < n[i]) mine[i] = __ldcg(&scratch->partial[c0 + warp * 32 + src_lane].e[lane]);
                    }
                }
                // (unrolled: with a run-time index the batch would live in local memory, and the store of each
                // loaded entry there would wait for its load before the next load could issue)
#pragma unroll
                for (int i = 0; i < kBatch; ++i) {
                    // a list whose first entry does not precede this warp's k-th entry adds nothing
                    const int64_t kth_key = __shfl_sync(kFull, ek, k - 1), head_key = __shfl_sync(kFull, mine[i].x, 0);
                    const uint64_t kth_idx = __shfl_sync(kFull, ei, k - 1);
                    const uint64_t head_idx = (uint64_t)__shfl_sync(kFull, mine[i].y, 0);
                    if (n[i] > 0 && pair_less(head_key, head_idx, kth_key, kth_idx))
                        reg_absorb(ek, ei, k, n[i], mine[i].x, (uint64_t)mine[i].y, lane);
                }
            }
        }
    }
    // The warps' lists are merged pairwise into warp 0's.
    if (lane < MMEE_MAX_TOPK) tops[warp][lane] = make_longlong2((long long)ek, (long long)ei);
    for (int stride = kWarps / 2; stride >= 1; stride >>= 1) {
        __syncthreads();
        if (warp < stride) {
            const longlong2 theirs = lane < MMEE_MAX_TOPK ? tops[warp + stride][lane] : make_longlong2(kInfKey, -1ll);
            const int n_theirs = __popc(__ballot_sync(kFull, theirs.x != kInfKey || theirs.y != -1ll));
            reg_absorb(ek, ei, k, n_theirs, theirs.x, (uint64_t)theirs.y, lane);
            if (lane < MMEE_MAX_TOPK) tops[warp][lane] = make_longlong2((long long)ek, (long long)ei);
        }
    }
    __syncthreads();
    // Every winner is evaluated in full, one warp per record (the parts of a record on different lanes); the key
    // it was ranked by must be the key of that evaluation.  A mismatch (a list entry whose key and index do not
    // belong together) is reported in out_best->status instead of being returned as a result.
    const longlong2 final_entry = lane < MMEE_MAX_TOPK ? tops[0][lane] : make_longlong2(kInfKey, -1ll);
    const int found = __popc(__ballot_sync(kFull, lane < k && (final_entry.x != kInfKey || final_entry.y != -1ll)));
    mmee_result_t r, first;
    for (int rec = warp; rec < k; rec += kWarps) {
        const long long rk = __shfl_sync(kFull, final_entry.x, rec);
        const uint64_t ri = (uint64_t)__shfl_sync(kFull, final_entry.y, rec);
        if (rec < found) {
            evaluate_candidate_warp(p, ri, lane, r);
            if (lane == 0) {
                int64_t key;
                switch (p.objective) {
                    case MMEE_OBJ_ENERGY: key = r.e_key; break;
                    case MMEE_OBJ_LATENCY: key = r.l_key; break;
                    case MMEE_OBJ_EDP: key = dbits(r.edp_key); break;
                    case MMEE_OBJ_ENERGY_LCAP: key = r.l_key <= p.key_cap ? r.e_key : kInfKey; break;
                    default: key = r.e_key <= p.key_cap ? r.l_key : kInfKey; break;
                }
                if (!(key == rk && r.feasible && r.t >= p.t_begin && r.t < p.t_end)) atomicOr(check_failed, 1u);
            }
        } else if (lane == 0) {
            // empty slot
            unsigned long long* raw = reinterpret_cast<unsigned long long*>(&r);
            for (unsigned i = 0; i < sizeof(r) / 8; ++i) raw[i] = 0;
            r.idx = MMEE_NO_INDEX;
            r.status = found ? MMEE_OK : MMEE_ERR_NO_FEASIBLE;
        }
        if (lane == 0) {
            if (out_topk) out_topk[rec] = r;
            if (rec == 0) first = r;
        }
    }
    __syncthreads();
    if (tid == 0) {
        first.n_total = (p.t_end - p.t_begin) * (uint64_t)p.rows_per_tiling * 9u;
        first.n_feasible = __ldcg(&scratch->feasible_rows) * (uint64_t)p.n_sm;
        if (*check_failed) first.status = MMEE_ERR_CHECK;
        *out_best = first;
        // ready for the next search on this scratch
        scratch->next_task = 0;
        scratch->feasible_rows = 0;
        scratch->G = kInfKey - 1;
        scratch->last_exact_visits = __ldcg(&scratch->exact_visits);
        scratch->exact_visits = 0;
        scratch->last_tested_rows = __ldcg(&scratch->tested_rows);
        scratch->tested_rows = 0;
        scratch->done_ctas = 0;
    }
}

// ------------------------------------------------------------------------------------------------
// the search kernel
// ------------------------------------------------------------------------------------------------

template <int OBJ, int MODE>
__global__ void __launch_bounds__(kSearchThreads, 2)
search_kernel(const __grid_constant__ Plan plan_arg, const LaunchShape shape, Scratch* __restrict__ scratch,
              int64_t* __restrict__ dump, mmee_result_t* __restrict__ out_best, mmee_result_t* __restrict__ out_topk) {
    constexpr bool DUMP = MODE == kModeDump;        // store every key instead of reducing
    constexpr bool PRUNE = MODE == kModePrune;      // visit only the rows kept by symbolic pruning
    constexpr bool FLAGS = MODE == kModeFlags;      // test mode: record which groups the filter flags (in `dump`)
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // The plan is copied to shared memory: lanes index its tables (query vectors, divisor lists,
    // block lists) with different indices, which the constant bank would serialise.
    Plan* plan_sm = reinterpret_cast<Plan*>(smem_raw);
    for (unsigned i = threadIdx.x; i < sizeof(Plan) / 4; i += kSearchThreads)
        reinterpret_cast<uint32_t*>(plan_sm)[i] = reinterpret_cast<const uint32_t*>(&plan_arg)[i];
    const Plan& p = *plan_sm;
    CtaShared* cs = reinterpret_cast<CtaShared*>(smem_raw + kPlanBytes);
    WarpTop* wtops = reinterpret_cast<WarpTop*>(smem_raw + kPlanBytes + sizeof(CtaShared));
    TilingTab* ttabs_all = reinterpret_cast<TilingTab*>(wtops + kSearchThreads / 32);
    OrderTab* otabs_all = reinterpret_cast<OrderTab*>(ttabs_all + 2 * shape.slots);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // (from the kernel argument: the shared copy of the plan is not complete before the barrier below)
    const int k = (int)plan_arg.topk;
    WarpTop* wt = &wtops[warp];
    // The last warp builds the tables of the next range while the other warps walk the tasks of
    // the current one (two table buffers); one barrier per range separates the two.
    const bool builder = warp == kWorkerWarps;

    if (tid == 0) {
        cs->G = scratch->G;
        cs->feasible_rows = 0;
        cs->exact_visits = 0;
        cs->tested_rows = 0;
        cs->check_failed = 0;
    }
    if (lane == 0) wt->count = 0;
    __syncthreads();      // the shared copy of the plan is complete

    const uint32_t tpt = shape.search_tpt;          // tasks per tiling in the searched task space
    const uint64_t task_begin = p.t_begin * tpt, task_end = p.t_end * tpt;
    const uint64_t dump_origin = task_begin * kCandPerTask;
    const uint32_t n_orders = p.n_orders;
    unsigned long long my_rows = 0;
    uint32_t my_visits = 0;
    uint32_t my_tested = 0;       // rows whose capacity test and bound this lane evaluated (fewer than 2^32 per lane)

    // Builder: pull the next range and build its tables into buffer `buf`.  The first n_spread pulls (one per
    // CTA) take ranges spread evenly over the index space, so that the pruning bound G is near its final value
    // from the start; the other ranges follow in ascending order.  Ascending matters where many mappings tie at
    // the best key (latency at the compute bound): a tie enters a list only with a lower index than the list's last
    // entry, and in ascending order the later candidates never have one.
    // `coop` (a std::bool_constant): the whole CTA builds together (the first range, when there is nothing to walk
    // yet) instead of the builder warp alone.
    auto build_next = [&](int buf, auto coop) {
        constexpr bool COOP = decltype(coop)::value;
        const uint32_t first = COOP ? (uint32_t)tid : (uint32_t)lane;
        const uint32_t step = COOP ? (uint32_t)kSearchThreads : 32u;
        auto sync = [] { if constexpr (COOP) __syncthreads(); else __syncwarp(); };
        if (first == 0) {
            const unsigned long long got = atomicAdd(&scratch->next_task, 1ull);
            // pull number -> range: multiples of `step` first, then the ranges between them, then the tail
            uint64_t range = got;
            if (shape.n_spread && got < shape.n_ranges) {
                const uint64_t step = shape.n_ranges / shape.n_spread;       // >= 2
                if (got < shape.n_spread) {
                    range = got * step;
                } else {
                    const uint64_t r = got - shape.n_spread;
                    const uint64_t block = r / (step - 1), offset = r % (step - 1);
                    range = block < shape.n_spread ? block * step + 1 + offset
                                                   : shape.n_spread * step + (r - shape.n_spread * (step - 1));
                }
            }
            // range -> tasks: n_big ranges of range_tasks, then short ones of tail_tasks
            auto first_task = [&](uint64_t r) {
                return r <= shape.n_big ? r * shape.range_tasks
                                        : shape.n_big * shape.range_tasks + (r - shape.n_big) * shape.tail_tasks;
            };
            const uint64_t b0 = task_begin + first_task(range), b1 = task_begin + first_task(range + 1);
            cs->range_begin[buf] = got < shape.n_ranges ? b0 : task_end;
            cs->range_end[buf] = b1 < task_end ? b1 : task_end;
            cs->cursor[buf] = 0;
        }
        sync();
        const uint64_t r0 = cs->range_begin[buf];
        if (r0 >= task_end) return;
        const uint64_t r1 = cs->range_end[buf];
        const uint64_t t_first = r0 / tpt, t_last = (r1 - 1) / tpt;
        const uint32_t n_slots = (uint32_t)(t_last - t_first + 1);
        TilingTab* ttabs = ttabs_all + buf * shape.slots;
        OrderTab* otabs = otabs_all + (size_t)buf * shape.slots * n_orders;
        for (uint32_t sl = first; sl < n_slots; sl += step) build_tiling_head(p, t_first + sl, &ttabs[sl]);
        sync();
        // subset products of the bounds: one lane per (slot, half, subset)
        for (uint32_t it = first; it < n_slots * 32u; it += step) {
            TilingTab* tb = &ttabs[it >> 5];
            const uint32_t h = (it >> 4) & 1u, m = it & 15u;
            int64_t v = 1;
#pragma unroll
            for (int d = 0; d < 4; ++d)
                if (m >> d & 1u) v *= (int64_t)tb->b[h * 4 + d];
            tb->half[h][m] = v;
        }
        sync();
        // Items are visited kind by kind, so that the 32 lanes always run the same code path.
        const uint32_t n_so = n_slots * n_orders;
        auto order_pass = [&](uint32_t first_item, uint32_t n_items) {
            for (uint32_t it = first; it < n_so * n_items; it += step) {
                const uint32_t so = it / n_items, e = first_item + it % n_items;
                const uint32_t slot = so / n_orders, os = so % n_orders;
                if (!ttabs[slot].live) { fill_dead_order_item(&otabs[so], (int)e); continue; }
                build_order_item<OBJ>(p, &ttabs[slot], p.order_id[os], &otabs[so], (int)e);
            }
        };
        order_pass(0, 10);      // A, B
        order_pass(10, 5);      // C
        order_pass(15, 10);     // D, E
        order_pass(25, 1);      // C read-back (unfused)
        auto tiling_pass = [&](uint32_t first_item, uint32_t n_items) {
            for (uint32_t it = first; it < n_slots * n_items; it += step) {
                const uint32_t slot = it / n_items, e = first_item + it % n_items;
                if (!ttabs[slot].live) { fill_dead_tiling_item(&ttabs[slot], (int)e); continue; }
                build_tiling_item(p, &ttabs[slot], (int)e);
            }
        };
        for (uint32_t it = first; it < n_slots * 6u; it += step)      // one tile of each operator under each mode
            if (ttabs[it / 6u].live) build_tile_terms(p, &ttabs[it / 6u], (int)(it % 6u));
        sync();
        tiling_pass(0, 18);     // stationary pairs x recompute flag
        tiling_pass(18, 3);     // unfused Op1 compute words
        sync();
        if (OBJ == MMEE_OBJ_LATENCY || OBJ == MMEE_OBJ_EDP) {
            // compute words relative to their minimum over the stationary pairs: fused without and with
            // recomputation, and Op2 of an unfused task
            for (uint32_t j = first; j < 3 * n_slots; j += step) {
                TilingTab* tb = &ttabs[j / 3];
                const int v = (int)(j % 3);
                const int64_t* src = v < 2 ? &tb->CB[0][v] : &tb->QU[0][0];
                int64_t m = kInfKey;       // over the stationary pairs the array offers (never none)
                for (int s = 0; s < 9; ++s)
                    if ((p.sm_mask >> s) & 1u) m = src[2 * s] < m ? src[2 * s] : m;
                tb->qmin[v] = m;
                if constexpr (OBJ == MMEE_OBJ_EDP) tb->fl[2 + v] = __ll2float_rd(m);
                for (int s = 0; s < 9; ++s) {
                    const int64_t qd = src[2 * s] - m;
                    const int64_t qs = qd >> p.rel_shift;
                    // (a pair the array does not offer: kUnfit, which no threshold part, clamped at -kUnfit, can
                    // bring below zero)
                    tb->Qrel[v][s] = !((p.sm_mask >> s) & 1u) ? kUnfit : (qs > (int64_t)kTermCap ? kTermCap : (int32_t)qs);
                }
                // entries 9..11: the least term of each Op1 stationary mode (kUnfit: none of its pairs is offered)
                for (int j2 = 0; j2 < 3; ++j2) {
                    const int32_t* r = &tb->Qrel[v][3 * j2];
                    tb->Qrel[v][9 + j2] = min(r[0], min(r[1], r[2]));
                }
                if (v == 2) {
                    int64_t c1 = kInfKey;
                    for (int j2 = 0; j2 < 3; ++j2)
                        if ((p.sm_mask >> (3 * j2)) & 7u) c1 = tb->C1w[j2] < c1 ? tb->C1w[j2] : c1;
                    tb->c1min = c1;
                }
            }
        }
        if (OBJ == MMEE_OBJ_ENERGY || OBJ == MMEE_OBJ_EDP) {
            // The least stationary-pair energy term, over the pairs the array offers (never none): a row's least
            // energy over its nine mappings is its row sum plus this.
            for (uint32_t j = first; j < 2 * n_slots; j += step) {
                TilingTab* tb = &ttabs[j >> 1];
                const int rc = (int)(j & 1);
                int64_t m = kInfKey;
                for (int s = 0; s < 9; ++s)
                    if ((p.sm_mask >> s) & 1u) m = tb->W[s][rc] < m ? tb->W[s][rc] : m;
                tb->wmin[rc] = m;
                if constexpr (OBJ == MMEE_OBJ_EDP) {
                    tb->fl[rc] = __ll2float_rd(m);
                    if (rc == 0) {
                        const int64_t c1 = min(tb->C1w[0], min(tb->C1w[1], tb->C1w[2]));
                        tb->fl[5] = __ll2float_rd(c1);
                        tb->fl[6] = __ll2float_rd(tb->cw);
                        tb->fl[7] = __ll2float_rd(tb->smx);
                    }
                }
            }
        }
    };

    build_next(0, std::true_type{});
    __syncthreads();

    for (int iter = 0;; ++iter) {
        const int buf = iter & 1;
        const uint64_t r0 = cs->range_begin[buf];
        if (r0 >= task_end) break;
        if (builder) build_next(buf ^ 1, std::false_type{});
        {       // every warp walks tasks; the builder warp joins once the next range's tables are done
        const uint64_t r1 = cs->range_end[buf];
        const uint64_t t_first = r0 / tpt;
        const TilingTab* ttabs = ttabs_all + buf * shape.slots;
        const OrderTab* otabs = otabs_all + (size_t)buf * shape.slots * n_orders;

        // ---- tasks
        const uint32_t w_first = (uint32_t)(r0 - t_first * tpt);      // task of r0 inside its tiling
        const uint32_t n_range = (uint32_t)(r1 - r0);
        // Worker warps take 32 tasks at a time from a cursor in shared memory: warps whose tasks fall
        // into pruned tilings come back sooner and take more.
        while (true) {
            uint32_t off = 0;
            if (lane == 0) off = atomicAdd(&cs->cursor[buf], 32u);
            off = __shfl_sync(kFull, off, 0);
            if (off >= n_range) break;
            const bool valid = off + lane < n_range;
            const uint32_t o = valid ? off + lane : n_range - 1;
            const uint32_t wa = w_first + o;
            const uint32_t slot = wa / tpt;
            const uint32_t wc = wa - slot * tpt;
            // With row pruning the searched task space lists only the tasks that still hold a kept
            // row: each searched unit is one middle level (kept_mid) of a task, `kept` the mask of its rows.
            uint32_t w = wc, kept = 0x1ffffffu, kept_mid = 0;
            if constexpr (PRUNE) {
                const PrunedTask pt = shape.pruned[wc];
                w = pt.task;
                kept_mid = pt.mid;
                kept = pt.rows;
            }
            const uint64_t tq = PRUNE ? (t_first + slot) * (uint64_t)p.tasks_per_tiling + w : r0 + o;
            const TilingTab* tb = &ttabs[slot];
            const bool live = valid && tb->live;
            if (DUMP && valid && !tb->live) {
                for (int c = 0; c < kCandPerTask; ++c) dump[tq * kCandPerTask - dump_origin + c] = kInfKey;
            }
            if (!__any_sync(kFull, live)) continue;

            const TaskChoice c = decode_task(p, w);
            const OrderTab* ot = &otabs[slot * n_orders + c.order_slot];
            const uint64_t task_first_idx = tq * kCandPerTask;
            // The other CTAs' pruning bound: the load is issued here and consumed at the end of the
            // task, so that its latency is covered by the task's own work.
            const long long g_seen = (lane == 0) ? *reinterpret_cast<volatile long long*>(&scratch->G) : 0;
            // (flags mode: 25 bytes per task, relative to the first task of the searched range)
            unsigned char* flags = (FLAGS && live) ? reinterpret_cast<unsigned char*>(dump) + (tq - task_begin) * 25u : nullptr;
            if constexpr (!DUMP && OBJ <= MMEE_OBJ_LATENCY) {
                my_rows += walk_task_relative<OBJ, PRUNE, FLAGS>(p, tb, ot, c, live, kept, kept_mid, task_first_idx, wt, cs,
                                                                 &scratch->G, k, lane, my_visits, my_tested, flags);
            } else {
                my_rows += walk_task_exact<OBJ, DUMP, PRUNE, FLAGS>(p, tb, ot, c, live, valid, kept, kept_mid, task_first_idx,
                                                                    wt, cs, &scratch->G, k, lane, dump, dump_origin, my_visits,
                                                                    my_tested, flags);
            }
            if (lane == 0 && g_seen < cs->G) atomicMin(&cs->G, g_seen);
        }
        }   // workers
        __syncthreads();      // this buffer is rebuilt during the next range
    }

    // ---- feasible count
    unsigned long long tested_rows = my_tested;
    for (int off = 16; off; off >>= 1) {
        my_rows += __shfl_down_sync(kFull, my_rows, off);
        tested_rows += __shfl_down_sync(kFull, tested_rows, off);
    }
    if (lane == 0 && my_rows) atomicAdd(&cs->feasible_rows, my_rows);
    if (lane == 0 && tested_rows) atomicAdd(&cs->tested_rows, tested_rows);
    if (lane == 0 && my_visits) atomicAdd(&cs->exact_visits, (unsigned long long)my_visits);
    __syncthreads();

    // ---- merge the warps' lists into warp 0's, then publish this CTA's partial list
    if (warp == 0) {
        // (in registers, lane j holding entry j: see reg_insert)
        int64_t ek = kInfKey;
        uint64_t ei = UINT64_MAX;
        if (lane < wt->count) {
            const longlong2 own = wt->e[lane];
            ek = own.x; ei = (uint64_t)own.y;
        }
        for (int w2 = 1; w2 < kSearchThreads / 32; ++w2) {
            const WarpTop* src = &wtops[w2];
            const int n = src->count;
            const longlong2 theirs = lane < n ? src->e[lane] : make_longlong2(kInfKey, -1ll);
            reg_absorb(ek, ei, k, n, theirs.x, (uint64_t)theirs.y, lane);
        }
        // An entry above the bound G (some full list's last key, here or in another CTA) cannot be among the
        // k best of the whole search: it is not published.
        Partial* out = &scratch->partial[blockIdx.x];
        long long g_end = (lane == 0) ? *reinterpret_cast<volatile long long*>(&scratch->G) : 0;
        g_end = __shfl_sync(kFull, g_end, 0);
        if (cs->G < g_end) g_end = cs->G;
        const int n = __popc(__ballot_sync(kFull, (ek != kInfKey || ei != UINT64_MAX) && ek <= g_end));
        if (lane < n) out->e[lane] = make_longlong2((long long)ek, (long long)ei);
        if (lane == 0) {
            out->count = n;
            if (cs->feasible_rows) atomicAdd(&scratch->feasible_rows, cs->feasible_rows);
            if (cs->exact_visits) atomicAdd(&scratch->exact_visits, cs->exact_visits);
            if (cs->tested_rows) atomicAdd(&scratch->tested_rows, cs->tested_rows);
        }
        if constexpr (!DUMP && !FLAGS) {
            // Grid reduction without a wait: every CTA makes its partial list visible, then draws a ticket; the
            // CTA that draws the last one knows that all lists are there and runs the finalize step.
            __threadfence();
            __syncwarp();
            if (lane == 0) cs->last_cta = atomicAdd(&scratch->done_ctas, 1u) == gridDim.x - 1 ? 1u : 0u;
        }
    }
    if constexpr (!DUMP && !FLAGS) {
        __syncthreads();
        if (cs->last_cta) {
            __threadfence();
            // (the table buffers are no longer in use: their first bytes hold the warps' lists of the merge)
            finalize_step(p, scratch, (int)gridDim.x, out_best, out_topk,
                          reinterpret_cast<longlong2 (*)[MMEE_MAX_TOPK]>(ttabs_all), &cs->check_failed);
        }
    }
}

__global__ void reset_kernel(Scratch* scratch) {
    scratch->next_task = 0;
    scratch->feasible_rows = 0;
    scratch->G = kInfKey - 1;
    scratch->exact_visits = 0;
    scratch->tested_rows = 0;
    scratch->done_ctas = 0;
}

__global__ void eval_kernel(const __grid_constant__ Plan p, uint64_t idx_begin, uint64_t count,
                            mmee_result_t* __restrict__ out) {
    for (uint64_t i = blockIdx.x * (uint64_t)blockDim.x + threadIdx.x; i < count;
         i += (uint64_t)gridDim.x * blockDim.x) {
        mmee_result_t r;
        evaluate_candidate(p, idx_begin + i, r);
        out[i] = r;
    }
}

// The kernels take more dynamic shared memory than the default limit: the limit of each instantiation is
// raised once per device, to the device's opt-in maximum, so that a launch is one driver call and two host
// threads with different table sizes cannot undo each other's setting.
template <int OBJ, int MODE>
cudaError_t allow_large_smem(int device) {
    static std::mutex mu;
    static unsigned long long done = 0;       // one bit per device
    std::lock_guard<std::mutex> lock(mu);
    if (device >= 0 && device < 64 && (done >> device & 1ull)) return cudaSuccess;
    int optin = 0;
    cudaError_t e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(search_kernel<OBJ, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, optin);
    if (e == cudaSuccess && device >= 0 && device < 64) done |= 1ull << device;
    return e;
}

template <int OBJ, int MODE>
cudaError_t launch_search_t(const Plan& p, const LaunchShape& shape, int device, Scratch* scratch, int64_t* dump,
                            mmee_result_t* out_best, mmee_result_t* out_topk, cudaStream_t st) {
    cudaError_t e = allow_large_smem<OBJ, MODE>(device);
    if (e != cudaSuccess) return e;
    search_kernel<OBJ, MODE><<<shape.grid, kSearchThreads, shape.smem_bytes, st>>>(p, shape, scratch, dump, out_best, out_topk);
    return cudaGetLastError();
}

template <int OBJ, int MODE>
cudaError_t occupancy_t(int device, int* blocks_per_sm, size_t smem) {
    cudaError_t e = allow_large_smem<OBJ, MODE>(device);
    if (e != cudaSuccess) return e;
    return cudaOccupancyMaxActiveBlocksPerMultiprocessor(blocks_per_sm, search_kernel<OBJ, MODE>, kSearchThreads, smem);
}

}  // namespace

size_t search_smem_bytes(const Plan& p, uint32_t slots) {
    return kPlanBytes + sizeof(CtaShared) + (kSearchThreads / 32) * sizeof(WarpTop) + 2 * slots * sizeof(TilingTab) +
           2 * (size_t)slots * p.n_orders * sizeof(OrderTab);
}

cudaError_t search_occupancy(const Plan& p, int device, size_t smem, int* blocks_per_sm) {
    switch (p.objective) {
        case MMEE_OBJ_ENERGY: return occupancy_t<MMEE_OBJ_ENERGY, kModeSearch>(device, blocks_per_sm, smem);
        case MMEE_OBJ_LATENCY: return occupancy_t<MMEE_OBJ_LATENCY, kModeSearch>(device, blocks_per_sm, smem);
        case MMEE_OBJ_EDP: return occupancy_t<MMEE_OBJ_EDP, kModeSearch>(device, blocks_per_sm, smem);
        case MMEE_OBJ_ENERGY_LCAP: return occupancy_t<MMEE_OBJ_ENERGY_LCAP, kModeSearch>(device, blocks_per_sm, smem);
        default: return occupancy_t<MMEE_OBJ_LATENCY_ECAP, kModeSearch>(device, blocks_per_sm, smem);
    }
}

cudaError_t launch_filter_flags(const Plan& p, const LaunchShape& shape, int device, Scratch* scratch, unsigned char* flags,
                                cudaStream_t st) {
    int64_t* out = reinterpret_cast<int64_t*>(flags);
    switch (p.objective) {
        case MMEE_OBJ_ENERGY: return launch_search_t<MMEE_OBJ_ENERGY, kModeFlags>(p, shape, device, scratch, out, nullptr, nullptr, st);
        case MMEE_OBJ_LATENCY: return launch_search_t<MMEE_OBJ_LATENCY, kModeFlags>(p, shape, device, scratch, out, nullptr, nullptr, st);
        case MMEE_OBJ_EDP: return launch_search_t<MMEE_OBJ_EDP, kModeFlags>(p, shape, device, scratch, out, nullptr, nullptr, st);
        default: return cudaErrorInvalidValue;
    }
}

cudaError_t launch_search(const Plan& p, const LaunchShape& shape, int device, Scratch* scratch, int64_t* dump,
                          mmee_result_t* out_best, mmee_result_t* out_topk, cudaStream_t st) {
    if (dump) {
        switch (p.objective) {
            case MMEE_OBJ_ENERGY: return launch_search_t<MMEE_OBJ_ENERGY, kModeDump>(p, shape, device, scratch, dump, out_best, out_topk, st);
            case MMEE_OBJ_LATENCY: return launch_search_t<MMEE_OBJ_LATENCY, kModeDump>(p, shape, device, scratch, dump, out_best, out_topk, st);
            case MMEE_OBJ_EDP: return launch_search_t<MMEE_OBJ_EDP, kModeDump>(p, shape, device, scratch, dump, out_best, out_topk, st);
            case MMEE_OBJ_ENERGY_LCAP: return launch_search_t<MMEE_OBJ_ENERGY_LCAP, kModeDump>(p, shape, device, scratch, dump, out_best, out_topk, st);
            default: return launch_search_t<MMEE_OBJ_LATENCY_ECAP, kModeDump>(p, shape, device, scratch, dump, out_best, out_topk, st);
        }
    }
    if (shape.pruned) {
        switch (p.objective) {
            case MMEE_OBJ_ENERGY: return launch_search_t<MMEE_OBJ_ENERGY, kModePrune>(p, shape, device, scratch, nullptr, out_best, out_topk, st);
            case MMEE_OBJ_LATENCY: return launch_search_t<MMEE_OBJ_LATENCY, kModePrune>(p, shape, device, scratch, nullptr, out_best, out_topk, st);
            case MMEE_OBJ_EDP: return launch_search_t<MMEE_OBJ_EDP, kModePrune>(p, shape, device, scratch, nullptr, out_best, out_topk, st);
            case MMEE_OBJ_ENERGY_LCAP: return launch_search_t<MMEE_OBJ_ENERGY_LCAP, kModePrune>(p, shape, device, scratch, nullptr, out_best, out_topk, st);
            default: return launch_search_t<MMEE_OBJ_LATENCY_ECAP, kModePrune>(p, shape, device, scratch, nullptr, out_best, out_topk, st);
        }
    }
    switch (p.objective) {
        case MMEE_OBJ_ENERGY: return launch_search_t<MMEE_OBJ_ENERGY, kModeSearch>(p, shape, device, scratch, nullptr, out_best, out_topk, st);
        case MMEE_OBJ_LATENCY: return launch_search_t<MMEE_OBJ_LATENCY, kModeSearch>(p, shape, device, scratch, nullptr, out_best, out_topk, st);
        case MMEE_OBJ_EDP: return launch_search_t<MMEE_OBJ_EDP, kModeSearch>(p, shape, device, scratch, nullptr, out_best, out_topk, st);
        case MMEE_OBJ_ENERGY_LCAP: return launch_search_t<MMEE_OBJ_ENERGY_LCAP, kModeSearch>(p, shape, device, scratch, nullptr, out_best, out_topk, st);
        default: return launch_search_t<MMEE_OBJ_LATENCY_ECAP, kModeSearch>(p, shape, device, scratch, nullptr, out_best, out_topk, st);
    }
}

cudaError_t launch_reset(Scratch* scratch, cudaStream_t st) {
    reset_kernel<<<1, 1, 0, st>>>(scratch);
    return cudaGetLastError();
}

cudaError_t launch_eval(const Plan& p, uint64_t idx_begin, uint64_t count, mmee_result_t* out, cudaStream_t st) {
    if (!count) return cudaSuccess;
    const uint64_t want = (count + 127) / 128;
    const int grid = (int)(want < 4096 ? want : 4096);
    eval_kernel<<<grid, 128, 0, st>>>(p, idx_begin, count, out);
    return cudaGetLastError();
}

}  // namespace mmee
