// Offline symbolic row pruning for single-optimum searches (Section VI-B), in a tie-safe form.
//
// The paper drops a row v when another row u of the same group needs no more buffer and no less
// DRAM traffic for every tiling, one of the two strictly (Eq. 12).  That keeps the optimum VALUE but
// may drop a row that merely ties with a kept one, and this library promises the lowest index among
// equal keys.  The rule used here is therefore: v is dropped iff some row u of the same fusion mode
// and recompute group with a LOWER row index has, symbolically, BS^Op1_u <= BS^Op1_v,
// BS^Op2_u <= BS^Op2_v and DA_u <= DA_v (for unfused rows: the DRAM sums of the two operators
// separately).  Then for every tiling and stationary pair u fits whenever v fits and
// (key_u, idx_u) < (key_v, idx_v) under each objective (energy is a sum, latency a max / a sum of
// maxima, EDP their product: all monotone), so v can never be the optimum.  Rows with identical
// symbolic sums are dropped too, except the one with the lowest index.  Valid for k = 1 only.
#include "mmee_plan.h"

#include <algorithm>
#include <map>
#include <vector>

namespace mmee {

namespace {

// A sum of monomials; each monomial is the set of loop bounds (query vector) it multiplies.
struct SymSum {
    int n = 0;
    uint8_t term[6] = {0, 0, 0, 0, 0, 0};
    void add(uint8_t q) { term[n++] = q; }
    void canon() { std::sort(term, term + n); }
    bool operator<(const SymSum& o) const {
        if (n != o.n) return n < o.n;
        for (int i = 0; i < n; ++i) if (term[i] != o.term[i]) return term[i] < o.term[i];
        return false;
    }
};

// q <= p for every assignment of bounds >= 1 if q's terms embed one-to-one into supersets among p's.
bool embeds(const SymSum& p, const SymSum& q, int qi, unsigned used) {
    if (qi == q.n) return true;
    for (int i = 0; i < p.n; ++i) {
        if (used & (1u << i)) continue;
        if ((q.term[qi] & p.term[i]) != q.term[qi]) continue;
        if (embeds(p, q, qi + 1, used | (1u << i))) return true;
    }
    return false;
}
bool sum_le(const SymSum& q, const SymSum& p) { return q.n <= p.n && embeds(p, q, 0, 0); }

struct Signature {
    SymSum part[4];       // BS^Op1, BS^Op2, DA (fused) or DA of Op1, DA of Op2 (unfused; part[3] empty when fused)
    int group;            // fusion mode * 2 + recompute flag
    bool operator<(const Signature& o) const {
        if (group != o.group) return group < o.group;
        for (int i = 0; i < 4; ++i) {
            if (part[i] < o.part[i]) return true;
            if (o.part[i] < part[i]) return false;
        }
        return false;
    }
};

bool sig_le(const Signature& u, const Signature& v) {
    if (u.group != v.group) return false;
    for (int i = 0; i < 4; ++i) if (!sum_le(u.part[i], v.part[i])) return false;
    return true;
}

Signature signature_of(const QueryTables& q, uint32_t phi, uint32_t order, const uint32_t lv[5]) {
    Signature s;
    const bool fused = phi == 0;
    const uint32_t rc = fused ? q.recompute[order][lv[OP_C]] : 0u;
    s.group = (int)(phi * 2 + rc);
    uint8_t bs[5];
    for (int x = 0; x < 5; ++x) bs[x] = q.bs[order][x][lv[x]];
    s.part[0].add(bs[OP_A]); s.part[0].add(bs[OP_B]); s.part[0].add(bs[OP_C]);
    s.part[1].add(bs[OP_C]); s.part[1].add(bs[OP_D]); s.part[1].add(bs[OP_E]);
    if (fused) {
        if (lv[OP_D]) s.part[0].add(bs[OP_D]);
        if (lv[OP_E]) s.part[0].add(bs[OP_E]);
        if (lv[OP_A]) s.part[1].add(bs[OP_A]);
        if (lv[OP_B]) s.part[1].add(bs[OP_B]);
        s.part[2].add(q.da[order][OP_A][lv[OP_A]][rc]);
        s.part[2].add(q.da[order][OP_B][lv[OP_B]][rc]);
        s.part[2].add(q.da[order][OP_D][lv[OP_D]][0]);
        s.part[2].add(q.da[order][OP_E][lv[OP_E]][0]);
    } else {
        s.part[2].add(q.da_unfused[order][OP_A][lv[OP_A]]);
        s.part[2].add(q.da_unfused[order][OP_B][lv[OP_B]]);
        s.part[3].add(q.da_unfused[order][OP_C][0]);
        s.part[3].add(q.da_unfused[order][OP_D][lv[OP_D]]);
        s.part[3].add(q.da_unfused[order][OP_E][lv[OP_E]]);
    }
    for (int i = 0; i < 4; ++i) s.part[i].canon();
    return s;
}

}  // namespace

namespace {

// Fills keep[row] (rows_per_tiling entries) for the plan's row space.
void build_row_keep(const Plan& p, std::vector<uint8_t>* keep) {
    const uint32_t R = p.rows_per_tiling;
    keep->assign(R, 1);
    std::vector<int> sig_of_row(R);
    std::map<Signature, int> ids;
    std::vector<Signature> sigs;
    std::vector<uint32_t> first_row;                      // lowest row index with this signature
    // rows in index order: fused r = o*3125 + lA*625 + lB*125 + lC*25 + lD*5 + lE, then per unfused
    // mode o*625 + lA*125 + lB*25 + lD*5 + lE
    const uint32_t fused_rows = p.n_fused_blocks * 3125u;
    for (uint32_t row = 0; row < R; ++row) {
        uint32_t block, lv[5];
        if (row < fused_rows) {
            block = row / 3125u;
            const uint32_t r = row % 3125u;
            lv[0] = r / 625u; lv[1] = (r / 125u) % 5u; lv[2] = (r / 25u) % 5u; lv[3] = (r / 5u) % 5u; lv[4] = r % 5u;
        } else {
            const uint32_t u = row - fused_rows;
            block = p.n_fused_blocks + u / 625u;
            const uint32_t r = u % 625u;
            lv[0] = r / 125u; lv[1] = (r / 25u) % 5u; lv[2] = 0; lv[3] = (r / 5u) % 5u; lv[4] = r % 5u;
        }
        const uint32_t phi = p.block_phi[block], order = p.order_id[p.block_order_slot[block]];
        {
            const Signature s = signature_of(p.q, phi, order, lv);
            auto it = ids.find(s);
            if (it == ids.end()) {
                it = ids.emplace(s, (int)sigs.size()).first;
                sigs.push_back(s);
                first_row.push_back(row);
            }
            sig_of_row[row] = it->second;
        }
    }
    // best_row[s] = lowest row index among the signatures that are <= s (itself included)
    const size_t n = sigs.size();
    std::vector<uint32_t> best_row(first_row);
    for (size_t v = 0; v < n; ++v)
        for (size_t u = 0; u < n; ++u)
            if (first_row[u] < best_row[v] && sig_le(sigs[u], sigs[v])) best_row[v] = first_row[u];
    for (uint32_t row = 0; row < R; ++row)
        if (best_row[sig_of_row[row]] < row) (*keep)[row] = 0;
}

}  // namespace

// The (task, middle level) groups of 25 rows that still hold a kept row, in index order, with their
// kept-row masks.  `out` has room for 5 * tasks_per_tiling entries.
int build_pruned_tasks(const Plan& p, PrunedTask* out, uint32_t* n_out, uint32_t* kept_rows) {
    std::vector<uint8_t> keep;
    build_row_keep(p, &keep);
    uint32_t n = 0, rows = 0;
    for (uint32_t w = 0; w < p.tasks_per_tiling; ++w) {
        for (uint32_t m = 0; m < 5; ++m) {
            PrunedTask t = {w, m, 0, 0};
            for (uint32_t de = 0; de < 25; ++de)
                if (keep[w * 125u + m * 25u + de]) { t.rows |= 1u << de; ++rows; }
            if (t.rows) out[n++] = t;
        }
    }
    *n_out = n;
    *kept_rows = rows;
    return MMEE_OK;
}

}  // namespace mmee
