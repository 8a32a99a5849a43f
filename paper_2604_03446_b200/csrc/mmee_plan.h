// Internal: the search plan handed to the kernels by value, and the host planner's interface.
#pragma once

#include <stdint.h>
#include "../../include/mmee.h"

namespace mmee {

constexpr int kMaxOrders = 6;
constexpr int kMaxBlocks = 18;     // (fusion mode, order) pairs
constexpr int kRowsPerTask = 125;   // one middle level (C when fused, B when unfused) x levels of D and E
constexpr int kCandPerTask = 1125;  // rows x 9 stationary pairs
constexpr int64_t kInfKey = INT64_MAX;

// Operand / loop numbering shared by host planner and kernels.
enum { OP_A = 0, OP_B = 1, OP_C = 2, OP_D = 3, OP_E = 4 };
enum { LOOP_I = 0, LOOP_K = 1, LOOP_L = 2, LOOP_J = 3 };

// Query vectors as 8-bit selector masks over b = [i_D,k_D,l_D,j_D,i_G,k_G,l_G,j_G]
// (bit d = x_D of loop d, bit 4+d = x_G).  Indexed by the ACTUAL order id 0..5.
struct QueryTables {
    uint8_t bs[6][5][5];          // [order][operand][beta-3]            operand buffer size
    uint8_t da[6][5][5][2];       // [order][operand][beta-3][recompute] fused DRAM access (C unused)
    uint8_t da_unfused[6][5][5];  // [order][operand][beta-3]            unfused; C: read-back at beta=3
    uint8_t recompute[6][5];      // [order][beta_C-3]
};

struct Plan {
    uint32_t dim[4];              // I, K, L, J of one instance
    uint32_t ndiv[4];
    uint32_t instances, n_arrays;
    uint32_t n_orders;            // orders in the search, in row order
    uint32_t order_id[kMaxOrders];
    uint32_t n_blocks;            // (phi, order) blocks in row order, fused first
    uint32_t n_fused_blocks;
    uint32_t fused_tasks;         // n_fused_blocks * 25
    uint8_t  block_phi[kMaxBlocks];
    uint8_t  block_order_slot[kMaxBlocks];   // position of the block's order in order_id[]
    uint32_t tasks_per_tiling;    // fused_tasks + 5 per unfused block
    uint32_t rows_per_tiling;     // R = 125 * tasks_per_tiling
    uint64_t n_tilings;           // T
    uint64_t t_begin, t_end;
    int64_t  cap_words;
    int64_t  c_dram_gb;           // quanta per DRAM word moved (DRAM + buffer side)
    int64_t  c_br;                // quanta per buffer<->PE word (buffer + register file side)
    int64_t  c_mac;               // quanta per MAC (MAC + 3 register-file accesses)
    int64_t  c_sfu;               // quanta per softmax element
    int64_t  cq[5];               // raw quantised energies: dram, gb, rf, mac, sfu
    uint32_t has_rf;
    uint32_t bw, pe_rows, pe_cols;
    uint32_t objective, topk;
    uint32_t row_pruning;
    uint32_t sm_mask, n_sm;       // stationary pairs in the space (bit s = 3*sm1+sm2; never 0) and their number
    int64_t  key_cap;             // capped objectives: bound on the other key
    uint32_t rel_shift;           // energy: threshold-relative keys are kept in units of 2^rel_shift quanta
    int32_t  unit;                // the constant 1, as a run-time value: x * unit + y is issued as an integer
                                  // multiply-add, which the FMA pipe executes beside the integer ALU pipe
    uint32_t rf_tiling;           // register-file-level tiling: the block of each operator's tile is searched
    uint32_t rf_words;            // register-file capacity of one PE in words
    double   quantum_pj;
    QueryTables q;
    uint32_t divs[4][MMEE_MAX_DIVISORS];
};

// Host planner (mmee_plan.cu).  Fills `plan`; returns an MMEE_* status.
int build_plan(const mmee_workload_t* w, const mmee_arch_t* a, const mmee_objective_t* o, Plan* plan);
void build_query_tables(QueryTables* q);

// Tie-safe symbolic row pruning (mmee_prune.cu): keep[row] for every row of a tiling.
struct PrunedTask { uint32_t task, mid, rows, pad; };   // task inside a tiling, middle level, 25-bit mask of kept rows
int build_pruned_tasks(const Plan& plan, PrunedTask* out, uint32_t* n_out, uint32_t* kept_rows);

}  // namespace mmee
