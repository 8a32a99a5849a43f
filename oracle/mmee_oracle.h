/*
 * CPU oracle for the MMEE search path -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, branch-per-decision evaluation of the analytical model for
 * fused two-GEMM (attention) dataflow mappings: every candidate index is
 * decoded into (tiling, fusion mode, loop order, five buffering levels, two
 * stationary modes) and its cost is computed directly from the model's
 * definitions.  It shares no code, header, table or constant with the CUDA
 * library and must never be linked or imported by it.  Only tests, the smoke
 * entry and the benchmark's CPU-baseline leg may call it.
 *
 * Parity pins (what fixes this code to something other than itself):
 *   - worked example of Section V (BS_A, DA_A, DA_D, Eq. 3, query vector q),
 *   - a tile-granular loop-nest simulator (mo_simulate, below) that executes
 *     the pseudo nested loop of Section IV and counts loads / occupancy,
 *   - MAC/softmax counts of Section V-D, Table I Accel.-1 closed-form latency,
 *   - row-count arithmetic of Sections VI-B / VII-C (18 750 rows, 18 groups),
 *   - brute-force sort for argmin / top-k.
 *   - an element-level execution of tiles on the PE array (mo_array_tile /
 *     mo_array_chain) for cycles, buffer<->array words, carried partial sums,
 *     MACs and register-file accesses,
 *   - a tile-granular execution of the two unfused loop nests
 *     (mo_simulate_unfused) for the rows of phi = 1, 2.
 * PARITY UNPINNED by the paper: absolute energies (its 28 nm energy table is
 * not printed); the array model itself (which operand each stationary mode
 * pins to which array dimension) is this build's reading, stated in
 * mo_array_tile.
 */
#ifndef MMEE_ORACLE_H
#define MMEE_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { MO_OBJ_ENERGY = 0, MO_OBJ_LATENCY = 1, MO_OBJ_EDP = 2 };
enum { MO_TILE_POW2 = 0, MO_TILE_ALL_DIVISORS = 1 };
enum { MO_ORD_NORECOMP2 = 0, MO_ORD_ALL6 = 1 };
enum { MO_OK = 0, MO_ERR_ARG = 1, MO_ERR_OVERFLOW = 2, MO_ERR_QUANTUM = 3 };
enum { MO_MAX_DIVISORS = 256, MO_MAX_TOPK = 64 };

typedef struct {
    uint32_t batch, q_heads, kv_heads;
    uint32_t seq_q, seq_kv, d_qk, d_v;
    uint32_t word_bytes;
} mo_workload;

typedef struct {
    uint32_t pe_rows, pe_cols, n_arrays;
    uint64_t gb_bytes, rf_bytes;
    uint32_t dram_words_per_cycle;
    double e_dram_pj, e_gb_pj, e_rf_pj, e_mac_pj, c_softmax;
    double energy_quantum_pj;
} mo_arch;

typedef struct {
    uint32_t objective, topk, tiling_set, order_set, fuse_mask;
    uint32_t stationary_mask;              /* bit 3*sm1+sm2 set: that stationary pair is in the space; 0 = all nine
                                              (a reconfigurable array offers several, a fixed one a single pair) */
    uint64_t t_begin, t_end;
    uint32_t rf_tiling;                    /* 1: register-file-level tiling (see mo_rf_block); energy / latency only */
    uint32_t pad;
} mo_objective;

/* Everything derived once from the three input structs. */
typedef struct {
    uint64_t dim[4];                       /* I, K, L, J of one instance            */
    uint32_t instances;                    /* batch * kv_heads                      */
    uint32_t ndiv[4];
    uint32_t divs[4][MO_MAX_DIVISORS];     /* ascending x_G candidates per dim      */
    uint64_t T;                            /* number of tilings                     */
    uint32_t n_orders;  uint32_t order_id[6];
    uint32_t n_phi;     uint32_t phi_id[3];
    uint64_t R;                            /* rows per tiling                       */
    uint64_t N;                            /* T * R * 9                             */
    uint64_t t_begin, t_end;               /* searched tiling range                 */
    int64_t  cq_dram, cq_gb, cq_rf, cq_mac, cq_sfu;   /* energies in quanta          */
    double   quantum_pj;
    int      has_rf;
    uint64_t cap_words;                    /* floor(gb_bytes / word_bytes)          */
    uint32_t pe_rows, pe_cols, n_arrays, bw;
    uint32_t objective, topk;
    uint32_t stationary_mask;              /* never 0 */
    uint32_t rf_tiling;
    uint64_t rf_words;                     /* floor(rf_bytes / word_bytes)          */
} mo_problem;

typedef struct {
    uint64_t idx, t;
    uint32_t row;
    uint32_t bound[8];                     /* i_D,k_D,l_D,j_D,i_G,k_G,l_G,j_G       */
    uint32_t phi, pi;
    uint32_t beta[5];                      /* A,B,C,D,E                             */
    uint32_t sm[2];
    uint32_t recompute, feasible;
    int64_t  bs_x[5];                      /* per-operand buffer words              */
    int64_t  bs_op1, bs_op2, bs;
    int64_t  da_x[5];                      /* A, B, C(write+read when unfused), D, E */
    int64_t  da_sm;                        /* separate softmax pass (phi = 2)       */
    int64_t  da1, da2;                     /* unfused per-operator DRAM words       */
    int64_t  br, cyc1, cyc2;
    int64_t  n[5];                         /* N_DRAM, N_GB, N_RF, N_MAC, N_SFU      */
    int64_t  e_key, l_key;
    double   edp_key;
    double   energy_pj, latency_cycles;
    uint32_t rf_block[6];                  /* register-file-level tiling: block (m, r, n) of Op1, then of Op2; 0 when off */
} mo_record;

typedef struct {
    int64_t  loads[5];                     /* tile loads per operand (C: always 0)  */
    int64_t  c_productions;                /* times a C tile was (re)generated      */
    int64_t  op1_stages, op2_stages;
    int64_t  peak_op1, peak_op2, peak;     /* occupancy in words                    */
    int32_t  n_trace;                      /* stages recorded in trace[]            */
    int64_t  trace[64];                    /* occupancy (words) of the first stages */
    int32_t  trace_kind[64];               /* 1 = Op1, 2 = softmax, 3 = Op2         */
} mo_sim_out;

int  mo_problem_init(const mo_workload*, const mo_arch*, const mo_objective*, mo_problem* out);
int  mo_eval(const mo_problem*, uint64_t idx, mo_record* out);
int  mo_eval_range(const mo_problem*, uint64_t begin, uint64_t count, mo_record* out);
/* key as the search orders it: int64 for energy/latency, IEEE bits of the product for EDP;
 * feasible[i] = 1 iff the candidate fits the global buffer and its stationary pair is in the space. */
int  mo_keys_range(const mo_problem*, uint64_t begin, uint64_t count, int64_t* keys, uint8_t* feasible);
/* k smallest (key, idx) among feasible candidates of tilings [t_begin, t_end); out_topk has topk
 * entries, unused ones carry idx = UINT64_MAX.  n_threads <= 0: all cores. */
int  mo_search(const mo_problem*, mo_record* out_topk, uint64_t* n_total, uint64_t* n_feasible,
               uint32_t* n_found, int n_threads);
int  mo_simulate(const uint32_t bound[8], uint32_t pi, const uint32_t beta[5], mo_sim_out* out);

/* Tile-granular execution of the two separate loop nests of an unfused mapping (phi = 1, 2): the
 * producer nest (k2 innermost, then i2 / l2 in the order's relative order; every finished C tile is
 * stored), the optional softmax pass over C, and the consumer nest (the order's three loops; C at L3
 * is read back).  Counts tile loads / stores per operand and the peak occupancy of each nest; uses
 * none of the closed forms. */
typedef struct {
    int64_t  loads[5];                     /* words loaded per operand; C: read back by the consumer nest */
    int64_t  c_stores;                     /* words of C stored by the producer nest                      */
    int64_t  softmax_words;                /* words moved by the separate softmax pass (phi = 2)          */
    int64_t  op1_stages, op2_stages;
    int64_t  peak_op1, peak_op2;           /* occupancy in words                                          */
} mo_sim_unfused_out;
int  mo_simulate_unfused(const uint32_t bound[8], uint32_t pi, const uint32_t beta[5], uint32_t phi,
                         mo_sim_unfused_out* out);

/* Element-level execution of tiles on a rows x cols PE array, for the array-level terms of the
 * model (compute cycles, buffer<->array words, MACs, register-file accesses).  Written as loops
 * over folds, streamed vectors and PEs that count events; none of the ceiling formulas appear. */
typedef struct {
    int64_t cycles;                        /* one per streamed vector per fold                            */
    int64_t words;                         /* words crossing the buffer<->array boundary, both directions */
    int64_t macs;                          /* multiply-accumulates performed by the PEs                   */
    int64_t rf;                            /* register-file accesses                                      */
} mo_array_counts;
/* One (m x r) * (r x n) tile; resume != 0: the output tile already holds partial sums of earlier
 * reduction steps in the buffer, which the array has to take in first.  Adds to *acc. */
int  mo_array_tile(uint32_t sm, uint32_t m, uint32_t r, uint32_t n, uint32_t rows, uint32_t cols,
                   int resume, mo_array_counts* acc);
/* Register-file-level tiling (third tiling level, below the buffer tile).  The stationary operand of a tile is
 * cut into blocks of a x b elements (a, b divisors of its two extents); one block at a time lives in the PEs'
 * register files, element (x, y) in PE (x mod rows, y mod cols), so that a PE holds ceil(a/rows) * ceil(b/cols)
 * of them, beside one register for the streamed operand and one for the partial sum: a block is admissible iff
 * that count + 2 <= rf_words.  The streamed vectors pass once per block; a vector takes one cycle per element a
 * PE holds.  mo_array_tile_blocked executes one tile that way, element by element (block (a, b) as the two
 * stationary extents: weight stationary (r, n), input stationary (m, r), output stationary (m, n)). */
int  mo_array_tile_blocked(uint32_t sm, uint32_t m, uint32_t r, uint32_t n, uint32_t rows, uint32_t cols,
                           uint32_t a, uint32_t b, int resume, mo_array_counts* acc);
/* The block the model picks for one tile: every admissible (a, b) is tried in ascending (a, b) order; the energy
 * objective keeps the block with the fewest buffer<->array words (then the fewest cycles, then the first), the
 * latency objective the one with the fewest cycles (then the fewest words, then the first).  Returns MO_ERR_ARG
 * if no block is admissible (cannot happen for rf_words >= 3). */
int  mo_rf_block(uint32_t objective, uint32_t sm, uint32_t m, uint32_t r, uint32_t n, uint32_t rows, uint32_t cols,
                 uint64_t rf_words, uint32_t block_mrn[3], int64_t* words, int64_t* cycles);

/* Every tile invocation of both operators of one tiling in loop order: Op1 = C(i2,l2) += A*B over
 * k2, the whole of it `productions` times (recomputation), Op2 = E(i2,j2) += C*D over l2. */
int  mo_array_chain(const uint32_t bound[8], uint32_t productions, uint32_t sm1, uint32_t sm2,
                    uint32_t rows, uint32_t cols, mo_array_counts out[2]);
int  mo_threads_used(void);

/* Symbolic form of one fused row (Section V-E): every BS_X / DA_X as the set of loop bounds it is the
 * product of, bit d = x_D of loop d (i,k,l,j), bit 4+d = x_G.  da_q[OPD_C] = 0 (no DRAM traffic). */
typedef struct {
    uint8_t bs_q[5], da_q[5];
    uint8_t tau[5];
    uint8_t recompute;
} mo_row_symbols;
int  mo_row_symbolic(uint32_t pi, const uint32_t beta[5], mo_row_symbols* out);

/* Offline symbolic pruning of the fused row space (Section VI-B, Eq. 12) over all six orders:
 * keep[r] = 0 for rows that another row of the same recompute group dominates for every tiling.
 * kept_per_group[g] / rows_per_group[g]: g = recompute flag.  18 750 rows. */
int  mo_symbolic_prune(uint8_t* keep, uint32_t kept_per_group[2], uint32_t rows_per_group[2]);

#ifdef __cplusplus
}
#endif
#endif
