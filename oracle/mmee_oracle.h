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
 * PARITY UNPINNED by the paper (builder-defined readings, checked only by hand
 * on one tile): buffer<->PE traffic BR, register-file count N_RF, the unfused
 * rows (phi = 1, 2), absolute energies.
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
