/*
 * libmmee -- exhaustive search over fused-attention dataflow mappings on one NVIDIA B200.
 *
 * The library evaluates the analytical buffer-size / DRAM-access / energy / latency model of
 * "Fast Cross-Operator Optimization of Attention Dataflow" (MMEE) for EVERY mapping of a fused
 * two-GEMM chain  C = A*B (Q*K^T), softmax, E = C*D (P*V)  onto a spatial accelerator, discards
 * the mappings that do not fit the on-chip buffer and returns the k best under one objective.
 * All model arithmetic runs in CUDA kernels (sm_100a); there is no CPU fallback.
 *
 * Plain C ABI: structs of fixed-width integers and doubles, raw pointers.  Every pointer
 * argument says below whether it is HOST or DEVICE memory.  All functions return an int status
 * (MMEE_OK = 0); nothing throws, aborts or traps.
 *
 * Candidate space (Sections III, IV, VI-A of the paper; dims I,K,L,J with I = query rows,
 * L = key/value rows, K = J = head dims):
 *   tiling t   : (i_G,k_G,l_G,j_G), each a divisor of its dim; x_D = X / x_G.  t is the mixed-radix
 *                number over the ascending divisor lists, j fastest.
 *   order pi   : order of the inter-tile loops (i2,l2,j2), outer->inner; k2 is always innermost
 *                (constraint "No Psum Propagation", Section III-C):
 *                0 (i,l,j) 1 (l,i,j) 2 (i,j,l) 3 (l,j,i) 4 (j,i,l) 5 (j,l,i)
 *   levels     : beta_X in 3..7 for X in A,B,C,D,E (Section IV-A "Buffering Level");
 *                L3 = one tile, L4 = k2, L5/L6/L7 = inner/middle/outer loop of the order
 *   stationary : sm1, sm2 in {0 weight, 1 input, 2 output} for the two operators (Section V-D)
 *   fusion phi : 0 fused (the paper's space), 1 unfused GEMMs with softmax in the first one's
 *                epilogue, 2 fully unfused (separate softmax pass)
 *   row r      : fused rows first, r = o*3125 + (bA-3)*625 + (bB-3)*125 + (bC-3)*25 + (bD-3)*5 + (bE-3)
 *                with o the position of pi in the order set; then one block of 625 rows per order for
 *                each unfused mode (bC = 3): o*625 + (bA-3)*125 + (bB-3)*25 + (bD-3)*5 + (bE-3)
 *   index      : idx = (t*R + r)*9 + 3*sm1 + sm2,  R rows per tiling,  N = T*R*9 candidates
 */
#ifndef MMEE_H
#define MMEE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* objective */
#define MMEE_OBJ_ENERGY   0u   /* energy-driven search (Section VII-D)                         */
#define MMEE_OBJ_LATENCY  1u   /* latency-driven search                                         */
#define MMEE_OBJ_EDP      2u   /* energy-delay product (Section VII-K)                          */
#define MMEE_OBJ_ENERGY_LCAP   3u   /* least energy among mappings with l_key <= key_cap          */
#define MMEE_OBJ_LATENCY_ECAP  4u   /* least latency among mappings with e_key <= key_cap         */
/* tiling_set */
#define MMEE_TILE_POW2          0u   /* only power-of-two tile extents                          */
#define MMEE_TILE_ALL_DIVISORS  1u   /* every integer factorisation (Section VI-A)              */
/* order_set */
#define MMEE_ORD_NORECOMP2  0u   /* orders 0 and 1 (j2 innermost: no recomputation)             */
#define MMEE_ORD_ALL6       1u   /* all six orders (recomputation included, Section III-C)      */
/* fuse_mask bits */
#define MMEE_FUSE_FUSED            1u
#define MMEE_FUSE_SOFTMAX_IN_OP1   2u
#define MMEE_FUSE_SEPARATE         4u

#define MMEE_MAX_TOPK      16u
#define MMEE_MAX_DIVISORS  64u    /* per dimension */
#define MMEE_NO_INDEX      UINT64_MAX

/* status codes */
#define MMEE_OK               0
#define MMEE_ERR_ARG          1   /* NULL pointer, zero dimension, value out of range              */
#define MMEE_ERR_OVERFLOW     2   /* a worst-case key of this problem does not fit 62 bits         */
#define MMEE_ERR_QUANTUM      3   /* an energy is not an integer multiple of energy_quantum_pj     */
#define MMEE_ERR_NO_FEASIBLE  4   /* no mapping fits the buffer (reported in mmee_result_t.status) */
#define MMEE_ERR_CUDA         5   /* a CUDA runtime call failed (no device, launch error, ...)     */
#define MMEE_ERR_TIMEOUT      6   /* reserved: the kernels contain no device-side wait             */
#define MMEE_ERR_RANGE        7   /* request exceeds a documented maximum                          */
#define MMEE_ERR_CHECK        8   /* a winner's ranking key is not the key of its full evaluation (internal
                                     consistency check of the finalize step): the records are not a result.
                                     In out_best->status after mmee_search; the return value of the
                                     synchronous entry points (mmee_solve_host, mmee_search_shapes, ...)  */

/* Attention workload.  Heads are independent instances of one search (Section V, first
 * paragraph); the q_heads/kv_heads query heads that share a K/V head are stacked along I. */
typedef struct {
    uint32_t batch, q_heads, kv_heads;       /* instances = batch*kv_heads                       */
    uint32_t seq_q, seq_kv, d_qk, d_v;       /* I = (q_heads/kv_heads)*seq_q, L = seq_kv, K, J   */
    uint32_t word_bytes;                     /* operand word size                                 */
} mmee_workload_t;

/* Spatial accelerator template (Section II-B): PE arrays with register files, one global
 * buffer, DRAM.  Energies are per word moved / per MAC, in pJ. */
typedef struct {
    uint32_t pe_rows, pe_cols, n_arrays;
    uint64_t gb_bytes;                       /* global buffer capacity                            */
    uint64_t rf_bytes;                       /* per-PE register file; 0 = no register-file level  */
    uint32_t dram_words_per_cycle;
    double   e_dram_pj, e_gb_pj, e_rf_pj, e_mac_pj;
    double   c_softmax;                      /* softmax cost per score element, in MAC energies   */
    double   energy_quantum_pj;              /* every energy must be an integer multiple of this  */
} mmee_arch_t;

typedef struct {
    uint32_t objective;                      /* MMEE_OBJ_*                                        */
    uint32_t topk;                           /* 1..MMEE_MAX_TOPK                                  */
    uint32_t tiling_set;                     /* MMEE_TILE_*                                       */
    uint32_t order_set;                      /* MMEE_ORD_*                                        */
    uint32_t fuse_mask;                      /* OR of MMEE_FUSE_*, at least one bit               */
    uint32_t row_pruning;                    /* 1: offline symbolic row pruning (Section VI-B); needs
                                                topk = 1.  Rows that a lower-index row dominates for every
                                                tiling are not evaluated: the optimum is unchanged, but
                                                n_feasible then counts only the evaluated rows.        */
    uint64_t t_begin, t_end;                 /* tiling sub-range [t_begin,t_end); the pair 0,0 stands for
                                                the whole space, so an empty range cannot start at 0   */
    int64_t  key_cap;                        /* MMEE_OBJ_*CAP: bound on the other key (energy in quanta,
                                                latency in words); ignored otherwise                   */
    uint32_t stationary_mask;                /* bit 3*sm1+sm2 set: the array offers that stationary pair
                                                (Section VII-K: a fixed array offers one, a reconfigurable
                                                one several); 0 = all nine.  A mapping with another pair
                                                is outside the space: never selected, not in n_feasible */
    uint32_t rf_tiling;                      /* 1: a third tiling level below the buffer tile, in the PEs' register files
                                                (the register-file level of the accelerator template, Section II-B).
                                                The stationary operand of each operator's tile is processed in blocks
                                                of a x b elements (divisors of its two extents; weight stationary:
                                                reduction x output columns, input stationary: output rows x reduction,
                                                output stationary: output rows x columns).  A block lives in the register
                                                files, element (x, y) in PE (x mod pe_rows, y mod pe_cols), beside one
                                                register each for the streamed operand and the partial sum: it is
                                                admissible iff ceil(a/pe_rows)*ceil(b/pe_cols) + 2 <= rf_bytes/word_bytes.
                                                The streamed vectors pass once per block, one cycle per element a PE
                                                holds.  Each mapping takes, per operator, the admissible block with the
                                                fewest buffer<->array words (energy objective; then the fewest cycles) or
                                                the fewest cycles (latency objective; then the fewest words), the first
                                                such block in ascending (a, b) order.  Energy and latency objectives on
                                                an architecture with a register file only; 0: one array fold per pass. */
} mmee_objective_t;

/* One fully evaluated mapping.  Counts are per instance. */
typedef struct {
    uint64_t idx;                            /* MMEE_NO_INDEX when the slot is empty              */
    uint64_t t;
    uint32_t row;
    uint32_t bound[8];                       /* i_D,k_D,l_D,j_D,i_G,k_G,l_G,j_G (Section V-E)     */
    uint8_t  phi, pi, beta[5], sm[2], recompute, feasible, reserved[5];
    int32_t  status;                         /* MMEE_OK, MMEE_ERR_NO_FEASIBLE or MMEE_ERR_CHECK   */
    int64_t  bs_x[5];                        /* buffer words of A,B,C,D,E (Section V-B)           */
    int64_t  bs_op1, bs_op2, bs;             /* Eq. (1), (2), (4)                                 */
    int64_t  da_x[5];                        /* DRAM words of A,B,C,D,E (Section V-C); C only unfused */
    int64_t  da_sm;                          /* separate softmax pass, phi = 2                    */
    int64_t  br, cyc1, cyc2;                 /* buffer<->PE words; compute cycles per operator    */
    int64_t  n[5];                           /* N_DRAM, N_GB, N_RF, N_MAC, N_SFU                  */
    int64_t  e_key;                          /* energy in quanta                                  */
    int64_t  l_key;                          /* latency in words = cycles * dram_words_per_cycle  */
    double   edp_key;                        /* (double)e_key * (double)l_key                     */
    double   energy_pj;                      /* e_key * quantum * instances                       */
    double   latency_cycles;                 /* l_key / words_per_cycle * ceil(instances/n_arrays) */
    uint64_t n_total;                        /* candidates of the searched range (in out_best)    */
    uint64_t n_feasible;                     /* of which fit the buffer, with an offered stationary pair (in out_best) */
    uint32_t rf_block[6];                    /* objective.rf_tiling: register-file block (m, r, n) of the first operator's
                                                tile, then of the second's (1 for the streamed extent); else 0        */
    uint32_t reserved2[2];
} mmee_result_t;

typedef struct mmee_handle mmee_handle_t;

/*
 * mmee_create -- plan one search (problem statement of Section VI-A: workload dims, accelerator,
 * objective in; optimal mapping out).  Enumerates the tilings by integer factorisation, derives
 * the query vectors of every (order, operand, level) (Section V-E, Section VI-A "offline"
 * enumeration), quantises the energies and bounds the largest possible key.
 *   workload, arch, objective : HOST, read only during the call.
 *   out                       : HOST, receives the handle.  The handle owns a few KB of DEVICE
 *                               scratch on the device that is current at the call.
 * Errors: MMEE_ERR_ARG, _OVERFLOW, _QUANTUM, _RANGE (more than MMEE_MAX_DIVISORS divisors), _CUDA.
 */
int mmee_create(const mmee_workload_t* workload, const mmee_arch_t* arch,
                const mmee_objective_t* objective, mmee_handle_t** out);

/*
 * mmee_search -- evaluate every mapping of the handle's range, drop those whose buffer need
 * (Eq. 4) exceeds the global buffer, and select the k smallest (key, idx) (Section VI-A; ties
 * broken by the lower index).  Asynchronous on `cuda_stream` (a cudaStream_t, may be 0).
 *   out_best : DEVICE, one mmee_result_t; also carries n_total / n_feasible and, when nothing
 *              fits, status = MMEE_ERR_NO_FEASIBLE with idx = MMEE_NO_INDEX.
 *   out_topk : DEVICE, objective.topk entries, best first, unused slots idx = MMEE_NO_INDEX;
 *              may be NULL.
 * Caller owns both buffers.  Calls on one handle must not overlap on the GPU.  The handle's device
 * must be the current device (MMEE_ERR_ARG otherwise; the same holds for mmee_eval, mmee_decode and
 * mmee_dump_keys).
 */
int mmee_search(mmee_handle_t* handle, void* cuda_stream, mmee_result_t* out_best,
                mmee_result_t* out_topk);

/*
 * mmee_search_host -- mmee_search on the default stream of the handle's device followed by the copy of
 * the records to HOST memory: the time to the optimal mapping of a planned search.  The first call on
 * a handle allocates 1 + topk records of pinned host memory that the kernel writes its records into;
 * later calls allocate nothing.  Synchronous.
 *   out_best : HOST, one record.   out_topk : HOST, objective.topk records, or NULL.
 * Returns MMEE_ERR_CHECK if the finalize step's self-check failed (the records are then not a result).
 */
int mmee_search_host(mmee_handle_t* handle, mmee_result_t* out_best, mmee_result_t* out_topk);

int mmee_destroy(mmee_handle_t* handle);

/*
 * mmee_search_static -- the same search as mmee_create + mmee_search + mmee_destroy, for callers
 * that must not allocate device memory.  (The paper has no counterpart: this is an interface
 * variant of the library, not a part of the method.)
 *
 * For whom: a process that has given the whole device to its own memory pool (a cudaMalloc from a
 * library then fails), or a latency-critical loop that cannot afford the device-wide
 * synchronisation of cudaMalloc / cudaFree.  This call makes no cudaMalloc, cudaFree or other
 * allocating call.  Its scratch (work counter, pruning bound, one partial top-k list per CTA) is a
 * fixed 139 328-byte array inside the library image, present on every device that loads the
 * library for as long as the process lives.
 *
 *   workload, arch, objective : HOST, as for mmee_create; planned on the host at every call.
 *   out_best, out_topk        : DEVICE, caller-owned, as for mmee_search (out_topk may be NULL).
 * Asynchronous on `cuda_stream`.  The first call on a device looks up the array's device address
 * (with that device current); make that first call before any stream capture begins.  The address
 * is kept for the life of the process: after a cudaDeviceReset it is stale, and this entry point
 * must not be called on that device again.
 * objective.row_pruning must be 0 here (its kept-row list would need a device allocation).
 * Limits: the array holds the partial lists of at most 512 persistent CTAs; a device whose launch
 * shape needs more is refused with MMEE_ERR_RANGE.  Other errors as mmee_create / mmee_search.
 * All calls on a device share the one array and it keeps the previous call's contents: the call
 * clears the header itself, but two mmee_search_static calls that overlap on the GPU (for instance
 * on different streams) race on it and give undefined results: serialise them.  Searches through
 * handles use their own scratch and are not affected.
 */
int mmee_search_static(const mmee_workload_t* workload, const mmee_arch_t* arch,
                       const mmee_objective_t* objective, void* cuda_stream,
                       mmee_result_t* out_best, mmee_result_t* out_topk);

/* Number of candidates / tilings / rows of the full space of the handle (HOST values). */
uint64_t mmee_num_candidates(const mmee_handle_t* handle);
uint64_t mmee_num_tilings(const mmee_handle_t* handle);
uint64_t mmee_num_rows(const mmee_handle_t* handle);

const char* mmee_strerror(int status);

/* Text of the CUDA runtime error behind the calling thread's most recent MMEE_ERR_CUDA. */
const char* mmee_last_cuda_error(void);

/*
 * mmee_eval -- evaluate `count` consecutive candidates from `idx_begin` on the device with the
 * query-vector form of the model, exp(q . ln b) taken exactly as an integer product
 * (Section V-E, Eq. 8), and write one full record each.
 *   out : DEVICE, count records.  Asynchronous on the stream.
 */
int mmee_eval(mmee_handle_t* handle, void* cuda_stream, uint64_t idx_begin, uint64_t count,
              mmee_result_t* out);

/*
 * mmee_decode -- one candidate index back to its mapping (tiling, order, levels, stationary pair;
 * index layout at the top of this file) with its full evaluation (Section VI-A: the output of the
 * search is the optimal tiling, order and buffering levels with their metrics).  The record is
 * computed on the device by the same code as mmee_eval and copied to the host.  Synchronous.
 *   host_out : HOST, one record.  MMEE_ERR_ARG for an index outside the handle's space.
 */
int mmee_decode(mmee_handle_t* handle, uint64_t idx, mmee_result_t* host_out);

/*
 * mmee_dump_keys -- run the search kernel in its key-dump mode over the handle's tiling range and
 * store every candidate's objective key instead of reducing (Eq. 11: the full result matrix).  The
 * dump mode shares the kernel's tables, decode and task walk, and forms every key exactly in 64 bits
 * (the path the search takes for the energy-delay and capped objectives and for every group of rows
 * that its 32-bit filter flags); the filter itself is not part of it.
 *   out_keys : DEVICE, (t_end - t_begin) * R * 9 int64; entry idx - t_begin*R*9.  Energy and
 *              latency keys as integers, EDP keys as the bit pattern of the double; INT64_MAX
 *              for a mapping that does not fit the buffer.
 * Meant for small ranges (parity checks).  MMEE_ERR_RANGE above 2^31 candidates.
 */
int mmee_dump_keys(mmee_handle_t* handle, void* cuda_stream, int64_t* out_keys);

/*
 * mmee_filter_flags -- test view of the search kernel's filter.  The search decides with a cheap bound per group of
 * five rows (45 mappings: one level of D, the five levels of E, nine stationary pairs) whether the group can hold a
 * key below the current threshold, and forms exact keys only for flagged groups (32-bit threshold-relative sums for
 * energy and latency, a single-precision product bound followed by double-precision products for the energy-delay
 * product).  This call runs that filter over the handle's tiling range against the FIXED threshold `threshold_key`
 * (a key as the search orders it; for the energy-delay product the bit pattern of the double), inserts nothing, and
 * stores one byte per group: 1 = flagged.  A group that holds a mapping that fits, with an offered stationary pair and
 * a key < threshold_key, must be flagged; the converse need not hold.
 *   out_flags : DEVICE, (t_end - t_begin) * (R / 125) * 25 bytes; group g of middle level m of task w (a task is 125
 *               consecutive rows of a tiling) at ((t - t_begin) * (R / 125) + w) * 25 + m * 5 + g.
 * Energy, latency and energy-delay objectives without row pruning; MMEE_ERR_ARG otherwise.  Asynchronous.
 */
int mmee_filter_flags(mmee_handle_t* handle, void* cuda_stream, int64_t threshold_key, uint8_t* out_flags);

/*
 * mmee_solve_host -- whole path with HOST buffers: plan, upload, search, copy the results back,
 * release.  Synchronous.  out_best: HOST, one record; out_topk: HOST, objective.topk records or
 * NULL.  h2d_bytes / d2h_bytes (HOST, may be NULL) receive the bytes copied in each direction.
 */
int mmee_solve_host(const mmee_workload_t* workload, const mmee_arch_t* arch,
                    const mmee_objective_t* objective, mmee_result_t* out_best,
                    mmee_result_t* out_topk, uint64_t* h2d_bytes, uint64_t* d2h_bytes);

/*
 * mmee_pareto_front -- the energy-latency trade-off of the whole mapping space (Section VII-E): every
 * pair (e_key, l_key) of a feasible mapping that no other feasible mapping improves in one key without
 * losing in the other, by increasing energy / decreasing latency, each with the lowest-index mapping
 * that attains it.  Computed by alternating capped searches on the device (least energy under a latency
 * bound, then least latency at that energy): two searches per point.  objective.objective, .topk,
 * .row_pruning and .key_cap are ignored.  Synchronous.
 *   out_points : HOST, `capacity` records; *n_points receives the number of points of the front, also
 *                when it exceeds capacity (then MMEE_ERR_RANGE is returned and the first `capacity`
 *                points are valid).
 */
int mmee_pareto_front(const mmee_workload_t* workload, const mmee_arch_t* arch,
                      const mmee_objective_t* objective, mmee_result_t* out_points, uint32_t capacity,
                      uint32_t* n_points);

/*
 * mmee_pareto_front_bs_da -- the buffer-size / DRAM-traffic trade-off of the whole mapping space (Section VI-A,
 * Section VII-C): every pair (BS, DA) of a mapping with BS <= arch.gb_bytes / word_bytes that no other mapping
 * improves in one of the two without losing in the other, by decreasing buffer size / increasing traffic, each
 * with the lowest-index mapping of least traffic among those that need no more buffer.  Computed by device
 * searches for the least DRAM traffic under a shrinking buffer (one search per distinct buffer need met on the
 * way down).  The energies of arch and objective.objective, .topk, .row_pruning, .key_cap are ignored: the key
 * of the returned records (e_key) is the DRAM word count n[0].  Synchronous.
 *   out_points : HOST, `capacity` records; *n_points receives the number of points of the front, also when it
 *                exceeds capacity (then MMEE_ERR_RANGE is returned and the first `capacity` points are valid).
 */
int mmee_pareto_front_bs_da(const mmee_workload_t* workload, const mmee_arch_t* arch,
                            const mmee_objective_t* objective, mmee_result_t* out_points, uint32_t capacity,
                            uint32_t* n_points);

/*
 * mmee_search_shapes -- reconfigurable PE arrays (Section VII-K): the same search on each of several logical
 * array shapes (the stationary modes the array can switch between are objective.stationary_mask), one device
 * search per shape, and the shape whose optimum has the least key.  arch.pe_rows / pe_cols are replaced by each
 * shape in turn; everything else is as given.  Synchronous.
 *   shapes      : HOST, n_shapes pairs (rows, cols), each >= 1.
 *   out_per_shape : HOST, n_shapes records: the optimum on that shape (idx = MMEE_NO_INDEX, status
 *                   MMEE_ERR_NO_FEASIBLE when nothing fits; n_total / n_feasible of that search).
 *   out_best_shape : HOST, index of the shape with the least key (the objective's; the first of equal ones),
 *                    UINT32_MAX when no shape has a feasible mapping.
 * objective.topk and .row_pruning are ignored (one optimum per shape, exhaustive).
 */
int mmee_search_shapes(const mmee_workload_t* workload, const mmee_arch_t* arch,
                       const mmee_objective_t* objective, const uint32_t* shapes, uint32_t n_shapes,
                       mmee_result_t* out_per_shape, uint32_t* out_best_shape);

/*
 * mmee_query_vector -- HOST only, no device needed.  The query vector q in {0,1}^8 over
 * b = [i_D,k_D,l_D,j_D,i_G,k_G,l_G,j_G] (Section V-E) of one metric of one operand:
 *   metric 0 = operand buffer size BS_X (Section V-B), 1 = operand DRAM access DA_X (Section V-C).
 *   phi, pi, operand (0..4 = A..E), beta (3..7), recompute (0/1; only read for DA of A and B).
 * Returns MMEE_ERR_ARG for values out of range or for DA of the fused intermediate C (which is 0).
 */
int mmee_query_vector(uint32_t metric, uint32_t phi, uint32_t pi, uint32_t operand, uint32_t beta,
                      uint32_t recompute, uint8_t out_q[8]);

/*
 * mmee_row_pruning_keep -- HOST only, no device needed.  The rows of one tiling that survive the
 * offline symbolic pruning (Section VI-B) for the order set and fusion modes of `objective`:
 * out_keep[r] = 1 if row r is evaluated when objective.row_pruning = 1, else 0.  A row is dropped iff
 * a row of the same fusion mode and recompute group with a lower index needs, for every tiling, no
 * more buffer in either operator and no more DRAM traffic (Eq. 12 made safe for ties: the dropped row
 * can then never be the lowest-index optimum).  out_keep: HOST, `capacity` bytes; *out_rows receives
 * the number of rows R; MMEE_ERR_RANGE if capacity < R.
 */
int mmee_row_pruning_keep(const mmee_objective_t* objective, uint8_t* out_keep, uint32_t capacity,
                          uint32_t* out_rows);

/* HOST only: whether order `pi` with C buffered at level `beta_c` regenerates C (Section III-C). */
int mmee_recompute_flag(uint32_t pi, uint32_t beta_c, uint32_t* out_flag);

/*
 * mmee_last_search_stats -- HOST counters of the most recent mmee_search on the handle, valid
 * after the stream has been synchronised (the call copies one counter from the device): kernels
 * launched by that call (one: the CTA that finishes last merges the partial results and writes the
 * records), persistent CTAs, threads per CTA, dynamic shared memory per CTA, tasks (groups of 1125
 * consecutive mappings) and, when mmee_kernel_timing is on, the device time of the search kernel in
 * milliseconds (CUDA events recorded on the search's stream; -1 when timing is off).  finalize_ms
 * is 0: the finalize step is part of the search kernel.
 */
typedef struct {
    uint32_t kernels_launched, grid, block, smem_bytes;
    uint64_t tasks;
    float    search_ms, finalize_ms;
    uint32_t rows_per_tiling;                /* R                                                  */
    uint32_t rows_evaluated_per_tiling;      /* R, or the rows that survive symbolic row pruning   */
    uint64_t exact_path_visits;              /* groups of rows the 32-bit (or floating-point) filter sent to the
                                                exact 64-bit path during that search               */
    float    create_ms;                      /* host wall clock of the mmee_create that made the handle */
    uint32_t reserved;
    uint64_t rows_tested;                    /* rows (of nine mappings each) whose capacity test (Eq. 4) and
                                                bound the search evaluated; the rest lay in tilings, middle
                                                levels or groups that a coarser test showed not to fit   */
} mmee_launch_stats_t;
int mmee_last_search_stats(const mmee_handle_t* handle, mmee_launch_stats_t* out);

/* mmee_kernel_timing -- switch per-kernel CUDA-event timing of mmee_search on (1) or off (0). */
int mmee_kernel_timing(mmee_handle_t* handle, int enable);

/*
 * mmee_alu_peak -- measure the integer instruction rates of the current device with register-only
 * kernels (the denominators of the search kernel's roofline).  out: HOST, four doubles:
 *   [0] 32-bit logic instructions, 10^9 per second (integer ALU pipe alone)
 *   [1] 32-bit add + logic pairs, 10^9 instructions per second
 *   [2] the search kernel's candidate mix -- a 64-bit add and a 64-bit signed compare, counted as
 *       four 32-bit instructions -- 10^9 instructions per second
 *   [3] SM clock in MHz during the measurement
 * Synchronous; a few milliseconds; allocates and frees 4 KB of device memory.
 */
int mmee_alu_peak(double out[4]);

#ifdef __cplusplus
}
#endif
#endif /* MMEE_H */
