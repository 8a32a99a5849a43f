// Internal: device scratch layout and kernel launchers (mmee_search.cu), used by the C ABI.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>

#include "mmee_plan.h"

namespace mmee {

constexpr int kSearchThreads = 256;
constexpr int kWorkerWarps = kSearchThreads / 32 - 1;     // the last warp builds tables
constexpr int kWorkerThreads = kWorkerWarps * 32;

// One CTA's k best (key, idx) pairs, best first.
struct alignas(16) Partial {
    longlong2 e[MMEE_MAX_TOPK];     // x = key, y = idx: one 16-byte word per pair, stored and loaded whole
    int32_t count;
    int32_t pad[3];
};

// Global scratch of one handle: a work counter, the feasible-row count, the shared pruning bound,
// the count of exact-path visits and one partial list per CTA.  The header is reset by the finalize
// step, which also keeps the finished search's visit count in `last_exact_visits`.
struct Scratch {
    unsigned long long next_task;
    unsigned long long feasible_rows;
    long long G;
    unsigned long long exact_visits;
    unsigned long long last_exact_visits;
    unsigned long long tested_rows;         // rows whose capacity test and bound were evaluated
    unsigned long long last_tested_rows;
    unsigned int done_ctas;         // ticket counter: the CTA that draws the last ticket runs the finalize step
    unsigned int pad;
    Partial partial[1];     // grid entries follow
};

struct LaunchShape {
    uint32_t grid;          // persistent CTAs
    uint32_t range_tasks;   // tasks a CTA takes per pull: those of `slots` whole tilings where that many fit
    uint32_t slots;         // tilings one range can touch
    uint32_t smem_bytes;
    uint32_t search_tpt;    // tasks per tiling in the searched task space (fewer with row pruning)
    uint32_t tail_tasks;    // tasks of each range from number n_big on (one tiling's; the last ranges are short)
    const PrunedTask* pruned;   // device: the kept tasks of a tiling (row pruning), else null
    uint64_t n_ranges;      // ranges of the searched task interval: n_big of range_tasks, the others of tail_tasks
    uint64_t n_big;
    uint64_t n_spread;      // the first n_spread pulls take ranges spread evenly over the interval (multiples of
                            // n_ranges / n_spread >= 2), the others follow in ascending order; 0: ascending only
};

inline size_t scratch_bytes(uint32_t grid) { return sizeof(Scratch) + (size_t)(grid ? grid - 1 : 0) * sizeof(Partial); }

size_t search_smem_bytes(const Plan& p, uint32_t slots);
cudaError_t search_occupancy(const Plan& p, int device, size_t smem, int* blocks_per_sm);
// One launch per search: the last CTA to finish merges the partial lists, evaluates the winners into
// out_best / out_topk (device) and resets the scratch header.  With `dump` set the kernel stores every
// key instead and writes no result (the caller resets the header).
cudaError_t launch_search(const Plan& p, const LaunchShape& shape, int device, Scratch* scratch, int64_t* dump,
                          mmee_result_t* out_best, mmee_result_t* out_topk, cudaStream_t st);
// Test mode: the search kernel's filter alone against the fixed threshold p.key_cap; flags[(task - first task) * 25
// + middle level * 5 + group] is set to 1 for every flagged group (the caller clears the buffer first and resets
// the scratch header afterwards).  Energy, latency and energy-delay objectives.
cudaError_t launch_filter_flags(const Plan& p, const LaunchShape& shape, int device, Scratch* scratch, unsigned char* flags,
                                cudaStream_t st);
cudaError_t launch_reset(Scratch* scratch, cudaStream_t st);
cudaError_t launch_eval(const Plan& p, uint64_t idx_begin, uint64_t count, mmee_result_t* out, cudaStream_t st);
cudaError_t measure_alu_peak(double* giops);

// Launch shape of a search on `device`: tasks per range, table slots, shared memory, persistent CTAs
// (at most max_ctas when that is not 0: MMEE_ERR_RANGE if the device would take more), range order.
int choose_launch_shape(const Plan& p, int device, uint32_t search_tpt, uint32_t max_ctas, LaunchShape* shape);

// MMEE_OK, or MMEE_ERR_CUDA with the error kept for mmee_last_cuda_error (per host thread).
int cuda_status(cudaError_t e);

}  // namespace mmee
