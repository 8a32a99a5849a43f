// C ABI of libmmee (declared and documented in include/mmee.h).
#include <cuda_runtime.h>

#include <chrono>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "mmee_search.h"

static_assert(sizeof(mmee_result_t) == 336, "mmee_result_t is part of the ABI");
static_assert(sizeof(mmee::Plan) <= 4096, "the plan travels as a kernel parameter");

struct mmee_handle {
    mmee::Plan plan;
    mmee::LaunchShape shape;
    mmee::Scratch* scratch;      // device
    mmee_result_t* decode_buf;   // device, one record (mmee_decode); part of the scratch allocation
    mmee_result_t* host_out;     // pinned host memory mapped into the device's address space, 1 + topk records:
                                 // mmee_search_host lets the kernel write its records there (made at its first call)
    mmee::PrunedTask* pruned;    // device, row pruning only
    uint32_t kept_rows;          // rows of a tiling that survive pruning (all rows without it)
    int device;
    mmee_launch_stats_t last;
    float create_ms;             // host wall clock of mmee_create
    bool dirty;                  // a launch failed half-way: the scratch header is reset before the next search
    bool timing;
    cudaEvent_t ev[2];           // before and after the search kernel
};

namespace {

using namespace mmee;

thread_local cudaError_t g_last_cuda_error = cudaSuccess;

}  // namespace

namespace mmee {

int cuda_status(cudaError_t e) {
    if (e == cudaSuccess) return MMEE_OK;
    g_last_cuda_error = e;
    return MMEE_ERR_CUDA;
}

// Tasks a CTA pulls per visit of the global counter, and the tilings such a range can touch.
int choose_launch_shape(const Plan& p, int device, uint32_t search_tpt, uint32_t max_ctas, LaunchShape* shape) {
    int sm_count = 0, smem_optin = 0;      // attribute queries: cudaGetDeviceProperties costs milliseconds
    cudaError_t e = cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device);
    if (e != cudaSuccess) return cuda_status(e);
    // A task is 1125 mappings (225 with row pruning, where the searched units are single middle levels).
    shape->search_tpt = search_tpt;
    shape->pruned = nullptr;
    // Two CTAs per SM under the 196 KB shared-memory carve-out, which leaves the row loops 60 KB of L1 (the next
    // carve-out, 228 KB, leaves 28 KB and costs the energy-delay search a tenth of its speed).
    constexpr size_t kSmemTarget = 97 * 1024;
    // Ranges of whole tilings, as many as the table slots hold: a tiling's tables are then built once, not once
    // by each of the two ranges it would straddle, and a range needs no slot for a tiling it only touches.
    constexpr uint32_t kAlignedMaxTasks = 2048;
    const uint64_t tilings = p.t_end - p.t_begin;
    bool aligned = search_tpt <= kAlignedMaxTasks && search_smem_bytes(p, 1) <= kSmemTarget;
    uint32_t per_range = 1;                          // aligned: tilings of a range
    if (aligned) {
        while ((per_range + 1) * search_tpt <= kAlignedMaxTasks && search_smem_bytes(p, per_range + 1) <= kSmemTarget)
            ++per_range;
        // (a small problem, with fewer than four such ranges per CTA of a full grid, keeps ranges of a fixed number
        // of tasks: whole tilings would leave most warps of a CTA without work)
        if (tilings / per_range < 4ull * 2u * (uint64_t)sm_count) aligned = false;
    }
    if (aligned) {
        shape->range_tasks = per_range * search_tpt;
        shape->slots = per_range;
    } else {
        const uint32_t rounds = p.row_pruning ? 9 : 3;
        shape->range_tasks = rounds * kWorkerThreads;
        shape->slots = (shape->range_tasks - 1) / search_tpt + 2;
        // Many small tilings per range need many table slots: shrink the range until they fit.
        // (Worker warps take 32 tasks at a time, so a range may be as short as one warp's share.)
        while (search_smem_bytes(p, shape->slots) > kSmemTarget && shape->range_tasks > 32) {
            shape->range_tasks -= shape->range_tasks > (uint32_t)kWorkerThreads ? kWorkerThreads : 32;
            shape->slots = (shape->range_tasks - 1) / search_tpt + 2;
        }
    }
    const size_t smem = search_smem_bytes(p, shape->slots);
    if (smem > (size_t)smem_optin) return MMEE_ERR_RANGE;
    shape->smem_bytes = (uint32_t)smem;
    int per_sm = 0;
    if ((e = search_occupancy(p, device, smem, &per_sm)) != cudaSuccess) return cuda_status(e);
    if (per_sm < 1) return MMEE_ERR_RANGE;
    if (per_sm > 2) per_sm = 2;
    uint64_t grid = (uint64_t)sm_count * (uint32_t)per_sm;
    const uint64_t tasks = tilings * search_tpt;
    if (aligned) {
        // The last tilings go out one per range, about half a full range's worth per CTA: the CTAs then finish
        // within one tiling of each other instead of within one full range.  (Measured with a whole, a half and a
        // quarter of a range per CTA: the searches differ in which they prefer, by 1 to 3 %.)
        uint64_t tail = grid * per_range / 2;
        shape->n_big = (tilings - tail) / per_range;
        tail = tilings - shape->n_big * per_range;
        shape->tail_tasks = search_tpt;
        shape->n_ranges = shape->n_big + tail;
    } else {
        shape->n_ranges = (tasks + shape->range_tasks - 1) / shape->range_tasks;
        shape->n_big = shape->n_ranges;
        shape->tail_tasks = shape->range_tasks;
    }
    const uint64_t ranges = shape->n_ranges;
    if (grid > ranges) grid = ranges ? ranges : 1;
    // (a caller with a fixed scratch: a device that would take more CTAs is refused, not silently under-used)
    if (max_ctas && grid > max_ctas) return MMEE_ERR_RANGE;
    shape->grid = (uint32_t)grid;
    // one spread range per CTA while at least as many ranges remain for the ascending part
    shape->n_spread = grid < ranges / 2 ? grid : ranges / 2;
    return MMEE_OK;
}

}  // namespace mmee

extern "C" {

int mmee_create(const mmee_workload_t* workload, const mmee_arch_t* arch, const mmee_objective_t* objective,
                mmee_handle_t** out) {
    if (!out) return MMEE_ERR_ARG;
    *out = nullptr;
    const auto t0 = std::chrono::steady_clock::now();
    mmee_handle* h = new (std::nothrow) mmee_handle;
    if (!h) return MMEE_ERR_ARG;
    std::memset(h, 0, sizeof(*h));
    int rc = build_plan(workload, arch, objective, &h->plan);
    if (rc) { delete h; return rc; }
    if ((rc = cuda_status(cudaGetDevice(&h->device)))) { delete h; return rc; }
    // Row pruning: the searched task space lists only the tasks that keep at least one row.
    std::vector<PrunedTask> kept_tasks;
    uint32_t search_tpt = h->plan.tasks_per_tiling;
    h->kept_rows = h->plan.rows_per_tiling;
    if (h->plan.row_pruning) {
        kept_tasks.resize(5 * (size_t)h->plan.tasks_per_tiling);
        uint32_t n = 0;
        build_pruned_tasks(h->plan, kept_tasks.data(), &n, &h->kept_rows);
        kept_tasks.resize(n);
        search_tpt = n;
    }
    rc = choose_launch_shape(h->plan, h->device, search_tpt, 0, &h->shape);
    if (rc) { delete h; return rc; }
    if (h->plan.row_pruning) {
        const size_t bytes = kept_tasks.size() * sizeof(PrunedTask);
        cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&h->pruned), bytes);
        if (e == cudaSuccess) e = cudaMemcpy(h->pruned, kept_tasks.data(), bytes, cudaMemcpyHostToDevice);
        if (e != cudaSuccess) {
            if (h->pruned) cudaFree(h->pruned);
            delete h;
            return cuda_status(e);
        }
        h->shape.pruned = h->pruned;
    }
    // one allocation: the search scratch, then one result record for mmee_decode
    const size_t sbytes = (scratch_bytes(h->shape.grid) + 15) / 16 * 16;
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(&h->scratch), sbytes + sizeof(mmee_result_t));
    if (e == cudaSuccess) {
        h->decode_buf = reinterpret_cast<mmee_result_t*>(reinterpret_cast<unsigned char*>(h->scratch) + sbytes);
        e = launch_reset(h->scratch, 0);
        if (e == cudaSuccess) e = cudaStreamSynchronize(0);
    }
    if (e != cudaSuccess) {
        if (h->scratch) cudaFree(h->scratch);
        if (h->pruned) cudaFree(h->pruned);
        delete h;
        return cuda_status(e);
    }
    h->create_ms = std::chrono::duration<float, std::milli>(std::chrono::steady_clock::now() - t0).count();
    *out = h;
    return MMEE_OK;
}

// The handle's device must be the current one: its scratch and tables live there, and a launch from another
// device's context would fail (or, with peer access enabled, silently run on the wrong device).
static int check_device(const mmee_handle* h) {
    int cur = -1;
    const cudaError_t e = cudaGetDevice(&cur);
    if (e != cudaSuccess) return cuda_status(e);
    return cur == h->device ? MMEE_OK : MMEE_ERR_ARG;
}

int mmee_search(mmee_handle_t* h, void* cuda_stream, mmee_result_t* out_best, mmee_result_t* out_topk) {
    if (!h || !out_best) return MMEE_ERR_ARG;
    int rc = check_device(h);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (h->dirty) {        // an earlier launch on this handle failed: the header may hold a used work counter
        if ((rc = cuda_status(launch_reset(h->scratch, st)))) return rc;
        h->dirty = false;
    }
    if (h->timing) cudaEventRecord(h->ev[0], st);
    const cudaError_t e = launch_search(h->plan, h->shape, h->device, h->scratch, nullptr, out_best, out_topk, st);
    if (e != cudaSuccess) { h->dirty = true; return cuda_status(e); }
    if (h->timing) cudaEventRecord(h->ev[1], st);
    h->last.kernels_launched = 1;
    h->last.grid = h->shape.grid;
    h->last.block = kSearchThreads;
    h->last.smem_bytes = h->shape.smem_bytes;
    h->last.tasks = (h->plan.t_end - h->plan.t_begin) * h->shape.search_tpt;
    h->last.rows_per_tiling = h->plan.rows_per_tiling;
    h->last.rows_evaluated_per_tiling = h->kept_rows;
    return MMEE_OK;
}

int mmee_search_host(mmee_handle_t* h, mmee_result_t* out_best, mmee_result_t* out_topk) {
    if (!h || !out_best) return MMEE_ERR_ARG;
    const uint32_t k = h->plan.topk;
    int rc;
    if (!h->host_out) {
        // Pinned, mapped host memory: the kernel's last CTA writes the records straight into it, so that the
        // host needs no copy call after the search, only the synchronisation.
        rc = cuda_status(cudaHostAlloc(reinterpret_cast<void**>(&h->host_out), (size_t)(1 + k) * sizeof(mmee_result_t),
                                       cudaHostAllocMapped));
        if (rc) { h->host_out = nullptr; return rc; }
    }
    mmee_result_t* dev = nullptr;
    if ((rc = cuda_status(cudaHostGetDevicePointer(reinterpret_cast<void**>(&dev), h->host_out, 0)))) return rc;
    if ((rc = mmee_search(h, nullptr, dev, dev + 1))) return rc;
    if ((rc = cuda_status(cudaStreamSynchronize(nullptr)))) return rc;
    std::memcpy(out_best, h->host_out, sizeof(mmee_result_t));
    if (out_topk) std::memcpy(out_topk, h->host_out + 1, (size_t)k * sizeof(mmee_result_t));
    return out_best->status == MMEE_ERR_CHECK ? MMEE_ERR_CHECK : MMEE_OK;
}

int mmee_destroy(mmee_handle_t* h) {
    if (!h) return MMEE_ERR_ARG;
    cudaError_t e = cudaSuccess;
    if (h->timing) for (int i = 0; i < 2; ++i) cudaEventDestroy(h->ev[i]);
    if (h->scratch) e = cudaFree(h->scratch);
    if (h->pruned) cudaFree(h->pruned);
    if (h->host_out) cudaFreeHost(h->host_out);
    delete h;
    return cuda_status(e);
}

uint64_t mmee_num_candidates(const mmee_handle_t* h) {
    return h ? h->plan.n_tilings * (uint64_t)h->plan.rows_per_tiling * 9u : 0;
}
uint64_t mmee_num_tilings(const mmee_handle_t* h) { return h ? h->plan.n_tilings : 0; }
uint64_t mmee_num_rows(const mmee_handle_t* h) { return h ? h->plan.rows_per_tiling : 0; }

const char* mmee_strerror(int status) {
    switch (status) {
        case MMEE_OK: return "ok";
        case MMEE_ERR_ARG: return "invalid argument";
        case MMEE_ERR_OVERFLOW: return "a worst-case key of this problem does not fit 62 bits";
        case MMEE_ERR_QUANTUM: return "an energy is not an integer multiple of the energy quantum";
        case MMEE_ERR_NO_FEASIBLE: return "no mapping fits the global buffer";
        case MMEE_ERR_CUDA: return "CUDA runtime error";
        case MMEE_ERR_TIMEOUT: return "device-side wait timed out";
        case MMEE_ERR_RANGE: return "request exceeds a documented maximum";
        case MMEE_ERR_CHECK: return "a winner's ranking key differs from its full evaluation";
        default: return "unknown status";
    }
}

int mmee_eval(mmee_handle_t* h, void* cuda_stream, uint64_t idx_begin, uint64_t count, mmee_result_t* out) {
    if (!h || (!out && count)) return MMEE_ERR_ARG;
    const uint64_t n = mmee_num_candidates(h);
    if (idx_begin > n || count > n - idx_begin) return MMEE_ERR_ARG;
    const int rc = check_device(h);
    if (rc) return rc;
    return cuda_status(launch_eval(h->plan, idx_begin, count, out, static_cast<cudaStream_t>(cuda_stream)));
}

int mmee_decode(mmee_handle_t* h, uint64_t idx, mmee_result_t* host_out) {
    if (!h || !host_out || idx >= mmee_num_candidates(h)) return MMEE_ERR_ARG;
    int rc = check_device(h);
    if (rc) return rc;
    if ((rc = cuda_status(launch_eval(h->plan, idx, 1, h->decode_buf, nullptr)))) return rc;
    return cuda_status(cudaMemcpy(host_out, h->decode_buf, sizeof(mmee_result_t), cudaMemcpyDeviceToHost));
}

int mmee_dump_keys(mmee_handle_t* h, void* cuda_stream, int64_t* out_keys) {
    if (!h || !out_keys || h->plan.row_pruning) return MMEE_ERR_ARG;
    const uint64_t n = (h->plan.t_end - h->plan.t_begin) * (uint64_t)h->plan.rows_per_tiling * 9u;
    if (n > (1ull << 31)) return MMEE_ERR_RANGE;
    int rc = check_device(h);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (h->dirty) {
        if ((rc = cuda_status(launch_reset(h->scratch, st)))) return rc;
        h->dirty = false;
    }
    cudaError_t e = launch_search(h->plan, h->shape, h->device, h->scratch, out_keys, nullptr, nullptr, st);
    if (e != cudaSuccess) { h->dirty = true; return cuda_status(e); }
    if ((e = launch_reset(h->scratch, st)) != cudaSuccess) { h->dirty = true; return cuda_status(e); }
    return MMEE_OK;
}

int mmee_filter_flags(mmee_handle_t* h, void* cuda_stream, int64_t threshold_key, uint8_t* out_flags) {
    if (!h || !out_flags || h->plan.row_pruning || h->plan.objective > MMEE_OBJ_EDP) return MMEE_ERR_ARG;
    int rc = check_device(h);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (h->dirty) {
        if ((rc = cuda_status(launch_reset(h->scratch, st)))) return rc;
        h->dirty = false;
    }
    const uint64_t bytes = (h->plan.t_end - h->plan.t_begin) * (uint64_t)h->plan.tasks_per_tiling * 25u;
    if ((rc = cuda_status(cudaMemsetAsync(out_flags, 0, bytes, st)))) return rc;
    Plan p = h->plan;
    p.key_cap = threshold_key;
    cudaError_t e = launch_filter_flags(p, h->shape, h->device, h->scratch, out_flags, st);
    if (e != cudaSuccess) { h->dirty = true; return cuda_status(e); }
    if ((e = launch_reset(h->scratch, st)) != cudaSuccess) { h->dirty = true; return cuda_status(e); }
    return MMEE_OK;
}

int mmee_solve_host(const mmee_workload_t* workload, const mmee_arch_t* arch, const mmee_objective_t* objective,
                    mmee_result_t* out_best, mmee_result_t* out_topk, uint64_t* h2d_bytes, uint64_t* d2h_bytes) {
    if (!out_best || !objective) return MMEE_ERR_ARG;
    mmee_handle_t* h = nullptr;
    int rc = mmee_create(workload, arch, objective, &h);
    if (rc) return rc;
    const uint32_t k = h->plan.topk;
    const size_t bytes = (size_t)(k + 1) * sizeof(mmee_result_t);
    mmee_result_t* dev = nullptr;
    if ((rc = cuda_status(cudaMalloc(reinterpret_cast<void**>(&dev), bytes)))) { mmee_destroy(h); return rc; }
    rc = mmee_search(h, nullptr, dev, dev + 1);
    if (rc == MMEE_OK) rc = cuda_status(cudaMemcpy(out_best, dev, sizeof(mmee_result_t), cudaMemcpyDeviceToHost));
    if (rc == MMEE_OK && out_topk)
        rc = cuda_status(cudaMemcpy(out_topk, dev + 1, (size_t)k * sizeof(mmee_result_t), cudaMemcpyDeviceToHost));
    // the finalize step's self-check failed: the records are not a result
    if (rc == MMEE_OK && out_best->status == MMEE_ERR_CHECK) rc = MMEE_ERR_CHECK;
    // The plan (divisor lists, query vectors, coefficients) travels to the device as the kernels'
    // parameter block: once per launch.
    if (h2d_bytes) *h2d_bytes = 2ull * sizeof(mmee::Plan);
    if (d2h_bytes) *d2h_bytes = sizeof(mmee_result_t) * (uint64_t)(1 + (out_topk ? k : 0));
    cudaFree(dev);
    const int rc2 = mmee_destroy(h);
    return rc ? rc : rc2;
}

int mmee_pareto_front(const mmee_workload_t* workload, const mmee_arch_t* arch, const mmee_objective_t* objective,
                      mmee_result_t* out_points, uint32_t capacity, uint32_t* n_points) {
    if (!objective || !n_points || (!out_points && capacity)) return MMEE_ERR_ARG;
    *n_points = 0;
    mmee_objective_t oe = *objective, ol = *objective;
    oe.objective = MMEE_OBJ_ENERGY_LCAP;  oe.topk = 1; oe.row_pruning = 0; oe.key_cap = INT64_MAX - 1;
    ol.objective = MMEE_OBJ_LATENCY_ECAP; ol.topk = 1; ol.row_pruning = 0; ol.key_cap = INT64_MAX - 1;
    mmee_handle_t *he = nullptr, *hl = nullptr;
    int rc = mmee_create(workload, arch, &oe, &he);
    if (rc) return rc;
    rc = mmee_create(workload, arch, &ol, &hl);
    if (rc) { mmee_destroy(he); return rc; }
    mmee_result_t* dev = nullptr;
    rc = cuda_status(cudaMalloc(reinterpret_cast<void**>(&dev), sizeof(mmee_result_t)));
    mmee_result_t r;
    int64_t latency_cap = INT64_MAX - 1;
    uint32_t n = 0;
    while (rc == MMEE_OK) {
        // least energy among the mappings that are still faster than the previous point
        he->plan.key_cap = latency_cap;
        if ((rc = mmee_search(he, nullptr, dev, nullptr))) break;
        if ((rc = cuda_status(cudaMemcpy(&r, dev, sizeof(r), cudaMemcpyDeviceToHost)))) break;
        if (r.idx == MMEE_NO_INDEX) break;                       // nothing faster is left
        // the fastest mapping at that energy: the point of the front, with its lowest index
        hl->plan.key_cap = r.e_key;
        if ((rc = mmee_search(hl, nullptr, dev, nullptr))) break;
        if ((rc = cuda_status(cudaMemcpy(&r, dev, sizeof(r), cudaMemcpyDeviceToHost)))) break;
        if (r.idx == MMEE_NO_INDEX) { rc = MMEE_ERR_CHECK; break; }   // cannot happen: the previous optimum qualifies
        if (n < capacity) out_points[n] = r;
        ++n;
        if (r.l_key == 0) break;
        latency_cap = r.l_key - 1;
    }
    if (dev) cudaFree(dev);
    mmee_destroy(he);
    mmee_destroy(hl);
    *n_points = n;
    if (rc == MMEE_OK && n > capacity) rc = MMEE_ERR_RANGE;
    return rc;
}

int mmee_pareto_front_bs_da(const mmee_workload_t* workload, const mmee_arch_t* arch, const mmee_objective_t* objective,
                            mmee_result_t* out_points, uint32_t capacity, uint32_t* n_points) {
    if (!arch || !objective || !n_points || (!out_points && capacity)) return MMEE_ERR_ARG;
    *n_points = 0;
    // DRAM words as the key: one quantum per DRAM word, nothing else costs anything
    mmee_arch_t a = *arch;
    a.e_dram_pj = 1.0; a.e_gb_pj = a.e_rf_pj = a.e_mac_pj = 0.0; a.c_softmax = 0.0; a.energy_quantum_pj = 1.0;
    mmee_objective_t o = *objective;
    o.objective = MMEE_OBJ_ENERGY; o.topk = 1; o.row_pruning = 0; o.key_cap = 0;
    mmee_handle_t* h = nullptr;
    int rc = mmee_create(workload, &a, &o, &h);
    if (rc) return rc;
    mmee_result_t* dev = nullptr;
    rc = cuda_status(cudaMalloc(reinterpret_cast<void**>(&dev), sizeof(mmee_result_t)));
    mmee_result_t r, held;
    bool have = false;
    uint32_t n = 0;
    // Searches with a shrinking buffer: each returns the least DRAM traffic that fits, with the buffer words its
    // mapping needs; the next one allows one word less than that.  While the traffic stays the same the mapping
    // found needs less buffer for the same traffic; when it rises, the mapping held is a point of the front.
    while (rc == MMEE_OK) {
        if ((rc = mmee_search(h, nullptr, dev, nullptr))) break;
        if ((rc = cuda_status(cudaMemcpy(&r, dev, sizeof(r), cudaMemcpyDeviceToHost)))) break;
        if (r.status == MMEE_ERR_CHECK) { rc = MMEE_ERR_CHECK; break; }
        const bool found = r.idx != MMEE_NO_INDEX;
        if (have && (!found || r.e_key != held.e_key)) {
            if (n < capacity) out_points[n] = held;
            ++n;
        }
        if (!found) break;
        held = r;
        have = true;
        if (r.bs <= 0) { if (n < capacity) out_points[n] = held; ++n; break; }      // (cannot happen: tiles take words)
        h->plan.cap_words = r.bs - 1;
    }
    if (dev) cudaFree(dev);
    mmee_destroy(h);
    *n_points = n;
    if (rc == MMEE_OK && n > capacity) rc = MMEE_ERR_RANGE;
    return rc;
}

int mmee_search_shapes(const mmee_workload_t* workload, const mmee_arch_t* arch, const mmee_objective_t* objective,
                       const uint32_t* shapes, uint32_t n_shapes, mmee_result_t* out_per_shape,
                       uint32_t* out_best_shape) {
    if (!arch || !objective || !shapes || !n_shapes || !out_per_shape || !out_best_shape) return MMEE_ERR_ARG;
    *out_best_shape = UINT32_MAX;
    mmee_objective_t o = *objective;
    o.topk = 1;
    o.row_pruning = 0;
    mmee_result_t* dev = nullptr;
    int rc = cuda_status(cudaMalloc(reinterpret_cast<void**>(&dev), sizeof(mmee_result_t)));
    if (rc) return rc;
    bool have = false;
    int64_t best_key = 0;
    for (uint32_t i = 0; i < n_shapes && rc == MMEE_OK; ++i) {
        mmee_arch_t a = *arch;
        a.pe_rows = shapes[2 * i];
        a.pe_cols = shapes[2 * i + 1];
        mmee_handle_t* h = nullptr;
        if ((rc = mmee_create(workload, &a, &o, &h))) break;
        rc = mmee_search(h, nullptr, dev, nullptr);
        if (rc == MMEE_OK)
            rc = cuda_status(cudaMemcpy(&out_per_shape[i], dev, sizeof(mmee_result_t), cudaMemcpyDeviceToHost));
        if (rc == MMEE_OK && out_per_shape[i].status == MMEE_ERR_CHECK) rc = MMEE_ERR_CHECK;
        const int rc2 = mmee_destroy(h);
        if (rc == MMEE_OK) rc = rc2;
        if (rc != MMEE_OK || out_per_shape[i].idx == MMEE_NO_INDEX) continue;
        const mmee_result_t& r = out_per_shape[i];
        // the key the search ordered by: energy, latency, or the bit pattern of the positive EDP product
        int64_t key;
        switch (o.objective) {
            case MMEE_OBJ_ENERGY: case MMEE_OBJ_ENERGY_LCAP: key = r.e_key; break;
            case MMEE_OBJ_LATENCY: case MMEE_OBJ_LATENCY_ECAP: key = r.l_key; break;
            default: std::memcpy(&key, &r.edp_key, sizeof(key)); break;
        }
        if (!have || key < best_key) { have = true; best_key = key; *out_best_shape = i; }
    }
    cudaFree(dev);
    return rc;
}

int mmee_query_vector(uint32_t metric, uint32_t phi, uint32_t pi, uint32_t operand, uint32_t beta,
                      uint32_t recompute, uint8_t out_q[8]) {
    if (!out_q || metric > 1 || phi > 2 || pi > 5 || operand > 4 || beta < 3 || beta > 7 || recompute > 1)
        return MMEE_ERR_ARG;
    QueryTables tables;
    build_query_tables(&tables);
    uint8_t q;
    if (metric == 0) {
        q = tables.bs[pi][operand][beta - 3];
    } else if (phi == 0) {
        if (operand == OP_C) return MMEE_ERR_ARG;
        q = tables.da[pi][operand][beta - 3][recompute];
    } else {
        q = tables.da_unfused[pi][operand][beta - 3];
    }
    for (int d = 0; d < 8; ++d) out_q[d] = (uint8_t)((q >> d) & 1u);
    return MMEE_OK;
}

int mmee_row_pruning_keep(const mmee_objective_t* objective, uint8_t* out_keep, uint32_t capacity,
                          uint32_t* out_rows) {
    if (!objective || !out_keep || !out_rows) return MMEE_ERR_ARG;
    // the row space depends on the objective's order set and fusion modes only: plan a unit workload
    const mmee_workload_t w = {1, 1, 1, 1, 1, 1, 1, 1};
    mmee_arch_t a;
    std::memset(&a, 0, sizeof(a));
    a.pe_rows = a.pe_cols = a.n_arrays = 1;
    a.gb_bytes = 16;
    a.dram_words_per_cycle = 1;
    a.energy_quantum_pj = 1.0;
    mmee_objective_t o = *objective;
    o.topk = 1;
    o.row_pruning = 1;
    o.t_begin = o.t_end = 0;
    Plan plan;
    const int rc = build_plan(&w, &a, &o, &plan);
    if (rc) return rc;
    *out_rows = plan.rows_per_tiling;
    if (capacity < plan.rows_per_tiling) return MMEE_ERR_RANGE;
    std::vector<PrunedTask> tasks(5 * (size_t)plan.tasks_per_tiling);
    uint32_t n = 0, kept = 0;
    build_pruned_tasks(plan, tasks.data(), &n, &kept);
    std::memset(out_keep, 0, plan.rows_per_tiling);
    for (uint32_t i = 0; i < n; ++i)
        for (uint32_t de = 0; de < 25; ++de)
            if (tasks[i].rows >> de & 1u) out_keep[tasks[i].task * 125u + tasks[i].mid * 25u + de] = 1;
    return MMEE_OK;
}

int mmee_recompute_flag(uint32_t pi, uint32_t beta_c, uint32_t* out_flag) {
    if (!out_flag || pi > 5 || beta_c < 3 || beta_c > 7) return MMEE_ERR_ARG;
    QueryTables tables;
    build_query_tables(&tables);
    *out_flag = tables.recompute[pi][beta_c - 3];
    return MMEE_OK;
}

int mmee_last_search_stats(const mmee_handle_t* h, mmee_launch_stats_t* out) {
    if (!h || !out) return MMEE_ERR_ARG;
    *out = h->last;
    out->search_ms = out->finalize_ms = -1.0f;
    out->create_ms = h->create_ms;
    out->exact_path_visits = 0;
    out->rows_tested = 0;
    if (h->last.kernels_launched) {
        unsigned long long counters[3] = {0, 0, 0};      // last_exact_visits, tested_rows, last_tested_rows
        const int rc = cuda_status(cudaMemcpy(counters, &h->scratch->last_exact_visits, sizeof(counters), cudaMemcpyDeviceToHost));
        if (rc) return rc;
        out->exact_path_visits = counters[0];
        out->rows_tested = counters[2];
    }
    if (h->timing && h->last.kernels_launched) {
        const cudaError_t e = cudaEventElapsedTime(&out->search_ms, h->ev[0], h->ev[1]);
        if (e != cudaSuccess) return cuda_status(e);
        out->finalize_ms = 0.0f;        // the finalize step runs inside the search kernel (its last CTA)
    }
    return MMEE_OK;
}

int mmee_kernel_timing(mmee_handle_t* h, int enable) {
    if (!h) return MMEE_ERR_ARG;
    if (enable && !h->timing) {
        for (int i = 0; i < 2; ++i) {
            const int rc = cuda_status(cudaEventCreate(&h->ev[i]));
            if (rc) return rc;
        }
        h->timing = true;
    } else if (!enable && h->timing) {
        for (int i = 0; i < 2; ++i) cudaEventDestroy(h->ev[i]);
        h->timing = false;
    }
    return MMEE_OK;
}

const char* mmee_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda_error); }

int mmee_alu_peak(double out[4]) {
    if (!out) return MMEE_ERR_ARG;
    return cuda_status(measure_alu_peak(out));
}

}  // extern "C"
