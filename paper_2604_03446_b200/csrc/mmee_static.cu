// mmee_search_static: the search without any device allocation (declared in include/mmee.h).
//
// Who needs this.  Some programs that embed the library cannot let it allocate device memory:
// a serving process that has handed the whole device to its own memory pool, so that a
// cudaMalloc issued by a library simply fails; or a latency-critical loop in which the implicit
// device-wide synchronisation of cudaMalloc / cudaFree would stall every other stream.  For them
// the work counter, the shared pruning bound and the per-CTA partial top-k lists -- the scratch
// that mmee_create otherwise allocates per handle -- live in one fixed array that is part of the
// library image.  Every device that loads the library carries that array until the process exits.
#include <cuda_runtime.h>

#include <mutex>

#include "mmee_search.h"

namespace {

using namespace mmee;

constexpr uint32_t kStaticMaxCtas = 512;       // persistent CTAs the fixed scratch has room for
constexpr int kMaxDevices = 64;
constexpr size_t kStaticScratchBytes = sizeof(Scratch) + (size_t)(kStaticMaxCtas - 1) * sizeof(Partial);

// 139 296 bytes on every device that loads the library.
static_assert(kStaticScratchBytes == 139296, "documented size of the fixed scratch");
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
Scratch* g_scratch_of_device[kMaxDevices];     // device address of the array, per device; null = not set up

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the
// address that kernels may use has to be asked for, with the device in question current.
int static_scratch(int device, Scratch** out) {
    if (device < 0 || device >= kMaxDevices) return MMEE_ERR_RANGE;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_of_device[device]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) return MMEE_ERR_CUDA;
        g_scratch_of_device[device] = static_cast<Scratch*>(ptr);
    }
    *out = g_scratch_of_device[device];
    return MMEE_OK;
}

// Same launch shape as a handle would get, but bounded by what the fixed scratch can hold.
int static_shape(const Plan& p, int device, LaunchShape* shape) {
    int sm_count = 0, smem_optin = 0;
    if (cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, device) != cudaSuccess)
        return MMEE_ERR_CUDA;
    shape->range_tasks = 3 * kWorkerThreads;
    shape->search_tpt = p.tasks_per_tiling;
    shape->pad = 0;
    shape->pruned = nullptr;
    shape->slots = (shape->range_tasks - 1) / p.tasks_per_tiling + 2;
    size_t smem = search_smem_bytes(p, shape->slots);
    while (smem > 110 * 1024 && shape->range_tasks > 32) {
        shape->range_tasks -= shape->range_tasks > (uint32_t)kWorkerThreads ? kWorkerThreads : 32;
        shape->slots = (shape->range_tasks - 1) / p.tasks_per_tiling + 2;
        smem = search_smem_bytes(p, shape->slots);
    }
    if (smem > (size_t)smem_optin) return MMEE_ERR_RANGE;
    shape->smem_bytes = (uint32_t)smem;
    int per_sm = 0;
    if (search_occupancy(p, smem, &per_sm) != cudaSuccess || per_sm < 1) return MMEE_ERR_CUDA;
    if (per_sm > 2) per_sm = 2;
    const uint64_t tasks = (p.t_end - p.t_begin) * p.tasks_per_tiling;
    const uint64_t ranges = (tasks + shape->range_tasks - 1) / shape->range_tasks;
    uint64_t grid = (uint64_t)sm_count * (uint32_t)per_sm;
    if (grid > ranges) grid = ranges ? ranges : 1;
    // The scratch need grows with the number of persistent CTAs, which grows with the SM count:
    // a device too large for the fixed array is refused rather than silently under-used.
    if (grid > kStaticMaxCtas) return MMEE_ERR_RANGE;
    shape->grid = (uint32_t)grid;
    shape->n_ranges = ranges;
    uint64_t stride = ranges > 2 ? (uint64_t)((double)ranges * 0.6180339887498949) : 1;
    if (stride < 1) stride = 1;
    auto gcd = [](uint64_t a, uint64_t b) { while (b) { const uint64_t t = a % b; a = b; b = t; } return a; };
    while (ranges > 1 && gcd(stride, ranges) != 1) ++stride;
    shape->range_stride = ranges > 1 ? stride % ranges : 0;
    if (ranges > 1 && shape->range_stride == 0) shape->range_stride = 1;
    return MMEE_OK;
}

}  // namespace

extern "C" int mmee_search_static(const mmee_workload_t* workload, const mmee_arch_t* arch,
                                  const mmee_objective_t* objective, void* cuda_stream,
                                  mmee_result_t* out_best, mmee_result_t* out_topk) {
    if (!out_best) return MMEE_ERR_ARG;
    Plan plan;
    int rc = build_plan(workload, arch, objective, &plan);      // host only
    if (rc) return rc;
    if (plan.row_pruning) return MMEE_ERR_ARG;      // the kept-task list would need a device allocation
    int device = 0;
    if (cudaGetDevice(&device) != cudaSuccess) return MMEE_ERR_CUDA;
    LaunchShape shape;
    if ((rc = static_shape(plan, device, &shape))) return rc;
    Scratch* scratch = nullptr;
    if ((rc = static_scratch(device, &scratch))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // The array keeps whatever the previous call left in it.  The header (work counter, feasible
    // count, pruning bound) must start clean; the partial lists need no clearing, every CTA of
    // this launch overwrites its own before the finalize kernel reads them.
    if (launch_reset(scratch, st) != cudaSuccess) return MMEE_ERR_CUDA;
    if (launch_search(plan, shape, scratch, nullptr, st) != cudaSuccess) return MMEE_ERR_CUDA;
    if (launch_finalize(plan, scratch, (int)shape.grid, out_best, out_topk, st) != cudaSuccess) return MMEE_ERR_CUDA;
    return MMEE_OK;
}
