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

// 139 328 bytes on every device that loads the library.
static_assert(kStaticScratchBytes == 139328, "documented size of the fixed scratch");
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::mutex g_setup_mutex;
Scratch* g_scratch_of_device[kMaxDevices];     // device address of the array, per device; null = not set up

// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the
// address that kernels may use has to be asked for, with the device in question current.  The
// address is kept for the life of the process; after a cudaDeviceReset it would be stale.
int static_scratch(int device, Scratch** out) {
    if (device < 0 || device >= kMaxDevices) return MMEE_ERR_RANGE;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_of_device[device]) {
        void* ptr = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return cuda_status(e);
        if (!ptr) return cuda_status(cudaErrorInvalidSymbol);
        g_scratch_of_device[device] = static_cast<Scratch*>(ptr);
    }
    *out = g_scratch_of_device[device];
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
    if ((rc = cuda_status(cudaGetDevice(&device)))) return rc;
    // The same launch shape as a handle would get, bounded by what the fixed scratch can hold.
    LaunchShape shape;
    if ((rc = choose_launch_shape(plan, device, plan.tasks_per_tiling, kStaticMaxCtas, &shape))) return rc;
    Scratch* scratch = nullptr;
    if ((rc = static_scratch(device, &scratch))) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // The array keeps whatever the previous call left in it.  The header (work counter, feasible
    // count, pruning bound) must start clean; the partial lists need no clearing, every CTA of
    // this launch overwrites its own before the finalize step reads them.
    if ((rc = cuda_status(launch_reset(scratch, st)))) return rc;
    return cuda_status(launch_search(plan, shape, device, scratch, nullptr, out_best, out_topk, st));
}
