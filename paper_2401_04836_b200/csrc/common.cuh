// Shared declarations of the CUDA library: handles, work items, small device helpers.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>
#include <cstring>
#include <mutex>
#include <string>

#include "../../include/const_b200.h"
#include "plan.h"
#include "tree_exec.h"

namespace cb {

constexpr uint32_t kCsfMagic = 0x31465343u;   // "CSF1"
constexpr uint32_t kPlanMagic = 0x314e4c50u;  // "PLN1"
constexpr int kMaxOrder = 4;

// One thread-block work item of the fused kernels.
//   kind 0: a group of light slices, one per warp: `slice` = first index into the light list, f0 = how many
//   kind 1: a whole slice handled by one block: level-1 nodes [f0, f1); result stored directly
//   kind 2: a chunk of a giant slice: level-1 nodes [f0, f1); result added atomically
struct WorkItem {
    int32_t slice;
    int32_t f0;
    int32_t f1;
    int32_t kind;
};

constexpr int kItemLight = 0, kItemBlock = 1, kItemChunk = 2;
constexpr int kWarpsPerBlock = 2;             // fused kernels run 64-thread blocks (small blocks keep warp slots busy)

// Number of work items, from the totals the load balancer left on the device.  The fused kernels are
// launched with an upper bound of it as their grid (the host never waits for the exact figure) and
// blocks beyond it return at once.
__device__ __forceinline__ int32_t work_item_count(const int32_t *__restrict__ totals) {
    return totals[0] + (totals[1] + kWarpsPerBlock - 1) / kWarpsPerBlock;
}

}  // namespace cb

// The public opaque handles.
struct const_csf {
    uint32_t magic = cb::kCsfMagic;
    int order = 0;
    const_dtype_t dtype = CONST_F32;
    int64_t dims[cb::kMaxOrder] = {0, 0, 0, 0};
    int mode_order[cb::kMaxOrder] = {0, 0, 0, 0};
    int64_t nnz = 0;
    int64_t n[cb::kMaxOrder] = {0, 0, 0, 0};            // nodes per level
    int32_t *pos[cb::kMaxOrder] = {nullptr, nullptr, nullptr, nullptr};
    int32_t *crd[cb::kMaxOrder] = {nullptr, nullptr, nullptr, nullptr};
    void *vals = nullptr;
    // load balancing
    int32_t *slice_ptr = nullptr;      // [n0 + 1] leaf offset of every root-level slice
    int32_t *light_list = nullptr;     // [n0] slice ids handled one per warp (the first n_light entries are used)
    cb::WorkItem *items = nullptr;     // [item_cap] (the first n_items entries are used)
    int32_t *bin_scratch = nullptr;    // [2 * (n0 + 1) + 8 + 64] scan outputs, size-class bases and fill counters
    const int32_t *bin_totals = nullptr;   // device: {block items of heavy and giant slices, n_light, n_heavy, n_giant}
    int64_t item_cap = 0;              // upper bound of n_items, known without asking the device: the launch grid
    // host copies of the totals, fetched on first request (csf_bin_totals): nothing on the execute path needs them
    bool totals_on_host = false;
    int64_t n_light = 0, n_heavy = 0, n_giant = 0, n_items = 0;
    int64_t light_max = 0, heavy_max = 0, chunk = 0;
    cudaStream_t stream = nullptr;     // stream of the build: the arrays are freed in its order
    cudaStream_t bin_stream = nullptr; // stream of the last (re)binning
    int device = 0;
};

struct const_plan {
    uint32_t magic = cb::kPlanMagic;
    cb::PlanDesc desc;
    int32_t *status_dev = nullptr;     // device status word written by kernels (allocated at the first execute)
    cudaStream_t status_stream = nullptr;   // stream that allocated and cleared it
    cudaEvent_t status_ready = nullptr;     // recorded behind the clear: other streams wait for it
    int tensor_stage = 0;              // run the dense per-slice stage on the tensor cores where a kernel has one
    cb::tree::Compiled tree;           // programs of the generic executor (compiled for every plan it can run)
    bool tree_ok = false;
    int use_tree = 0;                  // run the generic executor although a hand-written family matches
    int device = -1;
    std::mutex mu;                     // first-use set-up of the status word
};

namespace cb {

#define CB_CUDA(call)                                         \
    do {                                                      \
        cudaError_t _e = (call);                              \
        if (_e != cudaSuccess) return CONST_ERR_CUDA;         \
    } while (0)

// Runs `f` (typically a cudaFuncSetAttribute) once per device, whichever host thread gets there first.
struct PerDeviceOnce {
    std::mutex mu;
    bool done[64] = {};
};
template <class F>
inline cudaError_t once_per_device(PerDeviceOnce &o, F f) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(o.mu);
    const bool tracked = dev >= 0 && dev < 64;
    if (tracked && o.done[dev]) return cudaSuccess;
    e = f();
    if (e == cudaSuccess && tracked) o.done[dev] = true;
    return e;
}

// profile.cu: brackets a kernel launch with two events when profiling is on (no-op otherwise)
class ProfScope {
public:
    ProfScope(const char *name, cudaStream_t stream);
    ~ProfScope();
    ProfScope(const ProfScope &) = delete;
    ProfScope &operator=(const ProfScope &) = delete;
private:
    cudaStream_t stream_;
    long idx_;
};
#define CB_LAUNCH(name, stream, ...)             \
    do {                                         \
        cb::ProfScope _prof(name, stream);       \
        __VA_ARGS__;                             \
    } while (0)

// Test hooks (const_debug_set): limits of the bounded device-side waits and a switch that withholds the
// signal those waits are waiting for, so that a test can see a wait run out.  0 = library defaults.
struct DebugKnobs {
    int spin_limit;      // polls before a wait gives up (0: the kernel's own default)
    int withhold;        // nonzero: producers do not publish / the tensor-core stage does not commit
    int variant;         // kernel variant to launch where a launcher keeps several for measurement (0: the default)
};
DebugKnobs debug_knobs();

// csf_build.cu
const_status_t csf_build_impl(int order, const int64_t *dims, int64_t nnz, const int32_t *const *coords_dev,
                              const void *vals_dev, const_dtype_t dtype, const int *mode_order,
                              cudaStream_t stream, const_csf **out);
const_status_t csf_from_dense_impl(int order, const int64_t *dims, const void *dense, const_dtype_t dtype,
                                   const int *mode_order, cudaStream_t stream, const_csf **out);
const_status_t csf_rebin(const_csf *csf, cudaStream_t stream);
const_status_t csf_bin_totals(const_csf *csf);      // fills the host copies n_light .. n_items (waits for the device once)
void csf_free(const_csf *csf);
const_status_t csf_build_noalloc_impl(int order, const int64_t *dims, int64_t nnz, const int32_t *const *coords_dev,
                                      const void *vals_dev, const_dtype_t dtype, const int *mode_order,
                                      cudaStream_t stream, int32_t *const *pos_out, int32_t *const *crd_out,
                                      void *vals_out, int64_t *level_sizes);

// chain_kernels.cu
const_status_t run_ttmc3(const const_csf *X, const float *U, const float *V, int R2, int R3, float *Y,
                         int64_t n_rows, int32_t *status, cudaStream_t stream);
const_status_t run_mttkrp3(const const_csf *X, const float *B, const float *C, int R, float *A,
                           int64_t n_rows, int32_t *status, cudaStream_t stream);
const_status_t run_ttmc4(const const_csf *X, const float *U, const float *V, const float *W, int R, float *Y,
                         int64_t n_rows, int32_t *status, cudaStream_t stream);
// ttmc4_tc_kernel.cu: the same contraction with the per-slice dense stage on the tensor cores
const_status_t run_ttmc4_tensor(const const_csf *X, const float *U, const float *V, const float *W, int R, float *Y,
                                int64_t n_rows, int32_t *status, cudaStream_t stream);
// chain3_tc_kernel.cu: order-3 TTMc at rank 16 x 16 with the per-slice dense stage on the tensor cores
const_status_t run_ttmc3_tensor(const const_csf *X, const float *U, const float *V, int R2, int R3, float *Y,
                                int64_t n_rows, int32_t *status, cudaStream_t stream);
// network_kernels.cu
const_status_t run_network(const const_csf *U, const double *V, const const_csf *W, double *Z,
                           int64_t n_i, int64_t n_j, int64_t n_k, int64_t n_l, int64_t n_m,
                           int32_t *status, cudaStream_t stream);

// tree_kernel.cu: the generic executor; sparse[slot] and global_in[slot] follow cp.sparse_names / cp.global_names
const_status_t run_tree(const tree::Compiled &cp, const_dtype_t dtype, const const_csf *const *sparse,
                        void *const *global_in, void *out_dev, cudaStream_t stream);

}  // namespace cb
