// C-ABI entry points (include/const_b200.h): argument checking, handle management, dispatch.
#include <algorithm>
#include <atomic>
#include <cstring>
#include <new>

#include "common.cuh"

using namespace cb;

namespace {

const const_csf *as_csf(const void *h) {
    const const_csf *c = static_cast<const const_csf *>(h);
    return (c && c->magic == kCsfMagic) ? c : nullptr;
}
const const_plan *as_plan(const void *h) {
    const const_plan *p = static_cast<const const_plan *>(h);
    return (p && p->magic == kPlanMagic) ? p : nullptr;
}

const const_operand_t *find_operand(const const_operand_t *ops, int n, const std::string &name) {
    for (int i = 0; i < n; ++i)
        if (ops[i].name && name == ops[i].name) return &ops[i];
    return nullptr;
}

// the CSF handle must have been built with the mode order the plan was checked with
bool csf_matches(const const_csf *c, const PlanDesc &d, const std::string &name, const_dtype_t dtype) {
    auto it = d.mode_orders.find(name);
    if (!c || it == d.mode_orders.end() || c->order != (int)it->second.size() || c->dtype != dtype) return false;
    const TensorRef *ref = nullptr;
    for (const TensorRef &r : d.inputs) if (r.name == name) ref = &r;
    if (!ref) return false;
    for (int l = 0; l < c->order; ++l) {
        if (c->mode_order[l] != it->second[l]) return false;
        if (c->dims[l] != d.extents.at(ref->idx[l])) return false;
    }
    return true;
}

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

std::atomic<int> g_spin_limit{0}, g_withhold{0}, g_variant{0};

}  // namespace

namespace cb {
DebugKnobs debug_knobs() { return DebugKnobs{g_spin_limit.load(), g_withhold.load(), g_variant.load()}; }
}  // namespace cb

extern "C" {

const_status_t const_csf_build(int order, const int64_t *dims, int64_t nnz, const int32_t *const *coords_dev,
                               const void *vals_dev, const_dtype_t dtype, const int *mode_order, void *stream,
                               const_csf_t **out) {
    if (!out) return CONST_ERR_INVALID_ARG;
    *out = nullptr;
    if (order < 2 || order > kMaxOrder || !dims || nnz < 0 || !coords_dev || !mode_order ||
        (dtype != CONST_F32 && dtype != CONST_F64) || (nnz > 0 && !vals_dev))
        return CONST_ERR_INVALID_ARG;
    bool seen[kMaxOrder] = {false, false, false, false};
    for (int l = 0; l < order; ++l) {
        if (mode_order[l] < 0 || mode_order[l] >= order || seen[mode_order[l]]) return CONST_ERR_INVALID_ARG;
        seen[mode_order[l]] = true;
        if (dims[l] < 1) return CONST_ERR_INVALID_ARG;
        if (nnz > 0 && !coords_dev[l]) return CONST_ERR_INVALID_ARG;
    }
    if (nnz >= 2147483647ll) return CONST_ERR_UNSUPPORTED;
    const_csf *csf = nullptr;
    const_status_t rc = csf_build_impl(order, dims, nnz, coords_dev, vals_dev, dtype, mode_order,
                                       static_cast<cudaStream_t>(stream), &csf);
    if (rc == CONST_OK) *out = csf;
    return rc;
}

const_status_t const_csf_from_dense(int order, const int64_t *dims, const void *dense_dev, const_dtype_t dtype,
                                    const int *mode_order, void *stream, const_csf_t **out) {
    if (!out) return CONST_ERR_INVALID_ARG;
    *out = nullptr;
    if (order < 2 || order > kMaxOrder || !dims || !dense_dev || !mode_order || (dtype != CONST_F32 && dtype != CONST_F64))
        return CONST_ERR_INVALID_ARG;
    bool seen[kMaxOrder] = {false, false, false, false};
    for (int l = 0; l < order; ++l) {
        if (mode_order[l] < 0 || mode_order[l] >= order || seen[mode_order[l]] || dims[l] < 1) return CONST_ERR_INVALID_ARG;
        seen[mode_order[l]] = true;
    }
    const_csf *csf = nullptr;
    const_status_t rc = csf_from_dense_impl(order, dims, dense_dev, dtype, mode_order, static_cast<cudaStream_t>(stream), &csf);
    if (rc == CONST_OK) *out = csf;
    return rc;
}

const_status_t const_csf_build_noalloc(int order, const int64_t *dims, int64_t nnz, const int32_t *const *coords_dev,
                                       const void *vals_dev, const_dtype_t dtype, const int *mode_order, void *stream,
                                       int32_t *const *pos_out_dev, int32_t *const *crd_out_dev, void *vals_out_dev,
                                       int64_t *level_sizes) {
    if (order < 2 || order > kMaxOrder || !dims || nnz < 0 || !coords_dev || !mode_order || !pos_out_dev ||
        !crd_out_dev || (dtype != CONST_F32 && dtype != CONST_F64) || (nnz > 0 && (!vals_dev || !vals_out_dev)))
        return CONST_ERR_INVALID_ARG;
    bool seen[kMaxOrder] = {false, false, false, false};
    for (int l = 0; l < order; ++l) {
        if (mode_order[l] < 0 || mode_order[l] >= order || seen[mode_order[l]]) return CONST_ERR_INVALID_ARG;
        seen[mode_order[l]] = true;
        if (dims[l] < 1 || !pos_out_dev[l] || (nnz > 0 && (!coords_dev[l] || !crd_out_dev[l]))) return CONST_ERR_INVALID_ARG;
    }
    return csf_build_noalloc_impl(order, dims, nnz, coords_dev, vals_dev, dtype, mode_order,
                                  static_cast<cudaStream_t>(stream), pos_out_dev, crd_out_dev, vals_out_dev,
                                  level_sizes);
}

const_status_t const_csf_level(const const_csf_t *h, int level, const int32_t **pos, const int32_t **crd, int64_t *n) {
    const const_csf *c = as_csf(h);
    if (!c || level < 0 || level >= c->order) return CONST_ERR_INVALID_ARG;
    if (pos) *pos = c->pos[level];
    if (crd) *crd = c->crd[level];
    if (n) *n = c->n[level];
    return CONST_OK;
}

const_status_t const_csf_values(const const_csf_t *h, const void **vals, int64_t *nnz) {
    const const_csf *c = as_csf(h);
    if (!c) return CONST_ERR_INVALID_ARG;
    if (vals) *vals = c->vals;
    if (nnz) *nnz = c->nnz;
    return CONST_OK;
}

const_status_t const_csf_set_bins(const_csf_t *h, int64_t light_max_nnz, int64_t heavy_max_nnz, int64_t chunk_nnz,
                                  void *stream) {
    const_csf *c = const_cast<const_csf *>(as_csf(h));
    if (!c) return CONST_ERR_INVALID_ARG;
    if (light_max_nnz > 0) c->light_max = light_max_nnz;
    if (heavy_max_nnz > 0) c->heavy_max = heavy_max_nnz;
    if (chunk_nnz > 0) c->chunk = chunk_nnz;
    if (c->heavy_max < c->light_max) c->heavy_max = c->light_max;
    return csf_rebin(c, static_cast<cudaStream_t>(stream));
}

const_status_t const_csf_bin_counts(const const_csf_t *h, int64_t *n_light, int64_t *n_heavy, int64_t *n_giant,
                                    int64_t *n_items) {
    const_csf *c = const_cast<const_csf *>(as_csf(h));
    if (!c) return CONST_ERR_INVALID_ARG;
    const_status_t rc = csf_bin_totals(c);
    if (rc != CONST_OK) return rc;
    if (n_light) *n_light = c->n_light;
    if (n_heavy) *n_heavy = c->n_heavy;
    if (n_giant) *n_giant = c->n_giant;
    if (n_items) *n_items = c->n_items;
    return CONST_OK;
}

const_status_t const_csf_work_lists(const const_csf_t *h, const int32_t **slice_ptr, const int32_t **light_list,
                                    int64_t *n_light, const int32_t **items, int64_t *n_items) {
    const_csf *c = const_cast<const_csf *>(as_csf(h));
    if (!c) return CONST_ERR_INVALID_ARG;
    const_status_t rc = csf_bin_totals(c);
    if (rc != CONST_OK) return rc;
    static_assert(sizeof(WorkItem) == 4 * sizeof(int32_t), "a work item is four int32");
    if (slice_ptr) *slice_ptr = c->slice_ptr;
    if (light_list) *light_list = c->light_list;
    if (n_light) *n_light = c->n_light;
    if (items) *items = reinterpret_cast<const int32_t *>(c->items);
    if (n_items) *n_items = c->n_items;
    return CONST_OK;
}

const_status_t const_plan_create(const char *expression, const char *const *tree, int n_contractions,
                                 const char *const *sparse_names, const int *const *mode_orders, int n_sparse,
                                 const char *const *loop_orders, const const_extent_t *extents, int n_indices,
                                 const_dtype_t dtype, const_plan_t **out) {
    if (!out) return CONST_ERR_INVALID_ARG;
    *out = nullptr;
    const_plan *plan = new (std::nothrow) const_plan();
    if (!plan) return CONST_ERR_INVALID_ARG;
    const_status_t rc = parse_plan(expression, tree, n_contractions, sparse_names, mode_orders, n_sparse, loop_orders,
                                   extents, n_indices, dtype, plan->desc);
    if (rc == CONST_OK) rc = check_plan(plan->desc);
    if (rc == CONST_OK) {
        // every checked schedule is compiled for the generic executor; a hand-written family, where one
        // matches, takes precedence at execute time
        plan->tree_ok = tree::compile(plan->desc, plan->tree);
        rc = match_plan(plan->desc);
        if (rc == CONST_ERR_UNSUPPORTED && plan->tree_ok) {
            plan->desc.family = Family::Tree;
            rc = CONST_OK;
        }
    }
    if (rc != CONST_OK) {
        delete plan;
        return rc;
    }
    // the order-4 TTMc kernel with the per-slice stage on the tensor cores is the faster one at rank 8
    plan->tensor_stage = plan->desc.family == Family::Ttmc4 && plan->desc.ranks[0] == 8;
    *out = plan;
    return CONST_OK;
}

const_status_t const_schedule_check(const char *expression, const char *const *tree, int n_contractions,
                                    const char *const *sparse_names, const int *const *mode_orders, int n_sparse,
                                    const char *const *loop_orders, const const_extent_t *extents, int n_indices,
                                    int *reduced_orders) {
    PlanDesc d;
    const_status_t rc = parse_plan(expression, tree, n_contractions, sparse_names, mode_orders, n_sparse, loop_orders,
                                   extents, n_indices, CONST_F32, d);
    if (rc == CONST_OK) rc = check_plan(d);
    if (rc == CONST_OK && reduced_orders)
        for (int c = 0; c < n_contractions; ++c) reduced_orders[c] = d.reduced_order[c];
    return rc;
}

const_status_t const_schedule_cin(const char *expression, const char *const *tree, int n_contractions,
                                  const char *const *sparse_names, const int *const *mode_orders, int n_sparse,
                                  const char *const *loop_orders, const const_extent_t *extents, int n_indices,
                                  int validate, char *buf, int64_t buf_len, int64_t *needed) {
    PlanDesc d;
    const_status_t rc = parse_plan(expression, tree, n_contractions, sparse_names, mode_orders, n_sparse, loop_orders,
                                   extents, n_indices, CONST_F32, d);
    if (rc == CONST_OK && validate) rc = check_plan(d);
    if (rc != CONST_OK) return rc;
    const std::string text = schedule_cin(d);
    if (needed) *needed = (int64_t)text.size() + 1;
    if (buf && buf_len > 0) {
        const size_t n = std::min<size_t>(text.size(), (size_t)buf_len - 1);
        std::memcpy(buf, text.data(), n);
        buf[n] = 0;
        if (n < text.size()) return CONST_ERR_WORKSPACE;
    }
    return CONST_OK;
}

const_status_t const_plan_reduced_order(const const_plan_t *h, int contraction, int *order) {
    const const_plan *p = as_plan(h);
    if (!p || !order || contraction < 0 || contraction >= (int)p->desc.tree.size()) return CONST_ERR_INVALID_ARG;
    *order = p->desc.reduced_order[contraction];
    return CONST_OK;
}

const char *const_plan_family(const const_plan_t *h) {
    const const_plan *p = as_plan(h);
    if (!p) return "";
    switch (p->desc.family) {
        case Family::Ttmc3: return "ttmc3";
        case Family::Ttmc4: return "ttmc4";
        case Family::Mttkrp3: return "mttkrp3";
        case Family::Network: return "network";
        case Family::Tree: return "tree";
        default: return "";
    }
}

const_status_t const_execute(const_plan_t *h, const const_operand_t *operands, int n_operands, void *out_dev,
                             void *stream_v) {
    const_plan *p = const_cast<const_plan *>(as_plan(h));
    if (!p || !operands || n_operands < 1 || !out_dev) return CONST_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const PlanDesc &d = p->desc;
    // the kernels read factor rows and write results with 128-bit accesses: refuse a pointer they would fault on
    // (checked before anything touches the device)
    if (!aligned16(out_dev)) return CONST_ERR_INVALID_ARG;
    for (int i = 0; i < n_operands; ++i)
        if (operands[i].dense_dev && !aligned16(operands[i].dense_dev)) return CONST_ERR_INVALID_ARG;
    int dev = 0;
    CB_CUDA(cudaGetDevice(&dev));
    {
        // The status word is allocated and cleared in the order of the caller's stream at the first execute,
        // so that this call stays asynchronous; an execute on another stream waits (on the device) for the clear.
        std::lock_guard<std::mutex> lock(p->mu);
        if (p->status_dev && p->device != dev) return CONST_ERR_INVALID_ARG;   // a plan stays on the device of its first use
        if (!p->status_dev) {
            int32_t *word = nullptr;
            cudaEvent_t ready = nullptr;
            CB_CUDA(cudaMallocAsync((void **)&word, sizeof(int32_t), stream));
            if (cudaMemsetAsync(word, 0, sizeof(int32_t), stream) != cudaSuccess ||
                cudaEventCreateWithFlags(&ready, cudaEventDisableTiming) != cudaSuccess ||
                cudaEventRecord(ready, stream) != cudaSuccess) {
                if (ready) cudaEventDestroy(ready);
                cudaFreeAsync(word, stream);
                return CONST_ERR_CUDA;
            }
            p->status_dev = word;
            p->status_stream = stream;
            p->status_ready = ready;
            p->device = dev;
        } else if (stream != p->status_stream) {
            CB_CUDA(cudaStreamWaitEvent(stream, p->status_ready, 0));
        }
    }
    if (d.family == Family::Tree || p->use_tree) {
        const tree::Compiled &cp = p->tree;
        const const_csf *sparse[tree::kMaxSparse] = {nullptr};
        void *global_in[tree::kMaxDense] = {nullptr};
        for (size_t s = 0; s < cp.sparse_names.size(); ++s) {
            const const_operand_t *o = find_operand(operands, n_operands, cp.sparse_names[s]);
            if (!o || !o->csf || o->dense_dev) return CONST_ERR_INVALID_ARG;
            sparse[s] = as_csf(o->csf);
            if (!csf_matches(sparse[s], d, cp.sparse_names[s], d.dtype)) return CONST_ERR_INVALID_ARG;
        }
        for (size_t g = 0; g < cp.global_names.size(); ++g) {
            if (cp.global_is_workspace[g] || (int)g == cp.result_slot) continue;
            const const_operand_t *o = find_operand(operands, n_operands, cp.global_names[g]);
            if (!o || !o->dense_dev || o->csf) return CONST_ERR_INVALID_ARG;
            global_in[g] = const_cast<void *>(o->dense_dev);
        }
        return run_tree(cp, d.dtype, sparse, global_in, out_dev, stream);
    }
    // bind operands by name
    const const_operand_t *x = find_operand(operands, n_operands, d.sparse_name);
    if (!x || !x->csf || x->dense_dev) return CONST_ERR_INVALID_ARG;
    const const_csf *X = as_csf(x->csf);
    if (!csf_matches(X, d, d.sparse_name, d.dtype)) return CONST_ERR_INVALID_ARG;
    const void *dense[3] = {nullptr, nullptr, nullptr};
    for (size_t f = 0; f < d.factor_names.size(); ++f) {
        const const_operand_t *o = find_operand(operands, n_operands, d.factor_names[f]);
        if (!o || !o->dense_dev || o->csf) return CONST_ERR_INVALID_ARG;
        dense[f] = o->dense_dev;
    }
    const int64_t n_rows = d.extents.at(d.result.idx[0]);
    switch (d.family) {
        case Family::Ttmc3:
            if (p->tensor_stage)
                return run_ttmc3_tensor(X, (const float *)dense[0], (const float *)dense[1], d.ranks[0], d.ranks[1],
                                        (float *)out_dev, n_rows, p->status_dev, stream);
            return run_ttmc3(X, (const float *)dense[0], (const float *)dense[1], d.ranks[0], d.ranks[1],
                             (float *)out_dev, n_rows, p->status_dev, stream);
        case Family::Mttkrp3:
            return run_mttkrp3(X, (const float *)dense[0], (const float *)dense[1], d.ranks[0], (float *)out_dev,
                               n_rows, p->status_dev, stream);
        case Family::Ttmc4:
            if (p->tensor_stage)
                return run_ttmc4_tensor(X, (const float *)dense[0], (const float *)dense[1], (const float *)dense[2],
                                        d.ranks[0], (float *)out_dev, n_rows, p->status_dev, stream);
            return run_ttmc4(X, (const float *)dense[0], (const float *)dense[1], (const float *)dense[2], d.ranks[0],
                             (float *)out_dev, n_rows, p->status_dev, stream);
        case Family::Network: {
            const const_operand_t *w = find_operand(operands, n_operands, d.sparse2_name);
            if (!w || !w->csf || w->dense_dev) return CONST_ERR_INVALID_ARG;
            const const_csf *W = as_csf(w->csf);
            if (!csf_matches(W, d, d.sparse2_name, d.dtype)) return CONST_ERR_INVALID_ARG;
            // level extents of U (i,k,j) and W (l,m,k)
            const int64_t n_i = X->dims[X->mode_order[0]], n_k = X->dims[X->mode_order[1]],
                          n_j = X->dims[X->mode_order[2]];
            const int64_t n_l = W->dims[W->mode_order[0]], n_m = W->dims[W->mode_order[1]];
            return run_network(X, (const double *)dense[0], W, (double *)out_dev, n_i, n_j, n_k, n_l, n_m,
                               p->status_dev, stream);
        }
        default:
            return CONST_ERR_UNSUPPORTED;
    }
}

const_status_t const_plan_set_tensor_stage(const_plan_t *h, int enable) {
    const_plan *p = const_cast<const_plan *>(as_plan(h));
    if (!p) return CONST_ERR_INVALID_ARG;
    const bool has_stage = (p->desc.family == Family::Ttmc4 && p->desc.ranks[0] == 8) ||
                           (p->desc.family == Family::Ttmc3 && p->desc.ranks[0] == 16 && p->desc.ranks[1] == 16);
    if (enable && !has_stage) return CONST_ERR_UNSUPPORTED;
    p->tensor_stage = enable ? 1 : 0;
    return CONST_OK;
}

const_status_t const_plan_describe(const const_plan_t *h, char *buf, int64_t buf_len, int64_t *needed) {
    const const_plan *p = as_plan(h);
    if (!p) return CONST_ERR_INVALID_ARG;
    if (!p->tree_ok) return CONST_ERR_UNSUPPORTED;
    const std::string text = tree::describe(p->tree);
    if (needed) *needed = (int64_t)text.size() + 1;
    if (buf && buf_len > 0) {
        const size_t n = std::min<size_t>(text.size(), (size_t)buf_len - 1);
        std::memcpy(buf, text.data(), n);
        buf[n] = 0;
        if (n < text.size()) return CONST_ERR_WORKSPACE;
    }
    return CONST_OK;
}

const_status_t const_plan_set_generic_executor(const_plan_t *h, int enable) {
    const_plan *p = const_cast<const_plan *>(as_plan(h));
    if (!p) return CONST_ERR_INVALID_ARG;
    if (enable && !p->tree_ok) return CONST_ERR_UNSUPPORTED;
    if (!enable && p->desc.family == Family::Tree) return CONST_ERR_UNSUPPORTED;   // nothing else can run this plan
    p->use_tree = enable ? 1 : 0;
    return CONST_OK;
}

const_status_t const_last_device_status(const_plan_t *h, void *stream) {
    const_plan *p = const_cast<const_plan *>(as_plan(h));
    if (!p) return CONST_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    int32_t s = 0;
    if (p->status_dev) CB_CUDA(cudaMemcpyAsync(&s, p->status_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    CB_CUDA(cudaStreamSynchronize(st));
    return (const_status_t)s;
}

void const_destroy(void *handle) {
    if (!handle) return;
    if (const const_csf *c = as_csf(handle)) {
        csf_free(const_cast<const_csf *>(c));
        return;
    }
    if (const const_plan *pc = as_plan(handle)) {
        const_plan *p = const_cast<const_plan *>(pc);
        if (p->status_dev) {
            int prev = 0;
            cudaGetDevice(&prev);
            cudaSetDevice(p->device);
            cudaFree(p->status_dev);               // waits for outstanding work, then releases the stream-ordered allocation
            if (p->status_ready) cudaEventDestroy(p->status_ready);
            cudaSetDevice(prev);
        }
        p->magic = 0;
        delete p;
    }
}

const_status_t const_debug_set(int what, int64_t value) {
    if (value < 0 || value > 0x7fffffff) return CONST_ERR_INVALID_ARG;
    switch (what) {
        case 0: g_spin_limit.store((int)value); return CONST_OK;
        case 1: g_withhold.store(value != 0); return CONST_OK;
        case 2: g_variant.store((int)value); return CONST_OK;
    }
    return CONST_ERR_INVALID_ARG;
}

const char *const_status_string(const_status_t s) {
    switch (s) {
        case CONST_OK: return "ok";
        case CONST_ERR_INVALID_ARG: return "invalid argument";
        case CONST_ERR_UNSUPPORTED: return "unsupported (no kernel family for this schedule or size)";
        case CONST_ERR_ILLEGAL_SCHEDULE: return "illegal schedule";
        case CONST_ERR_DUPLICATE_COORD: return "duplicate coordinate";
        case CONST_ERR_COORD_RANGE: return "coordinate out of range";
        case CONST_ERR_WORKSPACE: return "internal capacity exceeded";
        case CONST_ERR_CUDA: return "CUDA error";
        case CONST_ERR_TIMEOUT: return "device-side wait timed out";
    }
    return "unknown status";
}

}  // extern "C"
