// Interpreter kernel of the generic executor: walks a compiled loop tree (tree_exec.h) for any legal
// schedule, e.g. the four-tensor running example R_ijk = A_ipq B_jpr C_kqr D_jkr with its two 2-D
// workspaces fused on r and j (Fig. 5), order-4 MTTKRP, TTMc at ranks the hand-written kernels do not
// cover, the scatter form of the two-contraction network, or a network multiplied by a sparse 0/1 map
// (Sec. 5.1, Eq. 2).  Slower than the hand-written families; it exists so that every schedule the checker
// accepts can run.
#include <vector>

#include "common.cuh"
#include "tree_exec.h"

namespace cb {
namespace tree {
namespace {

constexpr int kAbsentNone = 127;

struct State {
    int32_t idx[kMaxIdx];                       // value of every bound iteration index
    int32_t node[kMaxSparse][kMaxLevels];       // CSF node of every bound level of every sparse operand
    int8_t absent[kMaxSparse];                  // level at which the operand has no node for the bound coordinates
};

// children of the node the operand stands on above `level`
__device__ __forceinline__ void child_range(const SparsePtrs &s, const State &st, int slot, int level, int32_t &lo, int32_t &hi) {
    if (level == 0) { lo = 0; hi = s.n0; return; }
    const int32_t parent = st.node[slot][level - 1];
    lo = s.pos[level][parent];
    hi = s.pos[level][parent + 1];
}

// iteration range of a loop: positions in the driver's level, or coordinates of the dense range
__device__ __forceinline__ void loop_range(const Loop &L, const Bindings &b, const State &st, int32_t &lo, int32_t &hi) {
    if (L.driver < 0) { lo = 0; hi = L.extent; return; }
    if (st.absent[L.driver] < L.level) { lo = hi = 0; return; }
    child_range(b.sp[L.driver], st, L.driver, L.level, lo, hi);
}

// Binds iteration `it` of a loop; false when a located operand has no node there (the caller decides what that means).
__device__ __forceinline__ bool bind(const Loop &L, const Bindings &b, State &st, int32_t it) {
    int32_t coord = it;
    if (L.driver >= 0) {
        coord = b.sp[L.driver].crd[L.level][it];
        st.node[L.driver][L.level] = it;
        st.absent[L.driver] = kAbsentNone;
    }
    st.idx[L.index] = coord;
    bool all = true;
    for (int f = 0; f < L.n_follow; ++f) {
        const int slot = L.follow[f], level = L.flevel[f];
        if (st.absent[slot] < level) { all = false; continue; }     // already absent further out
        int32_t lo, hi;
        child_range(b.sp[slot], st, slot, level, lo, hi);
        int32_t at = -1;
        if (lo < hi) {
            const int32_t *crd = b.sp[slot].crd[level];
            int32_t a = lo, z = hi;
            while (a < z) {
                const int32_t mid = a + (z - a) / 2;
                if (crd[mid] < coord) a = mid + 1; else z = mid;
            }
            if (a < hi && crd[a] == coord) at = a;
        }
        st.node[slot][level] = at;
        st.absent[slot] = at < 0 ? (int8_t)level : (int8_t)kAbsentNone;
        all = all && at >= 0;
    }
    return all;
}

template <typename T>
__device__ __forceinline__ int64_t address(const Ref &r, const State &st) {
    int64_t a = 0;
    for (int k = 0; k < r.n; ++k) a += (int64_t)st.idx[r.idx[k]] * r.stride[k];
    return a;
}

template <typename T>
__device__ __forceinline__ T load_ref(const Ref &r, const Program &p, const Bindings &b, const State &st, const T *scratch) {
    if (r.kind == kRefSparse) {
        const SparsePtrs &s = b.sp[r.slot];
        return static_cast<const T *>(s.vals)[st.node[r.slot][s.order - 1]];
    }
    if (r.kind == kRefPrivate) return scratch[p.ws[r.slot].offset + address<T>(r, st)];
    return static_cast<const T *>(b.global[r.slot])[address<T>(r, st)];
}

template <typename T>
__device__ __forceinline__ void update(const Stmt &s, const Program &p, const Bindings &b, const State &st, T *scratch) {
    const T v = load_ref<T>(s.lhs, p, b, st, scratch) * load_ref<T>(s.rhs, p, b, st, scratch);
    T *dst = s.out.kind == kRefPrivate ? scratch + p.ws[s.out.slot].offset : static_cast<T *>(b.global[s.out.slot]);
    atomicAdd(dst + address<T>(s.out, st), v);
}

// One assignment with its private loops: loop 0 over the warps (over all threads when it is the only one),
// loop 1 over the lanes, deeper loops in sequence.
template <typename T>
__device__ void run_statement(const Stmt &s, const Program &p, const Bindings &b, State &st, T *scratch) {
    for (int k = 0; k < s.n_sparse; ++k)
        if (st.absent[s.sparse[k]] != kAbsentNone) return;           // an operand has nothing here (uniform over the block)
    const int n = s.n_priv;
    if (n == 0) {
        if (threadIdx.x == 0) update<T>(s, p, b, st, scratch);
        return;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    int32_t cur[kMaxPriv], end[kMaxPriv];
    auto first = [&](int d) { return n == 1 ? (int)threadIdx.x : d == 0 ? warp : d == 1 ? lane : 0; };
    auto step = [&](int d) { return n == 1 ? (int)blockDim.x : d == 0 ? warps : d == 1 ? 32 : 1; };
    int d = 0;
    loop_range(p.loops[s.priv[0]], b, st, cur[0], end[0]);
    cur[0] += first(0);
    while (d >= 0) {
        if (cur[d] >= end[d]) {
            --d;
            if (d >= 0) cur[d] += step(d);
            continue;
        }
        const Loop &L = p.loops[s.priv[d]];
        if (!bind(L, b, st, cur[d])) {                                // an operand of this assignment is absent
            cur[d] += step(d);
            continue;
        }
        if (d == n - 1) {
            update<T>(s, p, b, st, scratch);
            cur[d] += step(d);
        } else {
            ++d;
            loop_range(p.loops[s.priv[d]], b, st, cur[d], end[d]);
            cur[d] += first(d);
        }
    }
    // what the private loops bound is dead now; the operands stand where the uniform loops left them
    for (int k = 0; k < s.n_sparse; ++k) st.absent[s.sparse[k]] = kAbsentNone;
}

template <typename T>
__global__ void __launch_bounds__(kThreads) tree_kernel(const __grid_constant__ Program p, const __grid_constant__ Bindings b,
                                                        int64_t root_count) {
    State st;
    for (int k = 0; k < kMaxSparse; ++k) st.absent[k] = kAbsentNone;
    T *scratch = static_cast<T *>(b.scratch) + (int64_t)blockIdx.x * p.block_scratch;
    int32_t cur[kMaxLoops], end[kMaxLoops];
    const int64_t iterations = p.root_loop < 0 ? 1 : root_count;
    for (int64_t it = blockIdx.x; it < iterations; it += gridDim.x) {
        if (p.root_loop >= 0) bind(p.loops[p.root_loop], b, st, (int32_t)it);
        int pc = 0;
        while (pc < p.n_instr) {
            const Instr in = p.instr[pc];
            if (in.op == kOpZero) {
                T *w = scratch + p.ws[in.arg].offset;
                for (int64_t e = threadIdx.x; e < p.ws[in.arg].size; e += blockDim.x) w[e] = T(0);
                __syncthreads();
                ++pc;
            } else if (in.op == kOpStmt) {
                run_statement<T>(p.stmts[in.arg], p, b, st, scratch);
                __syncthreads();
                ++pc;
            } else if (in.op == kOpLoopBegin) {
                const Loop &L = p.loops[in.arg];
                loop_range(L, b, st, cur[in.arg], end[in.arg]);
                if (cur[in.arg] >= end[in.arg]) { pc = in.jump; continue; }
                bind(L, b, st, cur[in.arg]);
                ++pc;
            } else {                                                  // kOpLoopEnd
                if (++cur[in.arg] < end[in.arg]) {
                    bind(p.loops[in.arg], b, st, cur[in.arg]);
                    pc = in.jump;
                } else {
                    ++pc;
                }
            }
        }
    }
}

}  // namespace
}  // namespace tree

// Runs the compiled programs of a plan.  sparse[slot] / dense[slot] are the operands bound by name.
const_status_t run_tree(const tree::Compiled &cp, const_dtype_t dtype, const const_csf *const *sparse,
                        void *const *global_in, void *out_dev, cudaStream_t stream) {
    using namespace tree;
    const size_t esize = dtype == CONST_F32 ? 4 : 8;
    Bindings b;
    std::memset(&b, 0, sizeof(b));
    for (size_t s = 0; s < cp.sparse_names.size(); ++s) {
        const const_csf *c = sparse[s];
        for (int l = 0; l < c->order; ++l) { b.sp[s].pos[l] = c->pos[l]; b.sp[s].crd[l] = c->crd[l]; }
        b.sp[s].vals = c->vals;
        b.sp[s].n0 = (int32_t)c->n[0];
        b.sp[s].order = c->order;
    }
    // global workspaces behind one another in one stream-ordered allocation, cleared; the result is cleared too
    int64_t shared_elems = 0;
    for (size_t g = 0; g < cp.global_names.size(); ++g)
        if (cp.global_is_workspace[g]) shared_elems += (cp.global_elems[g] + 1) / 2 * 2;
    constexpr int64_t kScratchBudget = 1ll << 30;                     // bytes of private workspace over all blocks
    int sms = 148;
    {
        int dev = 0;
        CB_CUDA(cudaGetDevice(&dev));
        CB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    }
    std::vector<int64_t> grids, counts;
    int64_t private_bytes = 0;
    for (size_t r = 0; r < cp.programs.size(); ++r) {
        const Program &p = cp.programs[r];
        int64_t count = 1;
        if (p.root_loop >= 0) count = cp.root_driver[r] >= 0 ? sparse[cp.root_driver[r]]->n[0] : cp.root_extent[r];
        int64_t grid = std::max<int64_t>(1, std::min<int64_t>(count, (int64_t)sms * 8));
        const int64_t per_block = p.block_scratch * (int64_t)esize;
        if (per_block > kScratchBudget) return CONST_ERR_WORKSPACE;
        if (per_block > 0) grid = std::min<int64_t>(grid, std::max<int64_t>(1, kScratchBudget / per_block));
        grids.push_back(grid);
        counts.push_back(count);
        private_bytes = std::max<int64_t>(private_bytes, grid * per_block);
    }
    const int64_t total_bytes = shared_elems * (int64_t)esize + private_bytes + 256;
    unsigned char *scratch = nullptr;
    CB_CUDA(cudaMallocAsync((void **)&scratch, (size_t)total_bytes, stream));
    cudaError_t e = cudaMemsetAsync(scratch, 0, (size_t)(shared_elems * (int64_t)esize), stream);
    int64_t at = 0;
    for (size_t g = 0; g < cp.global_names.size(); ++g) {
        if (cp.global_is_workspace[g]) {
            b.global[g] = scratch + at * (int64_t)esize;
            at += (cp.global_elems[g] + 1) / 2 * 2;
        } else if ((int)g == cp.result_slot) {
            b.global[g] = out_dev;
        } else {
            b.global[g] = global_in[g];
        }
    }
    b.scratch = scratch + (shared_elems * (int64_t)esize + 255) / 256 * 256;
    if (e == cudaSuccess)                                             // "R[*] = 0" precedes the nest
        e = cudaMemsetAsync(out_dev, 0, (size_t)cp.global_elems[(size_t)cp.result_slot] * esize, stream);
    for (size_t r = 0; r < cp.programs.size() && e == cudaSuccess; ++r) {
        if (counts[r] == 0) continue;
        CB_LAUNCH("tree_kernel", stream, {
            if (dtype == CONST_F32)
                tree_kernel<float><<<(unsigned)grids[r], kThreads, 0, stream>>>(cp.programs[r], b, counts[r]);
            else
                tree_kernel<double><<<(unsigned)grids[r], kThreads, 0, stream>>>(cp.programs[r], b, counts[r]);
        });
        e = cudaGetLastError();
    }
    cudaFreeAsync(scratch, stream);
    return e == cudaSuccess ? CONST_OK : CONST_ERR_CUDA;
}

}  // namespace cb
