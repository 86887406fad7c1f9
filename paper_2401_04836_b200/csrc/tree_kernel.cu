// Interpreter kernel of the generic executor: walks a compiled loop tree (tree_exec.h) for any legal
// schedule, e.g. the four-tensor running example R_ijk = A_ipq B_jpr C_kqr D_jkr with its two 2-D
// workspaces fused on r and j (Fig. 5), order-4 MTTKRP, TTMc at ranks the hand-written kernels do not
// cover, the scatter form of the two-contraction network, or a network multiplied by a sparse 0/1 map
// (Sec. 5.1, Eq. 2).  Slower than the hand-written families; it exists so that every schedule the checker
// accepts can run.  One iteration of the outermost fused loop (of the two outermost, when both walk the same
// operand) goes to a block, or to a warp when its workspaces are small; the workspaces live in shared memory
// when they fit there.
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

// Who executes one iteration of the loops spread over the grid: a whole block, or (for small workspaces, where
// the work of one iteration is small too) one warp of it, eight iterations in flight per block.
template <bool WARP>
struct Group {
    static __device__ __forceinline__ int tid() { return WARP ? (int)(threadIdx.x & 31) : (int)threadIdx.x; }
    static __device__ __forceinline__ int size() { return WARP ? 32 : (int)blockDim.x; }
    static __device__ __forceinline__ int warp() { return WARP ? 0 : (int)(threadIdx.x >> 5); }
    static __device__ __forceinline__ int warps() { return WARP ? 1 : (int)(blockDim.x >> 5); }
    static __device__ __forceinline__ void sync() {
        if (WARP) __syncwarp();
        else __syncthreads();
    }
};

// One assignment with its private loops: loop 0 over the warps of the group (over all its threads when it is
// the only one), loop 1 over the lanes, deeper loops in sequence.  A dense innermost loop is first merged
// with the loop around it (Stmt::fuse_tail), so that short sparse ranges still fill the lanes.
template <typename T, bool WARP>
__device__ void run_statement(const Stmt &s, const Program &p, const Bindings &b, State &st, T *scratch) {
    using G = Group<WARP>;
    for (int k = 0; k < s.n_sparse; ++k)
        if (st.absent[s.sparse[k]] != kAbsentNone) return;           // an operand has nothing here (uniform over the group)
    const int n = s.n_priv;
    if (n == 0) {
        if (G::tid() == 0) update<T>(s, p, b, st, scratch);
        return;
    }
    const int lane = threadIdx.x & 31, warp = G::warp(), warps = G::warps();
    // m loops as they are dealt out: with fuse_tail the two innermost count as one, over (outer range) x (inner extent)
    const bool fuse = s.fuse_tail != 0;
    const int m = fuse ? n - 1 : n;
    const int32_t inner_extent = fuse ? p.loops[s.priv[n - 1]].extent : 1;
    int32_t cur[kMaxPriv], end[kMaxPriv];
    auto first = [&](int d) { return m == 1 ? G::tid() : d == 0 ? warp : d == 1 ? lane : 0; };
    auto step = [&](int d) { return m == 1 ? G::size() : d == 0 ? warps : d == 1 ? 32 : 1; };
    auto open = [&](int d) {                                        // range of dealt loop d (not the innermost) under the current bindings
        loop_range(p.loops[s.priv[d]], b, st, cur[d], end[d]);
        cur[d] += first(d);
    };
    // ---- the innermost dealt loop, entered with every loop around it bound
    auto innermost = [&]() {
        const int dl = m - 1;
        const Loop &LB = p.loops[s.priv[n - 1]];
        const Loop &LA = p.loops[s.priv[fuse ? n - 2 : n - 1]];           // the loop whose range is walked
        int32_t lo, hi;
        loop_range(LA, b, st, lo, hi);
        const int32_t f = first(dl), stp = step(dl);
        if (!s.fast) {                                                    // an operand is located per iteration
            if (fuse) {
                const int32_t total = (hi - lo) * inner_extent;
                for (int32_t c = f; c < total; c += stp) {
                    if (!bind(LA, b, st, lo + c / inner_extent)) continue;
                    bind(LB, b, st, c % inner_extent);
                    update<T>(s, p, b, st, scratch);
                }
            } else {
                for (int32_t it = lo + f; it < hi; it += stp)
                    if (bind(LB, b, st, it)) update<T>(s, p, b, st, scratch);
            }
            return;
        }
        // No operand is located here: every reference is affine in the two coordinates and positions
        // (Stmt::sA, sB, pA, pB), so the loop needs no bindings and no index-by-index addresses.
        st.idx[LB.index] = 0;
        if (fuse) st.idx[LA.index] = 0;
        const Ref *refs[3] = {&s.out, &s.lhs, &s.rhs};
        const T *ptr[3];
        int64_t base[3];
#pragma unroll
        for (int r = 0; r < 3; ++r) {
            const Ref &ref = *refs[r];
            if (ref.kind == kRefSparse) {
                const SparsePtrs &sp = b.sp[ref.slot];
                ptr[r] = static_cast<const T *>(sp.vals);
                base[r] = (s.pA[r] | s.pB[r]) ? 0 : st.node[ref.slot][sp.order - 1];
            } else {
                ptr[r] = ref.kind == kRefPrivate ? scratch + p.ws[ref.slot].offset : static_cast<const T *>(b.global[ref.slot]);
                base[r] = address<T>(ref, st);
            }
        }
        T *dst = const_cast<T *>(ptr[0]);
        const int32_t *crdA = LA.driver >= 0 ? b.sp[LA.driver].crd[LA.level] : nullptr;
        auto one = [&](int32_t itA, int32_t cA, int32_t itB, int32_t cB) {
            int64_t at[3];
#pragma unroll
            for (int r = 0; r < 3; ++r)
                at[r] = base[r] + (int64_t)cA * s.sA[r] + (int64_t)cB * s.sB[r] + (int64_t)itA * s.pA[r] + (int64_t)itB * s.pB[r];
            atomicAdd(dst + at[0], ptr[1][at[1]] * ptr[2][at[2]]);
        };
        if (fuse) {
            const int32_t total = (hi - lo) * inner_extent;
            int32_t qa = f / inner_extent, qb = f % inner_extent;          // place in the outer range, inner coordinate
            const int32_t da = stp / inner_extent, db = stp % inner_extent;
            for (int32_t c = f; c < total; c += stp) {
                const int32_t itA = lo + qa;
                one(itA, crdA ? crdA[itA] : itA, 0, qb);
                qa += da;
                qb += db;
                if (qb >= inner_extent) { qb -= inner_extent; ++qa; }
            }
        } else {
            for (int32_t it = lo + f; it < hi; it += stp) one(0, 0, it, crdA ? crdA[it] : it);
        }
    };
    if (m == 1) {
        innermost();
    } else {
        int d = 0;
        open(0);
        while (d >= 0) {
            if (cur[d] >= end[d]) {
                --d;
                if (d >= 0) cur[d] += step(d);
                continue;
            }
            if (!bind(p.loops[s.priv[d]], b, st, cur[d])) {               // an operand of this assignment is absent
                cur[d] += step(d);
                continue;
            }
            if (d == m - 2) {
                innermost();
                cur[d] += step(d);
            } else {
                ++d;
                open(d);
            }
        }
    }
    // what the private loops bound is dead now; the operands stand where the uniform loops left them
    for (int k = 0; k < s.n_sparse; ++k) st.absent[s.sparse[k]] = kAbsentNone;
}

// The instructions of one iteration of the loops spread over the grid.
template <typename T, bool WARP>
__device__ void run_body(const Program &p, const Bindings &b, State &st, T *scratch) {
    using G = Group<WARP>;
    int32_t cur[kMaxLoops], end[kMaxLoops];
    int pc = 0;
    while (pc < p.n_instr) {
        const Instr in = p.instr[pc];
        if (in.op == kOpZero) {
            T *w = scratch + p.ws[in.arg].offset;
            for (int64_t e = G::tid(); e < p.ws[in.arg].size; e += G::size()) w[e] = T(0);
            G::sync();
            ++pc;
        } else if (in.op == kOpStmt) {
            run_statement<T, WARP>(p.stmts[in.arg], p, b, st, scratch);
            G::sync();
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

// root_count: iterations of the loops spread over the grid (level-1 nodes of the driving operand when two
// loops are spread together).  Groups take runs of `chunk` consecutive iterations, so that the level-0 node
// above a level-1 node is searched for once per run and followed from there.
// local_scratch: the private workspaces of a group live in shared memory (b.scratch is then unused).
template <typename T, bool WARP>
__global__ void __launch_bounds__(kThreads) tree_kernel(const __grid_constant__ Program p, const __grid_constant__ Bindings b,
                                                        int64_t root_count, int32_t chunk, int32_t local_scratch) {
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    State st;
    for (int k = 0; k < kMaxSparse; ++k) st.absent[k] = kAbsentNone;
    const int groups_per_block = WARP ? (int)(blockDim.x >> 5) : 1;
    const int group_in_block = WARP ? (int)(threadIdx.x >> 5) : 0;
    const int64_t group = (int64_t)blockIdx.x * groups_per_block + group_in_block;
    const int64_t groups = (int64_t)gridDim.x * groups_per_block;
    T *scratch = local_scratch ? reinterpret_cast<T *>(dyn_smem) + (int64_t)group_in_block * p.block_scratch
                               : static_cast<T *>(b.scratch) + group * p.block_scratch;
    const int64_t iterations = p.root_loop < 0 ? 1 : root_count;
    for (int64_t run = group * chunk; run < iterations; run += groups * chunk) {
        const int64_t run_end = run + chunk < iterations ? run + chunk : iterations;
        int32_t above = -1;                                           // level-0 node over the current level-1 node
        for (int64_t it = run; it < run_end; ++it) {
            if (p.root_loop2 >= 0) {
                const Loop &L0 = p.loops[p.root_loop];
                const int32_t *pos1 = b.sp[L0.driver].pos[1];
                int32_t at = above;
                if (at < 0) {                                         // largest node whose children start at or before `it`
                    int32_t lo = 0, hi = b.sp[L0.driver].n0 - 1;
                    while (lo < hi) {
                        const int32_t mid = lo + (hi - lo + 1) / 2;
                        if ((int64_t)pos1[mid] <= it) lo = mid; else hi = mid - 1;
                    }
                    at = lo;
                } else {
                    while ((int64_t)pos1[at + 1] <= it) ++at;         // ends: the last entry of pos1 is the node count
                }
                if (at != above) bind(L0, b, st, at);
                above = at;
                bind(p.loops[p.root_loop2], b, st, (int32_t)it);
            } else if (p.root_loop >= 0) {
                bind(p.loops[p.root_loop], b, st, (int32_t)it);
            }
            run_body<T, WARP>(p, b, st, scratch);
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
    // per program: who runs an iteration (block or warp), where its workspaces live, how the iterations are dealt out
    constexpr int64_t kWarpScratchBytes = 4096;                       // up to here an iteration goes to one warp
    constexpr int64_t kLocalScratchBytes = 96 * 1024;                 // up to here the workspaces live in shared memory
    constexpr int kWarpsPerBlock = kThreads / 32;
    struct Launch { int64_t grid, count; int chunk; bool warp, local; size_t smem; };
    std::vector<Launch> launches;
    int64_t private_bytes = 0;
    for (size_t r = 0; r < cp.programs.size(); ++r) {
        const Program &p = cp.programs[r];
        Launch L{};
        L.count = 1;
        if (p.root_loop >= 0) {
            const int drv = cp.root_driver[r];
            L.count = drv < 0 ? cp.root_extent[r] : sparse[drv]->n[p.root_loop2 >= 0 ? 1 : 0];
        }
        const int64_t per_group = p.block_scratch * (int64_t)esize;
        if (per_group > kScratchBudget) return CONST_ERR_WORKSPACE;
        L.warp = p.root_loop >= 0 && p.n_instr > 1 && per_group <= kWarpScratchBytes;
        const int groups_per_block = L.warp ? kWarpsPerBlock : 1;
        L.local = per_group * groups_per_block <= kLocalScratchBytes;
        L.smem = L.local ? (size_t)(per_group * groups_per_block) : 0;
        L.grid = std::max<int64_t>(1, std::min<int64_t>((L.count + groups_per_block - 1) / groups_per_block, (int64_t)sms * 8));
        if (!L.local) {
            L.grid = std::min<int64_t>(L.grid, std::max<int64_t>(1, kScratchBudget / per_group));
            private_bytes = std::max<int64_t>(private_bytes, L.grid * per_group);
        }
        // runs of consecutive iterations per group: long enough to amortise the search for the node above,
        // short enough to leave every group several runs
        L.chunk = (int)std::max<int64_t>(1, std::min<int64_t>(32, L.count / (L.grid * groups_per_block * 8)));
        launches.push_back(L);
    }
    static PerDeviceOnce smem_once;
    CB_CUDA(once_per_device(smem_once, [] {
        cudaError_t e = cudaFuncSetAttribute(tree_kernel<float, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kLocalScratchBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<float, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kLocalScratchBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<double, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kLocalScratchBytes);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(tree_kernel<double, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kLocalScratchBytes);
        return e;
    }));
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
        const Launch &L = launches[r];
        if (L.count == 0) continue;
        const unsigned grid = (unsigned)L.grid;
        const int32_t local = L.local ? 1 : 0;
        CB_LAUNCH("tree_kernel", stream, {
            if (dtype == CONST_F32 && L.warp)
                tree_kernel<float, true><<<grid, kThreads, L.smem, stream>>>(cp.programs[r], b, L.count, L.chunk, local);
            else if (dtype == CONST_F32)
                tree_kernel<float, false><<<grid, kThreads, L.smem, stream>>>(cp.programs[r], b, L.count, L.chunk, local);
            else if (L.warp)
                tree_kernel<double, true><<<grid, kThreads, L.smem, stream>>>(cp.programs[r], b, L.count, L.chunk, local);
            else
                tree_kernel<double, false><<<grid, kThreads, L.smem, stream>>>(cp.programs[r], b, L.count, L.chunk, local);
        });
        e = cudaGetLastError();
    }
    cudaFreeAsync(scratch, stream);
    return e == cudaSuccess ? CONST_OK : CONST_ERR_CUDA;
}

}  // namespace cb
