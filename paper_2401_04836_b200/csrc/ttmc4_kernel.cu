// Fused order-4 TTMc:  Y[i,a,b,c] = sum_{j,k,l} X[i,j,k,l] U[j,a] V[k,b] W[l,c]  with the chain
//   P[c]   = sum_l X[i,j,k,l] W[l,c]      order-1 intermediate, reset per (i,j,k)
//   Q[b,c] = sum_k V[k,b] P[c]            order-2 intermediate, reset per (i,j)
//   Y[i,a,b,c] += U[j,a] Q[b,c]
// fused on i -> j -> k as in Fig. 4(b).
//
// Thread mapping (rank R = 8), the same warp-local two-phase scheme as the order-3 kernels:
//   phase 1 (producers)  The level-2 nodes (i,j,k) of a window of (i,j) fibres are dealt out to the
//     four 8-lane groups of the warp as equal contiguous runs.  Lane b of a group keeps P (8 floats,
//     a copy per lane) and row b of Q (8 floats) in registers; the W row of a leaf arrives with two
//     128-bit loads, V[k,b] with one coalesced 32-byte access per group.  Coordinates and rows of the
//     next nodes are requested while the current one is multiplied.  When a run leaves an (i,j)
//     fibre its Q is parked in shared memory (or handed over, if a neighbour began that fibre).
//   phase 2 (consumer)  Sixteen lanes cover the 8 x 8 x 8 result of one fibre: a lane owns all a for
//     one b and four c (32 accumulators), reads Q[b, 4 c] from shared memory and U[j, 8] from global
//     memory, 32 FMAs per fibre and lane; a warp consumes two fibres per step.
#include "common.cuh"

namespace cb {
namespace {

constexpr int R = 8;
constexpr int GL = 8;                 // lanes per producer group
constexpr int G = 32 / GL;            // producer groups per warp
constexpr int TILE = R * R * R;       // floats of one output row (slice)
constexpr int WF = 32;                // (i,j) fibres parked per warp
constexpr int QROW = R * R;           // floats of one parked Q

struct Csf4 {
    const int32_t *crd0, *pos1, *crd1, *pos2, *crd2, *pos3, *crd3;
    const float *vals;
};

__device__ __forceinline__ float4 ldg4(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }

__device__ __forceinline__ int32_t leaf_of(const Csf4 &x, int32_t f1) { return __ldg(x.pos3 + __ldg(x.pos2 + f1)); }

// first level-1 node f in [lo, hi] whose first leaf is at or beyond target
__device__ __forceinline__ int32_t lower_bound_leaf(const Csf4 &x, int32_t lo, int32_t hi, int64_t target) {
    while (lo < hi) {
        int32_t mid = lo + (hi - lo) / 2;
        if ((int64_t)leaf_of(x, mid) < target) lo = mid + 1; else hi = mid;
    }
    return lo;
}

struct NodeInfo { int32_t k, pa, pb, l; float xv; };      // one level-2 node and its first leaf

__device__ __forceinline__ NodeInfo load_node(const Csf4 &x, int32_t n, int32_t n_end) {
    NodeInfo r{0, 0, 0, 0, 0.f};
    if (n < n_end) {
        r.k = __ldg(x.crd2 + n);
        r.pa = __ldg(x.pos3 + n);
        r.pb = __ldg(x.pos3 + n + 1);
        r.l = __ldg(x.crd3 + r.pa);
        r.xv = __ldg(x.vals + r.pa);
    }
    return r;
}

// Producer for the window of (i,j) fibres [s0, s0 + cnt).
__device__ __forceinline__ void phase1(const Csf4 &x, const float *__restrict__ V, const float *__restrict__ W,
                                       int32_t s0, int cnt, int cnt_padded, int lane, float *__restrict__ Qs,
                                       int32_t *__restrict__ Js, int32_t *__restrict__ Ps, float *__restrict__ Hs,
                                       int32_t *__restrict__ Hf) {
    const int g = lane / GL, b = lane % GL;
    for (int e = lane; e < cnt_padded; e += 32) Js[e] = e < cnt ? __ldg(x.crd1 + s0 + e) : 0;
    for (int e = lane; e <= cnt; e += 32) Ps[e] = __ldg(x.pos2 + s0 + e);
    for (int e = cnt * (QROW / 4) + lane; e < cnt_padded * (QROW / 4); e += 32)
        reinterpret_cast<float4 *>(Qs)[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncwarp();

    const int32_t N0 = Ps[0], N1 = Ps[cnt];
    const int32_t per_group = (N1 - N0 + G - 1) / G;
    const int32_t na = N0 + g * per_group;
    const int32_t nb = na + per_group < N1 ? na + per_group : N1;
    int32_t head_fibre = -1;
    if (na < nb) {
        int lo = 0, hi = cnt - 1;                                 // fibre holding node na
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (Ps[mid] <= na) lo = mid; else hi = mid - 1;
        }
        int f = lo;
        int32_t fend = Ps[f + 1];
        bool head = Ps[f] < na;                                   // fibre f was begun by an earlier group
        float Q[R];
#pragma unroll
        for (int c = 0; c < R; ++c) Q[c] = 0.f;

        auto park = [&]() {
            float *dst = head ? Hs + g * QROW + b * R : Qs + f * QROW + b * R;
            *reinterpret_cast<float4 *>(dst) = make_float4(Q[0], Q[1], Q[2], Q[3]);
            *reinterpret_cast<float4 *>(dst + 4) = make_float4(Q[4], Q[5], Q[6], Q[7]);
            if (head) { head_fibre = f; head = false; }
        };

        // software pipeline over the nodes of the run: descriptors two nodes ahead, rows one node ahead
        NodeInfo cur = load_node(x, na, nb);
        NodeInfo nxt = load_node(x, na + 1, nb);
        float4 w0 = ldg4(W + (size_t)cur.l * R), w1 = ldg4(W + (size_t)cur.l * R + 4);
        float vb = __ldg(V + (size_t)cur.k * R + b);
        for (int32_t n = na; n < nb; ++n) {
            const NodeInfo nn = load_node(x, n + 2, nb);
            float4 w0n = w0, w1n = w1;
            float vbn = vb;
            if (n + 1 < nb) {
                w0n = ldg4(W + (size_t)nxt.l * R);
                w1n = ldg4(W + (size_t)nxt.l * R + 4);
                vbn = __ldg(V + (size_t)nxt.k * R + b);
            }
            // P = sum over the node's leaves of X * W[l, :]
            float P[R] = {cur.xv * w0.x, cur.xv * w0.y, cur.xv * w0.z, cur.xv * w0.w,
                          cur.xv * w1.x, cur.xv * w1.y, cur.xv * w1.z, cur.xv * w1.w};
            for (int32_t p = cur.pa + 1; p < cur.pb; ++p) {       // further leaves of the node (rare when sparse)
                const float xv = __ldg(x.vals + p);
                const float *w = W + (size_t)__ldg(x.crd3 + p) * R;
                const float4 a0 = ldg4(w), a1 = ldg4(w + 4);
                P[0] = fmaf(xv, a0.x, P[0]); P[1] = fmaf(xv, a0.y, P[1]);
                P[2] = fmaf(xv, a0.z, P[2]); P[3] = fmaf(xv, a0.w, P[3]);
                P[4] = fmaf(xv, a1.x, P[4]); P[5] = fmaf(xv, a1.y, P[5]);
                P[6] = fmaf(xv, a1.z, P[6]); P[7] = fmaf(xv, a1.w, P[7]);
            }
#pragma unroll
            for (int c = 0; c < R; ++c) Q[c] = fmaf(vb, P[c], Q[c]);   // Q[b, :] += V[k, b] * P[:]
            if (n + 1 == fend) {                                  // the run leaves fibre f
                park();
#pragma unroll
                for (int c = 0; c < R; ++c) Q[c] = 0.f;
                ++f;
                fend = Ps[f + 1 <= cnt ? f + 1 : cnt];
            }
            cur = nxt; nxt = nn; w0 = w0n; w1 = w1n; vb = vbn;
        }
        if (f < cnt && nb > Ps[f]) park();                        // the run ends inside fibre f
    }
    if (b == 0) Hf[g] = head_fibre;
    __syncwarp();
    if (g == 0) {                                                 // add the heads, in group order
        for (int gg = 1; gg < G; ++gg) {
            const int32_t hf = Hf[gg];
            if (hf >= 0) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    float4 *row = reinterpret_cast<float4 *>(Qs + hf * QROW + b * R + 4 * h);
                    const float4 v = *reinterpret_cast<const float4 *>(Hs + gg * QROW + b * R + 4 * h);
                    float4 r = *row;
                    r.x += v.x; r.y += v.y; r.z += v.z; r.w += v.w;
                    *row = r;
                }
            }
        }
    }
    __syncwarp();
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
ttmc4_kernel(const WorkItem *__restrict__ items, const int32_t *__restrict__ bin_totals,
             const int32_t *__restrict__ light_list, Csf4 x,
             const float *__restrict__ U, const float *__restrict__ V, const float *__restrict__ W,
             float *__restrict__ out) {
    extern __shared__ __align__(16) float Qs_all[];              // [warp][WF * 64] parked Q
    __shared__ int32_t Js_all[kWarpsPerBlock][WF];
    __shared__ int32_t Ps_all[kWarpsPerBlock][WF + 1];
    __shared__ __align__(16) float Hs_all[kWarpsPerBlock][G * QROW];
    __shared__ int32_t Hf_all[kWarpsPerBlock][G];
    __shared__ float tile[TILE];

    if ((int)blockIdx.x >= work_item_count(bin_totals)) return;      // the grid is an upper bound
    const WorkItem it = items[blockIdx.x];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool light = it.kind == kItemLight;

    int32_t slice = it.slice, fa = 0, fb = 0;
    if (light) {
        if (warp < it.f0) {
            slice = __ldg(light_list + it.slice + warp);
            fa = __ldg(x.pos1 + slice);
            fb = __ldg(x.pos1 + slice + 1);
        }
    } else {
        const int64_t lo = leaf_of(x, it.f0), hi = leaf_of(x, it.f1);
        fa = warp == 0 ? it.f0 : lower_bound_leaf(x, it.f0, it.f1, lo + (hi - lo) * warp / kWarpsPerBlock);
        fb = warp == kWarpsPerBlock - 1
                 ? it.f1
                 : lower_bound_leaf(x, it.f0, it.f1, lo + (hi - lo) * (warp + 1) / kWarpsPerBlock);
        for (int e = threadIdx.x; e < TILE; e += blockDim.x) tile[e] = 0.f;
        __syncthreads();
    }

    // consumer layout: 16 lanes per fibre; lane owns acc[a][4 c] for its b and its half of c
    const int slot = lane >> 4, b2 = (lane >> 1) & 7, ch = lane & 1;
    float acc[R][4];
#pragma unroll
    for (int a = 0; a < R; ++a) acc[a][0] = acc[a][1] = acc[a][2] = acc[a][3] = 0.f;
    float *Qs = Qs_all + warp * (WF * QROW);
    int32_t *Js = Js_all[warp];
    for (int32_t s0 = fa; s0 < fb; s0 += WF) {
        const int cnt = fb - s0 < WF ? fb - s0 : WF;
        const int cnt_padded = (cnt + 1) & ~1;
        phase1(x, V, W, s0, cnt, cnt_padded, lane, Qs, Js, Ps_all[warp], Hs_all[warp], Hf_all[warp]);
        for (int e = slot; e < cnt_padded; e += 2) {             // Y[a, b, c] += U[j, a] * Q[b, c]
            const float *up = U + (size_t)Js[e] * R;
            const float4 u0 = ldg4(up), u1 = ldg4(up + 4);
            const float4 q = *reinterpret_cast<const float4 *>(Qs + e * QROW + b2 * R + 4 * ch);
            const float ua[R] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
            for (int a = 0; a < R; ++a) {
                acc[a][0] = fmaf(ua[a], q.x, acc[a][0]);
                acc[a][1] = fmaf(ua[a], q.y, acc[a][1]);
                acc[a][2] = fmaf(ua[a], q.z, acc[a][2]);
                acc[a][3] = fmaf(ua[a], q.w, acc[a][3]);
            }
        }
        __syncwarp();
    }

    // the two fibre slots hold partial sums of the same entries
#pragma unroll
    for (int a = 0; a < R; ++a)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[a][c] += __shfl_xor_sync(0xffffffffu, acc[a][c], 16);

    if (light) {
        if (warp < it.f0 && lane < 16) {
            float *dst = out + (size_t)__ldg(x.crd0 + slice) * TILE;
#pragma unroll
            for (int a = 0; a < R; ++a)
                *reinterpret_cast<float4 *>(dst + (a * R + b2) * R + 4 * ch) =
                    make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
        }
        return;
    }
    if (fa < fb && lane < 16) {
#pragma unroll
        for (int a = 0; a < R; ++a)
#pragma unroll
            for (int c = 0; c < 4; ++c) atomicAdd(&tile[(a * R + b2) * R + 4 * ch + c], acc[a][c]);
    }
    __syncthreads();
    float *dst = out + (size_t)__ldg(x.crd0 + slice) * TILE;
    if (it.kind == kItemBlock) {
        for (int e = threadIdx.x; e < TILE; e += blockDim.x) dst[e] = tile[e];
    } else {
        for (int e = threadIdx.x; e < TILE; e += blockDim.x) atomicAdd(&dst[e], tile[e]);
    }
}

}  // namespace

const_status_t run_ttmc4(const const_csf *X, const float *U, const float *V, const float *W, int rank, float *Y,
                         int64_t n_rows, int32_t *, cudaStream_t stream) {
    if (rank != R) return CONST_ERR_UNSUPPORTED;
    CB_CUDA(cudaMemsetAsync(Y, 0, sizeof(float) * TILE * n_rows, stream));
    if (X->nnz == 0) return CONST_OK;
    Csf4 x{X->crd[0], X->pos[1], X->crd[1], X->pos[2], X->crd[2], X->pos[3], X->crd[3],
           static_cast<const float *>(X->vals)};
    constexpr size_t dyn = sizeof(float) * kWarpsPerBlock * WF * QROW;
    static PerDeviceOnce attr_once;                     // per template instance
    CB_CUDA(once_per_device(attr_once, [&] { return cudaFuncSetAttribute(ttmc4_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn); }));
    CB_LAUNCH("ttmc4_kernel", stream, ttmc4_kernel<<<(unsigned)X->item_cap, kWarpsPerBlock * 32, dyn, stream>>>(X->items, X->bin_totals, X->light_list, x, U, V, W, Y));
    CB_CUDA(cudaGetLastError());
    return CONST_OK;
}

}  // namespace cb
