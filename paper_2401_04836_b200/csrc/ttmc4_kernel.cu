// Fused order-4 TTMc:  Y[i,a,b,c] = sum_{j,k,l} X[i,j,k,l] U[j,a] V[k,b] W[l,c]  with the chain
//   P[c]   = sum_l X[i,j,k,l] W[l,c]      order-1 intermediate, reset per (i,j,k)
//   Q[b,c] = sum_k V[k,b] P[c]            order-2 intermediate, reset per (i,j)
//   Y[i,a,b,c] += U[j,a] Q[b,c]
// fused on i -> j -> k as in Fig. 4(b), both intermediates held in registers.
//
// Thread mapping (rank R = 8).  A group of 8 lanes owns one (i,j) fibre; lane b of the group holds
// row b of Q (8 floats), a full copy of P (8 floats) and the slice accumulator Y[a][b][*] for its b
// (64 floats).  A warp therefore works on four (i,j) fibres at once; the leaves of a fibre are
// walked in one flat loop, folding P into Q whenever a level-2 node ends.
#include "common.cuh"

namespace cb {
namespace {

constexpr int R = 8;
constexpr int GL = 8;            // lanes per group
constexpr int G = 32 / GL;       // (i,j) fibres in flight per warp
constexpr int TILE = R * R * R;

struct Csf4 {
    const int32_t *crd0, *pos1, *crd1, *pos2, *crd2, *pos3, *crd3;
    const float *vals;
};

__device__ __forceinline__ float4 ldg4(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }

__device__ __forceinline__ int32_t leaf_of(const Csf4 &x, int32_t f1) { return x.pos3[x.pos2[f1]]; }

// first level-1 node f in [lo, hi] whose first leaf is at or beyond target
__device__ __forceinline__ int32_t lower_bound_leaf(const Csf4 &x, int32_t lo, int32_t hi, int64_t target) {
    while (lo < hi) {
        int32_t mid = lo + (hi - lo) / 2;
        if ((int64_t)leaf_of(x, mid) < target) lo = mid + 1; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(kWarpsPerBlock * 32)
ttmc4_kernel(const WorkItem *__restrict__ items, const int32_t *__restrict__ light_list, Csf4 x,
             const float *__restrict__ U, const float *__restrict__ V, const float *__restrict__ W,
             float *__restrict__ out) {
    __shared__ float tile[kWarpsPerBlock][TILE];      // 16 KB

    const WorkItem it = items[blockIdx.x];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane / GL, b = lane % GL;
    const bool light = it.kind == kItemLight;

    int32_t slice = it.slice, fa = 0, fb = 0;
    if (light) {
        if (warp < it.f0) {
            slice = light_list[it.slice + warp];
            fa = x.pos1[slice];
            fb = x.pos1[slice + 1];
        }
    } else {
        const int64_t lo = leaf_of(x, it.f0), hi = leaf_of(x, it.f1);
        fa = warp == 0 ? it.f0 : lower_bound_leaf(x, it.f0, it.f1, lo + (hi - lo) * warp / kWarpsPerBlock);
        fb = warp == kWarpsPerBlock - 1
                 ? it.f1
                 : lower_bound_leaf(x, it.f0, it.f1, lo + (hi - lo) * (warp + 1) / kWarpsPerBlock);
    }
    float *my_tile = light ? tile[warp] : tile[0];
    for (int e = threadIdx.x; e < kWarpsPerBlock * TILE; e += blockDim.x) (&tile[0][0])[e] = 0.f;
    __syncthreads();

    if (fa < fb) {
        float acc[R][R];                     // acc[a][c] for this lane's b
#pragma unroll
        for (int a = 0; a < R; ++a)
#pragma unroll
            for (int c = 0; c < R; ++c) acc[a][c] = 0.f;

        for (int32_t fbase = fa; fbase < fb; fbase += G) {
            const int32_t f1 = fbase + g;
            const bool have = f1 < fb;
            int32_t n2 = 0, n2_end = 0, j = 0;          // level-2 node cursor
            if (have) { n2 = x.pos2[f1]; n2_end = x.pos2[f1 + 1]; j = x.crd1[f1]; }
            int32_t p = 0, p_end = 0, node_end = 0, k = 0;
            if (have) {
                p = x.pos3[n2];
                p_end = x.pos3[n2_end];
                node_end = x.pos3[n2 + 1];
                k = x.crd2[n2];
            }
            float P[R], Q[R];
#pragma unroll
            for (int c = 0; c < R; ++c) { P[c] = 0.f; Q[c] = 0.f; }
            while (__any_sync(0xffffffffu, p < p_end)) {
                if (p < p_end) {
                    const float xv = x.vals[p];
                    const float *w = W + (size_t)x.crd3[p] * R;
                    const float4 w0 = ldg4(w), w1 = ldg4(w + 4);
                    P[0] = fmaf(xv, w0.x, P[0]); P[1] = fmaf(xv, w0.y, P[1]);
                    P[2] = fmaf(xv, w0.z, P[2]); P[3] = fmaf(xv, w0.w, P[3]);
                    P[4] = fmaf(xv, w1.x, P[4]); P[5] = fmaf(xv, w1.y, P[5]);
                    P[6] = fmaf(xv, w1.z, P[6]); P[7] = fmaf(xv, w1.w, P[7]);
                    ++p;
                    if (p == node_end) {                 // level-2 node finished: Q[b,*] += V[k,b] * P[*]
                        const float vb = __ldg(V + (size_t)k * R + b);
#pragma unroll
                        for (int c = 0; c < R; ++c) { Q[c] = fmaf(vb, P[c], Q[c]); P[c] = 0.f; }
                        ++n2;
                        if (n2 < n2_end) { k = x.crd2[n2]; node_end = x.pos3[n2 + 1]; }
                    }
                }
            }
            if (have) {                                  // (i,j) fibre finished: Y[a,b,*] += U[j,a] * Q[b,*]
                const float4 u0 = ldg4(U + (size_t)j * R), u1 = ldg4(U + (size_t)j * R + 4);
                const float ua[R] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
                for (int a = 0; a < R; ++a)
#pragma unroll
                    for (int c = 0; c < R; ++c) acc[a][c] = fmaf(ua[a], Q[c], acc[a][c]);
            }
        }
#pragma unroll
        for (int a = 0; a < R; ++a)
#pragma unroll
            for (int c = 0; c < R; ++c) atomicAdd(&my_tile[(a * R + b) * R + c], acc[a][c]);
    }
    __syncthreads();

    if (light) {
        if (warp < it.f0) {
            float *dst = out + (size_t)x.crd0[slice] * TILE;
            for (int e = lane; e < TILE; e += 32) dst[e] = my_tile[e];
        }
    } else {
        float *dst = out + (size_t)x.crd0[slice] * TILE;
        if (it.kind == kItemBlock) {
            for (int e = threadIdx.x; e < TILE; e += blockDim.x) dst[e] = tile[0][e];
        } else {
            for (int e = threadIdx.x; e < TILE; e += blockDim.x) atomicAdd(&dst[e], tile[0][e]);
        }
    }
}

}  // namespace

const_status_t run_ttmc4(const const_csf *X, const float *U, const float *V, const float *W, int rank, float *Y,
                         int64_t n_rows, int32_t *, cudaStream_t stream) {
    if (rank != R) return CONST_ERR_UNSUPPORTED;
    CB_CUDA(cudaMemsetAsync(Y, 0, sizeof(float) * TILE * n_rows, stream));
    if (X->n_items == 0) return CONST_OK;
    Csf4 x{X->crd[0], X->pos[1], X->crd[1], X->pos[2], X->crd[2], X->pos[3], X->crd[3],
           static_cast<const float *>(X->vals)};
    CB_LAUNCH("ttmc4_kernel", stream, ttmc4_kernel<<<(unsigned)X->n_items, kWarpsPerBlock * 32, 0, stream>>>(X->items, X->light_list, x, U, V, W, Y));
    CB_CUDA(cudaGetLastError());
    return CONST_OK;
}

}  // namespace cb
