// Fused kernels of the "chain" family: one CSF tensor contracted leaf level first with one dense
// factor per level (TTMc, Sec. 5.3; MTTKRP, Sec. 5.2), executed as the fused loop nest of Fig. 4(b):
//
//   for i (slice)                     -- root level, fused
//     for j (fibre)                   -- level 1, fused
//       t[*] = 0                      -- order-1 intermediate, lives in registers, reset per fibre
//       for k: t[b] += X[i,j,k] * V[k,b]            (producer contraction)
//       for a,b: Y[i,a,b] += U[j,a] * t[b]          (consumer contraction; MTTKRP: A[i,r] += B[j,r] * t[r])
//
// Thread mapping.  A factor row of R floats is read by R/4 neighbouring lanes with one 128-bit load
// each; such a lane group owns one fibre at a time, so a warp works on 32/(R/4) fibres at once and
// the partial t never leaves the group's registers.  Fibres much longer than the group count are
// split over all groups of the warp: by linearity every group may apply the consumer to its own
// partial t.  Each lane accumulates its share of the slice result in registers; partial results
// are merged in shared memory and leave the block once per work item (plain store for a whole
// slice, atomic add for a chunk of a giant slice).
#include "common.cuh"

namespace cb {
namespace {

__device__ __forceinline__ float4 ldg4(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }

__device__ __forceinline__ void fma4(float4 &t, float x, const float4 &v) {
    t.x = fmaf(x, v.x, t.x);
    t.y = fmaf(x, v.y, t.y);
    t.z = fmaf(x, v.z, t.z);
    t.w = fmaf(x, v.w, t.w);
}

// first index f in [lo, hi] with pos[f] >= target
__device__ __forceinline__ int32_t lower_bound_pos(const int32_t *__restrict__ pos, int32_t lo, int32_t hi,
                                                   int64_t target) {
    while (lo < hi) {
        int32_t mid = lo + (hi - lo) / 2;
        if ((int64_t)pos[mid] < target) lo = mid + 1; else hi = mid;
    }
    return lo;
}

struct Csf3 {
    const int32_t *crd0, *pos1, *crd1, *pos2, *crd2;
    const float *vals;
};

// ROWS x 4 accumulators per lane.  TTMc: ROWS = R2 (outer product with the level-1 factor row);
// MTTKRP: ROWS = 1 (element-wise product with the level-1 factor row).
template <int R2, int R3, bool HADAMARD>
struct Acc {
    static constexpr int ROWS = HADAMARD ? 1 : R2;
    float a[ROWS][4];
    __device__ __forceinline__ void clear() {
#pragma unroll
        for (int r = 0; r < ROWS; ++r) a[r][0] = a[r][1] = a[r][2] = a[r][3] = 0.f;
    }
    // consumer contraction for one fibre: j = level-1 coordinate, t = this lane's 4 entries of the intermediate
    __device__ __forceinline__ void consume(const float *__restrict__ F1, int32_t j, const float4 &t, int q) {
        if (HADAMARD) {
            float4 b = ldg4(F1 + (size_t)j * R3 + 4 * q);
            a[0][0] = fmaf(b.x, t.x, a[0][0]);
            a[0][1] = fmaf(b.y, t.y, a[0][1]);
            a[0][2] = fmaf(b.z, t.z, a[0][2]);
            a[0][3] = fmaf(b.w, t.w, a[0][3]);
        } else {
            const float *u = F1 + (size_t)j * R2;
#pragma unroll
            for (int r4 = 0; r4 < R2 / 4; ++r4) {
                float4 uu = ldg4(u + 4 * r4);
                const float ur[4] = {uu.x, uu.y, uu.z, uu.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    a[4 * r4 + e][0] = fmaf(ur[e], t.x, a[4 * r4 + e][0]);
                    a[4 * r4 + e][1] = fmaf(ur[e], t.y, a[4 * r4 + e][1]);
                    a[4 * r4 + e][2] = fmaf(ur[e], t.z, a[4 * r4 + e][2]);
                    a[4 * r4 + e][3] = fmaf(ur[e], t.w, a[4 * r4 + e][3]);
                }
            }
        }
    }
};

// One warp walks the level-1 nodes [fa, fb) of one slice.
template <int R2, int R3, bool HADAMARD>
__device__ __forceinline__ void walk_fibres(const Csf3 &x, const float *__restrict__ F1, const float *__restrict__ F2,
                                            int32_t fa, int32_t fb, int lane, Acc<R2, R3, HADAMARD> &acc) {
    constexpr int LPR = R3 / 4;          // lanes per factor row
    constexpr int G = 32 / LPR;          // fibres in flight per warp
    constexpr int LONG = 8 * G;          // fibres at least this long are spread over all groups
    const int g = lane / LPR, q = lane % LPR;
    const float *F2q = F2 + 4 * q;

    for (int32_t fbase = fa; fbase < fb; fbase += G) {
        const int32_t f = fbase + g;
        const bool have = f < fb;
        int32_t p0 = 0, p1 = 0, j = 0;
        if (have) { p0 = x.pos2[f]; p1 = x.pos2[f + 1]; j = x.crd1[f]; }

        // long fibres first, one at a time, all groups cooperating
        unsigned longmask = __ballot_sync(0xffffffffu, have && (p1 - p0) >= LONG && q == 0);
        while (longmask) {
            const int src = __ffs(longmask) - 1;
            longmask &= longmask - 1;
            const int32_t lp0 = __shfl_sync(0xffffffffu, p0, src);
            const int32_t lp1 = __shfl_sync(0xffffffffu, p1, src);
            const int32_t lj = __shfl_sync(0xffffffffu, j, src);
            float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
            int32_t p = lp0 + g;
            for (; p + 3 * G < lp1; p += 4 * G) {
                int32_t k0 = x.crd2[p], k1 = x.crd2[p + G], k2 = x.crd2[p + 2 * G], k3 = x.crd2[p + 3 * G];
                float x0 = x.vals[p], x1 = x.vals[p + G], x2 = x.vals[p + 2 * G], x3 = x.vals[p + 3 * G];
                float4 v0 = ldg4(F2q + (size_t)k0 * R3), v1 = ldg4(F2q + (size_t)k1 * R3);
                float4 v2 = ldg4(F2q + (size_t)k2 * R3), v3 = ldg4(F2q + (size_t)k3 * R3);
                fma4(t, x0, v0); fma4(t, x1, v1); fma4(t, x2, v2); fma4(t, x3, v3);
            }
            for (; p < lp1; p += G) {
                float4 v = ldg4(F2q + (size_t)x.crd2[p] * R3);
                fma4(t, x.vals[p], v);
            }
            acc.consume(F1, lj, t, q);
            if (lane / LPR == src / LPR) p1 = p0;      // done: leave nothing for the short path
        }

        // short fibres: one per lane group, all groups in step
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
        int32_t p = p0;
        while (__any_sync(0xffffffffu, p < p1)) {
            if (p + 1 < p1) {
                int32_t k0 = x.crd2[p], k1 = x.crd2[p + 1];
                float x0 = x.vals[p], x1 = x.vals[p + 1];
                float4 v0 = ldg4(F2q + (size_t)k0 * R3), v1 = ldg4(F2q + (size_t)k1 * R3);
                fma4(t, x0, v0); fma4(t, x1, v1);
            } else if (p < p1) {
                float4 v = ldg4(F2q + (size_t)x.crd2[p] * R3);
                fma4(t, x.vals[p], v);
            }
            p += 2;
        }
        if (p0 < p1) acc.consume(F1, j, t, q);
    }
}

template <int R2, int R3, bool HADAMARD>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
chain3_kernel(const WorkItem *__restrict__ items, const int32_t *__restrict__ light_list, Csf3 x,
              const float *__restrict__ F1, const float *__restrict__ F2, float *__restrict__ out) {
    constexpr int LPR = R3 / 4;
    constexpr int ROWS = Acc<R2, R3, HADAMARD>::ROWS;
    constexpr int TILE = ROWS * R3;                 // floats of one output row (slice)
    __shared__ float tile[kWarpsPerBlock][TILE];

    const WorkItem it = items[blockIdx.x];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int q = lane % LPR;
    const bool light = it.kind == kItemLight;

    int32_t slice = it.slice, fa = 0, fb = 0;
    if (light) {
        if (warp < it.f0) {
            slice = light_list[it.slice + warp];
            fa = x.pos1[slice];
            fb = x.pos1[slice + 1];
        }
    } else {
        const int64_t lo = x.pos2[it.f0], hi = x.pos2[it.f1];
        fa = warp == 0 ? it.f0 : lower_bound_pos(x.pos2, it.f0, it.f1, lo + (hi - lo) * warp / kWarpsPerBlock);
        fb = warp == kWarpsPerBlock - 1
                 ? it.f1
                 : lower_bound_pos(x.pos2, it.f0, it.f1, lo + (hi - lo) * (warp + 1) / kWarpsPerBlock);
    }

    float *my_tile = light ? tile[warp] : tile[0];
    for (int e = threadIdx.x; e < kWarpsPerBlock * TILE; e += blockDim.x) (&tile[0][0])[e] = 0.f;
    __syncthreads();

    Acc<R2, R3, HADAMARD> acc;
    acc.clear();
    if (fa < fb) {
        walk_fibres<R2, R3, HADAMARD>(x, F1, F2, fa, fb, lane, acc);
#pragma unroll
        for (int r = 0; r < ROWS; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) atomicAdd(&my_tile[r * R3 + 4 * q + c], acc.a[r][c]);
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

template <int R2, int R3, bool HADAMARD>
const_status_t launch_chain3(const const_csf *X, const float *F1, const float *F2, float *out, int64_t n_rows,
                             cudaStream_t stream) {
    constexpr int TILE = Acc<R2, R3, HADAMARD>::ROWS * R3;
    CB_CUDA(cudaMemsetAsync(out, 0, sizeof(float) * TILE * n_rows, stream));       // "R[*] = 0" precedes the nest
    if (X->n_items == 0) return CONST_OK;
    Csf3 x{X->crd[0], X->pos[1], X->crd[1], X->pos[2], X->crd[2], static_cast<const float *>(X->vals)};
    CB_LAUNCH("chain3_kernel", stream, chain3_kernel<R2, R3, HADAMARD><<<(unsigned)X->n_items, kWarpsPerBlock * 32, 0, stream>>>(
        X->items, X->light_list, x, F1, F2, out));
    CB_CUDA(cudaGetLastError());
    return CONST_OK;
}

template <int R2>
const_status_t dispatch_ttmc3_r3(const const_csf *X, const float *U, const float *V, int R3, float *Y, int64_t n_rows,
                                 cudaStream_t s) {
    switch (R3) {
        case 8: return launch_chain3<R2, 8, false>(X, U, V, Y, n_rows, s);
        case 16: return launch_chain3<R2, 16, false>(X, U, V, Y, n_rows, s);
        case 32: return launch_chain3<R2, 32, false>(X, U, V, Y, n_rows, s);
    }
    return CONST_ERR_UNSUPPORTED;
}

}  // namespace

const_status_t run_ttmc3(const const_csf *X, const float *U, const float *V, int R2, int R3, float *Y,
                         int64_t n_rows, int32_t *, cudaStream_t stream) {
    switch (R2) {
        case 8: return dispatch_ttmc3_r3<8>(X, U, V, R3, Y, n_rows, stream);
        case 16: return dispatch_ttmc3_r3<16>(X, U, V, R3, Y, n_rows, stream);
        case 32: return dispatch_ttmc3_r3<32>(X, U, V, R3, Y, n_rows, stream);
    }
    return CONST_ERR_UNSUPPORTED;
}

const_status_t run_mttkrp3(const const_csf *X, const float *B, const float *C, int R, float *A, int64_t n_rows,
                           int32_t *, cudaStream_t stream) {
    switch (R) {
        case 8: return launch_chain3<8, 8, true>(X, B, C, A, n_rows, stream);
        case 16: return launch_chain3<16, 16, true>(X, B, C, A, n_rows, stream);
        case 32: return launch_chain3<32, 32, true>(X, B, C, A, n_rows, stream);
    }
    return CONST_ERR_UNSUPPORTED;
}

}  // namespace cb
