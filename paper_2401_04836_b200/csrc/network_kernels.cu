// Fused two-contraction network (paper Sec. 1):  Z[i,m] = sum_{j,k,l} U[i,j,k] V[j,l] W[k,l,m]
// with the tree  T[i,k,l] = sum_j U[i,j,k] V[j,l];  Z[i,m] = sum_{k,l} T[i,k,l] W[k,l,m],
// fused over i so that T is a per-i dense workspace T_i[k,l] (Fig. 4(b) structure: the workspace
// is reset inside the fused loop).
//
// Schedule this kernel implements (both contractions in gather form, no scatter into T or Z rows):
//   U in CSF order (i,k,j), loops i -> k -> j -> l :  T_i[k,l] = sum_{j in fibre (i,k)} U * V[j,l]
//   W in CSF order (m,l,k), loops i -> m -> l -> k :  Z[i,m]   = sum_{l} sum_{k in fibre (m,l)} T_i[k,l] * W
//
// Tiling.  T_i (n_k x n_l doubles, 1 MiB at the benchmark size) does not fit on chip, so a block
// owns a strip of IS consecutive i slices and a tile of LT consecutive l values and keeps
// T[IS][LT][n_k] in shared memory.  Strip-mining i lets every W nonzero fetched from L2 serve IS
// rows of Z; tiling l does not change the result because Z is a sum over l.  Partial sums over the
// l tiles are combined with fp64 atomic adds on Z.
#include "common.cuh"

namespace cb {
namespace {

constexpr int IS = 8;      // i slices per block
constexpr int LT = 16;     // l values per block
constexpr int kThreads = 256;

struct Csf3d {
    const int32_t *crd0, *pos1, *crd1, *pos2, *crd2;
    const double *vals;
    int32_t n0;
};

__global__ void __launch_bounds__(kThreads)
network_kernel(Csf3d u, const double *__restrict__ V, Csf3d w, double *__restrict__ Z, int n_k, int n_l, int n_m) {
    extern __shared__ double T[];                  // [IS][LT][KP], KP = n_k + 1 (padding avoids bank conflicts)
    const int KP = n_k + 1;
    const int strip = blockIdx.x, l0 = blockIdx.y * LT;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    for (int e = threadIdx.x; e < IS * LT * KP; e += kThreads) T[e] = 0.0;      // "T[*,*] = 0" per fused iteration
    __syncthreads();

    // ---- producer: T_i[k, l0 + l] = sum_j U[i,k,j] * V[j, l0 + l]; 16 lanes (one per l) per (i,k) fibre
    {
        const int hw = threadIdx.x / LT, l = threadIdx.x % LT;
        const bool l_ok = l0 + l < n_l;
        for (int ii = 0; ii < IS; ++ii) {
            const int s = strip * IS + ii;
            if (s >= u.n0) break;
            const int32_t fa = u.pos1[s], fb = u.pos1[s + 1];
            for (int32_t f = fa + hw; f < fb; f += kThreads / LT) {
                const int32_t k = u.crd1[f];
                double acc = 0.0;
                if (l_ok) {
                    const double *vcol = V + l0 + l;
                    for (int32_t p = u.pos2[f]; p < u.pos2[f + 1]; ++p)
                        acc = fma(u.vals[p], __ldg(vcol + (size_t)u.crd2[p] * n_l), acc);
                }
                T[(ii * LT + l) * KP + k] = acc;
            }
        }
    }
    __syncthreads();

    // ---- consumer: Z[i,m] += sum_{l in tile} sum_{k in fibre (m,l)} T_i[k,l] * W[m,l,k]; one warp per m
    int32_t rows[IS];
#pragma unroll
    for (int ii = 0; ii < IS; ++ii) {
        const int s = strip * IS + ii;
        rows[ii] = s < u.n0 ? u.crd0[s] : -1;
    }
    for (int32_t mbase = warp * 32; mbase < w.n0; mbase += (kThreads / 32) * 32) {
        // each lane finds, for its own m, the level-1 nodes whose l falls into [l0, l0 + LT)
        int32_t fl0 = 0, fl1 = 0;
        const int32_t mine = mbase + lane;
        if (mine < w.n0) {
            int32_t a = w.pos1[mine], b = w.pos1[mine + 1];
            int32_t lo = a, hi = b;
            while (lo < hi) { int32_t mid = lo + (hi - lo) / 2; if (w.crd1[mid] < l0) lo = mid + 1; else hi = mid; }
            fl0 = lo;
            hi = b;
            while (lo < hi) { int32_t mid = lo + (hi - lo) / 2; if (w.crd1[mid] < l0 + LT) lo = mid + 1; else hi = mid; }
            fl1 = lo;
        }
        unsigned todo = __ballot_sync(0xffffffffu, fl0 < fl1);
        while (todo) {
            const int src = __ffs(todo) - 1;
            todo &= todo - 1;
            const int32_t fa = __shfl_sync(0xffffffffu, fl0, src), fb = __shfl_sync(0xffffffffu, fl1, src);
            double acc[IS];
#pragma unroll
            for (int ii = 0; ii < IS; ++ii) acc[ii] = 0.0;
            for (int32_t f = fa; f < fb; ++f) {
                const int l = w.crd1[f] - l0;
                const int32_t pa = w.pos2[f], pb = w.pos2[f + 1];
                for (int32_t p = pa + lane; p < pb; p += 32) {
                    const int32_t k = w.crd2[p];
                    const double wv = w.vals[p];
                    const double *t = T + l * KP + k;
#pragma unroll
                    for (int ii = 0; ii < IS; ++ii) acc[ii] = fma(t[ii * LT * KP], wv, acc[ii]);
                }
            }
            // sum the lanes' partial dot products (butterfly), then lane ii adds row ii into Z
#pragma unroll
            for (int ii = 0; ii < IS; ++ii) {
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) acc[ii] += __shfl_xor_sync(0xffffffffu, acc[ii], off);
            }
            if (lane < IS && rows[lane] >= 0) {
                double v = 0.0;
#pragma unroll
                for (int ii = 0; ii < IS; ++ii) if (lane == ii) v = acc[ii];
                atomicAdd(Z + (size_t)rows[lane] * n_m + w.crd0[mbase + src], v);
            }
        }
    }
}

}  // namespace

const_status_t run_network(const const_csf *U, const double *V, const const_csf *W, double *Z, int64_t n_i,
                           int64_t n_j, int64_t n_k, int64_t n_l, int64_t n_m, int32_t *, cudaStream_t stream) {
    (void)n_j;
    CB_CUDA(cudaMemsetAsync(Z, 0, sizeof(double) * n_i * n_m, stream));
    if (U->nnz == 0 || W->nnz == 0) return CONST_OK;
    const size_t smem = sizeof(double) * IS * LT * (n_k + 1);
    if (smem > 200 * 1024 || n_l > (1ll << 30) || n_m > (1ll << 30)) return CONST_ERR_WORKSPACE;
    CB_CUDA(cudaFuncSetAttribute(network_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    Csf3d u{U->crd[0], U->pos[1], U->crd[1], U->pos[2], U->crd[2], static_cast<const double *>(U->vals), (int32_t)U->n[0]};
    Csf3d w{W->crd[0], W->pos[1], W->crd[1], W->pos[2], W->crd[2], static_cast<const double *>(W->vals), (int32_t)W->n[0]};
    dim3 grid((unsigned)((U->n[0] + IS - 1) / IS), (unsigned)((n_l + LT - 1) / LT));
    CB_LAUNCH("network_kernel", stream, network_kernel<<<grid, kThreads, smem, stream>>>(u, V, w, Z, (int)n_k, (int)n_l, (int)n_m));
    CB_CUDA(cudaGetLastError());
    return CONST_OK;
}

}  // namespace cb
