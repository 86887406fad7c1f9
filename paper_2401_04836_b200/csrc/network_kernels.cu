// Fused two-contraction network (paper Sec. 1):  Z[i,m] = sum_{j,k,l} U[i,j,k] V[j,l] W[k,l,m]
// with the tree  T[i,k,l] = sum_j U[i,j,k] V[j,l];  Z[i,m] = sum_{k,l} T[i,k,l] W[k,l,m],
// fused over i so that T is a per-i dense workspace T_i[k,l] (Fig. 4(b) structure: the workspace
// is reset inside the fused loop).
//
// Schedule this kernel implements (both contractions gather along a CSF fibre, nothing is scattered
// into T):
//   U in CSF order (i,k,j), loops i -> k -> j -> l :  T_i[k,l] = sum_{j in fibre (i,k)} U * V[j,l]
//   W in CSF order (l,m,k), loops i -> l -> m -> k :  Z[i,m]  += sum_{k in fibre (l,m)} T_i[k,l] * W
//
// Tiling.  T_i (n_k x n_l doubles, 1 MiB at the benchmark size) does not fit on chip, so a block
// owns a strip of IS consecutive i slices and a tile of LT consecutive l values and keeps
// T[LT][n_k][IS] in shared memory.  Strip-mining i lets every W nonzero fetched from L2 serve IS
// rows of Z; tiling l does not change the result because Z is a sum over l.  With l at the root of
// W, the nonzeros a block needs form one contiguous range of W's fibres.  The partial sums of the
// (l, m) fibres are combined with fp64 atomic adds on Z.
#include "common.cuh"

namespace cb {
namespace {

constexpr int IS = 8;      // i slices per block
constexpr int LT = 8;      // l values per block
constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct Csf3d {
    const int32_t *crd0, *pos1, *crd1, *pos2, *crd2;
    const double *vals;
    int32_t n0;
};

__global__ void __launch_bounds__(kThreads)
network_kernel(Csf3d u, const double *__restrict__ V, Csf3d w, double *__restrict__ Z, int n_k, int n_l, int n_m) {
    extern __shared__ double T[];                  // [LT][KP][IS], KP = n_k + 1 (odd row pitch spreads the banks)
    __shared__ int32_t w_pos[LT + 1];              // first fibre of every l node of the tile
    __shared__ int32_t w_l[LT];                    // l of those nodes, relative to the tile
    __shared__ int32_t w_nodes;
    const int KP = n_k + 1;
    const int strip = blockIdx.x, l0 = blockIdx.y * LT;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    for (int e = threadIdx.x; e < LT * KP * IS; e += kThreads) T[e] = 0.0;      // "T[*,*] = 0" per fused iteration
    if (warp == 0) {
        // root nodes of W whose l lies in [l0, l0 + LT): a contiguous range of at most LT nodes
        int32_t lo = 0, hi = w.n0;
        while (lo < hi) { int32_t mid = lo + (hi - lo) / 2; if (__ldg(w.crd0 + mid) < l0) lo = mid + 1; else hi = mid; }
        const int32_t first = lo;
        int32_t node = first + lane;
        const bool in = lane < LT && node < w.n0 && __ldg(w.crd0 + (node < w.n0 ? node : 0)) < l0 + LT;
        const unsigned m = __ballot_sync(0xffffffffu, in);
        const int cnt = __popc(m);                 // nodes are sorted, so the valid ones are lanes 0..cnt-1
        if (lane < cnt) { w_l[lane] = __ldg(w.crd0 + node) - l0; w_pos[lane] = __ldg(w.pos1 + node); }
        if (lane == 0) { w_nodes = cnt; w_pos[cnt] = __ldg(w.pos1 + first + cnt); }
    }
    __syncthreads();

    // ---- producer: T[l][k][ii] = sum_j U[i,k,j] * V[j, l0 + l]; LT/4 lanes per (i,k) fibre, four l per lane,
    //      so every (j, value) pair fetched feeds four multiply-adds
    {
        constexpr int LPU = LT / 4;                // lanes per fibre
        constexpr int UNITS = kThreads / LPU;      // fibres in flight per block
        const int slot = threadIdx.x / LPU, l4 = (threadIdx.x % LPU) * 4;
        const bool vec = (n_l % 2 == 0) && (l0 + l4 + 3 < n_l);     // 16-byte aligned, fully inside the row
        const double *vcol = V + l0 + l4;
        for (int ii = 0; ii < IS; ++ii) {
            const int s = strip * IS + ii;
            if (s >= u.n0) break;
            const int32_t fa = __ldg(u.pos1 + s), fb = __ldg(u.pos1 + s + 1);
            int32_t kn = 0, pan = 0, pbn = 0;                  // descriptor of the fibre after this one
            if (fa + slot < fb) {
                kn = __ldg(u.crd1 + fa + slot); pan = __ldg(u.pos2 + fa + slot); pbn = __ldg(u.pos2 + fa + slot + 1);
            }
            for (int32_t f = fa + slot; f < fb; f += UNITS) {
                const int32_t k = kn, pa = pan, pb = pbn;
                if (f + UNITS < fb) {
                    kn = __ldg(u.crd1 + f + UNITS); pan = __ldg(u.pos2 + f + UNITS); pbn = __ldg(u.pos2 + f + UNITS + 1);
                }
                double a[4] = {0.0, 0.0, 0.0, 0.0};
                if (vec) {
                    int32_t p = pa;
                    for (; p + 1 < pb; p += 2) {
                        const int32_t j0 = __ldg(u.crd2 + p), j1 = __ldg(u.crd2 + p + 1);
                        const double x0 = __ldg(u.vals + p), x1 = __ldg(u.vals + p + 1);
                        const double2 *r0 = reinterpret_cast<const double2 *>(vcol + (size_t)j0 * n_l);
                        const double2 *r1 = reinterpret_cast<const double2 *>(vcol + (size_t)j1 * n_l);
                        const double2 v00 = __ldg(r0), v01 = __ldg(r0 + 1), v10 = __ldg(r1), v11 = __ldg(r1 + 1);
                        a[0] = fma(x0, v00.x, a[0]); a[1] = fma(x0, v00.y, a[1]);
                        a[2] = fma(x0, v01.x, a[2]); a[3] = fma(x0, v01.y, a[3]);
                        a[0] = fma(x1, v10.x, a[0]); a[1] = fma(x1, v10.y, a[1]);
                        a[2] = fma(x1, v11.x, a[2]); a[3] = fma(x1, v11.y, a[3]);
                    }
                    if (p < pb) {
                        const double x0 = __ldg(u.vals + p);
                        const double2 *r0 = reinterpret_cast<const double2 *>(vcol + (size_t)__ldg(u.crd2 + p) * n_l);
                        const double2 v00 = __ldg(r0), v01 = __ldg(r0 + 1);
                        a[0] = fma(x0, v00.x, a[0]); a[1] = fma(x0, v00.y, a[1]);
                        a[2] = fma(x0, v01.x, a[2]); a[3] = fma(x0, v01.y, a[3]);
                    }
                } else {
                    for (int32_t p = pa; p < pb; ++p) {
                        const double x0 = __ldg(u.vals + p);
                        const double *r0 = vcol + (size_t)__ldg(u.crd2 + p) * n_l;
#pragma unroll
                        for (int c = 0; c < 4; ++c)
                            if (l0 + l4 + c < n_l) a[c] = fma(x0, __ldg(r0 + c), a[c]);
                    }
                }
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (l0 + l4 + c < n_l) T[((l4 + c) * KP + k) * IS + ii] = a[c];
            }
        }
    }
    __syncthreads();

    // ---- consumer: two lanes (four i of the strip each) per (l, m) fibre of W, so every (k, value) pair
    //      fetched feeds four multiply-adds and a warp has sixteen independent fibres in flight; the
    //      descriptor of the next fibre is fetched ahead
    constexpr int LPFIB = IS / 4;                               // lanes per fibre
    constexpr int SLOTS = kThreads / LPFIB;
    const int i4 = (threadIdx.x % LPFIB) * 4, slot = threadIdx.x / LPFIB;
    int32_t rows[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
        const int s_row = strip * IS + i4 + c;
        rows[c] = s_row < u.n0 ? __ldg(u.crd0 + s_row) : -1;
    }
    const int nodes = w_nodes;
    if (nodes == 0) return;
    const int32_t f_begin = w_pos[0], f_end = w_pos[nodes];
    int32_t f = f_begin + slot;
    int32_t m = 0, pa = 0, pb = 0;
    if (f < f_end) { m = __ldg(w.crd1 + f); pa = __ldg(w.pos2 + f); pb = __ldg(w.pos2 + f + 1); }
    while (f < f_end) {
        const int32_t fn = f + SLOTS;
        int32_t mn = 0, pan = 0, pbn = 0;
        if (fn < f_end) { mn = __ldg(w.crd1 + fn); pan = __ldg(w.pos2 + fn); pbn = __ldg(w.pos2 + fn + 1); }
        int node = 0;
        while (node + 1 < nodes && w_pos[node + 1] <= f) ++node;
        const double *t = T + (size_t)w_l[node] * KP * IS + i4;
        double a[4] = {0.0, 0.0, 0.0, 0.0};
        int32_t p = pa;
        for (; p + 1 < pb; p += 2) {
            const int32_t k0 = __ldg(w.crd2 + p), k1 = __ldg(w.crd2 + p + 1);
            const double w0 = __ldg(w.vals + p), w1 = __ldg(w.vals + p + 1);
            const double2 *t0 = reinterpret_cast<const double2 *>(t + k0 * IS);
            const double2 *t1 = reinterpret_cast<const double2 *>(t + k1 * IS);
            const double2 t00 = t0[0], t01 = t0[1], t10 = t1[0], t11 = t1[1];
            a[0] = fma(t00.x, w0, a[0]); a[1] = fma(t00.y, w0, a[1]);
            a[2] = fma(t01.x, w0, a[2]); a[3] = fma(t01.y, w0, a[3]);
            a[0] = fma(t10.x, w1, a[0]); a[1] = fma(t10.y, w1, a[1]);
            a[2] = fma(t11.x, w1, a[2]); a[3] = fma(t11.y, w1, a[3]);
        }
        if (p < pb) {
            const double w0 = __ldg(w.vals + p);
            const double2 *t0 = reinterpret_cast<const double2 *>(t + __ldg(w.crd2 + p) * IS);
            const double2 t00 = t0[0], t01 = t0[1];
            a[0] = fma(t00.x, w0, a[0]); a[1] = fma(t00.y, w0, a[1]);
            a[2] = fma(t01.x, w0, a[2]); a[3] = fma(t01.y, w0, a[3]);
        }
#pragma unroll
        for (int c = 0; c < 4; ++c)
            if (rows[c] >= 0) atomicAdd(Z + (size_t)rows[c] * n_m + m, a[c]);
        f = fn; m = mn; pa = pan; pb = pbn;
    }
}

}  // namespace

const_status_t run_network(const const_csf *U, const double *V, const const_csf *W, double *Z, int64_t n_i,
                           int64_t n_j, int64_t n_k, int64_t n_l, int64_t n_m, int32_t *, cudaStream_t stream) {
    (void)n_j;
    CB_CUDA(cudaMemsetAsync(Z, 0, sizeof(double) * n_i * n_m, stream));
    if (U->nnz == 0 || W->nnz == 0) return CONST_OK;
    const size_t smem = sizeof(double) * LT * (n_k + 1) * IS;
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
