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
// T[LT][n_k][IS] in shared memory.  Strip-mining i lets every W nonzero fetched serve IS rows of Z;
// tiling l does not change the result because Z is a sum over l.  With l at the root of W, the
// nonzeros a block needs form one contiguous range of W's fibres.
//
// Memory access.  A thread that walks its own fibre straight from global memory touches a
// different cache line than every other lane of its warp at every step, and the L1 tag stage
// becomes the limit.  So both phases sweep their fibre range in chunks: the chunk's (coordinate,
// value) pairs are copied into shared memory with coalesced loads as 16-byte records, and a group
// of GL lanes then walks one fibre, every lane of the group reading the same record (one broadcast
// 128-bit shared-memory load) and its own LT/GL entries of the V row (producer, contiguous
// in global memory) or of the T row (consumer, contiguous in shared memory).  The partial sums of
// the (l, m) fibres are combined with fp64 atomic adds on Z.
#include "common.cuh"

namespace cb {
namespace {

constexpr int kMaxLT = 32;     // most l values a block may own
constexpr int kThreads = 512;
constexpr int RB = 2048;       // records staged per chunk (a multiple of the block size)
constexpr int FPMAX = 1024;    // fibre descriptors staged per batch

struct Csf3d {
    const int32_t *crd0, *pos1, *crd1, *pos2, *crd2;
    const double *vals;
    int32_t n0;
};

struct __align__(16) Rec {
    int32_t c;
    int32_t pad;
    double v;
};

struct Stage {                 // shared-memory staging area of one sweep
    Rec *recs;                 // [RB]
    int32_t *fpos;             // [FPMAX + 1] first nonzero of every staged fibre
    int32_t *fcrd;             // [FPMAX]     level-1 coordinate of every staged fibre
    int32_t *first;            // staged fibre that holds the first nonzero of the current chunk
};

// Calls body(fibre, coordinate, records, count) once for every piece of every fibre in [fA, fB) of
// the tensor x; a fibre that straddles a chunk boundary is delivered in two pieces (in different
// chunks, i.e. separated by a block barrier).  Lane groups take the fibres of a chunk round-robin.
template <int GL, class Body>
__device__ __forceinline__ void sweep(const Csf3d &x, int32_t fA, int32_t fB, const Stage &st, Body body) {
    constexpr int NG = kThreads / GL;
    const int g = threadIdx.x / GL;
    for (int32_t fb0 = fA; fb0 < fB; fb0 += FPMAX) {
        const int nf = fB - fb0 < FPMAX ? fB - fb0 : FPMAX;
        __syncthreads();
        for (int e = threadIdx.x; e <= nf; e += kThreads) st.fpos[e] = __ldg(x.pos2 + fb0 + e);
        for (int e = threadIdx.x; e < nf; e += kThreads) st.fcrd[e] = __ldg(x.crd1 + fb0 + e);
        __syncthreads();
        const int32_t pA = st.fpos[0], pB = st.fpos[nf];
        // the records of a chunk are requested one chunk ahead and wait in registers while the chunk
        // before them is multiplied, so the global-memory latency of the staging is hidden
        constexpr int PER = RB / kThreads;
        int32_t pc[PER];
        double pv[PER];
        auto request = [&](int32_t c0) {
#pragma unroll
            for (int q = 0; q < PER; ++q) {
                const int32_t p = c0 + threadIdx.x + q * kThreads;
                pc[q] = 0;
                pv[q] = 0.0;
                if (p < pB) { pc[q] = __ldg(x.crd2 + p); pv[q] = __ldg(x.vals + p); }
            }
        };
        request(pA);
        for (int32_t c0 = pA; c0 < pB; c0 += RB) {
            const int32_t c1 = c0 + RB < pB ? c0 + RB : pB;
#pragma unroll
            for (int q = 0; q < PER; ++q) {
                Rec r;
                r.c = pc[q];
                r.pad = 0;
                r.v = pv[q];
                st.recs[threadIdx.x + q * kThreads] = r;
            }
            // the staged fibre that holds nonzero c0: every thread tests its candidates (exactly one fits),
            // which costs a few instructions where a search per thread costs a dependent chain
            for (int e = threadIdx.x; e < nf; e += kThreads)
                if (st.fpos[e] <= c0 && c0 < st.fpos[e + 1]) *st.first = e;
            __syncthreads();
            if (c1 < pB) request(c1);
            const int lo = *st.first;
            for (int f = lo + g; f < nf; f += NG) {
                const int32_t a = st.fpos[f], b = st.fpos[f + 1];
                if (a >= c1) break;
                const int32_t p0 = a > c0 ? a : c0, p1 = b < c1 ? b : c1;
                if (p0 < p1) body(fb0 + f, st.fcrd[f], st.recs + (p0 - c0), p1 - p0);
            }
            __syncthreads();
        }
    }
}

template <int IS, int LT, int GL>
__global__ void __launch_bounds__(kThreads)
network_kernel(Csf3d u, const double *__restrict__ V, Csf3d w, double *__restrict__ Z, int n_k, int n_l, int n_m,
               int v_vec_ok) {
    constexpr int VPT_P = LT / GL;                 // entries of a V row per lane (producer)
    constexpr int VPT_C = IS / GL;                 // entries of a T row per lane (consumer)
    static_assert(LT % GL == 0 && IS % GL == 0 && LT <= kMaxLT && (VPT_P == 1 || VPT_P % 2 == 0) &&
                  (VPT_C == 1 || VPT_C % 2 == 0), "a lane group covers the l of the tile or the i of the strip");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int TL = n_k * IS + 2;                   // doubles per l plane; the +2 staggers the banks of the 8 planes
    double *T = reinterpret_cast<double *>(smem_raw);                               // [LT][n_k][IS]
    Stage st;
    st.recs = reinterpret_cast<Rec *>(T + ((size_t)LT * TL + 1) / 2 * 2);
    st.fpos = reinterpret_cast<int32_t *>(st.recs + RB);
    st.fcrd = st.fpos + FPMAX + 1;
    __shared__ int32_t s_pos[IS + 1];              // first fibre of every slice of the strip
    __shared__ int32_t w_pos[LT + 1];              // first fibre of every l node of the tile
    __shared__ int32_t w_l[LT];                    // l of those nodes, relative to the tile
    __shared__ int32_t w_nodes;
    __shared__ int32_t s_first;
    st.first = &s_first;

    const int strip = blockIdx.x, l0 = blockIdx.y * LT;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int q = threadIdx.x % GL;                // position inside the lane group

    for (int e = threadIdx.x; e < LT * TL; e += kThreads) T[e] = 0.0;              // "T[*,*] = 0" per fused iteration
    if (threadIdx.x <= IS) {
        const int s = strip * IS + threadIdx.x;
        s_pos[threadIdx.x] = __ldg(u.pos1 + (s < u.n0 ? s : u.n0));
    }
    if (warp == 1) {
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
    const int nodes = w_nodes;
    if (nodes == 0) return;                        // no W nonzero has its l in this tile: nothing reaches Z

    // ---- producer: T[l][k][ii] = sum_j U[i,k,j] * V[j, l0 + l]
    {
        const int lq = q * VPT_P;                    // first l of this lane, relative to the tile
        const double *vcol = V + l0 + lq;
        const bool vec = v_vec_ok && VPT_P >= 2 && l0 + lq + VPT_P <= n_l;     // whole lane inside the row, 16-byte aligned
        sweep<GL>(u, s_pos[0], s_pos[IS], st, [&](int32_t f, int32_t k, const Rec *recs, int n) {
            int ii = 0;
            while (ii + 1 < IS && s_pos[ii + 1] <= f) ++ii;
            double a[VPT_P], b[VPT_P];                 // two accumulator sets: consecutive records alternate
#pragma unroll
            for (int c = 0; c < VPT_P; ++c) a[c] = b[c] = 0.0;
            if (vec) {
                auto row_fma = [&](const Rec &r, double (&acc)[VPT_P]) {
                    const double2 *row = reinterpret_cast<const double2 *>(vcol + (size_t)r.c * n_l);
#pragma unroll
                    for (int c = 0; c < VPT_P / 2; ++c) {
                        const double2 v = __ldg(row + c);
                        acc[2 * c] = fma(r.v, v.x, acc[2 * c]);
                        acc[2 * c + 1] = fma(r.v, v.y, acc[2 * c + 1]);
                    }
                };
                int e = 0;
                for (; e + 1 < n; e += 2) {
                    const Rec r0 = recs[e], r1 = recs[e + 1];
                    row_fma(r0, a);
                    row_fma(r1, b);
                }
                if (e < n) row_fma(recs[e], a);
            } else {
                for (int e = 0; e < n; ++e) {
                    const Rec r0 = recs[e];
                    const double *row = vcol + (size_t)r0.c * n_l;
#pragma unroll
                    for (int c = 0; c < VPT_P; ++c)
                        if (l0 + lq + c < n_l) a[c] = fma(r0.v, __ldg(row + c), a[c]);
                }
            }
            double *t = T + (size_t)lq * TL + k * IS + ii;
#pragma unroll
            for (int c = 0; c < VPT_P; ++c) t[c * TL] += a[c] + b[c];
        });
    }
    // (the sweep ends with a block barrier: T is complete)

    // ---- consumer: Z[i,m] += sum_{k in fibre (l,m)} T[l][k][ii] * W[l,m,k]
    {
        const int iq = q * VPT_C;                    // first slice of this lane, relative to the strip
        int32_t rows[VPT_C];
#pragma unroll
        for (int c = 0; c < VPT_C; ++c) {
            const int s = strip * IS + iq + c;
            rows[c] = s < u.n0 ? __ldg(u.crd0 + s) : -1;
        }
        sweep<GL>(w, w_pos[0], w_pos[nodes], st, [&](int32_t f, int32_t m, const Rec *recs, int n) {
            int node = 0;
            while (node + 1 < nodes && w_pos[node + 1] <= f) ++node;
            const double *t = T + (size_t)w_l[node] * TL + iq;
            double a[VPT_C], b[VPT_C];
#pragma unroll
            for (int c = 0; c < VPT_C; ++c) a[c] = b[c] = 0.0;
            auto row_fma = [&](const Rec &r, double (&acc)[VPT_C]) {
                const double *row = t + r.c * IS;
                if constexpr (VPT_C >= 2) {
#pragma unroll
                    for (int c = 0; c < VPT_C / 2; ++c) {
                        const double2 tv = *reinterpret_cast<const double2 *>(row + 2 * c);
                        acc[2 * c] = fma(tv.x, r.v, acc[2 * c]);
                        acc[2 * c + 1] = fma(tv.y, r.v, acc[2 * c + 1]);
                    }
                } else {
                    acc[0] = fma(row[0], r.v, acc[0]);
                }
            };
            int e = 0;
            for (; e + 1 < n; e += 2) {
                const Rec r0 = recs[e], r1 = recs[e + 1];
                row_fma(r0, a);
                row_fma(r1, b);
            }
            if (e < n) row_fma(recs[e], a);
#pragma unroll
            for (int c = 0; c < VPT_C; ++c)
                if (rows[c] >= 0) atomicAdd(Z + (size_t)rows[c] * n_m + m, a[c] + b[c]);
        });
    }
}

}  // namespace

namespace {

template <int IS, int LT, int GL>
const_status_t launch_network(const const_csf *U, const double *V, const const_csf *W, double *Z, int64_t n_k,
                              int64_t n_l, int64_t n_m, cudaStream_t stream) {
    const size_t t_doubles = ((size_t)LT * (n_k * IS + 2) + 1) / 2 * 2;
    const size_t smem = sizeof(double) * t_doubles + sizeof(Rec) * RB + sizeof(int32_t) * (2 * FPMAX + 1);
    if (smem > 220 * 1024 || n_l > (1ll << 30) || n_m > (1ll << 30)) return CONST_ERR_WORKSPACE;
    auto kernel = network_kernel<IS, LT, GL>;
    // the requested size depends on n_k: raise the limit once per device to the most a block may have
    static PerDeviceOnce attr_once;
    CB_CUDA(once_per_device(attr_once, [&] { return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024); }));
    Csf3d u{U->crd[0], U->pos[1], U->crd[1], U->pos[2], U->crd[2], static_cast<const double *>(U->vals), (int32_t)U->n[0]};
    Csf3d w{W->crd[0], W->pos[1], W->crd[1], W->pos[2], W->crd[2], static_cast<const double *>(W->vals), (int32_t)W->n[0]};
    const int v_vec_ok = (n_l % 2 == 0) && (reinterpret_cast<uintptr_t>(V) % 16 == 0);
    dim3 grid((unsigned)((U->n[0] + IS - 1) / IS), (unsigned)((n_l + LT - 1) / LT));
    CB_LAUNCH("network_kernel", stream,
              kernel<<<grid, kThreads, smem, stream>>>(u, V, w, Z, (int)n_k, (int)n_l, (int)n_m, v_vec_ok));
    CB_CUDA(cudaGetLastError());
    return CONST_OK;
}

}  // namespace

const_status_t run_network(const const_csf *U, const double *V, const const_csf *W, double *Z, int64_t n_i,
                           int64_t n_j, int64_t n_k, int64_t n_l, int64_t n_m, int32_t *, cudaStream_t stream) {
    (void)n_j;
    CB_CUDA(cudaMemsetAsync(Z, 0, sizeof(double) * n_i * n_m, stream));
    if (U->nnz == 0 || W->nnz == 0) return CONST_OK;
    // tile shape (slices per strip, l per tile, lanes per fibre); the variants are kept for measurement
    switch (debug_knobs().variant) {
        case 1: return launch_network<8, 16, 4>(U, V, W, Z, n_k, n_l, n_m, stream);
        case 2: return launch_network<16, 8, 4>(U, V, W, Z, n_k, n_l, n_m, stream);
        case 3: return launch_network<8, 16, 8>(U, V, W, Z, n_k, n_l, n_m, stream);
        case 4: return launch_network<16, 8, 8>(U, V, W, Z, n_k, n_l, n_m, stream);
        case 5: return launch_network<4, 16, 4>(U, V, W, Z, n_k, n_l, n_m, stream);
        default: return launch_network<8, 8, 4>(U, V, W, Z, n_k, n_l, n_m, stream);
    }
}

}  // namespace cb
