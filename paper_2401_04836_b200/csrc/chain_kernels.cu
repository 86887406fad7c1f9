// Fused kernels of the "chain" family: one CSF tensor contracted leaf level first with one dense
// factor per level (TTMc, Sec. 5.3; MTTKRP, Sec. 5.2), executed as the fused loop nest of Fig. 4(b):
//
//   for i (slice)                     -- root level, fused
//     for j (fibre)                   -- level 1, fused
//       t[*] = 0                      -- order-1 intermediate, reset per fibre
//       for k: t[b] += X[i,j,k] * V[k,b]            (producer contraction)
//       for a,b: Y[i,a,b] += U[j,a] * t[b]          (consumer contraction; MTTKRP: A[i,r] += B[j,r] * t[r])
//
// Thread mapping.  Each warp owns a run of fibres of one slice and alternates between two phases over
// windows of a few dozen fibres, entirely on its own (only __syncwarp, no block barrier), so warps of
// a block overlap their memory-bound and arithmetic-bound phases:
//
//   phase 1 (producer)  A factor row of R3 floats is read by R3/4 neighbouring lanes with one 128-bit
//     load each.  The nonzeros of the window are dealt out to the lane groups as equal contiguous
//     runs of 4-aligned blocks, independent of fibre lengths: a block's four coordinates and four
//     values arrive with one 128-bit load each and the four row gathers are issued together.  A
//     group stores its partial t when its run leaves a fibre (or hands it over, for a fibre begun
//     by its neighbour).  The finished t of every fibre of the window is thus parked in shared
//     memory (the reduced-order intermediate, one row per fibre), together with the fibre's j.
//   phase 2 (consumer)  The R2 x R3 slice result is cut into 8 x 4 register blocks; the lanes that
//     cover one result work on one fibre, so a warp consumes 32 / ((R2/8)(R3/4)) fibres per step:
//     t comes from shared memory, U[j, 8 rows] from global memory with two 128-bit loads, followed
//     by 32 FMAs per lane.  For MTTKRP a lane owns four rank entries and does four FMAs.
//
// The slice result therefore lives in registers and leaves the warp once: straight to global memory
// for a slice owned by one warp, through a shared-memory tile for a slice (or chunk of a giant
// slice) owned by a block -- stored once or, for a chunk, added atomically.
#include "common.cuh"

namespace cb {
namespace {

__device__ __forceinline__ float4 ldg4(const float *p) { return __ldg(reinterpret_cast<const float4 *>(p)); }

constexpr int kStreamAhead = 256;   // nonzeros between the L2 prefetch of a line of the leaf arrays and its use

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
        if ((int64_t)__ldg(pos + mid) < target) lo = mid + 1; else hi = mid;
    }
    return lo;
}

struct Csf3 {
    const int32_t *crd0, *pos1, *crd1, *pos2, *crd2;   // crd2 and vals are readable up to the next multiple of 4
    const float *vals;
};

template <int R2, int R3, bool HADAMARD>
struct Shape {
    // phase 1
    static constexpr int LPR1 = R3 / 4;                 // lanes per factor row
    static constexpr int G1 = 32 / LPR1;                // lane groups per warp
    static constexpr int WINDOW = R3 >= 32 ? 64 : 128;  // fibres parked per warp
    // phase 2: register block of RW rows x 4 columns per lane
    static constexpr int RW = HADAMARD ? 1 : 8;
    static constexpr int LPF = HADAMARD ? R3 / 4 : (R2 / 8) * (R3 / 4);   // lanes that cover one fibre
    static constexpr int FPW = 32 / LPF;                // fibres per warp and step
    static constexpr int NACC = RW * 4;
    static constexpr int TILE = HADAMARD ? R3 : R2 * R3;  // floats of one output row (slice)
    static_assert(LPF >= 1 && LPF <= 32 && WINDOW % FPW == 0, "unsupported rank combination");
};

// Producer for the window of fibres [s0, s0 + cnt): parks t and j in shared memory.
// A fibre that starts inside a group's run gets its row stored by that group; the part of a fibre
// that a group finds already begun (its run starts in the middle of it) goes to a per-group "head"
// slot and is added to the row afterwards, one group after the other, so no atomics and no clearing
// of the rows are needed.  Rows and j of the padding fibres [cnt, cnt_padded) are zeroed.
template <int R2, int R3, bool HADAMARD>
__device__ __forceinline__ void phase1(const Csf3 &x, const float *__restrict__ F2, int32_t s0, int cnt,
                                       int cnt_padded, int lane, float *__restrict__ Ts, int32_t *__restrict__ Js,
                                       int32_t *__restrict__ Ps, float *__restrict__ Hs, int32_t *__restrict__ Hf) {
    using S = Shape<R2, R3, HADAMARD>;
    const int g = lane / S::LPR1, q = lane % S::LPR1;
    const float *F2q = F2 + 4 * q;
    for (int e = lane; e < cnt_padded; e += 32) Js[e] = e < cnt ? __ldg(x.crd1 + s0 + e) : 0;
    for (int e = lane; e <= cnt; e += 32) Ps[e] = __ldg(x.pos2 + s0 + e);
    for (int e = cnt * (R3 / 4) + lane; e < cnt_padded * (R3 / 4); e += 32)
        reinterpret_cast<float4 *>(Ts)[e] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncwarp();

    const int32_t P0 = Ps[0], P1 = Ps[cnt];
    const int32_t A0 = P0 & ~3;                                   // 4-aligned blocks of the leaf arrays
    const int32_t blocks = (P1 - A0 + 3) >> 2;
    const int32_t per_group = (blocks + S::G1 - 1) / S::G1;
    const int32_t ba = A0 + g * per_group * 4;
    const int32_t bb = ba + per_group * 4;
    const int32_t pa = ba > P0 ? ba : P0;                         // nonzeros of this group: [pa, pb)
    const int32_t pb = bb < P1 ? bb : P1;
    int32_t head_fibre = -1;
    if (pa < pb) {
        int lo = 0, hi = cnt - 1;                                 // fibre holding nonzero pa
        while (lo < hi) {
            const int mid = (lo + hi + 1) >> 1;
            if (Ps[mid] <= pa) lo = mid; else hi = mid - 1;
        }
        int f = lo;
        int32_t fend = Ps[f + 1];
        bool head = Ps[f] < pa;                                   // fibre f was begun by an earlier group
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);

        auto park = [&]() {                                       // hand the partial t of fibre f over
            if (head) {
                *reinterpret_cast<float4 *>(Hs + g * R3 + 4 * q) = t;
                head_fibre = f;
                head = false;
            } else {
                *reinterpret_cast<float4 *>(Ts + f * R3 + 4 * q) = t;
            }
        };
        auto leave_fibre = [&]() {                                // the run leaves fibre f
            park();
            t = make_float4(0.f, 0.f, 0.f, 0.f);
            ++f;
            fend = Ps[f + 1 <= cnt ? f + 1 : cnt];
        };

        auto partial_block = [&](int32_t p) {                     // first or last block of the run
            const int4 kk = __ldg(reinterpret_cast<const int4 *>(x.crd2 + p));
            const float4 xx = __ldg(reinterpret_cast<const float4 *>(x.vals + p));
            const int32_t k[4] = {kk.x, kk.y, kk.z, kk.w};
            const float xv[4] = {xx.x, xx.y, xx.z, xx.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (p + u >= pa && p + u < pb) {
                    fma4(t, xv[u], ldg4(F2q + (size_t)k[u] * R3));
                    if (p + u + 1 == fend) leave_fibre();
                }
            }
        };

        // whole blocks [m0, m1) run through a software pipeline: coordinates two blocks ahead,
        // row gathers one block ahead of the multiply-adds
        const int32_t m0 = pa > ba ? ba + 4 : ba;
        const int32_t m1 = pb & ~3;
        if (pa > ba) partial_block(ba);
        if (m0 < m1) {
            int4 kn = __ldg(reinterpret_cast<const int4 *>(x.crd2 + m0));
            float4 xc = __ldg(reinterpret_cast<const float4 *>(x.vals + m0));
            float4 v0 = ldg4(F2q + (size_t)kn.x * R3), v1 = ldg4(F2q + (size_t)kn.y * R3);
            float4 v2 = ldg4(F2q + (size_t)kn.z * R3), v3 = ldg4(F2q + (size_t)kn.w * R3);
            float4 xn = xc;
            if (m0 + 4 < m1) {
                kn = __ldg(reinterpret_cast<const int4 *>(x.crd2 + m0 + 4));
                xn = __ldg(reinterpret_cast<const float4 *>(x.vals + m0 + 4));
            }
            for (int32_t p = m0; p < m1; p += 4) {
                if (q == 0 && ((p >> 2) & 7) == 0 && p + kStreamAhead < m1) {      // once per 128-byte line of the leaf arrays
                    asm volatile("prefetch.global.L2 [%0];" :: "l"(x.crd2 + p + kStreamAhead));
                    asm volatile("prefetch.global.L2 [%0];" :: "l"(x.vals + p + kStreamAhead));
                }
                float4 w0 = v0, w1 = v1, w2 = v2, w3 = v3, xw = xn;
                if (p + 4 < m1) {                                 // gathers of the next block
                    w0 = ldg4(F2q + (size_t)kn.x * R3); w1 = ldg4(F2q + (size_t)kn.y * R3);
                    w2 = ldg4(F2q + (size_t)kn.z * R3); w3 = ldg4(F2q + (size_t)kn.w * R3);
                }
                if (p + 8 < m1) {                                 // coordinates of the block after it
                    kn = __ldg(reinterpret_cast<const int4 *>(x.crd2 + p + 8));
                    xn = __ldg(reinterpret_cast<const float4 *>(x.vals + p + 8));
                }
                fma4(t, xc.x, v0);
                if (p + 1 == fend) leave_fibre();
                fma4(t, xc.y, v1);
                if (p + 2 == fend) leave_fibre();
                fma4(t, xc.z, v2);
                if (p + 3 == fend) leave_fibre();
                fma4(t, xc.w, v3);
                if (p + 4 == fend) leave_fibre();
                v0 = w0; v1 = w1; v2 = w2; v3 = w3; xc = xw;
            }
        }
        if (m1 >= m0 && m1 < pb) partial_block(m1);
        if (f < cnt && pb > Ps[f]) park();                        // the run ends inside fibre f
    }
    if (q == 0) Hf[g] = head_fibre;
    __syncwarp();
    if (g == 0) {                                                 // add the heads, in group order
        for (int gg = 1; gg < S::G1; ++gg) {
            const int32_t hf = Hf[gg];
            if (hf >= 0) {
                float4 *row = reinterpret_cast<float4 *>(Ts + hf * R3 + 4 * q);
                const float4 h = *reinterpret_cast<const float4 *>(Hs + gg * R3 + 4 * q);
                float4 r = *row;
                r.x += h.x; r.y += h.y; r.z += h.z; r.w += h.w;
                *row = r;
            }
        }
    }
    __syncwarp();
}

// Consumer for the parked window: acc += (factor row of j) (x) t.
template <int R2, int R3, bool HADAMARD>
__device__ __forceinline__ void phase2(const float *__restrict__ F1, int cnt_padded, int lane,
                                       const float *__restrict__ Ts, const int32_t *__restrict__ Js,
                                       float (&acc)[Shape<R2, R3, HADAMARD>::NACC]) {
    using S = Shape<R2, R3, HADAMARD>;
    const int slot = lane / S::LPF, inner = lane % S::LPF;
    if (HADAMARD) {
        // lane owns rank entries 4*inner .. 4*inner+3 of the fibre in its slot
        for (int e = slot; e < cnt_padded; e += S::FPW) {
            const float4 b = ldg4(F1 + (size_t)Js[e] * R3 + 4 * inner);
            const float4 tv = *reinterpret_cast<const float4 *>(Ts + e * R3 + 4 * inner);
            acc[0] = fmaf(b.x, tv.x, acc[0]);
            acc[1] = fmaf(b.y, tv.y, acc[1]);
            acc[2] = fmaf(b.z, tv.z, acc[2]);
            acc[3] = fmaf(b.w, tv.w, acc[3]);
        }
    } else {
        // lane owns rows 8*rg .. 8*rg+7 and columns 4*cg .. 4*cg+3 of the fibre in its slot
        const int rg = inner / (R3 / 4), cg = inner % (R3 / 4);
        const float *F1g = F1 + 8 * rg;
        for (int e = slot; e < cnt_padded; e += S::FPW) {
            const float *up = F1g + (size_t)Js[e] * R2;
            const float4 u0 = ldg4(up), u1 = ldg4(up + 4);
            const float4 tv = *reinterpret_cast<const float4 *>(Ts + e * R3 + 4 * cg);
            const float ur[8] = {u0.x, u0.y, u0.z, u0.w, u1.x, u1.y, u1.z, u1.w};
#pragma unroll
            for (int r = 0; r < 8; ++r) {
                acc[4 * r + 0] = fmaf(ur[r], tv.x, acc[4 * r + 0]);
                acc[4 * r + 1] = fmaf(ur[r], tv.y, acc[4 * r + 1]);
                acc[4 * r + 2] = fmaf(ur[r], tv.z, acc[4 * r + 2]);
                acc[4 * r + 3] = fmaf(ur[r], tv.w, acc[4 * r + 3]);
            }
        }
    }
    __syncwarp();
}

template <int R2, int R3, bool HADAMARD>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
chain3_kernel(const WorkItem *__restrict__ items, const int32_t *__restrict__ bin_totals,
              const int32_t *__restrict__ light_list, Csf3 x,
              const float *__restrict__ F1, const float *__restrict__ F2, float *__restrict__ out) {
    using S = Shape<R2, R3, HADAMARD>;
    extern __shared__ __align__(16) float Ts_all[];          // [warp][WINDOW * R3] parked rows
    __shared__ int32_t Js_all[kWarpsPerBlock][S::WINDOW];
    __shared__ int32_t Ps_all[kWarpsPerBlock][S::WINDOW + 1];
    __shared__ __align__(16) float Hs_all[kWarpsPerBlock][S::G1 * R3];
    __shared__ int32_t Hf_all[kWarpsPerBlock][S::G1];
    __shared__ float tile[S::TILE];

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
        const int64_t lo = __ldg(x.pos2 + it.f0), hi = __ldg(x.pos2 + it.f1);
        fa = warp == 0 ? it.f0 : lower_bound_pos(x.pos2, it.f0, it.f1, lo + (hi - lo) * warp / kWarpsPerBlock);
        fb = warp == kWarpsPerBlock - 1
                 ? it.f1
                 : lower_bound_pos(x.pos2, it.f0, it.f1, lo + (hi - lo) * (warp + 1) / kWarpsPerBlock);
        for (int e = threadIdx.x; e < S::TILE; e += blockDim.x) tile[e] = 0.f;
        __syncthreads();
    }

    float acc[S::NACC];
#pragma unroll
    for (int a = 0; a < S::NACC; ++a) acc[a] = 0.f;
    float *Ts = Ts_all + warp * (S::WINDOW * R3);
    int32_t *Js = Js_all[warp];
    for (int32_t s0 = fa; s0 < fb; s0 += S::WINDOW) {
        const int cnt = fb - s0 < S::WINDOW ? fb - s0 : S::WINDOW;
        const int cnt_padded = (cnt + S::FPW - 1) / S::FPW * S::FPW;
        phase1<R2, R3, HADAMARD>(x, F2, s0, cnt, cnt_padded, lane, Ts, Js, Ps_all[warp], Hs_all[warp], Hf_all[warp]);
        phase2<R2, R3, HADAMARD>(F1, cnt_padded, lane, Ts, Js, acc);
    }

    // lanes of different slots hold partial sums of the same result entries: add them up
#pragma unroll
    for (int off = S::LPF; off < 32; off <<= 1) {
#pragma unroll
        for (int a = 0; a < S::NACC; ++a) acc[a] += __shfl_xor_sync(0xffffffffu, acc[a], off);
    }
    const int inner = lane % S::LPF;
    const int rg = HADAMARD ? 0 : inner / (R3 / 4), cg = HADAMARD ? inner : inner % (R3 / 4);
    if (light) {
        if (warp < it.f0 && lane < S::LPF) {
            float *dst = out + (size_t)__ldg(x.crd0 + slice) * S::TILE;
#pragma unroll
            for (int r = 0; r < S::RW; ++r)
                *reinterpret_cast<float4 *>(dst + (S::RW * rg + r) * R3 + 4 * cg) =
                    make_float4(acc[4 * r], acc[4 * r + 1], acc[4 * r + 2], acc[4 * r + 3]);
        }
        return;
    }
    if (fa < fb && lane < S::LPF) {
#pragma unroll
        for (int r = 0; r < S::RW; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) atomicAdd(&tile[(S::RW * rg + r) * R3 + 4 * cg + c], acc[4 * r + c]);
    }
    __syncthreads();
    float *dst = out + (size_t)__ldg(x.crd0 + slice) * S::TILE;
    if (it.kind == kItemBlock) {
        for (int e = threadIdx.x; e < S::TILE; e += blockDim.x) dst[e] = tile[e];
    } else {
        for (int e = threadIdx.x; e < S::TILE; e += blockDim.x) atomicAdd(&dst[e], tile[e]);
    }
}

template <int R2, int R3, bool HADAMARD>
const_status_t launch_chain3(const const_csf *X, const float *F1, const float *F2, float *out, int64_t n_rows,
                             cudaStream_t stream) {
    constexpr int TILE = Shape<R2, R3, HADAMARD>::TILE;
    CB_CUDA(cudaMemsetAsync(out, 0, sizeof(float) * TILE * n_rows, stream));       // "R[*] = 0" precedes the nest
    if (X->nnz == 0) return CONST_OK;
    Csf3 x{X->crd[0], X->pos[1], X->crd[1], X->pos[2], X->crd[2], static_cast<const float *>(X->vals)};
    using S = Shape<R2, R3, HADAMARD>;
    constexpr size_t dyn = sizeof(float) * kWarpsPerBlock * S::WINDOW * R3;
    static PerDeviceOnce attr_once;                     // per template instance
    CB_CUDA(once_per_device(attr_once, [&] { return cudaFuncSetAttribute(chain3_kernel<R2, R3, HADAMARD>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn); }));
    CB_LAUNCH("chain3_kernel", stream,
              chain3_kernel<R2, R3, HADAMARD><<<(unsigned)X->item_cap, kWarpsPerBlock * 32, dyn, stream>>>(
                  X->items, X->bin_totals, X->light_list, x, F1, F2, out));
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
