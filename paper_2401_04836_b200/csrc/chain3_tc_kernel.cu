// Fused order-3 TTMc at rank 16 x 16 with the per-slice dense stage on the tensor cores (tcgen05):
//   t[b]      = sum_k X[i,j,k] V[k,b]        order-1 intermediate, reset per (i,j)   (Fig. 4(b))
//   Y[i,a,b] += U[j,a] t[b]
// The last statement, summed over the fibres of a slice, is the contraction
//   Y_i[b, a] = sum_f t_f[b] * U[j_f, a]          M = 16 (of 64), N = 16, K = fibres.
//
// Producer (CUDA cores).  The nonzeros of a warp's fibre range are dealt to eight streams of four lanes
// as equal contiguous runs; a stream walks its run with coordinates and values two nonzeros and the
// V row one nonzero ahead, lane h keeping t[4h .. 4h+3].  When the run leaves a fibre, or ends, the
// stream parks t with the fibre's j as one piece = one K slot (the contraction is linear in t, so a
// fibre cut between two streams takes two slots and nothing is merged).  When a stream has to park
// and its slot is still taken, the warp flushes the eight slots to the tensor core.
//
// Operands (no swizzle, K-major core matrices of 8 rows x 16 bytes):
//   A[m, k] at (k / 4) * 256 + (m / 8) * 128 + (m % 8) * 16 + (k % 4) * 4      m = b, 16 real rows
//   B[n, k] at (k / 4) * 272 + n * 16 + (k % 4) * 4                            n = a
// The MMA is M = 64: row m of the accumulator depends on row m of A only, so 48 rows are don't-cares.
// Warp q of the block places its 16 real rows at m = 16 q .. 16 q + 15 by starting the A descriptor
// 2 q row groups before its data (the other row groups then read neighbouring bytes of the warp's
// own shared-memory region, whatever they hold).  Those rows of the accumulator live in tensor-memory
// lanes 32 q .. 32 q + 15, the quarter that warp q can read: every warp is independent of the others
// until the block adds up the slice results in shared memory.
// fp32 accuracy from tf32: x = hi + lo with hi = tf32(x); hi*hi + lo*hi + hi*lo accumulated in fp32.
// Every mbarrier wait is bounded; on a timeout the block records CONST_ERR_TIMEOUT, stops issuing
// MMAs, skips its stores and still frees its tensor memory.
#include "common.cuh"
#include "umma.cuh"

namespace cb {
namespace {

using namespace umma;

constexpr int R = 16;
constexpr int TILE = R * R;
constexpr int SL = 4, NS = 8;     // lanes per stream, streams per warp
constexpr int SLOTS = NS;         // one K slot per stream
constexpr int kWarps = 4;
constexpr int kWarpsPerLight = kWarps / kWarpsPerBlock;
constexpr int kTmemCols = kWarps * R;     // one 16-column accumulator per warp
constexpr int RAW_ROW = 20;               // floats per parked piece (16 + 4 spare)
// per-warp shared memory, in floats; Raw comes first so that the 768 bytes in front of A belong to the warp
constexpr int RAW_FLOATS = 256, A_FLOATS = 128, B_QUAD = 68, B_FLOATS = 2 * B_QUAD;
constexpr int WARP_FLOATS = RAW_FLOATS + 2 * A_FLOATS + 2 * B_FLOATS + 32;
constexpr size_t kWarpBytes = (sizeof(float) * WARP_FLOATS + 127) / 128 * 128;
static_assert(SLOTS * RAW_ROW <= RAW_FLOATS && RAW_FLOATS * sizeof(float) >= 6 * 128, "row groups in front of A");
constexpr uint32_t kIdesc = idesc_tf32(64, R);

struct Csf3 {
    const int32_t *crd0, *pos1, *crd1, *pos2, *crd2;
    const float *vals;
};

// first level-1 node f in [lo, hi] with pos2[f] >= target
__device__ __forceinline__ int32_t lower_bound_pos(const int32_t *__restrict__ pos, int32_t lo, int32_t hi, int64_t target) {
    while (lo < hi) {
        int32_t mid = lo + (hi - lo) / 2;
        if ((int64_t)__ldg(pos + mid) < target) lo = mid + 1; else hi = mid;
    }
    return lo;
}

__global__ void __launch_bounds__(kWarps * 32, 8)
chain3_tc_kernel(const WorkItem *__restrict__ items, const int32_t *__restrict__ bin_totals,
                 const int32_t *__restrict__ light_list, Csf3 x,
                 const float *__restrict__ U, const float *__restrict__ V, float *__restrict__ out,
                 int32_t *__restrict__ status, int wait_polls, int withhold) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t mbar_all[kWarps];
    __shared__ uint32_t tmem_base_s;
    __shared__ float tile[kWarpsPerBlock][TILE];         // slice results of the block (two slices for a light item)
    __shared__ int32_t tile_row[kWarpsPerBlock];
    __shared__ int32_t failed;

    if ((int)blockIdx.x >= work_item_count(bin_totals)) return;      // the grid is an upper bound; nothing is held yet
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const WorkItem it = items[blockIdx.x];
    const bool light = it.kind == kItemLight;

    // this warp's share: part `part` of `parts` of the level-1 nodes [f0, f1) of `slice`, cut by nonzero count
    int32_t slice = it.slice, f0 = it.f0, f1 = it.f1, fa = 0, fb = 0;
    int part = warp, parts = kWarps, group = 0;
    if (light) {
        group = warp / kWarpsPerLight;
        part = warp % kWarpsPerLight;
        parts = kWarpsPerLight;
        f0 = f1 = 0;
        if (group < it.f0) {
            slice = __ldg(light_list + it.slice + group);
            f0 = __ldg(x.pos1 + slice);
            f1 = __ldg(x.pos1 + slice + 1);
        }
    }
    if (f0 < f1) {
        const int64_t lo = __ldg(x.pos2 + f0), hi = __ldg(x.pos2 + f1);
        fa = part == 0 ? f0 : lower_bound_pos(x.pos2, f0, f1, lo + (hi - lo) * part / parts);
        fb = part == parts - 1 ? f1 : lower_bound_pos(x.pos2, f0, f1, lo + (hi - lo) * (part + 1) / parts);
    }

    const uint32_t mbar = smem_u32(&mbar_all[warp]);
    for (int e = threadIdx.x; e < kWarpsPerBlock * TILE; e += kWarps * 32) (&tile[0][0])[e] = 0.f;
    if (lane == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(mbar) : "memory");
        if (part == 0 && group < kWarpsPerBlock) tile_row[group] = f0 < f1 ? __ldg(x.crd0 + slice) : -1;
        if (warp == 0) failed = 0;
    }
    __syncwarp();
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&tmem_base_s)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = tmem_base_s;
    const uint32_t d_tmem = tmem_base + (uint32_t)(R * warp);

    float *Raw = reinterpret_cast<float *>(smem_raw + kWarpBytes * warp);    // [SLOTS][RAW_ROW] parked pieces
    float *Ahi = Raw + RAW_FLOATS;
    float *Alo = Ahi + A_FLOATS;
    float *Bhi = Alo + A_FLOATS;
    float *Blo = Bhi + B_FLOATS;
    int32_t *Jslot = reinterpret_cast<int32_t *>(Blo + B_FLOATS);
    // row group 2 * warp of the 64-row A operand is the first real one
    const uint32_t ahi_s = smem_u32(Ahi) - 2u * warp * 128u, alo_s = smem_u32(Alo) - 2u * warp * 128u;
    const uint32_t bhi_s = smem_u32(Bhi), blo_s = smem_u32(Blo);

    uint32_t parity = 0;
    bool pending = false, ok = true, first = true, used = false;
    const int st = lane / SL, h = lane % SL;
    int cnt = 0;                                                  // 1: this stream's slot holds a piece

    // Hands the parked pieces to the tensor core: Y_i += T_J^T U_J over the eight slots.
    auto flush = [&]() {
        __syncwarp();
        const unsigned vm = __ballot_sync(0xffffffffu, cnt > 0);  // bit 4 s: slot s holds a piece
        const int slot_b = lane >> 2, quarter = lane & 3;         // B: lane writes entries 4 quarter .. + 3 of slot_b's U row
        float4 u = make_float4(0.f, 0.f, 0.f, 0.f);
        if ((vm >> (slot_b * SL)) & 1u) u = ldg4(U + (size_t)Jslot[slot_b] * R + 4 * quarter);
        if (pending) {                                            // the MMAs of the previous flush still read the operands
            bool done = lane == 0 ? mbar_wait(mbar, parity, wait_polls) : true;
            done = __shfl_sync(0xffffffffu, done, 0);
            parity ^= 1;
            pending = false;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (!done) ok = false;
        }
        if (ok) {
            {                                                     // A: lane = (K quad, m): column m of four pieces
                const int quad = lane >> 4, m = lane & 15;
                float e[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int slot = 4 * quad + q;
                    e[q] = ((vm >> (slot * SL)) & 1u) ? Raw[slot * RAW_ROW + m] : 0.f;
                }
                float4 hi4, lo4;
                split4(make_float4(e[0], e[1], e[2], e[3]), hi4, lo4);
                const int off = quad * 64 + (m >> 3) * 32 + (m & 7) * 4;
                *reinterpret_cast<float4 *>(Ahi + off) = hi4;
                *reinterpret_cast<float4 *>(Alo + off) = lo4;
            }
            {
                float4 hi4, lo4;
                split4(u, hi4, lo4);
                float *bh = Bhi + (slot_b >> 2) * B_QUAD + (4 * quarter) * 4 + (slot_b & 3);
                float *bl = Blo + (slot_b >> 2) * B_QUAD + (4 * quarter) * 4 + (slot_b & 3);
                bh[0] = hi4.x; bh[4] = hi4.y; bh[8] = hi4.z; bh[12] = hi4.w;
                bl[0] = lo4.x; bl[4] = lo4.y; bl[8] = lo4.z; bl[12] = lo4.w;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // operand stores -> visible to the tensor core
            __syncwarp();
            if (lane == 0) {
                const uint64_t a_hi = smem_desc(ahi_s, 256, 128), a_lo = smem_desc(alo_s, 256, 128);
                const uint64_t b_hi = smem_desc(bhi_s, 4 * B_QUAD, 128), b_lo = smem_desc(blo_s, 4 * B_QUAD, 128);
                if (!withhold) {      // (test hook: nothing issued, nothing committed -> the next bounded wait runs out)
                    umma_tf32(d_tmem, a_hi, b_hi, kIdesc, first ? 0u : 1u);
                    umma_tf32(d_tmem, a_lo, b_hi, kIdesc, 1u);
                    umma_tf32(d_tmem, a_hi, b_lo, kIdesc, 1u);
                    umma_commit(mbar);
                }
            }
            pending = true;
            first = false;
            used = true;
        }
        cnt = 0;
        __syncwarp();
    };

    if (fa < fb) {
        const int32_t P0 = __ldg(x.pos2 + fa), P1 = __ldg(x.pos2 + fb);
        const int32_t per = (P1 - P0 + NS - 1) / NS;
        const int32_t pa = P0 + st * per;
        const int32_t pb = pa + per < P1 ? pa + per : P1;
        int32_t f = fa;
        if (pa < pb) {                                            // fibre holding nonzero pa
            int32_t lo = fa, hi = fb - 1;
            while (lo < hi) {
                const int32_t mid = lo + (hi - lo + 1) / 2;
                if (__ldg(x.pos2 + mid) <= pa) lo = mid; else hi = mid - 1;
            }
            f = lo;
        }
        const int32_t flast = fb - 1;
        int32_t fend = __ldg(x.pos2 + f + 1);                     // end of fibre f; the fibre after it is fetched ahead
        int32_t fend_n = __ldg(x.pos2 + (f + 2 <= fb ? f + 2 : fb));
        int32_t jc = __ldg(x.crd1 + f), jn = __ldg(x.crd1 + (f + 1 <= flast ? f + 1 : flast));
        float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
        const float *Vh = V + 4 * h;

        // software pipeline: coordinate and value two nonzeros ahead, V row one nonzero ahead
        int32_t k1 = 0, k2 = 0;
        float x0 = 0.f, x1 = 0.f, x2 = 0.f;
        float4 v0 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (pa < pb) { x0 = __ldg(x.vals + pa); v0 = ldg4(Vh + (size_t)__ldg(x.crd2 + pa) * R); }
        if (pa + 1 < pb) { k1 = __ldg(x.crd2 + pa + 1); x1 = __ldg(x.vals + pa + 1); }
        for (int32_t s = 0; s < per && ok; ++s) {
            const int32_t p = pa + s;
            if (p + 2 < pb) { k2 = __ldg(x.crd2 + p + 2); x2 = __ldg(x.vals + p + 2); }
            float4 v1 = v0;
            if (p + 1 < pb) v1 = ldg4(Vh + (size_t)k1 * R);
            bool parks = false;
            if (p < pb) {
                t.x = fmaf(x0, v0.x, t.x); t.y = fmaf(x0, v0.y, t.y);
                t.z = fmaf(x0, v0.z, t.z); t.w = fmaf(x0, v0.w, t.w);
                parks = p + 1 == fend || p + 1 == pb;             // the run leaves fibre f, or ends inside it
            }
            if (__any_sync(0xffffffffu, parks && cnt > 0)) flush();
            if (parks && ok) {
                *reinterpret_cast<float4 *>(Raw + st * RAW_ROW + 4 * h) = t;
                t = make_float4(0.f, 0.f, 0.f, 0.f);
                if (h == 0) Jslot[st] = jc;
                cnt = 1;
                if (p + 1 == fend) {
                    ++f;
                    fend = fend_n;
                    jc = jn;
                    fend_n = __ldg(x.pos2 + (f + 2 <= fb ? f + 2 : fb));
                    jn = __ldg(x.crd1 + (f + 1 <= flast ? f + 1 : flast));
                }
            }
            x0 = x1; x1 = x2; k1 = k2; v0 = v1;
        }
        if (ok && __any_sync(0xffffffffu, cnt > 0)) flush();
    }
    if (pending) {
        bool done = lane == 0 ? mbar_wait(mbar, parity, wait_polls) : true;
        done = __shfl_sync(0xffffffffu, done, 0);
        if (!done) ok = false;
    }
    if (!ok && lane == 0) {
        failed = 1;
        atomicExch(status, (int32_t)CONST_ERR_TIMEOUT);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

    // ---- epilogue: lane b < 16 of warp q holds Y[a = 0..15][b] of the warp's accumulator
    if (!failed) {
        if (used) {                                               // warp-uniform
            uint32_t r[R];
            const uint32_t taddr = tmem_base + ((uint32_t)(32 * warp) << 16) + (uint32_t)(R * warp);
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                         : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                           "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                         : "r"(taddr));
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
            if (lane < R) {
#pragma unroll
                for (int a = 0; a < R; ++a) atomicAdd(&tile[group][a * R + lane], __uint_as_float(r[a]));
            }
        }
        __syncthreads();
        const int groups = light ? kWarpsPerBlock : 1;
        for (int e = threadIdx.x; e < groups * TILE; e += kWarps * 32) {
            const int g = e / TILE, o = e % TILE;
            const int row = tile_row[g];
            if (row >= 0) {
                float *dst = out + (size_t)row * TILE + o;
                if (it.kind == kItemChunk) atomicAdd(dst, tile[g][o]); else *dst = tile[g][o];
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(kTmemCols) : "memory");
}

}  // namespace

const_status_t run_ttmc3_tensor(const const_csf *X, const float *U, const float *V, int R2, int R3, float *Y,
                                int64_t n_rows, int32_t *status, cudaStream_t stream) {
    if (R2 != R || R3 != R) return CONST_ERR_UNSUPPORTED;
    CB_CUDA(cudaMemsetAsync(Y, 0, sizeof(float) * TILE * n_rows, stream));
    if (X->nnz == 0) return CONST_OK;
    Csf3 x{X->crd[0], X->pos[1], X->crd[1], X->pos[2], X->crd[2], static_cast<const float *>(X->vals)};
    constexpr size_t dyn = kWarpBytes * kWarps;
    const DebugKnobs knobs = debug_knobs();
    CB_LAUNCH("chain3_tc_kernel", stream,
              chain3_tc_kernel<<<(unsigned)X->item_cap, kWarps * 32, dyn, stream>>>(X->items, X->bin_totals, X->light_list, x, U, V, Y, status,
                                                                                 knobs.spin_limit > 0 ? knobs.spin_limit : kMbarPolls, knobs.withhold));
    CB_CUDA(cudaGetLastError());
    return CONST_OK;
}

}  // namespace cb
