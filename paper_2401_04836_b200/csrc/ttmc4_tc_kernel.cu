// Fused order-4 TTMc with the dense per-slice stage on the tensor cores (tcgen05, accumulators in
// tensor memory).  Same chain as ttmc4_kernel.cu (Fig. 4(b) structure, fused on i -> j -> k):
//   P[c]   = sum_l X[i,j,k,l] W[l,c]      order-1 intermediate, reset per (i,j,k)
//   Q[b,c] = sum_k V[k,b] P[c]            order-2 intermediate, reset per (i,j)
//   Y[i,a,b,c] += U[j,a] Q[b,c]
// The last statement, summed over the fibres of a slice, is the contraction
//   Y_i[(b,c), a] = sum_f Q_f[(b,c)] * U[j_f, a]          M = 64, N = 8, K = fibres,
// which one tcgen05.mma of kind::tf32 consumes eight fibres at a time.
//
// Producer (CUDA cores).  The level-2 nodes of a warp's fibre range are dealt to NS = 8 streams of
// four lanes as equal contiguous runs, which the streams walk from end to end with node descriptors
// two nodes and factor rows one node ahead; lane h of a stream keeps rows b = 2h, 2h+1 of Q in
// registers.  When a stream's run leaves a fibre, or ends, its lanes park their part of Q, with the
// fibre's j, as one piece.  The contraction is linear in Q, so a piece is simply one K slot: a fibre
// cut between two streams occupies two slots with the same j and nothing has to be merged.  Every
// stream owns C slots; when a stream has to park and finds them taken, the warp flushes all 8 C slots
// (empty ones as zeros).
// C = 1 keeps the shared memory of a warp under 7 KB, so five blocks (twenty warps) fit on an SM, which
// pays more than the fuller MMAs of a larger C.
//
// Flush.  Operands in shared memory (no swizzle, K-major, as the shared-memory matrix descriptor
// defines it: core matrices of 8 rows x 16 bytes, i.e. 8 values of m (or n) by 4 consecutive K slots):
//   A[m, k] at (k / 8) * 2048 + ((k % 8) / 4) * 1024 + (m / 8) * 128 + (m % 8) * 16 + (k % 4) * 4   m = 8 b + c
//   B[n, k] at (k / 4) * 144 + n * 16 + (k % 4) * 4                                                 n = a
// (the 16 spare bytes per K quad of B stagger the banks for the lanes that write it).  K-major puts
// four K slots of one m side by side, while a stream finishes one slot at a time, so pieces are parked
// as plain rows and the flush transposes them: a lane reads column m of four pieces, splits, and
// stores 16 bytes of each operand.  One lane then issues three MMAs per group of eight slots and
// commits them to the warp's mbarrier; the streams go on walking while the tensor core works, and
// the next flush waits for that commit before it overwrites the operands.
// fp32 precision from tf32 products: every operand x is split into hi = tf32(x) (round to nearest)
// and lo = x - hi, and the three products hi*hi, lo*hi, hi*lo are accumulated in fp32 in tensor
// memory; the dropped lo*lo term and the truncation of lo are below 2^-20 relative per term.
//
// A block has four warps because a warp can read only its own quarter of the 128 tensor-memory
// lanes (rows 16w..16w+15 of an M = 64 accumulator live in lanes 32w..32w+15).  A block takes one
// work item: the four warps cut the fibres of a heavy slice or chunk in four by leaf count, and a
// light item (up to kWarpsPerBlock slices) gives each slice to kWarps / kWarpsPerBlock warps.  Every
// warp owns an 8-column accumulator and the epilogue adds the accumulators that belong to one slice.
// Every wait on an mbarrier is bounded; on a timeout the block records CONST_ERR_TIMEOUT in the
// status word, stops issuing MMAs, skips its stores and still frees its tensor memory.
#include "common.cuh"
#include "umma.cuh"

namespace cb {
namespace {

using namespace umma;

constexpr int R = 8;
constexpr int TILE = R * R * R;   // floats of one output row (slice)
constexpr int SL = 4;             // lanes per node stream
constexpr int NS = 32 / SL;       // node streams per warp
constexpr int C = 1;              // K slots (parked pieces) per stream between two flushes
constexpr int SLOTS = NS * C;     // K slots per flush
constexpr int KG = SLOTS / 8;     // groups of eight slots = MMAs per operand pair
constexpr int kWarps = 4;
constexpr int kWarpsPerLight = kWarps / kWarpsPerBlock;    // warps per slice of a light item
constexpr int kTmemCols = 32;     // kWarps accumulators of 8 columns
static_assert(SLOTS % 8 == 0 && SLOTS <= 32, "one lane per slot when the B operand is written");

constexpr int A_FLOATS = KG * 512;        // one A operand: [KG][2 K quads][8 m groups][8 m][4 k]
constexpr int B_QUAD = 36;                // floats per K quad of B: [8 n][4 k] + 4 spare
constexpr int B_FLOATS = KG * 2 * B_QUAD;
constexpr int RAW_ROW = 68;               // floats per parked piece (64 + 4 spare: staggers the banks)
constexpr int WARP_FLOATS = 2 * A_FLOATS + 2 * B_FLOATS + SLOTS * RAW_ROW;
constexpr int WARP_INTS = 32;             // Jslot[SLOTS]
constexpr size_t kWarpBytes = (sizeof(float) * WARP_FLOATS + sizeof(int32_t) * WARP_INTS + 127) / 128 * 128;

// instruction descriptor: D fp32, A and B tf32, both K-major, N = 8, M = 64
constexpr uint32_t kIdesc = idesc_tf32(64, 8);

struct Csf4 {
    const int32_t *crd0, *pos1, *crd1, *pos2, *crd2, *pos3, *crd3;
    const float *vals;
};

__device__ __forceinline__ int32_t leaf_of(const Csf4 &x, int32_t f1) { return __ldg(x.pos3 + __ldg(x.pos2 + f1)); }

__device__ __forceinline__ int32_t lower_bound_leaf(const Csf4 &x, int32_t lo, int32_t hi, int64_t target) {
    while (lo < hi) {
        int32_t mid = lo + (hi - lo) / 2;
        if ((int64_t)leaf_of(x, mid) < target) lo = mid + 1; else hi = mid;
    }
    return lo;
}

struct NodeInfo { int32_t k, pa, pb, l; float xv; };      // one level-2 node and its first leaf

// `pa` is the node's first leaf: the end of the node before it, which the caller already holds, so no
// address here waits for a load of the same call.
__device__ __forceinline__ NodeInfo load_node(const Csf4 &x, int32_t n, int32_t n_end, int32_t pa) {
    NodeInfo r{0, pa, pa, 0, 0.f};
    if (n < n_end) {
        r.k = __ldg(x.crd2 + n);
        r.pb = __ldg(x.pos3 + n + 1);
        r.l = __ldg(x.crd3 + pa);
        r.xv = __ldg(x.vals + pa);
    }
    return r;
}

__global__ void __launch_bounds__(kWarps * 32, 5)
ttmc4_tc_kernel(const WorkItem *__restrict__ items, const int32_t *__restrict__ bin_totals,
                const int32_t *__restrict__ light_list, Csf4 x,
                const float *__restrict__ U, const float *__restrict__ V, const float *__restrict__ W,
                float *__restrict__ out, int32_t *__restrict__ status, int wait_polls, int withhold) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t mbar_all[kWarps];
    __shared__ uint32_t tmem_base_s;
    __shared__ int32_t acc_row[kWarps];          // output row of every warp's accumulator, -1: none
    __shared__ int32_t acc_used[kWarps];         // the warp issued at least one MMA
    __shared__ int32_t failed;

    if ((int)blockIdx.x >= work_item_count(bin_totals)) return;      // the grid is an upper bound; nothing is held yet
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const WorkItem it = items[blockIdx.x];
    const bool light = it.kind == kItemLight;

    // this warp's share: part `part` of `parts` of the level-1 nodes [f0, f1) of `slice`, cut by leaf count
    int32_t slice = it.slice, f0 = it.f0, f1 = it.f1, fa = 0, fb = 0;
    int part = warp, parts = kWarps;
    if (light) {
        const int sl = warp / kWarpsPerLight;
        part = warp % kWarpsPerLight;
        parts = kWarpsPerLight;
        f0 = f1 = 0;
        if (sl < it.f0) {
            slice = __ldg(light_list + it.slice + sl);
            f0 = __ldg(x.pos1 + slice);
            f1 = __ldg(x.pos1 + slice + 1);
        }
    }
    if (f0 < f1) {
        const int64_t lo = leaf_of(x, f0), hi = leaf_of(x, f1);
        fa = part == 0 ? f0 : lower_bound_leaf(x, f0, f1, lo + (hi - lo) * part / parts);
        fb = part == parts - 1 ? f1 : lower_bound_leaf(x, f0, f1, lo + (hi - lo) * (part + 1) / parts);
    }

    const uint32_t mbar = smem_u32(&mbar_all[warp]);
    if (lane == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(mbar) : "memory");
        acc_row[warp] = fa < fb ? __ldg(x.crd0 + slice) : -1;
        acc_used[warp] = 0;
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
    const uint32_t d_tmem = tmem_base + 8u * warp;

    float *Ahi = reinterpret_cast<float *>(smem_raw + kWarpBytes * warp);
    float *Alo = Ahi + A_FLOATS;
    float *Bhi = Alo + A_FLOATS;
    float *Blo = Bhi + B_FLOATS;
    float *Raw = Blo + B_FLOATS;                                  // [SLOTS][RAW_ROW] parked pieces
    int32_t *Jslot = reinterpret_cast<int32_t *>(Raw + SLOTS * RAW_ROW);
    const uint32_t ahi_s = smem_u32(Ahi), alo_s = smem_u32(Alo), bhi_s = smem_u32(Bhi), blo_s = smem_u32(Blo);

    uint32_t parity = 0;
    bool pending = false, ok = true, first = true;
    const int st = lane / SL, h = lane % SL;
    int cnt = 0;                                                  // pieces this stream has parked since the last flush

    // Hands the parked pieces to the tensor core: Y_i += U_J^T Q_J over the 8 C slots.
    auto flush = [&]() {
        __syncwarp();
        unsigned vm[C];                                           // bit s * SL of vm[c]: slot c of stream s holds a piece
#pragma unroll
        for (int c = 0; c < C; ++c) vm[c] = __ballot_sync(0xffffffffu, cnt > c);
        // U rows of the slots, requested before anything waits
        float4 u0 = make_float4(0.f, 0.f, 0.f, 0.f), u1 = u0;
        if (lane < SLOTS && ((vm[lane % C] >> ((lane / C) * SL)) & 1u)) {
            const float *up = U + (size_t)Jslot[lane] * R;
            u0 = ldg4(up);
            u1 = ldg4(up + 4);
        }
        if (pending) {                                            // the MMAs of the previous flush still read the operands
            bool done = lane == 0 ? mbar_wait(mbar, parity, wait_polls) : true;
            done = __shfl_sync(0xffffffffu, done, 0);
            parity ^= 1;
            pending = false;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (!done) ok = false;
        }
        if (ok) {
#pragma unroll
            for (int u = 0; u < SLOTS / 2; ++u) {                 // A: (K quad, half of m) pairs
                const int quad = u >> 1, m = lane + 32 * (u & 1);
                float e[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const int slot = 4 * quad + q;
                    e[q] = ((vm[slot % C] >> ((slot / C) * SL)) & 1u) ? Raw[slot * RAW_ROW + m] : 0.f;
                }
                float4 hi4, lo4;
                split4(make_float4(e[0], e[1], e[2], e[3]), hi4, lo4);
                const int off = (quad >> 1) * 512 + (quad & 1) * 256 + (m >> 3) * 32 + (m & 7) * 4;
                *reinterpret_cast<float4 *>(Ahi + off) = hi4;
                *reinterpret_cast<float4 *>(Alo + off) = lo4;
            }
            if (lane < SLOTS) {                                   // B: one lane per K slot
                float4 h0, l0, h1, l1;
                split4(u0, h0, l0);
                split4(u1, h1, l1);
                float *bh = Bhi + (lane >> 2) * B_QUAD + (lane & 3), *bl = Blo + (lane >> 2) * B_QUAD + (lane & 3);
                bh[0] = h0.x; bh[4] = h0.y; bh[8] = h0.z; bh[12] = h0.w; bh[16] = h1.x; bh[20] = h1.y; bh[24] = h1.z; bh[28] = h1.w;
                bl[0] = l0.x; bl[4] = l0.y; bl[8] = l0.z; bl[12] = l0.w; bl[16] = l1.x; bl[20] = l1.y; bl[24] = l1.z; bl[28] = l1.w;
            }
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // operand stores -> visible to the tensor core
            __syncwarp();
            if (lane == 0) {
#pragma unroll
                for (int kg = 0; kg < KG && !withhold; ++kg) {   // (test hook: nothing issued, nothing committed)
                    const uint64_t a_hi = smem_desc(ahi_s + kg * 2048, 1024, 128), a_lo = smem_desc(alo_s + kg * 2048, 1024, 128);
                    const uint64_t b_hi = smem_desc(bhi_s + kg * (8 * B_QUAD), 4 * B_QUAD, 128);
                    const uint64_t b_lo = smem_desc(blo_s + kg * (8 * B_QUAD), 4 * B_QUAD, 128);
                    umma_tf32(d_tmem, a_hi, b_hi, kIdesc, (first && kg == 0) ? 0u : 1u);
                    umma_tf32(d_tmem, a_lo, b_hi, kIdesc, 1u);
                    umma_tf32(d_tmem, a_hi, b_lo, kIdesc, 1u);
                }
                if (!withhold) umma_commit(mbar);               // withheld: the next bounded wait runs out
                acc_used[warp] = 1;
            }
            pending = true;
            first = false;
        }
        cnt = 0;
        __syncwarp();
    };

    if (fa < fb) {
        const int32_t N0 = __ldg(x.pos2 + fa), N1 = __ldg(x.pos2 + fb);
        const int32_t per = (N1 - N0 + NS - 1) / NS;
        const int32_t na = N0 + st * per;
        const int32_t nb = na + per < N1 ? na + per : N1;
        int32_t f = fa;
        if (na < nb) {                                            // fibre holding node na
            int32_t lo = fa, hi = fb - 1;
            while (lo < hi) {
                const int32_t mid = lo + (hi - lo + 1) / 2;
                if (__ldg(x.pos2 + mid) <= na) lo = mid; else hi = mid - 1;
            }
            f = lo;
        }
        const int32_t flast = fb - 1;
        int32_t fend = __ldg(x.pos2 + f + 1);                     // end of fibre f; the fibre after it is fetched ahead
        int32_t fend_n = __ldg(x.pos2 + (f + 2 <= fb ? f + 2 : fb));
        int32_t jc = __ldg(x.crd1 + f), jn = __ldg(x.crd1 + (f + 1 <= flast ? f + 1 : flast));
        float Q[2][R];
#pragma unroll
        for (int c = 0; c < R; ++c) Q[0][c] = Q[1][c] = 0.f;

        // software pipeline over the nodes of the run: descriptors two nodes ahead, rows one node ahead
        NodeInfo cur = load_node(x, na, nb, na < nb ? __ldg(x.pos3 + na) : 0);
        NodeInfo nxt = load_node(x, na + 1, nb, cur.pb);
        float4 w0 = ldg4(W + (size_t)cur.l * R), w1 = ldg4(W + (size_t)cur.l * R + 4);
        float2 vb = __ldg(reinterpret_cast<const float2 *>(V + (size_t)cur.k * R + 2 * h));
        for (int32_t t = 0; t < per && ok; ++t) {
            const int32_t n = na + t;
            const NodeInfo nn = load_node(x, n + 2, nb, nxt.pb);
            float4 w0n = w0, w1n = w1;
            float2 vbn = vb;
            if (n + 1 < nb) {
                w0n = ldg4(W + (size_t)nxt.l * R);
                w1n = ldg4(W + (size_t)nxt.l * R + 4);
                vbn = __ldg(reinterpret_cast<const float2 *>(V + (size_t)nxt.k * R + 2 * h));
            }
            bool parks = false;
            if (n < nb) {
                // P = sum over the node's leaves of X * W[l, :]
                float P[R] = {cur.xv * w0.x, cur.xv * w0.y, cur.xv * w0.z, cur.xv * w0.w,
                              cur.xv * w1.x, cur.xv * w1.y, cur.xv * w1.z, cur.xv * w1.w};
                for (int32_t p = cur.pa + 1; p < cur.pb; ++p) {   // further leaves of the node (rare when sparse)
                    const float xv = __ldg(x.vals + p);
                    const float *w = W + (size_t)__ldg(x.crd3 + p) * R;
                    const float4 a0 = ldg4(w), a1 = ldg4(w + 4);
                    P[0] = fmaf(xv, a0.x, P[0]); P[1] = fmaf(xv, a0.y, P[1]);
                    P[2] = fmaf(xv, a0.z, P[2]); P[3] = fmaf(xv, a0.w, P[3]);
                    P[4] = fmaf(xv, a1.x, P[4]); P[5] = fmaf(xv, a1.y, P[5]);
                    P[6] = fmaf(xv, a1.z, P[6]); P[7] = fmaf(xv, a1.w, P[7]);
                }
#pragma unroll
                for (int c = 0; c < R; ++c) {                     // Q[b, :] += V[k, b] * P[:]
                    Q[0][c] = fmaf(vb.x, P[c], Q[0][c]);
                    Q[1][c] = fmaf(vb.y, P[c], Q[1][c]);
                }
                parks = n + 1 == fend || n + 1 == nb;             // the run leaves fibre f, or ends inside it
            }
            // flush as late as possible: only when a stream that has to park finds its slots taken
            if (__any_sync(0xffffffffu, parks && cnt == C)) flush();
            if (parks && ok) {
                const int slot = st * C + cnt;
                float *dst = Raw + slot * RAW_ROW + 2 * h * R;
#pragma unroll
                for (int b2 = 0; b2 < 2; ++b2) {
                    *reinterpret_cast<float4 *>(dst + b2 * R) = make_float4(Q[b2][0], Q[b2][1], Q[b2][2], Q[b2][3]);
                    *reinterpret_cast<float4 *>(dst + b2 * R + 4) = make_float4(Q[b2][4], Q[b2][5], Q[b2][6], Q[b2][7]);
                    Q[b2][0] = Q[b2][1] = Q[b2][2] = Q[b2][3] = Q[b2][4] = Q[b2][5] = Q[b2][6] = Q[b2][7] = 0.f;
                }
                if (h == 0) Jslot[slot] = jc;
                ++cnt;
                if (n + 1 == fend) {
                    ++f;
                    fend = fend_n;
                    jc = jn;
                    fend_n = __ldg(x.pos2 + (f + 2 <= fb ? f + 2 : fb));
                    jn = __ldg(x.crd1 + (f + 1 <= flast ? f + 1 : flast));
                }
            }
            cur = nxt; nxt = nn; w0 = w0n; w1 = w1n; vb = vbn;
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

    // ---- epilogue: warp w holds rows m = 16 w + lane (lane < 16) of every accumulator
    if (!failed) {
        uint32_t r[kWarps][R];
#pragma unroll
        for (int a = 0; a < kWarps; ++a) {
            const uint32_t taddr = tmem_base + ((uint32_t)(32 * warp) << 16) + 8u * a;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                         : "=r"(r[a][0]), "=r"(r[a][1]), "=r"(r[a][2]), "=r"(r[a][3]), "=r"(r[a][4]), "=r"(r[a][5]),
                           "=r"(r[a][6]), "=r"(r[a][7])
                         : "r"(taddr));
        }
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        if (lane < 16) {
            const int m = 16 * warp + lane;
            // accumulators of the same slice are added: all four for a heavy slice or chunk,
            // kWarpsPerLight neighbours for every slice of a light item
            const int group = light ? kWarpsPerLight : kWarps;
#pragma unroll
            for (int g0 = 0; g0 < kWarps; g0 += kWarpsPerLight) {
                if (g0 % group != 0) continue;
                float sum[R];
                int row = -1;
#pragma unroll
                for (int n = 0; n < R; ++n) sum[n] = 0.f;
#pragma unroll
                for (int a = 0; a < kWarps; ++a) {
                    if (a >= g0 && a < g0 + group && acc_row[a] >= 0 && acc_used[a]) {
                        row = acc_row[a];
#pragma unroll
                        for (int n = 0; n < R; ++n) sum[n] += __uint_as_float(r[a][n]);
                    }
                }
                if (row >= 0) {
                    float *dst = out + (size_t)row * TILE + m;
                    if (it.kind == kItemChunk) {
#pragma unroll
                        for (int n = 0; n < R; ++n) atomicAdd(dst + n * 64, sum[n]);
                    } else {
#pragma unroll
                        for (int n = 0; n < R; ++n) dst[n * 64] = sum[n];
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem_base), "r"(kTmemCols) : "memory");
}

}  // namespace

const_status_t run_ttmc4_tensor(const const_csf *X, const float *U, const float *V, const float *W, int rank, float *Y,
                                int64_t n_rows, int32_t *status, cudaStream_t stream) {
    if (rank != R) return CONST_ERR_UNSUPPORTED;
    CB_CUDA(cudaMemsetAsync(Y, 0, sizeof(float) * TILE * n_rows, stream));
    if (X->nnz == 0) return CONST_OK;
    Csf4 x{X->crd[0], X->pos[1], X->crd[1], X->pos[2], X->crd[2], X->pos[3], X->crd[3],
           static_cast<const float *>(X->vals)};
    constexpr size_t dyn = kWarpBytes * kWarps;
    static PerDeviceOnce attr_once;                     // per template instance
    CB_CUDA(once_per_device(attr_once, [&] { return cudaFuncSetAttribute(ttmc4_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn); }));
    const unsigned grid = (unsigned)X->item_cap;
    const DebugKnobs knobs = debug_knobs();
    CB_LAUNCH("ttmc4_tc_kernel", stream,
              ttmc4_tc_kernel<<<grid, kWarps * 32, dyn, stream>>>(X->items, X->bin_totals, X->light_list, x, U, V, W, Y, status,
                                                               knobs.spin_limit > 0 ? knobs.spin_limit : kMbarPolls, knobs.withhold));
    CB_CUDA(cudaGetLastError());
    return CONST_OK;
}

}  // namespace cb
