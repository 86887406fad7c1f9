// GPU CSF builder (Sec. 2.1, CSF representation): pack -> LSD radix sort -> per-level compression,
// followed by the per-slice load-balancing lists used by the fused contraction kernels.
//
// Layout decisions
//   * The permuted coordinate tuple is packed into one 64-bit key, root level in the top bits, so a
//     single key sort orders the nonzeros lexicographically by the chosen mode order.
//   * The value travels with its key as the sort payload, so no gather pass is needed afterwards and
//     the sorted payload buffer *is* the leaf value array.
//   * The sort is a least-significant-digit radix sort with 8-bit digits.  Each pass is one kernel:
//     tiles are ranked in shared memory, the tile's digit counts are chained to earlier tiles with a
//     decoupled look-back (every spin is bounded and reports CONST_ERR_TIMEOUT), and keys are
//     reordered in shared memory so that global stores run over consecutive addresses.
//   * Compression is flag / scan / scatter: element e opens a node at level l when its length-(l+1)
//     prefix differs from that of e-1.
#include <algorithm>
#include <cstring>
#include <new>

#include "common.cuh"

namespace cb {
namespace {

// ------------------------------------------------------------------------------------------------
// pack
// ------------------------------------------------------------------------------------------------
struct PackArgs {
    const int32_t *c[kMaxOrder];   // coordinates of the mode stored at level l
    int64_t dim[kMaxOrder];
    int shift[kMaxOrder];
    int order;
};

enum DevErr : int32_t { kErrNone = 0 };

__device__ __forceinline__ void report(int32_t *status, int32_t code) { atomicCAS(status, 0, code); }

constexpr int kRsMaxBits = 9;                     // widest digit of a radix pass
constexpr int kRsMaxBins = 1 << kRsMaxBits;
constexpr int kMaxPasses = 8;

// Digits of the radix passes.  A pass sorts on `bits[p]` key bits starting at `shift[p]`; the widths
// are 8 or 9 bits (the width the pass kernel is instantiated for), chosen so that the key is covered
// in as few passes as possible.
struct DigitPlan { int shift[kMaxPasses]; int bits[kMaxPasses]; int passes; };

// Pack the permuted coordinates of every nonzero into its 64-bit sort key (range-checked) and, in the
// same read, count the digits of every radix pass.  Per-block counts live in shared memory and are
// flushed once; the grid is sized to a few blocks per SM so the flush stays small.
template <int ORDER>
__global__ void __launch_bounds__(256) pack_hist(PackArgs a, int64_t nnz, DigitPlan dp, uint64_t *__restrict__ keys,
                                                 uint32_t *__restrict__ hist, int32_t *status) {
    extern __shared__ uint32_t sh[];                 // [passes][kRsMaxBins]
    for (int x = threadIdx.x; x < dp.passes * kRsMaxBins; x += blockDim.x) sh[x] = 0;
    __syncthreads();
    bool bad = false;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < nnz; e += stride) {
        uint64_t key = 0;
#pragma unroll
        for (int l = 0; l < ORDER; ++l) {
            int64_t c = __ldg(a.c[l] + e);
            if (c < 0 || c >= a.dim[l]) { bad = true; c = 0; }
            key |= (uint64_t)c << a.shift[l];
        }
        keys[e] = key;
        // unrolled over the maximum so that the plan is read with constant indices (a runtime index would
        // send the parameter arrays through local memory, ten loads per nonzero)
#pragma unroll
        for (int p = 0; p < kMaxPasses; ++p)
            if (p < dp.passes)
                atomicAdd(&sh[p * kRsMaxBins + ((unsigned)(key >> dp.shift[p]) & ((1u << dp.bits[p]) - 1u))], 1u);
    }
    if (bad) report(status, CONST_ERR_COORD_RANGE);
    __syncthreads();
    for (int x = threadIdx.x; x < dp.passes * kRsMaxBins; x += blockDim.x)
        if (sh[x]) atomicAdd(&hist[x], sh[x]);
}

inline void launch_pack_hist(const PackArgs &pa, int64_t nnz, const DigitPlan &dp, uint64_t *keys, uint32_t *hist,
                             int32_t *status, cudaStream_t stream) {
    const int blocks = (int)std::min<int64_t>((nnz + 255) / 256, 148 * 8);
    const size_t sm = sizeof(uint32_t) * kRsMaxBins * std::max(dp.passes, 1);
    switch (pa.order) {
        case 2: pack_hist<2><<<blocks, 256, sm, stream>>>(pa, nnz, dp, keys, hist, status); break;
        case 3: pack_hist<3><<<blocks, 256, sm, stream>>>(pa, nnz, dp, keys, hist, status); break;
        default: pack_hist<4><<<blocks, 256, sm, stream>>>(pa, nnz, dp, keys, hist, status); break;
    }
}

// ------------------------------------------------------------------------------------------------
// radix sort
// ------------------------------------------------------------------------------------------------
constexpr int kRsThreads = 256;
constexpr int kRsItems = 16;
constexpr int kRsTile = kRsThreads * kRsItems;     // 4096 keys per tile
constexpr int kRsWarps = kRsThreads / 32;
constexpr int kSpinLimit = 1 << 21;
// Distance, in tiles, of the pass kernel's L2 prefetch: half a wave of its resident blocks (148 SMs x 3).  Measured on
// 38.5 M nonzeros: none 0.326 ms per pass, 56 to 444 tiles 0.311 ms, 888 and more 0.336 ms (evicted before use).
constexpr int kRsAheadTiles = 222;
// A tile's state for one digit is one 64-bit word: the count in the low half; in the high half
// (pass number << 2) | flag, flag 1 = the tile's own count, flag 2 = the count summed over this and
// every earlier tile.  A word counts only if it carries the current pass number, so the array is
// cleared once per sort, not once per pass.
constexpr unsigned kFlagOwn = 1u, kFlagPrefix = 2u;

__device__ __forceinline__ unsigned long long status_word(unsigned epoch, unsigned flag, uint32_t count) {
    return ((unsigned long long)((epoch << 2) | flag) << 32) | count;
}

// Exclusive scan of each pass's digit histogram: one block per pass.
__global__ void __launch_bounds__(256) rs_scan_hist(uint32_t *hist) {
    __shared__ uint32_t sh[kRsMaxBins];
    uint32_t *h = hist + blockIdx.x * kRsMaxBins;
    for (int x = threadIdx.x; x < kRsMaxBins; x += blockDim.x) sh[x] = h[x];
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t run = 0;
        for (int d = 0; d < kRsMaxBins; ++d) { uint32_t c = sh[d]; sh[d] = run; run += c; }
    }
    __syncthreads();
    for (int x = threadIdx.x; x < kRsMaxBins; x += blockDim.x) h[x] = sh[x];
}

// One radix pass over BITS key bits.  Thread t owns digits t, t + 256, ... (DPT of them).
template <typename V, int BITS>
__global__ void __launch_bounds__(kRsThreads, 3) rs_onesweep(const uint64_t *__restrict__ kin, uint64_t *__restrict__ kout,
                                                            const V *__restrict__ vin, V *__restrict__ vout, int64_t n,
                                                            int shift, const uint32_t *__restrict__ digit_base,
                                                            unsigned long long *status, uint32_t *counter,
                                                            int32_t *err, unsigned epoch, int spin_limit, int withhold, int ahead_tiles) {
    constexpr int kBins = 1 << BITS;
    constexpr unsigned kDigitMask = kBins - 1;
    constexpr int DPT = kBins / kRsThreads;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint64_t *keybuf = reinterpret_cast<uint64_t *>(smem_raw);
    V *valbuf = reinterpret_cast<V *>(smem_raw + kRsTile * sizeof(uint64_t));
    __shared__ uint32_t warp_hist[kRsWarps][kBins];
    __shared__ uint32_t digit_excl[kBins];
    __shared__ uint32_t s_gbase[kBins];
    __shared__ uint32_t warp_tot[DPT][kRsWarps];
    __shared__ uint32_t s_tile;
    __shared__ int s_abort;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { s_tile = atomicAdd(counter, 1u); s_abort = 0; }
    for (int x = threadIdx.x; x < kRsWarps * kBins; x += kRsThreads) (&warp_hist[0][0])[x] = 0;
    __syncthreads();
    const uint32_t tile = s_tile;
    const int64_t tile_base = (int64_t)tile * kRsTile;
    if (tile_base >= n) return;                       // never happens: the grid has exactly ceil(n / tile) blocks
    const int64_t left = n - tile_base;
    const int nvalid = left < kRsTile ? (int)left : kRsTile;

    // A tile that will be taken soon (half a wave of resident blocks ahead) is requested into L2 now, so that the
    // loads of the block that takes it find it there instead of in DRAM.
    {
        const int64_t ahead = tile_base + (int64_t)ahead_tiles * kRsTile;
        const int64_t kb = ahead * (int64_t)sizeof(uint64_t) + (int64_t)threadIdx.x * 128;       // keys: 32 KB = 256 lines
        if (ahead + kRsTile <= n) {
            asm volatile("prefetch.global.L2 [%0];" :: "l"(reinterpret_cast<const char *>(kin) + kb));
            const int64_t vb = ahead * (int64_t)sizeof(V) + (int64_t)threadIdx.x * 128;
            if ((int64_t)threadIdx.x * 128 < (int64_t)kRsTile * (int64_t)sizeof(V))
                asm volatile("prefetch.global.L2 [%0];" :: "l"(reinterpret_cast<const char *>(vin) + vb));
        }
    }

    // this thread's slots of the tile: local indices mine + 32 i
    const int mine = warp * (32 * kRsItems) + lane;
    const uint64_t *ktile = kin + tile_base + mine;
    uint64_t key[kRsItems];
#pragma unroll
    for (int i = 0; i < kRsItems; ++i)
        key[i] = mine + i * 32 < nvalid ? ktile[i * 32] : ~0ull;   // padding sorts after every real key of the tile

    // Digit counts of the tile first, so that later tiles can see them as early as possible:
    // the time from taking a tile to publishing its counts decides how long others wait.
    volatile unsigned long long *st = status;
    uint32_t count[DPT];

    // Rank inside the warp: keys with equal digits keep their order (item, lane).  The lanes holding
    // another digit are collected from one ballot per digit bit (the match instruction costs one
    // round per distinct value in the warp, which for random digits is far slower).
    int rank[kRsItems];
#pragma unroll
    for (int i = 0; i < kRsItems; ++i) {
        const unsigned dg = (unsigned)(key[i] >> shift) & kDigitMask;
        unsigned other = 0;
#pragma unroll
        for (int b = 0; b < BITS; ++b) {
            const bool bit = (dg >> b) & 1u;
            const unsigned m = __ballot_sync(0xffffffffu, bit);
            other |= bit ? ~m : m;                                     // lanes whose bit b differs from mine
        }
        const unsigned peers = ~other;
        const int leader = __ffs(peers) - 1;
        uint32_t old = 0;
        if (lane == leader) old = atomicAdd(&warp_hist[warp][dg], (uint32_t)__popc(peers));
        old = __shfl_sync(0xffffffffu, old, leader);
        rank[i] = (int)old + __popc(peers & ((1u << lane) - 1u));
    }
    __syncthreads();

    // offsets of each warp's run inside the digit, digit scan inside the tile (digits in order:
    // all of q = 0 first, then q = 1)
    uint32_t incl[DPT];
#pragma unroll
    for (int q = 0; q < DPT; ++q) {
        const int d = q * kRsThreads + threadIdx.x;
        uint32_t run = 0;
#pragma unroll
        for (int w = 0; w < kRsWarps; ++w) {
            uint32_t c = warp_hist[w][d];
            warp_hist[w][d] = run;
            run += c;
        }
        count[q] = run;     // the tile's count of digit d: published now, so that later tiles can go on
        if (!withhold)      // (test hook: with the counts withheld, every later tile's bounded wait runs out)
            st[(size_t)tile * kBins + d] = status_word(epoch, tile == 0 ? kFlagPrefix : kFlagOwn, count[q]);
        incl[q] = count[q];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            uint32_t v = __shfl_up_sync(0xffffffffu, incl[q], off);
            if (lane >= off) incl[q] += v;
        }
        if (lane == 31) warp_tot[q][warp] = incl[q];
    }
    __syncthreads();
    uint32_t excl[DPT];
    {
        uint32_t carry = 0;
#pragma unroll
        for (int q = 0; q < DPT; ++q) {
            uint32_t wbase = 0, total = 0;
#pragma unroll
            for (int w = 0; w < kRsWarps; ++w) {
                const uint32_t c = warp_tot[q][w];
                if (w < warp) wbase += c;
                total += c;
            }
            excl[q] = carry + wbase + incl[q] - count[q];
            digit_excl[q * kRsThreads + threadIdx.x] = excl[q];
            carry += total;
        }
    }
    __syncthreads();

    // Reorder in shared memory first (the payload is fetched only now: it is not needed for ranking).
    // This needs tile-local offsets only, so it runs before the look-back: by the time the global
    // prefix is needed, most predecessors have published theirs and little time is spent polling.
    {
        const V *vtile = vin + tile_base + mine;
#pragma unroll
        for (int i = 0; i < kRsItems; ++i) {
            const V val = mine + i * 32 < nvalid ? vtile[i * 32] : V(0);
            const unsigned dg = (unsigned)(key[i] >> shift) & kDigitMask;
            const int p = (int)digit_excl[dg] + (int)warp_hist[warp][dg] + rank[i];
            keybuf[p] = key[i];
            valbuf[p] = val;
        }
    }

    // Chained scan over tiles (decoupled look-back); every wait is bounded.  Most predecessors met
    // on the way have published only their own counts, so those are taken kLook at a time with one
    // test; a tile that is not ready yet, or one that carries a prefix, is handled one by one.
    const unsigned tag_own = (epoch << 2) | kFlagOwn, tag_prefix = (epoch << 2) | kFlagPrefix;
    bool ok = true;
#pragma unroll
    for (int q = 0; q < DPT; ++q) {
        const int d = q * kRsThreads + threadIdx.x;
        uint32_t before = 0;
        if (tile > 0) {
            constexpr int kLook = 8;
            volatile unsigned long long *p = st + (size_t)(tile - 1) * kBins + d;   // nearest tile not yet added
            uint32_t togo = tile;                                                    // tiles from p down to tile 0
            bool done = false;
            while (ok && !done) {
                if (togo >= (uint32_t)kLook) {
                    unsigned long long s[kLook];
#pragma unroll
                    for (int b = 0; b < kLook; ++b) s[b] = *(p - (ptrdiff_t)b * kBins);
                    bool all_own = true;
                    uint32_t sum = 0;
#pragma unroll
                    for (int b = 0; b < kLook; ++b) {
                        all_own = all_own && (unsigned)(s[b] >> 32) == tag_own;
                        sum += (uint32_t)s[b];
                    }
                    if (all_own) {
                        before += sum;
                        p -= (ptrdiff_t)kLook * kBins;
                        togo -= kLook;
                        continue;
                    }
                    // take the leading words that are ready; stop behind a prefix or at an unready one
                    int taken = 0;
                    bool stop = false;
#pragma unroll
                    for (int b = 0; b < kLook; ++b) {
                        const unsigned h = (unsigned)(s[b] >> 32);
                        if (!stop && (h == tag_own || h == tag_prefix)) {
                            before += (uint32_t)s[b];
                            ++taken;
                            if (h == tag_prefix) { done = true; stop = true; }
                        } else {
                            stop = true;
                        }
                    }
                    p -= (ptrdiff_t)taken * kBins;
                    togo -= taken;
                    if (done) break;
                }
                unsigned long long v = *p;
                int spins = 0;
                while ((unsigned)(v >> 32) != tag_own && (unsigned)(v >> 32) != tag_prefix) {
                    if (++spins > spin_limit) { ok = false; break; }
                    __nanosleep(spins < 8 ? 200 : 1000);   // back off at once: polling warps must not crowd the issue slots
                    v = *p;
                }
                if (!ok) break;
                before += (uint32_t)v;
                done = (unsigned)(v >> 32) == tag_prefix;   // tile 0 always carries a prefix, so the walk ends there at the latest
                p -= kBins;
                --togo;
            }
            if (ok && !withhold) st[(size_t)tile * kBins + d] = status_word(epoch, kFlagPrefix, before + count[q]);
        }
        s_gbase[d] = digit_base[d] + before - excl[q];      // modulo 2^32; adding a tile-local position gives the true offset
    }
    if (!ok) {
        report(err, CONST_ERR_TIMEOUT);
        s_abort = 1;
    }
    __syncthreads();
    if (s_abort) return;

    // store runs of consecutive addresses
#pragma unroll
    for (int m = 0; m < kRsItems; ++m) {
        const int p = threadIdx.x + m * kRsThreads;
        if (p < nvalid) {
            const uint64_t k = keybuf[p];
            const unsigned dg = (unsigned)(k >> shift) & kDigitMask;
            const uint32_t o = s_gbase[dg] + (uint32_t)p;
            kout[o] = k;
            vout[o] = valbuf[p];
        }
    }
}

// ------------------------------------------------------------------------------------------------
// compression: flags -> counts -> scan -> scatter
// ------------------------------------------------------------------------------------------------
constexpr int kCpThreads = 256;
constexpr int kCpIters = 8;                                   // 32-element steps per warp
constexpr int kCpTile = kCpThreads * kCpIters;                // 2048 elements per block
constexpr int kCpLevels = kMaxOrder - 1;                      // levels that need a scan (all but the leaf level)
constexpr int kCpAheadTiles = 592;                            // L2 prefetch distance of the one-shot tile kernels (half a wave)

// Requests the keys of the tile `kCpAheadTiles` after this block's into L2 (threads 0..127 take one line each).
__device__ __forceinline__ void prefetch_tile_ahead(const uint64_t *__restrict__ keys, int64_t n) {
    const int64_t first = ((int64_t)blockIdx.x + kCpAheadTiles) * kCpTile;
    if (threadIdx.x < kCpTile * (int)sizeof(uint64_t) / 128 && first + kCpTile <= n)
        asm volatile("prefetch.global.L2 [%0];" :: "l"(reinterpret_cast<const char *>(keys + first) + threadIdx.x * 128));
}

struct LevelShifts { int shift[kMaxOrder]; int order; };

// ballots of "opens a new node at level l" for the 32 elements starting at `base`
__device__ __forceinline__ void node_flags(const uint64_t *__restrict__ keys, int64_t n, int64_t base, int lane,
                                           const LevelShifts &ls, uint64_t &key, unsigned ballots[kCpLevels],
                                           bool &dup) {
    int64_t e = base + lane;
    bool in = e < n;
    key = in ? keys[e] : 0ull;
    uint64_t prev = __shfl_up_sync(0xffffffffu, key, 1);
    if (lane == 0 && in && e > 0) prev = keys[e - 1];
    bool first = (e == 0);
    dup = in && !first && key == prev;
#pragma unroll
    for (int l = 0; l < kCpLevels; ++l) {
        bool f = false;
        if (l < ls.order - 1) f = in && (first || (key >> ls.shift[l]) != (prev >> ls.shift[l]));
        ballots[l] = __ballot_sync(0xffffffffu, f);
    }
}

// the same flags from a key the caller already holds; `carry` = the element before `base` (unused when base == 0)
__device__ __forceinline__ void node_flags_of(int64_t n, int64_t base, int lane, const LevelShifts &ls, uint64_t key,
                                              uint64_t carry, unsigned ballots[kCpLevels]) {
    const int64_t e = base + lane;
    const bool in = e < n;
    uint64_t prev = __shfl_up_sync(0xffffffffu, key, 1);
    if (lane == 0) prev = carry;
    const bool first = (e == 0);
#pragma unroll
    for (int l = 0; l < kCpLevels; ++l) {
        bool f = false;
        if (l < ls.order - 1) f = in && (first || (key >> ls.shift[l]) != (prev >> ls.shift[l]));
        ballots[l] = __ballot_sync(0xffffffffu, f);
    }
}

__global__ void __launch_bounds__(kCpThreads) csf_count(const uint64_t *__restrict__ keys, int64_t n, LevelShifts ls,
                                                       uint32_t *__restrict__ block_counts, int32_t *status) {
    __shared__ uint32_t sh[kCpLevels];
    if (threadIdx.x < kCpLevels) sh[threadIdx.x] = 0;
    prefetch_tile_ahead(keys, n);
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t cnt[kCpLevels] = {0, 0, 0};
    bool any_dup = false;
    for (int it = 0; it < kCpIters; ++it) {
        int64_t base = (int64_t)blockIdx.x * kCpTile + (warp * kCpIters + it) * 32;
        uint64_t key; unsigned b[kCpLevels]; bool dup;
        node_flags(keys, n, base, lane, ls, key, b, dup);
        any_dup |= dup;
#pragma unroll
        for (int l = 0; l < kCpLevels; ++l) cnt[l] += __popc(b[l]);
    }
    if (any_dup) report(status, CONST_ERR_DUPLICATE_COORD);
    if (lane == 0)
        for (int l = 0; l < kCpLevels; ++l) atomicAdd(&sh[l], cnt[l]);
    __syncthreads();
    if (threadIdx.x < kCpLevels) block_counts[(int64_t)blockIdx.x * kCpLevels + threadIdx.x] = sh[threadIdx.x];
}

// In-place exclusive scan of the per-block counts, in two launches: every scan block adds up its chunk of
// kScanChunk counts; then every scan block adds the sums of the chunks before its own (a few dozen numbers) and
// scans its chunk.  totals[l] receives the level sizes.  `partials` has room for kCpLevels numbers per chunk.
constexpr int kScanThreads = 256, kScanPer = 4, kScanChunk = kScanThreads * kScanPer;

__device__ __forceinline__ uint32_t block_sum(uint32_t v, uint32_t *sh) {     // sum over the block, result in every thread
    v = __reduce_add_sync(0xffffffffu, v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    uint32_t s = 0;
    for (int w = 0; w < kScanThreads / 32; ++w) s += sh[w];
    return s;
}

__global__ void __launch_bounds__(kScanThreads) csf_scan_partials(const uint32_t *__restrict__ block_counts, int64_t nblocks,
                                                                  uint32_t *__restrict__ partials) {
    __shared__ uint32_t sh[kScanThreads / 32];
    uint32_t mine[kCpLevels] = {0, 0, 0};
    for (int k = 0; k < kScanPer; ++k) {
        const int64_t b = (int64_t)blockIdx.x * kScanChunk + k * kScanThreads + threadIdx.x;
        if (b < nblocks)
#pragma unroll
            for (int l = 0; l < kCpLevels; ++l) mine[l] += block_counts[b * kCpLevels + l];
    }
#pragma unroll
    for (int l = 0; l < kCpLevels; ++l) {
        const uint32_t s = block_sum(mine[l], sh);
        if (threadIdx.x == 0) partials[(int64_t)blockIdx.x * kCpLevels + l] = s;
    }
}

__global__ void __launch_bounds__(kScanThreads) csf_scan_apply(uint32_t *block_counts, int64_t nblocks,
                                                               const uint32_t *__restrict__ partials, uint32_t *totals) {
    __shared__ uint32_t sh[kScanThreads / 32];
    __shared__ uint32_t wsum[kScanThreads / 32][kCpLevels];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // counts of kScanPer consecutive blocks per thread
    uint32_t c[kScanPer][kCpLevels], mine[kCpLevels] = {0, 0, 0};
    const int64_t b0 = (int64_t)blockIdx.x * kScanChunk + (int64_t)threadIdx.x * kScanPer;
#pragma unroll
    for (int k = 0; k < kScanPer; ++k)
#pragma unroll
        for (int l = 0; l < kCpLevels; ++l) {
            c[k][l] = b0 + k < nblocks ? block_counts[(b0 + k) * kCpLevels + l] : 0;
            mine[l] += c[k][l];
        }
#pragma unroll
    for (int l = 0; l < kCpLevels; ++l) {
        // sum of the chunks in front of this one
        uint32_t before = 0;
        for (int q = threadIdx.x; q < (int)blockIdx.x; q += kScanThreads) before += partials[(int64_t)q * kCpLevels + l];
        before = block_sum(before, sh);
        // exclusive scan of the threads' sums
        uint32_t inc = mine[l];
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const uint32_t t = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += t;
        }
        if (lane == 31) wsum[warp][l] = inc;
        __syncthreads();
        uint32_t run = before + inc - mine[l];
        for (int w = 0; w < warp; ++w) run += wsum[w][l];
#pragma unroll
        for (int k = 0; k < kScanPer; ++k) {
            if (b0 + k < nblocks) block_counts[(b0 + k) * kCpLevels + l] = run;
            run += c[k][l];
        }
        if (b0 <= nblocks - 1 && nblocks - 1 < b0 + kScanPer) totals[l] = run;     // the thread that owns the last block
    }
}

inline void launch_csf_scan(uint32_t *block_counts, int64_t nblocks, uint32_t *totals, cudaStream_t stream) {
    const unsigned chunks = (unsigned)((nblocks + kScanChunk - 1) / kScanChunk);
    uint32_t *partials = block_counts + nblocks * kCpLevels;        // behind the counts (see scan_partials_room)
    CB_LAUNCH("csf_scan_partials", stream, csf_scan_partials<<<chunks, kScanThreads, 0, stream>>>(block_counts, nblocks, partials));
    CB_LAUNCH("csf_scan_apply", stream, csf_scan_apply<<<chunks, kScanThreads, 0, stream>>>(block_counts, nblocks, partials, totals));
}

// numbers to allocate behind the per-block counts for the chunk sums of the scan
inline int64_t scan_partials_room(int64_t nblocks) { return kCpLevels * ((nblocks + kScanChunk - 1) / kScanChunk + 1); }

struct CsfArrays {
    int32_t *pos[kMaxOrder];
    int32_t *crd[kMaxOrder];
    int bits[kMaxOrder];
};

// ORDER is a template parameter so that the per-level arrays are indexed by constants and stay in registers.
template <int ORDER>
__global__ void __launch_bounds__(kCpThreads) csf_scatter(const uint64_t *__restrict__ keys, int64_t n, LevelShifts ls,
                                                         const uint32_t *__restrict__ block_base, CsfArrays out) {
    __shared__ uint32_t wcnt[kCpThreads / 32][kCpLevels];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    prefetch_tile_ahead(keys, n);
    uint64_t key[kCpIters];
    unsigned bal[kCpIters][kCpLevels];
    uint32_t cnt[kCpLevels] = {0, 0, 0};
    // the warp's kCpIters * 32 consecutive keys and the one in front of them, all requested before the first is used
    const int64_t warp_base = (int64_t)blockIdx.x * kCpTile + (int64_t)warp * kCpIters * 32;
    uint64_t carry = warp_base > 0 && warp_base <= n ? keys[warp_base - 1] : 0ull;
#pragma unroll
    for (int it = 0; it < kCpIters; ++it) {
        const int64_t e = warp_base + it * 32 + lane;
        key[it] = e < n ? keys[e] : 0ull;
    }
#pragma unroll
    for (int it = 0; it < kCpIters; ++it) {
        node_flags_of(n, warp_base + it * 32, lane, ls, key[it], carry, bal[it]);
        carry = __shfl_sync(0xffffffffu, key[it], 31);
#pragma unroll
        for (int l = 0; l < kCpLevels; ++l) cnt[l] += __popc(bal[it][l]);
    }
    if (lane == 0)
        for (int l = 0; l < kCpLevels; ++l) wcnt[warp][l] = cnt[l];
    __syncthreads();
    uint32_t run[kCpLevels];
#pragma unroll
    for (int l = 0; l < kCpLevels; ++l) {
        run[l] = block_base[(int64_t)blockIdx.x * kCpLevels + l];
        for (int w = 0; w < warp; ++w) run[l] += wcnt[w][l];
    }
    constexpr int leaf = ORDER - 1;
    const unsigned below = (1u << lane) - 1u;
#pragma unroll
    for (int it = 0; it < kCpIters; ++it) {
        int64_t e = (int64_t)blockIdx.x * kCpTile + (warp * kCpIters + it) * 32 + lane;
        if (e < n) {
            uint32_t id[kMaxOrder];
#pragma unroll
            for (int l = 0; l < kCpLevels; ++l) id[l] = run[l] + __popc(bal[it][l] & below);
            id[leaf] = (uint32_t)e;
            out.crd[leaf][e] = (int32_t)((key[it] >> ls.shift[leaf]) & ((1ull << out.bits[leaf]) - 1ull));
#pragma unroll
            for (int l = 0; l < kCpLevels; ++l) {
                if (l < leaf && ((bal[it][l] >> lane) & 1u)) {
                    out.crd[l][id[l]] = (int32_t)((key[it] >> ls.shift[l]) & ((1ull << out.bits[l]) - 1ull));
                    out.pos[l + 1][id[l]] = (int32_t)id[l + 1];
                }
            }
        }
#pragma unroll
        for (int l = 0; l < kCpLevels; ++l) run[l] += __popc(bal[it][l]);
    }
}

inline void launch_csf_scatter(int order, int64_t blocks, const uint64_t *keys, int64_t n, const LevelShifts &ls,
                               const uint32_t *block_base, const CsfArrays &out, cudaStream_t stream) {
    switch (order) {
        case 1: csf_scatter<1><<<(unsigned)blocks, kCpThreads, 0, stream>>>(keys, n, ls, block_base, out); break;
        case 2: csf_scatter<2><<<(unsigned)blocks, kCpThreads, 0, stream>>>(keys, n, ls, block_base, out); break;
        case 3: csf_scatter<3><<<(unsigned)blocks, kCpThreads, 0, stream>>>(keys, n, ls, block_base, out); break;
        default: csf_scatter<4><<<(unsigned)blocks, kCpThreads, 0, stream>>>(keys, n, ls, block_base, out); break;
    }
}

struct LevelSizes { int64_t n[kMaxOrder]; int order; };

__global__ void csf_finish(CsfArrays out, LevelSizes sz) {
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        out.pos[0][0] = 0;
        out.pos[0][1] = (int32_t)sz.n[0];
        for (int l = 1; l < sz.order; ++l) out.pos[l][sz.n[l - 1]] = (int32_t)sz.n[l];
    }
}

// ------------------------------------------------------------------------------------------------
// load balancing (per-slice nonzero counts -> light / heavy / giant work lists)
// ------------------------------------------------------------------------------------------------
struct ChainPtrs { const int32_t *pos[kMaxOrder]; int order; };

// leaf offset of level-1 node f (or of the end when f = n1)
__device__ __forceinline__ int32_t leaf_of_fiber(const ChainPtrs &c, int32_t f) {
    int32_t x = f;
    for (int l = 2; l < c.order; ++l) x = c.pos[l][x];
    return x;
}

__global__ void bin_slice_ptr(ChainPtrs c, int64_t n0, int32_t *__restrict__ slice_ptr) {
    int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s > n0) return;
    slice_ptr[s] = leaf_of_fiber(c, c.pos[1][s]);
}

// Light slices are listed by falling size class (class = floor(log2(nonzeros))), so that the slices that
// share a block are about equally large and the largest start first.  kBinClasses classes; totals[8 + d] =
// first list position of class d (d = 0: largest), totals[8 + kBinClasses + d] = fill counter, cleared.
constexpr int kBinClasses = 32;
__device__ __forceinline__ int light_class(int64_t z) { return 31 - (63 - __clzll((unsigned long long)(z > 0 ? z : 1))); }

// Single-block scan over slices: per-slice work-item offset; totals in out[0..4), class bases behind them.
__global__ void __launch_bounds__(1024) bin_scan(const int32_t *__restrict__ slice_ptr, int64_t n0, int64_t light_max,
                                                 int64_t heavy_max, int64_t chunk, int32_t *__restrict__ item_off,
                                                 int32_t *__restrict__ light_idx, int32_t *__restrict__ totals) {
    __shared__ uint32_t wsum[32][2];
    __shared__ uint32_t carry[4];      // items, light, heavy, giant
    __shared__ uint32_t cls[kBinClasses];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x < 4) carry[threadIdx.x] = 0;
    if (threadIdx.x < kBinClasses) cls[threadIdx.x] = 0;
    __syncthreads();
    for (int64_t base = 0; base < n0; base += 1024) {
        int64_t s = base + threadIdx.x;
        uint32_t v[2] = {0, 0};
        uint32_t is_heavy = 0, is_giant = 0;
        if (s < n0) {
            int64_t z = (int64_t)slice_ptr[s + 1] - slice_ptr[s];
            if (z <= light_max) { v[1] = 1; atomicAdd(&cls[light_class(z)], 1u); }
            else if (z <= heavy_max) { v[0] = 1; is_heavy = 1; }
            else { v[0] = (uint32_t)((z + chunk - 1) / chunk); is_giant = 1; }
        }
        uint32_t inc[2];
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            inc[q] = v[q];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                uint32_t t = __shfl_up_sync(0xffffffffu, inc[q], off);
                if (lane >= off) inc[q] += t;
            }
            if (lane == 31) wsum[warp][q] = inc[q];
        }
        unsigned hb = __ballot_sync(0xffffffffu, is_heavy), gb = __ballot_sync(0xffffffffu, is_giant);
        __syncthreads();
        uint32_t wb[2] = {0, 0};
        for (int w = 0; w < warp; ++w) { wb[0] += wsum[w][0]; wb[1] += wsum[w][1]; }
        if (s < n0) {
            item_off[s] = (int32_t)(carry[0] + wb[0] + inc[0] - v[0]);
            light_idx[s] = (int32_t)(carry[1] + wb[1] + inc[1] - v[1]);
        }
        __syncthreads();
        if (lane == 0) { atomicAdd(&carry[2], __popc(hb)); atomicAdd(&carry[3], __popc(gb)); }
        if (threadIdx.x == 1023) { carry[0] += wb[0] + inc[0]; carry[1] += wb[1] + inc[1]; }
        __syncthreads();
    }
    if (threadIdx.x < 4) totals[threadIdx.x] = (int32_t)carry[threadIdx.x];
    if (threadIdx.x == 0) {
        uint32_t run = 0;
        for (int d = 0; d < kBinClasses; ++d) {
            totals[8 + d] = (int32_t)run;
            totals[8 + kBinClasses + d] = 0;
            run += cls[d];
        }
    }
}

__global__ void bin_fill(ChainPtrs c, const int32_t *__restrict__ slice_ptr, int64_t n0, int64_t light_max,
                         int64_t heavy_max, const int32_t *__restrict__ item_off,
                         int32_t *__restrict__ class_base, WorkItem *__restrict__ items,
                         int32_t *__restrict__ light_list) {
    int64_t s = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n0) return;
    const int64_t z = (int64_t)slice_ptr[s + 1] - slice_ptr[s];
    if (z <= light_max) {       // any order inside a class will do: slices are independent of one another
        const int d = light_class(z);
        light_list[class_base[d] + atomicAdd(&class_base[kBinClasses + d], 1)] = (int32_t)s;
    }
    else if (z <= heavy_max) items[item_off[s]] = WorkItem{(int32_t)s, c.pos[1][s], c.pos[1][s + 1], kItemBlock};
}

// One thread per block work item of the heavy/giant range: items of giant slices find their own
// level-1 node range (the slice is cut where the leaf offset passes q/parts of its nonzeros).
__global__ void bin_fill_chunks(ChainPtrs c, const int32_t *__restrict__ slice_ptr, int64_t n0, int64_t heavy_max,
                                int64_t chunk, const int32_t *__restrict__ item_off,
                                const int32_t *__restrict__ totals, WorkItem *__restrict__ items) {
    int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= totals[0]) return;                       // the grid covers the upper bound of the item count
    // slice owning item t: last s with item_off[s] <= t (slices without items share their successor's offset)
    int64_t lo = 0, hi = n0 - 1;
    while (lo < hi) {
        int64_t mid = lo + (hi - lo + 1) / 2;
        if (item_off[mid] <= t) lo = mid; else hi = mid - 1;
    }
    const int64_t s = lo;
    const int32_t p0 = slice_ptr[s], p1 = slice_ptr[s + 1];
    const int64_t z = (int64_t)p1 - p0;
    if (z <= heavy_max) return;                       // a whole-slice item, written by bin_fill
    const int64_t parts = (z + chunk - 1) / chunk, q = t - item_off[s];
    const int32_t f0 = c.pos[1][s], f1 = c.pos[1][s + 1];
    int32_t cut[2];
    for (int e = 0; e < 2; ++e) {
        const int64_t qq = q + e;
        if (qq == 0) { cut[e] = f0; continue; }
        if (qq >= parts) { cut[e] = f1; continue; }
        const int64_t target = p0 + (z * qq) / parts;
        int32_t a = f0, b = f1;
        while (a < b) {
            int32_t mid = a + (b - a) / 2;
            if ((int64_t)leaf_of_fiber(c, mid) < target) a = mid + 1; else b = mid;
        }
        cut[e] = a;
    }
    items[t] = WorkItem{(int32_t)s, cut[0], cut[1], kItemChunk};
}

__global__ void bin_light_items(WorkItem *__restrict__ items, const int32_t *__restrict__ totals) {
    const int64_t first_item = totals[0], n_light = totals[1];
    int64_t g = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    int64_t groups = (n_light + kWarpsPerBlock - 1) / kWarpsPerBlock;
    if (g >= groups) return;
    int64_t left = n_light - g * kWarpsPerBlock;
    items[first_item + g] = WorkItem{(int32_t)(g * kWarpsPerBlock),
                                     (int32_t)(left < kWarpsPerBlock ? left : kWarpsPerBlock), 0, kItemLight};
}

int bits_for(int64_t extent) {
    int b = 1;
    while (b < 63 && (1ll << b) < extent) ++b;
    return b;
}

// Stream-ordered memory comes from a pool the library owns (one per device) whose release threshold
// is unlimited, so buffers freed by one build are reused by the next without going back to the driver.
cudaMemPool_t library_pool(int device) {
    static cudaMemPool_t pools[64] = {nullptr};
    static std::mutex mu;
    if (device < 0 || device >= 64) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!pools[device]) {
        cudaMemPoolProps props;
        std::memset(&props, 0, sizeof(props));
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = device;
        cudaMemPool_t pool = nullptr;
        if (cudaMemPoolCreate(&pool, &props) != cudaSuccess) return nullptr;
        unsigned long long keep = ~0ull;
        cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
        pools[device] = pool;
    }
    return pools[device];
}

cudaError_t pool_alloc(void **p, size_t bytes, cudaStream_t stream) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    cudaMemPool_t pool = library_pool(dev);
    if (!pool) return cudaMallocAsync(p, bytes ? bytes : 16, stream);
    return cudaMallocFromPoolAsync(p, bytes ? bytes : 16, pool, stream);
}

struct Scratch {            // stream-ordered temporaries of one build
    cudaStream_t stream;
    void *ptrs[16];
    int n = 0;
    explicit Scratch(cudaStream_t s) : stream(s) {}
    cudaError_t alloc(void **p, size_t bytes) {
        cudaError_t e = pool_alloc(p, bytes, stream);
        if (e == cudaSuccess) ptrs[n++] = *p;
        return e;
    }
    void forget(void *p) {
        for (int i = 0; i < n; ++i) if (ptrs[i] == p) ptrs[i] = nullptr;
    }
    ~Scratch() {
        for (int i = 0; i < n; ++i) if (ptrs[i]) cudaFreeAsync(ptrs[i], stream);
    }
};

// Small buffers of one sort.  `zeroed` covers hist, counters, totals and the status word in one
// allocation so that a single memset clears them.
struct SortBufs {
    uint32_t *hist;                    // [kMaxPasses][kRsMaxBins] digit counts, then exclusive digit offsets
    uint32_t *counters;                // [kMaxPasses] tile tickets
    unsigned long long *tile_status;   // [ntiles][kRsMaxBins]
};

template <typename V, int BITS>
const_status_t launch_onesweep(const uint64_t *kin, uint64_t *kout, const V *vin, V *vout, int64_t n, int shift,
                               const uint32_t *digit_base, const SortBufs &b, uint32_t *counter, int32_t *status,
                               unsigned epoch, cudaStream_t stream) {
    const int64_t ntiles = (n + kRsTile - 1) / kRsTile;
    const size_t dyn = kRsTile * (sizeof(uint64_t) + sizeof(V));
    static PerDeviceOnce attr_once;                     // per template instance
    CB_CUDA(once_per_device(attr_once, [&] { return cudaFuncSetAttribute(rs_onesweep<V, BITS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn); }));
    const DebugKnobs knobs = debug_knobs();
    CB_LAUNCH("rs_onesweep", stream,
              rs_onesweep<V, BITS><<<(unsigned)ntiles, kRsThreads, dyn, stream>>>(
                  kin, kout, vin, vout, n, shift, digit_base, b.tile_status, counter, status, epoch,
                  knobs.spin_limit > 0 ? knobs.spin_limit : kSpinLimit, knobs.withhold,
                  kRsAheadTiles));
    return CONST_OK;
}

// Sorts (keys, payload) by key.  The first pass reads the payload from `vals_src` (the caller's
// array, never written); later passes alternate between vals_a and vals_b.  On return `keys` and
// `vals_sorted` name the buffers that hold the result.
template <typename V>
const_status_t sort_passes(uint64_t *&keys, uint64_t *&keys_alt, const V *vals_src, V *vals_a, V *vals_b,
                           V *&vals_sorted, int64_t n, const DigitPlan &dp, const SortBufs &b, int32_t *status,
                           cudaStream_t stream) {
    vals_sorted = vals_a;
    if (n == 0) return CONST_OK;
    if (dp.passes == 0) {
        CB_CUDA(cudaMemcpyAsync(vals_a, vals_src, sizeof(V) * n, cudaMemcpyDeviceToDevice, stream));
        return CONST_OK;
    }
    const int64_t ntiles = (n + kRsTile - 1) / kRsTile;
    CB_CUDA(cudaMemsetAsync(b.tile_status, 0, sizeof(unsigned long long) * ntiles * kRsMaxBins, stream));
    CB_LAUNCH("rs_scan_hist", stream, rs_scan_hist<<<dp.passes, 256, 0, stream>>>(b.hist));
    const V *vin = vals_src;
    V *vout = vals_a;
    for (int p = 0; p < dp.passes; ++p) {
        const_status_t s = dp.bits[p] > 8
            ? launch_onesweep<V, 9>(keys, keys_alt, vin, vout, n, dp.shift[p], b.hist + p * kRsMaxBins, b, b.counters + p,
                                    status, (unsigned)(p + 1), stream)
            : launch_onesweep<V, 8>(keys, keys_alt, vin, vout, n, dp.shift[p], b.hist + p * kRsMaxBins, b, b.counters + p,
                                    status, (unsigned)(p + 1), stream);
        if (s != CONST_OK) return s;
        std::swap(keys, keys_alt);
        vals_sorted = vout;
        vin = vout;
        vout = vout == vals_a ? vals_b : vals_a;
    }
    CB_CUDA(cudaGetLastError());
    return CONST_OK;
}

// Everything between "keys packed" and "level sizes known": sort, flag counts, block scan.
const_status_t sort_and_count(uint64_t *&keys, uint64_t *&keys_alt, const void *vals_src, void *vals_a, void *vals_b,
                              void *&vals_sorted, int64_t nnz, const DigitPlan &dp, const_dtype_t dtype,
                              const SortBufs &b, const LevelShifts &ls, uint32_t *block_counts, uint32_t *totals,
                              int32_t *status, cudaStream_t stream) {
    const_status_t s;
    if (dtype == CONST_F32) {
        uint32_t *out = nullptr;
        s = sort_passes<uint32_t>(keys, keys_alt, (const uint32_t *)vals_src, (uint32_t *)vals_a, (uint32_t *)vals_b, out,
                                  nnz, dp, b, status, stream);
        vals_sorted = out;
    } else {
        unsigned long long *out = nullptr;
        s = sort_passes<unsigned long long>(keys, keys_alt, (const unsigned long long *)vals_src,
                                            (unsigned long long *)vals_a, (unsigned long long *)vals_b, out, nnz, dp, b,
                                            status, stream);
        vals_sorted = out;
    }
    if (s != CONST_OK) return s;
    const int64_t cp_blocks = (nnz + kCpTile - 1) / kCpTile;
    CB_LAUNCH("csf_count", stream, csf_count<<<(unsigned)cp_blocks, kCpThreads, 0, stream>>>(keys, nnz, ls, block_counts, status));
    launch_csf_scan(block_counts, cp_blocks, totals, stream);
    return CONST_OK;
}

struct KeyLayout { int bits[kMaxOrder]; int shift[kMaxOrder]; int total_bits; DigitPlan digits; };

// Fewest passes with 8- or 9-bit digits: every pass is 8 bits wide unless 9-bit passes are needed to
// cover the key in that number of passes (43 bits -> 9 9 9 8 8).  A digit may reach past the top of
// the key; those bits are zero.
DigitPlan digit_plan(int total_bits) {
    DigitPlan dp;
    for (int p = 0; p < kMaxPasses; ++p) dp.shift[p] = dp.bits[p] = 0;
    const int p8 = (total_bits + 7) / 8, p9 = (total_bits + kRsMaxBits - 1) / kRsMaxBits;
    dp.passes = p9 < p8 ? p9 : p8;
    const int wide = std::max(0, total_bits - 8 * dp.passes);      // passes that must take 9 bits
    int acc = 0;
    for (int p = 0; p < dp.passes; ++p) {
        dp.bits[p] = p < wide ? kRsMaxBits : 8;
        dp.shift[p] = acc;
        acc += dp.bits[p];
    }
    return dp;
}

bool key_layout(int order, const int64_t *dims, const int *mode_order, KeyLayout &k) {
    k.total_bits = 0;
    for (int l = 0; l < kMaxOrder; ++l) k.bits[l] = k.shift[l] = 0;
    for (int l = 0; l < order; ++l) { k.bits[l] = bits_for(dims[mode_order[l]]); k.total_bits += k.bits[l]; }
    if (k.total_bits > 64) return false;
    int acc = 0;
    for (int l = order - 1; l >= 0; --l) { k.shift[l] = acc; acc += k.bits[l]; }
    k.digits = digit_plan(k.total_bits);
    return true;
}

PackArgs pack_args(int order, const int64_t *dims, const int *mode_order, const int32_t *const *coords_dev,
                   const KeyLayout &k) {
    PackArgs pa;
    pa.order = order;
    for (int l = 0; l < kMaxOrder; ++l) {
        pa.c[l] = l < order ? coords_dev[mode_order[l]] : nullptr;
        pa.dim[l] = l < order ? dims[mode_order[l]] : 0;
        pa.shift[l] = k.shift[l];
    }
    return pa;
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// host driver
// ------------------------------------------------------------------------------------------------
void csf_free(const_csf *csf) {
    if (!csf) return;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(csf->device);
    auto drop = [&](void *p) { if (p) cudaFreeAsync(p, csf->stream); };
    for (int l = 0; l < kMaxOrder; ++l) { drop(csf->pos[l]); drop(csf->crd[l]); }
    drop(csf->vals);
    drop(csf->slice_ptr);
    drop(csf->light_list);
    drop(csf->items);
    drop(csf->bin_scratch);
    csf->magic = 0;
    delete csf;
    cudaSetDevice(prev);
}

// Waits for everything queued on `stream` by polling an event instead of sleeping in the driver: the
// build needs two small results on the host (level sizes, work-list sizes) in the middle of a step that
// lasts a few milliseconds, and a blocking wait can cost a scheduler quantum when the host is busy.
cudaError_t wait_stream(cudaStream_t stream) {
    static thread_local cudaEvent_t ev[64] = {nullptr};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaStreamSynchronize(stream);
    if (!ev[dev] && cudaEventCreateWithFlags(&ev[dev], cudaEventDisableTiming) != cudaSuccess) {
        ev[dev] = nullptr;
        return cudaStreamSynchronize(stream);
    }
    e = cudaEventRecord(ev[dev], stream);
    if (e != cudaSuccess) return e;
    for (long spins = 0; spins < (1l << 26); ++spins) {
        e = cudaEventQuery(ev[dev]);
        if (e != cudaErrorNotReady) return e;
    }
    return cudaStreamSynchronize(stream);          // something takes seconds: stop burning a core
}

// Upper bound of the number of work items for the current thresholds: a light or heavy slice gives at most
// one item, a giant slice of z nonzeros ceil(z / chunk) <= z / chunk + 1.
int64_t item_capacity(const const_csf *csf) {
    return csf->n[0] + csf->nnz / std::max<int64_t>(csf->chunk, 1) + 1;
}

const_status_t csf_rebin(const_csf *csf, cudaStream_t stream) {
    const int64_t n0 = csf->n[0];
    csf->n_light = csf->n_heavy = csf->n_giant = csf->n_items = 0;
    csf->totals_on_host = n0 == 0;
    csf->bin_stream = stream;
    if (n0 == 0) { csf->item_cap = 0; return CONST_OK; }
    // Nothing below waits for the device: the lists are sized by their upper bounds, the fill kernels read
    // the counts the scan left in `totals`, and so do the fused kernels later on.
    const int64_t cap = item_capacity(csf);
    if (cap > 0x7fffffffll) return CONST_ERR_UNSUPPORTED;
    if (cap > csf->item_cap || !csf->items) {
        if (csf->items) cudaFreeAsync(csf->items, stream);
        csf->items = nullptr;
        CB_CUDA(pool_alloc((void **)&csf->items, sizeof(WorkItem) * cap, stream));
    }
    csf->item_cap = cap;
    if (!csf->light_list) CB_CUDA(pool_alloc((void **)&csf->light_list, sizeof(int32_t) * n0, stream));
    ChainPtrs c;
    c.order = csf->order;
    for (int l = 0; l < kMaxOrder; ++l) c.pos[l] = csf->pos[l];
    int32_t *item_off = csf->bin_scratch, *light_idx = csf->bin_scratch + (n0 + 1), *totals = csf->bin_scratch + 2 * (n0 + 1);
    csf->bin_totals = totals;
    CB_LAUNCH("bin_scan", stream, bin_scan<<<1, 1024, 0, stream>>>(csf->slice_ptr, n0, csf->light_max, csf->heavy_max, csf->chunk, item_off,
                                     light_idx, totals));
    CB_LAUNCH("bin_fill", stream, bin_fill<<<(unsigned)((n0 + 255) / 256), 256, 0, stream>>>(c, csf->slice_ptr, n0, csf->light_max, csf->heavy_max,
                                                              item_off, totals + 8, csf->items, csf->light_list));
    CB_LAUNCH("bin_fill_chunks", stream, bin_fill_chunks<<<(unsigned)((cap + 127) / 128), 128, 0, stream>>>(
                  c, csf->slice_ptr, n0, csf->heavy_max, csf->chunk, item_off, totals, csf->items));
    const int64_t max_groups = (n0 + kWarpsPerBlock - 1) / kWarpsPerBlock;
    CB_LAUNCH("bin_light_items", stream, bin_light_items<<<(unsigned)((max_groups + 255) / 256), 256, 0, stream>>>(csf->items, totals));
    CB_CUDA(cudaGetLastError());
    return CONST_OK;
}

// Host copies of the bin totals, for callers that ask (const_csf_bin_counts, const_csf_work_lists).
const_status_t csf_bin_totals(const_csf *csf) {
    if (csf->totals_on_host) return CONST_OK;
    int32_t h[4] = {0, 0, 0, 0};
    int prev = 0;
    CB_CUDA(cudaGetDevice(&prev));
    CB_CUDA(cudaSetDevice(csf->device));
    cudaError_t e = cudaMemcpyAsync(h, csf->bin_totals, sizeof(h), cudaMemcpyDeviceToHost, csf->bin_stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(csf->bin_stream);
    cudaSetDevice(prev);
    if (e != cudaSuccess) return CONST_ERR_CUDA;
    csf->n_light = h[1];
    csf->n_heavy = h[2];
    csf->n_giant = h[3];
    csf->n_items = h[0] + (h[1] + kWarpsPerBlock - 1) / kWarpsPerBlock;
    csf->totals_on_host = true;
    return CONST_OK;
}

const_status_t csf_build_impl(int order, const int64_t *dims, int64_t nnz, const int32_t *const *coords_dev,
                              const void *vals_dev, const_dtype_t dtype, const int *mode_order,
                              cudaStream_t stream, const_csf **out) {
    KeyLayout kl;
    if (!key_layout(order, dims, mode_order, kl)) return CONST_ERR_UNSUPPORTED;

    const_csf *csf = new (std::nothrow) const_csf();
    if (!csf) return CONST_ERR_INVALID_ARG;
    csf->order = order;
    csf->dtype = dtype;
    csf->nnz = nnz;
    csf->stream = stream;
    cudaGetDevice(&csf->device);
    for (int l = 0; l < order; ++l) { csf->dims[l] = dims[l]; csf->mode_order[l] = mode_order[l]; }
    csf->light_max = 4096;      // thresholds from sweeps over the three large benchmark tensors (with size-ordered light lists)
    csf->heavy_max = 16384;
    csf->chunk = 8192;

    const size_t vsize = dtype == CONST_F32 ? 4 : 8;
    const_status_t rc = CONST_OK;
    {
        Scratch tmp(stream);
        uint64_t *keys = nullptr, *keys_alt = nullptr;
        void *vals = nullptr, *vals_alt = nullptr, *vals_sorted = nullptr;
        unsigned char *small = nullptr;          // hist | counters | totals | status, cleared together
        uint32_t *block_counts = nullptr;
        SortBufs sb{nullptr, nullptr, nullptr};
        const int64_t cp_blocks = (nnz + kCpTile - 1) / kCpTile;
        const int64_t ntiles = (nnz + kRsTile - 1) / kRsTile;
        constexpr size_t kHistBytes = sizeof(uint32_t) * kMaxPasses * kRsMaxBins;
        constexpr size_t kSmallBytes = kHistBytes + 256;
        auto body = [&]() -> const_status_t {
            CB_CUDA(tmp.alloc((void **)&keys, sizeof(uint64_t) * nnz));
            CB_CUDA(tmp.alloc((void **)&keys_alt, sizeof(uint64_t) * nnz));
            CB_CUDA(tmp.alloc(&vals, vsize * (nnz + 4)));
            CB_CUDA(tmp.alloc(&vals_alt, vsize * (nnz + 4)));
            CB_CUDA(tmp.alloc((void **)&small, kSmallBytes));
            CB_CUDA(tmp.alloc((void **)&sb.tile_status, sizeof(unsigned long long) * std::max<int64_t>(ntiles, 1) * kRsMaxBins));
            CB_CUDA(tmp.alloc((void **)&block_counts, sizeof(uint32_t) * (kCpLevels * std::max<int64_t>(cp_blocks, 1) +
                                                                        scan_partials_room(cp_blocks))));
            CB_CUDA(cudaMemsetAsync(small, 0, kSmallBytes, stream));
            sb.hist = reinterpret_cast<uint32_t *>(small);
            sb.counters = reinterpret_cast<uint32_t *>(small + kHistBytes);
            uint32_t *totals = reinterpret_cast<uint32_t *>(small + kHistBytes + 64);
            int32_t *status = reinterpret_cast<int32_t *>(small + kHistBytes + 128);
            LevelShifts ls;
            ls.order = order;
            for (int l = 0; l < kMaxOrder; ++l) ls.shift[l] = kl.shift[l];
            if (nnz > 0) {
                PackArgs pa = pack_args(order, dims, mode_order, coords_dev, kl);
                CB_LAUNCH("pack_hist", stream, launch_pack_hist(pa, nnz, kl.digits, keys, sb.hist, status, stream));
                const_status_t s = sort_and_count(keys, keys_alt, vals_dev, vals, vals_alt, vals_sorted, nnz, kl.digits,
                                                  dtype, sb, ls, block_counts, totals, status, stream);
                if (s != CONST_OK) return s;
            }
            uint32_t h_small[32] = {0};          // totals at [0..4), status at [16]
            CB_CUDA(cudaMemcpyAsync(h_small, totals, sizeof(uint32_t) * 17, cudaMemcpyDeviceToHost, stream));
            CB_CUDA(wait_stream(stream));
            if (h_small[16] != 0) return (const_status_t)h_small[16];
            for (int l = 0; l < order - 1; ++l) csf->n[l] = h_small[l];
            csf->n[order - 1] = nnz;

            CsfArrays arr;
            for (int l = 0; l < kMaxOrder; ++l) { arr.pos[l] = arr.crd[l] = nullptr; arr.bits[l] = kl.bits[l]; }
            for (int l = 0; l < order; ++l) {
                const int64_t parents = l == 0 ? 1 : csf->n[l - 1];
                CB_CUDA(pool_alloc((void **)&csf->pos[l], sizeof(int32_t) * (parents + 1), stream));
                CB_CUDA(pool_alloc((void **)&csf->crd[l], sizeof(int32_t) * (csf->n[l] + 4), stream));
                arr.pos[l] = csf->pos[l];
                arr.crd[l] = csf->crd[l];
            }
            if (nnz > 0)
                CB_LAUNCH("csf_scatter", stream, launch_csf_scatter(order, cp_blocks, keys, nnz, ls, block_counts, arr, stream));
            LevelSizes sz;
            sz.order = order;
            for (int l = 0; l < kMaxOrder; ++l) sz.n[l] = csf->n[l];
            CB_LAUNCH("csf_finish", stream, csf_finish<<<1, 32, 0, stream>>>(arr, sz));
            if (!vals_sorted) vals_sorted = vals;
            csf->vals = vals_sorted;          // the sorted payload buffer becomes the leaf value array
            tmp.forget(vals_sorted);

            // per-slice leaf offsets and the default work lists
            const int64_t n0 = csf->n[0];
            CB_CUDA(pool_alloc((void **)&csf->slice_ptr, sizeof(int32_t) * (n0 + 1), stream));
            CB_CUDA(pool_alloc((void **)&csf->bin_scratch, sizeof(int32_t) * (2 * (n0 + 1) + 8 + 2 * kBinClasses), stream));
            ChainPtrs c;
            c.order = order;
            for (int l = 0; l < kMaxOrder; ++l) c.pos[l] = csf->pos[l];
            CB_LAUNCH("bin_slice_ptr", stream, bin_slice_ptr<<<(unsigned)((n0 + 1 + 255) / 256), 256, 0, stream>>>(c, n0, csf->slice_ptr));
            CB_CUDA(cudaGetLastError());
            return csf_rebin(csf, stream);
        };
        rc = body();
    }
    if (rc != CONST_OK) {
        csf_free(csf);
        return rc;
    }
    *out = csf;
    return CONST_OK;
}

// ------------------------------------------------------------------------------------------------
// const_csf_build_noalloc: the same COO -> CSF pipeline with every temporary in one static device
// array, for callers that must not allocate (see include/const_b200.h).
// ------------------------------------------------------------------------------------------------
namespace {

constexpr int64_t kNoAllocMaxNnz = 1 << 18;                               // 262 144 nonzeros
constexpr size_t kNaKeys = sizeof(uint64_t) * kNoAllocMaxNnz;             // one key buffer / one fp64 payload buffer
constexpr size_t kNaTiles = (kNoAllocMaxNnz + kRsTile - 1) / kRsTile;
constexpr size_t kNaCpBlocks = (kNoAllocMaxNnz + kCpTile - 1) / kCpTile;
// byte offsets inside the static array (every region 256-byte aligned)
constexpr size_t kNaOffKeys0 = 0;
constexpr size_t kNaOffKeys1 = kNaOffKeys0 + kNaKeys;
constexpr size_t kNaOffVals = kNaOffKeys1 + kNaKeys;                      // second payload buffer (the first is the caller's output)
constexpr size_t kNaOffTileStatus = kNaOffVals + kNaKeys;
constexpr size_t kNaOffHist = kNaOffTileStatus + sizeof(unsigned long long) * kNaTiles * kRsMaxBins;
constexpr size_t kNaHistBytes = sizeof(uint32_t) * kMaxPasses * kRsMaxBins;
constexpr size_t kNaOffSmall = kNaOffHist + kNaHistBytes;                 // pass counters, level totals, status word
constexpr size_t kNaSmallBytes = 256;
constexpr size_t kNaOffBlockCounts = kNaOffSmall + kNaSmallBytes;
constexpr size_t kNaBytes = kNaOffBlockCounts + ((sizeof(uint32_t) * kCpLevels * (kNaCpBlocks + 2) + 255) / 256) * 256;

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is not
// a device address and must never be handed to a kernel or to cudaMemset as if it were one.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNaBytes];

constexpr int kNaMaxDevices = 64;
unsigned char *g_noalloc_ptr[kNaMaxDevices] = {nullptr};                  // device address of the array, per device

const_status_t noalloc_scratch(unsigned char **out) {
    int dev = 0;
    CB_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kNaMaxDevices) return CONST_ERR_UNSUPPORTED;
    static std::mutex mu;                                                     // two host threads may arrive first together
    std::lock_guard<std::mutex> lock(mu);
    if (!g_noalloc_ptr[dev]) {
        void *p = nullptr;
        CB_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));                 // resolved with `dev` current
        g_noalloc_ptr[dev] = static_cast<unsigned char *>(p);
    }
    *out = g_noalloc_ptr[dev];
    return CONST_OK;
}

}  // namespace

const_status_t csf_build_noalloc_impl(int order, const int64_t *dims, int64_t nnz, const int32_t *const *coords_dev,
                                      const void *vals_dev, const_dtype_t dtype, const int *mode_order,
                                      cudaStream_t stream, int32_t *const *pos_out, int32_t *const *crd_out,
                                      void *vals_out, int64_t *level_sizes) {
    if (nnz > kNoAllocMaxNnz) return CONST_ERR_WORKSPACE;
    KeyLayout kl;
    if (!key_layout(order, dims, mode_order, kl)) return CONST_ERR_UNSUPPORTED;

    unsigned char *base = nullptr;
    const_status_t rc = noalloc_scratch(&base);
    if (rc != CONST_OK) return rc;
    uint64_t *keys = reinterpret_cast<uint64_t *>(base + kNaOffKeys0);
    uint64_t *keys_alt = reinterpret_cast<uint64_t *>(base + kNaOffKeys1);
    uint32_t *block_counts = reinterpret_cast<uint32_t *>(base + kNaOffBlockCounts);
    SortBufs sb{reinterpret_cast<uint32_t *>(base + kNaOffHist), reinterpret_cast<uint32_t *>(base + kNaOffSmall),
                reinterpret_cast<unsigned long long *>(base + kNaOffTileStatus)};
    uint32_t *totals = reinterpret_cast<uint32_t *>(base + kNaOffSmall + 64);
    int32_t *status = reinterpret_cast<int32_t *>(base + kNaOffSmall + 128);
    // everything that must start at zero: digit histograms, pass counters, level totals, status word
    // (the tile states are cleared by the sort itself)
    CB_CUDA(cudaMemsetAsync(base + kNaOffHist, 0, kNaHistBytes + kNaSmallBytes, stream));

    const size_t vsize = dtype == CONST_F32 ? 4 : 8;
    const int64_t cp_blocks = (nnz + kCpTile - 1) / kCpTile;
    LevelShifts ls;
    ls.order = order;
    for (int l = 0; l < kMaxOrder; ++l) ls.shift[l] = kl.shift[l];
    if (nnz > 0) {
        PackArgs pa = pack_args(order, dims, mode_order, coords_dev, kl);
        launch_pack_hist(pa, nnz, kl.digits, keys, sb.hist, status, stream);
        // the payload alternates between the caller's output and the static buffer; start on the side
        // that makes the last pass land in the caller's output
        const bool odd = kl.digits.passes % 2 == 1 || kl.digits.passes == 0;
        void *first = odd ? vals_out : (void *)(base + kNaOffVals);
        void *second = odd ? (void *)(base + kNaOffVals) : vals_out;
        void *sorted = nullptr;
        rc = sort_and_count(keys, keys_alt, vals_dev, first, second, sorted, nnz, kl.digits, dtype, sb, ls, block_counts,
                            totals, status, stream);
        if (rc != CONST_OK) return rc;
    }
    uint32_t h_small[32] = {0};                   // totals at [0..4), status at [16]
    CB_CUDA(cudaMemcpyAsync(h_small, totals, sizeof(uint32_t) * 17, cudaMemcpyDeviceToHost, stream));
    CB_CUDA(cudaStreamSynchronize(stream));
    if (h_small[16] != 0) return (const_status_t)h_small[16];
    LevelSizes sz;
    sz.order = order;
    for (int l = 0; l < kMaxOrder; ++l) sz.n[l] = 0;
    for (int l = 0; l < order - 1; ++l) sz.n[l] = h_small[l];
    sz.n[order - 1] = nnz;
    CsfArrays arr;
    for (int l = 0; l < kMaxOrder; ++l) {
        arr.pos[l] = l < order ? pos_out[l] : nullptr;
        arr.crd[l] = l < order ? crd_out[l] : nullptr;
        arr.bits[l] = kl.bits[l];
    }
    if (nnz > 0) launch_csf_scatter(order, cp_blocks, keys, nnz, ls, block_counts, arr, stream);
    csf_finish<<<1, 32, 0, stream>>>(arr, sz);
    CB_CUDA(cudaGetLastError());
    if (level_sizes)
        for (int l = 0; l < order; ++l) level_sizes[l] = sz.n[l];
    return CONST_OK;
}

// ------------------------------------------------------------------------------------------------
// const_csf_from_dense: a dense result as a CSF tensor (the entries that are not zero become its
// nonzeros; Sec. 2.1 defines nz(R) that way), so that the result of one network can be a sparse
// operand of the next, e.g. E of Sec. 5.1 Eq. 1 feeding the 4-index contraction of Eq. 3.
// ------------------------------------------------------------------------------------------------
namespace {

struct DenseShape { int64_t dim[kMaxOrder]; int order; };

template <typename T>
__global__ void __launch_bounds__(256) dense_count(const T *__restrict__ a, int64_t n, unsigned long long *total) {
    unsigned long long mine = 0;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += stride) mine += a[e] != T(0);
    mine = __reduce_add_sync(0xffffffffu, (unsigned)mine);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(total, mine);
}

// every stored entry gets the next free slot (one atomic per warp and step); the order is arbitrary, the sort
// of the CSF build establishes the final one
template <typename T>
__global__ void __launch_bounds__(256) dense_fill(const T *__restrict__ a, int64_t n, DenseShape sh, int32_t *c0,
                                                  int32_t *c1, int32_t *c2, int32_t *c3, T *__restrict__ vals,
                                                  unsigned long long *cursor, unsigned long long capacity) {
    const int lane = threadIdx.x & 31;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    const int64_t rounds = (n + stride - 1) / stride;
    for (int64_t r = 0; r < rounds; ++r) {
        const int64_t e = r * stride + (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
        const bool keep = e < n && a[e] != T(0);
        const unsigned m = __ballot_sync(0xffffffffu, keep);
        if (!m) continue;
        unsigned long long base = 0;
        if (lane == __ffs(m) - 1) base = atomicAdd(cursor, (unsigned long long)__popc(m));
        base = __shfl_sync(0xffffffffu, base, __ffs(m) - 1);
        if (!keep) continue;
        const unsigned long long at = base + __popc(m & ((1u << lane) - 1u));
        if (at >= capacity) continue;                     // cannot happen: the count pass saw the same array
        int64_t rest = e;
        int32_t c[kMaxOrder] = {0, 0, 0, 0};
        for (int d = sh.order - 1; d >= 0; --d) { c[d] = (int32_t)(rest % sh.dim[d]); rest /= sh.dim[d]; }
        c0[at] = c[0];
        c1[at] = c[1];
        if (sh.order > 2) c2[at] = c[2];
        if (sh.order > 3) c3[at] = c[3];
        vals[at] = a[e];
    }
}

}  // namespace

const_status_t csf_from_dense_impl(int order, const int64_t *dims, const void *dense, const_dtype_t dtype,
                                   const int *mode_order, cudaStream_t stream, const_csf **out) {
    int64_t n = 1;
    DenseShape sh;
    sh.order = order;
    for (int d = 0; d < kMaxOrder; ++d) sh.dim[d] = 1;
    for (int d = 0; d < order; ++d) {
        sh.dim[d] = dims[d];
        if (n > (1ll << 40) / dims[d]) return CONST_ERR_UNSUPPORTED;
        n *= dims[d];
    }
    Scratch tmp(stream);
    unsigned long long *counters = nullptr;
    CB_CUDA(tmp.alloc((void **)&counters, 64));
    CB_CUDA(cudaMemsetAsync(counters, 0, 64, stream));
    const int blocks = (int)std::min<int64_t>((n + 255) / 256, 148 * 8);
    if (dtype == CONST_F32) dense_count<float><<<blocks, 256, 0, stream>>>((const float *)dense, n, counters);
    else dense_count<double><<<blocks, 256, 0, stream>>>((const double *)dense, n, counters);
    unsigned long long h_nnz = 0;
    CB_CUDA(cudaMemcpyAsync(&h_nnz, counters, sizeof(h_nnz), cudaMemcpyDeviceToHost, stream));
    CB_CUDA(wait_stream(stream));
    if (h_nnz >= 2147483647ull) return CONST_ERR_UNSUPPORTED;
    const int64_t nnz = (int64_t)h_nnz;
    int32_t *c[kMaxOrder] = {nullptr, nullptr, nullptr, nullptr};
    void *vals = nullptr;
    for (int d = 0; d < order; ++d) CB_CUDA(tmp.alloc((void **)&c[d], sizeof(int32_t) * std::max<int64_t>(nnz, 1)));
    CB_CUDA(tmp.alloc(&vals, (dtype == CONST_F32 ? 4 : 8) * std::max<int64_t>(nnz, 1)));
    if (nnz > 0) {
        if (dtype == CONST_F32)
            dense_fill<float><<<blocks, 256, 0, stream>>>((const float *)dense, n, sh, c[0], c[1], c[2], c[3], (float *)vals,
                                                          counters + 1, h_nnz);
        else
            dense_fill<double><<<blocks, 256, 0, stream>>>((const double *)dense, n, sh, c[0], c[1], c[2], c[3],
                                                           (double *)vals, counters + 1, h_nnz);
        CB_CUDA(cudaGetLastError());
    }
    return csf_build_impl(order, dims, nnz, c, vals, dtype, mode_order, stream, out);
}

}  // namespace cb
