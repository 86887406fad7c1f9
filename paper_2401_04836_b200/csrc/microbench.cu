// Micro-benchmarks of the machine limits that the fused kernels are rated against (const_microbench):
// register-only FMA throughput in fp32 and fp64, tf32 throughput of the tensor pipe (tcgen05, operands in
// shared memory, accumulator in tensor memory), and the rate at which random factor rows can be gathered
// with 128-bit loads (the access pattern of the leaf-level producer).  Each is timed with CUDA events on
// the caller's stream in the same process, and therefore at the same clocks, as the kernels it is compared with.
#include <algorithm>

#include "common.cuh"
#include "umma.cuh"

namespace cb {
namespace {

constexpr int kFmaThreads = 256;
constexpr int kFmaChains = 8;          // independent dependency chains per thread
constexpr int kFmaIters = 4096;        // multiply-adds per chain

template <typename T>
__global__ void __launch_bounds__(kFmaThreads) fma_peak_kernel(T a, T b, T *sink) {
    T x[kFmaChains];
#pragma unroll
    for (int c = 0; c < kFmaChains; ++c) x[c] = a + (T)(threadIdx.x + c);
    for (int it = 0; it < kFmaIters; it += 8) {
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
            for (int c = 0; c < kFmaChains; ++c) x[c] = x[c] * a + b;     // contracted to one fused multiply-add
    }
    T s = 0;
#pragma unroll
    for (int c = 0; c < kFmaChains; ++c) s += x[c];
    if (s == (T)123456789) sink[0] = s;                                   // keeps the chains alive; practically never true
}

// ---- fp64 tensor path: mma.sync m8n8k4 (the only fp64 matrix instruction; tcgen05 has no fp64 kind) ----
constexpr int kDmmaIters = 4096, kDmmaChains = 4;
__global__ void __launch_bounds__(kFmaThreads) dmma_peak_kernel(double a, double b, double *sink) {
    double c[kDmmaChains][2];
#pragma unroll
    for (int k = 0; k < kDmmaChains; ++k) c[k][0] = c[k][1] = a * (double)(threadIdx.x + k);
    for (int it = 0; it < kDmmaIters; ++it) {
#pragma unroll
        for (int k = 0; k < kDmmaChains; ++k)
            asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
                         : "+d"(c[k][0]), "+d"(c[k][1]) : "d"(a), "d"(b));
    }
    double s = 0;
#pragma unroll
    for (int k = 0; k < kDmmaChains; ++k) s += c[k][0] + c[k][1];
    if (s == 123456789.0) sink[0] = s;
}

// ---- tf32 tensor pipe: M = 128, N = 256, K = 8 per instruction, the largest single-CTA shape ----
constexpr int kMmaM = 128, kMmaN = 256;
constexpr int kMmaPerBlock = 4096;
constexpr int kMmaABytes = 2 * kMmaM * 16;       // two K quads of 128 rows x 16 bytes
constexpr int kMmaBBytes = 2 * kMmaN * 16;
constexpr uint32_t kMmaIdesc = umma::idesc_tf32(kMmaM, kMmaN);

__global__ void __launch_bounds__(128) mma_peak_kernel(int32_t *status, int polls) {
    using namespace umma;
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t mbar_s;
    __shared__ uint32_t tmem_base_s;
    float *ops = reinterpret_cast<float *>(smem);
    for (int e = threadIdx.x; e < (kMmaABytes + kMmaBBytes) / 4; e += blockDim.x)
        ops[e] = tf32_rn(1.0f + (float)((e * 37) & 255) * (1.0f / 256.0f));
    const uint32_t mbar = smem_u32(&mbar_s);
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" :: "r"(mbar) : "memory");
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&tmem_base_s)), "r"(kMmaN) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t d_tmem = tmem_base_s;
    bool done = true;
    if (threadIdx.x == 0) {
        const uint32_t a_s = smem_u32(smem), b_s = a_s + kMmaABytes;
        const uint64_t a_desc = smem_desc(a_s, kMmaM * 16, 128), b_desc = smem_desc(b_s, kMmaN * 16, 128);
        for (int it = 0; it < kMmaPerBlock; ++it) umma_tf32(d_tmem, a_desc, b_desc, kMmaIdesc, it == 0 ? 0u : 1u);
        umma_commit(mbar);
        done = mbar_wait(mbar, 0, polls);
        if (!done) atomicExch(status, (int32_t)CONST_ERR_TIMEOUT);
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(d_tmem), "r"(kMmaN) : "memory");
}

// ---- random row gather: rows of R floats read by R / 4 neighbouring lanes, UNR rows in flight per lane ----
template <int R, int UNR>
__global__ void __launch_bounds__(256) gather_peak_kernel(const int32_t *__restrict__ rows, const float *__restrict__ table,
                                                          int64_t n, int64_t table_rows, float *sink) {
    constexpr int LPR = R / 4, G = 32 / LPR;
    const int lane = threadIdx.x & 31, g = lane / LPR, q = lane % LPR;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t per = (n + nwarps - 1) / nwarps;
    const int64_t a = warp * per, b = a + per < n ? a + per : n;
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int64_t p = a + g * UNR; p + UNR <= b; p += G * UNR) {
        int32_t k[UNR];
        float4 v[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) {
            k[u] = __ldg(rows + p + u);
            k[u] = k[u] >= 0 && k[u] < table_rows ? k[u] : 0;             // never leave the table, whatever the caller passed
        }
#pragma unroll
        for (int u = 0; u < UNR; ++u) v[u] = __ldg(reinterpret_cast<const float4 *>(table + (size_t)k[u] * R + 4 * q));
#pragma unroll
        for (int u = 0; u < UNR; ++u) { t.x += v[u].x; t.y += v[u].y; t.z += v[u].z; t.w += v[u].w; }
    }
    if (t.x + t.y + t.z + t.w == 1.2345f) sink[0] = t.x;
}

struct Timer {
    cudaEvent_t a = nullptr, b = nullptr;
    ~Timer() { if (a) cudaEventDestroy(a); if (b) cudaEventDestroy(b); }
};

}  // namespace
}  // namespace cb

using namespace cb;

extern "C" const_status_t const_microbench(int kind, const int32_t *rows_dev, int64_t n, int64_t table_rows, int rank,
                                           int repeats, void *stream_v, double *ms_per_launch, double *work_per_launch) {
    if (!ms_per_launch || !work_per_launch || repeats < 1 || repeats > 1000 || kind < CONST_BENCH_FP32_FMA ||
        kind > CONST_BENCH_FP64_MMA)
        return CONST_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    int dev = 0, sms = 0;
    CB_CUDA(cudaGetDevice(&dev));
    CB_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    Timer t;
    CB_CUDA(cudaEventCreate(&t.a));
    CB_CUDA(cudaEventCreate(&t.b));
    float *scratch = nullptr;              // sink / status word, and the gather table behind it
    size_t scratch_bytes = 256;
    if (kind == CONST_BENCH_ROW_GATHER) {
        if (!rows_dev || n < 1 || table_rows < 1 || (rank != 8 && rank != 16 && rank != 32)) return CONST_ERR_INVALID_ARG;
        scratch_bytes += sizeof(float) * (size_t)table_rows * rank;
    }
    CB_CUDA(cudaMallocAsync((void **)&scratch, scratch_bytes, stream));
    cudaError_t e = cudaMemsetAsync(scratch, 0, scratch_bytes, stream);
    double work = 0.0;
    auto launch = [&]() {
        switch (kind) {
            case CONST_BENCH_FP32_FMA:
                fma_peak_kernel<float><<<sms * 8, kFmaThreads, 0, stream>>>(1.0000001f, 1e-9f, scratch);
                work = 2.0 * kFmaChains * kFmaIters * kFmaThreads * (double)(sms * 8);
                break;
            case CONST_BENCH_FP64_FMA:
                fma_peak_kernel<double><<<sms * 8, kFmaThreads, 0, stream>>>(1.0000001, 1e-9, reinterpret_cast<double *>(scratch));
                work = 2.0 * kFmaChains * kFmaIters * kFmaThreads * (double)(sms * 8);
                break;
            case CONST_BENCH_FP64_MMA:
                dmma_peak_kernel<<<sms * 8, kFmaThreads, 0, stream>>>(1.0000001, 1e-9, reinterpret_cast<double *>(scratch));
                work = 2.0 * 8 * 8 * 4 * kDmmaChains * (double)kDmmaIters * (kFmaThreads / 32) * (double)(sms * 8);
                break;
            case CONST_BENCH_TF32_MMA:
                mma_peak_kernel<<<sms, 128, kMmaABytes + kMmaBBytes, stream>>>(reinterpret_cast<int32_t *>(scratch), umma::kMbarPolls);
                work = 2.0 * kMmaM * kMmaN * 8 * (double)kMmaPerBlock * sms;
                break;
            case CONST_BENCH_ROW_GATHER: {
                const float *table = scratch + 64;
                if (rank == 8) gather_peak_kernel<8, 4><<<sms * 8, 256, 0, stream>>>(rows_dev, table, n, table_rows, scratch);
                else if (rank == 16) gather_peak_kernel<16, 4><<<sms * 8, 256, 0, stream>>>(rows_dev, table, n, table_rows, scratch);
                else gather_peak_kernel<32, 4><<<sms * 8, 256, 0, stream>>>(rows_dev, table, n, table_rows, scratch);
                work = (double)n * rank * sizeof(float);
            }
        }
    };
    if (e == cudaSuccess) {
        launch();                                                        // warm-up
        e = cudaEventRecord(t.a, stream);
        for (int r = 0; r < repeats && e == cudaSuccess; ++r) launch();
        if (e == cudaSuccess) e = cudaEventRecord(t.b, stream);
        if (e == cudaSuccess) e = cudaGetLastError();
    }
    int32_t status = 0;
    if (e == cudaSuccess && kind == CONST_BENCH_TF32_MMA)
        e = cudaMemcpyAsync(&status, scratch, sizeof(status), cudaMemcpyDeviceToHost, stream);
    cudaFreeAsync(scratch, stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(stream);
    float ms = 0.f;
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, t.a, t.b);
    if (e != cudaSuccess) return CONST_ERR_CUDA;
    if (status != 0) return (const_status_t)status;
    *ms_per_launch = ms / repeats;
    *work_per_launch = work;
    return CONST_OK;
}
