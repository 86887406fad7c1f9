// Stand-alone microbenchmark: ceiling of random factor-row gathers (the access pattern of the fused
// kernels' producer) on this GPU.  Rows of R floats are read by R/4 neighbouring lanes with one 128-bit
// load each, row indices come from a 77 M entry stream over a 29 000 row table (the size of the
// level-2 factor of the large TTMc configuration), either uniform or Zipf(0.9) over a random
// permutation.  Not part of the library; build: nvcc -gencode arch=compute_100a,code=sm_100a -O3
// -o bench_row_gather bench_row_gather.cu ; run: ./bench_row_gather 1 (Zipf) or 0 (uniform).
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdlib>
#include <vector>
#include <cmath>
// rows of R floats gathered by R/4 lanes with float4 loads; idx[] random (zipf-ish or uniform)
template <int R, int UNR>
__global__ void gather(const int* __restrict__ idx, const float* __restrict__ tab, long n, float* out) {
    constexpr int LPR = R / 4, G = 32 / LPR;
    int lane = threadIdx.x & 31, g = lane / LPR, q = lane % LPR;
    long warp = (blockIdx.x * (long)blockDim.x + threadIdx.x) >> 5;
    long nwarps = ((long)gridDim.x * blockDim.x) >> 5;
    long per = (n + nwarps - 1) / nwarps;
    long a = warp * per, b = a + per < n ? a + per : n;
    float4 t = make_float4(0, 0, 0, 0);
    for (long p = a + g * UNR; p + UNR <= b; p += G * UNR) {
        int k[UNR]; float4 v[UNR];
#pragma unroll
        for (int u = 0; u < UNR; ++u) k[u] = __ldg(idx + p + u);
#pragma unroll
        for (int u = 0; u < UNR; ++u) v[u] = __ldg((const float4*)(tab + (size_t)k[u] * R + 4 * q));
#pragma unroll
        for (int u = 0; u < UNR; ++u) { t.x += v[u].x; t.y += v[u].y; t.z += v[u].z; t.w += v[u].w; }
    }
    if (t.x + t.y + t.z + t.w == 1.2345f) out[0] = t.x;
}
template <int R, int UNR>
void run(const int* idx, const float* tab, long n, float* out, int blocks, int threads, const char* name) {
    cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
    for (int i = 0; i < 3; ++i) gather<R, UNR><<<blocks, threads>>>(idx, tab, n, out);
    cudaEventRecord(e0);
    for (int i = 0; i < 10; ++i) gather<R, UNR><<<blocks, threads>>>(idx, tab, n, out);
    cudaEventRecord(e1); cudaEventSynchronize(e1);
    float ms; cudaEventElapsedTime(&ms, e0, e1); ms /= 10;
    printf("%s R=%d unr=%d blocks=%d thr=%d: %.3f ms  %.1f Grows/s  %.2f TB/s (row bytes)\n", name, R, UNR, blocks, threads, ms, n / ms / 1e6, n * (double)R * 4 / ms / 1e9);
}
int main(int argc, char** argv) {
    long n = 77000000; int rows = 29000;
    std::vector<int> h(n);
    bool zipf = argc > 1 && atoi(argv[1]) == 1;
    // zipf(0.9) over a random permutation, or uniform
    std::vector<double> cdf(rows); double s = 0; for (int r = 0; r < rows; ++r) { s += pow(r + 1.0, -0.9); cdf[r] = s; }
    std::vector<int> perm(rows); for (int r = 0; r < rows; ++r) perm[r] = r;
    srand(1); for (int r = rows - 1; r > 0; --r) { int j = rand() % (r + 1); std::swap(perm[r], perm[j]); }
    for (long i = 0; i < n; ++i) {
        if (zipf) { double u = (rand() / (RAND_MAX + 1.0)) * s; int lo = 0, hi = rows - 1; while (lo < hi) { int m = (lo + hi) / 2; if (cdf[m] < u) lo = m + 1; else hi = m; } h[i] = perm[lo]; }
        else h[i] = rand() % rows;
    }
    int* idx; float *tab, *out;
    cudaMalloc(&idx, n * 4); cudaMalloc(&tab, (size_t)rows * 32 * 4); cudaMalloc(&out, 4);
    cudaMemcpy(idx, h.data(), n * 4, cudaMemcpyHostToDevice); cudaMemset(tab, 0, (size_t)rows * 32 * 4);
    const char* nm = zipf ? "zipf0.9" : "uniform";
    run<16, 4>(idx, tab, n, out, 148 * 8, 256, nm);
    run<16, 8>(idx, tab, n, out, 148 * 8, 256, nm);
    run<16, 4>(idx, tab, n, out, 148 * 16, 256, nm);
    run<16, 8>(idx, tab, n, out, 148 * 4, 512, nm);
    run<32, 4>(idx, tab, n, out, 148 * 8, 256, nm);
    run<8, 4>(idx, tab, n, out, 148 * 8, 256, nm);
    return 0;
}
