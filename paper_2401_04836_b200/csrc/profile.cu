// Optional per-kernel timing with CUDA events, recorded on the stream the kernel is launched on.
// Off by default; when on, every kernel launch of the library is bracketed by two events and the
// elapsed times are summed per kernel name.  Used by the benchmark to report launch counts and
// durations measured inside the timed region.
#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "common.cuh"

namespace cb {
namespace {

struct Span { const char *name; cudaEvent_t a, b; };

std::mutex g_mu;
bool g_on = false;
std::vector<Span> g_spans;
std::vector<cudaEvent_t> g_pool;

cudaEvent_t get_event() {
    if (!g_pool.empty()) { cudaEvent_t e = g_pool.back(); g_pool.pop_back(); return e; }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

}  // namespace

ProfScope::ProfScope(const char *name, cudaStream_t stream) : stream_(stream), idx_(-1) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_on) return;
    Span s{name, get_event(), get_event()};
    if (!s.a || !s.b) return;
    cudaEventRecord(s.a, stream);
    g_spans.push_back(s);
    idx_ = (long)g_spans.size() - 1;
}

ProfScope::~ProfScope() {
    if (idx_ < 0) return;
    std::lock_guard<std::mutex> lock(g_mu);
    if (idx_ < (long)g_spans.size()) cudaEventRecord(g_spans[idx_].b, stream_);
}

}  // namespace cb

using namespace cb;

extern "C" {

const_status_t const_profile_enable(int on) {
    std::lock_guard<std::mutex> lock(g_mu);
    g_on = on != 0;
    for (Span &s : g_spans) { g_pool.push_back(s.a); g_pool.push_back(s.b); }
    g_spans.clear();
    // events are created here, not at the first launches that need them: creating one can take a
    // millisecond on some hosts, which would land inside the region that is being timed
    constexpr size_t kPrepared = 4096;
    while (g_on && g_pool.size() < kPrepared) {
        cudaEvent_t e = nullptr;
        if (cudaEventCreate(&e) != cudaSuccess || !e) break;
        g_pool.push_back(e);
    }
    return CONST_OK;
}

const_status_t const_profile_read(char *names, int64_t names_bytes, int64_t *launches, double *total_ms,
                                  int max_kernels, int *n_kernels) {
    if (!n_kernels || max_kernels < 0) return CONST_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_mu);
    std::vector<std::string> order;
    std::map<std::string, std::pair<int64_t, double>> acc;
    for (Span &s : g_spans) {
        if (cudaEventSynchronize(s.b) != cudaSuccess) return CONST_ERR_CUDA;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, s.a, s.b) != cudaSuccess) return CONST_ERR_CUDA;
        if (!acc.count(s.name)) order.push_back(s.name);
        acc[s.name].first += 1;
        acc[s.name].second += ms;
    }
    *n_kernels = (int)order.size();
    std::string joined;
    for (int k = 0; k < (int)order.size() && k < max_kernels; ++k) {
        if (launches) launches[k] = acc[order[k]].first;
        if (total_ms) total_ms[k] = acc[order[k]].second;
        joined += order[k];
        joined += '\n';
    }
    if (names && names_bytes > 0) {
        size_t n = joined.size() < (size_t)names_bytes - 1 ? joined.size() : (size_t)names_bytes - 1;
        std::memcpy(names, joined.data(), n);
        names[n] = 0;
    }
    return CONST_OK;
}

}  // extern "C"
