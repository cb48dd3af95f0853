// Launch accounting: a process-wide count of kernel launches per kind (always on) and, when enabled,
// CUDA-event timing of every launch on the stream it is issued on.  Host code only.
#include "kernels.h"

#include <atomic>
#include <cstdio>
#include <mutex>
#include <vector>

namespace tasc {
namespace {

const char* const KIND_NAMES[K_COUNT] = {
    "draft", "rows", "embed_norm", "gemm", "gemm_lm_head_argmax", "qkv_rope_append", "attention_split",
    "attention_combine", "residual_norm", "silu_mul", "accept", "other"};

std::atomic<unsigned long long> g_launches[K_COUNT];
std::atomic<int> g_enabled{0};
std::mutex g_mu;
struct Span { int kind; cudaEvent_t a, b; };
std::vector<Span> g_spans;
std::vector<cudaEvent_t> g_free;
thread_local cudaEvent_t t_open[K_COUNT];

cudaEvent_t get_event() {
    std::lock_guard<std::mutex> lk(g_mu);
    if (!g_free.empty()) {
        cudaEvent_t e = g_free.back();
        g_free.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) { (void)cudaGetLastError(); return nullptr; }
    return e;
}

char g_last_error[512] = "";

}  // namespace

void note_cuda_error(cudaError_t e, const char* expr, const char* file, int line) {
    std::lock_guard<std::mutex> lk(g_mu);
    const char* base = file;
    for (const char* c = file; *c; ++c)
        if (*c == '/') base = c + 1;
    snprintf(g_last_error, sizeof(g_last_error), "%s (%s) at %s:%d in `%s`", cudaGetErrorName(e), cudaGetErrorString(e), base, line, expr);
}

bool profiling_enabled() { return g_enabled.load(std::memory_order_relaxed) != 0; }

void prof_begin(int kind, cudaStream_t s) {
    g_launches[kind].fetch_add(1, std::memory_order_relaxed);
    t_open[kind] = nullptr;
    if (!g_enabled.load(std::memory_order_relaxed)) return;
    cudaEvent_t e = get_event();
    if (e && cudaEventRecord(e, s) == cudaSuccess) t_open[kind] = e;
}

void prof_end(int kind, cudaStream_t s) {
    cudaEvent_t a = t_open[kind];
    if (!a) return;
    t_open[kind] = nullptr;
    cudaEvent_t b = get_event();
    if (b && cudaEventRecord(b, s) == cudaSuccess) {
        std::lock_guard<std::mutex> lk(g_mu);
        g_spans.push_back(Span{kind, a, b});
    }
}

}  // namespace tasc

using namespace tasc;

extern "C" int32_t tasc_profile_kinds(void) { return K_COUNT; }
extern "C" const char* tasc_profile_kind_name(int32_t kind) { return kind >= 0 && kind < K_COUNT ? KIND_NAMES[kind] : ""; }

extern "C" tasc_status tasc_profile_enable(int32_t on) {
    g_enabled.store(on ? 1 : 0);
    return TASC_OK;
}

extern "C" tasc_status tasc_profile_read(double* ms_by_kind, int64_t* timed_launches_by_kind, int32_t n) {
    if (!ms_by_kind || !timed_launches_by_kind || n < K_COUNT) return TASC_EINVAL;
    for (int i = 0; i < n; ++i) { ms_by_kind[i] = 0.0; timed_launches_by_kind[i] = 0; }
    TASC_CUDA_TRY(cudaDeviceSynchronize());
    std::lock_guard<std::mutex> lk(g_mu);
    for (const Span& sp : g_spans) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, sp.a, sp.b) == cudaSuccess) {
            ms_by_kind[sp.kind] += ms;
            timed_launches_by_kind[sp.kind] += 1;
        } else {
            (void)cudaGetLastError();
        }
        g_free.push_back(sp.a);
        g_free.push_back(sp.b);
    }
    g_spans.clear();
    return TASC_OK;
}

extern "C" const char* tasc_last_error(void) { return g_last_error; }

extern "C" tasc_status tasc_launch_counts(int64_t* launches_by_kind, int32_t n) {
    if (!launches_by_kind || n < K_COUNT) return TASC_EINVAL;
    for (int i = 0; i < K_COUNT; ++i) launches_by_kind[i] = (int64_t)g_launches[i].load();
    return TASC_OK;
}
