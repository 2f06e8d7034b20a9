// Optional per-kernel-kind device timing with CUDA events (see benes.h).
#include "common.cuh"

#include <mutex>
#include <vector>

namespace benes {
namespace {

struct Span {
    int kind;
    cudaEvent_t start, stop;
    unsigned long long launches;
    int dev;                        // the device the events were created on
};

bool g_enabled = false;
std::vector<Span> g_spans;          // spans recorded since the last reset
std::vector<cudaEvent_t> g_pool[kMaxDevices];    // events free for reuse, per device (an event belongs to one)
std::mutex g_pmu;

cudaEvent_t take_event(int dev) {
    std::vector<cudaEvent_t> &pool = g_pool[dev];
    if (!pool.empty()) {
        cudaEvent_t e = pool.back();
        pool.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    return e;
}

const char *kNames[BENES_PROFILE_KINDS] = {"inverse", "full_label", "split", "fused", "apply", "walk",
                                           "combine", "list_walk", "list_label", "list_resolve",
                                           "colour", "apply_fused"};

}  // namespace

ProfileScope::ProfileScope(int kind, cudaStream_t s) : kind_(kind), s_(s), slot_(-1), launches0_(g_launches) {
    if (!g_enabled) return;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return; }
    std::lock_guard<std::mutex> lk(g_pmu);
    Span sp{kind, take_event(dev), take_event(dev), 0, dev};
    if (!sp.start || !sp.stop) return;
    if (cudaEventRecord(sp.start, s) != cudaSuccess) { cudaGetLastError(); return; }
    g_spans.push_back(sp);
    slot_ = int(g_spans.size()) - 1;
}

ProfileScope::~ProfileScope() {
    if (slot_ < 0) return;
    std::lock_guard<std::mutex> lk(g_pmu);
    if (slot_ >= int(g_spans.size())) return;
    if (cudaEventRecord(g_spans[slot_].stop, s_) != cudaSuccess) cudaGetLastError();
    g_spans[slot_].launches = g_launches - launches0_;
}

}  // namespace benes

using namespace benes;

extern "C" {

int benes_profile_enable(int on) {
    std::lock_guard<std::mutex> lk(g_pmu);
    g_enabled = on != 0;
    return BENES_OK;
}

int benes_profile_enabled(void) {
    std::lock_guard<std::mutex> lk(g_pmu);
    return g_enabled ? 1 : 0;
}

int benes_profile_reset(void) {
    std::lock_guard<std::mutex> lk(g_pmu);
    for (Span &sp : g_spans) {
        cudaEventSynchronize(sp.stop);
        g_pool[sp.dev].push_back(sp.start);
        g_pool[sp.dev].push_back(sp.stop);
    }
    g_spans.clear();
    return BENES_OK;
}

int benes_profile_read(int kind, unsigned long long *launches, double *milliseconds) {
    if (kind < 0 || kind >= BENES_PROFILE_KINDS || !launches || !milliseconds) return BENES_ERR_BADARG;
    std::lock_guard<std::mutex> lk(g_pmu);
    unsigned long long n = 0;
    double ms = 0.0;
    for (Span &sp : g_spans) {
        if (sp.kind != kind) continue;
        float t = 0.f;
        BENES_CUDA_TRY(cudaEventSynchronize(sp.stop));
        BENES_CUDA_TRY(cudaEventElapsedTime(&t, sp.start, sp.stop));
        ms += t;
        n += sp.launches;
    }
    *launches = n;
    *milliseconds = ms;
    return BENES_OK;
}

int benes_profile_span(int index, int *kind, unsigned long long *launches, double *milliseconds) {
    if (index < 0 || !kind || !launches || !milliseconds) return BENES_ERR_BADARG;
    std::lock_guard<std::mutex> lk(g_pmu);
    if (index >= int(g_spans.size())) return BENES_ERR_BADARG;
    Span &sp = g_spans[index];
    float t = 0.f;
    BENES_CUDA_TRY(cudaEventSynchronize(sp.stop));
    BENES_CUDA_TRY(cudaEventElapsedTime(&t, sp.start, sp.stop));
    *kind = sp.kind;
    *launches = sp.launches;
    *milliseconds = t;
    return BENES_OK;
}

const char *benes_profile_kind_name(int kind) {
    return (kind >= 0 && kind < BENES_PROFILE_KINDS) ? kNames[kind] : "?";
}

}  // extern "C"
