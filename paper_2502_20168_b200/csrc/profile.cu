// Measurement helpers: a count of kernel launches and optional per-stage CUDA-event timing.
// Both are process-wide and meant for single-threaded benchmarking; they never change results.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "kernels.h"

namespace ssm {

static std::atomic<long long> g_launches{0};
void count_launch(int n) { g_launches += n; }

struct StageRecord {
    const char* name;
    cudaEvent_t start, stop;
};
static bool g_profiling = false;
static std::vector<StageRecord> g_records;
static std::vector<cudaEvent_t> g_free_events;
constexpr size_t kMaxRecords = 1 << 16;

static cudaEvent_t get_event() {
    if (!g_free_events.empty()) {
        cudaEvent_t e = g_free_events.back();
        g_free_events.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

StageTimer::StageTimer(const char* name, cudaStream_t st) : st_(st), idx_(-1) {
    if (!g_profiling || g_records.size() >= kMaxRecords) return;
    StageRecord r{name, get_event(), get_event()};
    if (!r.start || !r.stop) return;
    cudaEventRecord(r.start, st);
    idx_ = (int)g_records.size();
    g_records.push_back(r);
}
StageTimer::~StageTimer() {
    if (idx_ >= 0) cudaEventRecord(g_records[idx_].stop, st_);
}

}  // namespace ssm

using namespace ssm;

#define SSM_API extern "C" __attribute__((visibility("default")))

SSM_API long long ssm_launch_count(void) { return g_launches.load(); }

SSM_API int ssm_profile_begin(void) {
    g_profiling = true;
    return SSM_OK;
}

SSM_API int ssm_profile_end(char* buf, size_t buf_bytes) {
    g_profiling = false;
    if (cudaDeviceSynchronize() != cudaSuccess) return SSM_ERR_CUDA;
    struct Acc { std::string name; int count; double ms; };
    std::vector<Acc> acc;
    for (const StageRecord& r : g_records) {
        float ms = 0.f;
        cudaEventElapsedTime(&ms, r.start, r.stop);
        size_t i = 0;
        for (; i < acc.size(); ++i)
            if (acc[i].name == r.name) break;
        if (i == acc.size()) acc.push_back({r.name, 0, 0.0});
        acc[i].count += 1;
        acc[i].ms += ms;
        g_free_events.push_back(r.start);
        g_free_events.push_back(r.stop);
    }
    g_records.clear();
    if (buf && buf_bytes) {
        size_t off = 0;
        buf[0] = 0;
        for (const Acc& a : acc) {
            int n = snprintf(buf + off, buf_bytes - off, "%s %d %.6f\n", a.name.c_str(), a.count, a.ms);
            if (n < 0 || (size_t)n >= buf_bytes - off) break;
            off += (size_t)n;
        }
    }
    return SSM_OK;
}
