// Launch accounting and optional per-stage timing with CUDA events on the launching stream.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>
#include <vector>

namespace od {
namespace prof {

enum Stage : int { S_MISC = 0, S_PACK, S_K1, S_GRAM, S_CHOL, S_APPLY, S_K3, S_COLNORM, S_K5, S_DIAG, S_COUNT };

inline const char* stage_name(int s) {
    static const char* names[S_COUNT] = {"misc", "pack", "k1_buffer_times_q", "gram", "cholesky_inverse",
                                         "apply_inverse", "k3_buffer_t_times_p", "colnorm", "k5_feedback_update",
                                         "diagnostics"};
    return (s >= 0 && s < S_COUNT) ? names[s] : "?";
}

struct Record { int stage; cudaEvent_t beg, end; };

inline std::atomic<int64_t> g_launches{0};
inline bool g_enabled = false;
inline std::vector<Record> g_records;
inline std::vector<cudaEvent_t> g_pool;
inline size_t g_pool_next = 0;

// Brackets one kernel launch: counts it and, when profiling is on, records an event pair.
struct Scope {
    cudaStream_t st;
    cudaEvent_t end = nullptr;
    Scope(int stage, cudaStream_t stream) : st(stream) {
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (g_enabled && g_pool_next + 2 <= g_pool.size()) {
            cudaEvent_t beg = g_pool[g_pool_next++];
            end = g_pool[g_pool_next++];
            cudaEventRecord(beg, st);
            g_records.push_back(Record{stage, beg, end});
        }
    }
    ~Scope() {
        if (end) cudaEventRecord(end, st);
    }
};

}  // namespace prof
}  // namespace od
