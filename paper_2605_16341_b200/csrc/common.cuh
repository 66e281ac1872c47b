// Shared device-side definitions of the Orth-Dion step library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace od {

// per-matrix status bits (mirrors include/orthdion.h)
constexpr int ST_SHIFT_L = 1, ST_SHIFT_R = 2, ST_RANKDEF = 4, ST_NONFINITE = 8, ST_ZEROCOL = 16,
              ST_WAIT = 32;
constexpr int ST_FAILED = ST_RANKDEF | ST_NONFINITE | ST_WAIT;

// Everything a kernel needs to know about one matrix of a launch batch.
struct MatWork {
    void* X;            // m x n, fp32 or bf16
    float* M;           // m x n
    const void* G;      // m x n, fp32 or bf16
    float* Q;           // n x r
    float* P;           // m x r   (workspace slot; holds Y = B Q_prev before the left QR)
    float* R;           // n x r   (workspace slot)
    int32_t* status;    // one word
    char* scratch;      // per-matrix scratch area
};

constexpr int MAXB = 128;   // matrices per launch batch
struct Batch {
    int32_t count;
    int32_t pad;
    MatWork w[MAXB];
};

// Where a kernel finds an fp32 matrix of one MatWork.
enum Where : int32_t { W_Q = 0, W_P = 1, W_R = 2, W_SCRATCH = 3 };
struct Sel {
    int32_t where;
    int32_t pad;
    int64_t off;   // byte offset into scratch (W_SCRATCH only)
};
__device__ __forceinline__ float* pick(const MatWork& w, Sel s) {
    switch (s.where) {
        case W_Q: return w.Q;
        case W_P: return w.P;
        case W_R: return w.R;
        default: return reinterpret_cast<float*>(w.scratch + s.off);
    }
}

__device__ __forceinline__ float load_elem(const void* p, int64_t idx, int is_bf16) {
    if (is_bf16) return __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(p)[idx]);
    return reinterpret_cast<const float*>(p)[idx];
}

}  // namespace od
