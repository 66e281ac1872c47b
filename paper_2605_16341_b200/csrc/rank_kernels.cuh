// Resize of the warm-start factor for the adaptive-rank rule (appendix algorithm "Ada-Orth-Dion
// Rank Selection", its last step: both factors are cut down or extended to the next rank).  Only
// V (here Q, n x r) is carried between steps; U (here P) is recomputed by every step.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace od {

// dst (n x r_new) <- leading columns of src (n x r_old), then the columns of pad (n x (r_new - r_old)).
// VEC = 4: all three row lengths are multiples of four and the pointers 16-byte aligned.
template <int VEC>
__global__ void __launch_bounds__(256)
resize_factor_kernel(const float* __restrict__ src, int64_t n, int r_old, float* __restrict__ dst, int r_new,
                     const float* __restrict__ pad) {
    const int keep = min(r_old, r_new), padw = r_new - keep;
    const int64_t per_row = r_new / VEC, total = n * per_row;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t i = idx / per_row;
        const int j = (int)(idx - i * per_row) * VEC;
        const float* from = j < keep ? src + i * r_old + j : pad + i * padw + (j - keep);
        if (VEC == 4) *reinterpret_cast<float4*>(dst + i * r_new + j) = *reinterpret_cast<const float4*>(from);
        else dst[i * r_new + j] = *from;
    }
}

}  // namespace od
