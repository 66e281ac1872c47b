// Plain fp32 FMA kernels: the SIMT engine's matrix products (any shape, any r >= 1).
// Used for tiny matrices and as an on-device cross-check of the tensor-core engine.
#pragma once
#include "common.cuh"

namespace od {

// ---- operand readers: value of the logical operand at (row i, depth k) ----------------------
struct RdPlain {            // fp32 matrix with arbitrary strides: elem(i,k) = p[i*rs + k*cs]
    Sel sel; int64_t rs, cs;
    static constexpr bool kBuf = false;
    __device__ __forceinline__ const float* base(const MatWork& w) const { return pick(w, sel); }
};
struct RdBuffer {           // B = M + G formed on the fly (Alg. 1, buffer step); trans: elem(i,k)=B[k][i]
    int64_t ld; int32_t g_bf16; int32_t trans;
    static constexpr bool kBuf = true;
};

template <class RD>
__device__ __forceinline__ float rd(const RD& r, const MatWork& w, int64_t i, int64_t k) {
    if constexpr (RD::kBuf) {
        int64_t idx = r.trans ? (k * r.ld + i) : (i * r.ld + k);
        return w.M[idx] + load_elem(w.G, idx, r.g_bf16);
    } else {
        return r.base(w)[i * r.rs + k * r.cs];
    }
}

// ---- epilogues ------------------------------------------------------------------------------
struct EpStore {            // C[i*ld + j] = acc ; destination may depend on the shift flag
    Sel dst, dst_if_shifted; int32_t shift_bit; int32_t skip_if_failed; int64_t ld;
    int32_t only_if_shifted;
    __device__ __forceinline__ bool active(const MatWork& w) const {
        int st = *w.status;
        if (skip_if_failed && (st & ST_FAILED)) return false;
        if (only_if_shifted && !(st & shift_bit)) return false;
        return true;
    }
    __device__ __forceinline__ void operator()(const MatWork& w, int64_t i, int64_t j, float acc) const {
        int st = *w.status;
        float* c = pick(w, (shift_bit && (st & shift_bit)) ? dst_if_shifted : dst);
        c[i * ld + j] = acc;
    }
};
struct EpErrorFeedback {    // M <- a*(M+G) - b*acc          (Alg. 1, error-feedback step)
    float a, b; int64_t ld; int32_t g_bf16;
    __device__ __forceinline__ bool active(const MatWork& w) const { return !(*w.status & ST_FAILED); }
    __device__ __forceinline__ void operator()(const MatWork& w, int64_t i, int64_t j, float acc) const {
        int64_t idx = i * ld + j;
        float bval = w.M[idx] + load_elem(w.G, idx, g_bf16);
        w.M[idx] = a * bval - b * acc;
    }
};
struct EpWeights {          // X <- c*X - d*acc              (Alg. 1, update step)
    float c, d; int64_t ld; int32_t x_bf16;
    __device__ __forceinline__ bool active(const MatWork& w) const { return !(*w.status & ST_FAILED); }
    __device__ __forceinline__ void operator()(const MatWork& w, int64_t i, int64_t j, float acc) const {
        int64_t idx = i * ld + j;
        if (x_bf16) {
            __nv_bfloat16* x = reinterpret_cast<__nv_bfloat16*>(w.X);
            x[idx] = __float2bfloat16_rn(c * __bfloat162float(x[idx]) - d * acc);
        } else {
            float* x = reinterpret_cast<float*>(w.X);
            x[idx] = c * x[idx] - d * acc;
        }
    }
};

// C(i,j) = sum_k A(i,k) * Bm(j,k): both operands are read as (row, depth).
// 64 x 64 tile per CTA, 256 threads, 4 x 4 outputs per thread, depth chunks of 16.
template <class RA, class RB, class EP>
__global__ void __launch_bounds__(256)
simt_gemm_kernel(const __grid_constant__ Batch batch, int64_t Md, int64_t Nd, int64_t Kd,
                 RA ra, RB rb, EP ep) {
    const MatWork& w = batch.w[blockIdx.z];
    if (!ep.active(w)) return;
    __shared__ float As[16][65];
    __shared__ float Bs[16][65];
    const int tid = threadIdx.x;
    const int tx = tid % 16, ty = tid / 16;
    const int64_t i0 = (int64_t)blockIdx.y * 64, j0 = (int64_t)blockIdx.x * 64;
    float acc[4][4] = {};
    for (int64_t k0 = 0; k0 < Kd; k0 += 16) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int idx = tid + 256 * e;
            int kk = idx % 16, ii = idx / 16;
            int64_t gi = i0 + ii, gj = j0 + ii, gk = k0 + kk;
            As[kk][ii] = (gi < Md && gk < Kd) ? rd(ra, w, gi, gk) : 0.f;
            Bs[kk][ii] = (gj < Nd && gk < Kd) ? rd(rb, w, gj, gk) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) { a[e] = As[kk][ty * 4 + e]; b[e] = Bs[kk][tx * 4 + e]; }
#pragma unroll
            for (int e = 0; e < 4; ++e)
#pragma unroll
                for (int f = 0; f < 4; ++f) acc[e][f] = fmaf(a[e], b[f], acc[e][f]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int f = 0; f < 4; ++f) {
            int64_t gi = i0 + ty * 4 + e, gj = j0 + tx * 4 + f;
            if (gi < Md && gj < Nd) ep(w, gi, gj, acc[e][f]);
        }
}

}  // namespace od
