// Optional per-step diagnostics, computed on the device from what the step leaves behind:
//   nu      = ||Q||_op, the dual-norm factor of the update P Q^T (Proposition 3.1: 1 for Orth-Dion,
//             in [1, sqrt(r)] for column-normalised Dion)
//   erank   = exp(-sum p log p), p_j proportional to the column norms of R (the effective-rank
//             estimator of the adaptive-rank section)
//   tr_t2   = <B, P Q^T> = <R, Q>     (Lemma 4.2: equals tr(T_2) for Orth-Dion)
//   norm_r  = ||R||_F = ||P^T B||_F   (energy of the buffer captured by the left factor)
//   norm_m, norm_g = ||M'||_F, ||G||_F (error-feedback diagnostics; one extra sweep over M and G)
//   norm_b  = ||B||_F, from ||M'||^2 = a^2 ||B||^2 - (2ab - b^2) ||R||^2  (P^T P = I)
// The r x r Gram matrix Q^T Q comes from the engine's Gram product; this file holds the small
// kernels around it.
#pragma once
#include "common.cuh"

namespace od {

constexpr int DIAG_RESULTS = 8;     // floats copied out per matrix
constexpr int DIAG_STRIDE = 16;     // floats reserved per matrix: results, then two double accumulators
constexpr int DIAG_THREADS = 1024;
constexpr int DIAG_MAX_ITERS = 96;

enum DiagSlot : int { DG_NU = 0, DG_ERANK, DG_TR_T2, DG_NORM_R, DG_NORM_M, DG_NORM_G, DG_NORM_B, DG_ITERS };

struct DiagBase { const int32_t* status_base; float* diag_base; };

__device__ __forceinline__ float* diag_record(const MatWork& w, const DiagBase& d) {
    return d.diag_base + (int64_t)(w.status - d.status_base) * DIAG_STRIDE;
}

__global__ void diag_init_kernel(const __grid_constant__ Batch batch, DiagBase d) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= batch.count * DIAG_STRIDE) return;
    diag_record(batch.w[i / DIAG_STRIDE], d)[i % DIAG_STRIDE] = 0.f;
}

// Column statistics of R and Q (both n x r fp32, row-major): stats[j] = sum_i R_ij^2,
// stats[r + j] = sum_i R_ij Q_ij, stats[2r + j] = sum_i Q_ij^2.  One CTA per 32 columns, lanes
// along columns.
__global__ void __launch_bounds__(1024)
diag_colstats_kernel(const __grid_constant__ Batch batch, int64_t n, int r, int64_t stats_off) {
    const MatWork& w = batch.w[blockIdx.z];
    __shared__ float part[3][32][33];
    const int lane = threadIdx.x % 32, ry = threadIdx.x / 32;
    const int j = blockIdx.x * 32 + lane;
    float s = 0.f, t = 0.f, u = 0.f;
    if (j < r)
        for (int64_t i = ry; i < n; i += 32) {
            const float v = w.R[i * r + j], q = w.Q[i * r + j];
            s = fmaf(v, v, s);
            t = fmaf(v, q, t);
            u = fmaf(q, q, u);
        }
    part[0][ry][lane] = s;
    part[1][ry][lane] = t;
    part[2][ry][lane] = u;
    __syncthreads();
    if (ry < 3 && j < r) {
        float acc = 0.f;
        for (int k = 0; k < 32; ++k) acc += part[ry][k][lane];
        reinterpret_cast<float*>(w.scratch + stats_off)[ry * r + j] = acc;
    }
}

// The same for r % 4 == 0: one CTA per 128 columns, a lane reads four adjacent columns.
__global__ void __launch_bounds__(1024)
diag_colstats4_kernel(const __grid_constant__ Batch batch, int64_t n, int r, int64_t stats_off) {
    const MatWork& w = batch.w[blockIdx.z];
    __shared__ __align__(16) float part[3][16][132];
    const int lane = threadIdx.x % 32, ry = threadIdx.x / 32;
    const int j = blockIdx.x * 128 + lane * 4;
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f), t = s, u = s;
    if (j < r)
        for (int64_t i = ry; i < n; i += 32) {
            const float4 a = *reinterpret_cast<const float4*>(w.R + i * r + j);
            const float4 q = *reinterpret_cast<const float4*>(w.Q + i * r + j);
            s.x = fmaf(a.x, a.x, s.x); s.y = fmaf(a.y, a.y, s.y); s.z = fmaf(a.z, a.z, s.z); s.w = fmaf(a.w, a.w, s.w);
            t.x = fmaf(a.x, q.x, t.x); t.y = fmaf(a.y, q.y, t.y); t.z = fmaf(a.z, q.z, t.z); t.w = fmaf(a.w, q.w, t.w);
            u.x = fmaf(q.x, q.x, u.x); u.y = fmaf(q.y, q.y, u.y); u.z = fmaf(q.z, q.z, u.z); u.w = fmaf(q.w, q.w, u.w);
        }
    if (ry >= 16) {
        *reinterpret_cast<float4*>(&part[0][ry - 16][lane * 4]) = s;
        *reinterpret_cast<float4*>(&part[1][ry - 16][lane * 4]) = t;
        *reinterpret_cast<float4*>(&part[2][ry - 16][lane * 4]) = u;
    }
    __syncthreads();
    if (ry < 16) {
        const float4 s2 = *reinterpret_cast<const float4*>(&part[0][ry][lane * 4]);
        const float4 t2 = *reinterpret_cast<const float4*>(&part[1][ry][lane * 4]);
        const float4 u2 = *reinterpret_cast<const float4*>(&part[2][ry][lane * 4]);
        *reinterpret_cast<float4*>(&part[0][ry][lane * 4]) = make_float4(s.x + s2.x, s.y + s2.y, s.z + s2.z, s.w + s2.w);
        *reinterpret_cast<float4*>(&part[1][ry][lane * 4]) = make_float4(t.x + t2.x, t.y + t2.y, t.z + t2.z, t.w + t2.w);
        *reinterpret_cast<float4*>(&part[2][ry][lane * 4]) = make_float4(u.x + u2.x, u.y + u2.y, u.z + u2.z, u.w + u2.w);
    }
    __syncthreads();
    if (threadIdx.x < 384) {
        const int which = threadIdx.x / 128, c = threadIdx.x % 128;
        if (blockIdx.x * 128 + c < r) {
            float acc = 0.f;
            for (int k = 0; k < 16; ++k) acc += part[which][k][c];
            reinterpret_cast<float*>(w.scratch + stats_off)[which * r + blockIdx.x * 128 + c] = acc;
        }
    }
}

// Sums of squares of M (fp32) and G over the whole matrix, accumulated in double.
__global__ void __launch_bounds__(256)
diag_frob_kernel(const __grid_constant__ Batch batch, int64_t elems, int g_bf16, DiagBase d) {
    const MatWork& w = batch.w[blockIdx.z];
    const int64_t quads = elems / 4;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    float sm = 0.f, sg = 0.f;
    double dm = 0.0, dg = 0.0;
    int since = 0;
    for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q < quads; q += stride) {
        const float4 mv = reinterpret_cast<const float4*>(w.M)[q];
        sm += mv.x * mv.x + mv.y * mv.y + mv.z * mv.z + mv.w * mv.w;
        if (g_bf16) {
            const uint2 gv = reinterpret_cast<const uint2*>(w.G)[q];
            const float g0 = bf16lo_to_f32(gv.x), g1 = bf16hi_to_f32(gv.x);
            const float g2 = bf16lo_to_f32(gv.y), g3 = bf16hi_to_f32(gv.y);
            sg += g0 * g0 + g1 * g1 + g2 * g2 + g3 * g3;
        } else {
            const float4 gv = reinterpret_cast<const float4*>(w.G)[q];
            sg += gv.x * gv.x + gv.y * gv.y + gv.z * gv.z + gv.w * gv.w;
        }
        if (++since == 64) { dm += sm; dg += sg; sm = sg = 0.f; since = 0; }   // short fp32 runs only
    }
    if (blockIdx.x == 0 && threadIdx.x == 0)
        for (int64_t e = quads * 4; e < elems; ++e) {
            const float mv = w.M[e];
            const float gv = g_bf16 ? __bfloat162float(reinterpret_cast<const __nv_bfloat16*>(w.G)[e])
                                    : reinterpret_cast<const float*>(w.G)[e];
            dm += (double)mv * mv; dg += (double)gv * gv;
        }
    dm += sm; dg += sg;
    for (int o = 16; o; o >>= 1) {
        dm += __shfl_xor_sync(0xffffffffu, dm, o);
        dg += __shfl_xor_sync(0xffffffffu, dg, o);
    }
    __shared__ double red[2][8];
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    if (lane == 0) { red[0][warp] = dm; red[1][warp] = dg; }
    __syncthreads();
    if (threadIdx.x < 2) {
        double t = 0.0;
        for (int k = 0; k < 8; ++k) t += red[threadIdx.x][k];
        double* acc = reinterpret_cast<double*>(diag_record(w, d) + DIAG_RESULTS);
        atomicAdd(acc + threadIdx.x, t);
    }
}

__device__ __forceinline__ float diag_block_sum(float v, float* red) {
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    __syncthreads();                       // red may still be read from the previous call
    if (lane == 0) red[warp] = v;
    __syncthreads();
    float t = 0.f;
    for (int k = 0; k < DIAG_THREADS / 32; ++k) t += red[k];
    return t;
}

// Largest eigenvalue of the symmetric tridiagonal matrix (alpha_1..k; beta_2..k off the
// diagonal), by one warp: each round cuts the bracket into 33 parts, every lane counts with the
// Sturm sequence how many eigenvalues lie below its point.
__device__ float diag_tridiag_max(const float* alpha, const float* beta, int k, int lane) {
    float lo = alpha[0], hi = 0.f;
    for (int i = 0; i < k; ++i) {
        const float off = (i > 0 ? fabsf(beta[i]) : 0.f) + (i + 1 < k ? fabsf(beta[i + 1]) : 0.f);
        lo = fmaxf(lo, alpha[i]);                     // lambda_max >= every diagonal entry
        hi = fmaxf(hi, fabsf(alpha[i]) + off);        // Gershgorin
    }
    hi = hi * (1.f + 1e-6f) + 1e-30f;
    if (k == 1) return alpha[0];
    for (int round = 0; round < 5; ++round) {
        const float step = (hi - lo) * (1.f / 33.f);
        const float x = lo + step * (float)(lane + 1);
        float dd = alpha[0] - x;
        int below = dd < 0.f;
        for (int i = 1; i < k; ++i) {
            if (dd == 0.f) dd = 1e-30f;
            dd = alpha[i] - x - beta[i] * beta[i] / dd;
            below += dd < 0.f;
        }
        const unsigned all_below = __ballot_sync(0xffffffffu, below == k);   // lambda_max < x
        const int first = all_below ? __ffs(all_below) - 1 : 32;
        const float nlo = lo + step * (float)first, nhi = first < 32 ? lo + step * (float)(first + 1) : hi;
        lo = nlo; hi = nhi;
    }
    return 0.5f * (lo + hi);
}

// One CTA per matrix: finishes the diagnostics.  `gram` holds Q^T Q (at least its lower
// triangle; it is mirrored in place first).  Its diagonal is replaced by the column squares of Q
// summed in fp32 registers: the tensor-core accumulation rounds towards zero, which lowers a sum
// of n positive terms by about 5e-9 n (relative), visible in nu of an orthonormal Q at n ~ 10^4;
// the off-diagonal entries keep that bias (it enters nu only through nu^2 - 1).  nu^2 is the largest eigenvalue of Q^T Q: Lanczos
// iteration from a fixed pseudo-random start (no re-orthogonalisation: only the top Ritz value is
// used, which converges regardless), the top Ritz value taken every fourth step and the iteration
// stopped once it has moved by less than 1e-6 (relative), the Krylov space is exhausted, or
// DIAG_MAX_ITERS products are done.
__global__ void __launch_bounds__(DIAG_THREADS)
diag_final_kernel(const __grid_constant__ Batch batch, int r, int64_t gram_off, int64_t stats_off, int mask,
                  float ef_a, float ef_b, DiagBase d) {
    const MatWork& w = batch.w[blockIdx.x];
    float* out = diag_record(w, d);
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    if (*w.status & ST_FAILED) {                 // the step left the state untouched
        if (tid < DIAG_RESULTS) out[tid] = __int_as_float(0x7fc00000);
        return;
    }
    __shared__ __align__(16) float vp[1024], v[1024], y[1024];
    __shared__ float red[DIAG_THREADS / 32];
    __shared__ float alpha[DIAG_MAX_ITERS], beta[DIAG_MAX_ITERS + 1], theta_sh;
    float* g = reinterpret_cast<float*>(w.scratch + gram_off);
    const float* colsq = reinterpret_cast<const float*>(w.scratch + stats_off);
    const float* rq = colsq + r;
    const float* qsq = colsq + 2 * r;

    // column norms of R: entropy of their distribution, ||R||_F, <R, Q>
    float s_sum = 0.f, sq_sum = 0.f, rq_sum = 0.f;
    for (int j = tid; j < r; j += DIAG_THREADS) {
        const float c = colsq[j];
        s_sum += sqrtf(c); sq_sum += c; rq_sum += rq[j];
    }
    s_sum = diag_block_sum(s_sum, red);
    sq_sum = diag_block_sum(sq_sum, red);
    rq_sum = diag_block_sum(rq_sum, red);
    float ent = 0.f;
    for (int j = tid; j < r; j += DIAG_THREADS) {
        const float p = sqrtf(colsq[j]) / s_sum;
        if (p > 0.f) ent -= p * logf(p);
    }
    ent = diag_block_sum(ent, red);

    // mirror the lower triangle
    for (int i = warp; i < r; i += DIAG_THREADS / 32)
        for (int j = i + 1 + lane; j < r; j += 32) g[(int64_t)i * r + j] = g[(int64_t)j * r + i];
    for (int j = tid; j < r; j += DIAG_THREADS) g[(int64_t)j * r + j] = qsq[j];
    float nrm2 = 0.f;
    for (int j = tid; j < r; j += DIAG_THREADS) {
        uint32_t h = (uint32_t)j * 2654435761u + 12345u;
        h ^= h >> 15; h *= 2246822519u; h ^= h >> 13;
        const float s0 = 0.5f + (float)(h & 0xffff) * (1.f / 65536.f);
        y[j] = s0; nrm2 += s0 * s0;
    }
    nrm2 = diag_block_sum(nrm2, red);
    for (int j = tid; j < r; j += DIAG_THREADS) { v[j] = y[j] * rsqrtf(nrm2); vp[j] = 0.f; }
    __syncthreads();

    float lambda = 0.f, beta_j = 0.f;
    int it = 0;
    bool done = false;
    while (!done) {
        // y = G v - beta_j v_prev ;  alpha = <y, v>
        for (int i = warp; i < r; i += DIAG_THREADS / 32) {
            const float* row = g + (int64_t)i * r;
            float acc = 0.f;
            if (r % 4 == 0) {
                for (int j = lane * 4; j < r; j += 128) {
                    const float4 gv = *reinterpret_cast<const float4*>(row + j);
                    const float4 vv = *reinterpret_cast<const float4*>(v + j);
                    acc = fmaf(gv.x, vv.x, fmaf(gv.y, vv.y, fmaf(gv.z, vv.z, fmaf(gv.w, vv.w, acc))));
                }
            } else {
                for (int j = lane; j < r; j += 32) acc = fmaf(row[j], v[j], acc);
            }
            for (int o = 16; o; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (lane == 0) y[i] = acc - beta_j * vp[i];
        }
        __syncthreads();
        float a = 0.f;
        for (int j = tid; j < r; j += DIAG_THREADS) a += y[j] * v[j];
        a = diag_block_sum(a, red);
        float bb = 0.f;
        for (int j = tid; j < r; j += DIAG_THREADS) {
            const float t = y[j] - a * v[j];
            y[j] = t; bb += t * t;
        }
        bb = sqrtf(diag_block_sum(bb, red));
        if (tid == 0) { alpha[it] = a; beta[it + 1] = bb; }
        ++it;
        const bool exhausted = !(bb > 1e-6f * fabsf(a)) || it >= r || it >= DIAG_MAX_ITERS;
        if (exhausted || it % 4 == 0) {
            __syncthreads();
            if (warp == 0) {
                const float th = diag_tridiag_max(alpha, beta, it, lane);
                if (lane == 0) theta_sh = th;
            }
            __syncthreads();
            const float th = theta_sh;
            done = exhausted || fabsf(th - lambda) <= 1e-6f * fabsf(th);
            lambda = th;
        }
        if (!done) {
            const float inv = 1.f / bb;
            for (int j = tid; j < r; j += DIAG_THREADS) { vp[j] = v[j]; v[j] = y[j] * inv; }
            beta_j = bb;
            __syncthreads();
        }
    }
    if (tid == 0) {
        out[DG_NU] = sqrtf(fmaxf(lambda, 0.f));
        out[DG_ERANK] = expf(ent);
        out[DG_TR_T2] = rq_sum;
        out[DG_NORM_R] = sqrtf(sq_sum);
        out[DG_ITERS] = (float)it;
        if (mask & 2) {
            const double* acc = reinterpret_cast<const double*>(out + DIAG_RESULTS);
            const double mm = acc[0], gg = acc[1];
            out[DG_NORM_M] = (float)sqrt(mm);
            out[DG_NORM_G] = (float)sqrt(gg);
            const double a = ef_a, b = ef_b;
            const double bb = a != 0.0 ? (mm + (2.0 * a * b - b * b) * (double)sq_sum) / (a * a) : 0.0;
            out[DG_NORM_B] = (float)sqrt(bb > 0.0 ? bb : 0.0);
        }
    }
}

}  // namespace od
