// r x r factor kernels of the tall-skinny QR (CholeskyQR): blocked Cholesky of the Gram matrix and
// the explicit inverse of its lower factor, one CTA per matrix; ColNorm; status initialisation.
#pragma once
#include "common.cuh"

namespace od {

constexpr int CH_THREADS = 512;               // two CTAs (two matrices) share an SM
constexpr int CH_NB = 32;                      // panel / diagonal block width
constexpr int CH_GROUPS = CH_THREADS / 256;    // groups of 256 threads run 64x64 tile products
constexpr int CH_DIAG_WARPS = 16;              // diagonal blocks inverted concurrently
constexpr size_t CH_SMEM_BYTES =
    (size_t)CH_GROUPS * 2 * 16 * 65 * 4 + (size_t)CH_DIAG_WARPS * 32 * 33 * 4 + 64;

__device__ __forceinline__ void group_bar(int g) {
    asm volatile("bar.sync %0, 256;" ::"r"(g + 1) : "memory");
}

// One group of 256 threads:  C(i,j) = beta*C(i,j) + alpha * sum_{k in [kbeg,kend)} A(i,k) B(k,j)
// for i < Mt <= 64, j < Nt <= 64.  Generic element strides.  lower_only: write only where the
// global column index (cg0 + j) does not exceed the global row index (rg0 + i).
__device__ void group_tile(float* C, int64_t c_rs, int64_t c_cs, const float* A, int64_t a_rs, int64_t a_cs,
                           const float* B, int64_t b_rs, int64_t b_cs, int Mt, int Nt, int kbeg, int kend,
                           float alpha, float beta, bool lower_only, int rg0, int cg0,
                           float* As, float* Bs, int gtid, int g) {
    const int tx = gtid % 16, ty = gtid / 16;
    float acc[4][4] = {};
    for (int k0 = kbeg; k0 < kend; k0 += 16) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            int idx = gtid + 256 * e;
            int ii, kk;
            if (a_cs == 1) { kk = idx % 16; ii = idx / 16; } else { ii = idx % 64; kk = idx / 64; }
            As[kk * 65 + ii] = (ii < Mt && k0 + kk < kend) ? A[(int64_t)ii * a_rs + (int64_t)(k0 + kk) * a_cs] : 0.f;
            int jj;
            if (b_cs == 1) { jj = idx % 64; kk = idx / 64; } else { kk = idx % 16; jj = idx / 16; }
            Bs[kk * 65 + jj] = (jj < Nt && k0 + kk < kend) ? B[(int64_t)(k0 + kk) * b_rs + (int64_t)jj * b_cs] : 0.f;
        }
        group_bar(g);
#pragma unroll
        for (int kk = 0; kk < 16; ++kk) {
            float a[4], b[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) { a[e] = As[kk * 65 + ty * 4 + e]; b[e] = Bs[kk * 65 + tx * 4 + e]; }
#pragma unroll
            for (int e = 0; e < 4; ++e)
#pragma unroll
                for (int f = 0; f < 4; ++f) acc[e][f] = fmaf(a[e], b[f], acc[e][f]);
        }
        group_bar(g);
    }
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
        for (int f = 0; f < 4; ++f) {
            int i = ty * 4 + e, j = tx * 4 + f;
            if (i < Mt && j < Nt && !(lower_only && (cg0 + j > rg0 + i))) {
                float* c = C + (int64_t)i * c_rs + (int64_t)j * c_cs;
                float v = alpha * acc[e][f];
                if (beta != 0.f) v += beta * *c;
                *c = v;
            }
        }
}

struct CholArgs {
    Sel gram;        // r x r Gram matrix (input, left intact)
    Sel work;        // r x r: receives L^{-1} (lower triangular, strict upper part zero)
    int32_t r;
    int32_t which;   // 0: left QR (P), 1: right QR (Q)
    int32_t pass;    // 1, 2 or 3
    float shift_rel; // shift = shift_rel * trace(Gram) on the retry of pass 1
    float cond_limit;// take the shifted path when max diag(L) / min diag(L) exceeds this (pass 1)
    // Optional fp32 column sums of squares, colsq[p * r + i] for p < MatWork::aux0 partial rows: when
    // use_colsq is set they replace the Gram diagonal.  (The tensor core truncates when it adds
    // into its fp32 accumulator, which biases long sums of squares low; the off-diagonal sums have
    // no such bias.)
    Sel colsq;
    int32_t use_colsq, pad;
    ImgRef img;      // img.off >= 0: also write L^{-1} as a split image (tensor-core operand)
    int64_t cnorm_off;   // >= 0: also leave the Gram diagonal (squared column norms) there, fp32 [r]
};

// Factor Gram = L L^T (blocked, right-looking) and overwrite `work` with L^{-1}.
// Pass 1 retries once with a diagonal shift when the factorisation breaks down or looks
// ill-conditioned, and records that in the status word so that a third QR pass is run.
__global__ void __launch_bounds__(CH_THREADS, 2)
chol_inv_kernel(const __grid_constant__ Batch batch, CholArgs a) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float* gemm_smem = reinterpret_cast<float*>(smem_raw);
    float* diag_smem = gemm_smem + CH_GROUPS * 2 * 16 * 65;
    __shared__ float red[32];
    __shared__ float s_diag[1024];
    __shared__ int s_fail;
    __shared__ float s_trace, s_dmin, s_dmax;
    __shared__ int s_status;

    const MatWork& w = batch.w[blockIdx.x];
    const int tid = threadIdx.x, lane = tid % 32, warp = tid / 32;
    const int g = tid / 256, gtid = tid % 256;
    float* As = gemm_smem + g * (2 * 16 * 65);
    float* Bs = As + 16 * 65;
    const int r = a.r;
    const int shift_bit = a.which ? ST_SHIFT_R : ST_SHIFT_L;

    if (tid == 0) s_status = *w.status;
    __syncthreads();
    const int st0 = s_status;
    if (st0 & ST_FAILED) return;
    if (a.pass == 3 && !(st0 & shift_bit)) return;

    const float* A = pick(w, a.gram);
    float* W = pick(w, a.work);

    // trace and finiteness of the Gram diagonal
    {
        float t = 0.f;
        for (int i = tid; i < r; i += CH_THREADS) {
            float d;
            if (a.use_colsq) {
                const float* cs = pick(w, a.colsq);
                d = 0.f;
                for (int kb = 0; kb < w.aux0; ++kb) d += cs[(int64_t)kb * r + i];
            } else {
                d = A[(int64_t)i * r + i];
            }
            s_diag[i] = d;
            if (a.cnorm_off >= 0) reinterpret_cast<float*>(w.scratch + a.cnorm_off)[i] = d;
            t += d;
        }
        for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (lane == 0) red[warp] = t;
        __syncthreads();
        if (warp == 0) {
            t = lane < CH_THREADS / 32 ? red[lane] : 0.f;
            for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
            if (lane == 0) s_trace = t;
        }
        __syncthreads();
    }
    const float trace = s_trace;
    if (!(fabsf(trace) <= 3.0e38f)) {   // Inf or NaN
        if (tid == 0) atomicOr(w.status, ST_NONFINITE);
        return;
    }

    bool ok = false;
    const int max_attempts = (a.pass == 1) ? 2 : 1;
    for (int attempt = 0; attempt < max_attempts && !ok; ++attempt) {
        const float shift = attempt ? a.shift_rel * trace : 0.f;
        // W <- lower(A) + shift*I, strict upper part zero
        for (int64_t e = tid; e < (int64_t)r * r; e += CH_THREADS) {
            int i = (int)(e / r), j = (int)(e % r);
            float v = (j <= i) ? A[e] : 0.f;
            if (i == j) v = s_diag[i] + shift;
            W[e] = v;
        }
        if (tid == 0) { s_fail = 0; s_dmin = 3.0e38f; s_dmax = 0.f; }
        __syncthreads();

        for (int k0 = 0; k0 < r; k0 += CH_NB) {
            const int nb = min(CH_NB, r - k0);
            float* D = diag_smem;   // 32 x 33, identity-padded
            for (int e = tid; e < 32 * 32; e += CH_THREADS) {
                int i = e / 32, j = e % 32;
                float v = (i == j) ? 1.f : 0.f;
                if (i < nb && j < nb && j <= i) v = W[(int64_t)(k0 + i) * r + k0 + j];
                D[i * 33 + j] = v;
            }
            __syncthreads();
            if (warp == 0) {
                // unblocked Cholesky of the 32 x 32 block: lane i owns row i
                float dmin = 3.0e38f, dmax = 0.f;
                int fail = 0;
                for (int j = 0; j < 32; ++j) {
                    float d = D[j * 33 + j];
                    if (!(d > 0.f) || !(d <= 3.0e38f)) { fail = 1; d = 1.f; }
                    float s = sqrtf(d);
                    if (j < nb) { dmin = fminf(dmin, s); dmax = fmaxf(dmax, s); }
                    float lij = 0.f;
                    if (lane > j) { lij = D[lane * 33 + j] / s; D[lane * 33 + j] = lij; }
                    if (lane == j) D[j * 33 + j] = s;
                    __syncwarp();
                    if (lane > j) {
                        for (int c = j + 1; c <= lane; ++c) D[lane * 33 + c] -= lij * D[c * 33 + j];
                    }
                    __syncwarp();
                }
                if (lane == 0) {
                    if (fail) s_fail = 1;
                    s_dmin = fminf(s_dmin, dmin);
                    s_dmax = fmaxf(s_dmax, dmax);
                }
            }
            __syncthreads();
            // write the factored block back (lower part)
            for (int e = tid; e < nb * nb; e += CH_THREADS) {
                int i = e / nb, j = e % nb;
                if (j <= i) W[(int64_t)(k0 + i) * r + k0 + j] = D[i * 33 + j];
            }
            const int t0 = k0 + nb;
            const int s = r - t0;
            if (s > 0) {
                // panel: rows below the block, x L_kk^T = w  (one thread per row)
                for (int i = tid; i < s; i += CH_THREADS) {
                    float* row = W + (int64_t)(t0 + i) * r + k0;
                    float x[CH_NB];
#pragma unroll
                    for (int c = 0; c < CH_NB; ++c) x[c] = (c < nb) ? row[c] : 0.f;
#pragma unroll
                    for (int c = 0; c < CH_NB; ++c) {
                        float v = x[c];
#pragma unroll
                        for (int p = 0; p < c; ++p) v = fmaf(-x[p], D[c * 33 + p], v);
                        x[c] = v / D[c * 33 + c];
                    }
#pragma unroll
                    for (int c = 0; c < CH_NB; ++c)
                        if (c < nb) row[c] = x[c];
                }
                __syncthreads();
                // trailing update: W[t0+i][t0+j] -= sum_c W[t0+i][k0+c] W[t0+j][k0+c], j <= i
                const int nt = (s + 63) / 64;
                int task = 0;
                for (int ti = 0; ti < nt; ++ti)
                    for (int tj = 0; tj <= ti; ++tj, ++task) {
                        if (task % CH_GROUPS != g) continue;
                        const int ri = t0 + ti * 64, cj = t0 + tj * 64;
                        group_tile(W + (int64_t)ri * r + cj, r, 1,
                                   W + (int64_t)ri * r + k0, r, 1,
                                   W + (int64_t)cj * r + k0, 1, r,
                                   min(64, r - ri), min(64, r - cj), 0, nb, -1.f, 1.f,
                                   ti == tj, ri, cj, As, Bs, gtid, g);
                    }
            }
            __syncthreads();
        }
        const bool fail = s_fail != 0;
        const bool ill = (a.pass == 1) && (s_dmax > a.cond_limit * s_dmin);
        if (!fail && !(ill && attempt == 0)) {
            ok = true;
        } else if (attempt == 0 && a.pass == 1) {
            if (tid == 0) atomicOr(w.status, shift_bit);
        }
        __syncthreads();
    }
    if (!ok) {
        if (tid == 0) atomicOr(w.status, ST_RANKDEF);
        return;
    }

    // ---- inverse of the lower factor, in place ------------------------------------------------
    // (1) 32 x 32 diagonal blocks: lane c solves for column c of the block inverse
    const int nblk = (r + 31) / 32;
    for (int b0 = 0; b0 < nblk; b0 += CH_DIAG_WARPS) {
        const int b = b0 + warp;
        float* Lb = diag_smem + (warp % CH_DIAG_WARPS) * (32 * 33);
        const bool mine = warp < CH_DIAG_WARPS && b < nblk;
        if (mine) {
            const int k0 = b * 32, nb = min(32, r - k0);
            for (int e = lane; e < 32 * 32; e += 32) {
                int i = e / 32, j = e % 32;
                float v = (i == j) ? 1.f : 0.f;
                if (i < nb && j < nb && j <= i) v = W[(int64_t)(k0 + i) * r + k0 + j];
                Lb[i * 33 + j] = v;
            }
            __syncwarp();
            float x[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                float sacc = (i == lane) ? 1.f : 0.f;
#pragma unroll
                for (int p = 0; p < i; ++p) sacc = fmaf(-Lb[i * 33 + p], x[p], sacc);
                x[i] = (i >= lane) ? sacc / Lb[i * 33 + i] : 0.f;
            }
            // lane = column c; write column c of the inverse (rows >= c)
#pragma unroll
            for (int i = 0; i < 32; ++i)
                if (i < nb && lane < nb && i >= lane) W[(int64_t)(k0 + i) * r + k0 + lane] = x[i];
        }
        __syncthreads();
    }
    // (2) combine blocks pairwise: inv [[A,0],[B,C]] = [[Ai,0],[-Ci B Ai, Ci]]
    for (int s = 32; s < r; s *= 2) {
        const int npairs = (r + 2 * s - 1) / (2 * s);
        // step 1: T = B * Ai, kept transposed in the (unused, zero) mirror block above the diagonal
        int task = 0;
        for (int pr = 0; pr < npairs; ++pr) {
            const int p = pr * 2 * s;
            const int sc = min(s, r - p - s);
            if (sc <= 0) continue;
            for (int ti = 0; ti < (sc + 63) / 64; ++ti)
                for (int tk = 0; tk < (s + 63) / 64; ++tk, ++task) {
                    if (task % CH_GROUPS != g) continue;
                    const int i0 = ti * 64, c0 = tk * 64;
                    group_tile(W + (int64_t)(p + c0) * r + (p + s + i0), 1, r,       // T(i,k) at W[p+k][p+s+i]
                               W + (int64_t)(p + s + i0) * r + p, r, 1,                // B(i,q)
                               W + (int64_t)p * r + (p + c0), r, 1,                    // Ai(q,k)
                               min(64, sc - i0), min(64, s - c0), c0, s, 1.f, 0.f,
                               false, 0, 0, As, Bs, gtid, g);
                }
        }
        __syncthreads();
        // step 2: B <- -Ci * T
        task = 0;
        for (int pr = 0; pr < npairs; ++pr) {
            const int p = pr * 2 * s;
            const int sc = min(s, r - p - s);
            if (sc <= 0) continue;
            for (int ti = 0; ti < (sc + 63) / 64; ++ti)
                for (int tk = 0; tk < (s + 63) / 64; ++tk, ++task) {
                    if (task % CH_GROUPS != g) continue;
                    const int i0 = ti * 64, c0 = tk * 64;
                    group_tile(W + (int64_t)(p + s + i0) * r + (p + c0), r, 1,        // Bnew(i,k)
                               W + (int64_t)(p + s + i0) * r + (p + s), r, 1,          // Ci(i,q)
                               W + (int64_t)(p + c0) * r + (p + s), 1, r,              // T(q,k) at W[p+k][p+s+q]
                               min(64, sc - i0), min(64, s - c0), 0, min(sc, i0 + 64), -1.f, 0.f,
                               false, 0, 0, As, Bs, gtid, g);
                }
        }
        __syncthreads();
        // clear the mirror blocks again
        for (int pr = 0; pr < npairs; ++pr) {
            const int p = pr * 2 * s;
            const int sc = min(s, r - p - s);
            if (sc <= 0) continue;
            for (int e = tid; e < s * sc; e += CH_THREADS) {
                int k = e / sc, i = e % sc;
                W[(int64_t)(p + k) * r + (p + s + i)] = 0.f;
            }
        }
        __syncthreads();
    }
    // ---- split image of L^{-1} for the tensor-core apply product ------------------------------
    if (a.img.off >= 0) {
        unsigned char* scr = reinterpret_cast<unsigned char*>(w.scratch);
        const int chunks = a.img.panels * a.img.rows_pad * 8;
        for (int q = tid; q < chunks; q += CH_THREADS) {
            const int c = q % 8, row = (q / 8) % a.img.rows_pad, panel = q / (8 * a.img.rows_pad);
            const int col = panel * 64 + c * 8;
            float v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = (row < r && col + i < r) ? W[(int64_t)row * r + col + i] : 0.f;
            uint4 t0, t1;
            split8(v, t0, t1);
            const int o = img_chunk_offset(row, c);
            *reinterpret_cast<uint4*>(scr + img_row_offset(a.img, 0, panel, row) + o) = t0;
            *reinterpret_cast<uint4*>(scr + img_row_offset(a.img, 1, panel, row) + o) = t1;
        }
    }
}

// ---- ColNorm (Alg. 1, normalisation step, Dion branch): Q[:,j] = R[:,j] / ||R[:,j]||_2 ----------------------
// One CTA per 32 columns: 32 x 32 threads, lanes along columns (coalesced rows).
// part: 0 = the whole operation; 1 = only the squared column norms of the rows at hand, left at
// cnorm_off (a column-sharded matrix sums them over the shards before it scales); 2 = only the
// scaling, with the squared norms taken from cnorm_off.
__global__ void __launch_bounds__(1024)
colnorm_kernel(const __grid_constant__ Batch batch, int64_t n, int r, int64_t cnorm_off, int part_sel) {
    const MatWork& w = batch.w[blockIdx.z];
    if (*w.status & ST_FAILED) return;
    __shared__ float part[32][33];
    __shared__ float inv[32];
    const int lane = threadIdx.x % 32, ry = threadIdx.x / 32;
    const int j = blockIdx.x * 32 + lane;
    float s = 0.f;
    if (j < r && part_sel != 2)
        for (int64_t i = ry; i < n; i += 32) { float v = w.R[i * r + j]; s = fmaf(v, v, s); }
    part[ry][lane] = s;
    __syncthreads();
    if (ry == 0) {
        float t = 0.f;
        if (part_sel == 2) {
            if (j < r) t = reinterpret_cast<const float*>(w.scratch + cnorm_off)[j];
        } else {
            for (int k = 0; k < 32; ++k) t += part[k][lane];
            if (cnorm_off >= 0 && j < r) reinterpret_cast<float*>(w.scratch + cnorm_off)[j] = t;
        }
        float nrm = sqrtf(t);
        if (j < r && !(nrm > 0.f) && part_sel != 1) atomicOr(w.status, ST_ZEROCOL);
        inv[lane] = (nrm > 0.f) ? 1.f / nrm : 0.f;
    }
    __syncthreads();
    if (j < r && part_sel != 1) {
        const float sc = inv[lane];
        for (int64_t i = ry; i < n; i += 32) w.Q[i * r + j] = w.R[i * r + j] * sc;
    }
}

// ---- helpers of the column-sharded step ---------------------------------------------------------
// Column sums of squares of an fp32 matrix S (rows x r) per block of 32 rows, in the layout the
// product kernels write next to their results: out[blk * r + j], blk < 4 * ceil(rows / 128)
// (blocks beyond the matrix hold zeros).  One CTA per (32-row block, 256 columns).
__global__ void __launch_bounds__(256)
colsq_blocks_kernel(const __grid_constant__ Batch batch, Sel src, int64_t rows, int r, int64_t colsq_off) {
    const MatWork& w = batch.w[blockIdx.z];
    if (*w.status & ST_FAILED) return;
    const float* S = pick(w, src);
    float* out = reinterpret_cast<float*>(w.scratch + colsq_off);
    const int j = blockIdx.y * 256 + threadIdx.x;
    if (j >= r) return;
    const int64_t i0 = (int64_t)blockIdx.x * 32;
    float s = 0.f;
    for (int k = 0; k < 32; ++k)
        if (i0 + k < rows) { const float v = S[(i0 + k) * r + j]; s = fmaf(v, v, s); }
    out[(int64_t)blockIdx.x * r + j] = s;
}

// Gram diagonal <- sum of the per-block column sums of squares (fp32 sums: the tensor core's
// truncating accumulation would bias the diagonal low), so that a reduction of the r x r matrix
// over the shards carries the exact diagonal along.
__global__ void __launch_bounds__(256)
gram_diag_kernel(const __grid_constant__ Batch batch, Sel gram, int r, int64_t colsq_off, int blocks) {
    const MatWork& w = batch.w[blockIdx.z];
    if (*w.status & ST_FAILED) return;
    const int j = blockIdx.x * 256 + threadIdx.x;
    if (j >= r) return;
    const float* cs = reinterpret_cast<const float*>(w.scratch + colsq_off);
    float d = 0.f;
    for (int b = 0; b < blocks; ++b) d += cs[(int64_t)b * r + j];
    pick(w, gram)[(int64_t)j * r + j] = d;
}

__global__ void init_status_kernel(const __grid_constant__ Batch batch) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < batch.count) *batch.w[i].status = 0;
}

}  // namespace od
