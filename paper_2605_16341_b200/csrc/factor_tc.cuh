// r x r factor kernel of the tensor-core engine: blocked Cholesky of the Gram matrix and the
// explicit inverse of its lower factor, one CTA (256 threads) per matrix, two CTAs per SM.
//
// Everything of cubic cost is a list of independent 64 x 64 tile products run on the warp-level
// tensor-core path (mma.sync m16n8k16, bf16 operands, fp32 accumulation).  Operands are split into
// two bf16 terms when they are staged in shared memory, and every 16 x 8 fragment is the sum of
// three products (hi*hi + hi*lo + lo*hi): about 2^-16 relative accuracy per product.  (The first
// QR pass only has to tame the condition number; in the second pass the factor is close to the
// identity, so its off-diagonal products are small and their absolute error far below 1e-6.)
// The global loads of the next 32-deep chunk (of this tile or of the next one) are issued before
// the current chunk is multiplied, so the L2 latency hides behind the work.
//
// Left-looking Cholesky with 32-wide block columns:
//   column update    W[:, k] -= L[:, <k] L[k, <k]^T                    (tile products, depth 32 k: one
//                    long pipelined run per 64 rows, every entry of the matrix updated once)
//   diagonal block   in shared memory: columns scaled by one warp, rank-one updates by all
//                    threads; then one warp inverts it (needed at the end anyway) in place
//   panel            rows below  <-  rows below * inv(L_kk)^T          (tile products, depth 32)
// then the inverse of the factor by combining diagonal blocks pairwise (32, 64, 128, ...):
//   inv [[A, 0], [B, C]] = [[Ai, 0], [-Ci B Ai, Ci]]                   (tile products)
// The later passes of a CholeskyQR see a Gram matrix I + E with E tiny; when a rigorous bound on
// |E|_2 is small enough, L^{-1} = I - Phi(E) (first order) replaces the factorisation.
//
// MULTI form: one matrix per thread-block CLUSTER.  When a launch has fewer matrices than the
// device has room for CTAs, a lone CTA per matrix leaves most of the device idle while it walks
// its lists of tile products one after the other.  The CTAs of a cluster share one matrix: every
// list of independent tile products (column update, panel, the two steps of the pairwise
// inverse) and every copy loop is dealt out over the CTAs, the 32 x 32 diagonal blocks are
// factored by CTA 0 alone, and phases are separated by cluster barriers.  The matrix stays in
// global memory (L2); loads of data another CTA of the cluster may have written bypass L1
// (ld.global.cg) and follow a release/acquire cluster barrier.  Decisions that steer control
// flow (first-order inverse or not, breakdown, retry) are taken by CTA 0 and read by the others
// from its shared memory, so all CTAs of a cluster always take the same path.
#pragma once
#include "common.cuh"
#include "factor_kernels.cuh"

namespace od {

constexpr int CT_THREADS = 256;
constexpr int CT_NB = 32;
constexpr int CT_KC = 32;             // depth of one staged chunk
constexpr int CT_LDK = 40;            // staged rows: 32 bf16 + 8 of padding (conflict-free fragment loads)
constexpr int CT_MAX_TASKS = 160;
constexpr float CT_THIRD_PASS_LIMIT = 0.02f; // bound on |Gram - I|_2 of the second pass above which a third follows
constexpr float CT_SERIES_LIMIT = 1.4e-3f;   // bound on |Gram - I|_2 below which L^{-1} = I - Phi(E) is used

// C(i,j) = beta*C(i,j) + alpha * sum_{k in [kbeg,kend)} A(i,k) B(k,j), i < Mt <= 64, j < Nt <= 64.
// A(i,k) = A[i*a_rs + k];  B(k,j) = B[k*b_rs + j*b_cs] with b_rs == 1 (k contiguous) or b_cs == 1.
struct TcTask {
    float* C; const float* A; const float* B;
    int32_t c_rs, c_cs, a_rs, b_rs, b_cs;
    int32_t Mt, Nt, kbeg, kend, lower_only, rg0, cg0;
    float alpha, beta;
};

// ---- cluster helpers of the MULTI form ----------------------------------------------------
__device__ __forceinline__ void ct_cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the int at `p` (a shared-memory variable of this kernel) as CTA 0 of the cluster holds it
__device__ __forceinline__ int ct_read_cta0(const int* p) {
    const uint32_t local = static_cast<uint32_t>(__cvta_generic_to_shared(p));
    uint32_t remote;
    int v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(0));
    asm volatile("ld.shared::cluster.b32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
    return v;
}
// loads of matrix data that another CTA of the cluster may have written: L2 only
template <bool MULTI> __device__ __forceinline__ float ct_ld(const float* p) { return MULTI ? __ldcg(p) : *p; }
template <bool MULTI> __device__ __forceinline__ float2 ct_ld2(const float* p) {
    return MULTI ? __ldcg(reinterpret_cast<const float2*>(p)) : *reinterpret_cast<const float2*>(p);
}
template <bool MULTI> __device__ __forceinline__ float4 ct_ld4(const float* p) {
    return MULTI ? __ldcg(reinterpret_cast<const float4*>(p)) : *reinterpret_cast<const float4*>(p);
}

__device__ __forceinline__ void mma_bf16_16x8x16(float (&c)[4], const uint32_t (&a)[4], const uint32_t (&b)[2]) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// All 256 threads.  Warp w owns rows 16*(w % 4).., columns 32*(w / 4).. of the tile.
// MULTI: this CTA takes the tasks first, first + stride, ... of the list (its share of a cluster's work).
template <bool MULTI>
__device__ void tc_run_tasks(const TcTask* tasks, int ntasks, __nv_bfloat16* stage, int first = 0, int stride = 1) {
    if (ntasks <= first) return;
    __nv_bfloat16* Ah = stage;
    __nv_bfloat16* Al = Ah + 64 * CT_LDK;
    __nv_bfloat16* Bh = Al + 64 * CT_LDK;
    __nv_bfloat16* Bl = Bh + 64 * CT_LDK;
    const int tid = threadIdx.x, warp = tid / 32, lane = tid % 32;
    const int gq = lane / 4, tq = lane % 4;
    const int row0 = (warp % 4) * 16, col0 = (warp / 4) * 32;
    // Staging: a thread handles pairs of adjacent depth indices (one float2 load, one packed
    // bf16x2 store per term): A rows a_ii + 16 e at depth a_kk, a_kk + 1; B likewise when depth is
    // contiguous in memory, else single elements (jj = tid % 64, depth tid / 64 + 4 e).
    const int a_kk = (tid % 16) * 2, a_ii = tid / 16;
    float2 ra[4];
    float rb[8];
    auto load = [&](int task, int k0) {
        const TcTask& t = tasks[task];
        // kbeg, kend, a_rs are even and rows 8-byte aligned in all task lists of this file
        const float* Ap = t.A + (a_ii * t.a_rs + k0 + a_kk);
        const bool ak = k0 + a_kk < t.kend;
#pragma unroll
        for (int e = 0; e < 4; ++e)
            ra[e] = (ak && a_ii + 16 * e < t.Mt) ? ct_ld2<MULTI>(Ap + e * 16 * t.a_rs) : make_float2(0.f, 0.f);
        if (t.b_rs == 1) {
            const float* Bp = t.B + (k0 + a_kk + a_ii * t.b_cs);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const float2 v = (ak && a_ii + 16 * e < t.Nt) ? ct_ld2<MULTI>(Bp + e * 16 * t.b_cs) : make_float2(0.f, 0.f);
                rb[2 * e] = v.x; rb[2 * e + 1] = v.y;
            }
        } else {
            const int jj = tid % 64, kk = tid / 64;
            const float* Bp = t.B + ((k0 + kk) * t.b_rs + jj);
#pragma unroll
            for (int e = 0; e < 8; ++e)
                rb[e] = (jj < t.Nt && k0 + kk + 4 * e < t.kend) ? ct_ld<MULTI>(Bp + e * 4 * t.b_rs) : 0.f;
        }
    };
    int ti = first, k0 = tasks[first].kbeg;
    load(ti, k0);
    float acc[4][4] = {};
    while (true) {
        {
            const bool b_kfast = tasks[ti].b_rs == 1;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const uint32_t hi = pack_bf16x2(ra[e].x, ra[e].y);
                const uint32_t lo = pack_bf16x2(ra[e].x - bf16lo_to_f32(hi), ra[e].y - bf16hi_to_f32(hi));
                const int oa = (a_ii + 16 * e) * CT_LDK + a_kk;
                *reinterpret_cast<uint32_t*>(Ah + oa) = hi;
                *reinterpret_cast<uint32_t*>(Al + oa) = lo;
                if (b_kfast) {
                    const uint32_t bhi = pack_bf16x2(rb[2 * e], rb[2 * e + 1]);
                    const uint32_t blo = pack_bf16x2(rb[2 * e] - bf16lo_to_f32(bhi), rb[2 * e + 1] - bf16hi_to_f32(bhi));
                    *reinterpret_cast<uint32_t*>(Bh + oa) = bhi;
                    *reinterpret_cast<uint32_t*>(Bl + oa) = blo;
                }
            }
            if (!b_kfast) {
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    const __nv_bfloat16 bh = __float2bfloat16_rn(rb[e]);
                    const int ob = (tid % 64) * CT_LDK + tid / 64 + 4 * e;
                    Bh[ob] = bh;
                    Bl[ob] = __float2bfloat16_rn(rb[e] - __bfloat162float(bh));
                }
            }
        }
        __syncthreads();
        const bool last_chunk = k0 + CT_KC >= tasks[ti].kend;
        int nti = ti, nk0 = k0 + CT_KC;
        if (last_chunk) { nti = ti + stride; nk0 = nti < ntasks ? tasks[nti].kbeg : 0; }
        const bool has_next = nti < ntasks;
        if (has_next) load(nti, nk0);
#pragma unroll
        for (int ks = 0; ks < CT_KC; ks += 16) {
            uint32_t ah[4], al[4];
            const int o0 = (row0 + gq) * CT_LDK + ks + tq * 2, o1 = o0 + 8 * CT_LDK;
            ah[0] = *reinterpret_cast<const uint32_t*>(Ah + o0);     al[0] = *reinterpret_cast<const uint32_t*>(Al + o0);
            ah[1] = *reinterpret_cast<const uint32_t*>(Ah + o1);     al[1] = *reinterpret_cast<const uint32_t*>(Al + o1);
            ah[2] = *reinterpret_cast<const uint32_t*>(Ah + o0 + 8); al[2] = *reinterpret_cast<const uint32_t*>(Al + o0 + 8);
            ah[3] = *reinterpret_cast<const uint32_t*>(Ah + o1 + 8); al[3] = *reinterpret_cast<const uint32_t*>(Al + o1 + 8);
#pragma unroll
            for (int nf = 0; nf < 4; ++nf) {
                const int o = (col0 + nf * 8 + gq) * CT_LDK + ks + tq * 2;
                uint32_t bh[2], bl[2];
                bh[0] = *reinterpret_cast<const uint32_t*>(Bh + o);     bl[0] = *reinterpret_cast<const uint32_t*>(Bl + o);
                bh[1] = *reinterpret_cast<const uint32_t*>(Bh + o + 8); bl[1] = *reinterpret_cast<const uint32_t*>(Bl + o + 8);
                mma_bf16_16x8x16(acc[nf], ah, bh);
                mma_bf16_16x8x16(acc[nf], ah, bl);
                mma_bf16_16x8x16(acc[nf], al, bh);
            }
        }
        __syncthreads();
        if (last_chunk) {
            const TcTask& t = tasks[ti];
            // all reads of C first, then all writes: a load behind a store that may alias it would
            // wait for that store, and the sixteen round trips would line up one after the other
            if (t.c_cs == 1) {
                // rows of C are contiguous: the two columns of a fragment row go as one float2
                float2 cv2[4][2];
                bool v0[4][2], v1[4][2];
#pragma unroll
                for (int nf = 0; nf < 4; ++nf)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int i = row0 + gq + h * 8, j = col0 + nf * 8 + tq * 2;
                        v0[nf][h] = i < t.Mt && j < t.Nt && !(t.lower_only && (t.cg0 + j > t.rg0 + i));
                        v1[nf][h] = i < t.Mt && j + 1 < t.Nt && !(t.lower_only && (t.cg0 + j + 1 > t.rg0 + i));
                        cv2[nf][h] = (v0[nf][h] && t.beta != 0.f) ? ct_ld2<MULTI>(t.C + i * t.c_rs + j) : make_float2(0.f, 0.f);
                    }
#pragma unroll
                for (int nf = 0; nf < 4; ++nf)
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const int i = row0 + gq + h * 8, j = col0 + nf * 8 + tq * 2;
                        const float o0 = fmaf(t.beta, cv2[nf][h].x, t.alpha * acc[nf][2 * h]);
                        const float o1 = fmaf(t.beta, cv2[nf][h].y, t.alpha * acc[nf][2 * h + 1]);
                        if (v0[nf][h] && v1[nf][h]) *reinterpret_cast<float2*>(t.C + i * t.c_rs + j) = make_float2(o0, o1);
                        else if (v0[nf][h]) t.C[i * t.c_rs + j] = o0;
                        acc[nf][2 * h] = 0.f; acc[nf][2 * h + 1] = 0.f;
                    }
            } else {
            float cv[4][4];
            bool valid[4][4];
#pragma unroll
            for (int nf = 0; nf < 4; ++nf)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i = row0 + gq + (e / 2) * 8, j = col0 + nf * 8 + tq * 2 + (e % 2);
                    valid[nf][e] = i < t.Mt && j < t.Nt && !(t.lower_only && (t.cg0 + j > t.rg0 + i));
                    cv[nf][e] = (valid[nf][e] && t.beta != 0.f) ? ct_ld<MULTI>(t.C + i * t.c_rs + j * t.c_cs) : 0.f;
                }
#pragma unroll
            for (int nf = 0; nf < 4; ++nf)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int i = row0 + gq + (e / 2) * 8, j = col0 + nf * 8 + tq * 2 + (e % 2);
                    if (valid[nf][e]) t.C[i * t.c_rs + j * t.c_cs] = fmaf(t.beta, cv[nf][e], t.alpha * acc[nf][e]);
                    acc[nf][e] = 0.f;
                }
            }
        }
        if (!has_next) break;
        ti = nti; k0 = nk0;
    }
    __syncthreads();
}

template <bool MULTI>
__global__ void __launch_bounds__(CT_THREADS, 2)
chol_inv_tc_kernel(const __grid_constant__ Batch batch, CholArgs a, int csize) {
    __shared__ __align__(16) __nv_bfloat16 s_stage[4 * 64 * CT_LDK];
    __shared__ TcTask s_tasks[CT_MAX_TASKS];
    __shared__ float s_blk[32 * 33];
    __shared__ float s_piv[32];
    extern __shared__ float s_dyn[];          // 2 r floats: Gram diagonal, row sums of |Gram - I|
    float* s_diag = s_dyn;
    float* s_rowsum = s_dyn + a.r;
    __shared__ float red[8];
    __shared__ int s_ntasks, s_fail, s_status, s_decision;
    __shared__ float s_trace, s_dmin, s_dmax;

    // MULTI: the csize CTAs of a cluster (ranks 0 .. csize-1) share matrix blockIdx.x / csize
    const int crank = MULTI ? (int)(blockIdx.x % (unsigned)csize) : 0;
    const int nshare = MULTI ? csize : 1;
    const MatWork& w = batch.w[MULTI ? blockIdx.x / (unsigned)csize : blockIdx.x];
    const int tid = threadIdx.x, lane = tid % 32, warp = tid / 32;
    const int r = a.r;
    const int shift_bit = a.which ? ST_SHIFT_R : ST_SHIFT_L;
    auto phase_sync = [&]() { if (MULTI) ct_cluster_sync(); else __syncthreads(); };

    if (tid == 0) s_status = *w.status;
    __syncthreads();
    // every CTA of the cluster has read the status word before any of them may change it
    if (MULTI) ct_cluster_sync();
    const int st0 = s_status;
    if (st0 & ST_FAILED) return;
    if (a.pass == 3 && !(st0 & shift_bit)) return;

    const float* __restrict__ A = pick(w, a.gram);     // Gram matrix: never written here
    float* W = pick(w, a.work);

    // diagonal (from the fp32 column sums of squares), trace, finiteness
    {
        float t = 0.f;
        for (int i = tid; i < r; i += CT_THREADS) {
            float d;
            if (a.use_colsq) {
                const float* cs = pick(w, a.colsq);
                d = 0.f;
                for (int kb = 0; kb < w.aux0; ++kb) d += cs[kb * r + i];
            } else {
                d = A[i * r + i];
            }
            s_diag[i] = d;
            if (a.cnorm_off >= 0 && crank == 0) reinterpret_cast<float*>(w.scratch + a.cnorm_off)[i] = d;
            t += d;
        }
        for (int o = 16; o; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
        if (lane == 0) red[warp] = t;
        __syncthreads();
        if (tid == 0) {
            float s = 0.f;
            for (int i = 0; i < CT_THREADS / 32; ++i) s += red[i];
            s_trace = s;
        }
        __syncthreads();
    }
    const float trace = s_trace;
    // (the same sum in the same order in every CTA of a cluster: all of them take this exit or none)
    if (!(fabsf(trace) <= 3.0e38f)) {   // Inf or NaN
        if (tid == 0 && crank == 0) atomicOr(w.status, ST_NONFINITE);
        return;
    }

    // ---- later passes of the QR: the Gram matrix is I + E with E small ------------------------
    // L = I + X with X + X^T + X X^T = E, so L^{-1} = I - Phi(E) + O(|E|^2), Phi = strict lower part
    // plus half the diagonal.  |E|_2 <= max row sum of |E| (E is symmetric); when that bound is
    // below CT_SERIES_LIMIT the dropped terms are below 2e-6 and the factorisation is skipped.
    bool series = false;
    if (a.pass >= 2) {
        for (int i = tid; i < r; i += CT_THREADS) s_rowsum[i] = fabsf(s_diag[i] - 1.f);
        __syncthreads();
        // strictly lower entries, in column blocks of 1024 (32 column sums per lane in registers)
        for (int cb = 0; cb < r; cb += 1024) {
            float colacc[32];
#pragma unroll
            for (int t = 0; t < 32; ++t) colacc[t] = 0.f;
            for (int i = cb + warp; i < r; i += CT_THREADS / 32) {
                float rs = 0.f;
#pragma unroll
                for (int t = 0; t < 32; ++t) {
                    const int j = cb + lane + 32 * t;
                    if (j < i) {
                        const float v = fabsf(A[(size_t)i * r + j]);
                        rs += v; colacc[t] += v;
                    }
                }
                for (int o = 16; o; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
                if (lane == 0) atomicAdd(&s_rowsum[i], rs);
            }
#pragma unroll
            for (int t = 0; t < 32; ++t)
                if (cb + lane + 32 * t < r && colacc[t] != 0.f) atomicAdd(&s_rowsum[cb + lane + 32 * t], colacc[t]);
        }
        __syncthreads();
        float mx = 0.f;
        for (int i = tid; i < r; i += CT_THREADS) mx = fmaxf(mx, s_rowsum[i]);
        for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (lane == 0) red[warp] = mx;
        __syncthreads();
        mx = 0.f;
        for (int i = 0; i < CT_THREADS / 32; ++i) mx = fmaxf(mx, red[i]);
        series = mx <= CT_SERIES_LIMIT;          // false for NaN
        if (MULTI) {
            // the row sums are accumulated with shared-memory atomics, whose order may differ from
            // CTA to CTA: CTA 0 decides for the cluster
            if (tid == 0) s_decision = series ? 1 : 0;
            ct_cluster_sync();
            series = ct_read_cta0(&s_decision) != 0;
            ct_cluster_sync();                   // nobody overwrites s_decision before all have read it
        }
        // Second pass with Q1 far from orthonormal (cond(Y)^2 u was not small): its result will
        // not be orthonormal to working accuracy either, so ask for the third pass.
        if (a.pass == 2 && !(mx <= CT_THIRD_PASS_LIMIT) && tid == 0 && crank == 0) atomicOr(w.status, shift_bit);
        __syncthreads();
    }
    if (series) {
        const int r4 = r / 4;
        for (int q = tid + crank * CT_THREADS; q < r * r4; q += CT_THREADS * nshare) {
            const int i = q / r4, j4 = (q - i * r4) * 4;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (j4 <= i) {
                const float4 g = *reinterpret_cast<const float4*>(A + i * r + j4);
                const float dg = 0.5f * (3.f - s_diag[i]);
                v.x = j4 + 0 < i ? -g.x : (j4 + 0 == i ? dg : 0.f);
                v.y = j4 + 1 < i ? -g.y : (j4 + 1 == i ? dg : 0.f);
                v.z = j4 + 2 < i ? -g.z : (j4 + 2 == i ? dg : 0.f);
                v.w = j4 + 3 < i ? -g.w : (j4 + 3 == i ? dg : 0.f);
            }
            *reinterpret_cast<float4*>(W + i * r + j4) = v;
        }
        phase_sync();
    }

    // Task lists longer than the table are run in windows of CT_MAX_TASKS: thread 0 walks the whole
    // list for every window and keeps the tasks that fall into it.
    int gen_base = 0, gen_count = 0;
    auto add_task = [&](float* C, int c_rs, int c_cs, const float* A_, int a_rs, const float* B_, int b_rs, int b_cs,
                        int Mt, int Nt, int kbeg, int kend, float alpha, float beta, bool lower_only, int rg0, int cg0) {
        const int k = gen_count++;
        if (k < gen_base || k >= gen_base + CT_MAX_TASKS) return;
        TcTask& t = s_tasks[k - gen_base];
        t.C = C; t.A = A_; t.B = B_;
        t.c_rs = c_rs; t.c_cs = c_cs; t.a_rs = a_rs; t.b_rs = b_rs; t.b_cs = b_cs;
        t.Mt = Mt; t.Nt = Nt; t.kbeg = kbeg; t.kend = kend; t.lower_only = lower_only ? 1 : 0; t.rg0 = rg0; t.cg0 = cg0;
        t.alpha = alpha; t.beta = beta;
    };
    // Runs the list of independent tile products that build() enumerates (always in the same
    // order); MULTI: task k of the list goes to CTA k % nshare, and the cluster meets afterwards.
    auto run_list = [&](auto build) {
        for (int base = 0;; base += CT_MAX_TASKS) {
            if (tid == 0) { gen_base = base; gen_count = 0; build(); s_ntasks = gen_count; }
            __syncthreads();
            const int total = s_ntasks;
            const int first = MULTI ? ((crank - base % nshare) % nshare + nshare) % nshare : 0;
            tc_run_tasks<MULTI>(s_tasks, min(CT_MAX_TASKS, total - base), s_stage, first, nshare);
            __syncthreads();
            if (base + CT_MAX_TASKS >= total) break;
        }
        if (MULTI) ct_cluster_sync();
    };

    bool ok = series;
    const int max_attempts = (a.pass == 1) ? 2 : 1;
    for (int attempt = 0; attempt < max_attempts && !ok; ++attempt) {
        const float shift = attempt ? a.shift_rel * trace : 0.f;
        // W <- lower(A) + shift*I (diagonal from s_diag), strict upper part zero; 4 columns per thread
        // (eight loads in flight per thread: one at a time, the L2 round trips of this copy alone
        // were 8 % of the kernel)
        const int r4 = r / 4;
        for (int q0 = tid + crank * 8 * CT_THREADS; q0 < r * r4; q0 += 8 * CT_THREADS * nshare) {
            float4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int q = q0 + u * CT_THREADS;
                const int i = q / r4, j4 = (q - i * r4) * 4;
                v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (q < r * r4 && j4 <= i) v[u] = *reinterpret_cast<const float4*>(A + i * r + j4);
            }
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int q = q0 + u * CT_THREADS;
                if (q >= r * r4) break;
                const int i = q / r4, j4 = (q - i * r4) * 4;
                if (j4 <= i) {
                    if (j4 + 0 > i) v[u].x = 0.f; else if (j4 + 0 == i) v[u].x = s_diag[i] + shift;
                    if (j4 + 1 > i) v[u].y = 0.f; else if (j4 + 1 == i) v[u].y = s_diag[i] + shift;
                    if (j4 + 2 > i) v[u].z = 0.f; else if (j4 + 2 == i) v[u].z = s_diag[i] + shift;
                    if (j4 + 3 > i) v[u].w = 0.f; else if (j4 + 3 == i) v[u].w = s_diag[i] + shift;
                }
                *reinterpret_cast<float4*>(W + i * r + j4) = v[u];
            }
        }
        if (tid == 0) { s_fail = 0; s_dmin = 3.0e38f; s_dmax = 0.f; }
        phase_sync();

        for (int k0 = 0; k0 < r; k0 += CT_NB) {
            const int nb = min(CT_NB, r - k0);
            // Left-looking update of block column k0 with everything to its left:
            //   W[i][k0 + j] -= sum_{c < k0} W[i][c] W[k0 + j][c],  i >= k0 + j
            // One tile product per 64 rows with the whole depth k0 in one run (its 32-deep chunks
            // pipelined), so that every entry of the matrix is read, updated and written once.
            // (A right-looking trailing update after every panel, 230 short products at r = 512
            // each with its own round trip for the tile it updates, took 12 % longer on one CTA;
            // shared by a cluster the two forms are within 4 % of each other, and both forms of the
            // kernel keep the same one so that a matrix gets the same bits in either.)
            if (k0 > 0) {
                run_list([&]() {
                    for (int i0 = k0; i0 < r; i0 += 64)
                        add_task(W + (size_t)i0 * r + k0, r, 1, W + (size_t)i0 * r, r, W + (size_t)k0 * r, 1, r,
                                 min(64, r - i0), nb, 0, k0, -1.f, 1.f, i0 == k0, i0, k0);
                });
            }
            // Diagonal block: factored in shared memory by all threads (column scaling by one warp,
            // rank-one update by everybody, two barriers per column), then inverted by one warp
            // (thread c solves L x = e_c with x in registers; L(i, p) are broadcast reads).  The
            // inverse replaces the block in place right away: it is needed at the end anyway.
            if (crank == 0) {
                for (int e = tid; e < 1024; e += CT_THREADS) {
                    const int i = e >> 5, c = e & 31;
                    float v = (i == c) ? 1.f : 0.f;          // rows beyond nb are identity rows
                    if (i < nb && c <= i) v = ct_ld<MULTI>(W + (k0 + i) * r + k0 + c);
                    s_blk[i * 33 + c] = v;
                }
                __syncthreads();
                bool fail = false;
                float dmin = 3.0e38f, dmax = 0.f;             // every thread tracks the same values
                for (int j = 0; j < 32; ++j) {
                    float d = s_blk[j * 33 + j];
                    if (!(d > 0.f) || !(d <= 3.0e38f)) { if (j < nb) fail = true; d = 1.f; }
                    const float sq = sqrtf(d);
                    if (j < nb) { dmin = fminf(dmin, sq); dmax = fmaxf(dmax, sq); }
                    if (tid == j) s_piv[j] = sq;
                    else if (tid > j && tid < 32) s_blk[tid * 33 + j] = s_blk[tid * 33 + j] / sq;
                    __syncthreads();
                    for (int e = tid; e < 1024; e += CT_THREADS) {
                        const int i = e >> 5, c = e & 31;
                        if (c > j && i >= c)
                            s_blk[i * 33 + c] = fmaf(-s_blk[i * 33 + j], s_blk[c * 33 + j], s_blk[i * 33 + c]);
                    }
                    __syncthreads();
                }
                if (warp == 0) {
                    float x[32];
#pragma unroll
                    for (int i = 0; i < 32; ++i) {
                        float sacc = (i == lane) ? 1.f : 0.f;
#pragma unroll
                        for (int p = 0; p < 32; ++p)
                            if (p < i) sacc = fmaf(-s_blk[i * 33 + p], x[p], sacc);
                        x[i] = (i >= lane) ? sacc / s_piv[i] : 0.f;
                    }
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (i < nb && lane < nb && i >= lane) W[(k0 + i) * r + k0 + lane] = x[i];
                    if (lane == 0) {
                        if (fail) s_fail = 1;
                        s_dmin = fminf(s_dmin, dmin);
                        s_dmax = fmaxf(s_dmax, dmax);
                    }
                }
            }
            phase_sync();
            const int t0 = k0 + nb, s = r - t0;
            if (s > 0) {
                // panel: rows below <- rows below * inv(L_kk)^T
                run_list([&]() {
                    for (int i0 = 0; i0 < s; i0 += 64)
                        add_task(W + (size_t)(t0 + i0) * r + k0, r, 1, W + (size_t)(t0 + i0) * r + k0, r,
                                 W + (size_t)k0 * r + k0, 1, r, min(64, s - i0), nb, 0, nb, 1.f, 0.f, false, 0, 0);
                });
            }
        }
        bool fail = s_fail != 0;
        bool ill = (a.pass == 1) && (s_dmax > a.cond_limit * s_dmin);
        if (MULTI) {
            // only CTA 0 has factored the diagonal blocks: its verdict holds for the cluster
            if (tid == 0) s_decision = (fail ? 1 : 0) | (ill ? 2 : 0);
            ct_cluster_sync();
            const int d = ct_read_cta0(&s_decision);
            fail = (d & 1) != 0; ill = (d & 2) != 0;
            ct_cluster_sync();
        }
        if (!fail && !(ill && attempt == 0)) {
            ok = true;
        } else if (attempt == 0 && a.pass == 1) {
            if (tid == 0 && crank == 0) atomicOr(w.status, shift_bit);
        }
        __syncthreads();
    }
    if (!ok) {
        if (tid == 0 && crank == 0) atomicOr(w.status, ST_RANKDEF);
        return;
    }

    // ---- inverse of the lower factor: the diagonal blocks are inverted already; combine pairwise
    for (int s = CT_NB; s < r && !series; s *= 2) {
        const int npairs = (r + 2 * s - 1) / (2 * s);
        // step 1: T = B * Ai, kept transposed in the (unused, zero) mirror block above the diagonal
        run_list([&]() {
            for (int pr = 0; pr < npairs; ++pr) {
                const int p = pr * 2 * s, sc = min(s, r - p - s);
                if (sc <= 0) continue;
                for (int i0 = 0; i0 < sc; i0 += 64)
                    for (int c0 = 0; c0 < s; c0 += 64)
                        add_task(W + (size_t)(p + c0) * r + (p + s + i0), 1, r,   // T(i,k) at W[p+k][p+s+i]
                                 W + (size_t)(p + s + i0) * r + p, r,             // B(i,q)
                                 W + (size_t)p * r + (p + c0), r, 1,              // Ai(q,k)
                                 min(64, sc - i0), min(64, s - c0), c0, s, 1.f, 0.f, false, 0, 0);
            }
        });
        // step 2: B <- -Ci * T
        run_list([&]() {
            for (int pr = 0; pr < npairs; ++pr) {
                const int p = pr * 2 * s, sc = min(s, r - p - s);
                if (sc <= 0) continue;
                for (int i0 = 0; i0 < sc; i0 += 64)
                    for (int c0 = 0; c0 < s; c0 += 64)
                        add_task(W + (size_t)(p + s + i0) * r + (p + c0), r, 1,   // Bnew(i,k)
                                 W + (size_t)(p + s + i0) * r + (p + s), r,       // Ci(i,q)
                                 W + (size_t)(p + c0) * r + (p + s), 1, r,        // T(q,k) at W[p+k][p+s+q]
                                 min(64, sc - i0), min(64, s - c0), 0, min(sc, i0 + 64), -1.f, 0.f, false, 0, 0);
            }
        });
        // clear the mirror blocks again
        for (int pr = 0; pr < npairs; ++pr) {
            const int p = pr * 2 * s, sc = min(s, r - p - s);
            if (sc <= 0) continue;
            for (int e = tid + crank * CT_THREADS; e < s * sc; e += CT_THREADS * nshare) {
                const int k = e / sc, i = e - k * sc;
                W[(p + k) * r + (p + s + i)] = 0.f;
            }
        }
        phase_sync();
    }

    // ---- split image of (L^{-1})^T for the tensor-core apply product ---------------------------
    // Image row k, column j holds L^{-1}(j, k): the apply product Y L^{-T} then reads its N-side
    // operand MN-major (depth along image rows) in 256-column instructions.
    if (a.img.off >= 0) {
        unsigned char* __restrict__ scr = reinterpret_cast<unsigned char*>(w.scratch);
        const float* Wr = W;
        const int chunks = a.img.panels * a.img.rows_pad * 8;
        for (int q0 = tid + crank * 4 * CT_THREADS; q0 < chunks; q0 += 4 * CT_THREADS * nshare) {
            // consecutive threads take consecutive image rows (consecutive k: contiguous in W);
            // four chunks (32 loads) in flight per thread
            float v[4][8];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int q = q0 + u * CT_THREADS;
                const int row = q % a.img.rows_pad, c = (q / a.img.rows_pad) % 8, panel = q / (8 * a.img.rows_pad);
                const int col = panel * 64 + c * 8;
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    v[u][i] = (q < chunks && row < r && col + i < r) ? ct_ld<MULTI>(Wr + (col + i) * r + row) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int q = q0 + u * CT_THREADS;
                if (q >= chunks) break;
                const int row = q % a.img.rows_pad, c = (q / a.img.rows_pad) % 8, panel = q / (8 * a.img.rows_pad);
                uint4 t0, t1;
                split8(v[u], t0, t1);
                const int o = img_chunk_offset(row, c);
                *reinterpret_cast<uint4*>(scr + img_row_offset(a.img, 0, panel, row) + o) = t0;
                *reinterpret_cast<uint4*>(scr + img_row_offset(a.img, 1, panel, row) + o) = t1;
            }
        }
    }
}

}  // namespace od
