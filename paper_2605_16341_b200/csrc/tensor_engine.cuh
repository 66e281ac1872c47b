// Tensor-core engine: tcgen05 (5th-generation tensor core) kernels with accumulators in tensor
// memory.  Every matrix product of the step is a sum of bf16 products with fp32 accumulation:
// an fp32 operand v is split as v = t0 + t1 (+ ...) with t0 = bf16(v), t1 = bf16(v - t0), and
// "3 passes" means t0*u0 + t0*u1 + t1*u0 (relative error about 2^-16), "1 pass" t0*u0.
//
// Operand staging.  Small operands (Q, P, R, L^{-1} and the QR intermediates) are first written by
// pack kernels as ready-made shared-memory images (128-row x 64-deep bf16 tiles, 128-byte rows,
// 16-byte chunks XOR-swizzled by row) and fetched with bulk asynchronous copies (TMA engine,
// cp.async.bulk) that complete on an mbarrier.  The big operand B = M + G (Alg. 1 line 1) is never
// stored: transform warps read M and G from HBM, add, split and write the image directly.
#pragma once
#include "common.cuh"
#include "profile.cuh"
#include "simt_kernels.cuh"

namespace od {
namespace tc {

constexpr int BM = 128;              // tile rows (MMA M)
constexpr int BK = 64;               // depth of one stage: 64 bf16 = one 128-byte swizzled row
constexpr int TILE_BYTES = 128 * 128;   // one 128 x 64 bf16 image
constexpr int STAGES = 2;
constexpr int NUM_EPI_WARPS = 4;
constexpr int NUM_XF_WARPS = 8;
constexpr int THREADS_PACKED = 32 * (2 + NUM_EPI_WARPS);
constexpr int THREADS_BUF = 32 * (2 + NUM_EPI_WARPS + NUM_XF_WARPS);
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // about two seconds

enum AMode : int { A_PACKED = 0, A_BUF_ROW = 1, A_BUF_COL = 2 };
enum EpiMode : int { EPI_STORE = 0, EPI_K5 = 1 };

// A packed operand inside a matrix's scratch area.  Tile (kb, term, row_tile) lives at
// off + ((kb * terms + term) * row_tiles + row_tile) * TILE_BYTES.
struct PackRef {
    int64_t off;
    int32_t row_tiles, terms, kblocks, pad;
};

struct GemmArgs {
    int32_t Mrows, Ncols, Kdim, BN;
    int32_t m_tiles, n_tiles, k_blocks, tri;
    int32_t passes, passes2, total_tiles, g_bf16;
    int32_t x_bf16, pad0;
    int64_t ld;
    PackRef a, b, b2;
    float ef_a, ef_b, wc, wd;
    EpStore st;
};

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after WAIT_LIMIT_CYCLES or as soon as another role of the CTA gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    int spins = 0;
    while (!mbar_try_wait(bar, parity)) {
        if ((++spins & 63) == 0) {
            if (*abort_flag) return false;
            if (clock64() - t0 > WAIT_LIMIT_CYCLES) { *abort_flag = 1; return false; }
        }
    }
    return true;
}
__device__ __forceinline__ void bulk_copy_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_async_smem() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]^T, bf16 inputs, fp32 accumulation; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                          uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// mbarrier arrives once every MMA issued so far by this thread has completed
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle.  K-major: rows of 128 bytes, 8-row groups
// 1024 bytes apart (stride offset), leading offset unused.  MN-major: lbo = distance between
// 64-element groups along M/N, sbo = distance between 8-deep groups along K.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;     // descriptor version of this architecture
    d |= (uint64_t)2 << 61;     // 128-byte swizzle
    return d;
}
// Instruction descriptor: fp32 accumulate, bf16 A and B, M = 128, N = n; a_mn = 1 for an MN-major A.
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, uint32_t a_mn) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (a_mn << 15) | ((n >> 3) << 17) | ((uint32_t)(BM >> 4) << 24);
}

// ---- bf16 splitting -----------------------------------------------------------------------------
// two fp32 -> packed bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float bf16lo_to_f32(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t p) { return __uint_as_float(p & 0xFFFF0000u); }

// 8 fp32 values -> chunk of term 0 and chunk of term 1 (each 8 bf16 = 16 bytes)
__device__ __forceinline__ void split8(const float (&v)[8], uint4& t0, uint4& t1) {
    uint32_t a[4], b[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        a[e] = pack_bf16x2(v[2 * e], v[2 * e + 1]);
        float r0 = v[2 * e] - bf16lo_to_f32(a[e]);
        float r1 = v[2 * e + 1] - bf16hi_to_f32(a[e]);
        b[e] = pack_bf16x2(r0, r1);
    }
    t0 = make_uint4(a[0], a[1], a[2], a[3]);
    t1 = make_uint4(b[0], b[1], b[2], b[3]);
}

__device__ __forceinline__ void load8(const void* base, int64_t idx, int is_bf16, float (&v)[8]) {
    if (is_bf16) {
        uint4 u = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(base) + idx);
        v[0] = bf16lo_to_f32(u.x); v[1] = bf16hi_to_f32(u.x);
        v[2] = bf16lo_to_f32(u.y); v[3] = bf16hi_to_f32(u.y);
        v[4] = bf16lo_to_f32(u.z); v[5] = bf16hi_to_f32(u.z);
        v[6] = bf16lo_to_f32(u.w); v[7] = bf16hi_to_f32(u.w);
    } else {
        const float4* p = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(base) + idx);
        float4 x = p[0], y = p[1];
        v[0] = x.x; v[1] = x.y; v[2] = x.z; v[3] = x.w;
        v[4] = y.x; v[5] = y.y; v[6] = y.z; v[7] = y.w;
    }
}

// ------------------------------------------------------------------------------------------
// Pack kernel: fp32 matrix S (rows_s x cols_s, row-major, leading dimension cols_s) -> packed operand.
//   trans = 0: operand row = S row,    depth = S column
//   trans = 1: operand row = S column, depth = S row
// One CTA per 128 x 64 tile (all terms), 256 threads.
// ------------------------------------------------------------------------------------------
struct PackArgs {
    Sel src;
    int32_t rows_s, cols_s;
    int32_t trans, only_if_shifted, shift_bit, colsq_ld;
    int64_t colsq_off;   // >= 0 (trans only): also write fp32 column sums of squares of this 64-row block
    PackRef dst;
};

__global__ void __launch_bounds__(256)
pack_kernel(const __grid_constant__ Batch batch, PackArgs a) {
    const MatWork& w = batch.w[blockIdx.z];
    const int st = *w.status;
    if (st & ST_FAILED) return;
    if (a.only_if_shifted && !(st & a.shift_bit)) return;
    const float* S = pick(w, a.src);
    const int rt = blockIdx.y, kb = blockIdx.x;
    unsigned char* out0 = reinterpret_cast<unsigned char*>(w.scratch + a.dst.off) +
                          ((int64_t)(kb * a.dst.terms + 0) * a.dst.row_tiles + rt) * TILE_BYTES;
    unsigned char* out1 = out0 + (int64_t)a.dst.row_tiles * TILE_BYTES;
    const int tid = threadIdx.x;
    if (!a.trans) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int q = tid + 256 * e;
            const int rho = q / 8, c = q % 8;
            const int64_t gr = (int64_t)rt * 128 + rho, gk = (int64_t)kb * 64 + c * 8;
            float v[8];
            if (gr < a.rows_s && gk < a.cols_s) {   // cols_s % 8 == 0
                load8(S, gr * a.cols_s + gk, 0, v);
            } else {
#pragma unroll
                for (int i = 0; i < 8; ++i) v[i] = 0.f;
            }
            uint4 t0, t1;
            split8(v, t0, t1);
            const int o = rho * 128 + ((c ^ (rho & 7)) << 4);
            *reinterpret_cast<uint4*>(out0 + o) = t0;
            if (a.dst.terms > 1) *reinterpret_cast<uint4*>(out1 + o) = t1;
        }
    } else {
        __shared__ float tile[64][129];
        // S rows kb*64 .. +63 (depth), S cols rt*128 .. +127 (operand rows)
        for (int e = tid; e < 64 * 32; e += 256) {
            const int kk = e / 32, c4 = e % 32;
            const int64_t gk = (int64_t)kb * 64 + kk, gc = (int64_t)rt * 128 + c4 * 4;
            float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
            if (gk < a.rows_s && gc < a.cols_s)     // cols_s % 4 == 0
                x = *reinterpret_cast<const float4*>(S + gk * a.cols_s + gc);
            tile[kk][c4 * 4 + 0] = x.x; tile[kk][c4 * 4 + 1] = x.y;
            tile[kk][c4 * 4 + 2] = x.z; tile[kk][c4 * 4 + 3] = x.w;
        }
        __syncthreads();
        if (a.colsq_off >= 0 && tid < 128 && rt * 128 + tid < a.cols_s) {
            float s = 0.f;
#pragma unroll 8
            for (int kk = 0; kk < 64; ++kk) s = fmaf(tile[kk][tid], tile[kk][tid], s);
            reinterpret_cast<float*>(w.scratch + a.colsq_off)[(int64_t)kb * a.colsq_ld + rt * 128 + tid] = s;
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int q = tid + 256 * e;
            const int rho = q % 128, c = q / 128;
            float v[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = tile[c * 8 + i][rho];
            uint4 t0, t1;
            split8(v, t0, t1);
            const int o = rho * 128 + ((c ^ (rho & 7)) << 4);
            *reinterpret_cast<uint4*>(out0 + o) = t0;
            if (a.dst.terms > 1) *reinterpret_cast<uint4*>(out1 + o) = t1;
        }
    }
}

// ------------------------------------------------------------------------------------------
// The GEMM kernel.  Persistent CTAs walk the tile list t = blockIdx.x, blockIdx.x + gridDim.x, ...
//   warp 0      bulk-copy producer (packed operands)
//   warp 1      MMA issuer, owns the tensor-memory allocation
//   warps 2-5   epilogue (tensor memory -> registers -> global)
//   warps 6-13  transform warps (A_BUF_* only): form B = M + G, split, write the A image
// Accumulators are double-buffered in tensor memory so that the epilogue of tile i overlaps the
// main loop of tile i+1.
// ------------------------------------------------------------------------------------------
struct TileCoord { int b, mt, nt, kb_end; bool active; };

template <int EPI>
__device__ __forceinline__ TileCoord decode_tile(const Batch& batch, const GemmArgs& g, int t) {
    TileCoord c;
    const int per = g.m_tiles * g.n_tiles;
    c.b = t / per;
    const int rem = t - c.b * per;
    c.mt = rem / g.n_tiles;
    c.nt = rem - c.mt * g.n_tiles;
    c.kb_end = g.k_blocks;
    if (g.tri) c.kb_end = min(g.k_blocks, ((c.nt + 1) * g.BN + BK - 1) / BK);
    const MatWork& w = batch.w[c.b];
    if (EPI == EPI_STORE) c.active = g.st.active(w);
    else c.active = !(*w.status & ST_FAILED);
    return c;
}

template <int AMODE, int EPI>
__global__ void __launch_bounds__(AMODE == A_PACKED ? THREADS_PACKED : THREADS_BUF, 1)
umma_gemm_kernel(const __grid_constant__ Batch batch, const __grid_constant__ GemmArgs g) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    unsigned char* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);
    const int BN = g.BN;
    const uint32_t b_term_bytes = (uint32_t)BN * 128u;
    const uint32_t nb_ops = (EPI == EPI_K5) ? 2u : 1u;
    const uint32_t stage_bytes = 2u * TILE_BYTES + 2u * b_term_bytes * nb_ops;
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * stage_bytes);
    const uint32_t full0 = smem_u32(bars), empty0 = full0 + 8 * STAGES;
    const uint32_t tfull0 = empty0 + 8 * STAGES, tempty0 = tfull0 + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t acc_cols = (EPI == EPI_K5) ? 2u * BN : (uint32_t)BN;
    uint32_t alloc_cols = 32;
    while (alloc_cols < 2 * acc_cols) alloc_cols *= 2;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full0 + 8 * s, AMODE == A_PACKED ? 1 : 1 + NUM_XF_WARPS);
            mbar_init(empty0 + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull0 + 8 * a, 1);
            mbar_init(tempty0 + 8 * a, NUM_EPI_WARPS);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) tmem_alloc(smem_u32(tmem_slot), alloc_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    const int a_terms = (g.passes == 3 || (EPI == EPI_K5 && g.passes2 == 3)) ? 2 : 1;
    const int b_terms = g.passes == 3 ? 2 : 1;
    const int b2_terms = g.passes2 == 3 ? 2 : 1;

    if (warp == 0) {
        // ---------------- producer ----------------
        if (lane == 0) {
            int stage = 0; uint32_t phase = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < g.total_tiles && ok; t += gridDim.x) {
                const TileCoord c = decode_tile<EPI>(batch, g, t);
                if (!c.active) continue;
                const unsigned char* scr = reinterpret_cast<const unsigned char*>(batch.w[c.b].scratch);
                const int n0 = c.nt * BN;
                const int b_rt = n0 / 128;
                const uint32_t b_row_off = (uint32_t)(n0 % 128) * 128u;
                for (int kb = 0; kb < c.kb_end; ++kb) {
                    if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
                    unsigned char* sbase = smem + stage * stage_bytes;
                    const uint32_t fb = full0 + 8 * stage;
                    uint32_t bytes = b_terms * b_term_bytes;
                    if (AMODE == A_PACKED) bytes += a_terms * TILE_BYTES;
                    if (EPI == EPI_K5) bytes += b2_terms * b_term_bytes;
                    mbar_arrive_expect_tx(fb, bytes);
                    if (AMODE == A_PACKED) {
                        for (int term = 0; term < a_terms; ++term) {
                            const unsigned char* src = scr + g.a.off +
                                ((int64_t)(kb * g.a.terms + term) * g.a.row_tiles + c.mt) * TILE_BYTES;
                            bulk_copy_g2s(smem_u32(sbase + term * TILE_BYTES), src, TILE_BYTES, fb);
                        }
                    }
                    for (int term = 0; term < b_terms; ++term) {
                        const unsigned char* src = scr + g.b.off +
                            ((int64_t)(kb * g.b.terms + term) * g.b.row_tiles + b_rt) * TILE_BYTES + b_row_off;
                        bulk_copy_g2s(smem_u32(sbase + 2 * TILE_BYTES + term * b_term_bytes), src, b_term_bytes, fb);
                    }
                    if (EPI == EPI_K5) {
                        for (int term = 0; term < b2_terms; ++term) {
                            const unsigned char* src = scr + g.b2.off +
                                ((int64_t)(kb * g.b2.terms + term) * g.b2.row_tiles + b_rt) * TILE_BYTES + b_row_off;
                            bulk_copy_g2s(smem_u32(sbase + 2 * TILE_BYTES + (2 + term) * b_term_bytes), src,
                                          b_term_bytes, fb);
                        }
                    }
                    if (++stage == STAGES) { stage = 0; phase ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        int stage = 0; uint32_t phase = 0;
        int acc = 0; uint32_t acc_phase = 0;
        bool ok = true;
        const uint32_t idesc = instr_desc((uint32_t)BN, AMODE == A_BUF_COL ? 1u : 0u);
        for (int t = blockIdx.x; t < g.total_tiles && ok; t += gridDim.x) {
            const TileCoord c = decode_tile<EPI>(batch, g, t);
            if (!c.active) continue;
            if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const uint32_t d1 = tmem_base + acc * acc_cols;
            const uint32_t d2 = d1 + BN;
            for (int kb = 0; kb < c.kb_end; ++kb) {
                if (!mbar_wait(full0 + 8 * stage, phase, abort_flag)) { ok = false; break; }
                tc_fence_after();
                if (lane == 0) {
                    const uint32_t sa = smem_u32(smem + stage * stage_bytes);
                    const uint32_t sb = sa + 2 * TILE_BYTES;
#pragma unroll
                    for (int j = 0; j < BK / 16; ++j) {
                        uint64_t a0, a1;
                        if (AMODE == A_BUF_COL) {
                            // MN-major A: 64-column groups 8192 bytes apart, 8-deep groups 1024 bytes apart
                            a0 = smem_desc(sa + j * 2048, 8192, 1024);
                            a1 = smem_desc(sa + TILE_BYTES + j * 2048, 8192, 1024);
                        } else {
                            a0 = smem_desc(sa + j * 32, 16, 1024);
                            a1 = smem_desc(sa + TILE_BYTES + j * 32, 16, 1024);
                        }
                        const uint64_t b0 = smem_desc(sb + j * 32, 16, 1024);
                        const uint64_t b1 = smem_desc(sb + b_term_bytes + j * 32, 16, 1024);
                        const uint32_t first = (kb > 0 || j > 0) ? 1u : 0u;
                        umma_bf16(d1, a0, b0, idesc, first);
                        if (g.passes == 3) {
                            umma_bf16(d1, a0, b1, idesc, 1u);
                            umma_bf16(d1, a1, b0, idesc, 1u);
                        }
                        if (EPI == EPI_K5) {
                            const uint64_t c0 = smem_desc(sb + 2 * b_term_bytes + j * 32, 16, 1024);
                            const uint64_t c1 = smem_desc(sb + 3 * b_term_bytes + j * 32, 16, 1024);
                            umma_bf16(d2, a0, c0, idesc, first);
                            if (g.passes2 == 3) {
                                umma_bf16(d2, a0, c1, idesc, 1u);
                                umma_bf16(d2, a1, c0, idesc, 1u);
                            }
                        }
                    }
                    umma_commit(empty0 + 8 * stage);
                }
                __syncwarp();
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
            if (!ok) break;
            if (lane == 0) umma_commit(tfull0 + 8 * acc);
            __syncwarp();
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
    } else if (warp < 2 + NUM_EPI_WARPS) {
        // ---------------- epilogue ----------------
        int acc = 0; uint32_t acc_phase = 0;
        bool ok = true;
        const int quarter = warp % 4;                    // tensor-memory lanes 32*quarter .. +31
        for (int t = blockIdx.x; t < g.total_tiles && ok; t += gridDim.x) {
            const TileCoord c = decode_tile<EPI>(batch, g, t);
            if (!c.active) continue;
            if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
            tc_fence_after();
            const MatWork& w = batch.w[c.b];
            const uint32_t taddr = tmem_base + acc * acc_cols + ((uint32_t)(quarter * 32) << 16);
            const int64_t gi = (int64_t)c.mt * BM + quarter * 32 + lane;
            const int n0 = c.nt * BN;
            if (EPI == EPI_STORE) {
                const int stw = *w.status;
                float* C = pick(w, (g.st.shift_bit && (stw & g.st.shift_bit)) ? g.st.dst_if_shifted : g.st.dst);
                for (int cc = 0; cc < BN; cc += 16) {
                    uint32_t v[16];
                    tmem_ld16(taddr + cc, v);
                    tmem_ld_wait();
                    if (gi < g.Mrows) {
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int gj = n0 + cc + 4 * u;
                            if (gj < g.Ncols)
                                *reinterpret_cast<uint4*>(C + gi * g.st.ld + gj) =
                                    make_uint4(v[4 * u], v[4 * u + 1], v[4 * u + 2], v[4 * u + 3]);
                        }
                    }
                }
            } else {
                for (int cc = 0; cc < BN; cc += 16) {
                    uint32_t v1[16], v2[16];
                    tmem_ld16(taddr + cc, v1);
                    tmem_ld16(taddr + BN + cc, v2);
                    tmem_ld_wait();
                    if (gi < g.Mrows) {
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const int gj = n0 + cc + 8 * h;
                            if (gj < g.Ncols) {     // Ncols % 8 == 0
                                const int64_t idx = gi * g.ld + gj;
                                float mv[8], gv[8], xv[8];
                                load8(w.M, idx, 0, mv);
                                load8(w.G, idx, g.g_bf16, gv);
                                load8(w.X, idx, g.x_bf16, xv);
                                float mo[8], xo[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e) {
                                    const float bval = mv[e] + gv[e];
                                    mo[e] = g.ef_a * bval - g.ef_b * __uint_as_float(v1[8 * h + e]);
                                    xo[e] = g.wc * xv[e] - g.wd * __uint_as_float(v2[8 * h + e]);
                                }
                                float4* mp = reinterpret_cast<float4*>(w.M + idx);
                                mp[0] = make_float4(mo[0], mo[1], mo[2], mo[3]);
                                mp[1] = make_float4(mo[4], mo[5], mo[6], mo[7]);
                                if (g.x_bf16) {
                                    uint4 xp = make_uint4(pack_bf16x2(xo[0], xo[1]), pack_bf16x2(xo[2], xo[3]),
                                                          pack_bf16x2(xo[4], xo[5]), pack_bf16x2(xo[6], xo[7]));
                                    *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(w.X) + idx) = xp;
                                } else {
                                    float4* xp = reinterpret_cast<float4*>(reinterpret_cast<float*>(w.X) + idx);
                                    xp[0] = make_float4(xo[0], xo[1], xo[2], xo[3]);
                                    xp[1] = make_float4(xo[4], xo[5], xo[6], xo[7]);
                                }
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(tempty0 + 8 * acc);
            if (++acc == 2) { acc = 0; acc_phase ^= 1; }
        }
    } else if (AMODE != A_PACKED) {
        // ---------------- transform warps: A image of B = M + G ----------------
        const int xt = threadIdx.x - 32 * (2 + NUM_EPI_WARPS);     // 0 .. 255
        int stage = 0; uint32_t phase = 0;
        bool ok = true;
        for (int t = blockIdx.x; t < g.total_tiles && ok; t += gridDim.x) {
            const TileCoord c = decode_tile<EPI>(batch, g, t);
            if (!c.active) continue;
            const MatWork& w = batch.w[c.b];
            const int64_t ld = g.ld;
            // chunk coordinates of this thread (4 chunks per stage)
            int64_t src_idx[4]; bool row_ok[4]; int kofs[4]; uint32_t dst_off[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int q = xt + 256 * e;
                if (AMODE == A_BUF_ROW) {
                    // operand row = B row, depth = B column: chunk (rho, c) = B[i0+rho][k0+8c .. +7]
                    const int rho = q / 8, ch = q % 8;
                    const int64_t gr = (int64_t)c.mt * BM + rho;
                    row_ok[e] = gr < g.Mrows;
                    src_idx[e] = gr * ld + ch * 8;           // + k0
                    kofs[e] = ch * 8;
                    dst_off[e] = rho * 128 + ((ch ^ (rho & 7)) << 4);
                } else {
                    // operand row = B column, depth = B row (MN-major image):
                    // chunk (k, cj) = B[k0+k][j0+8cj .. +7]
                    const int k = q / 16, cj = q % 16;
                    const int64_t gc = (int64_t)c.mt * BM + cj * 8;
                    row_ok[e] = gc < g.Mrows;                // Mrows = number of B columns (n), n % 8 == 0
                    src_idx[e] = (int64_t)k * ld + gc;       // + k0 * ld
                    kofs[e] = k;
                    dst_off[e] = (cj / 8) * 8192 + (k / 8) * 1024 + (k % 8) * 128 + (((cj % 8) ^ (k % 8)) << 4);
                }
            }
            float mv[4][8], gv[4][8];
            auto fetch = [&](int kb) {
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int64_t k0 = (int64_t)kb * BK;
                    bool okk = row_ok[e] && (k0 + kofs[e] < g.Kdim);
                    if (okk) {
                        const int64_t idx = src_idx[e] + (AMODE == A_BUF_ROW ? k0 : k0 * ld);
                        load8(w.M, idx, 0, mv[e]);
                        load8(w.G, idx, g.g_bf16, gv[e]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) { mv[e][i] = 0.f; gv[e][i] = 0.f; }
                    }
                }
            };
            fetch(0);
            for (int kb = 0; kb < c.kb_end; ++kb) {
                uint4 t0[4], t1[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float v[8];
#pragma unroll
                    for (int i = 0; i < 8; ++i) v[i] = mv[e][i] + gv[e][i];
                    split8(v, t0[e], t1[e]);
                }
                if (kb + 1 < c.kb_end) fetch(kb + 1);
                if (!mbar_wait(empty0 + 8 * stage, phase ^ 1, abort_flag)) { ok = false; break; }
                unsigned char* sa = smem + stage * stage_bytes;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    *reinterpret_cast<uint4*>(sa + dst_off[e]) = t0[e];
                    *reinterpret_cast<uint4*>(sa + TILE_BYTES + dst_off[e]) = t1[e];
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(full0 + 8 * stage);
                if (++stage == STAGES) { stage = 0; phase ^= 1; }
            }
        }
    }

    // ---------------- teardown ----------------
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (*abort_flag && threadIdx.x == 0) {
        for (int b = 0; b < batch.count; ++b) atomicOr(batch.w[b].status, ST_WAIT);
    }
    if (warp == 1) tmem_dealloc(tmem_base, alloc_cols);
}

// smem bytes a launch asks for: the stages, barriers, alignment slack, and enough to keep the number
// of resident CTAs per SM times their tensor-memory columns within the 512 columns of an SM.
inline size_t gemm_smem_bytes(int BN, bool k5) {
    const size_t stage = 2 * (size_t)TILE_BYTES + 2 * (size_t)BN * 128 * (k5 ? 2 : 1);
    size_t need = STAGES * stage + 256 + 1024;
    const size_t acc = (size_t)(k5 ? 2 * BN : BN);
    size_t cols = 32;
    while (cols < 2 * acc) cols *= 2;
    const size_t max_resident = 512 / cols;
    const size_t min_smem = (227 * 1024) / (max_resident + 1) + 1024;
    return std::max(need, max_resident >= 8 ? need : min_smem);
}

}  // namespace tc

// ------------------------------------------------------------------------------------------
// Host side of the engine
// ------------------------------------------------------------------------------------------
struct TensorScratch {
    int64_t q_t, src_t, src_n, linv, p_t, p_n, r_n, q_n;   // byte offsets of the packed operands
    int64_t colsq;                                          // fp32 [kblocks][r] column sums of squares
};

inline bool tensor_engine_supports(int64_t m, int64_t n, int32_t r) {
    return r % 16 == 0 && n % 8 == 0 && m >= 1;
}

inline int64_t pack_bytes(int64_t rows, int64_t depth, int terms) {
    return ((rows + 127) / 128) * ((depth + 63) / 64) * terms * (int64_t)tc::TILE_BYTES;
}

inline size_t tensor_scratch_layout(int64_t m, int64_t n, int32_t r, size_t off, TensorScratch* ts) {
    const int64_t kmax = std::max(m, n);
    auto take = [&](int64_t bytes) { int64_t o = (int64_t)off; off += (size_t)((bytes + 1023) / 1024 * 1024); return o; };
    off = (off + 1023) / 1024 * 1024;
    ts->q_t = take(pack_bytes(r, n, 2));
    ts->src_t = take(pack_bytes(r, kmax, 2));
    ts->src_n = take(pack_bytes(kmax, r, 2));
    ts->linv = take(pack_bytes(r, r, 2));
    ts->p_t = take(pack_bytes(r, m, 2));
    ts->p_n = take(pack_bytes(m, r, 2));
    ts->r_n = take(pack_bytes(n, r, 2));
    ts->q_n = take(pack_bytes(n, r, 2));
    ts->colsq = take(((kmax + 63) / 64) * (int64_t)r * 4);
    return off;
}

inline int tensor_bn(int64_t ncols) {
    int bn = 16;
    while (bn < 256 && bn < ncols) bn *= 2;
    return bn;
}

inline cudaError_t tensor_engine_set_attributes() {
    const int max_smem = 227 * 1024;
    cudaError_t e;
#define OD_SET(k) \
    if ((e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem)) != cudaSuccess) return e;
    OD_SET((tc::umma_gemm_kernel<tc::A_PACKED, tc::EPI_STORE>))
    OD_SET((tc::umma_gemm_kernel<tc::A_PACKED, tc::EPI_K5>))
    OD_SET((tc::umma_gemm_kernel<tc::A_BUF_ROW, tc::EPI_STORE>))
    OD_SET((tc::umma_gemm_kernel<tc::A_BUF_COL, tc::EPI_STORE>))
#undef OD_SET
    return cudaSuccess;
}

inline int sm_count() {
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

inline tc::PackRef make_pack(int64_t off, int64_t rows, int64_t depth, int terms) {
    tc::PackRef p;
    p.off = off;
    p.row_tiles = (int32_t)((rows + 127) / 128);
    p.terms = terms;
    p.kblocks = (int32_t)((depth + 63) / 64);
    p.pad = 0;
    return p;
}

// pack S (rows_s x cols_s) either as (operand rows = S rows) or transposed
inline void launch_pack(const Batch& b, Sel src, int64_t rows_s, int64_t cols_s, int trans, tc::PackRef dst,
                        int shift_bit_only, cudaStream_t st, int64_t colsq_off = -1) {
    tc::PackArgs a{};
    a.colsq_off = colsq_off; a.colsq_ld = (int32_t)cols_s;
    a.src = src; a.rows_s = (int32_t)rows_s; a.cols_s = (int32_t)cols_s; a.trans = trans;
    a.only_if_shifted = shift_bit_only ? 1 : 0; a.shift_bit = shift_bit_only; a.dst = dst;
    dim3 grid((unsigned)dst.kblocks, (unsigned)dst.row_tiles, (unsigned)b.count);
    prof::Scope scope(prof::S_PACK, st);
    tc::pack_kernel<<<grid, 256, 0, st>>>(b, a);
}

template <int AMODE, int EPI>
inline void launch_gemm(const Batch& b, tc::GemmArgs g, int stage, cudaStream_t st) {
    g.m_tiles = (g.Mrows + tc::BM - 1) / tc::BM;
    g.n_tiles = (g.Ncols + g.BN - 1) / g.BN;
    g.k_blocks = (g.Kdim + tc::BK - 1) / tc::BK;
    g.total_tiles = b.count * g.m_tiles * g.n_tiles;
    const size_t smem = tc::gemm_smem_bytes(g.BN, EPI == tc::EPI_K5);
    const int per_sm = std::max<int>(1, (int)((227 * 1024) / smem));
    const int grid = std::min(g.total_tiles, sm_count() * per_sm);
    const int threads = AMODE == tc::A_PACKED ? tc::THREADS_PACKED : tc::THREADS_BUF;
    prof::Scope scope(stage, st);
    tc::umma_gemm_kernel<AMODE, EPI><<<grid, threads, smem, st>>>(b, g);
}

// Y = (M + G) Q_prev  -> P slot                                   (Alg. 1 lines 1-2)
inline void tensor_k1(int64_t m, int64_t n, int r, int g_bf16, int passes, const Batch& b, const TensorScratch& ts,
                      cudaStream_t st) {
    const int terms = passes == 3 ? 2 : 1;
    tc::PackRef qt = make_pack(ts.q_t, r, n, terms);
    launch_pack(b, Sel{W_Q, 0, 0}, n, r, 1, qt, 0, st);
    tc::GemmArgs g{};
    g.Mrows = (int32_t)m; g.Ncols = r; g.Kdim = (int32_t)n; g.BN = tensor_bn(r);
    g.passes = passes; g.passes2 = 1; g.g_bf16 = g_bf16; g.ld = n; g.b = qt;
    g.st = EpStore{Sel{W_P, 0, 0}, Sel{W_P, 0, 0}, 0, 0, r, 0};
    launch_gemm<tc::A_BUF_ROW, tc::EPI_STORE>(b, g, prof::S_K1, st);
}

// R = (M + G)^T P  -> R slot                                      (Alg. 1 line 3)
inline void tensor_k3(int64_t m, int64_t n, int r, int g_bf16, int passes, const Batch& b, const TensorScratch& ts,
                      cudaStream_t st) {
    const int terms = passes == 3 ? 2 : 1;
    tc::PackRef pt = make_pack(ts.p_t, r, m, terms);
    launch_pack(b, Sel{W_P, 0, 0}, m, r, 1, pt, 0, st);
    tc::GemmArgs g{};
    g.Mrows = (int32_t)n; g.Ncols = r; g.Kdim = (int32_t)m; g.BN = tensor_bn(r);
    g.passes = passes; g.passes2 = 1; g.g_bf16 = g_bf16; g.ld = n; g.b = pt;
    g.st = EpStore{Sel{W_R, 0, 0}, Sel{W_R, 0, 0}, 0, 0, r, 0};
    launch_gemm<tc::A_BUF_COL, tc::EPI_STORE>(b, g, prof::S_K3, st);
}

// Gram = src^T src (src: rows x r)
inline void tensor_gram(int64_t, int64_t, int r, int passes, const Batch& b, const TensorScratch& ts, Sel src,
                        int64_t rows, Sel gram, int only_shift_bit, cudaStream_t st) {
    const int terms = passes == 3 ? 2 : 1;
    tc::PackRef sp = make_pack(ts.src_t, r, rows, terms);
    launch_pack(b, src, rows, r, 1, sp, only_shift_bit, st, ts.colsq);
    tc::GemmArgs g{};
    g.Mrows = r; g.Ncols = r; g.Kdim = (int32_t)rows; g.BN = tensor_bn(r);
    g.passes = passes; g.passes2 = 1; g.a = sp; g.b = sp;
    g.st = EpStore{gram, gram, only_shift_bit, 1, r, only_shift_bit ? 1 : 0};
    launch_gemm<tc::A_PACKED, tc::EPI_STORE>(b, g, prof::S_GRAM, st);
}

// dst = src * L^{-T}  (src: rows x r, L^{-1} lower triangular r x r)
inline void tensor_apply(int64_t, int64_t, int r, int passes, const Batch& b, const TensorScratch& ts, Sel src,
                         int64_t rows, Sel linv, EpStore ep, cudaStream_t st) {
    const int terms = passes == 3 ? 2 : 1;
    tc::PackRef sp = make_pack(ts.src_n, rows, r, terms);
    tc::PackRef lp = make_pack(ts.linv, r, r, terms);
    const int only_bit = ep.only_if_shifted ? ep.shift_bit : 0;
    launch_pack(b, src, rows, r, 0, sp, only_bit, st);
    launch_pack(b, linv, r, r, 0, lp, only_bit, st);
    tc::GemmArgs g{};
    g.Mrows = (int32_t)rows; g.Ncols = r; g.Kdim = r; g.BN = tensor_bn(r);
    g.passes = passes; g.passes2 = 1; g.a = sp; g.b = lp; g.tri = 1;
    g.st = ep;
    launch_gemm<tc::A_PACKED, tc::EPI_STORE>(b, g, prof::S_APPLY, st);
}

// M <- a (M + G) - b P R^T ;  X <- c X - d P Q^T                  (Alg. 1 lines 5-7)
inline void tensor_k5(int64_t m, int64_t n, int r, int g_bf16, int x_bf16, int passes_m, int passes_x, float ef_a,
                      float ef_b, float wc, float wd, const Batch& b, const TensorScratch& ts, cudaStream_t st) {
    const int pterms = (passes_m == 3 || passes_x == 3) ? 2 : 1;
    tc::PackRef pp = make_pack(ts.p_n, m, r, pterms);
    tc::PackRef rp = make_pack(ts.r_n, n, r, passes_m == 3 ? 2 : 1);
    tc::PackRef qp = make_pack(ts.q_n, n, r, passes_x == 3 ? 2 : 1);
    launch_pack(b, Sel{W_P, 0, 0}, m, r, 0, pp, 0, st);
    launch_pack(b, Sel{W_R, 0, 0}, n, r, 0, rp, 0, st);
    launch_pack(b, Sel{W_Q, 0, 0}, n, r, 0, qp, 0, st);
    tc::GemmArgs g{};
    g.Mrows = (int32_t)m; g.Ncols = (int32_t)n; g.Kdim = r; g.BN = 128;
    g.passes = passes_m; g.passes2 = passes_x; g.g_bf16 = g_bf16; g.x_bf16 = x_bf16; g.ld = n;
    g.a = pp; g.b = rp; g.b2 = qp;
    g.ef_a = ef_a; g.ef_b = ef_b; g.wc = wc; g.wd = wd;
    launch_gemm<tc::A_PACKED, tc::EPI_K5>(b, g, prof::S_K5, st);
}

}  // namespace od
