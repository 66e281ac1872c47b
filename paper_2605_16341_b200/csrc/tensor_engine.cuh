// Tensor-core engine: tcgen05 (5th-generation tensor core) kernels with accumulators in tensor
// memory.  Every matrix product of the step is a sum of bf16 products with fp32 accumulation:
// an fp32 operand v is split as v = t0 + t1 with t0 = bf16(v), t1 = bf16(v - t0), and "3 passes"
// means t0*u0 + t0*u1 + t1*u0 (relative error about 2^-16), "1 pass" t0*u0.
//
// Operands.  Every small operand (Q, Y, P, R, L^{-1} and the QR intermediates) lives in global
// memory as a split image (common.cuh): ready-made swizzled shared-memory tiles that one tiled
// TMA load (cp.async.bulk.tensor over a 5-d tensor map: 64 elements, rows, panels, terms,
// matrices of the launch batch) drops into an operand ring, usable both K-major and MN-major,
// so no kernel ever transposes.  Images are written by the epilogue of the kernel
// that produces the matrix; only Q_prev (caller-owned fp32) is packed by a kernel of its own.
// The big operand B = M + G (Alg. 1, buffer step) is never stored: transform warps read M and G from
// HBM, add, split and write the A tile directly.
//
// One CTA per SM walks a tile list.  Two rings in shared memory: A tiles of 128 x 64 (both terms,
// 32 KB) and N-side pieces (a slice of the other operand, at most 48 KB), each with full/empty
// mbarriers; accumulators (up to 128 x 512 fp32) sit in tensor memory.
#pragma once
#include <cuda.h>

#include <algorithm>
#include <atomic>
#include <cstdio>

#include "common.cuh"
#include "profile.cuh"
#include "simt_kernels.cuh"

namespace od {
namespace tc {

constexpr int BM = 128;                      // tile rows (MMA M)
constexpr int BK = 64;                       // depth of one A tile: 64 bf16 = one 128-byte row
constexpr int A_TERM_BYTES = 128 * 128;      // one 128 x 64 bf16 tile
constexpr int A_RING_BYTES = 4 * A_TERM_BYTES;   // two slots of two terms, or four slots of one
constexpr int MAX_A_SLOTS = 4;
constexpr int MAX_N_SLOTS = 6;
constexpr int NUM_XF_WARPS = 16;             // transform warps of the kernels that form B = M + G
constexpr int STAGING_BYTES_PER_WARP = 8192; // epilogue staging: one 32 x 64 fp32 block (or M, G, X slabs) per warp
constexpr int SMEM_LIMIT = 227 * 1024;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // about two seconds

enum AMode : int { A_IMG_K = 0, A_IMG_MN = 1, A_BUF_ROW = 2, A_BUF_COL = 3 };
enum NMode : int { N_IMG_K = 0, N_IMG_MN = 1 };
enum EpiMode : int { EPI_STORE = 0, EPI_K5 = 1 };

__host__ __device__ constexpr bool a_is_buf(int amode) { return amode == A_BUF_ROW || amode == A_BUF_COL; }
// Eight epilogue warps (two per tensor-memory lane quarter, splitting the columns) for the fused
// pass, whose epilogue is most of a tile's time.  Everywhere else four: the products that form B
// have sixteen transform warps already, and the image-to-image products of the QR do better with
// the 32 KB of staging that four more warps would take spent on a third A slot (they are bound by
// the latency of their operand tiles: measured apply 10.3 -> 9.4 ms, Gram 8.85 -> 8.5 ms).
__host__ __device__ constexpr int epi_warps(int amode, int epi) { (void)amode; return epi == EPI_K5 ? 8 : 4; }
__host__ __device__ constexpr int gemm_threads(int amode, int epi) {
    return 32 * (2 + epi_warps(amode, epi) + (a_is_buf(amode) ? NUM_XF_WARPS : 0));
}

// Where the result of an EPI_STORE product goes.
struct Dest {
    Sel f32;            // fp32 row-major copy (leading dimension OutSpec::ld) when has_f32
    ImgRef img;         // split image when img.off >= 0
    int32_t has_f32;
    int32_t colsq;      // also write per-(32-row block) column sums of squares (fp32)
};
struct OutSpec {
    Dest normal, shifted;      // `shifted` is used when the matrix's status has shift_bit set
    int32_t shift_bit;
    int32_t only_if_shifted;   // skip the matrix unless shift_bit is set
    int64_t ld;
};

struct GemmArgs {
    int32_t Mrows, Ncols, Kdim, BN;          // BN: nominal tile width (multiple of 16, <= 512)
    int32_t m_tiles, n_tiles, k_blocks, total_tiles;
    int32_t tri;                             // N-side is lower triangular (apply): skip depth beyond the tile
    int32_t lower_only;                      // symmetric result (Gram): skip tiles above the diagonal
    int32_t passes, passes2;                 // 1 or 3; passes2: second product of the fused pass
    int32_t ks;                              // N_IMG_MN: depth of one N-side piece (16, 32 or 64)
    int32_t n_slots, n_piece_bytes;          // N ring
    int32_t acc_bufs;                        // accumulator buffers in tensor memory (1 or 2)
    int32_t tmem_cols;                       // allocation (power of two >= 32)
    int32_t fp16;                            // single-pass fp16 products from plane 2 of the images
    int32_t a_slots, a_slot_bytes;           // A ring
    int32_t epi_bufs;                        // fused pass: 8 KB epilogue buffers per warp (1 or 2)
    int32_t pair;                            // launched as CTA pairs (clusters of two, M = 256 instructions)
    int32_t ksplit, kb_per_chunk;            // depth split: a tile is computed as `ksplit` partial products over
                                             // kb_per_chunk depth blocks each, stored split_stride floats apart
    int64_t split_stride;
    int64_t rscale_off;                      // fp16 fused pass: scratch offset of 1 / (scale of R's plane)
    int64_t ld;                              // leading dimension of M, G, X
    ImgRef a, n1, n2;
    int64_t colsq_off;                       // scratch offset of the column-square partials
    float ef_a, ef_b, wc, wd;
    OutSpec out;
    // tensor maps of the images a, n1, n2 over the whole launch batch; the box of each map is the
    // tile or piece this launch loads with one instruction
    alignas(64) CUtensorMap map_a;
    alignas(64) CUtensorMap map_n1;
    alignas(64) CUtensorMap map_n2;
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
// One tiled TMA load: the box of `map` at (0, row, panel, plane, matrix) -> shared memory, laid
// out [term][panel][row][128 bytes]; completes on the mbarrier with the full box size.
__device__ __forceinline__ void tma_load_box(uint32_t dst, const CUtensorMap* map, int row, int panel, int plane,
                                             int matrix, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(row), "r"(panel), "r"(plane), "r"(matrix), "r"(bar)
        : "memory");
}
// ---- CTA pairs (clusters of two CTAs on neighbouring SMs, tcgen05 cta_group::2) ----------------
// One MMA instruction of the pair's leader (cluster rank 0) multiplies M = 256 rows: each CTA
// supplies its own 128 rows of A and HALF of the N-side operand, and receives its 128 rows of the
// result in its own tensor memory.  Per CTA that halves the N-side bytes that are fetched from L2
// and read from shared memory by the tensor core.  Barriers that gather both CTAs (operand
// "full", accumulator "empty") live in the leader and are reached by remote arrives; barriers
// that release (operand "empty", accumulator "full") live in each CTA and are reached by the
// leader's multicast commit.  All of them keep the default (CTA-scope) semantics of the single-CTA
// barriers: with release/acquire at cluster scope on every arrive and wait the same kernels ran up
// to twice as long (the producer thread then pays a cluster-wide fence per load).
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the location `addr` (a shared::cta address) in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_rank(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx_remote(uint32_t cluster_addr, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cluster.b64 _, [%0], %1;"
                 ::"r"(cluster_addr), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Tiled TMA load of a CTA of a pair: the data lands in this CTA's shared memory, the bytes are
// counted on the mbarrier at cluster address `bar` (the leader's).
__device__ __forceinline__ void tma_load_box_pair(uint32_t dst, const CUtensorMap* map, int row, int panel, int plane,
                                                  int matrix, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.5d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(0), "r"(row), "r"(panel), "r"(plane), "r"(matrix), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// D[tmem of both CTAs] (+)= A * B^T with M = 256; issued by one thread of the leader.
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
// the mbarrier at offset `bar` of BOTH CTAs arrives once every MMA issued so far has completed
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
    asm volatile(
        "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
        ::"r"(bar), "h"((uint16_t)3) : "memory");
}

// Asynchronous 16-byte copy global -> shared (no register staging), grouped per thread.
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
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
// Instruction descriptor: fp32 accumulate, bf16 A and B, M = 128, N = n; a_mn / b_mn = 1 for an
// MN-major A / B operand (0: K-major).
// fmt: operand format, 1 = bf16, 0 = fp16 (both operands alike).
// m: rows of the instruction, 128, or 256 for an instruction of a CTA pair.
__device__ __forceinline__ uint32_t instr_desc(uint32_t n, uint32_t a_mn, uint32_t b_mn, uint32_t fmt = 1u,
                                               uint32_t m = (uint32_t)BM) {
    return (1u << 4) | (fmt << 7) | (fmt << 10) | (a_mn << 15) | (b_mn << 16) | ((n >> 3) << 17) |
           ((m >> 4) << 24);
}
template <bool PAIR>
__device__ __forceinline__ void umma_any(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                         uint32_t accumulate) {
    if (PAIR) umma_bf16_pair(d_tmem, adesc, bdesc, idesc, accumulate);
    else umma_bf16(d_tmem, adesc, bdesc, idesc, accumulate);
}
template <bool PAIR>
__device__ __forceinline__ void commit_any(uint32_t bar) {
    if (PAIR) umma_commit_pair(bar);
    else umma_commit(bar);
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
// Pack kernel: fp32 matrix S (rows x cols, row-major, cols % 8 == 0) -> split image.
// One CTA per (panel, 128-row block), 256 threads; rows beyond `rows` are written as zeros.
// ------------------------------------------------------------------------------------------
struct PackArgs {
    Sel src;
    int32_t rows, cols;
    ImgRef dst;
};

__global__ void __launch_bounds__(256)
pack_kernel(const __grid_constant__ Batch batch, PackArgs a) {
    const MatWork& w = batch.w[blockIdx.z];
    if (*w.status & ST_FAILED) return;
    const float* S = pick(w, a.src);
    const int panel = blockIdx.x, rb = blockIdx.y;
    unsigned char* out0 = reinterpret_cast<unsigned char*>(w.scratch) + img_row_offset(a.dst, 0, panel, (int64_t)rb * 128);
    unsigned char* out1 = reinterpret_cast<unsigned char*>(w.scratch) + img_row_offset(a.dst, 1, panel, (int64_t)rb * 128);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int q = threadIdx.x + 256 * e;
        const int rho = q / 8, c = q % 8;
        const int64_t gr = (int64_t)rb * 128 + rho, gk = (int64_t)panel * 64 + c * 8;
        float v[8];
        if (gr < a.rows && gk < a.cols) {
            load8(S, gr * a.cols + gk, 0, v);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = 0.f;
        }
        uint4 t0, t1;
        split8(v, t0, t1);
        const int o = rho * 128 + img_chunk_offset(rho, c);
        *reinterpret_cast<uint4*>(out0 + o) = t0;
        *reinterpret_cast<uint4*>(out1 + o) = t1;
        if (a.dst.planes == 3)
            *reinterpret_cast<uint4*>(reinterpret_cast<unsigned char*>(w.scratch) +
                                      img_row_offset(a.dst, 2, panel, (int64_t)rb * 128) + o) = half8(v, 1.f);
    }
}

// fp16 plane of R for the single-pass fused feedback/update product.  R is scaled by the power of
// two that brings its largest column norm to about 2^10 (no entry can then overflow fp16, and
// typical entries stay far from the subnormal range); the inverse scale is left at `rscale_off`
// for the epilogue.  cnorm holds the squared column norms of R (written by the Cholesky of the
// right QR, or by ColNorm).  One CTA per (panel, 128-row block), 256 threads.
struct PackHalfArgs {
    int32_t rows, cols;
    ImgRef dst;
    int64_t cnorm_off, rscale_off;
};

__global__ void __launch_bounds__(256)
pack_half_kernel(const __grid_constant__ Batch batch, PackHalfArgs a) {
    const MatWork& w = batch.w[blockIdx.z];
    if (*w.status & ST_FAILED) return;
    __shared__ float red[8];
    __shared__ float s_scale;
    const float* cn = reinterpret_cast<const float*>(w.scratch + a.cnorm_off);
    float mx = 0.f;
    for (int j = threadIdx.x; j < a.cols; j += 256) mx = fmaxf(mx, cn[j]);
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (threadIdx.x % 32 == 0) red[threadIdx.x / 32] = mx;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) mx = fmaxf(mx, red[i]);
        int e = 0;
        const float nrm = sqrtf(mx);
        if (nrm > 0.f && nrm <= 3.0e38f) frexpf(nrm, &e);      // nrm = f * 2^e, 0.5 <= f < 1
        const float scale = ldexpf(1.f, 10 - e);
        s_scale = scale;
        if (blockIdx.x == 0 && blockIdx.y == 0)
            *reinterpret_cast<float*>(w.scratch + a.rscale_off) = ldexpf(1.f, e - 10);
    }
    __syncthreads();
    const float scale = s_scale;
    const int panel = blockIdx.x, rb = blockIdx.y;
    unsigned char* out = reinterpret_cast<unsigned char*>(w.scratch) + img_row_offset(a.dst, 2, panel, (int64_t)rb * 128);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const int q = threadIdx.x + 256 * e;
        const int rho = q / 8, c = q % 8;
        const int64_t gr = (int64_t)rb * 128 + rho, gk = (int64_t)panel * 64 + c * 8;
        float v[8];
        if (gr < a.rows && gk < a.cols) {
            load8(w.R, gr * a.cols + gk, 0, v);
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) v[i] = 0.f;
        }
        *reinterpret_cast<uint4*>(out + rho * 128 + img_chunk_offset(rho, c)) = half8(v, scale);
    }
}

// ------------------------------------------------------------------------------------------
// Tile bookkeeping shared by all roles of the GEMM kernel
// ------------------------------------------------------------------------------------------
struct TileCoord { int b, mt, nt, n0, bn, kb_begin, kb_end, chunk; bool active; };
// Each role remembers the status word of the matrix it is working on (nothing changes it while
// the kernel runs), so that only the first tile of a matrix pays for the global load.
struct StatusCache { int b = -1; int st = 0; };

// Pair launches (g.pair): a scheduled row tile is 256 rows, CTA `rank` of the pair owns its
// rows 128 * rank .. ; c.mt stays the 128-row tile index (it may lie one past the last tile when
// the number of tiles is odd: that CTA multiplies zeros and stores nothing).
template <int EPI>
__device__ __forceinline__ TileCoord decode_tile(const Batch& batch, const GemmArgs& g, int t, StatusCache& sc,
                                                 int rank) {
    TileCoord c;
    const int per = g.m_tiles * g.n_tiles * g.ksplit;
    c.b = t / per;
    int rem = t - c.b * per;
    c.chunk = 0;
    if (g.ksplit > 1) { const int tl = rem / g.ksplit; c.chunk = rem - tl * g.ksplit; rem = tl; }
    const int mts = rem / g.n_tiles;
    c.nt = rem - mts * g.n_tiles;
    c.mt = g.pair ? 2 * mts + rank : mts;
    c.n0 = c.nt * g.BN;
    c.bn = min(g.BN, g.Ncols - c.n0);
    c.kb_begin = 0;
    c.kb_end = g.k_blocks;
    if (g.tri) c.kb_end = min(g.k_blocks, (c.n0 + c.bn + BK - 1) / BK);
    if (g.ksplit > 1) { c.kb_begin = c.chunk * g.kb_per_chunk; c.kb_end = min(g.k_blocks, c.kb_begin + g.kb_per_chunk); }
    if (c.b != sc.b) { sc.b = c.b; sc.st = *batch.w[c.b].status; }
    const int st = sc.st;
    c.active = !(st & ST_FAILED);
    if (EPI != EPI_K5 && g.out.only_if_shifted && !(st & g.out.shift_bit)) c.active = false;
    if (g.lower_only && c.n0 > (g.pair ? 2 * mts + 1 : c.mt) * BM + BM - 1) c.active = false;
    if (c.kb_begin >= c.kb_end) c.active = false;
    return c;
}

// N_IMG_MN: the pieces of depth block kb are its ks-deep slices that start below Kdim.
__device__ __forceinline__ int mn_pieces(const GemmArgs& g, int kb) {
    const int left = g.Kdim - kb * BK;
    return (min(left, BK) + g.ks - 1) / g.ks;
}
// N_IMG_K: the pieces of depth block kb are 128-row chunks of the tile's N range; with a lower
// triangular N-side a chunk is skipped once the depth block lies beyond its last row.
__device__ __forceinline__ bool k_piece_active(const GemmArgs& g, const TileCoord& c, int kb, int chunk) {
    return !g.tri || kb * BK <= c.n0 + min(c.bn, (chunk + 1) * 128) - 1;
}

// ------------------------------------------------------------------------------------------
// The GEMM kernel.  D (128 x bn, fp32 in tensor memory) = A (128 x K) * N^T (bn x K).
//   warp 0        producer: bulk copies of image tiles into the A ring and the N ring
//   warp 1        MMA issuer, owns the tensor-memory allocation
//   next 4 or 8   epilogue warps (tensor memory -> registers -> global)
//   last 16       transform warps (A_BUF_* only): form B = M + G, split, write the A tile
// AMODE  where the A tile comes from and how it lies in shared memory
//          A_IMG_K / A_IMG_MN   image tile, K-major / MN-major
//          A_BUF_ROW            rows of B = M + G      (K-major;  Y = B Q_prev, Alg. 1, left-factor step)
//          A_BUF_COL            columns of B = M + G   (MN-major; R = B^T P,    Alg. 1, right-factor step)
// NMODE  N_IMG_K   pieces = 128-row chunks of the N range, 64 deep (image K-major)
//        N_IMG_MN  pieces = ks-deep slices of the whole N range (image MN-major)
// EPI    EPI_STORE  fp32 copy and/or split image (+ column-square partials) of D
//        EPI_K5     M <- a (M+G) - b D1,  X <- c X - d D2     (Alg. 1, update and error-feedback steps), D1 = P R^T, D2 = P Q^T
// XG     bit 0: G is bf16, bit 1: X is bf16
// ------------------------------------------------------------------------------------------
template <int XG>
struct K5Pre {      // M, G, X of one 32 x 32 slab: 8 steps of (4 rows x 32 columns) per warp
    float4 m[8];
    uint32_t g[8][(XG & 1) ? 2 : 4];
    uint32_t x[8][(XG & 2) ? 2 : 4];
};

template <int AMODE, int NMODE, int EPI, int XG, bool PAIR>
__global__ void __launch_bounds__(gemm_threads(AMODE, EPI), 1)
gemm_kernel(const __grid_constant__ Batch batch, const __grid_constant__ GemmArgs g) {
    constexpr int NE = epi_warps(AMODE, EPI);
    // PAIR: launched in clusters of two; rank 0 (the leader) issues every MMA for both CTAs
    const int crank = PAIR ? (int)cluster_ctarank() : 0;
    const int tile0 = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int tstride = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
    constexpr bool A_BUF = a_is_buf(AMODE);
    constexpr bool A_MN = (AMODE == A_IMG_MN || AMODE == A_BUF_COL);
    constexpr bool G_BF16 = (XG & 1) != 0;
    constexpr bool X_BF16 = (XG & 2) != 0;

    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    unsigned char* smem = smem_raw + (((raw + 1023u) & ~1023u) - raw);
    unsigned char* a_ring = smem;
    unsigned char* n_ring = smem + g.a_slots * g.a_slot_bytes;
    unsigned char* staging = n_ring + (size_t)g.n_slots * g.n_piece_bytes;
    unsigned char* tail = staging + ((EPI == EPI_K5 || !A_BUF) ? NE * g.epi_bufs * STAGING_BYTES_PER_WARP : 0);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tail);
    const uint32_t a_full0 = smem_u32(bars), a_empty0 = a_full0 + 8 * MAX_A_SLOTS;
    const uint32_t n_full0 = a_empty0 + 8 * MAX_A_SLOTS, n_empty0 = n_full0 + 8 * MAX_N_SLOTS;
    const uint32_t tfull0 = n_empty0 + 8 * MAX_N_SLOTS, tempty0 = tfull0 + 16;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * MAX_A_SLOTS + 2 * MAX_N_SLOTS + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    StatusCache scache;

    // Pairs: the "full" barriers of the operand rings and the "empty" barriers of the accumulators
    // that are used are the leader's; they count the arrivals of both CTAs.
    constexpr uint32_t NCTA = PAIR ? 2u : 1u;
    if (threadIdx.x == 0) {
        for (int s = 0; s < MAX_A_SLOTS; ++s) {
            mbar_init(a_full0 + 8 * s, NCTA * (A_BUF ? NUM_XF_WARPS : 1));
            mbar_init(a_empty0 + 8 * s, 1);
        }
        for (int s = 0; s < MAX_N_SLOTS; ++s) {
            mbar_init(n_full0 + 8 * s, NCTA);
            mbar_init(n_empty0 + 8 * s, 1);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tfull0 + 8 * a, 1);
            mbar_init(tempty0 + 8 * a, NCTA * NE);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    if (warp == 1) {
        if (PAIR) tmem_alloc_pair(smem_u32(tmem_slot), (uint32_t)g.tmem_cols);
        else tmem_alloc(smem_u32(tmem_slot), (uint32_t)g.tmem_cols);
    }
    tc_fence_before();
    __syncthreads();
    if (PAIR) cluster_sync_all();       // the peer's barriers are initialised before anything reaches them
    tc_fence_after();
    // cluster addresses of the leader's gathering barriers (slot s: + 8 s)
    const uint32_t a_full_ld = PAIR ? map_to_rank(a_full0, 0) : a_full0;
    const uint32_t n_full_ld = PAIR ? map_to_rank(n_full0, 0) : n_full0;
    const uint32_t tempty_ld = PAIR ? map_to_rank(tempty0, 0) : tempty0;
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t acc_stride = (uint32_t)(g.tmem_cols / g.acc_bufs);

    const int a_terms = g.a_slot_bytes / A_TERM_BYTES;
    const int n1_terms = g.passes == 3 ? 2 : 1;
    const int plane = g.fp16 ? 2 : 0;
    const uint32_t fmt = g.fp16 ? 0u : 1u;
    // N_IMG_MN piece geometry: [term][64-column group][ks rows of 128 bytes]
    const uint32_t group_stride = (uint32_t)g.ks * 128u;
    const uint32_t mn_term_stride = PAIR ? 2u * group_stride : (uint32_t)((g.BN + 63) / 64) * group_stride;

    if (warp == 0) {
        // ---------------- producer ----------------
        // One thread feeds both rings.  It walks the schedule twice, with one cursor per ring, and
        // serves whichever ring has a free slot, so a full N ring never holds back A tiles (and
        // the other way round).  Every slot is filled by one tiled TMA load (two for the fused
        // pass: R and Q pieces).
        if (lane == 0) {
            int as = 0, ns = 0; uint32_t aph = 0, nph = 0;
            // cursor over (tile, depth block) for the A ring
            int at = tile0, akb = -1; TileCoord ac{}; bool a_done = A_BUF;      // akb < 0: tile not decoded yet
            // cursor over (tile, depth block, piece) for the N ring
            int nt_ = tile0, nkb = -1, npc = 0; TileCoord nc{}; bool n_done = false;
            auto a_seek = [&]() {           // make (at, akb) valid or finish
                while (!a_done) {
                    if (at >= g.total_tiles) { a_done = true; break; }
                    if (akb < 0) { ac = decode_tile<EPI>(batch, g, at, scache, crank); akb = ac.kb_begin; }
                    if (ac.active && akb < ac.kb_end) break;
                    at += tstride; akb = -1;
                }
            };
            auto n_pieces = [&](int kb) { return NMODE == N_IMG_MN ? mn_pieces(g, kb) : (nc.bn + 127) / 128; };
            auto n_seek = [&]() {           // make (nt_, nkb, npc) valid or finish
                while (!n_done) {
                    if (nt_ >= g.total_tiles) { n_done = true; break; }
                    if (nkb < 0) { nc = decode_tile<EPI>(batch, g, nt_, scache, crank); nkb = nc.kb_begin; npc = 0; }
                    if (!nc.active || nkb >= nc.kb_end) { nt_ += tstride; nkb = -1; npc = 0; continue; }
                    if (npc >= n_pieces(nkb)) { ++nkb; npc = 0; continue; }
                    if (NMODE == N_IMG_K && !k_piece_active(g, nc, nkb, npc)) { ++npc; continue; }
                    break;
                }
            };
            a_seek();
            n_seek();
            long long idle_since = -1;
            while (!a_done || !n_done) {
                bool progress = false;
                if (!a_done && mbar_try_wait(a_empty0 + 8 * as, aph ^ 1)) {
                    const uint32_t dst = smem_u32(a_ring + as * g.a_slot_bytes);
                    if (PAIR) {
                        const uint32_t fb = a_full_ld + 8 * as;
                        mbar_arrive_expect_tx_remote(fb, (uint32_t)a_terms * A_TERM_BYTES);
                        if (AMODE == A_IMG_K) tma_load_box_pair(dst, &g.map_a, ac.mt * BM, akb, plane, ac.b, fb);
                        else tma_load_box_pair(dst, &g.map_a, akb * BK, ac.mt * 2, plane, ac.b, fb);
                    } else {
                        const uint32_t fb = a_full0 + 8 * as;
                        mbar_arrive_expect_tx(fb, (uint32_t)a_terms * A_TERM_BYTES);
                        if (AMODE == A_IMG_K) tma_load_box(dst, &g.map_a, ac.mt * BM, akb, plane, ac.b, fb);
                        else tma_load_box(dst, &g.map_a, akb * BK, ac.mt * 2, plane, ac.b, fb);
                    }
                    if (++as == g.a_slots) { as = 0; aph ^= 1; }
                    ++akb;
                    if (akb >= ac.kb_end) { at += tstride; akb = -1; }
                    a_seek();
                    progress = true;
                }
                if (!n_done && mbar_try_wait(n_empty0 + 8 * ns, nph ^ 1)) {
                    const uint32_t fb = PAIR ? n_full_ld + 8 * ns : n_full0 + 8 * ns;
                    const uint32_t dst = smem_u32(n_ring + (size_t)ns * g.n_piece_bytes);
                    if (PAIR) {
                        // this CTA's half of the N-side: per 256-column block its two 64-column groups
                        // (MN-major), or the R piece (leader) / the Q piece (peer) of the fused pass
                        mbar_arrive_expect_tx_remote(fb, (uint32_t)g.n_piece_bytes);
                        if (NMODE == N_IMG_MN) {
                            const uint32_t blk_bytes = (uint32_t)n1_terms * 2u * group_stride;
                            for (int blk = 0; blk * 256 < nc.bn; ++blk)
                                tma_load_box_pair(dst + blk * blk_bytes, &g.map_n1, nkb * BK + npc * g.ks,
                                                  nc.n0 / 64 + blk * 4 + crank * 2, plane, nc.b, fb);
                        } else {
                            tma_load_box_pair(dst, crank == 0 ? &g.map_n1 : &g.map_n2, nc.n0 + npc * 128, nkb, plane,
                                              nc.b, fb);
                        }
                    } else {
                        mbar_arrive_expect_tx(fb, (uint32_t)g.n_piece_bytes);
                        if (NMODE == N_IMG_MN) {
                            tma_load_box(dst, &g.map_n1, nkb * BK + npc * g.ks, nc.n0 / 64, plane, nc.b, fb);
                        } else {
                            tma_load_box(dst, &g.map_n1, nc.n0 + npc * 128, nkb, plane, nc.b, fb);
                            if (EPI == EPI_K5)
                                tma_load_box(dst + n1_terms * A_TERM_BYTES, &g.map_n2, nc.n0 + npc * 128, nkb, plane, nc.b, fb);
                        }
                    }
                    if (++ns == g.n_slots) { ns = 0; nph ^= 1; }
                    ++npc;
                    n_seek();
                    progress = true;
                }
                if (progress) {
                    idle_since = -1;
                } else {
                    if (*abort_flag) break;
                    const long long now = clock64();
                    if (idle_since < 0) idle_since = now;
                    else if (now - idle_since > WAIT_LIMIT_CYCLES) { *abort_flag = 1; break; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        // One thread issues.  A tcgen05.mma of N = 256 occupies the tensor core for 128 cycles, so the
        // scalar work per instruction has to stay at a handful of operations: every descriptor is a
        // constant high part plus (shared address >> 4), advanced by additions only.
        int as = 0, ns = 0; uint32_t aph = 0, nph = 0;
        int acc = 0; uint32_t acc_phase = 0;
        bool ok = true;
        // descriptor high parts (layout, strides) and address units of 16 bytes
        const uint64_t a_hi = A_MN ? smem_desc(0, 8192, 1024) : smem_desc(0, 16, 1024);
        const uint64_t n_hi = (NMODE == N_IMG_MN) ? smem_desc(0, group_stride, 1024) : smem_desc(0, 16, 1024);
        const uint32_t a_slice16 = A_MN ? (2048u >> 4) : (32u >> 4);        // one 16-deep slice of the A tile
        const uint32_t n_slice16 = (NMODE == N_IMG_MN) ? (2048u >> 4) : (32u >> 4);
        const uint32_t a_term16 = A_TERM_BYTES >> 4;
        const uint32_t n_term16 = ((NMODE == N_IMG_MN) ? mn_term_stride : (uint32_t)A_TERM_BYTES) >> 4;
        const uint32_t a_ring16 = smem_u32(a_ring) >> 4, n_ring16 = smem_u32(n_ring) >> 4;
        const uint32_t a_slot16 = (uint32_t)g.a_slot_bytes >> 4, n_slot16 = (uint32_t)g.n_piece_bytes >> 4;
        const bool three = g.passes == 3;
        constexpr uint32_t MROWS = PAIR ? 256u : 128u;
        // pairs: a 256-column block of the N-side is this CTA's two 64-column groups, both terms
        const uint32_t n_block16 = (PAIR ? (uint32_t)n1_terms * 2u * group_stride : 4u * group_stride) >> 4;
        for (int t = tile0; t < g.total_tiles && ok && crank == 0; t += tstride) {
            const TileCoord c = decode_tile<EPI>(batch, g, t, scache, crank);
            if (!c.active) continue;
            if (!mbar_wait(tempty0 + 8 * acc, acc_phase ^ 1, abort_flag)) { ok = false; break; }
            // orders this tile's MMAs after the epilogue's tensor-memory loads.  (The operand waits
            // below need no tcgen05 fence: the operands arrive through the async proxy or behind
            // a proxy fence, and a fence per piece stalled the issuer for hundreds of cycles.)
            tc_fence_after();
            const uint32_t dacc = tmem_base + acc * acc_stride;
            for (int kb = c.kb_begin; kb < c.kb_end && ok; ++kb) {
                if (!mbar_wait(a_full0 + 8 * as, aph, abort_flag)) { ok = false; break; }
                const uint64_t a_kb = a_hi + (a_ring16 + as * a_slot16);
                if (NMODE == N_IMG_MN) {
                    const int pieces = mn_pieces(g, kb);
                    const int per_piece = g.ks / 16;
                    for (int sub = 0; sub < pieces && ok; ++sub) {
                        if (!mbar_wait(n_full0 + 8 * ns, nph, abort_flag)) { ok = false; break; }
                        if (lane == 0) {
                            const uint64_t n_pc = n_hi + (n_ring16 + ns * n_slot16);
                            const int k0 = kb * BK + sub * g.ks;
                            const int nsl = (min(g.ks, g.Kdim - k0) + 15) / 16;
                            for (int j = 0; j < nsl; ++j) {
                                const uint64_t a0 = a_kb + (uint32_t)(sub * per_piece + j) * a_slice16;
                                const uint64_t a1 = a0 + a_term16;
                                const uint32_t accum = (kb > c.kb_begin || sub > 0 || j > 0) ? 1u : 0u;
                                uint64_t b0 = n_pc + (uint32_t)j * n_slice16;
                                for (int cc = 0; cc < c.bn; cc += 256) {
                                    const uint32_t idesc = instr_desc((uint32_t)min(256, c.bn - cc), A_MN ? 1u : 0u, 1u, fmt, MROWS);
                                    umma_any<PAIR>(dacc + cc, a0, b0, idesc, accum);
                                    if (three) {
                                        umma_any<PAIR>(dacc + cc, a0, b0 + n_term16, idesc, 1u);
                                        umma_any<PAIR>(dacc + cc, a1, b0, idesc, 1u);
                                    }
                                    b0 += n_block16;                        // next 256 columns
                                }
                            }
                            commit_any<PAIR>(n_empty0 + 8 * ns);
                        }
                        __syncwarp();
                        if (++ns == g.n_slots) { ns = 0; nph ^= 1; }
                    }
                } else {
                    const int chunks = (c.bn + 127) / 128;
                    const int nsl = min(4, (g.Kdim - kb * BK + 15) / 16);
                    for (int ch = 0; ch < chunks && ok; ++ch) {
                        if (!k_piece_active(g, c, kb, ch)) continue;
                        if (!mbar_wait(n_full0 + 8 * ns, nph, abort_flag)) { ok = false; break; }
                        if (lane == 0) {
                            const uint32_t sa = smem_u32(a_ring + as * g.a_slot_bytes);
                            const uint32_t sn = smem_u32(n_ring + (size_t)ns * g.n_piece_bytes);
                            // N of the instruction must be a multiple of 16: round a ragged last chunk up
                            // (rows beyond the matrix are zero in the images; those columns of D are never stored)
                            const uint32_t ncols = (uint32_t)((min(128, c.bn - ch * 128) + 15) / 16 * 16);
                            const uint32_t idesc = instr_desc(ncols, A_MN ? 1u : 0u, 0u, fmt, MROWS);
                            // Fused pass with single-term operands: the R piece and the Q piece lie back
                            // to back in the slot (256 rows of one K-major tile) and their accumulators in
                            // adjacent columns, so one N = 256 instruction serves both products and reads
                            // the P slice from shared memory once.
                            const bool both = EPI == EPI_K5 && g.passes == 1 && g.passes2 == 1 && ncols == 128 && g.BN == 128;
                            const uint32_t idesc2 = instr_desc(256u, A_MN ? 1u : 0u, 0u, fmt, MROWS);
                            if (both) {
                                // one instruction per 16-deep slice; descriptors advanced by additions so
                                // that the issuing thread spends a handful of operations per instruction
                                uint64_t a0 = a_hi + (a_ring16 + as * a_slot16);
                                uint64_t b0 = n_hi + (n_ring16 + ns * n_slot16);
                                const uint32_t d1 = dacc + ch * 128;
                                umma_any<PAIR>(d1, a0, b0, idesc2, kb > c.kb_begin ? 1u : 0u);
                                for (int j = 1; j < nsl; ++j) {
                                    a0 += a_slice16; b0 += n_slice16;
                                    umma_any<PAIR>(d1, a0, b0, idesc2, 1u);
                                }
                            }
                            // (In the general form below the descriptors are rebuilt per instruction on
                            // purpose: its N = 128 instructions ran best when not issued back to back.)
                            for (int j = 0; j < nsl && !both; ++j) {
                                const uint64_t a0 = A_MN ? smem_desc(sa + j * 2048, 8192, 1024)
                                                         : smem_desc(sa + j * 32, 16, 1024);
                                const uint64_t a1 = A_MN ? smem_desc(sa + A_TERM_BYTES + j * 2048, 8192, 1024)
                                                         : smem_desc(sa + A_TERM_BYTES + j * 32, 16, 1024);
                                const uint64_t b0 = smem_desc(sn + j * 32, 16, 1024);
                                const uint64_t b1 = smem_desc(sn + A_TERM_BYTES + j * 32, 16, 1024);
                                const uint32_t accum = (kb > c.kb_begin || j > 0) ? 1u : 0u;
                                const uint32_t d1 = dacc + ch * 128;
                                umma_any<PAIR>(d1, a0, b0, idesc, accum);
                                if (g.passes == 3) {
                                    umma_any<PAIR>(d1, a0, b1, idesc, 1u);
                                    umma_any<PAIR>(d1, a1, b0, idesc, 1u);
                                }
                                if (EPI == EPI_K5) {
                                    const uint32_t s2 = sn + n1_terms * A_TERM_BYTES;
                                    const uint64_t c0 = smem_desc(s2 + j * 32, 16, 1024);
                                    const uint64_t c1 = smem_desc(s2 + A_TERM_BYTES + j * 32, 16, 1024);
                                    const uint32_t d2 = dacc + g.BN;
                                    umma_any<PAIR>(d2, a0, c0, idesc, accum);
                                    if (g.passes2 == 3) {
                                        umma_any<PAIR>(d2, a0, c1, idesc, 1u);
                                        umma_any<PAIR>(d2, a1, c0, idesc, 1u);
                                    }
                                }
                            }
                            commit_any<PAIR>(n_empty0 + 8 * ns);
                        }
                        __syncwarp();
                        if (++ns == g.n_slots) { ns = 0; nph ^= 1; }
                    }
                }
                if (!ok) break;
                if (lane == 0) commit_any<PAIR>(a_empty0 + 8 * as);
                __syncwarp();
                if (++as == g.a_slots) { as = 0; aph ^= 1; }
            }
            if (!ok) break;
            if (lane == 0) commit_any<PAIR>(tfull0 + 8 * acc);
            __syncwarp();
            if (++acc == g.acc_bufs) { acc = 0; acc_phase ^= 1; }
        }
    } else if (warp < 2 + NE) {
        // ---------------- epilogue ----------------
        int acc = 0; uint32_t acc_phase = 0;
        bool ok = true;
        const int quarter = warp % 4;                    // tensor-memory lanes 32*quarter .. +31
        if (EPI == EPI_STORE) {
            for (int t = tile0; t < g.total_tiles && ok; t += tstride) {
                const TileCoord c = decode_tile<EPI>(batch, g, t, scache, crank);
                if (!c.active) continue;
                if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const MatWork& w = batch.w[c.b];
                const int stw = scache.st;
                const Dest& d = (g.out.shift_bit && (stw & g.out.shift_bit)) ? g.out.shifted : g.out.normal;
                const uint32_t taddr = tmem_base + acc * acc_stride + ((uint32_t)(quarter * 32) << 16);
                float* C = d.has_f32 ? pick(w, d.f32) + (int64_t)c.chunk * g.split_stride : nullptr;
                unsigned char* scr = reinterpret_cast<unsigned char*>(w.scratch);
                const bool to_img = d.img.off >= 0;
                float* csq = d.colsq ? reinterpret_cast<float*>(w.scratch + g.colsq_off) +
                                           (int64_t)(c.mt * 4 + quarter) * g.Ncols : nullptr;
                if constexpr (A_BUF) {
                // One wide tile per long main loop: the epilogue is a small share of the time, so
                // it stores row per lane, 16 columns at a time, straight from the registers.
                const int64_t gi = (int64_t)c.mt * BM + quarter * 32 + lane;
                // (pairs: the CTA whose rows lie beyond the matrix stores nothing)
                const bool has_rows = !PAIR || (int64_t)c.mt * BM < g.Mrows;
                const int bn64 = !has_rows ? 0 : (to_img ? (c.bn + 63) / 64 * 64 : c.bn);
                for (int cc = 0; cc < bn64; cc += 16) {
                    uint32_t v[16];
                    if (cc < c.bn) {
                        tmem_ld16(taddr + cc, v);
                        tmem_ld_wait();
                    } else {
#pragma unroll
                        for (int i = 0; i < 16; ++i) v[i] = 0u;
                    }
                    const int gj = c.n0 + cc;
                    if (C && gi < g.Mrows && cc < c.bn) {
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            *reinterpret_cast<uint4*>(C + gi * g.out.ld + gj + 4 * u) =
                                make_uint4(v[4 * u], v[4 * u + 1], v[4 * u + 2], v[4 * u + 3]);
                    }
                    if (to_img) {
                        const int panel = gj / 64, ch0 = (gj % 64) / 8;
                        unsigned char* r0 = scr + img_row_offset(d.img, 0, panel, gi);
                        unsigned char* r1 = scr + img_row_offset(d.img, 1, panel, gi);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            float f[8];
#pragma unroll
                            for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[8 * h + i]);
                            uint4 t0, t1;
                            split8(f, t0, t1);
                            const int o = img_chunk_offset((int)(gi & 7), ch0 + h);
                            *reinterpret_cast<uint4*>(r0 + o) = t0;
                            *reinterpret_cast<uint4*>(r1 + o) = t1;
                            if (d.img.planes == 3)
                                *reinterpret_cast<uint4*>(scr + img_row_offset(d.img, 2, panel, gi) + o) = half8(f, 1.f);
                        }
                    }
                    if (csq && cc < c.bn) {
                        // column sums of squares over the 32 rows of this warp: fold 16 values over
                        // the lane bits 4..1, then add the two lanes that hold the same column
                        float s[16];
#pragma unroll
                        for (int i = 0; i < 16; ++i) { const float x = __uint_as_float(v[i]); s[i] = x * x; }
#pragma unroll
                        for (int half = 8, bit = 16; half >= 1; half >>= 1, bit >>= 1) {
                            const bool up = (lane & bit) != 0;
#pragma unroll
                            for (int i = 0; i < 8; ++i) {
                                if (i < half) {
                                    const float send = up ? s[i] : s[i + half];
                                    const float keep = up ? s[i + half] : s[i];
                                    s[i] = keep + __shfl_xor_sync(0xffffffffu, send, bit);
                                }
                            }
                        }
                        s[0] += __shfl_xor_sync(0xffffffffu, s[0], 1);
                        const int col = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
                        if (!(lane & 1)) csq[gj + col] = s[0];
                    }
                }
                } else {
                // 64 columns at a time: this warp's 32 x 64 block goes through an 8 KB staging
                // buffer so that global stores run along rows.  A plane's block is 32 image rows of
                // 128 bytes, byte for byte what the image holds, so it leaves as one 4 KB run.
                unsigned char* stg = staging + (warp - 2) * STAGING_BYTES_PER_WARP;
                const int64_t gi0 = (int64_t)c.mt * BM + quarter * 32;
                const bool has_rows = !PAIR || (int64_t)c.mt * BM < g.Mrows;
                const int groups = has_rows ? (c.bn + 63) / 64 : 0;
                for (int cg = (warp - 2) / 4; cg < groups; cg += NE / 4) {
                    const int valid = min(64, c.bn - cg * 64);          // multiple of 16
                    const int gj0 = c.n0 + cg * 64;
                    float f[64];
#pragma unroll
                    for (int q4 = 0; q4 < 4; ++q4) {
                        uint32_t v[16];
                        if (q4 * 16 < valid) {
                            tmem_ld16(taddr + cg * 64 + q4 * 16, v);
                            tmem_ld_wait();
                        } else {
#pragma unroll
                            for (int i = 0; i < 16; ++i) v[i] = 0u;
                        }
#pragma unroll
                        for (int i = 0; i < 16; ++i) f[q4 * 16 + i] = __uint_as_float(v[i]);
                        if (csq && q4 * 16 < valid) {
                            // column sums of squares over the 32 rows of this warp: fold 16 values
                            // over the lane bits 4..1, then add the two lanes that hold the same column
                            float s[16];
#pragma unroll
                            for (int i = 0; i < 16; ++i) { const float x = __uint_as_float(v[i]); s[i] = x * x; }
#pragma unroll
                            for (int half = 8, bit = 16; half >= 1; half >>= 1, bit >>= 1) {
                                const bool up = (lane & bit) != 0;
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    if (i < half) {
                                        const float send = up ? s[i] : s[i + half];
                                        const float keep = up ? s[i + half] : s[i];
                                        s[i] = keep + __shfl_xor_sync(0xffffffffu, send, bit);
                                    }
                                }
                            }
                            s[0] += __shfl_xor_sync(0xffffffffu, s[0], 1);
                            const int col = ((lane >> 4) & 1) * 8 + ((lane >> 3) & 1) * 4 + ((lane >> 2) & 1) * 2 + ((lane >> 1) & 1);
                            if (!(lane & 1)) csq[gj0 + q4 * 16 + col] = s[0];
                        }
                    }
                    if (C) {
                        // fp32 block: 32 rows x 256 bytes, 16-byte chunks swizzled by (row & 7)
#pragma unroll
                        for (int ch = 0; ch < 16; ++ch)
                            *reinterpret_cast<float4*>(stg + lane * 256 + ((ch ^ (lane & 7)) << 4)) =
                                make_float4(f[4 * ch], f[4 * ch + 1], f[4 * ch + 2], f[4 * ch + 3]);
                        __syncwarp();
#pragma unroll
                        for (int it = 0; it < 16; ++it) {
                            const int r = it * 2 + lane / 16, ch = lane % 16;
                            const float4 x = *reinterpret_cast<const float4*>(stg + r * 256 + ((ch ^ (r & 7)) << 4));
                            if (gi0 + r < g.Mrows && ch * 4 < valid)
                                *reinterpret_cast<float4*>(C + (gi0 + r) * g.out.ld + gj0 + ch * 4) = x;
                        }
                        __syncwarp();
                    }
                    if (to_img) {
                        // the two bf16 planes together (4 KB each in the staging buffer), then the fp16 plane
                        const int panel = gj0 / 64;
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch) {
                            const float fv[8] = {f[8 * ch], f[8 * ch + 1], f[8 * ch + 2], f[8 * ch + 3],
                                                 f[8 * ch + 4], f[8 * ch + 5], f[8 * ch + 6], f[8 * ch + 7]};
                            uint4 t0, t1;
                            split8(fv, t0, t1);
                            const int o = lane * 128 + img_chunk_offset(lane, ch);
                            *reinterpret_cast<uint4*>(stg + o) = t0;
                            *reinterpret_cast<uint4*>(stg + 4096 + o) = t1;
                        }
                        __syncwarp();
                        unsigned char* dst0 = scr + img_row_offset(d.img, 0, panel, gi0);
                        unsigned char* dst1 = scr + img_row_offset(d.img, 1, panel, gi0);
#pragma unroll
                        for (int it = 0; it < 8; ++it) {
                            *reinterpret_cast<uint4*>(dst0 + it * 512 + lane * 16) =
                                *reinterpret_cast<const uint4*>(stg + it * 512 + lane * 16);
                            *reinterpret_cast<uint4*>(dst1 + it * 512 + lane * 16) =
                                *reinterpret_cast<const uint4*>(stg + 4096 + it * 512 + lane * 16);
                        }
                        __syncwarp();
                        if (d.img.planes == 3) {
#pragma unroll
                            for (int ch = 0; ch < 8; ++ch) {
                                const float fv[8] = {f[8 * ch], f[8 * ch + 1], f[8 * ch + 2], f[8 * ch + 3],
                                                     f[8 * ch + 4], f[8 * ch + 5], f[8 * ch + 6], f[8 * ch + 7]};
                                *reinterpret_cast<uint4*>(stg + lane * 128 + img_chunk_offset(lane, ch)) = half8(fv, 1.f);
                            }
                            __syncwarp();
                            unsigned char* dst2 = scr + img_row_offset(d.img, 2, panel, gi0);
#pragma unroll
                            for (int it = 0; it < 8; ++it)
                                *reinterpret_cast<uint4*>(dst2 + it * 512 + lane * 16) =
                                    *reinterpret_cast<const uint4*>(stg + it * 512 + lane * 16);
                            __syncwarp();
                        }
                    }
                }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) { if (PAIR) mbar_arrive_remote(tempty_ld + 8 * acc); else mbar_arrive(tempty0 + 8 * acc); }
                if (++acc == g.acc_bufs) { acc = 0; acc_phase ^= 1; }
            }
        } else {
            // Fused error feedback and weight update.  Warp (quarter, half) owns rows
            // 32*quarter.. of the tile and columns 64*half.., in two slabs of 32 x 32.  The two
            // accumulator slabs go through a swizzled staging block so that global accesses run
            // along rows (8 lanes x 16 bytes per row).
            const int half = (warp - 2) / 4;
            auto next_tile = [&](int t) {
                for (t += tstride; t < g.total_tiles; t += tstride)
                    if (decode_tile<EPI>(batch, g, t, scache, crank).active) return t;
                return g.total_tiles;
            };
            // the slabs of this warp in order: (tile, 0), (tile, 1), (next tile, 0), ...
            auto advance = [&](int& t, int& slab) {
                if (++slab == 2) { slab = 0; t = next_tile(t); }
            };
            if constexpr (XG == 3) {
                // bf16 G and X.  The 32 x 32 slabs of M, G, X come in by asynchronous copies
                // (cp.async, no registers) into a per-warp buffer, one or two slabs ahead; each
                // lane then updates its own row in place (accumulators stay in the layout tensor
                // memory gives: one row per lane), and the buffer goes out along rows.
                //   buffer: M 32 x 128 B | G 32 x 64 B | X 32 x 64 B, 16-byte chunks swizzled so that
                //   both the row-per-lane and the 8-(or 4-)lanes-per-row accesses avoid bank conflicts
                const int nbuf = g.epi_bufs;
                unsigned char* bufs = staging + (size_t)(warp - 2) * nbuf * STAGING_BYTES_PER_WARP;
                const int mrow = lane / 8, mch = lane % 8;      // M: 4 rows x 8 chunks per step
                const int hrow = lane / 4, hch = lane % 4;      // G, X: 8 rows x 4 chunks per step
                auto m_off = [](int r, int ch) { return r * 128 + ((ch ^ (r & 7)) << 4); };
                auto h_off = [](int r, int ch) { return r * 64 + ((ch ^ ((r >> 1) & 3)) << 4); };
                auto issue = [&](int t, int slab, unsigned char* buf) {
                    const TileCoord c = decode_tile<EPI>(batch, g, t, scache, crank);
                    const MatWork& w = batch.w[c.b];
                    const int64_t gj0 = (int64_t)c.n0 + half * 64 + slab * 32;
                    const int64_t gi0 = (int64_t)c.mt * BM + quarter * 32;
                    const uint32_t sb = smem_u32(buf);
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int r = it * 4 + mrow;
                        const int64_t gi = gi0 + r, gj = gj0 + mch * 4;
                        if (gi < g.Mrows && gj < g.Ncols) cp_async16(sb + m_off(r, mch), w.M + gi * g.ld + gj);
                    }
#pragma unroll
                    for (int it = 0; it < 4; ++it) {
                        const int r = it * 8 + hrow;
                        const int64_t gi = gi0 + r, gj = gj0 + hch * 8;
                        if (gi < g.Mrows && gj < g.Ncols) {
                            const int64_t idx = gi * g.ld + gj;
                            cp_async16(sb + 4096 + h_off(r, hch), reinterpret_cast<const __nv_bfloat16*>(w.G) + idx);
                            cp_async16(sb + 6144 + h_off(r, hch), reinterpret_cast<const __nv_bfloat16*>(w.X) + idx);
                        }
                    }
                    cp_async_commit();
                };
                auto process = [&](int t, int slab, unsigned char* buf) -> bool {
                    const TileCoord c = decode_tile<EPI>(batch, g, t, scache, crank);
                    const MatWork& w = batch.w[c.b];
                    const float efb = g.fp16 ? g.ef_b * *reinterpret_cast<const float*>(w.scratch + g.rscale_off) : g.ef_b;
                    if (slab == 0) {
                        if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) return false;
                        tc_fence_after();
                    }
                    const uint32_t taddr = tmem_base + acc * acc_stride + ((uint32_t)(quarter * 32) << 16) +
                                           (uint32_t)(half * 64 + slab * 32);
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        uint32_t va[16], vc[16];
                        tmem_ld16(taddr + hh * 16, va);
                        tmem_ld16(taddr + g.BN + hh * 16, vc);
                        tmem_ld_wait();
                        uint4 gq[2], xq[2];
#pragma unroll
                        for (int k = 0; k < 2; ++k) {
                            gq[k] = *reinterpret_cast<const uint4*>(buf + 4096 + h_off(lane, hh * 2 + k));
                            xq[k] = *reinterpret_cast<const uint4*>(buf + 6144 + h_off(lane, hh * 2 + k));
                        }
                        const uint32_t gw[8] = {gq[0].x, gq[0].y, gq[0].z, gq[0].w, gq[1].x, gq[1].y, gq[1].z, gq[1].w};
                        const uint32_t xw[8] = {xq[0].x, xq[0].y, xq[0].z, xq[0].w, xq[1].x, xq[1].y, xq[1].z, xq[1].w};
                        uint32_t xo[8];
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            float4* mp = reinterpret_cast<float4*>(buf + m_off(lane, hh * 4 + k));
                            const float4 mv = *mp;
                            const float mvv[4] = {mv.x, mv.y, mv.z, mv.w};
                            float mo[4], xf[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int i = 4 * k + e;
                                const uint32_t gp = gw[i / 2], xp = xw[i / 2];
                                const float gval = (i & 1) ? bf16hi_to_f32(gp) : bf16lo_to_f32(gp);
                                const float xval = (i & 1) ? bf16hi_to_f32(xp) : bf16lo_to_f32(xp);
                                const float bval = mvv[e] + gval;
                                mo[e] = g.ef_a * bval - efb * __uint_as_float(va[i]);
                                xf[e] = g.wc * xval - g.wd * __uint_as_float(vc[i]);
                            }
                            *mp = make_float4(mo[0], mo[1], mo[2], mo[3]);
                            xo[2 * k] = pack_bf16x2(xf[0], xf[1]);
                            xo[2 * k + 1] = pack_bf16x2(xf[2], xf[3]);
                        }
#pragma unroll
                        for (int k = 0; k < 2; ++k)
                            *reinterpret_cast<uint4*>(buf + 6144 + h_off(lane, hh * 2 + k)) =
                                make_uint4(xo[4 * k], xo[4 * k + 1], xo[4 * k + 2], xo[4 * k + 3]);
                    }
                    if (slab == 1) {
                        // the accumulators of this tile are in registers / shared memory now
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) { if (PAIR) mbar_arrive_remote(tempty_ld + 8 * acc); else mbar_arrive(tempty0 + 8 * acc); }
                        if (++acc == g.acc_bufs) { acc = 0; acc_phase ^= 1; }
                    }
                    __syncwarp();
                    const int64_t gj0 = (int64_t)c.n0 + half * 64 + slab * 32;
                    const int64_t gi0 = (int64_t)c.mt * BM + quarter * 32;
#pragma unroll
                    for (int it = 0; it < 8; ++it) {
                        const int r = it * 4 + mrow;
                        const int64_t gi = gi0 + r, gj = gj0 + mch * 4;
                        if (gi < g.Mrows && gj < g.Ncols)
                            *reinterpret_cast<float4*>(w.M + gi * g.ld + gj) = *reinterpret_cast<const float4*>(buf + m_off(r, mch));
                    }
#pragma unroll
                    for (int it = 0; it < 4; ++it) {
                        const int r = it * 8 + hrow;
                        const int64_t gi = gi0 + r, gj = gj0 + hch * 8;
                        if (gi < g.Mrows && gj < g.Ncols)
                            *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(w.X) + gi * g.ld + gj) =
                                *reinterpret_cast<const uint4*>(buf + 6144 + h_off(r, hch));
                    }
                    __syncwarp();
                    return true;
                };
                int t = next_tile(tile0 - tstride), slab = 0, ib = 0;
                if (t < g.total_tiles) issue(t, slab, bufs);
                while (t < g.total_tiles) {
                    int t2 = t, slab2 = slab;
                    advance(t2, slab2);
                    if (nbuf == 2) {
                        if (t2 < g.total_tiles) issue(t2, slab2, bufs + (ib ^ 1) * STAGING_BYTES_PER_WARP);
                        else cp_async_commit();
                        cp_async_wait<1>();
                    } else {
                        cp_async_wait<0>();
                    }
                    __syncwarp();
                    if (!process(t, slab, bufs + ib * STAGING_BYTES_PER_WARP)) break;
                    if (nbuf == 2) ib ^= 1;
                    else if (t2 < g.total_tiles) issue(t2, slab2, bufs);
                    t = t2; slab = slab2;
                }
                cp_async_wait<0>();
            } else {
            unsigned char* S1 = staging + (warp - 2) * STAGING_BYTES_PER_WARP;
            unsigned char* S2 = S1 + 4096;
            const int rl = lane / 8, cq = lane % 8;      // row within a step, 4-column group

            auto fetch = [&](K5Pre<XG>& p, int t, int slab) {
                const TileCoord c = decode_tile<EPI>(batch, g, t, scache, crank);
                const MatWork& w = batch.w[c.b];
                const int64_t gj = (int64_t)c.n0 + half * 64 + slab * 32 + cq * 4;
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const int64_t gi = (int64_t)c.mt * BM + quarter * 32 + it * 4 + rl;
                    if (gi < g.Mrows && gj < g.Ncols) {
                        const int64_t idx = gi * g.ld + gj;
                        p.m[it] = *reinterpret_cast<const float4*>(w.M + idx);
                        if constexpr (G_BF16) {
                            const uint2 u = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(w.G) + idx);
                            p.g[it][0] = u.x; p.g[it][1] = u.y;
                        } else {
                            const uint4 u = *reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(w.G) + idx);
                            p.g[it][0] = u.x; p.g[it][1] = u.y; p.g[it][2] = u.z; p.g[it][3] = u.w;
                        }
                        if constexpr (X_BF16) {
                            const uint2 u = *reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(w.X) + idx);
                            p.x[it][0] = u.x; p.x[it][1] = u.y;
                        } else {
                            const uint4 u = *reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(w.X) + idx);
                            p.x[it][0] = u.x; p.x[it][1] = u.y; p.x[it][2] = u.z; p.x[it][3] = u.w;
                        }
                    }
                }
            };

            // one slab: accumulators -> staging -> row-wise update of M and X
            auto process = [&](const K5Pre<XG>& cur, int t, int slab) -> bool {
                const TileCoord c = decode_tile<EPI>(batch, g, t, scache, crank);
                const MatWork& w = batch.w[c.b];
                const float efb = g.fp16 ? g.ef_b * *reinterpret_cast<const float*>(w.scratch + g.rscale_off) : g.ef_b;
                if (slab == 0) {
                    if (!mbar_wait(tfull0 + 8 * acc, acc_phase, abort_flag)) return false;
                    tc_fence_after();
                }
                const uint32_t taddr = tmem_base + acc * acc_stride + ((uint32_t)(quarter * 32) << 16) +
                                       (uint32_t)(half * 64 + slab * 32);
                {
                    uint32_t va[16], vb[16], vc[16], vd[16];
                    tmem_ld16(taddr, va);
                    tmem_ld16(taddr + 16, vb);
                    tmem_ld16(taddr + g.BN, vc);
                    tmem_ld16(taddr + g.BN + 16, vd);
                    tmem_ld_wait();
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        const int o0 = lane * 128 + img_chunk_offset(lane, ch);
                        const int o1 = lane * 128 + img_chunk_offset(lane, ch + 4);
                        *reinterpret_cast<uint4*>(S1 + o0) = make_uint4(va[4 * ch], va[4 * ch + 1], va[4 * ch + 2], va[4 * ch + 3]);
                        *reinterpret_cast<uint4*>(S1 + o1) = make_uint4(vb[4 * ch], vb[4 * ch + 1], vb[4 * ch + 2], vb[4 * ch + 3]);
                        *reinterpret_cast<uint4*>(S2 + o0) = make_uint4(vc[4 * ch], vc[4 * ch + 1], vc[4 * ch + 2], vc[4 * ch + 3]);
                        *reinterpret_cast<uint4*>(S2 + o1) = make_uint4(vd[4 * ch], vd[4 * ch + 1], vd[4 * ch + 2], vd[4 * ch + 3]);
                    }
                }
                __syncwarp();
                const int64_t gj = (int64_t)c.n0 + half * 64 + slab * 32 + cq * 4;
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const int r = it * 4 + rl;
                    const int64_t gi = (int64_t)c.mt * BM + quarter * 32 + r;
                    const int o = r * 128 + img_chunk_offset(r, cq);
                    const float4 d1 = *reinterpret_cast<const float4*>(S1 + o);
                    const float4 d2 = *reinterpret_cast<const float4*>(S2 + o);
                    if (gi < g.Mrows && gj < g.Ncols) {
                        const int64_t idx = gi * g.ld + gj;
                        float gv[4], xv[4];
                        if constexpr (G_BF16) {
                            gv[0] = bf16lo_to_f32(cur.g[it][0]); gv[1] = bf16hi_to_f32(cur.g[it][0]);
                            gv[2] = bf16lo_to_f32(cur.g[it][1]); gv[3] = bf16hi_to_f32(cur.g[it][1]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e) gv[e] = __uint_as_float(cur.g[it][e]);
                        }
                        if constexpr (X_BF16) {
                            xv[0] = bf16lo_to_f32(cur.x[it][0]); xv[1] = bf16hi_to_f32(cur.x[it][0]);
                            xv[2] = bf16lo_to_f32(cur.x[it][1]); xv[3] = bf16hi_to_f32(cur.x[it][1]);
                        } else {
#pragma unroll
                            for (int e = 0; e < 4; ++e) xv[e] = __uint_as_float(cur.x[it][e]);
                        }
                        const float mv[4] = {cur.m[it].x, cur.m[it].y, cur.m[it].z, cur.m[it].w};
                        const float a1[4] = {d1.x, d1.y, d1.z, d1.w};
                        const float a2[4] = {d2.x, d2.y, d2.z, d2.w};
                        float mo[4], xo[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float bval = mv[e] + gv[e];
                            mo[e] = g.ef_a * bval - efb * a1[e];
                            xo[e] = g.wc * xv[e] - g.wd * a2[e];
                        }
                        *reinterpret_cast<float4*>(w.M + idx) = make_float4(mo[0], mo[1], mo[2], mo[3]);
                        if constexpr (X_BF16) {
                            *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(w.X) + idx) =
                                make_uint2(pack_bf16x2(xo[0], xo[1]), pack_bf16x2(xo[2], xo[3]));
                        } else {
                            *reinterpret_cast<float4*>(reinterpret_cast<float*>(w.X) + idx) =
                                make_float4(xo[0], xo[1], xo[2], xo[3]);
                        }
                    }
                }
                __syncwarp();
                if (slab == 1) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) { if (PAIR) mbar_arrive_remote(tempty_ld + 8 * acc); else mbar_arrive(tempty0 + 8 * acc); }
                    if (++acc == g.acc_bufs) { acc = 0; acc_phase ^= 1; }
                }
                return true;
            };
            int t = next_tile(tile0 - tstride), slab = 0;
            K5Pre<XG> pa;
            while (t < g.total_tiles) {
                fetch(pa, t, slab);
                if (!process(pa, t, slab)) break;
                advance(t, slab);
            }
            }
        }
    } else if (A_BUF) {
        // ---------------- transform warps: A tile of B = M + G (Alg. 1, buffer step) ----------------
        // 512 threads, two 8-element chunks each per 128 x 64 tile; the loads of the next two
        // tiles are in flight while the current one is split and stored.
        const int xt = threadIdx.x - 32 * (2 + NE);     // 0 .. 511
        int as = 0; uint32_t aph = 0;
        bool ok = true;
        struct Raw { float4 m[2][2]; uint32_t gq[2][G_BF16 ? 4 : 8]; };
        for (int t = tile0; t < g.total_tiles && ok; t += tstride) {
            const TileCoord c = decode_tile<EPI>(batch, g, t, scache, crank);
            if (!c.active) continue;
            const MatWork& w = batch.w[c.b];
            const int64_t ld = g.ld;
            int64_t src_idx[2]; bool row_ok[2]; int kofs[2]; uint32_t dst_off[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int q = xt + 512 * e;
                if (AMODE == A_BUF_ROW) {
                    // operand row = B row, depth = B column: chunk (rho, ch) = B[i0+rho][k0+8ch .. +7]
                    const int rho = q / 8, ch = q % 8;
                    const int64_t gr = (int64_t)c.mt * BM + rho;
                    row_ok[e] = gr < g.Mrows;
                    src_idx[e] = gr * ld + ch * 8;           // + k0
                    kofs[e] = ch * 8;
                    dst_off[e] = rho * 128 + img_chunk_offset(rho, ch);
                } else {
                    // operand row = B column, depth = B row (MN-major tile):
                    // chunk (k, cj) = B[k0+k][j0+8cj .. +7]
                    const int k = q / 16, cj = q % 16;
                    const int64_t gc = (int64_t)c.mt * BM + cj * 8;
                    row_ok[e] = gc < g.Mrows;                // Mrows = number of B columns, a multiple of 8
                    src_idx[e] = (int64_t)k * ld + gc;       // + k0 * ld
                    kofs[e] = k;
                    dst_off[e] = (cj / 8) * 8192 + k * 128 + img_chunk_offset(k, cj % 8);
                }
            }
            auto fetch = [&](Raw& r, int kb) {
                const int64_t k0 = (int64_t)kb * BK;
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const bool okk = row_ok[e] && (k0 + kofs[e] < g.Kdim);
                    if (okk) {
                        const int64_t idx = src_idx[e] + (AMODE == A_BUF_ROW ? k0 : k0 * ld);
                        const float4* mp = reinterpret_cast<const float4*>(w.M + idx);
                        r.m[e][0] = mp[0]; r.m[e][1] = mp[1];
                        if constexpr (G_BF16) {
                            const uint4 u = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(w.G) + idx);
                            r.gq[e][0] = u.x; r.gq[e][1] = u.y; r.gq[e][2] = u.z; r.gq[e][3] = u.w;
                        } else {
                            const uint4* gp = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(w.G) + idx);
                            const uint4 u0 = gp[0], u1 = gp[1];
                            r.gq[e][0] = u0.x; r.gq[e][1] = u0.y; r.gq[e][2] = u0.z; r.gq[e][3] = u0.w;
                            r.gq[e][4] = u1.x; r.gq[e][5] = u1.y; r.gq[e][6] = u1.z; r.gq[e][7] = u1.w;
                        }
                    } else {
                        r.m[e][0] = r.m[e][1] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                        for (int i = 0; i < (G_BF16 ? 4 : 8); ++i) r.gq[e][i] = 0u;
                    }
                }
            };
            // split the tile held in r into the two bf16 terms
            auto split_raw = [&](const Raw& r, uint4 (&t0)[2], uint4 (&t1)[2]) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    float gv[8];
                    if constexpr (G_BF16) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) { gv[2 * i] = bf16lo_to_f32(r.gq[e][i]); gv[2 * i + 1] = bf16hi_to_f32(r.gq[e][i]); }
                    } else {
#pragma unroll
                        for (int i = 0; i < 8; ++i) gv[i] = __uint_as_float(r.gq[e][i]);
                    }
                    const float v[8] = {r.m[e][0].x + gv[0], r.m[e][0].y + gv[1], r.m[e][0].z + gv[2], r.m[e][0].w + gv[3],
                                        r.m[e][1].x + gv[4], r.m[e][1].y + gv[5], r.m[e][1].z + gv[6], r.m[e][1].w + gv[7]};
                    split8(v, t0[e], t1[e]);
                }
            };
            // wait for the slot, store the tile, signal the MMA issuer
            auto store = [&](const uint4 (&t0)[2], const uint4 (&t1)[2]) -> bool {
                if (!mbar_wait(a_empty0 + 8 * as, aph ^ 1, abort_flag)) return false;
                unsigned char* sa = a_ring + as * g.a_slot_bytes;
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    *reinterpret_cast<uint4*>(sa + dst_off[e]) = t0[e];
                    *reinterpret_cast<uint4*>(sa + A_TERM_BYTES + dst_off[e]) = t1[e];
                }
                fence_async_smem();
                __syncwarp();
                if (lane == 0) { if (PAIR) mbar_arrive_remote(a_full_ld + 8 * as); else mbar_arrive(a_full0 + 8 * as); }
                if (++as == g.a_slots) { as = 0; aph ^= 1; }
                return true;
            };
            Raw r0, r1;
            fetch(r0, c.kb_begin);
            if (c.kb_begin + 1 < c.kb_end) fetch(r1, c.kb_begin + 1);
            for (int kb = c.kb_begin; kb < c.kb_end && ok; kb += 2) {
                uint4 t0[2], t1[2];
                split_raw(r0, t0, t1);
                if (kb + 2 < c.kb_end) fetch(r0, kb + 2);
                if (!store(t0, t1)) { ok = false; break; }
                if (kb + 1 < c.kb_end) {
                    split_raw(r1, t0, t1);
                    if (kb + 3 < c.kb_end) fetch(r1, kb + 3);
                    if (!store(t0, t1)) { ok = false; break; }
                }
            }
        }
    }

    // ---------------- teardown ----------------
    // A role that gave up on a bounded wait leaves bulk copies into this CTA's shared memory and
    // issued MMAs possibly still in flight.  Nothing more is issued once the flag is up, so a fixed
    // pause far longer than any copy or MMA takes (about a millisecond) lets them land before the
    // shared memory and the tensor memory are given back.
    if (*abort_flag) {
        const long long t0 = clock64();
        while (clock64() - t0 < 2000000LL) {}
    }
    tc_fence_before();
    __syncthreads();
    // pairs: neither CTA leaves (or frees tensor memory) while the other may still reach its barriers
    if (PAIR) cluster_sync_all();
    tc_fence_after();
    if (*abort_flag && threadIdx.x == 0) {
        for (int b = 0; b < batch.count; ++b) atomicOr(batch.w[b].status, ST_WAIT);
    }
    if (warp == 1) {
        if (PAIR) tmem_dealloc_pair(tmem_base, (uint32_t)g.tmem_cols);
        else tmem_dealloc(tmem_base, (uint32_t)g.tmem_cols);
    }
}

}  // namespace tc

// ------------------------------------------------------------------------------------------
// Host side of the engine
// ------------------------------------------------------------------------------------------
struct TensorScratch {      // where the images of one matrix live inside its scratch area
    ImgRef linv;            // (L^{-1})^T of the current Cholesky        (r x r)
    ImgRef qprev;           // Q_prev                                    (n x r)
    ImgRef w0, w1;          // Y = B Q_prev and the QR intermediates     (max(m,n) x r)
    ImgRef p, r, q;         // P (m x r), R (n x r), Q (n x r); three planes when the fused pass runs in fp16
    int64_t colsq;          // fp32 [4 * ceil(max(m,n)/128)][r] column-square partials
    int64_t cnorm;          // fp32 [r] squared column norms of R
    int64_t rscale;         // fp32 inverse of the scale of R's fp16 plane
};

inline bool tensor_engine_supports(int64_t m, int64_t n, int32_t r) {
    return r % 16 == 0 && n % 8 == 0 && m >= 1;
}

inline ImgRef make_img(int64_t off, int64_t rows, int64_t cols, int planes = 2) {
    ImgRef im;
    im.off = off;
    im.rows_pad = (int32_t)((rows + 127) / 128 * 128);
    im.panels = (int32_t)((cols + 63) / 64);
    im.planes = planes;
    im.pad = 0;
    return im;
}
inline int64_t img_bytes(int64_t rows, int64_t cols, int planes = 2) {
    return planes * ((cols + 63) / 64) * ((rows + 127) / 128 * 128) * 128;
}
inline ImgRef no_img() { ImgRef im; im.off = -1; im.rows_pad = 0; im.panels = 0; im.planes = 0; im.pad = 0; return im; }

// The offsets of linv, cnorm, rscale and colsq depend on r only (everything whose size depends on
// the matrix shape comes after them), so that one Cholesky launch can serve matrices of
// different shapes.
// half_planes: P, R, Q carry the fp16 plane (fused pass in fp16).
inline size_t tensor_scratch_layout(int64_t m, int64_t n, int32_t r, bool half_planes, size_t off, TensorScratch* ts) {
    const int64_t kmax = std::max(m, n);
    off = (off + 1023) / 1024 * 1024;
    auto take = [&](int64_t bytes) { int64_t o = (int64_t)off; off += (size_t)((bytes + 1023) / 1024 * 1024); return o; };
    ts->linv = make_img(take(img_bytes(r, r)), r, r);
    ts->cnorm = take((int64_t)r * 4);
    ts->rscale = take(16);
    ts->colsq = take(4 * ((kmax + 127) / 128) * (int64_t)r * 4);
    const int pl = half_planes ? 3 : 2;
    ts->w0 = make_img(take(img_bytes(kmax, r)), kmax, r);
    ts->w1 = make_img(take(img_bytes(kmax, r)), kmax, r);
    // the image of Q_prev is read by the first product of a step only; w1 is first written after
    // it (first apply of the left QR, same stream): they share their bytes
    ts->qprev = make_img(ts->w1.off, n, r);
    ts->p = make_img(take(img_bytes(m, r, pl)), m, r, pl);
    ts->r = make_img(take(img_bytes(n, r, pl)), n, r, pl);
    ts->q = make_img(take(img_bytes(n, r, pl)), n, r, pl);
    return off;
}
// the work images are sized for max(m, n) rows; a product over `rows` rows sees this view
inline ImgRef img_view(const ImgRef& im, int64_t rows) {
    ImgRef v = im;
    v.rows_pad = (int32_t)((rows + 127) / 128 * 128);
    return v;
}

// cuTensorMapEncodeTiled, fetched through the runtime so that the library does not link libcuda.
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                      const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                      CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
inline TensorMapEncodeFn tensor_map_encoder() {
    static TensorMapEncodeFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<TensorMapEncodeFn>(p);
    }
    return fn;
}
// First error met while preparing launches of the current step call (0 = none); one per host
// thread, so that concurrent step calls do not see each other's.
inline int& engine_error() { static thread_local int e = 0; return e; }

// 5-d map over the images `img` of all matrices of a batch: (64 bf16, rows, panels, terms, matrix),
// with the box (64, box_rows, box_panels, box_terms, 1).  The images are stored pre-swizzled, so
// the copy itself does not swizzle; out-of-range parts of a box read as zeros.
inline void encode_img_map(CUtensorMap* map, const Batch& b, const ImgRef& img, int box_rows, int box_panels,
                           int box_terms) {
    TensorMapEncodeFn enc = tensor_map_encoder();
    if (!enc) { engine_error() = 1; return; }
    const cuuint64_t term_bytes = (cuuint64_t)img.panels * img.rows_pad * 128;
    cuuint64_t dims[5] = {64, (cuuint64_t)img.rows_pad, (cuuint64_t)img.panels, (cuuint64_t)img.planes,
                          (cuuint64_t)b.count};
    cuuint64_t strides[4] = {128, (cuuint64_t)img.rows_pad * 128, term_bytes,
                             b.count > 1 ? (cuuint64_t)b.scratch_stride : img.planes * term_bytes};
    cuuint32_t box[5] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_panels, (cuuint32_t)box_terms, 1};
    cuuint32_t estr[5] = {1, 1, 1, 1, 1};
    void* base = b.w[0].scratch + img.off;
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, base, dims, strides, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        std::fprintf(stderr, "orthdion: cuTensorMapEncodeTiled failed (%d)\n", (int)r);
        engine_error() = 2;
    }
}

// Multiprocessor count of the current device (looked up once per device ordinal).
constexpr int kMaxDevices = 64;
inline int sm_count() {
    static std::atomic<int> cached[kMaxDevices] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= kMaxDevices) dev = 0;
    int n = cached[dev].load(std::memory_order_relaxed);
    if (n <= 0) {
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
        cached[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

// Which instantiations exist as CTA-pair kernels: every product with an MN-major N-side (the two
// products with B, Gram, apply) and the fused pass on bf16 G and X in its single-term form, where
// the leader loads the R pieces and the peer the Q pieces (operand bytes per element 24 -> 16).
constexpr bool pair_capable(int nmode, int epi, int xg) {
    return nmode == tc::N_IMG_MN || (epi == tc::EPI_K5 && xg == 3);
}

template <int AMODE, int NMODE, int EPI, int XG>
inline cudaError_t set_gemm_attr() {
    cudaError_t e = cudaFuncSetAttribute(tc::gemm_kernel<AMODE, NMODE, EPI, XG, false>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_LIMIT);
    if constexpr (pair_capable(NMODE, EPI, XG)) {
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(tc::gemm_kernel<AMODE, NMODE, EPI, XG, true>,
                                     cudaFuncAttributeMaxDynamicSharedMemorySize, tc::SMEM_LIMIT);
    }
    return e;
}

inline cudaError_t tensor_engine_set_attributes() {
    cudaError_t e;
#define OD_SET(...) if ((e = set_gemm_attr<__VA_ARGS__>()) != cudaSuccess) return e;
    OD_SET(tc::A_BUF_ROW, tc::N_IMG_MN, tc::EPI_STORE, 0)
    OD_SET(tc::A_BUF_ROW, tc::N_IMG_MN, tc::EPI_STORE, 1)
    OD_SET(tc::A_BUF_COL, tc::N_IMG_MN, tc::EPI_STORE, 0)
    OD_SET(tc::A_BUF_COL, tc::N_IMG_MN, tc::EPI_STORE, 1)
    OD_SET(tc::A_IMG_MN, tc::N_IMG_MN, tc::EPI_STORE, 0)
    OD_SET(tc::A_IMG_K, tc::N_IMG_MN, tc::EPI_STORE, 0)
    OD_SET(tc::A_IMG_K, tc::N_IMG_K, tc::EPI_K5, 0)
    OD_SET(tc::A_IMG_K, tc::N_IMG_K, tc::EPI_K5, 1)
    OD_SET(tc::A_IMG_K, tc::N_IMG_K, tc::EPI_K5, 2)
    OD_SET(tc::A_IMG_K, tc::N_IMG_K, tc::EPI_K5, 3)
#undef OD_SET
    return cudaSuccess;
}

inline void launch_pack_half(const Batch& b, int64_t rows, int64_t cols, const TensorScratch& ts, cudaStream_t st) {
    tc::PackHalfArgs a{};
    a.rows = (int32_t)rows; a.cols = (int32_t)cols; a.dst = ts.r; a.cnorm_off = ts.cnorm; a.rscale_off = ts.rscale;
    dim3 grid((unsigned)ts.r.panels, (unsigned)(ts.r.rows_pad / 128), (unsigned)b.count);
    prof::Scope scope(prof::S_PACK, st);
    tc::pack_half_kernel<<<grid, 256, 0, st>>>(b, a);
}

inline void launch_pack(const Batch& b, Sel src, int64_t rows, int64_t cols, ImgRef dst, cudaStream_t st) {
    tc::PackArgs a{};
    a.src = src; a.rows = (int32_t)rows; a.cols = (int32_t)cols; a.dst = dst;
    dim3 grid((unsigned)dst.panels, (unsigned)(dst.rows_pad / 128), (unsigned)b.count);
    prof::Scope scope(prof::S_PACK, st);
    tc::pack_kernel<<<grid, 256, 0, st>>>(b, a);
}

// Fills in the tiling, ring and tensor-memory fields and launches.
template <int AMODE, int NMODE, int EPI, int XG>
inline void launch_gemm(const Batch& b, tc::GemmArgs g, int stage, cudaStream_t st) {
    if (g.fp16) { g.passes = 1; g.passes2 = 1; }
    // CTA pairs need full 256-column instructions: every tile 256 or 512 columns wide (MN-major
    // N-side), or the fused pass in its single-term form with full 128-column tiles.
    bool pair = false;
    if constexpr (pair_capable(NMODE, EPI, XG)) {
        if (NMODE == tc::N_IMG_MN) pair = g.BN % 256 == 0 && g.Ncols % g.BN == 0;
        else pair = g.passes == 1 && g.passes2 == 1 && g.BN == 128 && g.Ncols % 128 == 0;
        if (sm_count() < 2) pair = false;
    }
    g.pair = pair ? 1 : 0;
    g.m_tiles = (g.Mrows + tc::BM - 1) / tc::BM;
    if (pair) g.m_tiles = (g.m_tiles + 1) / 2;      // scheduled row tiles of 256 rows
    g.n_tiles = (g.Ncols + g.BN - 1) / g.BN;
    g.k_blocks = (g.Kdim + tc::BK - 1) / tc::BK;
    if (g.ksplit < 1) g.ksplit = 1;
    if (g.ksplit > 1) g.kb_per_chunk = (g.k_blocks + g.ksplit - 1) / g.ksplit;
    g.total_tiles = b.count * g.m_tiles * g.n_tiles * g.ksplit;
    const int n1_terms = g.passes == 3 ? 2 : 1, n2_terms = g.passes2 == 3 ? 2 : 1;
    const int bn64 = (g.BN + 63) / 64 * 64;
    const int a_terms = (tc::a_is_buf(AMODE) || g.passes == 3 || (EPI == tc::EPI_K5 && g.passes2 == 3)) ? 2 : 1;
    g.a_slot_bytes = a_terms * tc::A_TERM_BYTES;
    g.a_slots = tc::A_RING_BYTES / g.a_slot_bytes;
    // image-to-image products: a third two-term slot (the N ring then holds three pieces as well)
    if (EPI == tc::EPI_STORE && !tc::a_is_buf(AMODE)) g.a_slots = std::min(tc::MAX_A_SLOTS, 6 * tc::A_TERM_BYTES / g.a_slot_bytes);
    g.epi_bufs = 1;
    if (EPI == tc::EPI_K5) {
        // the fused pass: 64 KB of A slots (four single-term ones or two two-term ones) and one
        // epilogue buffer per warp (a second one, paid for with ring slots, measured slower)
        g.a_slots = (a_terms == 1) ? 4 : 2;
    }
    if (NMODE == tc::N_IMG_MN) {
        if (pair) {
            // each CTA holds half of the columns: same bytes per piece at twice the depth
            g.ks = bn64 <= 256 ? 64 : 32;
            g.n_piece_bytes = n1_terms * (bn64 / 128) * g.ks * 128;
        } else {
            g.ks = bn64 <= 128 ? 64 : (bn64 <= 256 ? 32 : 16);
            g.n_piece_bytes = n1_terms * (bn64 / 64) * g.ks * 128;
        }
    } else {
        g.ks = 64;
        g.n_piece_bytes = (n1_terms + (EPI == tc::EPI_K5 ? n2_terms : 0)) * tc::A_TERM_BYTES;
        if (pair) g.n_piece_bytes = tc::A_TERM_BYTES;    // the R piece (leader) or the Q piece (peer)
    }
    const int accw = (EPI == tc::EPI_K5) ? 2 * g.BN : g.BN;
    g.acc_bufs = (2 * accw <= 512) ? 2 : 1;
    int cols = 32;
    while (cols < g.acc_bufs * accw) cols *= 2;
    g.tmem_cols = cols;
    const size_t fixed = (size_t)g.a_slots * g.a_slot_bytes +
                         (tc::a_is_buf(AMODE) ? 0 : (size_t)tc::epi_warps(AMODE, EPI) * g.epi_bufs * tc::STAGING_BYTES_PER_WARP) +
                         256 + 1024;
    g.n_slots = (int)std::min<size_t>(tc::MAX_N_SLOTS, (tc::SMEM_LIMIT - fixed) / (size_t)g.n_piece_bytes);
    // more than half of an SM's shared memory: one CTA per SM, whatever its tensor-memory share
    const size_t smem = std::max<size_t>(fixed + (size_t)g.n_slots * g.n_piece_bytes, 120 * 1024);
    if (AMODE == tc::A_IMG_K) encode_img_map(&g.map_a, b, g.a, 128, 1, a_terms);
    else if (AMODE == tc::A_IMG_MN) encode_img_map(&g.map_a, b, g.a, 64, 2, a_terms);
    if (NMODE == tc::N_IMG_MN) encode_img_map(&g.map_n1, b, g.n1, g.ks, pair ? 2 : bn64 / 64, n1_terms);
    else encode_img_map(&g.map_n1, b, g.n1, 128, 1, n1_terms);
    if (EPI == tc::EPI_K5) encode_img_map(&g.map_n2, b, g.n2, 128, 1, n2_terms);
    if (engine_error()) return;
    prof::Scope scope(stage, st);
    if constexpr (pair_capable(NMODE, EPI, XG)) {
        if (pair) {
            cudaLaunchConfig_t cfg{};
            cfg.gridDim = dim3((unsigned)(2 * std::min(g.total_tiles, sm_count() / 2)), 1, 1);
            cfg.blockDim = dim3((unsigned)tc::gemm_threads(AMODE, EPI), 1, 1);
            cfg.dynamicSmemBytes = smem;
            cfg.stream = st;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr; cfg.numAttrs = 1;
            if (cudaLaunchKernelEx(&cfg, tc::gemm_kernel<AMODE, NMODE, EPI, XG, true>, b, g) != cudaSuccess)
                engine_error() = 3;
            return;
        }
    }
    const int grid = std::min(g.total_tiles, sm_count());
    tc::gemm_kernel<AMODE, NMODE, EPI, XG, false><<<grid, tc::gemm_threads(AMODE, EPI), smem, st>>>(b, g);
}

inline tc::Dest dest_none() {
    tc::Dest d{};
    d.f32 = Sel{W_P, 0, 0}; d.img = no_img(); d.has_f32 = 0; d.colsq = 0;
    return d;
}

// Depth split of the two products with the buffer.  With one matrix (or a few) in a call and a
// small rank, the output has too few 256-row tile pairs for the device (16 for a 4096-wide
// factor) and every one of them runs over the whole depth: the depth is cut into chunks that run
// as separate tiles and leave fp32 partial results, which are then added in a fixed order, packed
// into the operand image and given their column squares by small kernels.  Like the split of the
// Gram product, the chunk count depends on the plan only (rank, rows of the result, depth), so a
// matrix gets the same bits alone and in any group; ranks above 256 never split.
inline int buffer_ksplit(int r, int64_t out_rows, int64_t depth) {
    if (r > 256) return 1;
    const int tiles = (int)((out_rows + 255) / 256);
    const int kb = (int)((depth + tc::BK - 1) / tc::BK);
    if (tiles >= 37 || kb < 32) return 1;
    const int want = std::min({8, 74 / tiles, kb / 8});
    if (want < 2) return 1;
    const int per = (kb + want - 1) / want;
    return (kb + per - 1) / per;             // every chunk non-empty
}

__global__ void gram_reduce_kernel(const __grid_constant__ Batch batch, Sel gram, Sel part, int64_t total4, int ksplit,
                                   int only_shift_bit);

// after a depth-split product: dst (rows x r fp32) <- sum of the partials, then its image and its
// column squares per 32-row block
inline void finish_split_product(const Batch& b, Sel dst, Sel part, int64_t rows, int r, int ksplit, ImgRef img,
                                 int64_t colsq_off, int stage, cudaStream_t st) {
    {
        prof::Scope scope(stage, st);
        const int64_t total4 = rows * r / 4;
        dim3 grid((unsigned)((total4 + 255) / 256), 1, (unsigned)b.count);
        gram_reduce_kernel<<<grid, 256, 0, st>>>(b, dst, part, total4, ksplit, 0);
    }
    launch_pack(b, dst, rows, r, img, st);
    {
        prof::Scope scope(stage, st);
        dim3 grid((unsigned)(4 * ((rows + 127) / 128)), (unsigned)((r + 255) / 256), (unsigned)b.count);
        colsq_blocks_kernel<<<grid, 256, 0, st>>>(b, dst, rows, r, colsq_off);
    }
}

// Y = (M + G) Q_prev  -> image w0 (+ column squares)              (Alg. 1, buffer and left-factor steps)
// partial: the columns at hand are one shard of the matrix; the product goes to the fp32 P slot
// only, to be summed over the shards before it is orthonormalised.
// part: scratch for the partial results of a depth split (buffer_ksplit(r, m, n) > 1).
inline void tensor_k1(int64_t m, int64_t n, int r, int g_bf16, int passes, const Batch& b, const TensorScratch& ts,
                      Sel part, cudaStream_t st, bool partial = false) {
    launch_pack(b, Sel{W_Q, 0, 0}, n, r, ts.qprev, st);
    const int ksplit = partial ? 1 : buffer_ksplit(r, m, n);
    tc::GemmArgs g{};
    g.Mrows = (int32_t)m; g.Ncols = r; g.Kdim = (int32_t)n; g.BN = std::min(r, 512);
    g.passes = passes; g.passes2 = 1; g.ld = n; g.n1 = ts.qprev; g.a = no_img(); g.n2 = no_img();
    g.colsq_off = ts.colsq;
    g.out.normal = dest_none();
    if (ksplit > 1) { g.out.normal.f32 = part; g.out.normal.has_f32 = 1; g.ksplit = ksplit; g.split_stride = m * r; }
    else if (partial) { g.out.normal.f32 = Sel{W_P, 0, 0}; g.out.normal.has_f32 = 1; }
    else { g.out.normal.img = img_view(ts.w0, m); g.out.normal.colsq = 1; }
    g.out.shifted = g.out.normal; g.out.ld = r;
    if (g_bf16) launch_gemm<tc::A_BUF_ROW, tc::N_IMG_MN, tc::EPI_STORE, 1>(b, g, prof::S_K1, st);
    else launch_gemm<tc::A_BUF_ROW, tc::N_IMG_MN, tc::EPI_STORE, 0>(b, g, prof::S_K1, st);
    // (the sum goes through the fp32 P slot, which holds nothing yet at this point of a step)
    if (ksplit > 1) finish_split_product(b, Sel{W_P, 0, 0}, part, m, r, ksplit, img_view(ts.w0, m), ts.colsq, prof::S_K1, st);
}

// R = (M + G)^T P  -> fp32 R slot, image r (+ column squares)     (Alg. 1, right-factor step)
inline void tensor_k3(int64_t m, int64_t n, int r, int g_bf16, int passes, const Batch& b, const TensorScratch& ts,
                      Sel part, cudaStream_t st) {
    const int ksplit = buffer_ksplit(r, n, m);
    tc::GemmArgs g{};
    g.Mrows = (int32_t)n; g.Ncols = r; g.Kdim = (int32_t)m; g.BN = std::min(r, 512);
    g.passes = passes; g.passes2 = 1; g.ld = n; g.n1 = ts.p; g.a = no_img(); g.n2 = no_img();
    g.colsq_off = ts.colsq;
    g.out.normal = dest_none(); g.out.normal.has_f32 = 1;
    if (ksplit > 1) { g.out.normal.f32 = part; g.ksplit = ksplit; g.split_stride = n * r; }
    else { g.out.normal.f32 = Sel{W_R, 0, 0}; g.out.normal.img = ts.r; g.out.normal.colsq = 1; }
    g.out.shifted = g.out.normal; g.out.ld = r;
    if (g_bf16) launch_gemm<tc::A_BUF_COL, tc::N_IMG_MN, tc::EPI_STORE, 1>(b, g, prof::S_K3, st);
    else launch_gemm<tc::A_BUF_COL, tc::N_IMG_MN, tc::EPI_STORE, 0>(b, g, prof::S_K3, st);
    if (ksplit > 1) finish_split_product(b, Sel{W_R, 0, 0}, part, n, r, ksplit, ts.r, ts.colsq, prof::S_K3, st);
}

// Depth split of the Gram product.  At small ranks the whole Gram matrix is one output tile whose
// main loop runs over all rows of the tall matrix on a single CTA (pair): the depth is cut into
// chunks that run side by side and leave partial sums, which a small kernel adds up in a fixed
// order.  The number of chunks depends on the rank and the row count only, never on how many
// matrices a launch holds, so a matrix gets the same bits alone and in any group.
inline int gram_ksplit(int r, int64_t rows) {
    if (r > 256) return 1;
    const int kb = (int)((rows + tc::BK - 1) / tc::BK);
    const int want = std::min(16, kb / 8);
    if (want < 2) return 1;
    const int per = (kb + want - 1) / want;
    return (kb + per - 1) / per;             // every chunk non-empty
}

// dst <- sum of the `ksplit` partial results at `part` (4 * total4 floats each, one after the
// other), added in the order of the chunks
__global__ void __launch_bounds__(256)
gram_reduce_kernel(const __grid_constant__ Batch batch, Sel gram, Sel part, int64_t total4, int ksplit, int only_shift_bit) {
    const MatWork& w = batch.w[blockIdx.z];
    const int st = *w.status;
    if ((st & ST_FAILED) || (only_shift_bit && !(st & only_shift_bit))) return;
    const int64_t q = (int64_t)blockIdx.x * 256 + threadIdx.x;      // float4 index
    if (q >= total4) return;
    const float4* P = reinterpret_cast<const float4*>(pick(w, part));
    float4 acc = P[q];
    for (int s2 = 1; s2 < ksplit; ++s2) {
        const float4 v = P[(int64_t)s2 * total4 + q];
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    reinterpret_cast<float4*>(pick(w, gram))[q] = acc;
}

// Gram = src^T src (src: image of a rows x r matrix); only tiles that touch the lower triangle.
// part: scratch for gram_ksplit(r, rows) partial matrices (used when that is more than one).
inline void tensor_gram(int r, int passes, const Batch& b, ImgRef src, int64_t rows, Sel gram, Sel part,
                        int only_shift_bit, cudaStream_t st) {
    const int ksplit = gram_ksplit(r, rows);
    tc::GemmArgs g{};
    g.Mrows = r; g.Ncols = r; g.Kdim = (int32_t)rows; g.BN = std::min(r, 256);
    g.passes = passes; g.passes2 = 1; g.a = src; g.n1 = src; g.n2 = no_img(); g.lower_only = 1;
    g.out.normal = dest_none(); g.out.normal.f32 = ksplit > 1 ? part : gram; g.out.normal.has_f32 = 1;
    g.out.shifted = g.out.normal; g.out.ld = r;
    g.out.shift_bit = only_shift_bit; g.out.only_if_shifted = only_shift_bit ? 1 : 0;
    g.ksplit = ksplit; g.split_stride = (int64_t)r * r;
    launch_gemm<tc::A_IMG_MN, tc::N_IMG_MN, tc::EPI_STORE, 0>(b, g, prof::S_GRAM, st);
    if (ksplit > 1) {
        prof::Scope scope(prof::S_GRAM, st);
        dim3 grid((unsigned)(((int64_t)r * r / 4 + 255) / 256), 1, (unsigned)b.count);
        gram_reduce_kernel<<<grid, 256, 0, st>>>(b, gram, part, (int64_t)r * r / 4, ksplit, only_shift_bit);
    }
}

// dst = src * L^{-T}  (src: image of a rows x r matrix; image linv holds (L^{-1})^T, read MN-major)
inline void tensor_apply(int r, int passes, const Batch& b, const TensorScratch& ts, ImgRef src, int64_t rows,
                         tc::OutSpec out, cudaStream_t st) {
    tc::GemmArgs g{};
    g.Mrows = (int32_t)rows; g.Ncols = r; g.Kdim = r; g.BN = std::min(r, 256);
    g.passes = passes; g.passes2 = 1; g.a = src; g.n1 = ts.linv; g.n2 = no_img(); g.tri = 1;
    g.colsq_off = ts.colsq;
    g.out = out;
    launch_gemm<tc::A_IMG_K, tc::N_IMG_MN, tc::EPI_STORE, 0>(b, g, prof::S_APPLY, st);
}

// M <- a (M + G) - b P R^T ;  X <- c X - d P Q^T                  (Alg. 1, update and error-feedback steps)
// fp16 = 1: both products run as one fp16 pass from the fp16 planes of P, R, Q (R's plane must
// have been written by launch_pack_half).
inline void tensor_k5(int64_t m, int64_t n, int r, int g_bf16, int x_bf16, int passes_m, int passes_x, int fp16,
                      float ef_a, float ef_b, float wc, float wd, const Batch& b, const TensorScratch& ts,
                      cudaStream_t st) {
    tc::GemmArgs g{};
    g.fp16 = fp16; g.rscale_off = ts.rscale;
    g.Mrows = (int32_t)m; g.Ncols = (int32_t)n; g.Kdim = r; g.BN = 128;
    g.passes = passes_m; g.passes2 = passes_x; g.ld = n;
    g.a = ts.p; g.n1 = ts.r; g.n2 = ts.q;
    g.ef_a = ef_a; g.ef_b = ef_b; g.wc = wc; g.wd = wd;
    g.out.normal = dest_none(); g.out.shifted = dest_none();
    const int xg = (g_bf16 ? 1 : 0) | (x_bf16 ? 2 : 0);
    switch (xg) {
        case 0: launch_gemm<tc::A_IMG_K, tc::N_IMG_K, tc::EPI_K5, 0>(b, g, prof::S_K5, st); break;
        case 1: launch_gemm<tc::A_IMG_K, tc::N_IMG_K, tc::EPI_K5, 1>(b, g, prof::S_K5, st); break;
        case 2: launch_gemm<tc::A_IMG_K, tc::N_IMG_K, tc::EPI_K5, 2>(b, g, prof::S_K5, st); break;
        default: launch_gemm<tc::A_IMG_K, tc::N_IMG_K, tc::EPI_K5, 3>(b, g, prof::S_K5, st); break;
    }
}

}  // namespace od
