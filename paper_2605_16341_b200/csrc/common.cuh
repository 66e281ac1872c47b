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
    int32_t aux0;       // launch-specific per-matrix integer (Cholesky: rows of column-square partials)
    int32_t aux1;
};

constexpr int MAXB = 256;   // matrices per launch batch
struct Batch {
    int32_t count;
    int32_t pad;
    int64_t scratch_stride;   // w[k].scratch = w[0].scratch + k * scratch_stride (one class per batch)
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

// ---- bf16 splitting ---------------------------------------------------------------------------
// An fp32 value v is carried through the tensor cores as v = t0 + t1 with t0 = bf16(v),
// t1 = bf16(v - t0) (round to nearest even): the two terms together hold 16 significand bits.

// two fp32 -> packed bf16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float bf16lo_to_f32(uint32_t p) { return __uint_as_float(p << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t p) { return __uint_as_float(p & 0xFFFF0000u); }

// two fp32 -> packed f16x2 (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
    uint32_t r;
    asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}
// 8 fp32 values (times scale) -> 16-byte chunk of fp16
__device__ __forceinline__ uint4 half8(const float (&v)[8], float scale) {
    return make_uint4(pack_f16x2(v[0] * scale, v[1] * scale), pack_f16x2(v[2] * scale, v[3] * scale),
                      pack_f16x2(v[4] * scale, v[5] * scale), pack_f16x2(v[6] * scale, v[7] * scale));
}

// 8 fp32 values -> 16-byte chunk of term 0 and of term 1
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

// Split image of an fp32 matrix S (rows x cols): the operand format of every tensor-core product.
// Columns are cut into panels of 64; a panel stores one 128-byte row (64 bf16) per matrix row,
// rows padded with zeros to a multiple of 128, and the eight 16-byte chunks of a row are
// XOR-swizzled with (row & 7) (the 128-byte shared-memory swizzle of the MMA descriptors).  Term t
// of panel p starts at off + (t * panels + p) * rows_pad * 128.  128 consecutive rows of a panel
// are a K-major operand tile (depth = S columns); 64 consecutive rows of two or more panels are an
// MN-major operand tile (depth = S rows): bulk copies move either into shared memory unchanged.
// An image may carry a third plane (index 2): the matrix rounded once to fp16 (times a power of
// two chosen by the writer), for products that run as a single fp16 pass.
struct ImgRef {
    int64_t off;        // byte offset in the matrix's scratch area; < 0: absent
    int32_t rows_pad;   // multiple of 128
    int32_t panels;     // ceil(cols / 64)
    int32_t planes;     // 2 (bf16 terms) or 3 (+ fp16 plane)
    int32_t pad;
};
__device__ __forceinline__ int64_t img_row_offset(const ImgRef& im, int term, int panel, int64_t row) {
    return im.off + (((int64_t)term * im.panels + panel) * im.rows_pad + row) * 128;
}
__device__ __forceinline__ int img_chunk_offset(int row, int chunk) { return ((chunk ^ (row & 7)) << 4); }

}  // namespace od
