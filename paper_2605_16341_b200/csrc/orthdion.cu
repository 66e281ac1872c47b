// Host side of liborthdion: plans, workspace layout, packing of equal plans into launch batches
// and the stage sequence of one optimizer step.  All device work is enqueued on the caller's stream.
#include "../../include/orthdion.h"

#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

#include "common.cuh"
#include "profile.cuh"
#include "factor_kernels.cuh"
#include "factor_tc.cuh"
#include "diag_kernels.cuh"
#include "rank_kernels.cuh"
#include "simt_kernels.cuh"
#include "tensor_engine.cuh"

using namespace od;

struct orthdion_plan {
    uint32_t magic;
    int64_t m, n;
    int32_t r;
    float mu, eta, wd, scale, ef_a, ef_b;
    int32_t mode, x_dtype, g_dtype, engine;
    int32_t passes[4];
    int32_t passes_set[4]; // 1: chosen by the caller, 0: follows the default rule
    int32_t diag;          // bit 0: factor diagnostics, bit 1: buffer norms (extra sweep over M, G)
};

namespace {

constexpr uint32_t kMagic = 0x0D10A5E7u;
constexpr int32_t kMaxRank = 4096;        // tensor engine; the SIMT engine and the diagnostics take r <= 1024
constexpr int32_t kMaxRankSimt = 1024;
constexpr size_t kScratchBudget = (size_t)24 << 30;   // per launch batch
constexpr float kShiftRel = 1e-5f;
// max/min diag(L) of the first Cholesky above which the QR takes the shifted three-pass path.
// CholeskyQR2 needs cond(Y)^2 * u well below 1, u the accuracy of the Gram/apply products:
// fp32 for the SIMT engine, about 2^-16 for the split-bf16 products of the tensor engine.
constexpr float kCondLimit = 1024.f;
constexpr float kCondLimitTensor = 96.f;

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
inline bool valid(orthdion_t h) { return h && h->magic == kMagic; }

bool same_class(const orthdion_plan* a, const orthdion_plan* b) {
    return a->m == b->m && a->n == b->n && a->r == b->r && a->mode == b->mode &&
           a->x_dtype == b->x_dtype && a->g_dtype == b->g_dtype && a->engine == b->engine &&
           a->eta == b->eta && a->wd == b->wd && a->scale == b->scale && a->ef_a == b->ef_a &&
           a->ef_b == b->ef_b && a->diag == b->diag &&
           std::memcmp(a->passes, b->passes, sizeof(a->passes)) == 0;
}

// Per-matrix scratch carving (byte offsets).  gram, linv and the tensor engine's first entries
// depend on r only, so one Cholesky launch can serve matrices of different shapes.
struct Scratch {
    int64_t gram, linv, tmpA, tmpB;
    int64_t gram_part;     // partial results of a depth-split product (tensor engine, small ranks)
    TensorScratch ts;
    size_t bytes;
};

// The fused feedback/update pass runs as one fp16 pass when both of its products ask for one pass.
bool fused_fp16(const orthdion_plan* p) {
    return p->engine == ORTHDION_ENGINE_TENSOR && p->passes[2] == 1 && p->passes[3] == 1;
}

Scratch scratch_layout(const orthdion_plan* p) {
    Scratch s{};
    const size_t rr = align_up((size_t)p->r * p->r * 4, 256);
    size_t off = 0;
    s.gram = off; off += rr;
    s.linv = off; off += rr;
    if (p->engine == ORTHDION_ENGINE_TENSOR) {
        off = tensor_scratch_layout(p->m, p->n, p->r, fused_fp16(p), off, &s.ts);
        // (after everything whose offset must depend on r only)
        const int parts = std::max(gram_ksplit(p->r, p->m), gram_ksplit(p->r, p->n));
        const int s1 = buffer_ksplit(p->r, p->m, p->n), s3 = buffer_ksplit(p->r, p->n, p->m);
        size_t part_bytes = parts > 1 ? (size_t)parts * rr : 0;
        if (s1 > 1) part_bytes = std::max(part_bytes, align_up((size_t)s1 * p->m * p->r * 4, 256));
        if (s3 > 1) part_bytes = std::max(part_bytes, align_up((size_t)s3 * p->n * p->r * 4, 256));
        s.gram_part = (int64_t)off;
        off += part_bytes;
    } else {
        const size_t kr = align_up((size_t)std::max(p->m, p->n) * p->r * 4, 256);
        s.tmpA = off; off += kr;
        s.tmpB = off; off += kr;
    }
    s.bytes = align_up(off, 1024);
    return s;
}

// A launch batch: matrices of one class.  A group: batches that are stepped together, stage by
// stage, so that the short serial kernels (the r x r Cholesky) of all of them run side by side.
struct Batching {
    std::vector<std::vector<int>> batches;   // matrix indices per launch batch
    std::vector<std::vector<int>> groups;    // batch indices per group
    std::vector<size_t> batch_off;           // scratch offset of each batch inside its group
    size_t scratch_bytes = 0;                // max over groups
};

Batching make_batches(const orthdion_t* hs, int32_t count) {
    Batching out;
    std::vector<char> done(count, 0);
    size_t group_bytes = 0;
    for (int i = 0; i < count; ++i) {
        if (done[i]) continue;
        std::vector<int> cls;
        for (int j = i; j < count; ++j)
            if (!done[j] && same_class(hs[i], hs[j])) { cls.push_back(j); done[j] = 1; }
        const size_t per = scratch_layout(hs[i]).bytes;
        size_t cap = std::max<size_t>(1, kScratchBudget / std::max<size_t>(per, 1));
        cap = std::min<size_t>(cap, MAXB);
        const size_t nb = (cls.size() + cap - 1) / cap;
        const size_t bs = (cls.size() + nb - 1) / nb;
        for (size_t b = 0; b < cls.size(); b += bs) {
            std::vector<int> one(cls.begin() + b, cls.begin() + std::min(cls.size(), b + bs));
            const size_t bytes = one.size() * per;
            if (out.groups.empty() || group_bytes + bytes > kScratchBudget) {
                out.groups.emplace_back();
                group_bytes = 0;
            }
            out.groups.back().push_back((int)out.batches.size());
            out.batch_off.push_back(group_bytes);
            group_bytes += bytes;
            out.scratch_bytes = std::max(out.scratch_bytes, group_bytes);
            out.batches.push_back(std::move(one));
        }
    }
    return out;
}

// Workspace: [status words][diagnostic records][P_0 R_0][P_1 R_1]...[scratch of the largest group]
struct Layout {
    std::vector<size_t> p_off, r_off;
    size_t status_off = 0, diag_off = 0, scratch_off = 0, total = 0;
};

Layout make_layout(const orthdion_t* hs, int32_t count, size_t scratch_bytes) {
    Layout l;
    size_t off = align_up((size_t)count * 4, 256);
    l.diag_off = off;
    off += align_up((size_t)count * DIAG_STRIDE * 4, 256);
    l.p_off.resize(count);
    l.r_off.resize(count);
    for (int i = 0; i < count; ++i) {
        l.p_off[i] = off; off += align_up((size_t)hs[i]->m * hs[i]->r * 4, 256);
        l.r_off[i] = off; off += align_up((size_t)hs[i]->n * hs[i]->r * 4, 256);
    }
    l.scratch_off = align_up(off, 1024);
    l.total = l.scratch_off + scratch_bytes;
    return l;
}

#define CU_CHECK(expr)                                                     \
    do {                                                                   \
        cudaError_t e__ = (expr);                                          \
        if (e__ != cudaSuccess) {                                          \
            std::fprintf(stderr, "orthdion: %s failed: %s\n", #expr, cudaGetErrorString(e__)); \
            return ORTHDION_ERR_CUDA;                                      \
        }                                                                  \
    } while (0)

// Kernel attributes (dynamic shared-memory limits) belong to a device: they are set once per
// device ordinal, on the first step call made with that device current.
signed char g_factor_cluster_max[kMaxDevices] = {};   // written under ensure_attributes()'s lock

int ensure_attributes() {
    static std::mutex mu;
    static signed char state[kMaxDevices] = {};   // 0 unknown, 1 ok, -1 failed
    int dev = -1;
    CU_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return ORTHDION_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (state[dev]) return state[dev] > 0 ? 0 : ORTHDION_ERR_CUDA;
    cudaError_t e = cudaFuncSetAttribute(chol_inv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)CH_SMEM_BYTES);
    // the r x r factor kernel keeps 2 r floats in dynamic shared memory next to its static tables
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(chol_inv_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * kMaxRank * 4);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(chol_inv_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * kMaxRank * 4);
    // clusters of 16 CTAs are beyond the portable size: allowed per kernel, and used only where the
    // device says that it can place one
    g_factor_cluster_max[dev] = 8;
    if (e == cudaSuccess &&
        cudaFuncSetAttribute(chol_inv_tc_kernel<true>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess) {
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(16, 1, 1); cfg.blockDim = dim3(CT_THREADS, 1, 1);
        cfg.dynamicSmemBytes = (size_t)2 * kMaxRank * 4;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 16; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        int clusters = 0;
        if (cudaOccupancyMaxActiveClusters(&clusters, chol_inv_tc_kernel<true>, &cfg) == cudaSuccess && clusters >= 1)
            g_factor_cluster_max[dev] = 16;
        else
            (void)cudaGetLastError();
    }
    if (e == cudaSuccess) e = tensor_engine_set_attributes();
    if (e != cudaSuccess) {
        std::fprintf(stderr, "orthdion: kernel attribute setup failed on device %d: %s\n", dev, cudaGetErrorString(e));
        state[dev] = -1;
        return ORTHDION_ERR_CUDA;
    }
    state[dev] = 1;
    return 0;
}

int factor_cluster_max() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 8;
    return g_factor_cluster_max[dev] == 16 ? 16 : 8;
}

// ---- internal streams of the grouped step ---------------------------------------------------
// The steps of two launch batches (matrices of different plans) share nothing, so a grouped call
// may run them side by side: the caller's stream forks into up to kMaxLanes internal streams,
// every batch runs its whole stage sequence on one of them, and the caller's stream joins them
// again before the call returns.  Order on the device is fixed by events only; the host never
// waits.  The latency-bound r x r factor kernel of one batch and the ramp-up and tail of every
// persistent kernel then overlap the kernels of the other batches.  Results per matrix do not
// depend on this: every matrix goes through the same kernels with the same launch geometry.
constexpr int kMaxLanes = 8;
std::atomic<int> g_lanes{4};

struct DeviceLanes {
    std::mutex mu;                   // one grouped call at a time forks into the lanes of a device
    bool ready = false;
    cudaStream_t lane[kMaxLanes] = {};
    cudaEvent_t fork = nullptr, done[kMaxLanes] = {};
};

// Lanes of the current device; streams and events are created on the first call that needs them
// (no device memory is allocated).
DeviceLanes* device_lanes() {
    static DeviceLanes table[kMaxDevices];
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    DeviceLanes* d = &table[dev];
    std::lock_guard<std::mutex> lock(d->mu);
    if (!d->ready) {
        bool ok = cudaEventCreateWithFlags(&d->fork, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < kMaxLanes && ok; ++i)
            ok = cudaStreamCreateWithFlags(&d->lane[i], cudaStreamNonBlocking) == cudaSuccess &&
                 cudaEventCreateWithFlags(&d->done[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return nullptr;
        d->ready = true;
    }
    return d;
}

template <class RA, class RB, class EP>
void launch_simt(const Batch& b, int64_t Md, int64_t Nd, int64_t Kd, RA ra, RB rb, EP ep, int stage,
                 cudaStream_t st) {
    dim3 grid((unsigned)((Nd + 63) / 64), (unsigned)((Md + 63) / 64), (unsigned)b.count);
    prof::Scope scope(stage, st);
    simt_gemm_kernel<RA, RB, EP><<<grid, 256, 0, st>>>(b, Md, Nd, Kd, ra, rb, ep);
}

Sel sel(int where, int64_t off = 0) { return Sel{where, 0, off}; }

// One class of a group while it is being stepped.
struct ClassRun {
    const orthdion_plan* p;
    Batch* b;
    Scratch sc;
    bool tensor() const { return p->engine == ORTHDION_ENGINE_TENSOR; }
};

// Cholesky + inverse of every class's Gram matrix: classes of equal (r, engine) share launches.
// diag_from_gram: take the diagonal from the Gram matrix itself instead of the column-square
// partials of the producing kernel (column-sharded matrices: the reduced Gram matrix carries it).
void chol_stage(std::vector<ClassRun>& cls, const std::vector<int>& which_cls, int which, int pass,
                Batch* merged, int call_matrices, cudaStream_t st, bool diag_from_gram = false) {
    std::vector<char> done(which_cls.size(), 0);
    for (size_t i = 0; i < which_cls.size(); ++i) {
        if (done[i]) continue;
        const ClassRun& lead = cls[which_cls[i]];
        const int r = lead.p->r;
        CholArgs ca{};
        ca.gram = sel(W_SCRATCH, lead.sc.gram); ca.work = sel(W_SCRATCH, lead.sc.linv);
        ca.r = r; ca.which = which; ca.pass = pass; ca.shift_rel = kShiftRel;
        ca.cond_limit = lead.tensor() ? kCondLimitTensor : kCondLimit;
        ca.colsq = sel(W_SCRATCH, 0); ca.use_colsq = 0; ca.img = no_img(); ca.cnorm_off = -1;
        if (lead.tensor()) {
            ca.colsq = sel(W_SCRATCH, lead.sc.ts.colsq); ca.use_colsq = diag_from_gram ? 0 : 1; ca.img = lead.sc.ts.linv;
            if (which == 1 && pass == 1) ca.cnorm_off = lead.sc.ts.cnorm;
        }
        merged->count = 0; merged->pad = 0; merged->scratch_stride = 0;
        auto flush = [&]() {
            if (!merged->count) return;
            prof::Scope scope(prof::S_CHOL, st);
            if (lead.tensor()) {
                // Fewer matrices than the device has room for CTAs (two per multiprocessor): share
                // each matrix among the CTAs of a cluster (2, 4 or 8; 16 from rank 512 up, where the
                // tile lists are long enough to feed them and the device can place such a cluster).
                // (counted over the whole grouped call: with more matrices than that, the other
                // launch batches keep the rest of the device busy on their own streams.)
                int csize = 1;
                const int room = 2 * sm_count();
                const int cmax = r >= 512 ? factor_cluster_max() : 8;
                while (csize < cmax && std::max(merged->count, call_matrices) * csize * 2 <= room) csize *= 2;
                const size_t dyn = (size_t)2 * r * sizeof(float);
                if (csize == 1) {
                    chol_inv_tc_kernel<false><<<merged->count, CT_THREADS, dyn, st>>>(*merged, ca, 1);
                } else {
                    cudaLaunchConfig_t cfg{};
                    cfg.gridDim = dim3((unsigned)(merged->count * csize), 1, 1);
                    cfg.blockDim = dim3(CT_THREADS, 1, 1);
                    cfg.dynamicSmemBytes = dyn;
                    cfg.stream = st;
                    cudaLaunchAttribute attr[1];
                    attr[0].id = cudaLaunchAttributeClusterDimension;
                    attr[0].val.clusterDim.x = (unsigned)csize; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
                    cfg.attrs = attr; cfg.numAttrs = 1;
                    if (cudaLaunchKernelEx(&cfg, chol_inv_tc_kernel<true>, *merged, ca, csize) != cudaSuccess)
                        engine_error() = 4;
                }
            } else {
                chol_inv_kernel<<<merged->count, CH_THREADS, CH_SMEM_BYTES, st>>>(*merged, ca);
            }
            merged->count = 0;
        };
        for (size_t j = i; j < which_cls.size(); ++j) {
            const ClassRun& c = cls[which_cls[j]];
            if (done[j] || c.p->r != r || c.tensor() != lead.tensor()) continue;
            done[j] = 1;
            const int64_t rows = which ? c.p->n : c.p->m;
            for (int k = 0; k < c.b->count; ++k) {
                MatWork& w = merged->w[merged->count++];
                w = c.b->w[k];
                w.aux0 = (int32_t)(4 * ((rows + 127) / 128));
                if (merged->count == MAXB) flush();
            }
        }
        flush();
    }
}

// ---- tall-skinny QR of every class in `which_cls` (CholeskyQR2; third pass when flagged) --------
// which = 0: P = orth(Y) (Alg. 1, left-factor step), which = 1: Q = orth(R) (Alg. 1, normalisation step).
// Tensor engine: the input is an image (w0 holds Y, image r holds R); SIMT engine: fp32 slots.
void qr_stage(std::vector<ClassRun>& cls, const std::vector<int>& which_cls, int which, Batch* merged,
              int call_matrices, cudaStream_t st) {
    const int shift_bit = which ? ST_SHIFT_R : ST_SHIFT_L;
    for (int pass = 1; pass <= 3; ++pass) {
        const int only_shift = pass == 3;
        for (int ci : which_cls) {
            ClassRun& c = cls[ci];
            const int r = c.p->r;
            const int64_t rows = which ? c.p->n : c.p->m;
            const Sel gram = sel(W_SCRATCH, c.sc.gram);
            if (c.tensor()) {
                const TensorScratch& ts = c.sc.ts;
                const ImgRef in = which ? ts.r : img_view(ts.w0, rows);
                const ImgRef src = pass == 1 ? in : (pass == 2 ? img_view(ts.w1, rows) : img_view(ts.w0, rows));
                tensor_gram(r, c.p->passes[1], *c.b, src, rows, gram, sel(W_SCRATCH, c.sc.gram_part),
                            only_shift ? shift_bit : 0, st);
            } else {
                const Sel in = which ? sel(W_R) : sel(W_P);
                const Sel src = pass == 1 ? in : (pass == 2 ? sel(W_SCRATCH, c.sc.tmpA) : sel(W_SCRATCH, c.sc.tmpB));
                EpStore eg{gram, gram, only_shift ? shift_bit : 0, 1, r, only_shift};
                launch_simt(*c.b, r, r, rows, RdPlain{src, 1, r}, RdPlain{src, 1, r}, eg, prof::S_GRAM, st);
            }
        }
        chol_stage(cls, which_cls, which, pass, merged, call_matrices, st);
        for (int ci : which_cls) {
            ClassRun& c = cls[ci];
            const int r = c.p->r;
            const int64_t rows = which ? c.p->n : c.p->m;
            const Sel fin = which ? sel(W_Q) : sel(W_P);
            if (c.tensor()) {
                const TensorScratch& ts = c.sc.ts;
                const ImgRef in = which ? ts.r : img_view(ts.w0, rows);
                const ImgRef w0 = img_view(ts.w0, rows), w1 = img_view(ts.w1, rows);
                const ImgRef src = pass == 1 ? in : (pass == 2 ? w1 : w0);
                tc::Dest to_fin = dest_none();
                to_fin.f32 = fin; to_fin.has_f32 = 1; to_fin.img = which ? ts.q : ts.p;
                tc::Dest to_w1 = dest_none(); to_w1.img = w1; to_w1.colsq = 1;
                tc::Dest to_w0 = dest_none(); to_w0.img = w0; to_w0.colsq = 1;
                tc::OutSpec out{};
                out.ld = r; out.shift_bit = 0; out.only_if_shifted = 0;
                if (pass == 1) { out.normal = to_w1; out.shifted = to_w1; }
                else if (pass == 2) { out.normal = to_fin; out.shifted = to_w0; out.shift_bit = shift_bit; }
                else { out.normal = to_fin; out.shifted = to_fin; out.shift_bit = shift_bit; out.only_if_shifted = 1; }
                tensor_apply(r, c.p->passes[1], *c.b, ts, src, rows, out, st);
            } else {
                const Sel in = which ? sel(W_R) : sel(W_P);
                const Sel tmpA = sel(W_SCRATCH, c.sc.tmpA), tmpB = sel(W_SCRATCH, c.sc.tmpB);
                const Sel linv = sel(W_SCRATCH, c.sc.linv);
                const Sel src = pass == 1 ? in : (pass == 2 ? tmpA : tmpB);
                EpStore ea{};
                if (pass == 1) ea = EpStore{tmpA, tmpA, 0, 1, r, 0};
                else if (pass == 2) ea = EpStore{fin, tmpB, shift_bit, 1, r, 0};
                else ea = EpStore{fin, fin, shift_bit, 1, r, 1};
                launch_simt(*c.b, rows, r, r, RdPlain{src, r, 1}, RdPlain{linv, r, 1}, ea, prof::S_APPLY, st);
            }
        }
    }
}

// Diagnostics of one class, after its step: Q^T Q from the engine's Gram product, column
// statistics of R, optionally the norms of M' and G, then one CTA per matrix for the rest.
void diag_stage(ClassRun& c, DiagBase db, cudaStream_t st) {
    const orthdion_plan* p = c.p;
    const Batch& b = *c.b;
    const int r = p->r;
    const Sel gram = sel(W_SCRATCH, c.sc.gram);
    const int64_t stats_off = c.sc.linv;          // 3 r floats of the (now free) inverse slot
    {
        prof::Scope scope(prof::S_DIAG, st);
        diag_init_kernel<<<(b.count * DIAG_STRIDE + 255) / 256, 256, 0, st>>>(b, db);
    }
    if (c.tensor()) {
        tensor_gram(r, p->passes[1], b, c.sc.ts.q, p->n, gram, sel(W_SCRATCH, c.sc.gram_part), 0, st);
    } else {
        const Sel sQ = sel(W_Q);
        launch_simt(b, r, r, p->n, RdPlain{sQ, 1, r}, RdPlain{sQ, 1, r}, EpStore{gram, gram, 0, 1, r, 0},
                    prof::S_GRAM, st);
    }
    {
        prof::Scope scope(prof::S_DIAG, st);
        if (r % 4 == 0) {
            dim3 grid((unsigned)((r + 127) / 128), 1, (unsigned)b.count);
            diag_colstats4_kernel<<<grid, 1024, 0, st>>>(b, p->n, r, stats_off);
        } else {
            dim3 grid((unsigned)((r + 31) / 32), 1, (unsigned)b.count);
            diag_colstats_kernel<<<grid, 1024, 0, st>>>(b, p->n, r, stats_off);
        }
    }
    if (p->diag & 2) {
        const int64_t elems = p->m * p->n;
        const int64_t want = (elems / 4 + 256 * 32 - 1) / (256 * 32);
        dim3 grid((unsigned)std::max<int64_t>(1, std::min<int64_t>(want, 1184 / std::max(1, b.count) + 1)), 1,
                  (unsigned)b.count);
        prof::Scope scope(prof::S_DIAG, st);
        diag_frob_kernel<<<grid, 256, 0, st>>>(b, elems, p->g_dtype == ORTHDION_DTYPE_BF16, db);
    }
    {
        prof::Scope scope(prof::S_DIAG, st);
        diag_final_kernel<<<b.count, DIAG_THREADS, 0, st>>>(b, r, c.sc.gram, stats_off, p->diag, p->ef_a, p->ef_b, db);
    }
}

// One step of every class of a group, stage by stage.
void run_group(std::vector<ClassRun>& cls, Batch* merged, DiagBase db, int call_matrices, cudaStream_t st) {
    const Sel sP = sel(W_P), sR = sel(W_R), sQ = sel(W_Q);
    std::vector<int> all, orth;
    for (size_t i = 0; i < cls.size(); ++i) {
        all.push_back((int)i);
        if (cls[i].p->mode == ORTHDION_MODE_ORTH) orth.push_back((int)i);
    }
    for (ClassRun& c : cls) {
        prof::Scope scope(prof::S_MISC, st);
        init_status_kernel<<<(c.b->count + 255) / 256, 256, 0, st>>>(*c.b);
    }
    // Alg. 1, buffer and left-factor steps:  Y = (M + G) Q_prev
    for (ClassRun& c : cls) {
        const orthdion_plan* p = c.p;
        const int gb = p->g_dtype == ORTHDION_DTYPE_BF16;
        if (c.tensor()) tensor_k1(p->m, p->n, p->r, gb, p->passes[0], *c.b, c.sc.ts, sel(W_SCRATCH, c.sc.gram_part), st);
        else launch_simt(*c.b, p->m, p->r, p->n, RdBuffer{p->n, gb, 0}, RdPlain{sQ, 1, p->r},
                         EpStore{sP, sP, 0, 0, p->r, 0}, prof::S_K1, st);
    }
    qr_stage(cls, all, 0, merged, call_matrices, st);
    // Alg. 1, right-factor step:  R = (M + G)^T P
    for (ClassRun& c : cls) {
        const orthdion_plan* p = c.p;
        const int gb = p->g_dtype == ORTHDION_DTYPE_BF16;
        if (c.tensor()) tensor_k3(p->m, p->n, p->r, gb, p->passes[0], *c.b, c.sc.ts, sel(W_SCRATCH, c.sc.gram_part), st);
        else launch_simt(*c.b, p->n, p->r, p->m, RdBuffer{p->n, gb, 1}, RdPlain{sP, 1, p->r},
                         EpStore{sR, sR, 0, 0, p->r, 0}, prof::S_K3, st);
    }
    // Alg. 1, normalisation step
    qr_stage(cls, orth, 1, merged, call_matrices, st);
    for (ClassRun& c : cls) {
        const orthdion_plan* p = c.p;
        if (p->mode == ORTHDION_MODE_ORTH) continue;
        {
            dim3 grid((unsigned)((p->r + 31) / 32), 1, (unsigned)c.b->count);
            prof::Scope scope(prof::S_COLNORM, st);
            colnorm_kernel<<<grid, 1024, 0, st>>>(*c.b, p->n, p->r, c.tensor() ? c.sc.ts.cnorm : (int64_t)-1, 0);
        }
        if (c.tensor()) launch_pack(*c.b, sQ, p->n, p->r, c.sc.ts.q, st);
    }
    // Alg. 1, update and error-feedback steps:  M <- a B - b P R^T ;  X <- c X - d P Q^T
    for (ClassRun& c : cls) {
        const orthdion_plan* p = c.p;
        const int gb = p->g_dtype == ORTHDION_DTYPE_BF16, xb = p->x_dtype == ORTHDION_DTYPE_BF16;
        const float cc = 1.f - p->eta * p->wd, dd = p->eta * p->scale;
        if (c.tensor()) {
            const int fp16 = fused_fp16(p) ? 1 : 0;
            if (fp16) launch_pack_half(*c.b, p->n, p->r, c.sc.ts, st);
            tensor_k5(p->m, p->n, p->r, gb, xb, p->passes[2], p->passes[3], fp16, p->ef_a, p->ef_b, cc, dd, *c.b,
                      c.sc.ts, st);
        } else {
            launch_simt(*c.b, p->m, p->n, p->r, RdPlain{sP, p->r, 1}, RdPlain{sR, p->r, 1},
                        EpErrorFeedback{p->ef_a, p->ef_b, p->n, gb}, prof::S_K5, st);
            launch_simt(*c.b, p->m, p->n, p->r, RdPlain{sP, p->r, 1}, RdPlain{sQ, p->r, 1},
                        EpWeights{cc, dd, p->n, xb}, prof::S_K5, st);
        }
    }
    for (ClassRun& c : cls)
        if (c.p->diag) diag_stage(c, db, st);
}

// Default pass counts of the fused feedback/update pass.  One fp16 pass carries P R^T with about
// 4e-4 relative error; in M' = a B - b P R^T that is harmless while b is small against a (the
// momentum form, b = 1 - mu), but not in the residual form a = b, where M' is what is left after
// the projection has been subtracted: then P R^T comes from split terms (three passes).
void default_passes(orthdion_plan* p) {
    const bool x32 = p->x_dtype == ORTHDION_DTYPE_F32;
    if (!p->passes_set[0]) p->passes[0] = 3;
    if (!p->passes_set[1]) p->passes[1] = 3;
    if (!p->passes_set[2]) p->passes[2] = (x32 || std::fabs(p->ef_b) > 0.1f * std::fabs(p->ef_a)) ? 3 : 1;
    if (!p->passes_set[3]) p->passes[3] = x32 ? 3 : 1;
}

int check_ptr(const void* p) {
    if (!p) return ORTHDION_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(p) % 16) return ORTHDION_ERR_ALIGNMENT;
    return 0;
}

}  // namespace

extern "C" {

int orthdion_create(orthdion_t* out, int64_t m, int64_t n, int32_t r, float mu, float eta, float wd,
                    int32_t mode) {
    if (!out) return ORTHDION_ERR_NULL;
    *out = nullptr;
    if (m < 1 || n < 1 || m > (1 << 24) || n > (1 << 24)) return ORTHDION_ERR_INVALID_ARG;
    if (mode != ORTHDION_MODE_ORTH && mode != ORTHDION_MODE_COLNORM) return ORTHDION_ERR_INVALID_ARG;
    if (!(mu == mu) || !(eta == eta) || !(wd == wd)) return ORTHDION_ERR_INVALID_ARG;
    if (r < 1 || r > m || r > n || r > kMaxRank) return ORTHDION_ERR_RANK;
    orthdion_plan* p = new orthdion_plan();
    p->magic = kMagic;
    p->m = m; p->n = n; p->r = r;
    p->mu = mu; p->eta = eta; p->wd = wd; p->scale = 1.f;
    p->ef_a = 1.f; p->ef_b = 1.f - mu;
    p->mode = mode;
    p->x_dtype = ORTHDION_DTYPE_BF16; p->g_dtype = ORTHDION_DTYPE_BF16;
    p->engine = tensor_engine_supports(m, n, r) ? ORTHDION_ENGINE_TENSOR : ORTHDION_ENGINE_SIMT;
    if (p->engine == ORTHDION_ENGINE_SIMT && r > kMaxRankSimt) { delete p; return ORTHDION_ERR_RANK; }
    for (int k = 0; k < 4; ++k) p->passes_set[k] = 0;
    default_passes(p);
    p->diag = 0;
    *out = p;
    return ORTHDION_OK;
}

int orthdion_destroy(orthdion_t h) {
    if (!valid(h)) return ORTHDION_ERR_INVALID_ARG;
    h->magic = 0;
    delete h;
    return ORTHDION_OK;
}

int orthdion_set_dtypes(orthdion_t h, int32_t x_dtype, int32_t g_dtype) {
    if (!valid(h)) return ORTHDION_ERR_INVALID_ARG;
    if ((x_dtype != ORTHDION_DTYPE_F32 && x_dtype != ORTHDION_DTYPE_BF16) ||
        (g_dtype != ORTHDION_DTYPE_F32 && g_dtype != ORTHDION_DTYPE_BF16))
        return ORTHDION_ERR_INVALID_ARG;
    h->x_dtype = x_dtype; h->g_dtype = g_dtype;
    // bf16 weights: the update is rounded to bf16 anyway, one pass carries P Q^T.  An fp32 weight
    // matrix shows the update at full precision: both products from split terms.
    default_passes(h);
    return ORTHDION_OK;
}

int orthdion_set_lr(orthdion_t h, float eta) {
    if (!valid(h) || !(eta == eta)) return ORTHDION_ERR_INVALID_ARG;
    h->eta = eta;
    return ORTHDION_OK;
}

int orthdion_set_scale(orthdion_t h, float scale) {
    if (!valid(h) || !(scale == scale)) return ORTHDION_ERR_INVALID_ARG;
    h->scale = scale;
    return ORTHDION_OK;
}

int orthdion_set_ef(orthdion_t h, float a, float b) {
    if (!valid(h) || !(a == a) || !(b == b)) return ORTHDION_ERR_INVALID_ARG;
    h->ef_a = a; h->ef_b = b;
    default_passes(h);
    return ORTHDION_OK;
}

int orthdion_set_engine(orthdion_t h, int32_t engine) {
    if (!valid(h)) return ORTHDION_ERR_INVALID_ARG;
    if (engine == ORTHDION_ENGINE_SIMT) {
        if (h->r > kMaxRankSimt) return ORTHDION_ERR_RANK;
        h->engine = engine;
        return ORTHDION_OK;
    }
    if (engine != ORTHDION_ENGINE_TENSOR) return ORTHDION_ERR_INVALID_ARG;
    if (!tensor_engine_supports(h->m, h->n, h->r)) return ORTHDION_ERR_RANK;
    h->engine = engine;
    return ORTHDION_OK;
}

int orthdion_set_passes(orthdion_t h, int32_t which, int32_t passes) {
    if (!valid(h) || which < 0 || which > 3) return ORTHDION_ERR_INVALID_ARG;
    if (passes <= 0) {
        h->passes_set[which] = 0;
        default_passes(h);
        return ORTHDION_OK;
    }
    if (passes != 1 && passes != 3) return ORTHDION_ERR_INVALID_ARG;
    h->passes[which] = passes;
    h->passes_set[which] = 1;
    return ORTHDION_OK;
}

int orthdion_set_diagnostics(orthdion_t h, int32_t mask) {
    if (!valid(h) || mask < 0 || mask > 3) return ORTHDION_ERR_INVALID_ARG;
    if (mask && h->r > kMaxRankSimt) return ORTHDION_ERR_RANK;   // the eigenvalue iteration holds r-vectors in shared memory
    if (mask == 2) mask = 3;      // the buffer norms are reported together with the factor diagnostics
    h->diag = mask;
    return ORTHDION_OK;
}

size_t orthdion_workspace_bytes_grouped(const orthdion_t* hs, int32_t count) {
    if (!hs || count < 1) return 0;
    for (int i = 0; i < count; ++i)
        if (!valid(hs[i])) return 0;
    Batching bt = make_batches(hs, count);
    return make_layout(hs, count, bt.scratch_bytes).total;
}

size_t orthdion_workspace_bytes(orthdion_t h) { return orthdion_workspace_bytes_grouped(&h, 1); }

int orthdion_step_grouped(const orthdion_t* hs, int32_t count, void* const* X, float* const* M,
                          const void* const* G, float* const* Q, void* workspace, size_t workspace_bytes,
                          void* stream) {
    if (!hs || !X || !M || !G || !Q || !workspace) return ORTHDION_ERR_NULL;
    if (count < 1) return ORTHDION_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i) {
        if (!valid(hs[i])) return ORTHDION_ERR_INVALID_ARG;
        int e;
        if ((e = check_ptr(X[i])) || (e = check_ptr(M[i])) || (e = check_ptr(G[i])) || (e = check_ptr(Q[i])))
            return e;
    }
    if (reinterpret_cast<uintptr_t>(workspace) % 256) return ORTHDION_ERR_WORKSPACE;
    Batching bt = make_batches(hs, count);
    Layout lay = make_layout(hs, count, bt.scratch_bytes);
    if (workspace_bytes < lay.total) return ORTHDION_ERR_WORKSPACE;
    int e = ensure_attributes();
    if (e) return e;

    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    char* ws = reinterpret_cast<char*>(workspace);
    std::vector<Batch> pool(bt.batches.size() + 1);
    Batch* merged = &pool[bt.batches.size()];
    int rc = ORTHDION_OK;
    for (const auto& grp : bt.groups) {
        std::vector<ClassRun> cls;
        for (int bi : grp) {
            const auto& idx = bt.batches[bi];
            ClassRun c{hs[idx[0]], &pool[bi], scratch_layout(hs[idx[0]])};
            c.b->count = (int32_t)idx.size();
            c.b->pad = 0;
            c.b->scratch_stride = (int64_t)c.sc.bytes;
            for (size_t k = 0; k < idx.size(); ++k) {
                const int i = idx[k];
                MatWork& w = c.b->w[k];
                w.X = X[i]; w.M = M[i]; w.G = G[i]; w.Q = Q[i];
                w.P = reinterpret_cast<float*>(ws + lay.p_off[i]);
                w.R = reinterpret_cast<float*>(ws + lay.r_off[i]);
                w.status = reinterpret_cast<int32_t*>(ws + lay.status_off) + i;
                w.scratch = ws + lay.scratch_off + bt.batch_off[bi] + k * c.sc.bytes;
                w.aux0 = 0; w.aux1 = 0;
            }
            cls.push_back(c);
        }
        engine_error() = 0;
        const DiagBase db{reinterpret_cast<const int32_t*>(ws + lay.status_off),
                          reinterpret_cast<float*>(ws + lay.diag_off)};
        const int lanes = std::min<int>({g_lanes.load(), kMaxLanes, (int)cls.size()});
        DeviceLanes* dl = lanes > 1 ? device_lanes() : nullptr;
        if (dl) {
            // heaviest batch first, each batch a lane of its own (round robin beyond `lanes`)
            std::vector<int> order(cls.size());
            for (size_t i = 0; i < cls.size(); ++i) order[i] = (int)i;
            auto cost = [&](int i) {
                const orthdion_plan* p = cls[i].p;
                return (double)cls[i].b->count * ((double)p->m * p->n * p->r + (double)(p->m + p->n) * p->r * p->r);
            };
            std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return cost(a) > cost(b); });
            std::lock_guard<std::mutex> lock(dl->mu);
            cudaEventRecord(dl->fork, st);
            for (int l = 0; l < lanes; ++l) cudaStreamWaitEvent(dl->lane[l], dl->fork, 0);
            for (size_t k = 0; k < order.size(); ++k) {
                std::vector<ClassRun> one(1, cls[order[k]]);
                run_group(one, merged, db, count, dl->lane[k % lanes]);
            }
            for (int l = 0; l < lanes; ++l) {
                cudaEventRecord(dl->done[l], dl->lane[l]);
                cudaStreamWaitEvent(st, dl->done[l], 0);
            }
        } else {
            run_group(cls, merged, db, count, st);
        }
        if (engine_error()) {
            std::fprintf(stderr, "orthdion: tensor map setup failed (%d)\n", engine_error());
            rc = ORTHDION_ERR_CUDA;
            break;
        }
        cudaError_t ce = cudaGetLastError();
        if (ce != cudaSuccess) {
            std::fprintf(stderr, "orthdion: launch failed: %s\n", cudaGetErrorString(ce));
            rc = ORTHDION_ERR_CUDA;
            break;
        }
    }
    return rc;
}

int orthdion_step(orthdion_t h, void* X, float* M, const void* G, float* Q, void* workspace,
                  size_t workspace_bytes, void* stream) {
    void* const xs[1] = {X};
    float* const ms[1] = {M};
    const void* const gs[1] = {G};
    float* const qs[1] = {Q};
    return orthdion_step_grouped(&h, 1, xs, ms, gs, qs, workspace, workspace_bytes, stream);
}

}  // extern "C"

// ---- column-sharded step (Section 2, "FSDP communication") --------------------------------------
// A matrix split by columns over k ranks, rank j holding X_j, M_j, G_j (m x n_j) and the rows Q_j
// (n_j x r) of the right factor:  B Q_prev = sum_j B_j Q_j,  R_j = B_j^T P,  R^T R = sum_j R_j^T R_j.
// The step becomes four local phases with one reduction (a sum over the ranks, made by the
// caller: NCCL all-reduce on real ranks) of a small buffer between them:
//   phase 0   Y_j = (M_j + G_j) Q_j                                       -> reduce Y   (m x r)
//   phase 1   P = orth(Y) (the same on every rank);  R_j = (M_j + G_j)^T P;
//             ORTH: Gram matrix of R_j;  COLNORM: squared column norms of R_j  -> reduce (r x r | r)
//   phase 2   ORTH: first CholeskyQR pass of R_j with the reduced Gram matrix, Gram matrix of the
//             result -> reduce (r x r).   COLNORM: Q_j = R_j / norms, fused update pass: done.
//   phase 3   ORTH: second pass -> Q_j, fused update pass.
// The traffic per step is (m + 2 r) r floats (ORTH) or (m + 1) r floats (COLNORM) per rank: the
// O((m + n) r) of the paper.  The right QR is CholeskyQR2 here; a flagged third pass is not taken.
namespace {
struct ShardRun {
    Batch batch;
    ClassRun c;
    Layout lay;
};

int shard_setup(orthdion_t h, void* X, float* M, const void* G, float* Q, void* workspace, size_t workspace_bytes,
                ShardRun* sr) {
    if (!valid(h)) return ORTHDION_ERR_INVALID_ARG;
    if (h->engine != ORTHDION_ENGINE_TENSOR || h->diag) return ORTHDION_ERR_INVALID_ARG;
    int e;
    if ((e = check_ptr(X)) || (e = check_ptr(M)) || (e = check_ptr(G)) || (e = check_ptr(Q))) return e;
    if (!workspace) return ORTHDION_ERR_NULL;
    if (reinterpret_cast<uintptr_t>(workspace) % 256) return ORTHDION_ERR_WORKSPACE;
    Batching bt = make_batches(&h, 1);
    sr->lay = make_layout(&h, 1, bt.scratch_bytes);
    if (workspace_bytes < sr->lay.total) return ORTHDION_ERR_WORKSPACE;
    if ((e = ensure_attributes())) return e;
    char* ws = reinterpret_cast<char*>(workspace);
    sr->c = ClassRun{h, &sr->batch, scratch_layout(h)};
    sr->batch.count = 1; sr->batch.pad = 0; sr->batch.scratch_stride = (int64_t)sr->c.sc.bytes;
    MatWork& w = sr->batch.w[0];
    w.X = X; w.M = M; w.G = G; w.Q = Q;
    w.P = reinterpret_cast<float*>(ws + sr->lay.p_off[0]);
    w.R = reinterpret_cast<float*>(ws + sr->lay.r_off[0]);
    w.status = reinterpret_cast<int32_t*>(ws + sr->lay.status_off);
    w.scratch = ws + sr->lay.scratch_off;
    w.aux0 = 0; w.aux1 = 0;
    return ORTHDION_OK;
}

// Gram matrix of the image `src` (rows x r) with its diagonal from the fp32 column squares
void shard_gram(ShardRun& sr, const ImgRef& src, int64_t rows, cudaStream_t st) {
    const orthdion_plan* p = sr.c.p;
    const Sel gram = sel(W_SCRATCH, sr.c.sc.gram);
    tensor_gram(p->r, p->passes[1], sr.batch, src, rows, gram, sel(W_SCRATCH, sr.c.sc.gram_part), 0, st);
    prof::Scope scope(prof::S_MISC, st);
    gram_diag_kernel<<<dim3((unsigned)((p->r + 255) / 256), 1, 1), 256, 0, st>>>(
        sr.batch, gram, p->r, sr.c.sc.ts.colsq, (int)(4 * ((rows + 127) / 128)));
}

void shard_fused_pass(ShardRun& sr, cudaStream_t st) {
    const orthdion_plan* p = sr.c.p;
    const int gb = p->g_dtype == ORTHDION_DTYPE_BF16, xb = p->x_dtype == ORTHDION_DTYPE_BF16;
    const float cc = 1.f - p->eta * p->wd, dd = p->eta * p->scale;
    const int fp16 = fused_fp16(p) ? 1 : 0;
    if (fp16) launch_pack_half(sr.batch, p->n, p->r, sr.c.sc.ts, st);
    tensor_k5(p->m, p->n, p->r, gb, xb, p->passes[2], p->passes[3], fp16, p->ef_a, p->ef_b, cc, dd, sr.batch,
              sr.c.sc.ts, st);
}
}  // namespace

extern "C" {

int orthdion_shard_phase(orthdion_t h, int32_t phase, void* X, float* M, const void* G, float* Q, void* workspace,
                         size_t workspace_bytes, void* stream) {
    ShardRun* sr = new ShardRun();
    int rc = shard_setup(h, X, M, G, Q, workspace, workspace_bytes, sr);
    if (rc) { delete sr; return rc; }
    const orthdion_plan* p = h;
    const bool orth = p->mode == ORTHDION_MODE_ORTH;
    if (phase < 0 || phase > (orth ? 3 : 2)) { delete sr; return ORTHDION_ERR_INVALID_ARG; }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int gb = p->g_dtype == ORTHDION_DTYPE_BF16;
    const TensorScratch& ts = sr->c.sc.ts;
    const int r = p->r;
    std::vector<ClassRun> cls(1, sr->c);
    const std::vector<int> only(1, 0);
    Batch* merged = new Batch();
    engine_error() = 0;
    if (phase == 0) {
        {
            prof::Scope scope(prof::S_MISC, st);
            init_status_kernel<<<1, 256, 0, st>>>(sr->batch);
        }
        tensor_k1(p->m, p->n, r, gb, p->passes[0], sr->batch, ts, sel(W_SCRATCH, sr->c.sc.gram_part), st, true);
    } else if (phase == 1) {
        // the summed Y sits in the P slot: image and column squares, then the usual left QR
        launch_pack(sr->batch, sel(W_P), p->m, r, img_view(ts.w0, p->m), st);
        {
            prof::Scope scope(prof::S_MISC, st);
            colsq_blocks_kernel<<<dim3((unsigned)(4 * ((p->m + 127) / 128)), (unsigned)((r + 255) / 256), 1), 256, 0, st>>>(
                sr->batch, sel(W_P), p->m, r, ts.colsq);
        }
        qr_stage(cls, only, 0, merged, 1, st);
        tensor_k3(p->m, p->n, r, gb, p->passes[0], sr->batch, ts, sel(W_SCRATCH, sr->c.sc.gram_part), st);
        if (orth) {
            shard_gram(*sr, ts.r, p->n, st);
        } else {
            prof::Scope scope(prof::S_COLNORM, st);
            colnorm_kernel<<<dim3((unsigned)((r + 31) / 32), 1, 1), 1024, 0, st>>>(sr->batch, p->n, r, ts.cnorm, 1);
        }
    } else if (phase == 2 && orth) {
        chol_stage(cls, only, 1, 1, merged, 1, st, true);
        tc::Dest to_w1 = dest_none(); to_w1.img = img_view(ts.w1, p->n); to_w1.colsq = 1;
        tc::OutSpec out{};
        out.ld = r; out.normal = to_w1; out.shifted = to_w1;
        tensor_apply(r, p->passes[1], sr->batch, ts, ts.r, p->n, out, st);
        shard_gram(*sr, img_view(ts.w1, p->n), p->n, st);
    } else if (phase == 2) {
        {
            prof::Scope scope(prof::S_COLNORM, st);
            colnorm_kernel<<<dim3((unsigned)((r + 31) / 32), 1, 1), 1024, 0, st>>>(sr->batch, p->n, r, ts.cnorm, 2);
        }
        launch_pack(sr->batch, sel(W_Q), p->n, r, ts.q, st);
        shard_fused_pass(*sr, st);
    } else {
        chol_stage(cls, only, 1, 2, merged, 1, st, true);
        tc::Dest to_fin = dest_none();
        to_fin.f32 = sel(W_Q); to_fin.has_f32 = 1; to_fin.img = ts.q;
        tc::OutSpec out{};
        out.ld = r; out.normal = to_fin; out.shifted = to_fin;
        tensor_apply(r, p->passes[1], sr->batch, ts, img_view(ts.w1, p->n), p->n, out, st);
        shard_fused_pass(*sr, st);
    }
    delete merged;
    delete sr;
    if (engine_error()) return ORTHDION_ERR_CUDA;
    cudaError_t ce = cudaGetLastError();
    if (ce != cudaSuccess) {
        std::fprintf(stderr, "orthdion: launch failed: %s\n", cudaGetErrorString(ce));
        return ORTHDION_ERR_CUDA;
    }
    return ORTHDION_OK;
}

int orthdion_shard_reduce_buffer(orthdion_t h, int32_t phase, void* workspace, float** buffer, int64_t* count) {
    if (!valid(h) || !workspace || !buffer || !count) return ORTHDION_ERR_NULL;
    if (h->engine != ORTHDION_ENGINE_TENSOR) return ORTHDION_ERR_INVALID_ARG;
    const bool orth = h->mode == ORTHDION_MODE_ORTH;
    if (phase < 0 || phase > (orth ? 2 : 1)) return ORTHDION_ERR_INVALID_ARG;
    Batching bt = make_batches(&h, 1);
    Layout lay = make_layout(&h, 1, bt.scratch_bytes);
    Scratch sc = scratch_layout(h);
    char* ws = reinterpret_cast<char*>(workspace);
    if (phase == 0) {
        *buffer = reinterpret_cast<float*>(ws + lay.p_off[0]);
        *count = h->m * (int64_t)h->r;
    } else if (orth) {
        *buffer = reinterpret_cast<float*>(ws + lay.scratch_off + sc.gram);
        *count = (int64_t)h->r * h->r;
    } else {
        *buffer = reinterpret_cast<float*>(ws + lay.scratch_off + sc.ts.cnorm);
        *count = h->r;
    }
    return ORTHDION_OK;
}

}  // extern "C"

// Scratch of orthdion_step_noalloc: part of the library image, so every GPU that loads the library
// holds these bytes until the process exits.  In host code the name below is only a handle for
// cudaGetSymbolAddress; it is not a device address and must never be handed to a kernel.
static __device__ __align__(256) unsigned char g_noalloc_scratch[ORTHDION_NOALLOC_SCRATCH_BYTES];

namespace {
// Device address of g_noalloc_scratch on the current device, looked up once per device.
int noalloc_scratch_address(void** out) {
    static std::mutex mu;
    static void* addr[kMaxDevices] = {};
    int dev = -1;
    CU_CHECK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return ORTHDION_ERR_CUDA;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        CU_CHECK(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        if (!p) return ORTHDION_ERR_CUDA;
        addr[dev] = p;
    }
    *out = addr[dev];
    return ORTHDION_OK;
}
}  // namespace

extern "C" {

int orthdion_step_noalloc(orthdion_t h, void* X, float* M, const void* G, float* Q, int32_t* status_dev,
                          void* stream) {
    if (!valid(h)) return ORTHDION_ERR_INVALID_ARG;
    const size_t need = orthdion_workspace_bytes(h);
    if (need == 0) return ORTHDION_ERR_INVALID_ARG;
    if (need > ORTHDION_NOALLOC_SCRATCH_BYTES) {
        std::fprintf(stderr,
                     "orthdion_step_noalloc: this plan (m=%lld, n=%lld, r=%d) needs %zu bytes of scratch, the "
                     "built-in array holds %zu; use orthdion_step with a caller-provided workspace\n",
                     (long long)h->m, (long long)h->n, (int)h->r, need, (size_t)ORTHDION_NOALLOC_SCRATCH_BYTES);
        return ORTHDION_ERR_WORKSPACE;
    }
    void* scratch = nullptr;
    int rc = noalloc_scratch_address(&scratch);
    if (rc) return rc;
    rc = orthdion_step(h, X, M, G, Q, scratch, ORTHDION_NOALLOC_SCRATCH_BYTES, stream);
    if (rc) return rc;
    if (status_dev) {
        // the status word of the only matrix is the first word of the scratch
        CU_CHECK(cudaMemcpyAsync(status_dev, scratch, sizeof(int32_t), cudaMemcpyDeviceToDevice,
                                 reinterpret_cast<cudaStream_t>(stream)));
    }
    return ORTHDION_OK;
}

int orthdion_get_factors(const orthdion_t* hs, int32_t count, int32_t index, void* workspace,
                         const float** P, const float** R) {
    if (!hs || !workspace || !P || !R) return ORTHDION_ERR_NULL;
    if (count < 1 || index < 0 || index >= count) return ORTHDION_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i)
        if (!valid(hs[i])) return ORTHDION_ERR_INVALID_ARG;
    Layout lay = make_layout(hs, count, 0);
    char* ws = reinterpret_cast<char*>(workspace);
    *P = reinterpret_cast<const float*>(ws + lay.p_off[index]);
    *R = reinterpret_cast<const float*>(ws + lay.r_off[index]);
    return ORTHDION_OK;
}

int orthdion_last_status(const orthdion_t* hs, int32_t count, void* workspace, void* stream, int32_t* flags) {
    if (!hs || !workspace || !flags) return ORTHDION_ERR_NULL;
    if (count < 1) return ORTHDION_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    CU_CHECK(cudaMemcpyAsync(flags, workspace, (size_t)count * 4, cudaMemcpyDeviceToHost, st));
    CU_CHECK(cudaStreamSynchronize(st));
    return ORTHDION_OK;
}

int orthdion_last_diagnostics(const orthdion_t* hs, int32_t count, void* workspace, void* stream, float* out) {
    if (!hs || !workspace || !out) return ORTHDION_ERR_NULL;
    if (count < 1) return ORTHDION_ERR_INVALID_ARG;
    for (int i = 0; i < count; ++i)
        if (!valid(hs[i])) return ORTHDION_ERR_INVALID_ARG;
    Layout lay = make_layout(hs, count, 0);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const char* ws = reinterpret_cast<const char*>(workspace);
    CU_CHECK(cudaMemcpy2DAsync(out, ORTHDION_DIAG_FLOATS * 4, ws + lay.diag_off, DIAG_STRIDE * 4,
                               ORTHDION_DIAG_FLOATS * 4, (size_t)count, cudaMemcpyDeviceToHost, st));
    CU_CHECK(cudaStreamSynchronize(st));
    for (int i = 0; i < count; ++i)
        if (!hs[i]->diag)
            for (int k = 0; k < ORTHDION_DIAG_FLOATS; ++k) out[(size_t)i * ORTHDION_DIAG_FLOATS + k] = 0.f;
    return ORTHDION_OK;
}

int orthdion_rank_policy(double e_t, int32_t r_t, double ema_prev, int32_t r_min, int32_t r_max, double alpha,
                         double gamma, int32_t multiple, double* ema_out, int32_t* r_next) {
    (void)r_t;   // part of the rule's statement; the caller resizes when *r_next differs from it
    if (!ema_out || !r_next) return ORTHDION_ERR_NULL;
    if (multiple < 1 || r_min < multiple || r_max < r_min || r_min % multiple || r_max % multiple)
        return ORTHDION_ERR_INVALID_ARG;
    if (!(e_t == e_t) || !(ema_prev == ema_prev) || !(alpha >= 0.0 && alpha <= 1.0) || !(gamma > 0.0))
        return ORTHDION_ERR_INVALID_ARG;
    const double ema = alpha * e_t + (1.0 - alpha) * ema_prev;
    double target = std::ceil(gamma * ema);
    if (!(target >= (double)r_min)) target = (double)r_min;
    if (target > (double)r_max) target = (double)r_max;
    *ema_out = ema;
    *r_next = (int32_t)std::floor(target / multiple + 0.5) * multiple;
    return ORTHDION_OK;
}

int orthdion_resize_factor(const float* Q_old, int64_t n, int32_t r_old, float* Q_new, int32_t r_new,
                           const float* pad, void* stream) {
    if (!Q_old || !Q_new) return ORTHDION_ERR_NULL;
    if (n < 1 || n > (1 << 24) || r_old < 1 || r_new < 1 || r_old > kMaxRank || r_new > kMaxRank)
        return ORTHDION_ERR_INVALID_ARG;
    if (r_new > r_old && !pad) return ORTHDION_ERR_NULL;
    if (Q_old == Q_new) return ORTHDION_ERR_INVALID_ARG;
    int e;
    if ((e = check_ptr(Q_old)) || (e = check_ptr(Q_new)) || (r_new > r_old && (e = check_ptr(pad)))) return e;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    const int padw = r_new > r_old ? r_new - r_old : 0;
    const bool vec = r_old % 4 == 0 && r_new % 4 == 0 && padw % 4 == 0;
    const int64_t total = n * (vec ? r_new / 4 : r_new);
    const unsigned grid = (unsigned)std::max<int64_t>(1, std::min<int64_t>((total + 255) / 256, 148 * 16));
    prof::Scope scope(prof::S_MISC, st);
    if (vec) resize_factor_kernel<4><<<grid, 256, 0, st>>>(Q_old, n, r_old, Q_new, r_new, pad);
    else resize_factor_kernel<1><<<grid, 256, 0, st>>>(Q_old, n, r_old, Q_new, r_new, pad);
    cudaError_t ce = cudaGetLastError();
    if (ce != cudaSuccess) {
        std::fprintf(stderr, "orthdion: launch failed: %s\n", cudaGetErrorString(ce));
        return ORTHDION_ERR_CUDA;
    }
    return ORTHDION_OK;
}

int orthdion_set_concurrency(int32_t lanes) {
    if (lanes < 1 || lanes > kMaxLanes) return ORTHDION_ERR_INVALID_ARG;
    g_lanes.store(lanes);
    return ORTHDION_OK;
}

int64_t orthdion_launch_count(void) { return prof::g_launches.load(); }

int orthdion_profile_begin(int32_t max_launches) {
    if (max_launches < 1 || max_launches > (1 << 20)) return ORTHDION_ERR_INVALID_ARG;
    while (prof::g_pool.size() < (size_t)max_launches * 2) {
        cudaEvent_t e;
        CU_CHECK(cudaEventCreate(&e));
        prof::g_pool.push_back(e);
    }
    prof::g_pool_next = 0;
    prof::g_records.clear();
    prof::g_enabled = true;
    return ORTHDION_OK;
}

int orthdion_profile_end(int32_t n_stages, double* ms, int64_t* launches) {
    if (!ms || !launches) return ORTHDION_ERR_NULL;
    if (n_stages < prof::S_COUNT) return ORTHDION_ERR_INVALID_ARG;
    prof::g_enabled = false;
    for (int s = 0; s < n_stages; ++s) { ms[s] = 0.0; launches[s] = 0; }
    for (const prof::Record& rec : prof::g_records) {
        CU_CHECK(cudaEventSynchronize(rec.end));
        float t = 0.f;
        CU_CHECK(cudaEventElapsedTime(&t, rec.beg, rec.end));
        ms[rec.stage] += t;
        launches[rec.stage] += 1;
    }
    prof::g_records.clear();
    return ORTHDION_OK;
}

int32_t orthdion_stage_count(void) { return prof::S_COUNT; }
const char* orthdion_stage_name(int32_t stage) { return prof::stage_name(stage); }

const char* orthdion_version(void) {
    return "orthdion sm_100a: engines tensor(tcgen05, bf16-split) + simt(fp32)";
}

}  // extern "C"
