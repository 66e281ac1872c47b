// Tensor-core engine (tcgen05 / TMEM) -- placeholder until the kernels land.
#pragma once
#include "common.cuh"
#include "simt_kernels.cuh"
namespace od {
struct TensorScratch { int64_t dummy; };
inline bool tensor_engine_supports(int64_t, int64_t, int32_t) { return false; }
inline size_t tensor_scratch_layout(int64_t, int64_t, int32_t, size_t off, TensorScratch*) { return off; }
inline cudaError_t tensor_engine_set_attributes() { return cudaSuccess; }
inline void tensor_k1(int64_t, int64_t, int, int, int, const Batch&, const TensorScratch&, cudaStream_t) {}
inline void tensor_k3(int64_t, int64_t, int, int, int, const Batch&, const TensorScratch&, cudaStream_t) {}
inline void tensor_k5(int64_t, int64_t, int, int, int, int, int, float, float, float, float, const Batch&, const TensorScratch&, cudaStream_t) {}
inline void tensor_gram(int64_t, int64_t, int, int, const Batch&, const TensorScratch&, Sel, int64_t, Sel, int, cudaStream_t) {}
inline void tensor_apply(int64_t, int64_t, int, int, const Batch&, const TensorScratch&, Sel, int64_t, Sel, EpStore, cudaStream_t) {}
}
