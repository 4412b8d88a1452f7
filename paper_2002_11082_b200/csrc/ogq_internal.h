// Host-side launchers behind the C ABI (one per kernel family).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace ogq {

// Instrumentation: counts launches and, when profiling is on, brackets them with events.
void launch_begin(const char* name, cudaStream_t stream);
void launch_end(cudaStream_t stream);

constexpr int kMaxFlatCtas = 4096;  // upper bound on CTAs of a flat streaming grid (scratch sizing)

// d_tau: per-tensor clipping thresholds applied to the values as they are read, or null
cudaError_t launch_levels_bingrad_b(const float* d_grad, const int64_t* d_off, int T, int64_t total,
                                    int lloyd_iters, const float* d_tau, float* d_levels, float* d_thresh,
                                    int32_t* d_status, void* d_ws, int sm_count, cudaStream_t stream);
cudaError_t launch_clip_threshold(const float* d_grad, const int64_t* d_off, int T, int64_t total, float c,
                                  float* d_tau, int32_t* d_status, void* d_ws, int sm_count, cudaStream_t stream);
size_t ws_bytes_bingrad_b(int T, int64_t total);

constexpr int kNoAllocMaxTensors = 1024;  // tensors per call of the fixed-scratch BinGrad-b variant
constexpr int kNoAllocMaxDevices = 64;
cudaError_t launch_levels_bingrad_b_static(const float* d_grad, const int64_t* d_off, int T, int64_t total,
                                           int lloyd_iters, float* d_levels, float* d_thresh,
                                           int32_t* d_status, int sm_count, cudaStream_t stream);

cudaError_t launch_levels_select(const float* d_grad, const int64_t* d_off, int T, int64_t total,
                                 int scheme, int s, const float* d_tau, float* d_levels, int32_t* d_status,
                                 void* d_ws, size_t ws_bytes, int sm_count, cudaStream_t stream);
size_t ws_bytes_select(int T, int64_t total, int s);

cudaError_t launch_quantize_pack(const float* d_grad, const int64_t* d_off, int T, int64_t total,
                                 int scheme, int s, const float* d_levels, const float* d_thresh,
                                 const float* d_tau, uint64_t seed, uint32_t stream_id,
                                 const int64_t* d_packed_off, uint32_t* d_packed, int sm_count,
                                 cudaStream_t stream);

cudaError_t launch_unpack_sum(const uint32_t* const* d_packed_k, const float* const* d_levels_k, int K,
                              const int64_t* d_off, const int64_t* d_packed_off, int T, int64_t total,
                              int s, float scale, float* d_out, int sm_count, cudaStream_t stream);

cudaError_t launch_bucket_encode(const float* d_grad, int64_t total, int d, int scheme, int s, int iters,
                                 float clip_c, uint64_t seed, uint32_t stream_id, float* d_levels, float* d_thresh,
                                 int32_t* d_status, uint32_t* d_packed, int sm_count, cudaStream_t stream);

// d_packed null: expected error of random rounding; else the realised error of those codes
cudaError_t launch_quant_error(const float* d_grad, const int64_t* d_off, int T, int64_t total, int s,
                               const float* d_levels, const int64_t* d_packed_off, const uint32_t* d_packed,
                               double* d_err, int sm_count, cudaStream_t stream);
cudaError_t launch_bucket_decode_sum(const uint32_t* const* d_packed_k, const float* const* d_levels_k, int K,
                                     int64_t total, int d, int s, float scale, float* d_out, int sm_count,
                                     cudaStream_t stream);
int dense_digits(int s);  // codes per 32-bit word of the base-s format (0: unsupported s)
cudaError_t launch_quantize_pack_dense(const float* d_grad, const int64_t* d_off, int T, int64_t total, int s,
                                       const float* d_levels, uint64_t seed, uint32_t stream_id,
                                       const int64_t* d_packed_off, uint32_t* d_packed, int sm_count,
                                       cudaStream_t stream);
cudaError_t launch_unpack_sum_dense(const uint32_t* const* d_packed_k, const float* const* d_levels_k, int K,
                                    const int64_t* d_off, const int64_t* d_packed_off, int T, int64_t total, int s,
                                    float scale, float* d_out, int sm_count, cudaStream_t stream);

}  // namespace ogq
