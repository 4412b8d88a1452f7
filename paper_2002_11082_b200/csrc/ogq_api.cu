// extern "C" entry points: argument validation, scratch layout, kernel launches.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>
#include <string.h>

#include <atomic>
#include <vector>

#include "../../include/ogq.h"
#include "ogq_internal.h"

static_assert(OGQ_NOALLOC_MAX_TENSORS == ogq::kNoAllocMaxTensors, "header and library limits differ");

namespace ogq {

struct ProfRec {
    const char* name;
    cudaEvent_t a, b;
};
static std::vector<ProfRec> g_prof;
static bool g_prof_on = false;
static std::atomic<unsigned long long> g_launches{0};  // data-path calls may come from several host threads

void launch_begin(const char* name, cudaStream_t stream)
{
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (!g_prof_on) return;
    ProfRec r;
    r.name = name;
    if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return;
    cudaEventRecord(r.a, stream);
    g_prof.push_back(r);
}

void launch_end(cudaStream_t stream)
{
    if (!g_prof_on || g_prof.empty()) return;
    cudaEventRecord(g_prof.back().b, stream);
}

}  // namespace ogq

namespace {

int sm_count_of_current_device()
{
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    return sms;
}

bool aligned16(const void* p) { return ((uintptr_t)p & 15u) == 0; }

// One NVTX range per data-path call, named after the entry point (a stage of the path on a profiler's
// host timeline; a no-op when no tool is attached).
struct StageRange {
    explicit StageRange(const char* name) { nvtxRangePushA(name); }
    ~StageRange() { nvtxRangePop(); }
    StageRange(const StageRange&) = delete;
    StageRange& operator=(const StageRange&) = delete;
};

bool valid_orq_levels(int s) { return s == 3 || s == 5 || s == 9 || s == 17; }

// The selection solvers count the elements of a tensor in 32-bit cells.
bool select_size_ok(int64_t total_elems) { return total_elems < ((int64_t)1 << 32); }

}  // namespace

extern "C" {

const char* ogq_version(void) { return "ogq 0.2 (sm_100a)"; }

unsigned long long ogq_launch_count(void) { return ogq::g_launches.load(std::memory_order_relaxed); }

int ogq_profile_enable(int on)
{
    if (on) {
        for (auto& r : ogq::g_prof) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
        ogq::g_prof.clear();
    }
    ogq::g_prof_on = on != 0;
    return 0;
}

int ogq_profile_collect(float* h_ms, char* h_names, int name_stride, int max_records)
{
    int n = 0;
    for (auto& r : ogq::g_prof) {
        if (n < max_records && h_ms && cudaEventSynchronize(r.b) == cudaSuccess) {
            float ms = 0.f;
            cudaEventElapsedTime(&ms, r.a, r.b);
            h_ms[n] = ms;
            if (h_names && name_stride > 0) {
                strncpy(h_names + (size_t)n * name_stride, r.name, (size_t)name_stride - 1);
                h_names[(size_t)n * name_stride + name_stride - 1] = 0;
            }
            ++n;
        }
        cudaEventDestroy(r.a);
        cudaEventDestroy(r.b);
    }
    ogq::g_prof.clear();
    return n;
}

int ogq_bits_for_levels(int s)
{
    if (s < 2 || s > 32) return 0;
    int bits = 1;
    while ((1 << bits) < s) ++bits;
    return bits;
}

ogq_status ogq_packed_layout(const int64_t* h_off, int T, int bits, int64_t* h_packed_off)
{
    if (!h_off || !h_packed_off || T < 0 || bits < 1 || bits > 5) return OGQ_ERR_INVALID_ARG;
    h_packed_off[0] = 0;
    for (int t = 0; t < T; ++t) {
        const int64_t n = h_off[t + 1] - h_off[t];
        if (n < 0) return OGQ_ERR_INVALID_ARG;
        const int64_t w = (n * bits + 31) / 32;
        h_packed_off[t + 1] = h_packed_off[t] + (w + 3) / 4 * 4;
    }
    return OGQ_OK;
}

size_t ogq_workspace_bytes(int num_tensors, int64_t total_elems, int max_levels)
{
    if (num_tensors < 0 || total_elems < 0) return 0;
    size_t a = ogq::ws_bytes_bingrad_b(num_tensors, total_elems);
    size_t b = ogq::ws_bytes_select(num_tensors, total_elems, max_levels < 3 ? 3 : max_levels);
    return (a > b ? a : b) + 256;
}

static ogq_status levels_bingrad_impl(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems,
                                      int variant, int lloyd_iters, const float* d_tau, float* d_levels,
                                      float* d_thresh, int32_t* d_status, void* d_ws, size_t ws_bytes,
                                      ogq_stream_t stream)
{
    if (T < 0 || total_elems < 0 || !d_off || !d_levels || !d_status || lloyd_iters < 0 ||
        lloyd_iters > 1024)
        return OGQ_ERR_INVALID_ARG;
    if (variant != OGQ_BINGRAD_PB && variant != OGQ_BINGRAD_B) return OGQ_ERR_UNSUPPORTED;
    if (variant == OGQ_BINGRAD_PB && !select_size_ok(total_elems)) return OGQ_ERR_UNSUPPORTED;
    if (total_elems > 0 && (!d_grad || !aligned16(d_grad))) return OGQ_ERR_INVALID_ARG;
    if (variant == OGQ_BINGRAD_B && !d_thresh) return OGQ_ERR_INVALID_ARG;
    if (T == 0) return OGQ_OK;
    if (!d_ws || ((uintptr_t)d_ws & 255u)) return OGQ_ERR_WORKSPACE;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e;
    if (variant == OGQ_BINGRAD_B) {
        if (ws_bytes < ogq::ws_bytes_bingrad_b(T, total_elems)) return OGQ_ERR_WORKSPACE;
        e = ogq::launch_levels_bingrad_b(d_grad, d_off, T, total_elems, lloyd_iters, d_tau, d_levels, d_thresh,
                                         d_status, d_ws, sms, (cudaStream_t)stream);
    } else {
        if (ws_bytes < ogq::ws_bytes_select(T, total_elems, 2)) return OGQ_ERR_WORKSPACE;
        e = ogq::launch_levels_select(d_grad, d_off, T, total_elems, OGQ_BINGRAD_PB, 2, d_tau, d_levels, d_status,
                                      d_ws, ws_bytes, sms, (cudaStream_t)stream);
    }
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

ogq_status ogq_levels_bingrad(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems,
                              int variant, int lloyd_iters, float* d_levels, float* d_thresh,
                              int32_t* d_status, void* d_ws, size_t ws_bytes, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_levels_bingrad");
    return levels_bingrad_impl(d_grad, d_off, T, total_elems, variant, lloyd_iters, nullptr, d_levels, d_thresh,
                               d_status, d_ws, ws_bytes, stream);
}

ogq_status ogq_levels_bingrad_clipped(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems,
                                      int variant, int lloyd_iters, const float* d_tau, float* d_levels,
                                      float* d_thresh, int32_t* d_status, void* d_ws, size_t ws_bytes,
                                      ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_levels_bingrad_clipped");
    if (!d_tau) return OGQ_ERR_INVALID_ARG;
    return levels_bingrad_impl(d_grad, d_off, T, total_elems, variant, lloyd_iters, d_tau, d_levels, d_thresh,
                               d_status, d_ws, ws_bytes, stream);
}

ogq_status ogq_clip_threshold(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems, float c,
                              float* d_tau, int32_t* d_status, void* d_ws, size_t ws_bytes, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_clip_threshold");
    if (T < 0 || total_elems < 0 || !d_off || !d_tau || !d_status || !(c > 0.f) || !(c < 1e30f))
        return OGQ_ERR_INVALID_ARG;
    if (total_elems > 0 && (!d_grad || !aligned16(d_grad))) return OGQ_ERR_INVALID_ARG;
    if (T == 0) return OGQ_OK;
    if (!d_ws || ((uintptr_t)d_ws & 255u) || ws_bytes < ogq::ws_bytes_bingrad_b(T, total_elems)) return OGQ_ERR_WORKSPACE;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e = ogq::launch_clip_threshold(d_grad, d_off, T, total_elems, c, d_tau, d_status, d_ws, sms,
                                               (cudaStream_t)stream);
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

ogq_status ogq_levels_bingrad_b_noalloc(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems,
                                        int lloyd_iters, float* d_levels, float* d_thresh,
                                        int32_t* d_status, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_levels_bingrad_b_noalloc");
    if (T < 0 || total_elems < 0 || !d_off || !d_levels || !d_thresh || !d_status || lloyd_iters < 0 ||
        lloyd_iters > 1024)
        return OGQ_ERR_INVALID_ARG;
    if (T > OGQ_NOALLOC_MAX_TENSORS) return OGQ_ERR_LIMIT;
    if (total_elems > 0 && (!d_grad || !aligned16(d_grad))) return OGQ_ERR_INVALID_ARG;
    if (T == 0) return OGQ_OK;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e = ogq::launch_levels_bingrad_b_static(d_grad, d_off, T, total_elems, lloyd_iters, d_levels,
                                                        d_thresh, d_status, sms, (cudaStream_t)stream);
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

static ogq_status levels_orq_impl(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems, int s,
                                  const float* d_tau, float* d_levels, int32_t* d_status, void* d_ws,
                                  size_t ws_bytes, ogq_stream_t stream)
{
    if (T < 0 || total_elems < 0 || !d_off || !d_levels || !d_status) return OGQ_ERR_INVALID_ARG;
    if (!valid_orq_levels(s) || !select_size_ok(total_elems)) return OGQ_ERR_UNSUPPORTED;
    if (total_elems > 0 && (!d_grad || !aligned16(d_grad))) return OGQ_ERR_INVALID_ARG;
    if (T == 0) return OGQ_OK;
    if (!d_ws || ((uintptr_t)d_ws & 255u)) return OGQ_ERR_WORKSPACE;
    if (ws_bytes < ogq::ws_bytes_select(T, total_elems, s)) return OGQ_ERR_WORKSPACE;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e = ogq::launch_levels_select(d_grad, d_off, T, total_elems, OGQ_ORQ, s, d_tau, d_levels, d_status,
                                              d_ws, ws_bytes, sms, (cudaStream_t)stream);
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

ogq_status ogq_levels_orq(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems, int s,
                          float* d_levels, int32_t* d_status, void* d_ws, size_t ws_bytes,
                          ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_levels_orq");
    return levels_orq_impl(d_grad, d_off, T, total_elems, s, nullptr, d_levels, d_status, d_ws, ws_bytes, stream);
}

ogq_status ogq_levels_orq_clipped(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems, int s,
                                  const float* d_tau, float* d_levels, int32_t* d_status, void* d_ws,
                                  size_t ws_bytes, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_levels_orq_clipped");
    if (!d_tau) return OGQ_ERR_INVALID_ARG;
    return levels_orq_impl(d_grad, d_off, T, total_elems, s, d_tau, d_levels, d_status, d_ws, ws_bytes, stream);
}

static ogq_status quantize_pack_impl(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems,
                             ogq_scheme scheme, int s, const float* d_levels, const float* d_thresh,
                             const float* d_tau, uint64_t seed, uint32_t stream_id, const int64_t* d_packed_off,
                             uint32_t* d_packed, ogq_stream_t stream)
{
    if (T < 0 || total_elems < 0 || !d_off || !d_packed_off) return OGQ_ERR_INVALID_ARG;
    if (scheme == OGQ_BINGRAD_B) {
        if (s != 2) return OGQ_ERR_UNSUPPORTED;
        if (!d_thresh) return OGQ_ERR_INVALID_ARG;
    } else if (scheme == OGQ_BINGRAD_PB) {
        if (s != 2) return OGQ_ERR_UNSUPPORTED;
        if (!d_levels) return OGQ_ERR_INVALID_ARG;
    } else if (scheme == OGQ_ORQ) {
        if (!valid_orq_levels(s)) return OGQ_ERR_UNSUPPORTED;
        if (!d_levels) return OGQ_ERR_INVALID_ARG;
    } else {
        return OGQ_ERR_UNSUPPORTED;
    }
    if (total_elems > 0 && (!d_grad || !d_packed || !aligned16(d_grad) || !aligned16(d_packed)))
        return OGQ_ERR_INVALID_ARG;
    if (T == 0 || total_elems == 0) return OGQ_OK;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e = ogq::launch_quantize_pack(d_grad, d_off, T, total_elems, (int)scheme, s, d_levels,
                                              d_thresh, d_tau, seed, stream_id, d_packed_off, d_packed, sms,
                                              (cudaStream_t)stream);
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

ogq_status ogq_quantize_pack(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems,
                             ogq_scheme scheme, int s, const float* d_levels, const float* d_thresh,
                             uint64_t seed, uint32_t stream_id, const int64_t* d_packed_off,
                             uint32_t* d_packed, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_quantize_pack");
    return quantize_pack_impl(d_grad, d_off, T, total_elems, scheme, s, d_levels, d_thresh, nullptr, seed,
                              stream_id, d_packed_off, d_packed, stream);
}

ogq_status ogq_quantize_pack_clipped(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems,
                                     ogq_scheme scheme, int s, const float* d_levels, const float* d_thresh,
                                     const float* d_tau, uint64_t seed, uint32_t stream_id,
                                     const int64_t* d_packed_off, uint32_t* d_packed, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_quantize_pack_clipped");
    if (!d_tau) return OGQ_ERR_INVALID_ARG;
    return quantize_pack_impl(d_grad, d_off, T, total_elems, scheme, s, d_levels, d_thresh, d_tau, seed,
                              stream_id, d_packed_off, d_packed, stream);
}

ogq_status ogq_unpack_sum(const uint32_t* const* d_packed_k, const float* const* d_levels_k, int K,
                          const int64_t* d_off, const int64_t* d_packed_off, int T, int64_t total_elems,
                          int s, float scale, float* d_out, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_unpack_sum");
    if (T < 0 || total_elems < 0 || !d_off || !d_packed_off || !d_packed_k || !d_levels_k)
        return OGQ_ERR_INVALID_ARG;
    if (K < 1 || K > 64) return OGQ_ERR_INVALID_ARG;
    if (!(s == 2 || valid_orq_levels(s))) return OGQ_ERR_UNSUPPORTED;
    if (total_elems > 0 && (!d_out || !aligned16(d_out))) return OGQ_ERR_INVALID_ARG;
    if (T == 0 || total_elems == 0) return OGQ_OK;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e = ogq::launch_unpack_sum(d_packed_k, d_levels_k, K, d_off, d_packed_off, T, total_elems, s,
                                           scale, d_out, sms, (cudaStream_t)stream);
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

static ogq_status quant_error_impl(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems, int s,
                                   const float* d_levels, const int64_t* d_packed_off, const uint32_t* d_packed,
                                   bool realised, double* d_err, ogq_stream_t stream)
{
    if (T < 0 || total_elems < 0 || !d_off || !d_levels || !d_err) return OGQ_ERR_INVALID_ARG;
    if (realised && (!d_packed_off || (total_elems > 0 && !d_packed))) return OGQ_ERR_INVALID_ARG;
    if (!(s == 2 || valid_orq_levels(s))) return OGQ_ERR_UNSUPPORTED;
    if (total_elems > 0 && !d_grad) return OGQ_ERR_INVALID_ARG;
    if (T == 0) return OGQ_OK;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e = ogq::launch_quant_error(d_grad, d_off, T, total_elems, s, d_levels, d_packed_off,
                                            realised ? d_packed : nullptr, d_err, sms, (cudaStream_t)stream);
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

ogq_status ogq_quant_error(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems, int s,
                           const float* d_levels, const int64_t* d_packed_off, const uint32_t* d_packed,
                           double* d_err, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_quant_error");
    return quant_error_impl(d_grad, d_off, T, total_elems, s, d_levels, d_packed_off, d_packed, true, d_err, stream);
}

ogq_status ogq_expected_error(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems, int s,
                              const float* d_levels, double* d_err, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_expected_error");
    return quant_error_impl(d_grad, d_off, T, total_elems, s, d_levels, nullptr, nullptr, false, d_err, stream);
}

int ogq_dense_digits(int s) { return ogq::dense_digits(s); }

ogq_status ogq_dense_layout(const int64_t* h_off, int T, int s, int64_t* h_packed_off)
{
    const int m = ogq::dense_digits(s);
    if (!h_off || !h_packed_off || T < 0) return OGQ_ERR_INVALID_ARG;
    if (m == 0) return OGQ_ERR_UNSUPPORTED;
    h_packed_off[0] = 0;
    for (int t = 0; t < T; ++t) {
        const int64_t n = h_off[t + 1] - h_off[t];
        if (n < 0) return OGQ_ERR_INVALID_ARG;
        const int64_t w = (n + m - 1) / m;
        h_packed_off[t + 1] = h_packed_off[t] + (w + 3) / 4 * 4;
    }
    return OGQ_OK;
}

ogq_status ogq_quantize_pack_dense(const float* d_grad, const int64_t* d_off, int T, int64_t total_elems, int s,
                                   const float* d_levels, uint64_t seed, uint32_t stream_id,
                                   const int64_t* d_packed_off, uint32_t* d_packed, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_quantize_pack_dense");
    if (T < 0 || total_elems < 0 || !d_off || !d_packed_off || !d_levels) return OGQ_ERR_INVALID_ARG;
    if (!valid_orq_levels(s)) return OGQ_ERR_UNSUPPORTED;
    if (total_elems > 0 && (!d_grad || !d_packed || !aligned16(d_grad) || !aligned16(d_packed)))
        return OGQ_ERR_INVALID_ARG;
    if (T == 0 || total_elems == 0) return OGQ_OK;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e = ogq::launch_quantize_pack_dense(d_grad, d_off, T, total_elems, s, d_levels, seed, stream_id,
                                                    d_packed_off, d_packed, sms, (cudaStream_t)stream);
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

ogq_status ogq_unpack_sum_dense(const uint32_t* const* d_packed_k, const float* const* d_levels_k, int K,
                                const int64_t* d_off, const int64_t* d_packed_off, int T, int64_t total_elems,
                                int s, float scale, float* d_out, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_unpack_sum_dense");
    if (T < 0 || total_elems < 0 || !d_off || !d_packed_off || !d_packed_k || !d_levels_k)
        return OGQ_ERR_INVALID_ARG;
    if (K < 1 || K > 64) return OGQ_ERR_INVALID_ARG;
    if (!valid_orq_levels(s)) return OGQ_ERR_UNSUPPORTED;
    if (total_elems > 0 && (!d_out || !aligned16(d_out))) return OGQ_ERR_INVALID_ARG;
    if (T == 0 || total_elems == 0) return OGQ_OK;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e = ogq::launch_unpack_sum_dense(d_packed_k, d_levels_k, K, d_off, d_packed_off, T, total_elems, s,
                                                 scale, d_out, sms, (cudaStream_t)stream);
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

int64_t ogq_bucket_packed_words(int64_t total_elems, int d, int bits)
{
    if (total_elems < 0 || d < 128 || d > 32768 || (d & 127) || bits < 1 || bits > 5) return -1;
    if (total_elems == 0) return 0;
    const int64_t nb = (total_elems + d - 1) / d;
    const int64_t last = total_elems - (nb - 1) * d;
    const int64_t w = (last * bits + 31) / 32;
    return (nb - 1) * ((int64_t)d * bits / 32) + (w + 3) / 4 * 4;
}

ogq_status ogq_bucket_encode(const float* d_grad, int64_t total_elems, int d, ogq_scheme scheme, int s, int iters,
                             float clip_c, uint64_t seed, uint32_t stream_id, float* d_levels, float* d_thresh,
                             int32_t* d_status, uint32_t* d_packed, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_bucket_encode");
    if (total_elems < 0 || iters < 0 || iters > 1024 || !d_levels || !d_status || !(clip_c >= 0.f) || !(clip_c < 1e30f))
        return OGQ_ERR_INVALID_ARG;
    if (d < 128 || d > 32768 || (d & 127)) return OGQ_ERR_UNSUPPORTED;
    if (scheme == OGQ_BINGRAD_B) {
        if (s != 2) return OGQ_ERR_UNSUPPORTED;
        if (!d_thresh) return OGQ_ERR_INVALID_ARG;
    } else if (scheme == OGQ_BINGRAD_PB) {
        if (s != 2) return OGQ_ERR_UNSUPPORTED;
    } else if (scheme == OGQ_ORQ) {
        if (!valid_orq_levels(s)) return OGQ_ERR_UNSUPPORTED;
    } else {
        return OGQ_ERR_UNSUPPORTED;
    }
    if ((total_elems + d - 1) / d > 0x7fffffff) return OGQ_ERR_UNSUPPORTED;
    if (total_elems > 0 && (!d_grad || !d_packed || !aligned16(d_grad) || !aligned16(d_packed)))
        return OGQ_ERR_INVALID_ARG;
    if (total_elems == 0) return OGQ_OK;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e = ogq::launch_bucket_encode(d_grad, total_elems, d, (int)scheme, s, iters, clip_c, seed, stream_id,
                                              d_levels, d_thresh, d_status, d_packed, sms, (cudaStream_t)stream);
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

ogq_status ogq_bucket_decode_sum(const uint32_t* const* d_packed_k, const float* const* d_levels_k, int K,
                                 int64_t total_elems, int d, int s, float scale, float* d_out, ogq_stream_t stream)
{
    StageRange nvtx_range("ogq_bucket_decode_sum");
    if (total_elems < 0 || !d_packed_k || !d_levels_k) return OGQ_ERR_INVALID_ARG;
    if (K < 1 || K > 64) return OGQ_ERR_INVALID_ARG;
    if (d < 128 || d > 32768 || (d & 127)) return OGQ_ERR_UNSUPPORTED;
    if (!(s == 2 || valid_orq_levels(s))) return OGQ_ERR_UNSUPPORTED;
    if (total_elems > 0 && (!d_out || !aligned16(d_out))) return OGQ_ERR_INVALID_ARG;
    if (total_elems == 0) return OGQ_OK;
    const int sms = sm_count_of_current_device();
    if (sms <= 0) return OGQ_ERR_CUDA;
    cudaError_t e = ogq::launch_bucket_decode_sum(d_packed_k, d_levels_k, K, total_elems, d, s, scale, d_out, sms,
                                                  (cudaStream_t)stream);
    return e == cudaSuccess ? OGQ_OK : OGQ_ERR_CUDA;
}

}  // extern "C"
