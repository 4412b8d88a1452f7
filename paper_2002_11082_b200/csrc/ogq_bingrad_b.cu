// BinGrad-b level solver: Eq. (bingrad-b optimal condition).
//
// Pass 0 streams the bucket once for the per-tensor sum (b_0 = mean).  Every
// further pass streams it again for the counts and sums of {v < b_0} and
// {v >= b_0}, i.e. the two conditional means; with Lloyd iterations requested
// the last CTA to finish a tensor moves b_0 to the midpoint and the next pass
// repeats.  Partial sums are fp64, written to fixed slots and combined in CTA
// order by the last CTA to arrive, so results do not depend on scheduling.
#include <math.h>

#include <atomic>

#include "ogq_common.cuh"
#include "ogq_internal.h"
#include "ogq_ws.h"

namespace ogq {

// CLIP: every value is first clamped to [-tau_arr[t], tau_arr[t]] (gradient clipping).
template <bool CLIP>
__global__ void __launch_bounds__(kThreads)
k_bb_pass(const float* __restrict__ grad, const int64_t* __restrict__ off, int T, int64_t total,
          int64_t chunk, int pass, int lloyd_iters, const float* __restrict__ tau_arr, float* __restrict__ levels,
          float* __restrict__ thresh, int32_t* __restrict__ status, BbWs ws)
{
    __shared__ double sh_d[kWarps];
    __shared__ long long sh_l[kWarps];
    __shared__ int sh_last;

    const int64_t lo = (int64_t)blockIdx.x * chunk;
    const int64_t hi = (lo + chunk < total) ? lo + chunk : total;

    if (pass == 0 && blockIdx.x == 0) {
        // empty tensors have no piece anywhere: settle them here
        for (int t = threadIdx.x; t < T; t += kThreads) {
            if (__ldg(off + t + 1) <= __ldg(off + t)) {
                levels[2 * t] = 0.f;
                levels[2 * t + 1] = 0.f;
                thresh[t] = 0.f;
                status[t] = OGQ_ST_EMPTY;
                ws.done[t] = 1;
            }
        }
    }

    for_each_piece(off, T, lo, hi, [&](int t, int64_t tb, int64_t te, int64_t pb, int64_t pe) {
        if (pass > 0 && __ldcg(ws.done + t)) return;
        const float b0 = (pass == 0) ? -INFINITY : __ldcg(thresh + t);
        const float tau = CLIP ? __ldg(tau_arr + t) : 0.f;
        double s_lo = 0.0, s_hi = 0.0;
        long long c_lo = 0;
        visit_piece(grad, pb, pe, [&](float raw) {
            const float v = CLIP ? copysignf(fminf(fabsf(raw), tau), raw) : raw;
            const bool below = v < b0;
            const double d = (double)v;
            s_lo += below ? d : 0.0;
            s_hi += below ? 0.0 : d;
            c_lo += below ? 1 : 0;
        });
        s_lo = block_sum(s_lo, sh_d);
        s_hi = block_sum(s_hi, sh_d);
        c_lo = block_sum(c_lo, sh_l);

        const int64_t c0 = tb / chunk, c1 = (te - 1) / chunk;
        if (threadIdx.x == 0) {
            BbPart p;
            p.s_lo = s_lo; p.s_hi = s_hi; p.c_lo = c_lo; p.c_hi = (pe - pb) - c_lo;
            BbPart* dst = (c0 == c1) ? ws.direct + t : ((tb < lo) ? ws.slot_a + blockIdx.x : ws.slot_b + blockIdx.x);
            *dst = p;
            __threadfence();
            unsigned prev = atomicAdd(ws.arrive + t, 1u);
            sh_last = (prev == (unsigned)(c1 - c0));
        }
        __syncthreads();
        if (!sh_last) return;
        __threadfence();

        // last CTA of this tensor: combine the pieces in CTA order
        double a_lo = 0.0, a_hi = 0.0;
        long long n_lo = 0, n_hi = 0;
        if (c0 == c1) {
            if (threadIdx.x == 0) {
                a_lo = s_lo; a_hi = s_hi; n_lo = c_lo; n_hi = (pe - pb) - c_lo;
            }
        } else {
            for (int64_t c = c0 + threadIdx.x; c <= c1; c += kThreads) {
                const BbPart* src = (c == c0) ? ws.slot_b + c : ws.slot_a + c;
                a_lo += __ldcg(&src->s_lo);
                a_hi += __ldcg(&src->s_hi);
                n_lo += __ldcg(&src->c_lo);
                n_hi += __ldcg(&src->c_hi);
            }
            a_lo = block_sum(a_lo, sh_d);
            a_hi = block_sum(a_hi, sh_d);
            n_lo = block_sum(n_lo, sh_l);
            n_hi = block_sum(n_hi, sh_l);
        }
        if (threadIdx.x == 0) {
            ws.arrive[t] = 0;
            if (pass == 0) {
                int st = 0;
                if (!isfinite(a_hi)) st |= OGQ_ST_NONFINITE;
                thresh[t] = (float)(a_hi / (double)n_hi);
                status[t] = st;
                ws.prev_lo[t] = -1;
                ws.done[t] = 0;
            } else {
                const int it = pass - 1;
                if (n_lo == 0 || n_hi == 0) {
                    const double m = (n_lo == 0) ? a_hi / (double)n_hi : a_lo / (double)n_lo;
                    levels[2 * t] = (float)m;
                    levels[2 * t + 1] = (float)m;
                    status[t] |= OGQ_ST_CONSTANT;
                    ws.done[t] = 1;
                } else {
                    const double m_lo = a_lo / (double)n_lo, m_hi = a_hi / (double)n_hi;
                    levels[2 * t] = (float)m_lo;
                    levels[2 * t + 1] = (float)m_hi;
                    if (n_lo == ws.prev_lo[t]) {
                        ws.done[t] = 1;
                    } else if (it >= lloyd_iters) {
                        ws.done[t] = 1;
                        if (lloyd_iters > 0) status[t] |= OGQ_ST_ITER_CAP;
                    } else {
                        ws.prev_lo[t] = n_lo;
                        thresh[t] = (float)((m_lo + m_hi) * 0.5);
                    }
                }
            }
            __threadfence();
        }
    });
}

cudaError_t launch_levels_bingrad_b(const float* d_grad, const int64_t* d_off, int T, int64_t total,
                                    int lloyd_iters, const float* d_tau, float* d_levels, float* d_thresh,
                                    int32_t* d_status, void* d_ws, int sm_count, cudaStream_t stream)
{
    int target = sm_count * 4 < kMaxFlatCtas ? sm_count * 4 : kMaxFlatCtas;
    FlatGrid g = make_flat_grid(total, target, 8192);
    BbWs ws = bb_ws_carve(d_ws, T, g.ctas);
    cudaError_t e = cudaMemsetAsync(d_ws, 0, bb_ws_bytes(T, g.ctas), stream);
    if (e != cudaSuccess) return e;
    for (int pass = 0; pass <= lloyd_iters + 1; ++pass) {
        launch_begin("k_bb_pass", stream);
        if (d_tau)
            k_bb_pass<true><<<g.ctas, kThreads, 0, stream>>>(d_grad, d_off, T, total, g.chunk, pass, lloyd_iters, d_tau,
                                                             d_levels, d_thresh, d_status, ws);
        else
            k_bb_pass<false><<<g.ctas, kThreads, 0, stream>>>(d_grad, d_off, T, total, g.chunk, pass, lloyd_iters, d_tau,
                                                              d_levels, d_thresh, d_status, ws);
        launch_end(stream);
    }
    return cudaGetLastError();
}

size_t ws_bytes_bingrad_b(int T, int64_t /*total*/) { return bb_ws_bytes(T, kMaxFlatCtas); }

// ---------------------------------------------------------------------------
// Variant for callers that cannot allocate device memory: the scratch of the
// BinGrad-b solver lives in a fixed array inside the library image.  The array
// is sized for kNoAllocMaxTensors tensors and the largest flat grid; every GPU
// that loads the library keeps these ~304 KB until the process exits.
// ---------------------------------------------------------------------------
constexpr size_t kNoAllocBytes = 2 * ((sizeof(BbPart) * kMaxFlatCtas + 255) / 256 * 256) +
                                 (sizeof(BbPart) * kNoAllocMaxTensors + 255) / 256 * 256 +
                                 (sizeof(unsigned) * kNoAllocMaxTensors + 255) / 256 * 256 +
                                 (sizeof(int) * kNoAllocMaxTensors + 255) / 256 * 256 +
                                 (sizeof(long long) * kNoAllocMaxTensors + 255) / 256 * 256;

static __device__ __align__(256) unsigned char g_bb_static_scratch[kNoAllocBytes];

// Device address of the array above, looked up once per device.  In host code the symbol's name is
// only a handle, not an address the GPU can use, so the address has to come from the runtime.
// Two host threads that make the first call on a device at the same time both look the address up and
// store the same value: the slot is atomic so that this is well defined.
static std::atomic<void*> g_bb_static_ptr[kNoAllocMaxDevices];

cudaError_t launch_levels_bingrad_b_static(const float* d_grad, const int64_t* d_off, int T, int64_t total,
                                           int lloyd_iters, float* d_levels, float* d_thresh,
                                           int32_t* d_status, int sm_count, cudaStream_t stream)
{
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kNoAllocMaxDevices) return cudaErrorInvalidDevice;
    void* scratch = g_bb_static_ptr[dev].load(std::memory_order_acquire);
    if (scratch == nullptr) {
        e = cudaGetSymbolAddress(&scratch, g_bb_static_scratch);
        if (e != cudaSuccess) return e;
        g_bb_static_ptr[dev].store(scratch, std::memory_order_release);
    }
    int target = sm_count * 4 < kMaxFlatCtas ? sm_count * 4 : kMaxFlatCtas;
    FlatGrid g = make_flat_grid(total, target, 8192);
    // cannot happen for T <= kNoAllocMaxTensors (the caller checked): the array is sized for that many
    // tensors and the largest grid
    if (bb_ws_bytes(T, g.ctas) > kNoAllocBytes) return cudaErrorUnknown;
    BbWs ws = bb_ws_carve(scratch, T, g.ctas);
    // the array still holds the previous call's counters: clear the part this call uses
    e = cudaMemsetAsync(scratch, 0, bb_ws_bytes(T, g.ctas), stream);
    if (e != cudaSuccess) return e;
    for (int pass = 0; pass <= lloyd_iters + 1; ++pass) {
        launch_begin("k_bb_pass", stream);
        k_bb_pass<false><<<g.ctas, kThreads, 0, stream>>>(d_grad, d_off, T, total, g.chunk, pass, lloyd_iters, nullptr,
                                                          d_levels, d_thresh, d_status, ws);
        launch_end(stream);
    }
    return cudaGetLastError();
}

}  // namespace ogq
