// Quantization error per tensor: the realised ||Q(G) - G||^2 of given packed codes (the quantity the
// paper tracks in its training curves), or its expectation over the random rounding,
// sum (v - lo)(hi - v), the functional the optimal condition minimises (proof of Theorem 1).
//
// A diagnostic, not part of the encode / decode path.  fp64 per thread, one fp64 atomic per CTA and
// tensor piece: the result does not depend on the data layout but its last bits depend on the order
// in which the CTAs arrive.
#include <math.h>

#include "ogq_common.cuh"
#include "ogq_internal.h"
#include "ogq_quant.cuh"

namespace ogq {

__global__ void __launch_bounds__(kThreads)
k_quant_error(const float* __restrict__ grad, const int64_t* __restrict__ off, int T, int64_t total, int64_t chunk,
              int s, int bits, const float* __restrict__ levels, const int64_t* __restrict__ packed_off,
              const uint32_t* __restrict__ packed, double* __restrict__ err)
{
    __shared__ double sh_lv[kMaxLevels];
    __shared__ double sh_d[kWarps];
    const int64_t lo = (int64_t)blockIdx.x * chunk;
    const int64_t hi = (lo + chunk < total) ? lo + chunk : total;
    const uint32_t mask = (1u << bits) - 1u;

    for_each_piece(off, T, lo, hi, [&](int t, int64_t tb, int64_t te, int64_t pb, int64_t pe) {
        __syncthreads();
        if (threadIdx.x < s) sh_lv[threadIdx.x] = (double)__ldg(levels + (int64_t)t * s + threadIdx.x);
        __syncthreads();
        const uint32_t* words = packed ? packed + __ldg(packed_off + t) : nullptr;
        const int64_t region = packed ? __ldg(packed_off + t + 1) - __ldg(packed_off + t) : 0;
        double acc = 0.0;
        for (int64_t i = pb + threadIdx.x; i < pe; i += kThreads) {
            const double x = (double)__ldg(grad + i);
            if (words) {
                const int64_t bit = (i - tb) * bits;
                const int64_t wi = bit >> 5;
                const int sh = (int)(bit & 31);
                const uint32_t w_lo = __ldg(words + wi);
                const uint32_t w_hi = (sh + bits > 32 && wi + 1 < region) ? __ldg(words + wi + 1) : 0u;
                uint32_t code = __funnelshift_r(w_lo, w_hi, sh) & mask;
                if (code > (uint32_t)(s - 1)) code = s - 1;
                const double d = sh_lv[code] - x;
                acc += d * d;
            } else {
                const double b0 = sh_lv[0], bs = sh_lv[s - 1];
                if (x < b0) acc += (b0 - x) * (b0 - x);
                else if (x > bs) acc += (x - bs) * (x - bs);
                else {
                    int k = 0;
                    for (int q = 0; q < s; ++q) k += (sh_lv[q] <= x) ? 1 : 0;
                    k = k < 1 ? 1 : (k > s - 1 ? s - 1 : k);
                    acc += (x - sh_lv[k - 1]) * (sh_lv[k] - x);
                }
            }
        }
        acc = block_sum(acc, sh_d);
        if (threadIdx.x == 0) atomicAdd(err + t, acc);
    });
}

cudaError_t launch_quant_error(const float* d_grad, const int64_t* d_off, int T, int64_t total, int s,
                               const float* d_levels, const int64_t* d_packed_off, const uint32_t* d_packed,
                               double* d_err, int sm_count, cudaStream_t stream)
{
    int target = sm_count * 8 < kMaxFlatCtas ? sm_count * 8 : kMaxFlatCtas;
    FlatGrid g = make_flat_grid(total, target, 8192);
    cudaError_t e = cudaMemsetAsync(d_err, 0, sizeof(double) * (size_t)T, stream);
    if (e != cudaSuccess) return e;
    launch_begin("k_quant_error", stream);
    k_quant_error<<<g.ctas, kThreads, 0, stream>>>(d_grad, d_off, T, total, g.chunk, s, ogq_bits_for_levels(s), d_levels,
                                                   d_packed_off, d_packed, d_err);
    launch_end(stream);
    return cudaGetLastError();
}

}  // namespace ogq
