// Gradient clipping threshold: tau = c * sigma per tensor, sigma^2 the variance of the tensor about
// its mean (Section "Experiments", paragraph after the list of methods: clip(v) = sign(v) min(|v|, c sigma)).
//
// One streaming read.  Sums of (v - v0) and (v - v0)^2 with v0 the tensor's first element are
// accumulated in fp64 per thread and combined in a fixed order (per-CTA slots, the last CTA of a
// tensor adds them up in CTA order); the variance is (S2 - S1^2 / n) / n, which the shift by v0
// keeps free of the cancellation a large mean would cause.  The clamp itself is applied by the level
// solvers as they read the gradient (the clipped gradient is never written out).
#include <math.h>

#include "ogq_common.cuh"
#include "ogq_internal.h"
#include "ogq_ws.h"

namespace ogq {

__global__ void __launch_bounds__(kThreads)
k_clip_threshold(const float* __restrict__ grad, const int64_t* __restrict__ off, int T, int64_t total,
                 int64_t chunk, float c, float* __restrict__ tau, int32_t* __restrict__ status, BbWs ws)
{
    __shared__ double sh_d[kWarps];
    __shared__ long long sh_l[kWarps];
    __shared__ int sh_last;

    const int64_t lo = (int64_t)blockIdx.x * chunk;
    const int64_t hi = (lo + chunk < total) ? lo + chunk : total;

    if (blockIdx.x == 0) {
        for (int t = threadIdx.x; t < T; t += kThreads) {
            if (__ldg(off + t + 1) <= __ldg(off + t)) {
                tau[t] = 0.f;
                status[t] = OGQ_ST_EMPTY;
            }
        }
    }

    for_each_piece(off, T, lo, hi, [&](int t, int64_t tb, int64_t te, int64_t pb, int64_t pe) {
        const double v0 = (double)__ldg(grad + tb);
        double s1 = 0.0, s2 = 0.0;
        long long bad = 0;
        visit_piece(grad, pb, pe, [&](float v) {
            bad |= ((__float_as_uint(v) & 0x7f800000u) == 0x7f800000u) ? 1 : 0;
            const double d = (double)v - v0;
            s1 += d;
            s2 += d * d;
        });
        s1 = block_sum(s1, sh_d);
        s2 = block_sum(s2, sh_d);
        bad = block_sum(bad, sh_l);

        const int64_t c0 = tb / chunk, c1 = (te - 1) / chunk;
        if (threadIdx.x == 0) {
            BbPart p;
            p.s_lo = s1; p.s_hi = s2; p.c_lo = bad; p.c_hi = 0;
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
        double a1 = 0.0, a2 = 0.0;
        long long nbad = 0;
        if (c0 == c1) {
            if (threadIdx.x == 0) { a1 = s1; a2 = s2; nbad = bad; }
        } else {
            for (int64_t cc = c0 + threadIdx.x; cc <= c1; cc += kThreads) {
                const BbPart* src = (cc == c0) ? ws.slot_b + cc : ws.slot_a + cc;
                a1 += __ldcg(&src->s_lo);
                a2 += __ldcg(&src->s_hi);
                nbad += __ldcg(&src->c_lo);
            }
            a1 = block_sum(a1, sh_d);
            a2 = block_sum(a2, sh_d);
            nbad = block_sum(nbad, sh_l);
        }
        if (threadIdx.x == 0) {
            const double n = (double)(te - tb);
            if (nbad) {
                tau[t] = 0.f;
                status[t] = OGQ_ST_NONFINITE;
            } else {
                double var = (a2 - a1 * a1 / n) / n;
                if (!(var > 0.0)) var = 0.0;
                tau[t] = (float)((double)c * sqrt(var));
                status[t] = 0;
            }
        }
    });
}

cudaError_t launch_clip_threshold(const float* d_grad, const int64_t* d_off, int T, int64_t total, float c,
                                  float* d_tau, int32_t* d_status, void* d_ws, int sm_count, cudaStream_t stream)
{
    int target = sm_count * 4 < kMaxFlatCtas ? sm_count * 4 : kMaxFlatCtas;
    FlatGrid g = make_flat_grid(total, target, 8192);
    BbWs ws = bb_ws_carve(d_ws, T, g.ctas);
    cudaError_t e = cudaMemsetAsync(d_ws, 0, bb_ws_bytes(T, g.ctas), stream);
    if (e != cudaSuccess) return e;
    launch_begin("k_clip_threshold", stream);
    k_clip_threshold<<<g.ctas, kThreads, 0, stream>>>(d_grad, d_off, T, total, g.chunk, c, d_tau, d_status, ws);
    launch_end(stream);
    return cudaGetLastError();
}

}  // namespace ogq
