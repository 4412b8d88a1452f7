// Entropy-dense wire format: M consecutive codes are the base-s digits of one 32-bit word (least
// significant first), M the largest count with s^M <= 2^32: 20 codes per word for s = 3, 13 for
// s = 5, 10 for s = 9, 7 for s = 17, i.e. 1.6 / 2.46 / 3.2 / 4.57 bits per element instead of
// 2 / 3 / 4 / 5.  The paper's compression ratios (x20.2, x13.8, x10.1) assume log2(s) bits per code;
// this is the closest whole-word format.  Quantization itself (segment search, Philox draw, rounding
// decision) is the one of the bit-packed path: only the packing differs.
//
// Unit of work: a group of U = lcm(4, M) consecutive elements of a tensor, which is a whole number of
// 128-bit loads and Philox blocks (U / 4) and of output words (U / M).  A lane takes one group per
// trip, a warp 32 consecutive groups; a group belongs to the CTA whose chunk holds its first element.
#include <math.h>

#include "ogq_common.cuh"
#include "ogq_internal.h"
#include "ogq_quant.cuh"

namespace ogq {

template <int S> struct Dense;
template <> struct Dense<3>  { static constexpr int M = 20, U = 20, BITS = 2; };
template <> struct Dense<5>  { static constexpr int M = 13, U = 52, BITS = 3; };
template <> struct Dense<9>  { static constexpr int M = 10, U = 20, BITS = 4; };
template <> struct Dense<17> { static constexpr int M = 7,  U = 28, BITS = 5; };

__host__ __device__ constexpr uint32_t dense_pow(int s, int q)
{
    uint32_t p = 1;
    for (int i = 0; i < q; ++i) p *= (uint32_t)s;
    return p;
}

int dense_digits(int s)
{
    switch (s) {
        case 3: return 20;
        case 5: return 13;
        case 9: return 10;
        case 17: return 7;
        default: return 0;
    }
}

template <int S>
__global__ void __launch_bounds__(kThreads)
k_quantize_pack_dense(const float* __restrict__ grad, const int64_t* __restrict__ off, int T, int64_t total,
                      int64_t chunk, const float* __restrict__ levels, const __grid_constant__ PhiloxKeys keys,
                      uint32_t stream_id, const int64_t* __restrict__ packed_off, uint32_t* __restrict__ packed)
{
    constexpr int M = Dense<S>::M, U = Dense<S>::U, BITS = Dense<S>::BITS, W = U / M, Q = U / 4;
    __shared__ float sh_lv[kMaxLevels];
    __shared__ float sh_w[kMaxLevels];
    __shared__ float2 sh_tab[kMaxLevels];

    const int64_t lo = (int64_t)blockIdx.x * chunk;
    const int64_t hi = (lo + chunk < total) ? lo + chunk : total;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    for_each_piece(off, T, lo, hi, [&](int t, int64_t tb, int64_t te, int64_t pb, int64_t pe) {
        const int64_t n = te - tb;
        const int64_t g_beg = (pb - tb + U - 1) / U, g_end = (pe - tb + U - 1) / U;
        if (g_beg >= g_end) return;
        __syncthreads();
        if (threadIdx.x < S) {
            const float cur = __ldg(levels + (int64_t)t * S + threadIdx.x);
            const float prv = threadIdx.x > 0 ? __ldg(levels + (int64_t)t * S + threadIdx.x - 1) : cur;
            const float nxt = (int)threadIdx.x + 1 < S ? __ldg(levels + (int64_t)t * S + threadIdx.x + 1) : cur;
            sh_lv[threadIdx.x] = cur;
            sh_w[threadIdx.x] = __fsub_rn(cur, prv);
            sh_tab[threadIdx.x] = make_float2(cur, __fsub_rn(nxt, cur));
        }
        __syncthreads();
        const int64_t region = __ldg(packed_off + t + 1) - __ldg(packed_off + t);
        uint32_t* out = packed + __ldg(packed_off + t);
        const float* base = grad + tb;
        const bool aligned = (tb & 3) == 0;

        int64_t g_rest = g_beg;
        if (aligned && n <= ((int64_t)1 << 34)) {
            const int64_t g_full = (n / U) < g_end ? (n / U) : g_end;
            if (g_full > g_beg) {
                g_rest = g_full;
                const uint32_t tabaddr = (uint32_t)__cvta_generic_to_shared(sh_tab);
                const float mid = sh_tab[1 << (BITS - 2)].x;
                const PhiloxHoist hz = philox_hoist(0u, (uint32_t)t, stream_id, keys);
                for (int64_t g = g_beg + (int64_t)warp * 32 + lane; g < g_full; g += (int64_t)kWarps * 32) {
                    const float4* src = reinterpret_cast<const float4*>(base + g * U);
                    float4 v[Q];
#pragma unroll
                    for (int q = 0; q < Q; ++q) v[q] = __ldg(src + q);
                    uint32_t word[W];
#pragma unroll
                    for (int w = 0; w < W; ++w) word[w] = 0u;
                    const uint32_t c0 = (uint32_t)(g * Q);
#pragma unroll
                    for (int q = 0; q < Q; ++q) {
                        const uint4 r = philox4x32_10_tail(c0 + (uint32_t)q, hz, keys);
                        const float x[4] = {v[q].x, v[q].y, v[q].z, v[q].w};
                        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const int e = 4 * q + j;  // position in the group (compile time after unrolling)
                            const uint32_t code = (entry_after_rounding<BITS>(x[j], rw[j], tabaddr, mid) - tabaddr) >> 3;
                            word[e / M] += code * dense_pow(S, e % M);
                        }
                    }
                    uint32_t* dst = out + g * W;
                    if constexpr (W == 1) dst[0] = word[0];
                    else if constexpr (W == 2) *reinterpret_cast<uint2*>(dst) = make_uint2(word[0], word[1]);
                    else *reinterpret_cast<uint4*>(dst) = make_uint4(word[0], word[1], word[2], word[3]);
                }
            }
        }

        // generic path: one thread per output word, element by element (the last, partial group;
        // everything when the tensor does not start on a 16-byte boundary)
        // (the CTA that owns the tensor's last group also writes the zero padding of the region)
        const int64_t w_beg = g_rest * W;
        const int64_t w_end = (g_end == (n + U - 1) / U) ? region : g_end * W;
        for (int64_t wi = w_beg + threadIdx.x; wi < w_end; wi += kThreads) {
            uint32_t word = 0u, p = 1u;
            for (int d = 0; d < M; ++d) {
                const int64_t i = wi * M + d;
                if (i < n) {
                    const float x = __ldg(base + i);
                    const uint64_t blk = (uint64_t)i >> 2;
                    const uint4 r = philox4x32_10((uint32_t)blk, (uint32_t)(blk >> 32), (uint32_t)t, stream_id, keys);
                    const uint32_t rnd = (i & 3) == 0 ? r.x : ((i & 3) == 1 ? r.y : ((i & 3) == 2 ? r.z : r.w));
                    int idx = 0;
                    for (int step = 1 << (BITS - 2); step >= 1; step >>= 1)
                        if (sh_lv[idx + step] <= x) idx += step;
                    const float dd = __fsub_rn(x, sh_lv[idx]);
                    const float lhs = __fmul_rn((float)(rnd >> 8), sh_w[idx + 1]);
                    const float rhs = __fmul_rn(dd, 16777216.0f);
                    word += ((uint32_t)idx + ((lhs < rhs) ? 1u : 0u)) * p;
                }
                p *= (uint32_t)S;
            }
            out[wi] = word;
        }
    });
}

template <int S>
__global__ void __launch_bounds__(kThreads)
k_unpack_sum_dense(const uint32_t* const* __restrict__ packed_k, const float* const* __restrict__ levels_k, int K,
                   const int64_t* __restrict__ off, const int64_t* __restrict__ packed_off, int T, int64_t total,
                   int64_t chunk, float scale, float* __restrict__ outp)
{
    constexpr int M = Dense<S>::M, U = Dense<S>::U, W = U / M, Q = U / 4;
    __shared__ float sh_lv[kMaxWorkers][kMaxLevels + 1];
    __shared__ const uint32_t* sh_pk[kMaxWorkers];

    const int64_t lo = (int64_t)blockIdx.x * chunk;
    const int64_t hi = (lo + chunk < total) ? lo + chunk : total;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    for_each_piece(off, T, lo, hi, [&](int t, int64_t tb, int64_t te, int64_t pb, int64_t pe) {
        const int64_t n = te - tb;
        const int64_t g_beg = (pb - tb + U - 1) / U, g_end = (pe - tb + U - 1) / U;
        if (g_beg >= g_end) return;
        __syncthreads();
        for (int i = threadIdx.x; i < K * 32; i += kThreads) {
            const int k = i >> 5, q = i & 31;
            sh_lv[k][q] = __ldg(levels_k[k] + (int64_t)t * S + (q < S ? q : S - 1));
        }
        const int64_t pofs = __ldg(packed_off + t);
        if (threadIdx.x < K) sh_pk[threadIdx.x] = packed_k[threadIdx.x] + pofs;
        __syncthreads();
        float* dst = outp + tb;
        const bool aligned = (tb & 3) == 0;

        int64_t g_rest = g_beg;
        if (aligned) {
            const int64_t g_full = (n / U) < g_end ? (n / U) : g_end;
            if (g_full > g_beg) {
                g_rest = g_full;
                for (int64_t g = g_beg + (int64_t)warp * 32 + lane; g < g_full; g += (int64_t)kWarps * 32) {
                    float acc[U];
#pragma unroll
                    for (int e = 0; e < U; ++e) acc[e] = 0.f;
                    for (int k = 0; k < K; ++k) {
                        const uint32_t* src = sh_pk[k] + g * W;
                        uint32_t word[W];
                        if constexpr (W == 1) word[0] = __ldg(src);
                        else if constexpr (W == 2) { const uint2 x = __ldg(reinterpret_cast<const uint2*>(src)); word[0] = x.x; word[1] = x.y; }
                        else { const uint4 x = __ldg(reinterpret_cast<const uint4*>(src)); word[0] = x.x; word[1] = x.y; word[2] = x.z; word[3] = x.w; }
                        const float* row = sh_lv[k];
#pragma unroll
                        for (int w = 0; w < W; ++w) {
                            uint32_t rest = word[w];
#pragma unroll
                            for (int d = 0; d < M; ++d) {
                                const uint32_t qd = rest / (uint32_t)S;  // constant divisor: multiply and shift
                                const uint32_t digit = rest - qd * (uint32_t)S;
                                rest = qd;
                                acc[w * M + d] = __fadd_rn(acc[w * M + d], row[digit]);
                            }
                        }
                    }
                    float4* d4 = reinterpret_cast<float4*>(dst + g * U);
#pragma unroll
                    for (int q = 0; q < Q; ++q)
                        d4[q] = make_float4(__fmul_rn(acc[4 * q], scale), __fmul_rn(acc[4 * q + 1], scale),
                                            __fmul_rn(acc[4 * q + 2], scale), __fmul_rn(acc[4 * q + 3], scale));
                }
            }
        }

        // generic path: one thread per element
        const int64_t e_beg = g_rest * U;
        int64_t e_end = g_end * U;
        if (e_end > n) e_end = n;
        for (int64_t i = e_beg + threadIdx.x; i < e_end; i += kThreads) {
            const int64_t wi = i / M;
            const int d = (int)(i - wi * M);
            float acc = 0.f;
            for (int k = 0; k < K; ++k) {
                uint32_t rest = __ldg(sh_pk[k] + wi);
                for (int q = 0; q < d; ++q) rest /= (uint32_t)S;
                acc = __fadd_rn(acc, sh_lv[k][rest % (uint32_t)S]);
            }
            dst[i] = __fmul_rn(acc, scale);
        }
    });
}

static int dense_flat_target(int sm_count)
{
    int t = sm_count * 8;
    return t < kMaxFlatCtas ? t : kMaxFlatCtas;
}

cudaError_t launch_quantize_pack_dense(const float* d_grad, const int64_t* d_off, int T, int64_t total, int s,
                                       const float* d_levels, uint64_t seed, uint32_t stream_id,
                                       const int64_t* d_packed_off, uint32_t* d_packed, int sm_count,
                                       cudaStream_t stream)
{
    FlatGrid g = make_flat_grid(total, dense_flat_target(sm_count), 16640);  // a multiple of every group length
    const PhiloxKeys keys = philox_round_keys((uint32_t)seed, (uint32_t)(seed >> 32));
    launch_begin("k_quantize_pack_dense", stream);
#define OGQ_LAUNCH_D(SS)                                                                                     \
    k_quantize_pack_dense<SS><<<g.ctas, kThreads, 0, stream>>>(d_grad, d_off, T, total, g.chunk, d_levels,  \
                                                               keys, stream_id, d_packed_off, d_packed)
    switch (s) {
        case 3: OGQ_LAUNCH_D(3); break;
        case 5: OGQ_LAUNCH_D(5); break;
        case 9: OGQ_LAUNCH_D(9); break;
        case 17: OGQ_LAUNCH_D(17); break;
        default: return cudaErrorInvalidValue;
    }
#undef OGQ_LAUNCH_D
    launch_end(stream);
    return cudaGetLastError();
}

cudaError_t launch_unpack_sum_dense(const uint32_t* const* d_packed_k, const float* const* d_levels_k, int K,
                                    const int64_t* d_off, const int64_t* d_packed_off, int T, int64_t total, int s,
                                    float scale, float* d_out, int sm_count, cudaStream_t stream)
{
    FlatGrid g = make_flat_grid(total, dense_flat_target(sm_count), 16640);
    launch_begin("k_unpack_sum_dense", stream);
#define OGQ_LAUNCH_UD(SS)                                                                                       \
    k_unpack_sum_dense<SS><<<g.ctas, kThreads, 0, stream>>>(d_packed_k, d_levels_k, K, d_off, d_packed_off, T, \
                                                            total, g.chunk, scale, d_out)
    switch (s) {
        case 3: OGQ_LAUNCH_UD(3); break;
        case 5: OGQ_LAUNCH_UD(5); break;
        case 9: OGQ_LAUNCH_UD(9); break;
        case 17: OGQ_LAUNCH_UD(17); break;
        default: return cudaErrorInvalidValue;
    }
#undef OGQ_LAUNCH_UD
    launch_end(stream);
    return cudaGetLastError();
}

}  // namespace ogq
