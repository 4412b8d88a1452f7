// Quantize + bit-pack, and unpack + dequantize + sum over K workers.
//
// Both kernels walk the flat bucket in chunks.  Inside a tensor the unit of work
// is a group of 128 consecutive elements (tensor-relative), which fills exactly
// 4*bits output words; a group belongs to the CTA whose chunk holds its first
// element, so no two CTAs ever touch the same word.  A warp takes one group per
// iteration: lane l handles elements 4l..4l+3 (one 128-bit load, one Philox
// block), and the words are assembled with shuffles inside each 8-lane set,
// which produces exactly `bits` words.
#include <math.h>

#include "ogq_common.cuh"
#include "ogq_internal.h"
#include "ogq_quant.cuh"

namespace ogq {

// CLIP: every value is first clamped to [-tau_arr[t], tau_arr[t]] (gradient clipping).
template <int BITS, bool THRESHOLD, bool CLIP>
__global__ void __launch_bounds__(kThreads)
k_quantize_pack(const float* __restrict__ grad, const int64_t* __restrict__ off, int T, int64_t total,
                int64_t chunk, int s, const float* __restrict__ levels, const float* __restrict__ thresh,
                const float* __restrict__ tau_arr,
                const __grid_constant__ PhiloxKeys keys, uint32_t stream_id,
                const int64_t* __restrict__ packed_off, uint32_t* __restrict__ packed)
{
    __shared__ float sh_lv[kMaxLevels];
    __shared__ float sh_w[kMaxLevels];
    __shared__ float2 sh_tab[kMaxLevels];  // {level k, width of the segment above it}
    // 3- and 5-bit codes: the 4*BITS words of a warp's group are OR-ed together here (kept zero between uses)
    __shared__ uint32_t sh_words[kWarps][(BITS == 3 || BITS == 5) ? 4 * BITS : 1];
    if ((BITS == 3 || BITS == 5) && (threadIdx.x & 31) < 4 * BITS) sh_words[threadIdx.x >> 5][threadIdx.x & 31] = 0u;
    __syncthreads();

    const int64_t lo = (int64_t)blockIdx.x * chunk;
    const int64_t hi = (lo + chunk < total) ? lo + chunk : total;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    for_each_piece(off, T, lo, hi, [&](int t, int64_t tb, int64_t te, int64_t pb, int64_t pe) {
        const int64_t n = te - tb;
        const int64_t g_beg = (pb - tb + 127) >> 7, g_end = (pe - tb + 127) >> 7;
        if (g_beg >= g_end) return;
        float b0 = 0.f;
        const float tau = CLIP ? __ldg(tau_arr + t) : 0.f;
        auto clip = [&](float x) -> float { return CLIP ? copysignf(fminf(fabsf(x), tau), x) : x; };
        if (THRESHOLD) {
            b0 = __ldg(thresh + t);
        } else {
            __syncthreads();
            if (threadIdx.x < s) {
                const float cur = __ldg(levels + (int64_t)t * s + threadIdx.x);
                const float prv = threadIdx.x > 0 ? __ldg(levels + (int64_t)t * s + threadIdx.x - 1) : cur;
                sh_lv[threadIdx.x] = cur;
                sh_w[threadIdx.x] = __fsub_rn(cur, prv);  // width of the segment below level k
                const float nxt = (int)threadIdx.x + 1 < s ? __ldg(levels + (int64_t)t * s + threadIdx.x + 1) : cur;
                sh_tab[threadIdx.x] = make_float2(cur, __fsub_rn(nxt, cur));
            }
            __syncthreads();
        }
        const int64_t region = __ldg(packed_off + t + 1) - __ldg(packed_off + t);
        uint32_t* out = packed + __ldg(packed_off + t);
        const bool aligned = (tb & 3) == 0;
        const float* base = grad + tb;

        // Fast path: groups that lie wholly inside the tensor, 128-bit loads, four groups in flight
        // per warp, no bounds checks.  The generic loop below takes what is left (the last, partial
        // group; everything when the tensor does not start on a 16-byte boundary, or when its Philox
        // counters do not fit 32 bits).
        int64_t g_rest = g_beg;
        if (aligned && n <= ((int64_t)1 << 34)) {
            const int64_t g_full = (n >> 7) < g_end ? (n >> 7) : g_end;
            if (g_full > g_beg) {
                g_rest = g_full;
                constexpr bool kPow2 = (BITS == 1 || BITS == 2 || BITS == 4);
                constexpr int L = kPow2 ? 8 / BITS : 1;  // lanes per word when a word is a whole number of lanes
                const int ng = (int)(g_full - g_beg);
                const float4* src = reinterpret_cast<const float4*>(base + (g_beg << 7)) + lane;
                // which word of the group this lane stores: the first lane of each set of L lanes (see
                // assemble_words), or, for 3 and 5 bits, lane w stores word w after the shared-memory OR
                const bool writer = kPow2 ? (lane & (L - 1)) == 0 : lane < 4 * BITS;
                uint32_t* dstw = out + g_beg * (4 * BITS) + (kPow2 ? lane / L : lane);
                uint32_t* wsm = sh_words[warp];
                const int obit = (lane * 4 * BITS) & 31, oword = (lane * 4 * BITS) >> 5;  // kPow2 == false only
                const uint32_t c0_first = (uint32_t)(g_beg << 5) + (uint32_t)lane;  // counters fit 32 bits here
                const uint32_t tabaddr = (uint32_t)__cvta_generic_to_shared(sh_tab);
                // the sum of the four entry addresses of a lane carries this multiple of the table's base
                const uint32_t tab4 = tabaddr * (1u + (1u << BITS) + (1u << (2 * BITS)) + (1u << (3 * BITS)));
                float mid = 0.f;
                PhiloxHoist hz = {};
                if constexpr (!THRESHOLD) {
                    mid = sh_tab[(BITS >= 2) ? (1 << (BITS - 2)) : 0].x;
                    hz = philox_hoist(0u, (uint32_t)t, stream_id, keys);
                }
                auto code4 = [&](float4 v, int gl) -> uint32_t {
                    if constexpr (CLIP) { v.x = clip(v.x); v.y = clip(v.y); v.z = clip(v.z); v.w = clip(v.w); }
                    if constexpr (THRESHOLD) {
                        const uint32_t b4 = ((v.x >= b0) ? 1u : 0u) | ((v.y >= b0) ? 2u : 0u) |
                                            ((v.z >= b0) ? 4u : 0u) | ((v.w >= b0) ? 8u : 0u);
                        return assemble_words<BITS>(b4, lane);
                    } else {
                        const uint4 r = philox4x32_10_tail(c0_first + ((uint32_t)gl << 5), hz, keys);
                        const uint32_t a0 = entry_after_rounding<BITS>(v.x, r.x, tabaddr, mid),
                                       a1 = entry_after_rounding<BITS>(v.y, r.y, tabaddr, mid),
                                       a2 = entry_after_rounding<BITS>(v.z, r.z, tabaddr, mid),
                                       a3 = entry_after_rounding<BITS>(v.w, r.w, tabaddr, mid);
                        // entries are 8 bytes apart: (address - base) / 8 is the code
                        const uint32_t bits4 =
                            (a0 + (a1 << BITS) + (a2 << (2 * BITS)) + (a3 << (3 * BITS)) - tab4) >> 3;
                        if constexpr (kPow2) {
                            return assemble_words<BITS>(bits4, lane);
                        } else {
                            // a lane's 4*BITS bits touch at most two words of the group
                            atomicOr(wsm + oword, bits4 << obit);
                            if (obit + 4 * BITS > 32) atomicOr(wsm + oword + 1, bits4 >> (32 - obit));
                            __syncwarp();
                            const uint32_t word = writer ? atomicExch(wsm + lane, 0u) : 0u;
                            __syncwarp();
                            return word;
                        }
                    }
                };
                constexpr int U = 4;  // groups per warp and trip: all loads are issued before the first use
                for (int gl = warp; gl < ng; gl += U * kWarps) {
                    float4 v[U];
#pragma unroll
                    for (int u = 0; u < U; ++u)
                        if (gl + u * kWarps < ng) v[u] = __ldg(src + (size_t)(gl + u * kWarps) * 32);
#pragma unroll
                    for (int u = 0; u < U; ++u)
                        if (gl + u * kWarps < ng) {
                            const uint32_t w = code4(v[u], gl + u * kWarps);
                            if (writer) dstw[(size_t)(gl + u * kWarps) * (4 * BITS)] = w;
                        }
                }
            }
        }

        for (int64_t g = g_rest + warp; g < g_end; g += kWarps) {
            const int64_t i0 = (g << 7) + 4 * lane;
            float x[4];
            if (aligned && i0 + 3 < n) {
                const float4 v = __ldg(reinterpret_cast<const float4*>(base + i0));
                x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) x[j] = (i0 + j < n) ? __ldg(base + i0 + j) : 0.f;
            }
            if constexpr (CLIP) {
#pragma unroll
                for (int j = 0; j < 4; ++j) x[j] = clip(x[j]);
            }
            uint32_t c[4];
            if (THRESHOLD) {
#pragma unroll
                for (int j = 0; j < 4; ++j) c[j] = (x[j] >= b0) ? 1u : 0u;
            } else {
                const uint64_t q = (uint64_t)i0 >> 2;
                const uint4 r = philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), (uint32_t)t, stream_id, keys);
                const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    // s = 2^(BITS-1) + 1 levels (s = 2 for BITS = 1): BITS - 1 halving steps
                    int idx = 0;
#pragma unroll
                    for (int step = (BITS >= 2) ? (1 << (BITS - 2)) : 0; step >= 1; step >>= 1)
                        if (sh_lv[idx + step] <= x[j]) idx += step;
                    const float d = __fsub_rn(x[j], sh_lv[idx]);
                    const float lhs = __fmul_rn((float)(rw[j] >> 8), sh_w[idx + 1]);
                    const float rhs = __fmul_rn(d, 16777216.0f);
                    c[j] = (uint32_t)idx + ((lhs < rhs) ? 1u : 0u);
                }
            }
            if (i0 + 3 >= n) {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (i0 + j >= n) c[j] = 0u;  // zero padding beyond the tensor
            }
            const uint32_t bits4 = c[0] | (c[1] << BITS) | (c[2] << (2 * BITS)) | (c[3] << (3 * BITS));
            if constexpr (BITS == 1 || BITS == 2 || BITS == 4) {
                const uint32_t word = assemble_words<BITS>(bits4, lane);
                constexpr int L = 8 / (BITS == 3 || BITS == 5 ? 1 : BITS);
                if ((lane & (L - 1)) == 0) {
                    const int64_t widx = g * (4 * BITS) + lane / L;
                    if (widx < region) out[widx] = word;
                }
            } else {
                // 3 and 5 bits: OR the lanes' bits into the group's 4*BITS words in shared memory
                uint32_t* wsm = sh_words[warp];
                const int obit = (lane * 4 * BITS) & 31, oword = (lane * 4 * BITS) >> 5;
                atomicOr(wsm + oword, bits4 << obit);
                if (obit + 4 * BITS > 32) atomicOr(wsm + oword + 1, bits4 >> (32 - obit));
                __syncwarp();
                if (lane < 4 * BITS) {
                    const uint32_t word = atomicExch(wsm + lane, 0u);
                    const int64_t widx = g * (4 * BITS) + lane;
                    if (widx < region) out[widx] = word;
                }
                __syncwarp();
            }
        }
    });
}

// Two fp32 additions in one instruction (each rounded to nearest): (a0, a1) += (b0, b1).
__device__ __forceinline__ void add2(float& a0, float& a1, float b0, float b1)
{
    unsigned long long a, b;
    asm("mov.b64 %0, {%1, %2};" : "=l"(a) : "f"(a0), "f"(a1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(b) : "f"(b0), "f"(b1));
    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(a) : "l"(b));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(a));
}

template <int BITS>
__global__ void __launch_bounds__(kThreads)
k_unpack_sum(const uint32_t* const* __restrict__ packed_k, const float* const* __restrict__ levels_k, int K,
             const int64_t* __restrict__ off, const int64_t* __restrict__ packed_off, int T, int64_t total,
             int64_t chunk, int s, float scale, float* __restrict__ outp)
{
    __shared__ float sh_lv[kMaxWorkers][kMaxLevels + 1];
    __shared__ const uint32_t* sh_pk[kMaxWorkers];

    const int64_t lo = (int64_t)blockIdx.x * chunk;
    const int64_t hi = (lo + chunk < total) ? lo + chunk : total;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr uint32_t kMask4 = (BITS * 4 >= 32) ? 0xffffffffu : ((1u << (BITS * 4)) - 1u);
    constexpr uint32_t kMask1 = (1u << BITS) - 1u;

    for_each_piece(off, T, lo, hi, [&](int t, int64_t tb, int64_t te, int64_t pb, int64_t pe) {
        const int64_t n = te - tb;
        const int64_t g_beg = (pb - tb + 127) >> 7, g_end = (pe - tb + 127) >> 7;
        if (g_beg >= g_end) return;
        __syncthreads();
        // every code a BITS-bit field can hold gets an entry: codes above s - 1 (never produced by the
        // quantizer) read the top level, so the inner loops need no clamp
        for (int i = threadIdx.x; i < K * 32; i += kThreads) {
            const int k = i >> 5, q = i & 31;
            sh_lv[k][q] = __ldg(levels_k[k] + (int64_t)t * s + (q < s ? q : s - 1));
        }
        const int64_t pofs = __ldg(packed_off + t);
        if (threadIdx.x < K) sh_pk[threadIdx.x] = packed_k[threadIdx.x] + pofs;
        __syncthreads();
        const int64_t region = __ldg(packed_off + t + 1) - pofs;
        const bool aligned = (tb & 3) == 0;
        float* dst = outp + tb;

        // Fast path (1, 2 or 4 bits per code): groups wholly inside the tensor, eight workers' words in
        // flight per lane, level rows addressed with compile-time offsets.  All lanes of a warp read the
        // same few level entries, so the shared-memory loads are broadcasts.
        int64_t g_rest = g_beg;
        if ((BITS == 1 || BITS == 2 || BITS == 4) && aligned) {
            const int64_t g_full = (n >> 7) < g_end ? (n >> 7) : g_end;
            if (g_full > g_beg) {
                g_rest = g_full;
                constexpr int L = 8 / BITS;                       // lanes per packed word
                const int shift = (lane & (L - 1)) * 4 * BITS;    // this lane's 4 codes inside its word
                const int64_t w0 = g_beg * (4 * BITS) + lane / L;
                float4* dst4 = reinterpret_cast<float4*>(dst + (g_beg << 7)) + lane;
                const int ng = (int)(g_full - g_beg);
                const char* rows = reinterpret_cast<const char*>(&sh_lv[0][0]);
                constexpr int kRow = (kMaxLevels + 1) * (int)sizeof(float);
                constexpr int kAhead = 16;  // trips (of kWarps groups) between two prefetch requests
                // adds the levels of the four codes of this lane in word w (worker row r) to a[0..3]
                auto add4 = [&](uint32_t w, const char* r, float* a) {
                    const uint32_t f = (w >> shift) << 2;  // byte offsets of the 4 codes
                    const float l0 = *reinterpret_cast<const float*>(r + (f & (kMask1 << 2)));
                    const float l1 = *reinterpret_cast<const float*>(r + ((f >> BITS) & (kMask1 << 2)));
                    const float l2 = *reinterpret_cast<const float*>(r + ((f >> (2 * BITS)) & (kMask1 << 2)));
                    const float l3 = *reinterpret_cast<const float*>(r + ((f >> (3 * BITS)) & (kMask1 << 2)));
                    add2(a[0], a[1], l0, l1);  // same fp32 additions, two per instruction
                    add2(a[2], a[3], l2, l3);
                };
                // two groups per warp and trip: sixteen word loads in flight per lane
                for (int gl = warp; gl < ng; gl += 2 * kWarps) {
                    // every kAhead trips the first K threads ask L2 for the K workers' words of the
                    // kAhead trips after the next kAhead (no gain at one bit per code)
                    const int tr = gl / kWarps;
                    if (BITS >= 2 && (tr & (kAhead - 1)) == 0 && (int)threadIdx.x < K && (tr + 2 * kAhead) * kWarps <= ng)
                        prefetch_l2(sh_pk[threadIdx.x] + (g_beg + (int64_t)(tr + kAhead) * kWarps) * (4 * BITS),
                                    kAhead * kWarps * 4u * BITS * 4u);
                    const bool two = gl + kWarps < ng;
                    const int64_t wa = w0 + (int64_t)gl * (4 * BITS);
                    const int64_t wb = two ? wa + (int64_t)kWarps * (4 * BITS) : wa;
                    float a[4] = {0.f, 0.f, 0.f, 0.f}, b[4] = {0.f, 0.f, 0.f, 0.f};
                    int k0 = 0;
                    for (; k0 + 8 <= K; k0 += 8) {
                        uint32_t xa[8], xb[8];
#pragma unroll
                        for (int u = 0; u < 8; ++u) xa[u] = __ldg(sh_pk[k0 + u] + wa);
#pragma unroll
                        for (int u = 0; u < 8; ++u) xb[u] = __ldg(sh_pk[k0 + u] + wb);
                        const char* r0 = rows + k0 * kRow;
#pragma unroll
                        for (int u = 0; u < 8; ++u) add4(xa[u], r0 + u * kRow, a);
#pragma unroll
                        for (int u = 0; u < 8; ++u) add4(xb[u], r0 + u * kRow, b);
                    }
                    for (; k0 < K; ++k0) {
                        const uint32_t xa = __ldg(sh_pk[k0] + wa), xb = __ldg(sh_pk[k0] + wb);
                        add4(xa, rows + k0 * kRow, a);
                        add4(xb, rows + k0 * kRow, b);
                    }
                    dst4[(size_t)gl * 32] = make_float4(__fmul_rn(a[0], scale), __fmul_rn(a[1], scale),
                                                        __fmul_rn(a[2], scale), __fmul_rn(a[3], scale));
                    if (two)
                        dst4[(size_t)(gl + kWarps) * 32] = make_float4(__fmul_rn(b[0], scale), __fmul_rn(b[1], scale),
                                                                       __fmul_rn(b[2], scale), __fmul_rn(b[3], scale));
                }
            }
        }

        for (int64_t g = g_rest + warp; g < g_end; g += kWarps) {
            const int64_t i0 = (g << 7) + 4 * lane;
            if (i0 >= n) continue;
            const int64_t bit = i0 * BITS;
            const int64_t wi = bit >> 5;
            const int sh = (int)(bit & 31);
            const bool two = (sh + 4 * BITS > 32) && (wi + 1 < region);
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
            for (int k = 0; k < K; ++k) {
                const uint32_t* p = sh_pk[k];
                const uint32_t w_lo = __ldg(p + wi);
                const uint32_t w_hi = two ? __ldg(p + wi + 1) : 0u;
                const uint32_t bits4 = __funnelshift_r(w_lo, w_hi, sh) & kMask4;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t code = (bits4 >> (j * BITS)) & kMask1;
                    acc[j] = __fadd_rn(acc[j], sh_lv[k][code]);
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) acc[j] = __fmul_rn(acc[j], scale);
            if (aligned && i0 + 3 < n) {
                *reinterpret_cast<float4*>(dst + i0) = make_float4(acc[0], acc[1], acc[2], acc[3]);
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    if (i0 + j < n) dst[i0 + j] = acc[j];
            }
        }
    });
}

static int flat_target(int sm_count)
{
    int t = sm_count * 8;
    return t < kMaxFlatCtas ? t : kMaxFlatCtas;
}

cudaError_t launch_quantize_pack(const float* d_grad, const int64_t* d_off, int T, int64_t total,
                                 int scheme, int s, const float* d_levels, const float* d_thresh,
                                 const float* d_tau, uint64_t seed, uint32_t stream_id,
                                 const int64_t* d_packed_off, uint32_t* d_packed, int sm_count,
                                 cudaStream_t stream)
{
    FlatGrid g = make_flat_grid(total, flat_target(sm_count), 8192);
    const PhiloxKeys keys = philox_round_keys((uint32_t)seed, (uint32_t)(seed >> 32));
    const int bits = ogq_bits_for_levels(s);
#define OGQ_LAUNCH_QC(B, TH, CL)                                                                        \
    k_quantize_pack<B, TH, CL><<<g.ctas, kThreads, 0, stream>>>(d_grad, d_off, T, total, g.chunk, s,    \
                                                                d_levels, d_thresh, d_tau, keys,        \
                                                                stream_id, d_packed_off, d_packed)
#define OGQ_LAUNCH_Q(B, TH)                    \
    do {                                       \
        if (d_tau) OGQ_LAUNCH_QC(B, TH, true); \
        else OGQ_LAUNCH_QC(B, TH, false);      \
    } while (0)
    launch_begin(scheme == OGQ_BINGRAD_B ? "k_quantize_pack_threshold" : "k_quantize_pack_random", stream);
    if (scheme == OGQ_BINGRAD_B) {
        OGQ_LAUNCH_Q(1, true);
    } else {
        switch (bits) {
            case 1: OGQ_LAUNCH_Q(1, false); break;
            case 2: OGQ_LAUNCH_Q(2, false); break;
            case 3: OGQ_LAUNCH_Q(3, false); break;
            case 4: OGQ_LAUNCH_Q(4, false); break;
            case 5: OGQ_LAUNCH_Q(5, false); break;
            default: return cudaErrorInvalidValue;
        }
    }
#undef OGQ_LAUNCH_Q
#undef OGQ_LAUNCH_QC
    launch_end(stream);
    return cudaGetLastError();
}

cudaError_t launch_unpack_sum(const uint32_t* const* d_packed_k, const float* const* d_levels_k, int K,
                              const int64_t* d_off, const int64_t* d_packed_off, int T, int64_t total,
                              int s, float scale, float* d_out, int sm_count, cudaStream_t stream)
{
    FlatGrid g = make_flat_grid(total, flat_target(sm_count), 8192);
    const int bits = ogq_bits_for_levels(s);
#define OGQ_LAUNCH_U(B)                                                                               \
    k_unpack_sum<B><<<g.ctas, kThreads, 0, stream>>>(d_packed_k, d_levels_k, K, d_off, d_packed_off, T, \
                                                     total, g.chunk, s, scale, d_out)
    launch_begin("k_unpack_sum", stream);
    switch (bits) {
        case 1: OGQ_LAUNCH_U(1); break;
        case 2: OGQ_LAUNCH_U(2); break;
        case 3: OGQ_LAUNCH_U(3); break;
        case 4: OGQ_LAUNCH_U(4); break;
        case 5: OGQ_LAUNCH_U(5); break;
        default: return cudaErrorInvalidValue;
    }
#undef OGQ_LAUNCH_U
    launch_end(stream);
    return cudaGetLastError();
}

}  // namespace ogq
