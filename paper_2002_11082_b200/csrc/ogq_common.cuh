// Shared device helpers of the gradient-quantization kernels (sm_100a).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/ogq.h"

namespace ogq {

constexpr int kThreads = 256;       // threads per CTA of every streaming kernel
constexpr int kWarps = kThreads / 32;
constexpr int kChunkAlign = 1024;   // flat chunk boundaries are multiples of this many elements

// ---------------------------------------------------------------------------
// Flat partition of the bucket: CTA c owns elements [c*chunk, (c+1)*chunk).
// ---------------------------------------------------------------------------
struct FlatGrid {
    int64_t chunk;  // elements per CTA, multiple of kChunkAlign
    int ctas;       // number of CTAs
};

inline FlatGrid make_flat_grid(int64_t total, int target_ctas, int64_t min_chunk)
{
    FlatGrid g;
    if (total <= 0) {
        g.chunk = kChunkAlign;
        g.ctas = 1;
        return g;
    }
    int64_t c = (total + target_ctas - 1) / target_ctas;
    if (c < min_chunk) c = min_chunk;
    c = (c + kChunkAlign - 1) / kChunkAlign * kChunkAlign;
    g.chunk = c;
    g.ctas = (int)((total + c - 1) / c);
    return g;
}

// Largest t < T with off[t] <= x (the tensor that contains flat index x; 0 when there is none).
// Called by all 32 lanes of a warp with the same arguments: every step probes 32 evenly spaced
// offsets at once, so a bucket of a few hundred tensors costs two dependent loads instead of eight.
__device__ __forceinline__ int find_tensor(const int64_t* __restrict__ off, int T, int64_t x)
{
    const int lane = threadIdx.x & 31;
    int lo = 0, hi = T;  // answer in [lo, hi)
    while (hi - lo > 1) {
        const int step = (hi - lo + 31) >> 5;
        const int idx = lo + lane * step;
        const bool le = idx < hi && __ldg(off + idx) <= x;
        const unsigned m = __ballot_sync(0xffffffffu, le);  // offsets ascend: a prefix of the lanes
        const int k = m ? 31 - __clz(m) : 0;
        lo += k * step;
        hi = (lo + step < hi) ? lo + step : hi;
    }
    return lo;
}

// Calls f(t, tensor_begin, tensor_end, piece_begin, piece_end) for every non-empty
// intersection of the flat range [lo, hi) with a tensor, in ascending order.
template <class F>
__device__ __forceinline__ void for_each_piece(const int64_t* __restrict__ off, int T, int64_t lo,
                                               int64_t hi, F f)
{
    if (lo >= hi || T <= 0) return;
    int t = find_tensor(off, T, lo);
    int64_t pos = lo;
    while (pos < hi && t < T) {
        int64_t tb = __ldg(off + t), te = __ldg(off + t + 1);
        int64_t pe = te < hi ? te : hi;
        if (pe > pos) {
            f(t, tb, te, pos, pe);
            pos = pe;
        }
        if (pe >= te) ++t;
    }
}

// Asks L2 to fetch `bytes` (a multiple of 16) from a 16-byte aligned global address.  One thread of
// a CTA issues it for the block the CTA will read a couple of loop trips later: the loads then find
// their lines in L2, which keeps far more DRAM requests in flight than the registers of the loop can.
// It pays in loops that compute for a while between loads (round 2 of the selection); loops that are
// already bound by DRAM (BinGrad-b passes, the threshold quantizer) ran slower with it.
__device__ __forceinline__ void prefetch_l2(const void* p, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" :: "l"(p), "r"(bytes) : "memory");
}

// Block-cooperative visit of grad[pb, pe): 128-bit loads on the aligned body,
// scalar loads on the ragged head and tail.  f(float) is called once per element.
template <class F>
__device__ __forceinline__ void visit_piece(const float* __restrict__ grad, int64_t pb, int64_t pe, F f)
{
    int64_t a = (pb + 3) & ~(int64_t)3;
    if (a > pe) a = pe;
    int64_t b = pe & ~(int64_t)3;
    if (b < a) b = a;
    const int tid = threadIdx.x;
    if (tid < (int)(a - pb)) f(__ldg(grad + pb + tid));
    if (tid < (int)(pe - b)) f(__ldg(grad + b + tid));
    const float4* g4 = reinterpret_cast<const float4*>(grad);
    int64_t i = (a >> 2) + tid, e = b >> 2;
    for (; i + 3 * kThreads < e; i += 4 * kThreads) {
        float4 x0 = __ldg(g4 + i);
        float4 x1 = __ldg(g4 + i + kThreads);
        float4 x2 = __ldg(g4 + i + 2 * kThreads);
        float4 x3 = __ldg(g4 + i + 3 * kThreads);
        f(x0.x); f(x0.y); f(x0.z); f(x0.w);
        f(x1.x); f(x1.y); f(x1.z); f(x1.w);
        f(x2.x); f(x2.y); f(x2.z); f(x2.w);
        f(x3.x); f(x3.y); f(x3.z); f(x3.w);
    }
    for (; i < e; i += kThreads) {
        float4 x = __ldg(g4 + i);
        f(x.x); f(x.y); f(x.z); f(x.w);
    }
}

// ---------------------------------------------------------------------------
// Order-preserving map between fp32 values and unsigned 32-bit keys.
// -0.0 is folded onto +0.0 first so that equal values have equal keys.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t float_to_key(float v)
{
    uint32_t b = __float_as_uint(v);
    if (b == 0x80000000u) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ float key_to_float(uint32_t k)
{
    uint32_t b = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    return __uint_as_float(b);
}

// ---------------------------------------------------------------------------
// Philox4x32 with 10 rounds (Salmon et al., SC'11).
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               uint32_t k0, uint32_t k1)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;  // one wide multiply gives both halves
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c0 = n0; c1 = (uint32_t)p1; c2 = n2; c3 = (uint32_t)p0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// The ten round keys of one Philox4x32-10 key (the Weyl sequence of the key schedule), computed on
// the host and handed to a kernel by value: a kernel parameter can be an ALU operand directly, so the
// schedule costs no instruction on the device.
struct PhiloxKeys {
    uint32_t k0[10], k1[10];
};

inline PhiloxKeys philox_round_keys(uint32_t k0, uint32_t k1)
{
    PhiloxKeys K;
    for (int r = 0; r < 10; ++r) {
        K.k0[r] = k0 + (uint32_t)r * 0x9E3779B9u;
        K.k1[r] = k1 + (uint32_t)r * 0xBB67AE85u;
    }
    return K;
}

__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const PhiloxKeys& K)
{
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ K.k0[r];
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ K.k1[r];
        c0 = n0; c1 = (uint32_t)p1; c2 = n2; c3 = (uint32_t)p0;
    }
    return make_uint4(c0, c1, c2, c3);
}

// Rounds 1 and 2 of Philox4x32-10 split into the part that depends only on (c1, c2, c3) and the key,
// computed once per tensor, and the part that depends on c0.  c1..c3 = (counter high word, tensor
// index, stream id) are the same for every element of a tensor whose counters fit 32 bits: the
// product of round 1's second multiplier, round 1's first output word and therefore round 2's first
// product are all uniform.
struct PhiloxHoist {
    uint32_t n0;          // first word after round 1
    uint32_t lo1;         // low half of round 1's second product (second word after round 1)
    uint32_t c3k1;        // c3 ^ k1[0]
    uint32_t hi0b, lo0b;  // round 2's first product (multiplier * n0)
};

__device__ __forceinline__ PhiloxHoist philox_hoist(uint32_t c1, uint32_t c2, uint32_t c3, const PhiloxKeys& K)
{
    PhiloxHoist h;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    h.n0 = (uint32_t)(p1 >> 32) ^ c1 ^ K.k0[0];
    h.lo1 = (uint32_t)p1;
    h.c3k1 = c3 ^ K.k1[0];
    const uint64_t p0b = (uint64_t)0xD2511F53u * h.n0;
    h.hi0b = (uint32_t)(p0b >> 32);
    h.lo0b = (uint32_t)p0b;
    return h;
}

__device__ __forceinline__ uint4 philox4x32_10_tail(uint32_t c0, const PhiloxHoist& h, const PhiloxKeys& K)
{
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;  // round 1: only this product depends on c0
    uint32_t a0, a1, a2 = (uint32_t)(p0 >> 32) ^ h.c3k1, a3 = (uint32_t)p0;
    {  // round 2: the first product is uniform
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * a2;
        a0 = (uint32_t)(p1 >> 32) ^ h.lo1 ^ K.k0[1];
        a1 = (uint32_t)p1;
        a2 = h.hi0b ^ a3 ^ K.k1[1];
        a3 = h.lo0b;
    }
#pragma unroll
    for (int r = 2; r < 10; ++r) {
        const uint64_t q0 = (uint64_t)0xD2511F53u * a0;
        const uint64_t q1 = (uint64_t)0xCD9E8D57u * a2;
        const uint32_t n0 = (uint32_t)(q1 >> 32) ^ a1 ^ K.k0[r];
        const uint32_t n2 = (uint32_t)(q0 >> 32) ^ a3 ^ K.k1[r];
        a0 = n0; a1 = (uint32_t)q1; a2 = n2; a3 = (uint32_t)q0;
    }
    return make_uint4(a0, a1, a2, a3);
}

// ---------------------------------------------------------------------------
// Warp / block reductions with a fixed combination order (reproducible).
// ---------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

__device__ __forceinline__ long long warp_sum(long long x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Sum over the CTA; the result is valid in thread 0.  `scratch` holds kWarps values.
template <class Tv>
__device__ __forceinline__ Tv block_sum(Tv x, Tv* scratch)
{
    x = warp_sum(x);
    const int w = threadIdx.x >> 5, l = threadIdx.x & 31;
    __syncthreads();
    if (l == 0) scratch[w] = x;
    __syncthreads();
    Tv r = 0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int i = 0; i < kWarps; ++i) r += scratch[i];
    }
    return r;
}

}  // namespace ogq
