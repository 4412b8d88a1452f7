// Per-element pieces of the quantizer shared by the bucket-wide kernel and the fixed-length-bucket
// kernel: segment search in a shared-memory level table, the rounding decision, word assembly.
#pragma once

#include "ogq_common.cuh"

namespace ogq {

constexpr int kMaxLevels = 32;
constexpr int kMaxWorkers = 64;

// OR-combine the 4*BITS-bit chunk of each lane into words, BITS = 1, 2 or 4: a word is made of
// 8, 4, 2 neighbouring lanes and the first lane of each such set returns it (word index lane / L).
template <int BITS>
__device__ __forceinline__ uint32_t assemble_words(uint32_t chunk, int lane)
{
    static_assert(BITS == 1 || BITS == 2 || BITS == 4, "other widths are combined in shared memory");
    constexpr int L = 8 / BITS;
    uint32_t x = chunk << (4 * BITS * (lane & (L - 1)));
#pragma unroll
    for (int o = 1; o < L; o <<= 1) x |= __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Segment search and rounding decision of one element on the fast path.  `tabaddr` is the shared
// address of the table {level k, width of the segment above it} (8 bytes per entry) and `mid` its
// middle level.  Returns the address of the entry whose index is the element's code: the entry of the
// segment's lower level, or the next one when the element rounds up.  The halving steps are written
// as "load, compare, predicated add" so that each costs three instructions.
template <int STEP>
__device__ __forceinline__ void search_step(uint32_t& a, float v)
{
    asm("{ .reg .pred p; .reg .f32 t; ld.shared.f32 t, [%0+%2]; setp.le.f32 p, t, %1; @p add.u32 %0, %0, %2; }"
        : "+r"(a) : "f"(v), "n"(STEP * 8));
}

template <int BITS>
__device__ __forceinline__ uint32_t entry_after_rounding(float v, uint32_t rnd, uint32_t tabaddr, float mid)
{
    uint32_t a = tabaddr;
    if constexpr (BITS >= 2) {
        if (mid <= v) a += 8u << (BITS - 2);
        if constexpr (BITS >= 5) search_step<4>(a, v);
        if constexpr (BITS >= 4) search_step<2>(a, v);
        if constexpr (BITS >= 3) search_step<1>(a, v);
    }
    float lo, w;
    asm("ld.shared.v2.f32 {%0, %1}, [%2];" : "=f"(lo), "=f"(w) : "r"(a));
    const float lhs = __fmul_rn((float)(rnd >> 8), w);
    const float rhs = __fmul_rn(__fsub_rn(v, lo), 16777216.0f);
    asm("{ .reg .pred p; setp.lt.f32 p, %1, %2; @p add.u32 %0, %0, 8; }" : "+r"(a) : "f"(lhs), "f"(rhs));
    return a;
}

}  // namespace ogq
