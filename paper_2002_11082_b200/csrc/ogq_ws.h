// Host-side layout of the caller-provided scratch buffer.
#pragma once

#include <stddef.h>
#include <stdint.h>

namespace ogq {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Partial sums of one split pass of the BinGrad-b solver.
struct BbPart {
    double s_lo, s_hi;     // sums of {v < b_0} and {v >= b_0}
    long long c_lo, c_hi;  // their counts
};

struct BbWs {
    BbPart* slot_a;      // [ctas]  piece of a tensor that began before the CTA's chunk
    BbPart* slot_b;      // [ctas]  piece of a tensor that begins in the chunk and runs past it
    BbPart* direct;      // [T]     tensors that lie inside one chunk
    unsigned* arrive;    // [T]     pieces finished in the current pass
    int* done;           // [T]     tensor needs no further pass
    long long* prev_lo;  // [T]     |{v < b_0}| of the previous pass
};

inline size_t bb_ws_bytes(int T, int ctas)
{
    size_t b = 0;
    b += align_up(sizeof(BbPart) * (size_t)ctas, 256) * 2;
    b += align_up(sizeof(BbPart) * (size_t)T, 256);
    b += align_up(sizeof(unsigned) * (size_t)T, 256);
    b += align_up(sizeof(int) * (size_t)T, 256);
    b += align_up(sizeof(long long) * (size_t)T, 256);
    return b;
}

inline BbWs bb_ws_carve(void* base, int T, int ctas)
{
    char* p = (char*)base;
    BbWs w;
    w.slot_a = (BbPart*)p; p += align_up(sizeof(BbPart) * (size_t)ctas, 256);
    w.slot_b = (BbPart*)p; p += align_up(sizeof(BbPart) * (size_t)ctas, 256);
    w.direct = (BbPart*)p; p += align_up(sizeof(BbPart) * (size_t)T, 256);
    w.arrive = (unsigned*)p; p += align_up(sizeof(unsigned) * (size_t)T, 256);
    w.done = (int*)p; p += align_up(sizeof(int) * (size_t)T, 256);
    w.prev_lo = (long long*)p;
    return w;
}

}  // namespace ogq
