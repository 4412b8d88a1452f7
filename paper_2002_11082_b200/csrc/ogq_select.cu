// ORQ and BinGrad-pb level solvers: exact selection by histogram refinement.
//
// Round 1 streams the bucket once: per tensor it finds min, max and a histogram
// over key cells (128 cells per binade inside a 16-binade window anchored at a
// sampled magnitude, one cell per binade outside), each cell with an exact
// count and an exact integer sum of the low key bits.  The last CTA to finish a
// tensor runs the scalar solver (ogq_select_solver.cuh), which turns the cell
// prefix sums into a few narrow candidate intervals.  Round 2 streams the bucket
// again, copies the few percent of elements inside the intervals to scratch and
// histograms them on a finer grid; round 3 and later work on the copied keys
// only, until every level's rank falls into a single-key cell.  As soon as the
// elements still in question fit one shared-memory sort, the next pass only
// copies them and the tensor is finished from the sorted keys.  Tensors of at
// most kSmallN elements are sorted in shared memory right away; mid-size ones
// run on a CTA of their own (round 1 in the first launch, the rest in the
// second).  The key buffers hold one eighth of the bucket: a pass whose copies
// do not fit is repeated on the gradient with the narrower intervals.
//
// All cross-CTA accumulation is integer (atomic adds, min, max), and the
// per-tensor prefix sums are built in a fixed order, so results are
// bit-reproducible.  No kernel waits on another CTA: the "last CTA to arrive"
// is found with one atomic counter per tensor.
#include <math.h>

#include <atomic>

#include "ogq_common.cuh"
#include "ogq_internal.h"
#include "ogq_select_solver.cuh"
#include "ogq_ws.h"

namespace ogq {

constexpr int kSelThreads = 512;    // two CTAs are resident per SM: a CTA in a solver pass, a sort or a
                                    // set-up phase leaves the other half of the SM streaming
constexpr int kSelResident = 2;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelW = 16;          // binades in the fine window of round 1
constexpr int kSelM = 7;           // log2(cells per binade) in the window
constexpr int kSmallN = 4096;      // tensors up to this size are sorted in shared memory
constexpr int kMidN = 131072;      // tensors up to this size are solved start to finish by one CTA of their own
constexpr int kStageCap = 320;     // per-warp staging entries for compaction
constexpr int kParkMax = 256;      // values one warp can park between two checks in the tail of round 2 (32 lanes x 8)
constexpr int kMaxSlices = 64;     // CTAs that share one tensor's copied keys in round 3
constexpr int kSliceElems = 16384;
constexpr int kMaxRounds = 32;
constexpr int kSortScanMax = 65536;  // longest copied-key list one CTA filters for the sorting finish

constexpr int kRound1Mag = 256 - kSelW + (kSelW << kSelM);  // round-1 cells per sign
constexpr int kRound1Cells = 2 * kRound1Mag;
static_assert(kRound1Cells <= kCells, "round-1 cells exceed the budget");

struct TState {
    int done, round, m, hi_e;
    unsigned kmin_inv, kmax, nonfinite, arrive;
    unsigned long long arrived;  // elements of the current pass whose counts have been flushed
    unsigned expected;
    int compact_only;  // the next pass only copies the keys inside the intervals: they fit one sort
    int overflow;      // the current pass dropped copies that did not fit the tensor's region
    int from_grad;     // the current pass (round >= 3) reads the gradient, not the previous pass's copies
    unsigned long long cursor[2];
    long long n;
    double stot;
    Interval iv[kMaxIv];
    ExactLv lv[kMaxLv];
};

struct SelWs {
    TState* st;                  // [T]
    uint32_t* gcnt;              // [T][kCells]
    unsigned long long* glsum;   // [T][kCells]
    unsigned* nitems;            // [1] work items of round 3
    int2* items;                 // [T * kMaxSlices]
    uint32_t* buf[2];            // [total / kBufDiv] copied keys: tensor t owns [sel_region(off[t]), sel_region(off[t+1]))
};

// The copied keys of a tensor are normally a few percent of it, so the two key buffers hold one eighth
// of the bucket: the tensor that starts at element x owns the words from sel_region(x) on, up to where
// the next tensor's region starts.  A pass whose copies do not fit drops the surplus and marks the
// tensor (TState::overflow); the next pass then reads the gradient again instead of the buffer, with
// narrower intervals, until the copies fit.
constexpr int kBufDiv = 8;
__host__ __device__ __forceinline__ int64_t sel_region(int64_t x) { return (x / kBufDiv) & ~(int64_t)3; }

static size_t sel_zero_bytes(int T)
{
    return align_up(sizeof(TState) * (size_t)T, 256) + align_up(sizeof(uint32_t) * (size_t)T * kCells, 256) +
           align_up(sizeof(unsigned long long) * (size_t)T * kCells, 256) + 256;
}

size_t ws_bytes_select(int T, int64_t total, int /*s*/)
{
    return sel_zero_bytes(T) + align_up(sizeof(int2) * (size_t)T * kMaxSlices, 256) +
           2 * align_up(sizeof(uint32_t) * (size_t)(total / kBufDiv + 8), 256);
}

static SelWs sel_carve(void* base, int T, int64_t total)
{
    char* p = (char*)base;
    SelWs w;
    w.st = (TState*)p; p += align_up(sizeof(TState) * (size_t)T, 256);
    w.gcnt = (uint32_t*)p; p += align_up(sizeof(uint32_t) * (size_t)T * kCells, 256);
    w.glsum = (unsigned long long*)p; p += align_up(sizeof(unsigned long long) * (size_t)T * kCells, 256);
    w.nitems = (unsigned*)p; p += 256;
    w.items = (int2*)p; p += align_up(sizeof(int2) * (size_t)T * kMaxSlices, 256);
    w.buf[0] = (uint32_t*)p; p += align_up(sizeof(uint32_t) * (size_t)(total / kBufDiv + 8), 256);
    w.buf[1] = (uint32_t*)p;
    return w;
}

// ---------------------------------------------------------------------------
// Shared-memory layout of a streaming CTA (dynamic): cell counters, low-bit sums
// (two 32-bit halves with carry), and the per-warp compaction stages.  The
// solver reuses the same bytes for its prefix arrays.
// ---------------------------------------------------------------------------
constexpr size_t kSmemHist = 3 * kCells * sizeof(uint32_t);
constexpr size_t kSmemStage = kSelWarps * kStageCap * sizeof(uint32_t);
constexpr size_t kSmemSolver = kSlots * (sizeof(uint32_t) + sizeof(double) + 1) + 32;
constexpr size_t kSmemBytes = (kSmemHist + kSmemStage > kSmemSolver) ? kSmemHist + kSmemStage : kSmemSolver;

struct Table {  // interval lookup table of the tensor being streamed
    uint32_t klo[kMaxIv];
    uint32_t khi[kMaxIv];
    int sh[kMaxIv];
    int cellbase[kMaxIv];
    int m, ncells;
    int lo_e;                                      // bottom binade of the round-1 fine window
    uint32_t coarse[1024];                         // one bit per block of 2^17 keys that touches an interval
};

__device__ __forceinline__ void table_from_intervals(Table& tb, const Interval* iv, int m)
{
    // called by one thread
    int nc = 0;
    for (int j = 0; j < kMaxIv; ++j) {
        if (j < m) {
            tb.klo[j] = iv[j].klo; tb.khi[j] = iv[j].khi; tb.sh[j] = iv[j].sh; tb.cellbase[j] = iv[j].cellbase;
            nc = iv[j].cellbase + iv[j].ncell;
        } else {
            tb.klo[j] = 0xffffffffu; tb.khi[j] = 0u; tb.sh[j] = 0; tb.cellbase[j] = 0;
        }
    }
    tb.m = m;
    tb.ncells = nc;
}

// The same, spread over the first kMaxIv threads of the CTA (called by all threads; the caller
// synchronises afterwards).
__device__ __forceinline__ void table_from_intervals_cta(Table& tb, const Interval* iv, int m)
{
    const int j = threadIdx.x;
    if (j < kMaxIv) {
        if (j < m) {
            tb.klo[j] = iv[j].klo; tb.khi[j] = iv[j].khi; tb.sh[j] = iv[j].sh; tb.cellbase[j] = iv[j].cellbase;
        } else {
            tb.klo[j] = 0xffffffffu; tb.khi[j] = 0u; tb.sh[j] = 0; tb.cellbase[j] = 0;
        }
    }
    if (j == 0) {
        tb.m = m;
        tb.ncells = (m > 0) ? iv[m - 1].cellbase + iv[m - 1].ncell : 0;
    }
}

// Round-1 intervals: coarse (one cell per binade) outside a window of kSelW binades that ends
// at binade hi_e, fine inside.  Negative values only for signed keys.
__device__ __forceinline__ int round1_intervals(int hi_e, bool magnitude_only, Interval* iv)
{
    const int lo_e = hi_e - kSelW;
    int m = 0, cb = 0;
    auto add = [&](uint32_t klo, int ncell, int sh) {
        if (ncell <= 0) return;
        Interval& x = iv[m++];
        x.klo = klo; x.sh = sh; x.ncell = ncell;
        x.khi = klo + (uint32_t)((((unsigned long long)ncell) << sh) - 1ull);
        x.cellbase = cb; x.pad = 0; x.cbefore = 0; x.sbefore = 0.0;
        cb += ncell;
    };
    if (!magnitude_only) {
        add(0u, 256 - hi_e, 23);
        add(0x80000000u - ((uint32_t)hi_e << 23), kSelW << kSelM, 23 - kSelM);
        add(0x80000000u - ((uint32_t)lo_e << 23), lo_e, 23);
    }
    add(0x80000000u, lo_e, 23);
    add(0x80000000u + ((uint32_t)lo_e << 23), kSelW << kSelM, 23 - kSelM);
    add(0x80000000u + ((uint32_t)hi_e << 23), 256 - hi_e, 23);
    return m;
}

// Round-1 cell of a value, computed directly (same layout as round1_intervals produces):
// magnitude cells ascend with |v|; negative values mirror them below, non-negative ones above.
__device__ __forceinline__ void round1_cell(uint32_t bits, int lo_e, bool magnitude_only, int& cell,
                                            uint32_t& lowkey)
{
    const uint32_t mag = bits & 0x7fffffffu;
    const uint32_t rel = mag - ((uint32_t)lo_e << 23);
    const int e = (int)(mag >> 23);
    const bool fine = rel < ((uint32_t)kSelW << 23);
    const int mi = fine ? lo_e + (int)(rel >> (23 - kSelM)) : ((e < lo_e) ? e : e - kSelW + (kSelW << kSelM));
    const uint32_t mask = fine ? ((1u << (23 - kSelM)) - 1u) : 0x7fffffu;
    const uint32_t low = mag & mask;
    if (magnitude_only) { cell = mi; lowkey = low; }
    else if (bits >> 31) { cell = kRound1Mag - 1 - mi; lowkey = mask - low; }
    else { cell = kRound1Mag + mi; lowkey = low; }
}

__device__ __forceinline__ uint32_t key_to_bits(uint32_t k) { return (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k; }

__device__ __forceinline__ bool classify(const Table& tb, uint32_t key, int& cell, uint32_t& low, int& sh)
{
    int idx = 0;
#pragma unroll
    for (int step = kMaxIv / 2; step >= 1; step >>= 1)
        if (tb.klo[idx + step] <= key) idx += step;
    sh = tb.sh[idx];
    const uint32_t rel = key - tb.klo[idx];
    cell = tb.cellbase[idx] + (int)(rel >> sh);
    low = rel & ((1u << sh) - 1u);
    return key >= tb.klo[idx] && key <= tb.khi[idx];
}

__device__ __forceinline__ void hist_add(uint32_t* cnt, uint32_t* lo, uint32_t* hi, int cell, uint32_t low)
{
    atomicAdd(cnt + cell, 1u);
    if (low) {
        const uint32_t old = atomicAdd(lo + cell, low);
        if (old + low < old) atomicAdd(hi + cell, 1u);
    }
}

// Warp-uniform visit of base[pb, pe): every lane of a warp calls f(x, nvalid) the same number of
// times (nvalid = 0, 1 or 4), so f may use warp collectives.  128-bit loads on the aligned body.
__device__ __forceinline__ float4 ld4(const float4* p) { return __ldg(p); }
__device__ __forceinline__ uint4 ld4(const uint4* p) { return __ldcg(p); }
__device__ __forceinline__ float ld1(const float* p) { return __ldg(p); }
__device__ __forceinline__ uint32_t ld1(const uint32_t* p) { return __ldcg(p); }

template <class E4, class E, class F>
__device__ __forceinline__ void warp_visit4(const E* __restrict__ base, int64_t pb, int64_t pe, F f)
{
    int64_t a = (pb + 3) & ~(int64_t)3;
    if (a > pe) a = pe;
    int64_t b = pe & ~(int64_t)3;
    if (b < a) b = a;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (warp == 0) {
        E x[4];
        int nv = 0;
        if (lane < (int)(a - pb)) { x[0] = ld1(base + pb + lane); nv = 1; }
        else if (lane >= 4 && lane - 4 < (int)(pe - b)) { x[0] = ld1(base + b + lane - 4); nv = 1; }
        f(x, nv);
    }
    const E4* b4 = reinterpret_cast<const E4*>(base);
    const int64_t e = b >> 2;
    for (int64_t i0 = (a >> 2) + warp * 32; i0 < e; i0 += 4 * kSelThreads) {
        E x[4][4];
        int nx[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t i = i0 + (int64_t)u * kSelThreads + lane;
            nx[u] = 0;
            if (i < e) {
                const E4 v = ld4(b4 + i);
                x[u][0] = v.x; x[u][1] = v.y; x[u][2] = v.z; x[u][3] = v.w;
                nx[u] = 4;
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (i0 + (int64_t)u * kSelThreads < e) f(x[u], nx[u]);
    }
}

struct Stager {  // per-warp compaction stage
    uint32_t* stage;            // this warp's kStageCap entries in shared memory
    uint32_t* dst;              // tensor's region in the destination buffer
    unsigned long long* cursor; // tensor's append cursor
    int fill;

    __device__ __forceinline__ void flush()
    {
        const int lane = threadIdx.x & 31;
        if (fill > 0) {
            unsigned long long pos = 0;
            if (lane == 0) pos = atomicAdd(cursor, (unsigned long long)fill);
            pos = __shfl_sync(0xffffffffu, pos, 0);
            for (int i = lane; i < fill; i += 32) dst[pos + i] = stage[i];
        }
        __syncwarp();
        fill = 0;
    }

    // every lane passes its own keys (c of them, c <= 4)
    __device__ __forceinline__ void append(const uint32_t* kk, int c)
    {
        const int lane = threadIdx.x & 31;
        int incl = c;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int nb = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += nb;
        }
        const int total = __shfl_sync(0xffffffffu, incl, 31);
        if (total == 0) return;
        const int at = fill + incl - c;
        for (int i = 0; i < c; ++i) stage[at + i] = kk[i];
        fill += total;
        __syncwarp();
        if (fill > kStageCap - 128) flush();
    }
};

// Block-cooperative visit of grad[pb, pe) without warp collectives: 128-bit loads on the aligned
// body (four in flight per thread), scalar loads on the ragged head and tail.
template <class F>
__device__ __forceinline__ void visit_plain(const float* __restrict__ grad, int64_t pb, int64_t pe, F f)
{
    int64_t a = (pb + 3) & ~(int64_t)3;
    if (a > pe) a = pe;
    int64_t b = pe & ~(int64_t)3;
    if (b < a) b = a;
    const int tid = threadIdx.x;
    if (tid < (int)(a - pb)) f(__ldg(grad + pb + tid));
    if (tid < (int)(pe - b)) f(__ldg(grad + b + tid));
    const float4* g4 = reinterpret_cast<const float4*>(grad);
    int64_t i = (a >> 2) + tid;
    const int64_t e = b >> 2;
    for (; i + 3 * kSelThreads < e; i += 4 * kSelThreads) {
        const float4 x0 = __ldg(g4 + i);
        const float4 x1 = __ldg(g4 + i + kSelThreads);
        const float4 x2 = __ldg(g4 + i + 2 * kSelThreads);
        const float4 x3 = __ldg(g4 + i + 3 * kSelThreads);
        f(x0.x); f(x0.y); f(x0.z); f(x0.w);
        f(x1.x); f(x1.y); f(x1.z); f(x1.w);
        f(x2.x); f(x2.y); f(x2.z); f(x2.w);
        f(x3.x); f(x3.y); f(x3.z); f(x3.w);
    }
    for (; i < e; i += kSelThreads) {
        const float4 x = __ldg(g4 + i);
        f(x.x); f(x.y); f(x.z); f(x.w);
    }
}


__device__ __forceinline__ float min3f(float a, float b, float c)
{
    float r;
    asm("min.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));  // a NaN operand is skipped
    return r;
}
__device__ __forceinline__ float max3f(float a, float b, float c)
{
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}
constexpr int kPrefetchTrips = 2;                         // how far ahead of the loads L2 is asked for a block
constexpr uint32_t kTripBytes = 4u * kSelThreads * 16u;  // one trip of a CTA's streaming loop
// shared-memory add without a return value, on a 32-bit shared address
__device__ __forceinline__ void red_shared_add(uint32_t addr, uint32_t v)
{
    asm volatile("red.shared.add.u32 [%0], %1;" :: "r"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ uint32_t atom_shared_add(uint32_t addr, uint32_t v)
{
    uint32_t old;
    asm volatile("atom.shared.add.u32 %0, [%1], %2;" : "=r"(old) : "r"(addr), "r"(v) : "memory");
    return old;
}

constexpr int kPackedPerSign = kSelW << kSelM;  // fine cells per sign (2048)
constexpr int kPackedCells = 2 * kPackedPerSign;
constexpr int kPackTrips = 8;                    // loop trips between two folds of the packed cells
static_assert(kPackedCells * sizeof(uint32_t) <= kSelWarps * kStageCap * sizeof(uint32_t),
              "the packed cells live in the (otherwise unused) compaction stages during round 1");

template <bool MAG, bool CLIP>
struct Round1Body {
    uint32_t lo23;
    uint32_t neg_lo23x2;  // -(lo23 << 1), the addend of the doubled window offset
    int lo_e;
    uint32_t cnt;  // shared address of the count of the first non-negative magnitude cell; the low
                   // sums lie kCells words above the counts, their carries 2 kCells words above
    uint32_t pk;   // shared address of the packed words: kPackedPerSign cells of the non-negative values,
                   // then (signed keys only) kPackedPerSign cells of the negative ones, both by magnitude
    uint32_t coarse;  // shared address of the counter of values that bypassed the packed cells
    uint32_t one24;   // 1 << 24 (the count field of a packed word), kept in a register
    float mn, mx;
    uint32_t nonfinite;
    float tau;  // clipping threshold (CLIP only)

    // clip to [-tau, tau] (CLIP), magnitude for BinGrad-pb, and fold -0 into +0
    __device__ __forceinline__ float canon(float v) const
    {
        if (CLIP) {
            const float m = fminf(fabsf(v), tau);
            return (MAG ? m : copysignf(m, v)) + 0.0f;
        }
        return (MAG ? fabsf(v) : v) + 0.0f;
    }

    // A value inside the fine window, the slow way: two adds into the wide counters (cells and low bits
    // mirrored for negative values, so that both ascend with the key).  rel = magnitude bits - lo23.
    __device__ __forceinline__ void fine_wide(uint32_t bits, uint32_t rel)
    {
        const int sgn = MAG ? 0 : ((int)bits >> 31);  // 0 or -1
        const uint32_t low = (bits ^ (uint32_t)sgn) & ((1u << (23 - kSelM)) - 1u);
        const uint32_t c = cnt + (uint32_t)(((lo_e + (int)(rel >> (23 - kSelM))) ^ sgn) << 2);
        red_shared_add(c, 1u);
        const uint32_t old = atom_shared_add(c + 4u * kCells, low);
        if (old + low < old) red_shared_add(c + 8u * kCells, 1u);
    }

    // The fast way: one shared-memory add of {count 1 in the top 8 bits, low magnitude bits in the other
    // 24} into the cell's packed word (r2 = rel << 1, below kSelW << 24).  The caller folds the packed
    // words into the wide counters every few trips, before a cell can have taken 256 values (and redoes
    // the trips the slow way if one did); the mirroring of the negative half happens there.  The
    // instruction mix matters here: the loop is bound by the integer/logic pipe, so the address is put
    // together with multiply-adds and the sign is not branched on.
    __device__ __forceinline__ void fine_packed(uint32_t bits, uint32_t r2)
    {
        // pk + 4 * cell, cell = r2 >> (24 - kSelM): the high half of a multiply-add by a power of two,
        // which the compiler turns into one shift-and-add
        static_assert(kSelM == 7, "the shift below is 32 - (24 - kSelM - 2)");
        uint32_t addr;
        asm("mad.hi.u32 %0, %1, 131072, %2;" : "=r"(addr) : "r"(r2 & ~((1u << (24 - kSelM)) - 1u)), "r"(pk));
        if (!MAG) asm("mad.lo.u32 %0, %1, %2, %0;" : "+r"(addr) : "r"(bits >> 31), "r"(4u * kPackedPerSign));
        red_shared_add(addr, (bits & ((1u << (23 - kSelM)) - 1u)) | one24);
    }

    // any value (already canonical)
    template <bool PACKED>
    __device__ __forceinline__ void any(uint32_t bits)
    {
        const int sgn = MAG ? 0 : ((int)bits >> 31);
        const uint32_t mag = bits & 0x7fffffffu;
        const uint32_t rel = mag - lo23;
        if (rel < ((uint32_t)kSelW << 23)) {
            if (PACKED) fine_packed(bits, rel << 1);
            else fine_wide(bits, rel);
        } else {  // outside the fine window: one cell per binade
            const int e = (int)(mag >> 23);
            const int mi = (e < lo_e) ? e : e - kSelW + (kSelW << kSelM);
            if (e == 255) nonfinite = 1u;  // the window never reaches binade 255
            const uint32_t c = cnt + (uint32_t)((mi ^ sgn) << 2);
            const uint32_t low = (mag ^ (uint32_t)sgn) & 0x7fffffu;
            red_shared_add(c, 1u);
            const uint32_t old = atom_shared_add(c + 4u * kCells, low);
            if (old + low < old) red_shared_add(c + 8u * kCells, 1u);
            if (PACKED) red_shared_add(coarse, 1u);
        }
    }

    __device__ __forceinline__ void one(float v)
    {
        v = canon(v);
        mn = fminf(mn, v);
        mx = fmaxf(mx, v);
        any<false>(__float_as_uint(v));
    }

    template <bool PACKED>
    __device__ __forceinline__ void four(float4 x)
    {
        const float v0 = canon(x.x), v1 = canon(x.y), v2 = canon(x.z), v3 = canon(x.w);
        mn = min3f(min3f(mn, v0, v1), v2, v3);
        mx = max3f(max3f(mx, v0, v1), v2, v3);
        const uint32_t b0 = __float_as_uint(v0), b1 = __float_as_uint(v1), b2 = __float_as_uint(v2),
                       b3 = __float_as_uint(v3);
        // doubled offset into the window, (magnitude bits - lo23) << 1: the doubling drops the sign bit,
        // and a multiply-add does both steps outside the integer/logic pipe
        uint32_t r0, r1, r2, r3;
        asm("mad.lo.u32 %0, %1, 2, %2;" : "=r"(r0) : "r"(b0), "r"(neg_lo23x2));
        asm("mad.lo.u32 %0, %1, 2, %2;" : "=r"(r1) : "r"(b1), "r"(neg_lo23x2));
        asm("mad.lo.u32 %0, %1, 2, %2;" : "=r"(r2) : "r"(b2), "r"(neg_lo23x2));
        asm("mad.lo.u32 %0, %1, 2, %2;" : "=r"(r3) : "r"(b3), "r"(neg_lo23x2));
        // the window spans kSelW = 2^4 binades, so "all four inside" is one test on the OR (a value
        // below the window wraps to at least kSelW << 24 as well, because lo23 < 2^31 - 2^27)
        static_assert((kSelW & (kSelW - 1)) == 0, "window size must be a power of two");
        if ((r0 | r1 | r2 | r3) < ((uint32_t)kSelW << 24)) {
            if (PACKED) {
                fine_packed(b0, r0); fine_packed(b1, r1); fine_packed(b2, r2); fine_packed(b3, r3);
            } else {
                fine_wide(b0, r0 >> 1); fine_wide(b1, r1 >> 1); fine_wide(b2, r2 >> 1); fine_wide(b3, r3 >> 1);
            }
        } else {
            any<PACKED>(b0); any<PACKED>(b1); any<PACKED>(b2); any<PACKED>(b3);
        }
    }
};

// Round 1 over grad[pb, pe): per element min / max and the cell histogram (count, sum of the low key
// bits).  The bulk goes through packed cells (one shared-memory add per element instead of two, see
// Round1Body::fine), folded into the wide counters every kPackTrips loop trips; the sum of the folded
// counts is checked against the number of values that went in, and a mismatch (a cell took 256 values
// or more within the trips: heavily repeated values) redoes those trips with the two-add path.
// packed: kPackedCells zeroed words of shared memory, zero again on return.
template <bool MAG, bool CLIP>
__device__ __noinline__ void stream_round1(const float* __restrict__ grad, int64_t pb, int64_t pe, int lo_e,
                                              uint32_t* hist, uint32_t* packed, float& vmin, float& vmax,
                                              uint32_t& nonfinite, float tau)
{
    __shared__ uint32_t sh_coarse, sh_total;
    Round1Body<MAG, CLIP> f;
    f.tau = tau;
    f.lo23 = (uint32_t)lo_e << 23;
    f.neg_lo23x2 = 0u - (f.lo23 << 1);
    f.one24 = 0x01000000u;
    f.lo_e = lo_e;
    f.cnt = (uint32_t)__cvta_generic_to_shared(hist + (MAG ? 0 : kRound1Mag));
    f.pk = (uint32_t)__cvta_generic_to_shared(packed);
    f.coarse = (uint32_t)__cvta_generic_to_shared(&sh_coarse);
    f.mn = vmin; f.mx = vmax; f.nonfinite = nonfinite;
    int64_t a = (pb + 3) & ~(int64_t)3;
    if (a > pe) a = pe;
    int64_t b = pe & ~(int64_t)3;
    if (b < a) b = a;
    const int tid = threadIdx.x;
    if (tid < (int)(a - pb)) f.one(__ldg(grad + pb + tid));
    if (tid < (int)(pe - b)) f.one(__ldg(grad + b + tid));
    const float4* g4 = reinterpret_cast<const float4*>(grad);
    const int64_t first = a >> 2, e = b >> 2;
    const int64_t ntrips = (e - first) / (4 * kSelThreads);  // full trips: the same for every thread
    constexpr int kNp = MAG ? kPackedPerSign : kPackedCells;
    const float4* src = g4 + first + tid;                                              // this thread's next load
    const float4* pfp = g4 + first + (int64_t)kPrefetchTrips * 4 * kSelThreads;       // next block to ask L2 for
    const float4* const pf_end = g4 + e - 4 * kSelThreads;
    for (int64_t t0 = 0; t0 < ntrips; t0 += kPackTrips) {
        const int nt = (int)((ntrips - t0 < kPackTrips) ? ntrips - t0 : kPackTrips);
        if (tid == 0) { sh_coarse = 0u; sh_total = 0u; }
        __syncthreads();
        const float4* const period = src;
        for (int tt = 0; tt < nt; ++tt) {
            if (tid == 0 && pfp <= pf_end) prefetch_l2(pfp, kTripBytes);
            pfp += 4 * kSelThreads;
            float4 x[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) x[u] = __ldg(src + u * kSelThreads);
            src += 4 * kSelThreads;
#pragma unroll
            for (int u = 0; u < 4; ++u) f.template four<true>(x[u]);
        }
        __syncthreads();
        // fold, phase 1: do the packed counts add up to the values that went in?
        uint32_t mine = 0u;
        uint32_t wv[kNp / kSelThreads];  // this thread's packed words, read once
#pragma unroll
        for (int k = 0; k < kNp / kSelThreads; ++k) {
            wv[k] = packed[tid + k * kSelThreads];
            mine += wv[k] >> 24;
        }
        mine = __reduce_add_sync(0xffffffffu, mine);
        if ((tid & 31) == 0 && mine) atomicAdd(&sh_total, mine);
        __syncthreads();
        const bool ok = sh_total + sh_coarse == (uint32_t)nt * 16u * kSelThreads;
        // phase 2: into the wide counters (packed index p: negative values mirror below the middle)
#pragma unroll
        for (int k = 0; k < kNp / kSelThreads; ++k) {
            const int p = tid + k * kSelThreads;
            const uint32_t w = wv[k];
            if (w) {
                packed[p] = 0u;
                if (ok) {
                    // non-negative half: cell and low bits ascend with the magnitude; negative half: mirrored
                    const uint32_t c = w >> 24, sum = w & 0xffffffu;
                    const bool neg = !MAG && p >= kPackedPerSign;
                    const int cell = MAG ? lo_e + p
                                         : (neg ? kRound1Mag - 1 - lo_e - (p - kPackedPerSign) : kRound1Mag + lo_e + p);
                    hist[cell] += c;
                    const uint32_t add = neg ? c * ((1u << (23 - kSelM)) - 1u) - sum : sum;
                    const uint32_t old = hist[kCells + cell];
                    hist[kCells + cell] = old + add;
                    if (old + add < old) hist[2 * kCells + cell] += 1u;  // carry into the high word
                }
            }
        }
        if (!ok) {
            // a packed count wrapped: the fine values of these trips again, two adds each (the values outside
            // the window were counted directly the first time and are skipped now)
            __syncthreads();
            for (int tt = 0; tt < nt; ++tt) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float4 x = __ldg(period + (tt * 4 + u) * kSelThreads);
                    const float vv[4] = {f.canon(x.x), f.canon(x.y), f.canon(x.z), f.canon(x.w)};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t bits = __float_as_uint(vv[j]);
                        const uint32_t rel = (bits & 0x7fffffffu) - f.lo23;
                        if (rel < ((uint32_t)kSelW << 23)) f.fine_wide(bits, rel);
                    }
                }
            }
        }
        __syncthreads();  // everyone has read the totals before they are reset
    }
    __syncthreads();
    for (int64_t i = first + ntrips * 4 * kSelThreads + tid; i < e; i += kSelThreads) f.template four<false>(__ldg(g4 + i));
    vmin = f.mn; vmax = f.mx; nonfinite = f.nonfinite;
}

// Round 2 over grad[pb, pe).  Phase A: a one-bit-per-2^17-bit-patterns test on the raw fp32 bits
// rejects almost every element; values that pass are parked in the warp's stage (no classification
// yet).  Phase B, whenever the stage fills up: the parked values are turned into keys and classified
// exactly 32 at a time, so that the expensive part runs with all lanes busy; keys inside an interval
// are histogrammed and copied out.
struct Round2Ctx {  // per-CTA constants of round 2, kept in shared memory to spare registers
    uint32_t *cnt, *lo, *hi;
    uint32_t* dst;
    unsigned long long* cursor;
    uint32_t clear;  // 0x7fffffff when only magnitudes count
    int nohist;      // copy the keys inside the intervals without counting them
    unsigned long long cap;  // words of the tensor's region in the destination buffer
    int* overflow;           // set when a copy did not fit
};

// Phase B of round 2 for one warp: classifies `fill` parked values 32 at a time.  A free function
// taking values, so that the caller's per-warp state can stay in registers.
__device__ __noinline__ void round2_drain(const Table* tb, const Round2Ctx* ctx, const uint32_t* stage, int fill)
{
    const int lane = threadIdx.x & 31;
    const uint32_t lt = (1u << lane) - 1u;
    const uint32_t clear = ctx->clear;
    __syncwarp();
    for (int base = 0; base < fill; base += 32) {
        const int i = base + lane;
        uint32_t key = 0;
        bool in = false;
        if (i < fill) {
            uint32_t bits = stage[i] & clear;
            if (bits == 0x80000000u) bits = 0u;
            key = bits ^ ((uint32_t)((int)bits >> 31) | 0x80000000u);
            int cell, sh;
            uint32_t low;
            in = classify(*tb, key, cell, low, sh);
            if (in && !ctx->nohist) hist_add(ctx->cnt, ctx->lo, ctx->hi, cell, low);
        }
        const uint32_t m2 = __ballot_sync(0xffffffffu, in);
        if (m2) {
            unsigned long long pos = 0;
            if (lane == 0) pos = atomicAdd(ctx->cursor, (unsigned long long)__popc(m2));
            pos = __shfl_sync(0xffffffffu, pos, 0);
            if (in) {
                const unsigned long long at = pos + __popc(m2 & lt);
                if (at < ctx->cap) ctx->dst[at] = key;
                else *(volatile int*)ctx->overflow = 1;
            }
        }
    }
    __syncwarp();
}

// Marks, in the space of raw fp32 bit patterns, every block of 2^17 patterns that can hold a value
// whose key lies in one of the table's intervals (called by all threads).  A block of 2^17 aligned
// keys is a block of 2^17 aligned patterns; -0 shares the block of the smallest negative values, and
// with magnitude_only both signs of a pattern are marked.  Block b of a word sits at bit 31 - (b & 31):
// a left shift by the block index brings its bit to the top of the word.
__device__ __forceinline__ void build_prefilter(Table& tb, bool magnitude_only)
{
    for (int i = threadIdx.x; i < 1024; i += kSelThreads) tb.coarse[i] = 0u;
    __syncthreads();
    if ((int)threadIdx.x < tb.m) {
        const uint32_t ba = tb.klo[threadIdx.x] >> 17, bb = tb.khi[threadIdx.x] >> 17;
        for (uint32_t b = ba; b <= bb; ++b) {
            const uint32_t pblk = (b & 0x4000u) ? (b ^ 0x4000u) : (~b & 0x7fffu);
            atomicOr(&tb.coarse[pblk >> 5], 0x80000000u >> (pblk & 31));
            if (magnitude_only || pblk == 0u) {
                const uint32_t twin = pblk ^ 0x4000u;
                atomicOr(&tb.coarse[twin >> 5], 0x80000000u >> (twin & 31));
            }
        }
    }
    __syncthreads();
}

template <bool CLIP>
struct Round2Warp {
    uint32_t coarse;  // shared addresses: the table's prefilter bitmap,
    uint32_t stage;   // this warp's kStageCap parking slots,
    uint32_t fillp;   // and their fill counter (bumped by the lanes that hit)
    float tau;        // clipping threshold (CLIP only)

    __device__ __forceinline__ float clip(float v) const { return CLIP ? copysignf(fminf(fabsf(v), tau), v) : v; }

    // Phase A for one element: no warp collective, only the lanes that pass the bitmap test do work.
    __device__ __forceinline__ void park(uint32_t bits)
    {
        const uint32_t pos = atom_shared_add(fillp, 1u);
        asm volatile("st.shared.u32 [%0], %1;" :: "r"(stage + (pos << 2)), "r"(bits) : "memory");
    }
    // Word address = coarse + ((bits & ~(2^22 - 1)) >> 20), written as the high half of a multiply-add
    // by 2^12: the compiler makes one shift-and-add of it (a real multiplication, with the factor
    // hidden in a kernel argument, was measured slower).  The funnel shift takes its count modulo 32.
    __device__ __forceinline__ uint32_t top_is_hit(uint32_t bits) const
    {
        uint32_t addr, word;
        asm("mad.hi.u32 %0, %1, 4096, %2;" : "=r"(addr) : "r"(bits & 0xffc00000u), "r"(coarse));
        asm("ld.shared.u32 %0, [%1];" : "=r"(word) : "r"(addr));
        return __funnelshift_l(0u, word, bits >> 17);  // the block's bit is now bit 31
    }
    __device__ __forceinline__ void one(float v)
    {
        const uint32_t bits = __float_as_uint(clip(v));
        if (top_is_hit(bits) >> 31) park(bits);
    }
    // Branch-free form for the main loop: shifts `hits` left and appends this element's bit.
    __device__ __forceinline__ void test(float v, uint32_t& hits) const
    {
        hits = __funnelshift_l(top_is_hit(__float_as_uint(clip(v))), hits, 1);
    }
    // Parks the elements marked in `hits` (bit 15 = the first of the sixteen elements tested: p[0].x,
    // ..., p[0].w, p[stride].x, ..., p[3 * stride].w).  The values are read again, from L1: a hit is
    // rare, and a register cannot be picked by a run-time index.
    __device__ __forceinline__ void park_hits(uint32_t hits, const float4* p, int stride)
    {
        while (hits) {
            const int b = 31 - __clz(hits);
            hits &= ~(1u << b);
            const int j = 15 - b;
            const float* src = reinterpret_cast<const float*>(p + (j >> 2) * stride) + (j & 3);
            park(__float_as_uint(clip(__ldg(src))));
        }
    }
};

template <bool CLIP>
__device__ __noinline__ void stream_round2(const float* __restrict__ grad, int64_t pb, int64_t pe,
                                              bool magnitude_only, const Table& tb, uint32_t* cnt, uint32_t* lo,
                                              uint32_t* hi, uint32_t* stage, uint32_t* dst, int64_t cap,
                                              unsigned long long* cursor, int* overflow, bool nohist, float tau)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __shared__ Round2Ctx ctx;
    __shared__ int fills[kSelWarps];
    __syncthreads();
    if (threadIdx.x == 0) {
        ctx.cnt = cnt; ctx.lo = lo; ctx.hi = hi; ctx.dst = dst; ctx.cursor = cursor;
        ctx.clear = magnitude_only ? 0x7fffffffu : 0xffffffffu;
        ctx.nohist = nohist ? 1 : 0;
        ctx.cap = (unsigned long long)cap;
        ctx.overflow = overflow;
    }
    if (lane == 0) fills[warp] = 0;
    __syncthreads();
    Round2Warp<CLIP> w;
    w.tau = tau;
    w.coarse = (uint32_t)__cvta_generic_to_shared(tb.coarse);
    w.stage = (uint32_t)__cvta_generic_to_shared(stage);
    w.fillp = (uint32_t)__cvta_generic_to_shared(&fills[warp]);
    int64_t a = (pb + 3) & ~(int64_t)3;
    if (a > pe) a = pe;
    int64_t b = pe & ~(int64_t)3;
    if (b < a) b = a;
    if (warp == 0) {  // ragged head and tail, one element per lane
        if (lane < (int)(a - pb)) w.one(__ldg(grad + pb + lane));
        else if (lane >= 4 && lane - 4 < (int)(pe - b)) w.one(__ldg(grad + b + lane - 4));
        __syncwarp();
    }
    // The tail below parks at most kParkMax values between two checks of the stage's fill.
    auto check = [&]() {
        __syncwarp();
        const int f = *(volatile int*)&fills[warp];
        if (f > kStageCap - kParkMax) {
            round2_drain(&tb, &ctx, stage, f);
            if (lane == 0) fills[warp] = 0;
            __syncwarp();
        }
    };
    const float4* g4 = reinterpret_cast<const float4*>(grad);
    const int64_t e = b >> 2;
    int64_t i0 = (a >> 2) + warp * 32;  // the trip counts below are warp-uniform
    // Trips of 4 x kSelThreads float4 (one contiguous block of kTripBytes per CTA).  One thread asks
    // L2 for the block kPrefetchTrips ahead, so that the loads below find their lines there.
    // A lane tests its sixteen values of a trip without branching; the warp then parks the trip's
    // hits in one go (nearly every trip has a hit in some lane, so the divergent parking code is
    // paid once per trip, not once per few values).  `fill` mirrors the stage's fill counter in a
    // register: it is the same in all lanes, so whether to drain first is a uniform decision.
    int64_t pf = (a >> 2) + (int64_t)kPrefetchTrips * 4 * kSelThreads;
    __syncwarp();
    int fill = *(volatile int*)&fills[warp];
    for (; i0 + 3 * kSelThreads + 32 <= e; i0 += 4 * kSelThreads) {
        if (threadIdx.x == 0 && pf + 4 * kSelThreads <= e) prefetch_l2(g4 + pf, kTripBytes);
        pf += 4 * kSelThreads;
        float4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) x[u] = __ldg(g4 + i0 + lane + u * kSelThreads);
        uint32_t hits = 0u;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            w.test(x[u].x, hits); w.test(x[u].y, hits); w.test(x[u].z, hits); w.test(x[u].w, hits);
        }
        for (;;) {  // one turn, unless the stage has to be drained to make room
            const int tot = (int)__reduce_add_sync(0xffffffffu, (uint32_t)__popc(hits));
            if (tot == 0) break;
            if (fill + tot <= kStageCap) {
                if (hits) w.park_hits(hits, g4 + i0 + lane, kSelThreads);
                fill += tot;
                break;
            }
            if (fill) {
                round2_drain(&tb, &ctx, stage, fill);
                if (lane == 0) fills[warp] = 0;
                __syncwarp();
                fill = 0;
                continue;
            }
            // more hits in one trip than the empty stage holds: the first eight values of every lane now
            const uint32_t first = hits & 0xff00u;
            if (first) w.park_hits(first, g4 + i0 + lane, kSelThreads);
            fill = (int)__reduce_add_sync(0xffffffffu, (uint32_t)__popc(first));
            hits &= 0xffu;
        }
    }
    if (i0 < e) {
        check();  // the trips above may have left the stage nearly full
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int64_t i = i0 + lane + (int64_t)u * kSelThreads;
            if (i < e) {
                const float4 x = __ldg(g4 + i);
                w.one(x.x); w.one(x.y); w.one(x.z); w.one(x.w);
            }
            if (u & 1) check();
        }
    }
    __syncwarp();
    round2_drain(&tb, &ctx, stage, *(volatile int*)&fills[warp]);
}

// Streams one piece of a tensor's working set: histogram of the keys inside the intervals,
// optional copy of those keys, and (round 1) min / max / non-finite tracking.
template <bool FIRST, bool FROM_GRAD, bool COMPACT>
__device__ __forceinline__ void stream_piece(const void* __restrict__ src, int64_t pb, int64_t pe,
                                             bool magnitude_only, const Table& tb, uint32_t* cnt,
                                             uint32_t* lo, uint32_t* hi, Stager& stg, uint32_t& kmin,
                                             uint32_t& kmax, uint32_t& nonfinite, bool nohist = false)
{
    auto handle = [&](uint32_t key, uint32_t* kk, int& c) {
        int cell, sh;
        uint32_t low;
        if (classify(tb, key, cell, low, sh)) {
            if (!nohist) hist_add(cnt, lo, hi, cell, low);
            if (COMPACT) kk[c++] = key;
        }
    };
    static_assert(!FROM_GRAD && !FIRST, "fp32 input goes through stream_round1 / stream_round2");
    {
        warp_visit4<uint4, uint32_t>((const uint32_t*)src, pb, pe, [&](const uint32_t* x, int nv) {
            uint32_t kk[4];
            int c = 0;
#pragma unroll
            for (int j = 0; j < 4; ++j)
                if (j < nv) handle(x[j], kk, c);
            if (COMPACT) stg.append(kk, c);
        });
    }
}

__device__ __forceinline__ void zero_hist(uint32_t* smem_hist, int ncells)
{
    for (int i = threadIdx.x; i < ncells; i += kSelThreads) {
        smem_hist[i] = 0u;
        smem_hist[kCells + i] = 0u;
        smem_hist[2 * kCells + i] = 0u;
    }
}

__device__ __forceinline__ void flush_hist(const uint32_t* smem_hist, int ncells, uint32_t* gcnt,
                                           unsigned long long* glsum)
{
    for (int i = threadIdx.x; i < ncells; i += kSelThreads) {
        const uint32_t c = smem_hist[i];
        if (c) {
            atomicAdd(gcnt + i, c);
            const unsigned long long l =
                ((unsigned long long)smem_hist[2 * kCells + i] << 32) | smem_hist[kCells + i];
            if (l) atomicAdd(glsum + i, l);
        }
    }
}

// Sum of a double over the CTA in a fixed order; valid in thread 0.  scratch: kSelWarps doubles.
__device__ __forceinline__ double sel_block_sum(double x, double* scratch)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = x;
    __syncthreads();
    double r = 0.0;
    if (threadIdx.x == 0)
        for (int i = 0; i < kSelWarps; ++i) r += scratch[i];
    return r;
}

// ---------------------------------------------------------------------------
// Block-wide exclusive scan of (count, sum) pairs in thread order (fixed order).
// ---------------------------------------------------------------------------
__device__ __forceinline__ void block_excl_scan(unsigned long long& c, double& s, unsigned long long* sc,
                                                double* ss, unsigned long long& tot_c, double& tot_s)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long ic = c;
    double is = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long nc = __shfl_up_sync(0xffffffffu, ic, o);
        const double ns = __shfl_up_sync(0xffffffffu, is, o);
        if (lane >= o) { ic += nc; is = ns + is; }
    }
    const unsigned long long pc = __shfl_up_sync(0xffffffffu, ic, 1);
    const double ps = __shfl_up_sync(0xffffffffu, is, 1);
    __syncthreads();
    if (lane == 31) { sc[warp] = ic; ss[warp] = is; }
    __syncthreads();
    unsigned long long bc = 0;
    double bs = 0.0;
    tot_c = 0;
    tot_s = 0.0;
#pragma unroll
    for (int w = 0; w < kSelWarps; ++w) {
        if (w < warp) { bc += sc[w]; bs += ss[w]; }
        tot_c += sc[w];
        tot_s += ss[w];
    }
    c = (lane == 0) ? bc : bc + pc;
    s = (lane == 0) ? bs : bs + ps;
}

struct SolverShared {
    Interval iv[kMaxIv];
    Interval niv[kMaxIv];
    LvInfo lv[kMaxLv];
    SolverView view;
    unsigned long long sc[kSelWarps];
    double ss[kSelWarps];
    int pb_a, pb_b, pb_c;
    int done, nm, internal;
    uint32_t offc[kMaxIv];    // per-interval shifts of the scanned prefix arrays
    double offs[kMaxIv];
    int nr, ra[kMaxLv], rb[kMaxLv];  // open slot ranges of this pass
    int pa[kMaxIv], pb[kMaxIv];      // pieces cut out of them
    long long cand;           // elements inside the new intervals
    int n_keys, n_unique;     // sorting finish
    int ivstart[kMaxIv], ivufirst[kMaxIv];
    double ivpre[kMaxIv];
};

__device__ __forceinline__ int find_new_interval(const SolverShared& S, uint32_t key)
{
    int lo = 0, hi = S.nm;  // last interval with klo <= key
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (S.niv[mid].klo <= key) lo = mid; else hi = mid;
    }
    return (key >= S.niv[lo].klo && key <= S.niv[lo].khi) ? lo : -1;
}

// ---------------------------------------------------------------------------
// Ascending bitonic sort of P keys in shared memory (P a power of two, at most 8 * kSelThreads),
// called by all threads of the CTA; the keys are ordered on return (a barrier has been passed).
// Compare-exchange distances of 256 and more are done by the whole CTA with a barrier per stage;
// distances 8..128 stay inside an aligned block of 256 keys, which one warp owns and orders with
// warp barriers only; distances 4, 2, 1 stay inside 8 consecutive keys, which one lane holds in
// registers.  For 4096 keys that is 10 CTA barriers instead of 78.
// ---------------------------------------------------------------------------
__device__ __forceinline__ void cmpx(uint32_t& a, uint32_t& b, bool up)
{
    const uint32_t lo = a < b ? a : b, hi = a < b ? b : a;
    a = up ? lo : hi;
    b = up ? hi : lo;
}

__device__ void block_bitonic_sort(uint32_t* keys, int P)
{
    if (P < 256) {  // few stages: the plain network
        for (int k = 2; k <= P; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                for (int i = threadIdx.x; i < P; i += kSelThreads) {
                    const int ixj = i ^ j;
                    if (ixj > i) {
                        const uint32_t a = keys[i], b = keys[ixj];
                        const bool up = (i & k) == 0;
                        if ((a > b) == up) { keys[i] = b; keys[ixj] = a; }
                    }
                }
                __syncthreads();
            }
        }
        return;
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int k = 2; k <= P; k <<= 1) {
        int j = k >> 1;
        for (; j >= 256; j >>= 1) {  // CTA-wide stages
            for (int q = threadIdx.x; q < (P >> 1); q += kSelThreads) {
                const int i = ((q & ~(j - 1)) << 1) | (q & (j - 1));
                uint32_t a = keys[i], b = keys[i | j];
                cmpx(a, b, (i & k) == 0);
                keys[i] = a; keys[i | j] = b;
            }
            __syncthreads();
        }
        for (int wb = warp * 256; wb < P; wb += kSelWarps * 256) {  // the 256-key blocks of this warp
            uint32_t* blk = keys + wb;
            int jj = j;
            for (; jj >= 8; jj >>= 1) {
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int q = lane + 32 * u;
                    const int i = ((q & ~(jj - 1)) << 1) | (q & (jj - 1));
                    uint32_t a = blk[i], b = blk[i | jj];
                    cmpx(a, b, ((wb + i) & k) == 0);
                    blk[i] = a; blk[i | jj] = b;
                }
                __syncwarp();
            }
            // distances 4, 2, 1 (those not above k / 2) on this lane's 8 consecutive keys
            uint4* v4 = reinterpret_cast<uint4*>(blk + 8 * lane);
            uint4 lo4 = v4[0], hi4 = v4[1];
            uint32_t r[8] = {lo4.x, lo4.y, lo4.z, lo4.w, hi4.x, hi4.y, hi4.z, hi4.w};
            const int i0 = wb + 8 * lane;
#pragma unroll
            for (int d = 4; d >= 1; d >>= 1) {
                if (d <= jj) {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if ((e & d) == 0) cmpx(r[e], r[e | d], ((i0 + e) & k) == 0);
                }
            }
            v4[0] = make_uint4(r[0], r[1], r[2], r[3]);
            v4[1] = make_uint4(r[4], r[5], r[6], r[7]);
            __syncwarp();
        }
        // the next k starts with a CTA-wide stage only when k >= 256
        if ((k << 1) >= 512 || k == P) __syncthreads();
    }
}

// Sorting finish (ORQ): when the elements left inside the candidate intervals fit in shared
// memory, they are sorted, run-length encoded into single-key cells with exact prefix counts
// and sums, and one more solver pass resolves every open level at once.
__device__ void sort_finish(TState* st, int t, int s, const uint32_t* buf, long long src_cnt,
                            float* __restrict__ levels, int32_t* __restrict__ status, unsigned char* smem,
                            SolverShared& S)
{
    constexpr int kPer = kSmallN / kSelThreads;
    uint32_t* skeys = reinterpret_cast<uint32_t*>(smem);
    uint32_t* xkeys = skeys + kSmallN;
    uint32_t* xcpre = xkeys + kSmallN;
    double* xspre = reinterpret_cast<double*>(smem + ((3 * kSmallN + kMaxIv + 2) * sizeof(uint32_t) + 15) / 16 * 16);
    __syncthreads();
    if (threadIdx.x == 0) S.n_keys = 0;
    if (threadIdx.x < kMaxIv) { S.ivstart[threadIdx.x] = 0; S.ivufirst[threadIdx.x] = -1; S.ivpre[threadIdx.x] = 0.0; }
    __syncthreads();
    // Filter of the copied keys: the lower and upper keys of the new intervals in two compact arrays
    // (padded to 64 entries), a six-step search without branches, eight keys per thread in flight, and
    // one shared counter update per warp and key column instead of one per accepted key.
    __shared__ uint32_t f_lo[kMaxIv], f_hi[kMaxIv];
    static_assert(kMaxIv == 64, "the search below takes six halving steps");
    if (threadIdx.x < kMaxIv) {
        const bool real = (int)threadIdx.x < S.nm;
        f_lo[threadIdx.x] = real ? S.niv[threadIdx.x].klo : 0xffffffffu;  // no key has this value (NaN pattern)
        f_hi[threadIdx.x] = real ? S.niv[threadIdx.x].khi : 0u;
    }
    __syncthreads();
    {
        const int lane = threadIdx.x & 31;
        constexpr int kCols = 8;
        // the keys come from L2 (another SM wrote them): the loads of the next trip are issued before
        // this trip's keys are searched, so that one round trip is hidden behind the other's work
        auto fetch = [&](uint32_t* k, long long at) {
#pragma unroll
            for (int u = 0; u < kCols; ++u) {
                const long long i = at + u * 32 + lane;
                k[u] = (i < src_cnt) ? __ldcg(buf + i) : 0u;
            }
        };
        int top = 2;
        while (top < S.nm) top <<= 1;
        uint32_t nxt[kCols];
        long long i0 = (long long)(threadIdx.x & ~31) * kCols;
        if (i0 < src_cnt) fetch(nxt, i0);
        for (; i0 < src_cnt; i0 += (long long)kCols * kSelThreads) {
            uint32_t key[kCols];
            bool in[kCols];
#pragma unroll
            for (int u = 0; u < kCols; ++u) key[u] = nxt[u];
            if (i0 + (long long)kCols * kSelThreads < src_cnt) fetch(nxt, i0 + (long long)kCols * kSelThreads);
            int idx[kCols];
#pragma unroll
            for (int u = 0; u < kCols; ++u) idx[u] = 0;
            // halving steps over the first `top` entries only (top = the power of two that covers the
            // intervals): the table reads of 16 warps are what this loop is bound by
            for (int step = top >> 1; step >= 1; step >>= 1) {
#pragma unroll
                for (int u = 0; u < kCols; ++u)
                    if (f_lo[idx[u] + step] <= key[u]) idx[u] += step;
            }
            unsigned m[kCols];
            int total = 0;
#pragma unroll
            for (int u = 0; u < kCols; ++u) {
                in[u] = (i0 + u * 32 + lane < src_cnt) && key[u] >= f_lo[idx[u]] && key[u] <= f_hi[idx[u]];
                m[u] = __ballot_sync(0xffffffffu, in[u]);
                total += __popc(m[u]);
            }
            if (total) {  // one counter update per warp and trip
                int pos = 0;
                if (lane == 0) pos = atomicAdd(&S.n_keys, total);
                pos = __shfl_sync(0xffffffffu, pos, 0);
#pragma unroll
                for (int u = 0; u < kCols; ++u) {
                    const int at = pos + __popc(m[u] & ((1u << lane) - 1u));
                    if (in[u] && at < kSmallN) skeys[at] = key[u];
                    pos += __popc(m[u]);
                }
            }
        }
    }
    __syncthreads();
    const int c = S.n_keys < kSmallN ? S.n_keys : kSmallN;
    int P = 1;
    while (P < c) P <<= 1;
    for (int i = c + threadIdx.x; i < kSmallN; i += kSelThreads) skeys[i] = 0xffffffffu;
    __syncthreads();
    block_bitonic_sort(skeys, P);
    // pass 1: run starts and value sums of this thread's kPer consecutive sorted elements
    const int base = threadIdx.x * kPer;
    uint32_t k[kPer];
    unsigned long long lu = 0;
    double ls = 0.0;
    uint32_t prev = (base > 0 && base <= c) ? skeys[base - 1] : 0u;
#pragma unroll
    for (int e = 0; e < kPer; ++e) {
        const int i = base + e;
        k[e] = (i < c) ? skeys[i] : 0xffffffffu;
        if (i < c) {
            const bool flag = (i == 0) || (k[e] != (e == 0 ? prev : k[e - 1]));
            lu += flag ? 1 : 0;
            ls += (double)sel_key_to_float(k[e]);
        }
    }
    unsigned long long ubase = lu, tu;
    double sbase = ls, tsum;
    block_excl_scan(ubase, sbase, S.sc, S.ss, tu, tsum);
    if (threadIdx.x == 0) S.n_unique = (int)tu;
    // interval of each of this thread's keys, of the key before them and of the key after them
    // (searched once; the passes below reuse them)
    int jv[kPer];
#pragma unroll
    for (int e = 0; e < kPer; ++e) jv[e] = (base + e < c) ? find_new_interval(S, k[e]) : -1;
    const int jprev = (base > 0 && base <= c) ? find_new_interval(S, prev) : -2;
    const uint32_t knext = (base + kPer < c) ? skeys[base + kPer] : 0u;
    const int jnext = (base + kPer < c) ? find_new_interval(S, knext) : -3;
    // pass 2: first element of every interval
    {
        int nf = 0;
        double run = sbase;
#pragma unroll
        for (int e = 0; e < kPer; ++e) {
            const int i = base + e;
            if (i < c) {
                const uint32_t pk = (e == 0) ? prev : k[e - 1];
                const bool flag = (i == 0) || (k[e] != pk);
                if (flag) {
                    const int j = jv[e];
                    const int jp = (i == 0) ? -2 : ((e == 0) ? jprev : jv[e - 1]);
                    if (j >= 0 && j != jp) {
                        S.ivstart[j] = i;
                        S.ivpre[j] = run;
                        S.ivufirst[j] = (int)ubase + nf;
                    }
                    ++nf;
                }
                run += (double)sel_key_to_float(k[e]);
            }
        }
    }
    __syncthreads();
    // pass 3: explicit cells (slot = unique index + interval index) and the end slot of every interval
    {
        int nf = 0;
        double run = sbase;
#pragma unroll
        for (int e = 0; e < kPer; ++e) {
            const int i = base + e;
            if (i < c) {
                const uint32_t pk = (e == 0) ? prev : k[e - 1];
                const bool flag = (i == 0) || (k[e] != pk);
                const int j = jv[e];
                const double val = (double)sel_key_to_float(k[e]);
                if (flag) {
                    const int u = (int)ubase + nf;
                    xkeys[u] = k[e];
                    if (j >= 0) {
                        xcpre[u + j] = (uint32_t)(S.niv[j].cbefore + (long long)(i - S.ivstart[j]));
                        xspre[u + j] = S.niv[j].sbefore + (run - S.ivpre[j]);
                    }
                    ++nf;
                }
                const int jn = (i + 1 < c) ? ((e + 1 < kPer) ? jv[e + 1] : jnext) : -4;
                const bool last_of_iv = (i + 1 >= c) || (jn != j);
                if (last_of_iv && j >= 0) {
                    const int u = (int)ubase + nf - 1;
                    xcpre[u + 1 + j] = (uint32_t)(S.niv[j].cbefore + (long long)(i + 1 - S.ivstart[j]));
                    xspre[u + 1 + j] = S.niv[j].sbefore + ((run + val) - S.ivpre[j]);
                    S.niv[j].ncell = u - S.ivufirst[j] + 1;
                }
                run += val;
            }
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int next = S.n_unique;
        for (int j = S.nm - 1; j >= 0; --j) {
            if (S.ivufirst[j] < 0) {  // no element left in this interval: only its end slot
                S.niv[j].ncell = 0;
                xcpre[next + j] = (uint32_t)S.niv[j].cbefore;
                xspre[next + j] = S.niv[j].sbefore;
            } else {
                next = S.ivufirst[j];
            }
        }
        int cb = 0;
        for (int j = 0; j < S.nm; ++j) { S.niv[j].sh = 0; S.niv[j].cellbase = cb; cb += S.niv[j].ncell; }
        S.view.slot_iv = nullptr; S.view.xkeys = xkeys; S.view.cpre = xcpre; S.view.spre = xspre;
        S.view.iv = S.niv; S.view.m = S.nm;
        sel_init_slots(S.view);
        S.internal = (S.n_keys > kSmallN) ? 1 : 0;
    }
    // one thread per level, one depth at a time (every cell is a single key now, so each solve is exact)
    for (int stride = (s - 1) >> 1; stride >= 1; stride >>= 1) {
        __syncthreads();
        const int q = threadIdx.x >> 5;  // one warp per level, as in solver_round
        if ((threadIdx.x & 31) == 0 && !S.internal && q < s - 1 && q >= stride && ((q - stride) % (2 * stride)) == 0 &&
            !S.lv[q].exact) {
            if (!sel_orq_solve(S.view, S.lv[q - stride], S.lv[q + stride], S.lv[q])) S.internal = 1;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        bool ok = !S.internal;
        for (int q = 0; q < s; ++q) ok = ok && S.lv[q].exact;
        if (ok) {
            for (int q = 0; q < s; ++q) levels[(int64_t)t * s + q] = sel_key_to_float(S.lv[q].key);
        } else {
            status[t] |= OGQ_ST_INTERNAL;
            for (int q = 0; q < s; ++q) levels[(int64_t)t * s + q] = 0.f;
        }
        st->done = 1;
        __threadfence();
    }
    __syncthreads();
}

// Warp-parallel version of the common case of sel_refine: the open ranges are sorted and do not
// touch, every range yields at most four pieces, there are at most 32 pieces and none is wider
// than an equal share of the cell budget.  Lane i first cuts range i into pieces, then lane k
// builds interval k.  Returns false (nothing written) when the case is not the common one; the
// caller then runs the general single-thread routine.  Called by the 32 lanes of warp 0.
__device__ bool refine_parallel(SolverShared& S, bool trim_empty)
{
    const SolverView& v = S.view;
    const int lane = threadIdx.x & 31;
    const int nr = S.nr;
    int p_a[4], p_b[4], np = 0;
    bool fail = nr > 32;
    if (lane < nr && !fail) {
        const int a = S.ra[lane], b = S.rb[lane];
        if (lane > 0 && a <= S.rb[lane - 1] + 1) fail = true;
        int first = a, last = b;
        long long cnt = 1;
        if (trim_empty) {
            cnt = (long long)v.cpre[b + 1] - (long long)v.cpre[a];
            if (cnt > 0) {
                bool gap;
                first = sel_locate(v, (long long)v.cpre[a], true, &gap);
                last = sel_locate(v, (long long)v.cpre[b + 1] - 1, false, &gap);
                if (first < a || last > b || first > last) fail = true;
            }
        }
        if (cnt > 0 && !fail) {
            const int width = last - first + 1;
            if (trim_empty && width <= 12) {
                int run_a = -1, lastp = -1;
                for (int c = first; c <= last + 1; ++c) {
                    const bool boundary = (c > last) || sel_is_end_slot(v, c);
                    const bool populated = !boundary && v.cpre[c + 1] != v.cpre[c];
                    if (run_a >= 0 && (boundary || (!populated && c - lastp > 1))) {
                        if (np >= 4) { fail = true; break; }
#pragma unroll
                        for (int u = 0; u < 4; ++u) if (u == np) { p_a[u] = run_a; p_b[u] = lastp; }
                        ++np;
                        run_a = -1;
                    }
                    if (populated) { if (run_a < 0) run_a = c; lastp = c; }
                }
            } else {
                // wide: the trimmed hull, cut where it crosses into another interval (if it is too wide
                // for its share of the cells the general routine takes over below)
                const int j0 = sel_interval_of_slot(v, first), j1 = sel_interval_of_slot(v, last);
                for (int j = j0; j <= j1; ++j) {
                    const int lo = v.slotbase[j], hi = v.slotbase[j] + v.iv[j].ncell - 1;
                    const int x = first > lo ? first : lo, y = last < hi ? last : hi;
                    if (x > y) continue;
                    if (np >= 4) { fail = true; break; }
#pragma unroll
                    for (int u = 0; u < 4; ++u) if (u == np) { p_a[u] = x; p_b[u] = y; }
                    ++np;
                }
            }
        }
    }
    if (__any_sync(0xffffffffu, fail)) return false;
    // piece offsets
    int incl = np;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int nb = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += nb;
    }
    const int m = __shfl_sync(0xffffffffu, incl, 31);
    if (m == 0 || m > 32) return false;
#pragma unroll
    for (int u = 0; u < 4; ++u)
        if (u < np) { S.pa[incl - np + u] = p_a[u]; S.pb[incl - np + u] = p_b[u]; }
    __syncwarp();
    // one lane per piece: equal share of the cell budget
    const int share = kCells / m;
    int cells = 0, sh = 0, r = 0, j = 0, pa = 0, pb = 0;
    long long elems = 0;
    if (lane < m) {
        pa = S.pa[lane]; pb = S.pb[lane];
        cells = pb - pa + 1;
        j = sel_interval_of_slot(v, pa);
        sh = v.iv[j].sh;
        r = (cells <= share) ? sel_floor_log2(share / cells) : -1;
        if (r > sh) r = sh;
        elems = (long long)v.cpre[pb + 1] - (long long)v.cpre[pa];
    }
    if (__any_sync(0xffffffffu, lane < m && r < 0)) return false;  // a piece wider than its share
    const int ncell = (lane < m) ? (cells << r) : 0;
    int cinc = ncell;
    long long einc = elems;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int nb = __shfl_up_sync(0xffffffffu, cinc, o);
        const long long eb = __shfl_up_sync(0xffffffffu, einc, o);
        if (lane >= o) { cinc += nb; einc += eb; }
    }
    const bool progress = __any_sync(0xffffffffu, lane < m && r > 0);
    const bool open_shift = __any_sync(0xffffffffu, lane < m && sh - r > 0);
    if (open_shift && !progress) return false;
    if (lane < m) {
        const Interval& o = v.iv[j];
        Interval& ni = S.niv[lane];
        ni.sh = sh - r;
        ni.ncell = ncell;
        ni.klo = o.klo + ((uint32_t)(pa - v.slotbase[j]) << o.sh);
        ni.khi = ni.klo + (uint32_t)((((unsigned long long)ncell) << ni.sh) - 1ull);
        ni.cellbase = cinc - ncell;
        ni.pad = 0;
        ni.cbefore = v.cpre[pa];
        ni.sbefore = v.spre[pa];
    }
    if (lane == 31) { S.cand = einc; S.nm = m; }
    __syncwarp();
    return true;
}

// Runs one solver pass for tensor t after all of its pieces of the current round arrived.
// Called by every thread of the CTA; returns true when the tensor is finished.
__device__ bool solver_round(TState* st, int t, uint32_t* gcnt, unsigned long long* glsum, int scheme,
                             int s, float* __restrict__ levels, int32_t* __restrict__ status,
                             unsigned* nitems, int2* items, const uint32_t* round_buf, bool enqueue,
                             unsigned char* smem, SolverShared& S, int64_t cap)
{
    constexpr size_t kOffSpre = (kSlots * sizeof(uint32_t) + 15) / 16 * 16;
    uint32_t* cpre = reinterpret_cast<uint32_t*>(smem);
    double* spre = reinterpret_cast<double*>(smem + kOffSpre);
    uint8_t* slot_iv = smem + kOffSpre + kSlots * sizeof(double);
    const bool pb = scheme == OGQ_BINGRAD_PB;
    const int round = st->round;

    __syncthreads();
    if ((int)threadIdx.x < st->m) S.iv[threadIdx.x] = st->iv[threadIdx.x];
    __syncthreads();
    if (threadIdx.x == 0) {
        S.view.m = st->m;
        S.view.iv = S.iv;
        S.view.slot_iv = slot_iv;
        S.view.xkeys = nullptr;
        S.view.cpre = cpre;
        S.view.spre = spre;
        S.view.n = st->n;
        sel_init_slots(S.view);
        S.done = 0; S.nm = 0; S.internal = 0;
        S.pb_a = -1; S.pb_b = -1; S.pb_c = -1;
    }
    __syncthreads();

    // ---- prefix arrays over all slots: raw cell values, one block scan, per-interval shifts
    const int nslots = S.view.nslots, m = S.view.m;
    const int per = (nslots + kSelThreads - 1) / kSelThreads;
    const int s0 = (int)threadIdx.x * per < nslots ? (int)threadIdx.x * per : nslots;
    const int s1 = s0 + per < nslots ? s0 + per : nslots;
    {
        // interval index of every slot (blocked over threads, no global traffic)
        int j = 0;
        if (s0 < nslots) {
            int lo = 0, hi = m;
            while (hi - lo > 1) { const int mid = (lo + hi) >> 1; if (S.view.slotbase[mid] <= s0) lo = mid; else hi = mid; }
            j = lo;
        }
        for (int slot = s0; slot < s1; ++slot) {
            while (slot >= S.view.slotbase[j + 1]) ++j;
            slot_iv[slot] = (uint8_t)j;
        }
        __syncthreads();
        // raw (count, sum) of every cell: strided so that the global loads are coalesced and independent
        // (all of a thread's loads are issued before the first is used: they come from L2)
        constexpr int kPerThread = (kSlots + kSelThreads - 1) / kSelThreads;
        uint32_t rc[kPerThread];
        unsigned long long rl[kPerThread];
#pragma unroll
        for (int u = 0; u < kPerThread; ++u) {
            const int slot = threadIdx.x + u * kSelThreads;
            rc[u] = 0u;
            rl[u] = 0ull;
            if (slot < nslots) {
                const int jj = slot_iv[slot];
                const int c = slot - S.view.slotbase[jj];
                if (c < S.iv[jj].ncell) {
                    rc[u] = __ldcg(gcnt + S.iv[jj].cellbase + c);
                    rl[u] = __ldcg(glsum + S.iv[jj].cellbase + c);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kPerThread; ++u) {
            const int slot = threadIdx.x + u * kSelThreads;
            if (slot < nslots) {
                double sm = 0.0;
                if (rc[u]) {
                    const int jj = slot_iv[slot];
                    const int c = slot - S.view.slotbase[jj];
                    sm = sel_cell_sum(S.iv[jj].klo + ((uint32_t)c << S.iv[jj].sh), S.iv[jj].sh, rc[u], rl[u]);
                }
                cpre[slot] = rc[u];
                spre[slot] = sm;
            }
        }
        __syncthreads();
        // exclusive prefix: per-thread blocks, one block scan, in place
        unsigned long long lc = 0;
        double ls = 0.0;
        for (int slot = s0; slot < s1; ++slot) { lc += cpre[slot]; ls += spre[slot]; }
        unsigned long long tc;
        double ts;
        block_excl_scan(lc, ls, S.sc, S.ss, tc, ts);
        for (int slot = s0; slot < s1; ++slot) {
            const unsigned long long cn = cpre[slot];
            const double sm = spre[slot];
            cpre[slot] = (uint32_t)lc;
            spre[slot] = ls;
            lc += cn;
            ls += sm;
        }
    }
    __syncthreads();
    if ((int)threadIdx.x < m) {
        // rounds >= 2: shift every interval so that it starts from the exact (count, sum) before it
        const int sb = S.view.slotbase[threadIdx.x];
        S.offc[threadIdx.x] = (round == 1) ? 0u : (uint32_t)((unsigned long long)S.iv[threadIdx.x].cbefore - cpre[sb]);
        S.offs[threadIdx.x] = (round == 1) ? 0.0 : S.iv[threadIdx.x].sbefore - spre[sb];
    }
    __syncthreads();
    if (round != 1)
        for (int slot = s0; slot < s1; ++slot) {
            const int j = slot_iv[slot];
            cpre[slot] += S.offc[j];
            spre[slot] += S.offs[j];
        }
    __syncthreads();
    if (threadIdx.x == 0) {
        if (round == 1) {
            st->stot = spre[nslots - 1];
            if ((long long)cpre[nslots - 1] != st->n) S.internal = 1;
        }
        S.view.stot = st->stot;
    }
    __syncthreads();

    if (pb && !S.internal && S.view.stot > 0.0) {
        // bracket of the sign change of g, evaluated at the lower edge of every cell
        int a = -1, b = -1, cs = -1;
        for (int sl = threadIdx.x; sl < nslots; sl += kSelThreads) {
            if (sel_is_end_slot(S.view, sl)) continue;
            double x;
            const double g = sel_pb_g(S.view, sl, &x);
            if (!(x < INFINITY)) continue;
            const double eps = 1e-11 * (x * (double)S.view.n + S.view.stot);
            if (g < -eps) a = sl;
            if (g <= eps) b = sl;
            if (g <= 0.0) cs = sl;
        }
        if (a >= 0) atomicMax(&S.pb_a, a);
        if (b >= 0) atomicMax(&S.pb_b, b);
        if (cs >= 0) atomicMax(&S.pb_c, cs);
    }
    if (!pb && !S.internal) {
        // one thread per level, one depth of Algorithm 1 at a time
        if ((int)threadIdx.x < s) {
            LvInfo& l = S.lv[threadIdx.x];
            if (round == 1) {
                l.exact = 0;
                if (threadIdx.x == 0) {
                    l.exact = 1; l.key = ~__ldcg(&st->kmin_inv); l.val = (double)sel_key_to_float(l.key);
                    l.c_lt = 0; l.s_lt = 0.0; l.c_le = 0; l.s_le = 0.0;
                } else if ((int)threadIdx.x == s - 1) {
                    l.exact = 1; l.key = __ldcg(&st->kmax); l.val = (double)sel_key_to_float(l.key);
                    l.c_lt = 0; l.s_lt = 0.0; l.c_le = S.view.n; l.s_le = S.view.stot;
                }
            } else {
                const ExactLv& e = st->lv[threadIdx.x];
                l.exact = e.exact; l.key = e.key; l.val = (double)sel_key_to_float(e.key);
                l.c_lt = e.c_lt; l.c_le = e.c_le; l.s_lt = e.s_lt; l.s_le = e.s_le;
            }
        }
        // (one warp per level: the solves of one depth are long chains of dependent shared-memory
        // reads and fp64 divisions, and lanes of one warp that take different branches would run
        // one after the other)
        static_assert(kSelWarps >= kMaxLv - 1, "one warp per interior level");
        for (int stride = (s - 1) >> 1; stride >= 1; stride >>= 1) {
            __syncthreads();
            const int q = threadIdx.x >> 5;
            if ((threadIdx.x & 31) == 0 && q < s - 1 && q >= stride && ((q - stride) % (2 * stride)) == 0 &&
                !S.lv[q].exact) {
                if (!sel_orq_solve(S.view, S.lv[q - stride], S.lv[q + stride], S.lv[q])) S.internal = 1;
            }
        }
    }
    __syncthreads();

    if (threadIdx.x == 0) {
        int open = 0;
        int stbits = 0;
        if (S.internal) {
            stbits = OGQ_ST_INTERNAL;
            S.done = 1;
        } else if (pb) {
            if (!(S.view.stot > 0.0)) {
                levels[2 * t] = 0.f; levels[2 * t + 1] = 0.f;
                stbits = OGQ_ST_CONSTANT;
                S.done = 1;
            } else {
                int a = S.pb_a < 0 ? 0 : S.pb_a;
                int b = S.pb_b < a ? a : S.pb_b;
                int cs = S.pb_c < a ? a : S.pb_c;
                if (cs > b) cs = b;
                bool fine = true;
                for (int sl = a; sl <= b; ++sl)
                    if (!sel_is_end_slot(S.view, sl) && sel_slot_shift(S.view, sl) != 0) fine = false;
                if (fine && !sel_is_end_slot(S.view, cs)) {
                    const float b1 = (float)sel_pb_final(S.view, cs);
                    levels[2 * t] = -b1; levels[2 * t + 1] = b1;
                    S.done = 1;
                } else {
                    S.ra[0] = a; S.rb[0] = b; open = 1;
                }
            }
        } else {
            for (int q = 1; q < s - 1; ++q)
                if (!S.lv[q].exact) { S.ra[open] = S.lv[q].sa; S.rb[open] = S.lv[q].sb; ++open; }
            if (open == 0) S.done = 1;
        }
        S.nr = open;
        S.nm = -100;
        S.cand = 0;
        if (!S.done && round + 1 > kMaxRounds) { stbits = OGQ_ST_ITER_CAP; S.done = 1; }
        if (stbits) {
            // unresolved: leave zeros rather than garbage
            if (pb) { levels[2 * t] = 0.f; levels[2 * t + 1] = 0.f; }
            else for (int q = 0; q < s; ++q) levels[(int64_t)t * s + q] = 0.f;
            status[t] |= stbits;
        }
    }
    __syncthreads();
    if (!pb && !S.internal && (int)threadIdx.x < s) {
        if (S.done) {
            if (S.nr == 0 && !(status[t] & (OGQ_ST_ITER_CAP | OGQ_ST_INTERNAL)))
                levels[(int64_t)t * s + threadIdx.x] = sel_key_to_float(S.lv[threadIdx.x].key);
        } else {
            ExactLv& e = st->lv[threadIdx.x];
            const LvInfo& l = S.lv[threadIdx.x];
            e.exact = l.exact; e.key = l.key; e.c_lt = l.c_lt; e.c_le = l.c_le; e.s_lt = l.s_lt; e.s_le = l.s_le;
        }
    }
    if (!S.done) {
        // intervals of the next round: warp-parallel common case, single-thread general case
        bool ok = true;
        if (threadIdx.x < 32) ok = refine_parallel(S, !pb);
        if (threadIdx.x == 0 && !ok) {
            const int nm = sel_refine(S.view, S.nr, S.ra, S.rb, !pb, S.niv, &S.cand);
            if (nm < 0) {
                if (pb) { levels[2 * t] = 0.f; levels[2 * t + 1] = 0.f; }
                else for (int q = 0; q < s; ++q) levels[(int64_t)t * s + q] = 0.f;
                status[t] |= OGQ_ST_INTERNAL;
                S.done = 1;
            } else {
                S.nm = nm;
            }
        }
    }
    __syncthreads();

    if (S.done) {
        if (threadIdx.x == 0) { st->done = 1; __threadfence(); }
        return true;
    }
    // (the copies of the pass that just ended are complete unless it overflowed its region)
    const bool incomplete = round >= 2 && __ldcg(&st->overflow) != 0;
    if (!pb && round >= 2 && S.cand <= kSmallN && round_buf != nullptr && !incomplete) {
        const long long src_cnt = (long long)__ldcg(&st->cursor[round & 1]);
        if (src_cnt <= kSortScanMax) {
            sort_finish(st, t, s, round_buf, src_cnt, levels, status, smem, S);
            return true;
        }
    }
    // prepare the next round: clear the cells it will use, publish the new intervals.  When the
    // elements inside the new intervals already fit one sort (ORQ), the next pass only copies them
    // and its last CTA sorts and finishes the tensor (finish_sorted): no cells, no further solver pass.
    const bool compact_only = !pb && S.cand <= kSmallN && S.cand <= cap;
    const int ncells_next = S.niv[S.nm - 1].cellbase + S.niv[S.nm - 1].ncell;
    if (!compact_only)
        for (int i = threadIdx.x; i < ncells_next; i += kSelThreads) {
            gcnt[i] = 0u;
            glsum[i] = 0ull;
        }
    if ((int)threadIdx.x < S.nm) st->iv[threadIdx.x] = S.niv[threadIdx.x];
    if (threadIdx.x == 0) {
        st->m = S.nm;
        st->compact_only = compact_only ? 1 : 0;
        st->from_grad = incomplete ? 1 : 0;  // the next pass cannot read copies that were cut short
        st->overflow = 0;
        st->round = round + 1;
        st->arrive = 0;
        st->arrived = 0ull;
        const int next = round + 1;
        st->cursor[next & 1] = 0ull;  // buffer the next round writes
        if (next == 3 && enqueue) {
            // work items of the round-3 kernel: slices of the copied keys, or of the tensor itself when
            // the copies were cut short
            const unsigned long long cntk = incomplete ? (unsigned long long)(st->n / 16) : __ldcg(&st->cursor[0]);
            unsigned ns = (unsigned)((cntk + kSliceElems - 1) / kSliceElems);
            if (ns < 1) ns = 1;
            if (ns > kMaxSlices) ns = kMaxSlices;
            st->expected = ns;
            const unsigned base = atomicAdd(nitems, ns);
            for (unsigned i = 0; i < ns; ++i) items[base + i] = make_int2(t, (int)i);
        }
    }
    __threadfence();
    __syncthreads();
    return false;
}

// Finishes a tensor whose last pass only copied the keys inside its intervals (TState::compact_only):
// the solver state the previous pass left in global memory is loaded back, then the copied keys are
// sorted and every open level is solved on single-key cells.  Called by every thread of the CTA that
// arrived last for the tensor.
__device__ void finish_sorted(TState* st, int t, int s, const uint32_t* copied, float* __restrict__ levels,
                              int32_t* __restrict__ status, unsigned char* smem, SolverShared& S, int cursor_idx)
{
    __syncthreads();
    const int m = __ldcg(&st->m);
    if ((int)threadIdx.x < m) S.niv[threadIdx.x] = st->iv[threadIdx.x];
    if ((int)threadIdx.x < s) {
        const ExactLv& e = st->lv[threadIdx.x];
        LvInfo& l = S.lv[threadIdx.x];
        l.exact = e.exact; l.key = e.key; l.val = (double)sel_key_to_float(e.key);
        l.c_lt = e.c_lt; l.c_le = e.c_le; l.s_lt = e.s_lt; l.s_le = e.s_le;
        l.sa = l.sb = 0; l.vlo = l.vhi = l.val;
    }
    if (threadIdx.x == 0) {
        S.nm = m;
        S.view.n = st->n;
        S.view.stot = st->stot;
        S.internal = 0;
    }
    __syncthreads();
    const long long src_cnt = (long long)__ldcg(&st->cursor[cursor_idx]);
    sort_finish(st, t, s, copied, src_cnt, levels, status, smem, S);
}

// ---------------------------------------------------------------------------
// Small tensors: sort the keys in shared memory and apply the definitions directly.
// ---------------------------------------------------------------------------
__device__ __forceinline__ int lower_bound_u32(const uint32_t* a, int n, uint32_t k)
{
    int lo = 0, hi = n;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (a[mid] < k) lo = mid + 1; else hi = mid; }
    return lo;
}

__device__ __forceinline__ int upper_bound_u32(const uint32_t* a, int n, uint32_t k)
{
    int lo = 0, hi = n;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (a[mid] <= k) lo = mid + 1; else hi = mid; }
    return lo;
}

__device__ void small_tensor(const float* __restrict__ grad, int64_t tb, int n, int t, int scheme, int s,
                             float* __restrict__ levels, int32_t* __restrict__ status, TState* st,
                             unsigned char* smem, float tau)
{
    __shared__ double sh_d[kSelWarps];
    __shared__ uint32_t sh_lvkey[kMaxLv];
    __shared__ int sh_flag;
    __shared__ double sh_bcast;
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem);
    const bool pb = scheme == OGQ_BINGRAD_PB;
    int P = 1;
    while (P < n) P <<= 1;
    if (threadIdx.x == 0) sh_flag = 0;
    __syncthreads();
    for (int i = threadIdx.x; i < P; i += kSelThreads) {
        uint32_t key = 0xffffffffu;
        if (i < n) {
            const float raw = __ldg(grad + tb + i);
            uint32_t bits = __float_as_uint(copysignf(fminf(fabsf(raw), tau), raw));
            if ((bits & 0x7f800000u) == 0x7f800000u) sh_flag = 1;
            if (pb) key = bits | 0x80000000u;
            else {
                if (bits == 0x80000000u) bits = 0u;
                key = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
            }
        }
        keys[i] = key;
    }
    __syncthreads();
    block_bitonic_sort(keys, P);  // ascending
    int stbits = 0;
    if (sh_flag) {
        if (threadIdx.x == 0) {
            const int nl = pb ? 2 : s;
            for (int q = 0; q < nl; ++q) levels[(int64_t)t * nl + q] = 0.f;
            status[t] = OGQ_ST_NONFINITE;
            st->done = 1;
        }
        return;
    }
    if (!pb) {
        if (keys[0] == keys[n - 1]) stbits |= OGQ_ST_CONSTANT;
        if (threadIdx.x == 0) {
            for (int q = 0; q < s; ++q) sh_lvkey[q] = keys[0];
            sh_lvkey[s - 1] = keys[n - 1];
        }
        __syncthreads();
        for (int stride = (s - 1) >> 1; stride >= 1; stride >>= 1) {
            for (int q = stride; q < s - 1; q += 2 * stride) {
                const uint32_t kl = sh_lvkey[q - stride], kr = sh_lvkey[q + stride];
                uint32_t res = kl;
                if (kr > kl) {
                    const int i0 = lower_bound_u32(keys, n, kl), i1 = upper_bound_u32(keys, n, kr);
                    const double Lv = (double)sel_key_to_float(kl), Rv = (double)sel_key_to_float(kr);
                    double a = 0.0;
                    for (int i = i0 + threadIdx.x; i < i1; i += kSelThreads) a += (double)sel_key_to_float(keys[i]) - Lv;
                    a = sel_block_sum(a, sh_d);
                    if (threadIdx.x == 0) sh_bcast = a;
                    __syncthreads();
                    a = sh_bcast;
                    const double T = a / (Rv - Lv);
                    long long k = (long long)floor(T);
                    const long long m = i1 - i0;
                    if (k < 0) k = 0;
                    if (k > m - 1) k = m - 1;
                    res = keys[i1 - 1 - (int)k];
                }
                __syncthreads();
                if (threadIdx.x == 0) sh_lvkey[q] = res;
                __syncthreads();
            }
        }
        if (threadIdx.x < s) levels[(int64_t)t * s + threadIdx.x] = sel_key_to_float(sh_lvkey[threadIdx.x]);
        if (threadIdx.x == 0) { status[t] = stbits; st->done = 1; }
        return;
    }
    // BinGrad-pb: prefix sums of the sorted magnitudes, then the sign change of g
    double* pre = reinterpret_cast<double*>(smem + kSmallN * sizeof(uint32_t));  // [n + 1]
    __shared__ unsigned long long sc_[kSelWarps];
    __shared__ double ss_[kSelWarps];
    __shared__ int sh_c;
    const int per = (n + kSelThreads - 1) / kSelThreads;
    const int c0 = threadIdx.x * per < n ? threadIdx.x * per : n;
    const int c1 = c0 + per < n ? c0 + per : n;
    unsigned long long dummy = 0, dt;
    double ls = 0.0, tot;
    for (int i = c0; i < c1; ++i) ls += (double)sel_key_to_float(keys[i]);
    block_excl_scan(dummy, ls, sc_, ss_, dt, tot);
    double run = ls;
    for (int i = c0; i < c1; ++i) { pre[i] = run; run += (double)sel_key_to_float(keys[i]); }
    if (threadIdx.x == 0) { pre[n] = tot; sh_c = -1; }
    __syncthreads();
    int best = -1;
    for (int i = threadIdx.x; i < n; i += kSelThreads) {
        const double x = (double)sel_key_to_float(keys[i]);
        const int first = lower_bound_u32(keys, n, keys[i]);
        const double g = x * (double)n - (tot - pre[first]);
        if (g <= 0.0) best = i;
    }
    if (best >= 0) atomicMax(&sh_c, best);
    __syncthreads();
    if (threadIdx.x == 0) {
        float b1 = 0.f;
        if (!(tot > 0.0)) stbits |= OGQ_ST_CONSTANT;
        else {
            const int c = sh_c < 0 ? 0 : sh_c;
            const double x = (double)sel_key_to_float(keys[c]);
            const int up = upper_bound_u32(keys, n, keys[c]);
            const double stat_up = (tot - pre[up]) / (double)n;
            b1 = (float)(stat_up > x ? stat_up : x);
        }
        levels[2 * t] = -b1; levels[2 * t + 1] = b1;
        status[t] = stbits;
        st->done = 1;
    }
}

// ---------------------------------------------------------------------------
// Kernels
// ---------------------------------------------------------------------------
struct SelArgs {
    const float* grad;
    const float* tau;  // per-tensor clipping thresholds, or null
    const int64_t* off;
    int T;
    int64_t total, chunk;
    int flat_ctas, scheme, s;
    float* levels;
    int32_t* status;
    SelWs ws;
};

// One pass over grad[pb_, pe_) of tensor t with the tensor's current intervals (table and prefilter
// already built in tb): the values inside the intervals are copied to key buffer k (what fits the
// tensor's region) and, unless copy_only, counted on the cells.
__device__ __forceinline__ void grad_pass(const SelArgs& A, int t, int64_t tbeg, int64_t tend, int64_t pb_, int64_t pe_,
                                          int k, const Table& tb, uint32_t* hist, unsigned char* smem, bool copy_only)
{
    TState* st = A.ws.st + t;
    uint32_t* stage = reinterpret_cast<uint32_t*>(smem + kSmemHist) + (threadIdx.x >> 5) * kStageCap;
    uint32_t* dst = A.ws.buf[k] + sel_region(tbeg);
    const int64_t cap = sel_region(tend) - sel_region(tbeg);
    const bool mag = A.scheme == OGQ_BINGRAD_PB;
    if (A.tau)
        stream_round2<true>(A.grad, pb_, pe_, mag, tb, hist, hist + kCells, hist + 2 * kCells, stage, dst, cap,
                            &st->cursor[k], &st->overflow, copy_only, __ldg(A.tau + t));
    else
        stream_round2<false>(A.grad, pb_, pe_, mag, tb, hist, hist + kCells, hist + 2 * kCells, stage, dst, cap,
                             &st->cursor[k], &st->overflow, copy_only, 0.f);
}

// Continues the rounds of one tensor on a single CTA until it is finished (the working set is
// tiny by then).  Called by the CTA that completed round >= 3.
__device__ void finish_alone(const SelArgs& A, int t, unsigned char* smem, Table& tb, SolverShared& S)
{
    TState* st = A.ws.st + t;
    uint32_t* gcnt = A.ws.gcnt + (size_t)t * kCells;
    unsigned long long* glsum = A.ws.glsum + (size_t)t * kCells;
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem);
    const int64_t tbeg = __ldg(A.off + t), tend = __ldg(A.off + t + 1);
    for (int guard = 0; guard < kMaxRounds; ++guard) {
        const int round = st->round;
        const uint32_t* src = A.ws.buf[(round - 1) & 1];  // 16-byte aligned base; indices are absolute
        const int64_t cnt = (int64_t)__ldcg(&st->cursor[(round - 1) & 1]);
        const bool copy_only = st->compact_only != 0;
        __syncthreads();
        if (threadIdx.x == 0) table_from_intervals(tb, st->iv, st->m);
        __syncthreads();
        if (!copy_only) zero_hist(hist, tb.ncells);
        __syncthreads();
        if (st->from_grad) {
            // the previous pass's copies did not fit: this pass reads the tensor itself again
            build_prefilter(tb, A.scheme == OGQ_BINGRAD_PB);
            grad_pass(A, t, tbeg, tend, tbeg, tend, round & 1, tb, hist, smem, copy_only);
        } else {
            Stager stg;
            stg.stage = reinterpret_cast<uint32_t*>(smem + kSmemHist) + (threadIdx.x >> 5) * kStageCap;
            stg.dst = A.ws.buf[round & 1] + sel_region(tbeg);
            stg.cursor = &st->cursor[round & 1];
            stg.fill = 0;
            uint32_t kmin = 0, kmax = 0, nf = 0;
            stream_piece<false, false, true>(src, sel_region(tbeg), sel_region(tbeg) + cnt, false, tb, hist, hist + kCells,
                                             hist + 2 * kCells, stg, kmin, kmax, nf, copy_only);
            stg.flush();
        }
        __syncthreads();
        if (copy_only) {
            __threadfence();
            __syncthreads();
            finish_sorted(st, t, A.s, A.ws.buf[round & 1] + sel_region(tbeg), A.levels, A.status, smem, S, round & 1);
            return;
        }
        flush_hist(hist, tb.ncells, gcnt, glsum);
        __threadfence();
        __syncthreads();
        if (solver_round(st, t, gcnt, glsum, A.scheme, A.s, A.levels, A.status, A.ws.nitems, A.ws.items,
                         A.ws.buf[round & 1] + sel_region(tbeg), false, smem, S, sel_region(tend) - sel_region(tbeg)))
            return;
    }
    if (threadIdx.x == 0) {
        A.status[t] |= OGQ_ST_ITER_CAP;
        st->done = 1;
    }
}

__global__ void __launch_bounds__(kSelThreads, kSelResident) k_sel_round1(SelArgs A)
{
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ SolverShared S;
    __shared__ Interval r1iv[kMaxIv];
    __shared__ int sh_i[kSelWarps];
    __shared__ int sh_last;
    const bool pb = A.scheme == OGQ_BINGRAD_PB;
    const int nl = pb ? 2 : A.s;

    uint32_t* hist = reinterpret_cast<uint32_t*>(smem);

    // Anchor of the fine window of tensor [tbeg, tbeg + n): largest binade among strided samples, plus
    // two (every CTA of the tensor samples the same elements and so arrives at the same window).
    auto window_anchor = [&](int64_t tbeg, int64_t n) -> int {
        int hi_e;
        {
            const int64_t idx = tbeg + (int64_t)threadIdx.x * n / kSelThreads;
            int e = (int)((__float_as_uint(__ldg(A.grad + idx)) >> 23) & 255u);
            if (e == 255) e = 0;
            e = __reduce_max_sync(0xffffffffu, e);
            __syncthreads();  // earlier readers of sh_i are done
            if ((threadIdx.x & 31) == 0) sh_i[threadIdx.x >> 5] = e;
            __syncthreads();
            hi_e = __reduce_max_sync(0xffffffffu, ((threadIdx.x & 31) < kSelWarps) ? sh_i[threadIdx.x & 31] : 0) + 2;
            if (hi_e < kSelW) hi_e = kSelW;
            if (hi_e > 255) hi_e = 255;  // binade 255 (Inf / NaN) always stays outside the fine window
        }
        return hi_e;
    };

    // Round 1 of a tensor on this CTA, in three steps: r1_begin clears the CTA's cells, r1_add streams
    // a piece of the tensor into them (any number of pieces), r1_flush adds the cells to the tensor's
    // global ones, reports `elems` streamed elements and returns true when that completes the tensor;
    // the CTA for which it does runs r1_solve.
    float r1_vmin = 0.f, r1_vmax = 0.f, r1_tau = 0.f;
    uint32_t r1_nf = 0u;
    int r1_lo_e = 0;
    uint32_t* packed_cells = reinterpret_cast<uint32_t*>(smem + kSmemHist);
    const int r1_ncells = pb ? kRound1Mag : kRound1Cells;
    auto r1_begin = [&](int t, int64_t tbeg, int64_t tend) {
        r1_lo_e = window_anchor(tbeg, tend - tbeg) - kSelW;
        r1_tau = A.tau ? __ldg(A.tau + t) : 0.f;
        r1_vmin = __int_as_float(0x7f800000);
        r1_vmax = __int_as_float(0xff800000);
        r1_nf = 0u;
        __syncthreads();
        zero_hist(hist, r1_ncells);
        for (int i = threadIdx.x; i < kPackedCells; i += kSelThreads) packed_cells[i] = 0u;
        __syncthreads();
    };
    auto r1_add = [&](int64_t pb_, int64_t pe_) {
        const bool clip = A.tau != nullptr;
        if (pb) {
            if (clip) stream_round1<true, true>(A.grad, pb_, pe_, r1_lo_e, hist, packed_cells, r1_vmin, r1_vmax, r1_nf, r1_tau);
            else stream_round1<true, false>(A.grad, pb_, pe_, r1_lo_e, hist, packed_cells, r1_vmin, r1_vmax, r1_nf, r1_tau);
        } else {
            if (clip) stream_round1<false, true>(A.grad, pb_, pe_, r1_lo_e, hist, packed_cells, r1_vmin, r1_vmax, r1_nf, r1_tau);
            else stream_round1<false, false>(A.grad, pb_, pe_, r1_lo_e, hist, packed_cells, r1_vmin, r1_vmax, r1_nf, r1_tau);
        }
    };
    auto r1_flush = [&](int t, int64_t n, int64_t elems) -> bool {
        TState* st = A.ws.st + t;
        __syncthreads();
        flush_hist(hist, r1_ncells, A.ws.gcnt + (size_t)t * kCells, A.ws.glsum + (size_t)t * kCells);
        // min / max / non-finite: one atomic per warp
        {
            const uint32_t kmin = __reduce_min_sync(0xffffffffu, float_to_key(r1_vmin));  // +Inf / -Inf when the
            const uint32_t kmax = __reduce_max_sync(0xffffffffu, float_to_key(r1_vmax));  // thread saw nothing
            const bool anynf = __any_sync(0xffffffffu, r1_nf != 0u);
            if ((threadIdx.x & 31) == 0) {
                atomicMax(&st->kmin_inv, ~kmin);
                atomicMax(&st->kmax, kmax);
                if (anynf) atomicOr(&st->nonfinite, 1u);
            }
        }
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) {
            const unsigned long long prev = atomicAdd(&st->arrived, (unsigned long long)elems);
            sh_last = (prev + (unsigned long long)elems == (unsigned long long)n);
        }
        __syncthreads();
        if (!sh_last) return false;
        __threadfence();
        return true;
    };

    // Last CTA of tensor t: sets up the state and runs the first solver pass.  Returns true when the
    // tensor is finished.
    auto r1_solve = [&](int t, int64_t tbeg, int64_t tend, bool alone) -> bool {
        const int64_t n = tend - tbeg;
        TState* st = A.ws.st + t;
        const int hi_e = window_anchor(tbeg, n);
        __syncthreads();
        if (threadIdx.x == 0) {
            st->n = n;
            st->round = 1;
            st->hi_e = hi_e;
            const int m = round1_intervals(hi_e, pb, r1iv);
            st->m = m;
            for (int j = 0; j < m; ++j) st->iv[j] = r1iv[j];
            int stb = 0;
            const uint32_t kmn = ~__ldcg(&st->kmin_inv), kmx = __ldcg(&st->kmax);
            if (__ldcg(&st->nonfinite)) stb |= OGQ_ST_NONFINITE;
            else if (!pb && kmn == kmx) stb |= OGQ_ST_CONSTANT;
            A.status[t] = stb;
            sh_last = stb;
            if (stb & OGQ_ST_NONFINITE) {
                for (int q = 0; q < nl; ++q) A.levels[(int64_t)t * nl + q] = 0.f;
                st->done = 1;
            } else if (stb & OGQ_ST_CONSTANT) {
                const float v = sel_key_to_float(kmn);
                for (int q = 0; q < nl; ++q) A.levels[(int64_t)t * nl + q] = v;
                st->done = 1;
            }
        }
        __syncthreads();
        if (sh_last & (OGQ_ST_NONFINITE | OGQ_ST_CONSTANT)) return true;
        bool done;
        done = solver_round(st, t, A.ws.gcnt + (size_t)t * kCells, A.ws.glsum + (size_t)t * kCells,
                                           A.scheme, A.s, A.levels, A.status, A.ws.nitems, A.ws.items, nullptr,
                                           !alone, smem, S, sel_region(tend) - sel_region(tbeg));
        return done;
    };

    if ((int)blockIdx.x < A.T) {
        // the first T CTAs, one per tensor, settle the empty, small and mid-size tensors; they come
        // first in the grid because the mid-size ones run longest
        [&]() {
        const int t = blockIdx.x;
        const int64_t tbeg = __ldg(A.off + t), tend = __ldg(A.off + t + 1);
        const int64_t n = tend - tbeg;
        if (n <= 0) {
            if (threadIdx.x < nl) A.levels[(int64_t)t * nl + threadIdx.x] = 0.f;
            if (threadIdx.x == 0) { A.status[t] = OGQ_ST_EMPTY; A.ws.st[t].done = 1; }
        } else if (n <= kSmallN) {
            small_tensor(A.grad, tbeg, (int)n, t, A.scheme, A.s, A.levels, A.status, A.ws.st + t, smem,
                         A.tau ? __ldg(A.tau + t) : __int_as_float(0x7f800000));
        } else if (n <= kMidN) {
            // round 1 and its solver pass on this CTA; the tensor's CTA of the round-2 kernel goes on from there
            r1_begin(t, tbeg, tend);
            r1_add(tbeg, tend);
            r1_flush(t, n, n);
            r1_solve(t, tbeg, tend, true);
        }
        }();
        return;
    }

    // Flat CTAs: one chunk of the bucket each.  The solver passes of the tensors this CTA completed wait
    // until its chunk has been streamed, so that a solver pass never holds up another tensor's arrival.
    // (Handing smaller chunks out from a counter was tried and lost: the CTAs of a launch already finish
    // within a few percent of one another, what ends late are the solver passes, and every extra chunk
    // boundary costs a set-up and, in round 2, a drain of the compaction stages.)
    constexpr int kDefer = 8;
    int dt[kDefer];
    int nd = 0;
    int cur_t = -1;
    int64_t cur_n = 0, cur_elems = 0;
    auto done_with_current = [&]() {
        if (cur_t < 0) return;
        if (r1_flush(cur_t, cur_n, cur_elems)) {
            if (nd < kDefer) {
#pragma unroll
                for (int u = 0; u < kDefer; ++u)
                    if (u == nd) dt[u] = cur_t;
                ++nd;
            } else {
                r1_solve(cur_t, __ldg(A.off + cur_t), __ldg(A.off + cur_t + 1), false);
            }
        }
        cur_t = -1;
    };
    {
        const int64_t lo = (int64_t)(blockIdx.x - A.T) * A.chunk;
        const int64_t hi = (lo + A.chunk < A.total) ? lo + A.chunk : A.total;
        for_each_piece(A.off, A.T, lo, hi, [&](int t, int64_t tbeg, int64_t tend, int64_t pb_, int64_t pe_) {
            if (tend - tbeg <= kMidN) return;
            if (t != cur_t) {
                done_with_current();
                r1_begin(t, tbeg, tend);
                cur_t = t;
                cur_n = tend - tbeg;
                cur_elems = 0;
            }
            r1_add(pb_, pe_);
            cur_elems += pe_ - pb_;
        });
    }
    done_with_current();
#pragma unroll
    for (int u = 0; u < kDefer; ++u)
        if (u < nd) r1_solve(dt[u], __ldg(A.off + dt[u]), __ldg(A.off + dt[u] + 1), false);
}

__global__ void __launch_bounds__(kSelThreads, kSelResident) k_sel_round2(SelArgs A)
{
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ Table tb;
    __shared__ SolverShared S;
    __shared__ int sh_last;
    const bool pb = A.scheme == OGQ_BINGRAD_PB;
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem);

    // Second pass over a tensor on this CTA, in three steps like round 1: r2_begin builds the tensor's
    // interval table and prefilter and clears the CTA's cells, r2_add streams a piece (copies the values
    // inside the intervals and counts them on the finer cells, unless they already fit one sort),
    // r2_flush adds the cells to the tensor's global ones.
    bool r2_copy_only = false;
    auto r2_begin = [&](int t) {
        TState* st = A.ws.st + t;
        __syncthreads();
        table_from_intervals_cta(tb, st->iv, __ldcg(&st->m));
        __syncthreads();
        build_prefilter(tb, pb);
        r2_copy_only = __ldcg(&st->compact_only) != 0;
        if (!r2_copy_only) zero_hist(hist, tb.ncells);
        __syncthreads();
    };
    auto r2_add = [&](int t, int64_t tbeg, int64_t tend, int64_t pb_, int64_t pe_) {
        grad_pass(A, t, tbeg, tend, pb_, pe_, 0, tb, hist, smem, r2_copy_only);
    };
    auto r2_flush = [&](int t) {
        __syncthreads();
        if (!r2_copy_only) flush_hist(hist, tb.ncells, A.ws.gcnt + (size_t)t * kCells, A.ws.glsum + (size_t)t * kCells);
        __threadfence();
        __syncthreads();
    };

    if ((int)blockIdx.x < A.T) {
        // the first T CTAs, one per tensor, take the mid-size tensors from where their CTA of the
        // round-1 kernel left them to the end (the tensor stays in L2, later rounds read copied keys)
        const int t = blockIdx.x;
        const int64_t tbeg = __ldg(A.off + t), tend = __ldg(A.off + t + 1);
        const int64_t n = tend - tbeg;
        TState* st = A.ws.st + t;
        if (n <= kSmallN || n > kMidN || __ldcg(&st->done)) return;
        r2_begin(t);
        r2_add(t, tbeg, tend, tbeg, tend);
        r2_flush(t);
        if (r2_copy_only) {
            finish_sorted(st, t, A.s, A.ws.buf[0] + sel_region(tbeg), A.levels, A.status, smem, S, 0);
            return;
        }
        if (solver_round(st, t, A.ws.gcnt + (size_t)t * kCells, A.ws.glsum + (size_t)t * kCells, A.scheme, A.s,
                         A.levels, A.status, A.ws.nitems, A.ws.items, A.ws.buf[0] + sel_region(tbeg), false, smem, S, sel_region(tend) - sel_region(tbeg)))
            return;
        finish_alone(A, t, smem, tb, S);
        return;
    }

    // flat CTAs: one chunk each, solver passes last (as in round 1)
    constexpr int kDefer = 8;
    int dt[kDefer];
    int nd = 0;
    auto finish = [&](int t) {
        TState* st = A.ws.st + t;
        const int64_t tbeg = __ldg(A.off + t), tend = __ldg(A.off + t + 1);
        if (__ldcg(&st->compact_only) != 0) {
            finish_sorted(st, t, A.s, A.ws.buf[0] + sel_region(tbeg), A.levels, A.status, smem, S, 0);
            return;
        }
        solver_round(st, t, A.ws.gcnt + (size_t)t * kCells, A.ws.glsum + (size_t)t * kCells, A.scheme, A.s,
                     A.levels, A.status, A.ws.nitems, A.ws.items, A.ws.buf[0] + sel_region(tbeg), true, smem, S, sel_region(tend) - sel_region(tbeg));
    };
    int cur_t = -1;
    int64_t cur_n = 0, cur_elems = 0;
    auto done_with_current = [&]() {
        if (cur_t < 0) return;
        r2_flush(cur_t);
        TState* st = A.ws.st + cur_t;
        if (threadIdx.x == 0) {
            const unsigned long long prev = atomicAdd(&st->arrived, (unsigned long long)cur_elems);
            sh_last = (prev + (unsigned long long)cur_elems == (unsigned long long)cur_n);
        }
        __syncthreads();
        if (sh_last) {
            __threadfence();
            if (nd < kDefer) {
#pragma unroll
                for (int u = 0; u < kDefer; ++u)
                    if (u == nd) dt[u] = cur_t;
                ++nd;
            } else {
                finish(cur_t);
            }
        }
        cur_t = -1;
    };
    {
        const int64_t lo = (int64_t)(blockIdx.x - A.T) * A.chunk;
        const int64_t hi = (lo + A.chunk < A.total) ? lo + A.chunk : A.total;
        for_each_piece(A.off, A.T, lo, hi, [&](int t, int64_t tbeg, int64_t tend, int64_t pb_, int64_t pe_) {
            const int64_t n = tend - tbeg;
            if (n <= kMidN) return;
            if (t != cur_t) {
                done_with_current();
                if (__ldcg(&A.ws.st[t].done)) return;  // settled in round 1
                r2_begin(t);
                cur_t = t;
                cur_n = n;
                cur_elems = 0;
            }
            r2_add(t, tbeg, tend, pb_, pe_);
            cur_elems += pe_ - pb_;
        });
    }
    done_with_current();
#pragma unroll
    for (int u = 0; u < kDefer; ++u)
        if (u < nd) finish(dt[u]);
}

__global__ void __launch_bounds__(kSelThreads, kSelResident) k_sel_round3(SelArgs A)
{
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ Table tb;
    __shared__ SolverShared S;
    __shared__ int sh_last;
    uint32_t* hist = reinterpret_cast<uint32_t*>(smem);
    const unsigned nitems = __ldcg(A.ws.nitems);

    for (unsigned w = blockIdx.x; w < nitems; w += gridDim.x) {
        const int2 it = A.ws.items[w];
        const int t = it.x;
        TState* st = A.ws.st + t;
        const int64_t tbeg = __ldg(A.off + t), tend = __ldg(A.off + t + 1);
        const unsigned ns = __ldcg(&st->expected);
        const bool from_grad = __ldcg(&st->from_grad) != 0;  // round 2's copies were cut short: slices of the tensor
        const int64_t cnt = from_grad ? tend - tbeg : (int64_t)__ldcg(&st->cursor[0]);
        int64_t per = (cnt + ns - 1) / ns;
        per = (per + 3) & ~(int64_t)3;
        int64_t pb_ = per * it.y, pe_ = pb_ + per;
        if (pb_ > cnt) pb_ = cnt;
        if (pe_ > cnt) pe_ = cnt;
        __syncthreads();
        if (threadIdx.x == 0) table_from_intervals(tb, st->iv, __ldcg(&st->m));
        const bool copy_only = __ldcg(&st->compact_only) != 0;
        __syncthreads();
        if (!copy_only) zero_hist(hist, tb.ncells);
        __syncthreads();
        if (from_grad) {
            build_prefilter(tb, A.scheme == OGQ_BINGRAD_PB);
            grad_pass(A, t, tbeg, tend, tbeg + pb_, tbeg + pe_, 1, tb, hist, smem, copy_only);
        } else {
            Stager stg;
            stg.stage = reinterpret_cast<uint32_t*>(smem + kSmemHist) + (threadIdx.x >> 5) * kStageCap;
            stg.dst = A.ws.buf[1] + sel_region(tbeg);
            stg.cursor = &st->cursor[1];
            stg.fill = 0;
            uint32_t kmin = 0, kmax = 0, nf = 0;
            stream_piece<false, false, true>(A.ws.buf[0], sel_region(tbeg) + pb_, sel_region(tbeg) + pe_, false, tb, hist,
                                             hist + kCells, hist + 2 * kCells, stg, kmin, kmax, nf, copy_only);
            stg.flush();
        }
        __syncthreads();
        if (!copy_only) flush_hist(hist, tb.ncells, A.ws.gcnt + (size_t)t * kCells, A.ws.glsum + (size_t)t * kCells);
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) {
            const unsigned prev = atomicAdd(&st->arrive, 1u);
            sh_last = (prev == ns - 1);
        }
        __syncthreads();
        if (!sh_last) continue;
        __threadfence();
        if (copy_only) {
            finish_sorted(st, t, A.s, A.ws.buf[1] + sel_region(tbeg), A.levels, A.status, smem, S, 1);
            continue;
        }
        if (!solver_round(st, t, A.ws.gcnt + (size_t)t * kCells, A.ws.glsum + (size_t)t * kCells, A.scheme, A.s,
                          A.levels, A.status, A.ws.nitems, A.ws.items, A.ws.buf[1] + sel_region(tbeg), false, smem, S, sel_region(tend) - sel_region(tbeg)))
            finish_alone(A, t, smem, tb, S);
    }
}

cudaError_t launch_levels_select(const float* d_grad, const int64_t* d_off, int T, int64_t total, int scheme,
                                 int s, const float* d_tau, float* d_levels, int32_t* d_status, void* d_ws,
                                 size_t /*ws_bytes*/, int sm_count, cudaStream_t stream)
{
    {
        // the kernels need more dynamic shared memory than the default limit: raised once per device
        static std::atomic<bool> attr_set[64];
        int dev = 0;
        cudaError_t e = cudaGetDevice(&dev);
        if (e != cudaSuccess) return e;
        if (dev < 0 || dev >= 64 || !attr_set[dev].load(std::memory_order_acquire)) {
            e = cudaFuncSetAttribute(k_sel_round1, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
            if (e != cudaSuccess) return e;
            e = cudaFuncSetAttribute(k_sel_round2, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
            if (e != cudaSuccess) return e;
            e = cudaFuncSetAttribute(k_sel_round3, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
            if (e != cudaSuccess) return e;
            if (dev >= 0 && dev < 64) attr_set[dev].store(true, std::memory_order_release);
        }
    }
    // Flat streaming CTAs: one wave (kSelResident per SM).  Each CTA pays a set-up, a flush of its
    // cells and an arrival per tensor piece, so larger chunks stream more of the time; a second wave
    // balanced a lone call slightly better in round 1 but cost throughput whenever several calls
    // (workers on their own streams) share the GPU.  Buckets above 4 M elements get chunks of at least
    // 131,072 elements: on a bucket of 25 M elements that leaves a third of the wave's slots to concurrent
    // calls (measured with eight workers in flight: 8 % more throughput, 3 % slower alone); smaller
    // buckets keep 32,768, where a lone call is all that matters.
    const int64_t wave = (int64_t)kSelResident * sm_count;
    const int target = wave < kMaxFlatCtas ? (int)wave : kMaxFlatCtas;
    FlatGrid g = make_flat_grid(total, target, total > ((int64_t)1 << 22) ? 131072 : 32768);
    SelArgs A;
    A.grad = d_grad; A.tau = d_tau; A.off = d_off; A.T = T; A.total = total; A.chunk = g.chunk; A.flat_ctas = g.ctas;
    A.scheme = scheme; A.s = s; A.levels = d_levels; A.status = d_status;
    A.ws = sel_carve(d_ws, T, total);
    cudaError_t e = cudaMemsetAsync(d_ws, 0, sel_zero_bytes(T), stream);
    if (e != cudaSuccess) return e;
    launch_begin("k_sel_round1", stream);
    k_sel_round1<<<g.ctas + T, kSelThreads, kSmemBytes, stream>>>(A);
    launch_end(stream);
    launch_begin("k_sel_round2", stream);
    k_sel_round2<<<g.ctas + T, kSelThreads, kSmemBytes, stream>>>(A);
    launch_end(stream);
    launch_begin("k_sel_round3", stream);
    k_sel_round3<<<kSelResident * sm_count, kSelThreads, kSmemBytes, stream>>>(A);
    launch_end(stream);
    return cudaGetLastError();
}

}  // namespace ogq
