// Fixed-length bucket mode: the gradient is cut into buckets of d elements and every bucket is
// quantized on its own (the setting of all the paper's experiments, d = 128 ... 32768).
//
// One CTA takes one bucket at a time and does the whole path on it from a single read: the bucket's
// keys are sorted in shared memory, the levels follow from the definitions applied to the sorted
// keys (Algorithm 1 with Q* for ORQ, optionally followed by refinement sweeps; the sign change of g
// for BinGrad-pb; the conditional means for BinGrad-b), then the bucket is read once more (from L2)
// to be quantized and packed.  Results are those of the per-tensor entry points called with tensor
// offsets j * d: same level definitions, same Philox counters (tensor index = bucket index), same
// packed layout.
#include <math.h>

#include <atomic>

#include "ogq_common.cuh"
#include "ogq_internal.h"
#include "ogq_quant.cuh"

namespace ogq {

constexpr int kBktMaxD = 32768;        // longest bucket (its keys take 128 KB of shared memory)
constexpr int kBktPrefixMaxD = 4096;   // buckets up to this length also keep fp64 prefix sums of the sorted values
constexpr int kBktMaxThreads = 1024;
static_assert(kBktMaxD * sizeof(uint32_t) <= 160 * 1024, "the keys of the longest bucket must fit the shared-memory limit set at launch");
constexpr int kBktMaxWarps = kBktMaxThreads / 32;

struct BktArgs {
    const float* grad;
    int64_t total;
    int d, nb, scheme, s, iters;  // iters: refinement sweeps (ORQ) or Lloyd updates (BinGrad-b)
    float clip_c;                 // > 0: clip every bucket to c times its standard deviation first
    uint32_t stream_id;
    float* levels;
    float* thresh;
    int32_t* status;
    uint32_t* packed;
    int64_t words_per_bucket;
};

// Ascending bitonic sort of P = KPT * blockDim.x keys held in registers, KPT per thread: thread t
// owns positions t * KPT ... t * KPT + KPT - 1 of the sequence.  The network is the variant whose
// merges start with a "flip" (position i against i ^ (k - 1)) followed by halvings (i against
// i ^ j): every compare-exchange then puts the smaller key at the lower position, so no direction
// has to be computed.  Distances inside a thread's registers cost a min and a max; distances up to
// 16 * KPT cross lanes by shuffle; only the larger ones (a few stages, none when the CTA is one
// warp) go through shared memory with a barrier.  xch: P words of shared memory.
__device__ __forceinline__ void bkt_cmpx(uint32_t& a, uint32_t& b)
{
    const uint32_t lo = min(a, b), hi = max(a, b);
    a = lo;
    b = hi;
}

// Exchange with thread t ^ m: this thread's register e against the partner's register e (REV false)
// or KPT - 1 - e (REV true); the thread on the lower side keeps the smaller keys.
template <int KPT, bool REV>
__device__ __forceinline__ void bkt_cross(uint32_t (&r)[KPT], uint32_t* xch, int m, bool keep_min)
{
    const int t = threadIdx.x, nt = blockDim.x;
    uint32_t o[KPT];
    if (m < 32) {
#pragma unroll
        for (int e = 0; e < KPT; ++e) o[e] = __shfl_xor_sync(0xffffffffu, r[REV ? KPT - 1 - e : e], m);
    } else {
        __syncthreads();
#pragma unroll
        for (int e = 0; e < KPT; ++e) xch[e * nt + t] = r[e];
        __syncthreads();
#pragma unroll
        for (int e = 0; e < KPT; ++e) o[e] = xch[(REV ? KPT - 1 - e : e) * nt + (t ^ m)];
    }
    // the side of the exchange decides once whether this thread keeps minima or maxima: one predicated
    // instruction pair per key instead of a minimum, a maximum and a select
#pragma unroll
    for (int e = 0; e < KPT; ++e)
        asm("{ .reg .pred p; setp.ne.u32 p, %2, 0; @p min.u32 %0, %0, %1; @!p max.u32 %0, %0, %1; }"
            : "+r"(r[e]) : "r"(o[e]), "r"((uint32_t)keep_min));
}

// The stages of a merge that stay inside a warp, written out at compile time (no run-time dispatch on
// the merge size, so the registers never have to be moved between code paths): halvings at lane
// distances 16 ... 1 (FROM_LANES) or only those inside a thread's registers.
template <int KPT, bool FROM_LANES>
__device__ __forceinline__ void bkt_merge_tail(uint32_t (&r)[KPT], uint32_t* xch)
{
    const int t = threadIdx.x;
    if constexpr (FROM_LANES) {
#pragma unroll
        for (int m = 16; m >= 1; m >>= 1) bkt_cross<KPT, false>(r, xch, m, (t & m) == 0);
    }
#pragma unroll
    for (int j = KPT / 2; j >= 1; j >>= 1) {
#pragma unroll
        for (int e = 0; e < KPT; ++e)
            if ((e & j) == 0) bkt_cmpx(r[e], r[e | j]);
    }
}

// Sorts the 32 * KPT keys of every warp ascending: the whole network unrolled at compile time.
template <int KPT>
__device__ __forceinline__ void bkt_sort_warp(uint32_t (&r)[KPT], uint32_t* xch)
{
    const int t = threadIdx.x;
#pragma unroll
    for (int k = 2; k <= 32 * KPT; k <<= 1) {
        if (k <= KPT) {
#pragma unroll
            for (int e = 0; e < KPT; ++e)
                if ((e & (k >> 1)) == 0) bkt_cmpx(r[e], r[e ^ (k - 1)]);
#pragma unroll
            for (int j = k >> 2; j >= 1; j >>= 1) {
#pragma unroll
                for (int e = 0; e < KPT; ++e)
                    if ((e & j) == 0) bkt_cmpx(r[e], r[e | j]);
            }
        } else {
            const int m = k / KPT - 1;  // flip: lane t against t ^ m, registers reversed
            bkt_cross<KPT, true>(r, xch, m, (t & ((m + 1) >> 1)) == 0);
#pragma unroll
            for (int j = k >> 2; j >= KPT; j >>= 1) bkt_cross<KPT, false>(r, xch, j / KPT, (t & (j / KPT)) == 0);
            bkt_merge_tail<KPT, false>(r, xch);
        }
    }
}

template <int KPT>
__device__ __forceinline__ void bkt_sort_regs(uint32_t (&r)[KPT], uint32_t* xch, int P)
{
    const int t = threadIdx.x;
    bkt_sort_warp<KPT>(r, xch);
    // merges across warps: the flip and the halvings at 32 threads or more go through shared memory
    for (int k = 64 * KPT; k <= P; k <<= 1) {
        const int m = k / KPT - 1;
        bkt_cross<KPT, true>(r, xch, m, (t & ((m + 1) >> 1)) == 0);
        for (int j = k >> 2; j >= 32 * KPT; j >>= 1) bkt_cross<KPT, false>(r, xch, j / KPT, (t & (j / KPT)) == 0);
        bkt_merge_tail<KPT, true>(r, xch);
    }
}

__device__ __forceinline__ int bkt_lower(const uint32_t* a, int n, uint32_t k)
{
    int lo = 0, hi = n;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (a[mid] < k) lo = mid + 1; else hi = mid; }
    return lo;
}

__device__ __forceinline__ int bkt_upper(const uint32_t* a, int n, uint32_t k)
{
    int lo = 0, hi = n;
    while (lo < hi) { const int mid = (lo + hi) >> 1; if (a[mid] <= k) lo = mid + 1; else hi = mid; }
    return lo;
}

// Sum of a double over the CTA, valid in every thread.  scratch: kBktMaxWarps + 1 doubles.
__device__ __forceinline__ double bkt_block_sum(double x, double* scratch)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = x;
    __syncthreads();
    if (threadIdx.x == 0) {
        double r = 0.0;
        const int nw = (blockDim.x + 31) >> 5;
        for (int i = 0; i < nw; ++i) r += scratch[i];
        scratch[kBktMaxWarps] = r;
    }
    __syncthreads();
    return scratch[kBktMaxWarps];
}

// Q*(L, R) on sorted keys with prefix sums (pre[i] = sum of the values of keys[0..i)): called by one
// thread.  With T = sum_{L <= v <= R} (v - L) / (R - L) the result is the (floor(T) + 1)-th largest
// element of the segment.
__device__ __forceinline__ uint32_t bkt_qstar_prefix(const uint32_t* keys, const double* pre, int n, uint32_t kl,
                                                     uint32_t kr)
{
    if (kr <= kl) return kl;
    const int i0 = bkt_lower(keys, n, kl), i1 = bkt_upper(keys, n, kr);
    const double Lv = (double)key_to_float(kl), Rv = (double)key_to_float(kr);
    const int m = i1 - i0;
    const double A = (pre[i1] - pre[i0]) - Lv * (double)m;
    long long k = (long long)floor(A / (Rv - Lv));
    if (k < 0) k = 0;
    if (k > m - 1) k = m - 1;
    return keys[i1 - 1 - (int)k];
}

// One depth of Algorithm 1 for a bucket held by ONE warp, called by all its lanes with the sorted keys
// still in their registers.  The positions of the brackets come from counting (a compare per key and
// one warp reduction per bracket) instead of binary searches in shared memory, whose dependent loads
// are what a lone lane spends its time on; the levels of the depth are counted one after the other,
// then lane i finishes level i (the fp64 division of every level of the depth at the same time).
// Positions past n hold the largest key, which no bracket reaches.  lvkey: the level keys in shared
// memory, the brackets of this depth already in place.
template <int KPT>
__device__ __forceinline__ void bkt_depth_warp(const uint32_t (&r)[KPT], const uint32_t* keys, const double* pre,
                                               uint32_t* lvkey, int s, int stride, int lane)
{
    int my_i0 = 0, my_i1 = 0, my_q = -1;
    uint32_t my_kl = 0u, my_kr = 0u;
    int idx = 0;
    for (int q = stride; q < s - 1; q += 2 * stride, ++idx) {
        const uint32_t kl = lvkey[q - stride], kr = lvkey[q + stride];
        int i0 = 0, i1 = 0;
        if (kr > kl) {
            uint32_t below = 0u, upto = 0u;
#pragma unroll
            for (int e = 0; e < KPT; ++e) {
                below += (r[e] < kl) ? 1u : 0u;
                upto += (r[e] <= kr) ? 1u : 0u;
            }
            i0 = (int)__reduce_add_sync(0xffffffffu, below);
            i1 = (int)__reduce_add_sync(0xffffffffu, upto);
        }
        if (lane == idx) { my_i0 = i0; my_i1 = i1; my_kl = kl; my_kr = kr; my_q = q; }
    }
    __syncwarp();
    if (my_q >= 0) {
        uint32_t res = my_kl;
        if (my_kr > my_kl) {
            const double Lv = (double)key_to_float(my_kl), Rv = (double)key_to_float(my_kr);
            const int m = my_i1 - my_i0;
            const double A = (pre[my_i1] - pre[my_i0]) - Lv * (double)m;
            long long k = (long long)floor(A / (Rv - Lv));
            if (k < 0) k = 0;
            if (k > m - 1) k = m - 1;
            res = keys[my_i1 - 1 - (int)k];
        }
        lvkey[my_q] = res;
    }
    __syncwarp();
}

// The same without prefix sums: called by every thread of the CTA, the segment's sum is a block sum.
__device__ __forceinline__ uint32_t bkt_qstar_block(const uint32_t* keys, int n, uint32_t kl, uint32_t kr,
                                                    double* scratch)
{
    if (kr <= kl) return kl;
    const int i0 = bkt_lower(keys, n, kl), i1 = bkt_upper(keys, n, kr);
    const double Lv = (double)key_to_float(kl), Rv = (double)key_to_float(kr);
    double a = 0.0;
    for (int i = i0 + threadIdx.x; i < i1; i += blockDim.x) a += (double)key_to_float(keys[i]) - Lv;
    a = bkt_block_sum(a, scratch);
    const int m = i1 - i0;
    long long k = (long long)floor(a / (Rv - Lv));
    if (k < 0) k = 0;
    if (k > m - 1) k = m - 1;
    return keys[i1 - 1 - (int)k];
}

template <int BITS, int KPT>
__global__ void __launch_bounds__(kBktMaxThreads)
k_bucket_encode(BktArgs A, const __grid_constant__ PhiloxKeys pk)
{
    extern __shared__ __align__(16) unsigned char smem[];
    __shared__ double sh_d[kBktMaxWarps + 1];
    __shared__ uint32_t sh_lvkey[kMaxLevels];
    __shared__ float sh_lv[kMaxLevels];
    __shared__ float sh_w[kMaxLevels];
    __shared__ float2 sh_tab[kMaxLevels];
    __shared__ uint32_t sh_words[kBktMaxWarps][(BITS == 3 || BITS == 5) ? 4 * BITS : 1];
    __shared__ int sh_flag, sh_changed;
    __shared__ float sh_b0;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (blockDim.x + 31) >> 5;
    const int s = A.s;
    const bool orq = A.scheme == OGQ_ORQ, pbs = A.scheme == OGQ_BINGRAD_PB;
    uint32_t* keys = reinterpret_cast<uint32_t*>(smem);
    const int Pmax = KPT * blockDim.x;
    double* pre = (A.d <= kBktPrefixMaxD) ? reinterpret_cast<double*>(smem + (size_t)Pmax * sizeof(uint32_t)) : nullptr;
    if ((BITS == 3 || BITS == 5) && lane < 4 * BITS) sh_words[warp][lane] = 0u;

    for (int j = blockIdx.x; j < A.nb; j += gridDim.x) {
        const int64_t base_i = (int64_t)j * A.d;
        const int n = (int)((A.total - base_i < (int64_t)A.d) ? A.total - base_i : (int64_t)A.d);
        const float* src = A.grad + base_i;
        int stbits = 0;
        __syncthreads();
        if (threadIdx.x == 0) { sh_flag = 0; sh_b0 = 0.f; }
        __syncthreads();
        // The bucket's values, KPT per thread (element e * blockDim.x + threadIdx.x: coalesced), all loads
        // issued before the first use; positions past n read element 0 and are not used.  Every later
        // pass over the bucket but the quantizer's runs from these registers.
        float rawv[KPT];
#pragma unroll
        for (int e = 0; e < KPT; ++e) {
            const int i = e * blockDim.x + threadIdx.x;
            rawv[e] = __ldg(src + (i < n ? i : 0));
        }
        // clipping threshold of this bucket: c times the standard deviation about the mean (none: +Inf)
        float tau = __int_as_float(0x7f800000);
        if (A.clip_c > 0.f) {
            const double v0 = (double)__ldg(src);
            double s1 = 0.0, s2 = 0.0;
#pragma unroll
            for (int e = 0; e < KPT; ++e) {
                if (e * (int)blockDim.x + (int)threadIdx.x < n) {
                    const double dv = (double)rawv[e] - v0;
                    s1 += dv;
                    s2 += dv * dv;
                }
            }
            s1 = bkt_block_sum(s1, sh_d);
            s2 = bkt_block_sum(s2, sh_d);
            double var = (s2 - s1 * s1 / (double)n) / (double)n;
            if (!(var > 0.0)) var = 0.0;  // also a non-finite bucket: everything clips to 0
            tau = (float)((double)A.clip_c * sqrt(var));
        }

        if (A.scheme == OGQ_BINGRAD_B) {
            // ---- BinGrad-b: b_0 = mean, b_{-1}, b_1 = conditional means, optional Lloyd updates
            double sum = 0.0;
            int bad = 0;
#pragma unroll
            for (int e = 0; e < KPT; ++e) {
                if (e * (int)blockDim.x + (int)threadIdx.x < n) {
                    const float raw = rawv[e];
                    bad |= ((__float_as_uint(raw) & 0x7f800000u) == 0x7f800000u);
                    sum += (double)copysignf(fminf(fabsf(raw), tau), raw);
                }
            }
            sum = bkt_block_sum(sum, sh_d);
            if (__syncthreads_or(bad)) stbits |= OGQ_ST_NONFINITE;
            float b0 = (float)(sum / (double)n);
            long long prev_lo = -1;
            float l_lo = 0.f, l_hi = 0.f;
            for (int it = 0;; ++it) {
                double s_lo = 0.0, s_hi = 0.0, c_lo = 0.0;
#pragma unroll
                for (int e = 0; e < KPT; ++e) {
                    if (e * (int)blockDim.x + (int)threadIdx.x < n) {
                        const float raw = rawv[e];
                        const float v = copysignf(fminf(fabsf(raw), tau), raw);
                        const bool below = v < b0;
                        s_lo += below ? (double)v : 0.0;
                        s_hi += below ? 0.0 : (double)v;
                        c_lo += below ? 1.0 : 0.0;
                    }
                }
                s_lo = bkt_block_sum(s_lo, sh_d);
                s_hi = bkt_block_sum(s_hi, sh_d);
                c_lo = bkt_block_sum(c_lo, sh_d);
                const long long n_lo = (long long)c_lo, n_hi = (long long)n - n_lo;
                if (n_lo == 0 || n_hi == 0) {
                    const double m = (n_lo == 0) ? s_hi / (double)n_hi : s_lo / (double)n_lo;
                    l_lo = l_hi = (float)m;
                    stbits |= OGQ_ST_CONSTANT;
                    break;
                }
                const double m_lo = s_lo / (double)n_lo, m_hi = s_hi / (double)n_hi;
                l_lo = (float)m_lo;
                l_hi = (float)m_hi;
                if (n_lo == prev_lo) break;
                if (it >= A.iters) {
                    if (A.iters > 0) stbits |= OGQ_ST_ITER_CAP;
                    break;
                }
                prev_lo = n_lo;
                b0 = (float)((m_lo + m_hi) * 0.5);
            }
            if (threadIdx.x == 0) {
                A.levels[2 * (int64_t)j] = l_lo;
                A.levels[2 * (int64_t)j + 1] = l_hi;
                A.thresh[j] = b0;
                A.status[j] = stbits;
                sh_b0 = b0;
            }
            __syncthreads();
        } else {
            // ---- sorted keys of the bucket (magnitudes for BinGrad-pb): KPT keys per thread, loaded
            // coalesced (the arrangement before the sort does not matter), sorted in registers, then
            // written to shared memory in order.  P = KPT * blockDim.x >= d; positions past n hold
            // the largest key.
            const int P = KPT * blockDim.x;
            uint32_t r[KPT];
            int bad = 0;
#pragma unroll
            for (int e = 0; e < KPT; ++e) {
                const int i = e * blockDim.x + threadIdx.x;
                uint32_t key = 0xffffffffu;
                if (i < n) {
                    const float raw = rawv[e];
                    bad |= ((__float_as_uint(raw) & 0x7f800000u) == 0x7f800000u);
                    uint32_t bits = __float_as_uint(copysignf(fminf(fabsf(raw), tau), raw));
                    if (pbs) key = bits | 0x80000000u;
                    else {
                        if (bits == 0x80000000u) bits = 0u;
                        key = (bits & 0x80000000u) ? ~bits : (bits | 0x80000000u);
                    }
                }
                r[e] = key;
            }
            const bool nonfinite = __syncthreads_or(bad) != 0;
            const int nl = pbs ? 2 : s;
            if (nonfinite) {
                stbits |= OGQ_ST_NONFINITE;
                if (threadIdx.x < nl) sh_lv[threadIdx.x] = 0.f;
            } else {
                bkt_sort_regs<KPT>(r, keys, P);
                __syncthreads();
                static_assert(KPT % 4 == 0, "a thread's keys are stored as 128-bit words");
#pragma unroll
                for (int e = 0; e < KPT; e += 4)
                    *reinterpret_cast<uint4*>(keys + threadIdx.x * KPT + e) = make_uint4(r[e], r[e + 1], r[e + 2], r[e + 3]);
                __syncthreads();
                if (pre != nullptr) {
                    // fp64 prefix sums of the sorted values, from the registers that hold them (thread t
                    // owns positions t * KPT ...): local sums, one scan over the threads, running sums out
                    const int p0 = threadIdx.x * KPT;
                    double ls = 0.0;
#pragma unroll
                    for (int e = 0; e < KPT; ++e)
                        if (p0 + e < n) ls += (double)key_to_float(r[e]);
                    // exclusive scan of ls in thread order
                    double inc = ls;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const double nbv = __shfl_up_sync(0xffffffffu, inc, o);
                        if (lane >= o) inc = nbv + inc;
                    }
                    double wbase = 0.0;
                    if (nwarps > 1) {
                        __syncthreads();
                        if (lane == 31) sh_d[warp] = inc;
                        __syncthreads();
                        for (int w = 0; w < warp; ++w) wbase += sh_d[w];
                    }
                    double run = wbase + (inc - ls);
#pragma unroll
                    for (int e = 0; e < KPT; ++e)
                        if (p0 + e < n) { pre[p0 + e] = run; run += (double)key_to_float(r[e]); }
                    if (n > p0 && n <= p0 + KPT) pre[n] = run;
                    if (n == 0 && threadIdx.x == 0) pre[0] = 0.0;
                    __syncthreads();
                }
                if (orq) {
                    if (keys[0] == keys[n - 1]) stbits |= OGQ_ST_CONSTANT;
                    if (threadIdx.x < s) sh_lvkey[threadIdx.x] = (threadIdx.x == s - 1) ? keys[n - 1] : keys[0];
                    __syncthreads();
                    // Algorithm 1: a level after its two brackets, the levels of one depth side by side
                    for (int stride = (s - 1) >> 1; stride >= 1; stride >>= 1) {
                        if (pre != nullptr && nwarps == 1) {
                            // one warp holds the bucket
                            bkt_depth_warp<KPT>(r, keys, pre, sh_lvkey, s, stride, lane);
                        } else if (pre != nullptr) {
                            const int q = threadIdx.x;
                            uint32_t res = 0u;
                            const bool mine = q < s - 1 && q >= stride && ((q - stride) % (2 * stride)) == 0;
                            if (mine) res = bkt_qstar_prefix(keys, pre, n, sh_lvkey[q - stride], sh_lvkey[q + stride]);
                            __syncthreads();
                            if (mine) sh_lvkey[q] = res;
                            __syncthreads();
                        } else {
                            for (int q = stride; q < s - 1; q += 2 * stride) {
                                const uint32_t res = bkt_qstar_block(keys, n, sh_lvkey[q - stride], sh_lvkey[q + stride], sh_d);
                                __syncthreads();
                                if (threadIdx.x == 0) sh_lvkey[q] = res;
                                __syncthreads();
                            }
                        }
                    }
                    // refinement sweeps: every interior level again from its two current neighbours, ascending
                    for (int it = 0; it < A.iters; ++it) {
                        if (threadIdx.x == 0) sh_changed = 0;
                        __syncthreads();
                        if (pre != nullptr) {
                            if (threadIdx.x == 0) {
                                for (int q = 1; q < s - 1; ++q) {
                                    const uint32_t res = bkt_qstar_prefix(keys, pre, n, sh_lvkey[q - 1], sh_lvkey[q + 1]);
                                    if (res != sh_lvkey[q]) { sh_lvkey[q] = res; sh_changed = 1; }
                                }
                            }
                            __syncthreads();
                        } else {
                            for (int q = 1; q < s - 1; ++q) {
                                const uint32_t res = bkt_qstar_block(keys, n, sh_lvkey[q - 1], sh_lvkey[q + 1], sh_d);
                                __syncthreads();
                                if (threadIdx.x == 0 && res != sh_lvkey[q]) { sh_lvkey[q] = res; sh_changed = 1; }
                                __syncthreads();
                            }
                        }
                        if (!sh_changed) break;
                    }
                    if (threadIdx.x < s) sh_lv[threadIdx.x] = key_to_float(sh_lvkey[threadIdx.x]);
                } else {
                    // BinGrad-pb: the last sorted magnitude x_c with g(x_c) = x_c n - sum_{|v| >= x_c} |v| <= 0;
                    // the sign change lies in [x_c, next magnitude)
                    auto suffix = [&](int from) -> double {  // sum of the magnitudes keys[from..n)
                        if (pre != nullptr) return pre[n] - pre[from];
                        double a = 0.0;
                        for (int i = from + threadIdx.x; i < n; i += blockDim.x) a += (double)key_to_float(keys[i]);
                        return bkt_block_sum(a, sh_d);
                    };
                    const double tot = suffix(0);
                    float b1 = 0.f;
                    if (!(tot > 0.0)) {
                        stbits |= OGQ_ST_CONSTANT;
                    } else {
                        // g is non-decreasing along the sorted magnitudes: bisection on the index (all threads alike)
                        int lo = -1, hi = n;  // g(x_lo) <= 0 < g(x_hi)
                        while (hi - lo > 1) {
                            const int mid = (lo + hi) >> 1;
                            const int first = bkt_lower(keys, n, keys[mid]);
                            const double g = (double)key_to_float(keys[mid]) * (double)n - suffix(first);
                            if (g <= 0.0) lo = mid; else hi = mid;
                        }
                        const int c = lo < 0 ? 0 : lo;
                        const double x = (double)key_to_float(keys[c]);
                        const int up = bkt_upper(keys, n, keys[c]);
                        const double stat_up = suffix(up) / (double)n;
                        b1 = (float)(stat_up > x ? stat_up : x);
                    }
                    if (threadIdx.x == 0) { sh_lv[0] = -b1; sh_lv[1] = b1; }
                }
            }
            __syncthreads();
            if (threadIdx.x < nl) {
                const float cur = sh_lv[threadIdx.x];
                const float prv = threadIdx.x > 0 ? sh_lv[threadIdx.x - 1] : cur;
                const float nxt = (int)threadIdx.x + 1 < nl ? sh_lv[threadIdx.x + 1] : cur;
                sh_w[threadIdx.x] = __fsub_rn(cur, prv);
                sh_tab[threadIdx.x] = make_float2(cur, __fsub_rn(nxt, cur));
                A.levels[(int64_t)j * nl + threadIdx.x] = cur;
            }
            if (threadIdx.x == 0) A.status[j] = stbits;
            __syncthreads();
        }

        // ---- quantize + pack: the bucket is read again (it is in L2), 128 elements per warp and trip
        uint32_t* out = A.packed + (int64_t)j * A.words_per_bucket;
        const int64_t region = ((int64_t)n * BITS + 31) / 32;
        const int64_t region4 = (region + 3) / 4 * 4;
        const bool threshold = A.scheme == OGQ_BINGRAD_B;
        const float b0 = sh_b0;
        const int ngroups = (n + 127) >> 7, nfull = n >> 7;
        const int nl = (orq ? s : 2);
        constexpr bool kPow2 = (BITS == 1 || BITS == 2 || BITS == 4);
        constexpr int L = kPow2 ? 8 / BITS : 1;
        const uint32_t tabaddr = (uint32_t)__cvta_generic_to_shared(sh_tab);
        const uint32_t tab4 = tabaddr * (1u + (1u << BITS) + (1u << (2 * BITS)) + (1u << (3 * BITS)));
        float mid = 0.f;
        PhiloxHoist hz = {};
        if (!threshold) {
            mid = sh_tab[(BITS >= 2) ? (1 << (BITS - 2)) : 0].x;
            hz = philox_hoist(0u, (uint32_t)j, A.stream_id, pk);
        }
        uint32_t* wsm = sh_words[warp];
        const int obit = (lane * 4 * BITS) & 31, oword = (lane * 4 * BITS) >> 5;
        // (the next group's values are loaded before the current group is worked on)
        const float4* src4 = reinterpret_cast<const float4*>(src) + lane;
        float4 vnext = make_float4(0.f, 0.f, 0.f, 0.f);
        if (warp < nfull) vnext = __ldg(src4 + ((int64_t)warp << 5));
        for (int g = warp; g < ngroups; g += nwarps) {
            uint32_t bits4;
            float4 v = vnext;
            if (g + nwarps < nfull) vnext = __ldg(src4 + ((int64_t)(g + nwarps) << 5));
            if (g < nfull) {
                v.x = copysignf(fminf(fabsf(v.x), tau), v.x);  // clipping (tau = +Inf: none)
                v.y = copysignf(fminf(fabsf(v.y), tau), v.y);
                v.z = copysignf(fminf(fabsf(v.z), tau), v.z);
                v.w = copysignf(fminf(fabsf(v.w), tau), v.w);
                if (threshold) {
                    bits4 = ((v.x >= b0) ? 1u : 0u) | ((v.y >= b0) ? 2u : 0u) | ((v.z >= b0) ? 4u : 0u) |
                            ((v.w >= b0) ? 8u : 0u);
                } else {
                    const uint4 r = philox4x32_10_tail(((uint32_t)g << 5) + (uint32_t)lane, hz, pk);
                    const uint32_t a0 = entry_after_rounding<BITS>(v.x, r.x, tabaddr, mid),
                                   a1 = entry_after_rounding<BITS>(v.y, r.y, tabaddr, mid),
                                   a2 = entry_after_rounding<BITS>(v.z, r.z, tabaddr, mid),
                                   a3 = entry_after_rounding<BITS>(v.w, r.w, tabaddr, mid);
                    bits4 = (a0 + (a1 << BITS) + (a2 << (2 * BITS)) + (a3 << (3 * BITS)) - tab4) >> 3;
                }
            } else {
                // the ragged end of the last bucket: element by element
                const int i0 = (g << 7) + 4 * lane;
                uint32_t c[4] = {0u, 0u, 0u, 0u};
                uint4 r = make_uint4(0u, 0u, 0u, 0u);
                if (!threshold) r = philox4x32_10((uint32_t)(i0 >> 2), 0u, (uint32_t)j, A.stream_id, pk);
                const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    if (i0 + e < n) {
                        const float raw = __ldg(src + i0 + e);
                        const float x = copysignf(fminf(fabsf(raw), tau), raw);
                        if (threshold) {
                            c[e] = (x >= b0) ? 1u : 0u;
                        } else {
                            int idx = 0;
                            for (int step = (BITS >= 2) ? (1 << (BITS - 2)) : 0; step >= 1; step >>= 1)
                                if (sh_lv[idx + step] <= x) idx += step;
                            const float dd = __fsub_rn(x, sh_lv[idx]);
                            const float lhs = __fmul_rn((float)(rw[e] >> 8), sh_w[idx + 1]);
                            const float rhs = __fmul_rn(dd, 16777216.0f);
                            c[e] = (uint32_t)idx + ((lhs < rhs) ? 1u : 0u);
                        }
                    }
                }
                bits4 = c[0] | (c[1] << BITS) | (c[2] << (2 * BITS)) | (c[3] << (3 * BITS));
            }
            if constexpr (kPow2) {
                const uint32_t word = assemble_words<BITS>(bits4, lane);
                if ((lane & (L - 1)) == 0) {
                    const int64_t widx = (int64_t)g * (4 * BITS) + lane / L;
                    if (widx < region4) out[widx] = word;
                }
            } else {
                atomicOr(wsm + oword, bits4 << obit);
                if (obit + 4 * BITS > 32) atomicOr(wsm + oword + 1, bits4 >> (32 - obit));
                __syncwarp();
                if (lane < 4 * BITS) {
                    const uint32_t word = atomicExch(wsm + lane, 0u);
                    const int64_t widx = (int64_t)g * (4 * BITS) + lane;
                    if (widx < region4) out[widx] = word;
                }
                __syncwarp();
            }
        }
        (void)nl;
    }
}

// Server step for fixed-length buckets: out[i] = scale * sum_k levels_k[i / d][code_k[i]].  Because d is
// a multiple of 128, the packed codes of consecutive buckets form one contiguous bit stream (only the
// last, shorter bucket is padded), so a warp takes 128 consecutive elements of the flat gradient at a
// time and only has to fetch the level rows of the bucket they lie in.  Same additions in the same
// (worker) order as ogq_unpack_sum with offsets j * d.
constexpr int kDecWorkers = 8;  // workers per batch: their level rows and packed words are loaded before any is used

template <int BITS>
__global__ void __launch_bounds__(kThreads)
k_bucket_decode_sum(const uint32_t* const* __restrict__ packed_k, const float* const* __restrict__ levels_k, int K,
                    int64_t total, int d, int s, int64_t total_words, float scale, float* __restrict__ outp)
{
    __shared__ float sh_lv[kWarps][kDecWorkers][kMaxLevels];
    __shared__ const uint32_t* sh_pk[kMaxWorkers];
    __shared__ const float* sh_lp[kMaxWorkers];
    for (int k = threadIdx.x; k < K; k += kThreads) { sh_pk[k] = packed_k[k]; sh_lp[k] = levels_k[k]; }
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr uint32_t kMask4 = (BITS * 4 >= 32) ? 0xffffffffu : ((1u << (BITS * 4)) - 1u);
    constexpr uint32_t kMask1 = (1u << BITS) - 1u;
    const int64_t ngroups = (total + 127) >> 7;
    for (int64_t g = (int64_t)blockIdx.x * kWarps + warp; g < ngroups; g += (int64_t)gridDim.x * kWarps) {
        const int64_t i0 = (g << 7) + 4 * lane;
        const int64_t j = (g << 7) / d;  // the bucket of this group
        const int64_t bit = i0 * BITS;
        const int64_t wi = bit >> 5;
        const int sh = (int)(bit & 31);
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int k0 = 0; k0 < K; k0 += kDecWorkers) {
            const int kn = (K - k0 < kDecWorkers) ? K - k0 : kDecWorkers;
            // all loads of the batch first (level rows: every code a BITS-bit field can hold gets an entry)
            float row[kDecWorkers];
            uint32_t w_lo[kDecWorkers], w_hi[kDecWorkers];
            const bool straddle = sh + 4 * BITS > 32;
#pragma unroll
            for (int u = 0; u < kDecWorkers; ++u) {
                row[u] = 0.f; w_lo[u] = 0u; w_hi[u] = 0u;
                if (u < kn) {
                    row[u] = __ldg(sh_lp[k0 + u] + j * s + (lane < s ? lane : s - 1));
                    if (i0 < total) {
                        const uint32_t* p = sh_pk[k0 + u];
                        if (wi < total_words) w_lo[u] = __ldg(p + wi);
                        if (straddle && wi + 1 < total_words) w_hi[u] = __ldg(p + wi + 1);
                    }
                }
            }
            __syncwarp();
#pragma unroll
            for (int u = 0; u < kDecWorkers; ++u)
                if (u < kn) sh_lv[warp][u][lane] = row[u];
            __syncwarp();
#pragma unroll
            for (int u = 0; u < kDecWorkers; ++u) {
                if (u < kn) {
                    const uint32_t bits4 = __funnelshift_r(w_lo[u], w_hi[u], sh) & kMask4;
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        acc[e] = __fadd_rn(acc[e], sh_lv[warp][u][(bits4 >> (e * BITS)) & kMask1]);
                }
            }
        }
        if (i0 + 3 < total) {
            *reinterpret_cast<float4*>(outp + i0) = make_float4(__fmul_rn(acc[0], scale), __fmul_rn(acc[1], scale),
                                                                __fmul_rn(acc[2], scale), __fmul_rn(acc[3], scale));
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (i0 + e < total) outp[i0 + e] = __fmul_rn(acc[e], scale);
        }
    }
}

cudaError_t launch_bucket_decode_sum(const uint32_t* const* d_packed_k, const float* const* d_levels_k, int K,
                                     int64_t total, int d, int s, float scale, float* d_out, int sm_count,
                                     cudaStream_t stream)
{
    const int bits = ogq_bits_for_levels(s);
    const int64_t nb = (total + d - 1) / d;
    const int64_t last = total - (nb - 1) * d;
    const int64_t total_words = (nb - 1) * ((int64_t)d * bits / 32) + ((last * bits + 31) / 32 + 3) / 4 * 4;
    const int64_t ngroups = (total + 127) >> 7;
    int64_t ctas = (ngroups + kWarps - 1) / kWarps;
    if (ctas > (int64_t)sm_count * 8) ctas = (int64_t)sm_count * 8;
    launch_begin("k_bucket_decode_sum", stream);
#define OGQ_LAUNCH_BD(B)                                                                                        \
    k_bucket_decode_sum<B><<<(int)ctas, kThreads, 0, stream>>>(d_packed_k, d_levels_k, K, total, d, s, total_words, \
                                                               scale, d_out)
    switch (bits) {
        case 1: OGQ_LAUNCH_BD(1); break;
        case 2: OGQ_LAUNCH_BD(2); break;
        case 3: OGQ_LAUNCH_BD(3); break;
        case 4: OGQ_LAUNCH_BD(4); break;
        case 5: OGQ_LAUNCH_BD(5); break;
        default: return cudaErrorInvalidValue;
    }
#undef OGQ_LAUNCH_BD
    launch_end(stream);
    return cudaGetLastError();
}

static int bkt_pow2(int d);

static size_t bkt_smem_bytes(int d)
{
    const size_t P = (size_t)bkt_pow2(d);
    size_t b = P * sizeof(uint32_t);
    if (d <= kBktPrefixMaxD) b += (P + 1) * sizeof(double);
    return (b + 15) / 16 * 16;
}

static int bkt_pow2(int d)
{
    int P = 128;
    while (P < d) P <<= 1;
    return P;
}

// keys per thread of the register sort: 4 for the shortest buckets, 32 for the longest, else 16
// (measured on 512- and 2048-element buckets: 16 keys per thread beat 8 and 4, although fewer
// warps are resident: the stages that stay in registers are the cheapest)
static int bkt_kpt(int d)
{
    const int P = bkt_pow2(d);
    return P <= 256 ? 4 : (P <= 16384 ? 16 : 32);
}

template <int BITS, int KPT>
static cudaError_t bkt_launch(const BktArgs& A, const PhiloxKeys& pk, int sm_count, cudaStream_t stream)
{
    const size_t smem = bkt_smem_bytes(A.d);
    const int threads = bkt_pow2(A.d) / KPT;
    static std::atomic<size_t> attr_bytes[64];  // dynamic shared-memory limit set so far, per device
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (smem > 48 * 1024 && (dev < 0 || dev >= 64 || attr_bytes[dev].load(std::memory_order_acquire) < smem)) {
        e = cudaFuncSetAttribute(k_bucket_encode<BITS, KPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(160 * 1024));
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_bytes[dev].store(160 * 1024, std::memory_order_release);
    }
    int per_sm = 1;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_bucket_encode<BITS, KPT>, threads, smem);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    int64_t ctas = (int64_t)per_sm * sm_count;
    if (ctas > A.nb) ctas = A.nb;
    launch_begin("k_bucket_encode", stream);
    k_bucket_encode<BITS, KPT><<<(int)ctas, threads, smem, stream>>>(A, pk);
    launch_end(stream);
    return cudaGetLastError();
}

template <int BITS>
static cudaError_t bkt_dispatch(const BktArgs& A, const PhiloxKeys& pk, int sm_count, cudaStream_t stream)
{
    switch (bkt_kpt(A.d)) {
        case 4: return bkt_launch<BITS, 4>(A, pk, sm_count, stream);
        case 16: return bkt_launch<BITS, 16>(A, pk, sm_count, stream);
        default: return bkt_launch<BITS, 32>(A, pk, sm_count, stream);
    }
}

cudaError_t launch_bucket_encode(const float* d_grad, int64_t total, int d, int scheme, int s, int iters,
                                 float clip_c, uint64_t seed, uint32_t stream_id, float* d_levels, float* d_thresh,
                                 int32_t* d_status, uint32_t* d_packed, int sm_count, cudaStream_t stream)
{
    BktArgs A;
    A.grad = d_grad; A.total = total; A.d = d; A.nb = (int)((total + d - 1) / d);
    A.scheme = scheme; A.s = s; A.iters = iters; A.clip_c = clip_c; A.stream_id = stream_id;
    A.levels = d_levels; A.thresh = d_thresh; A.status = d_status; A.packed = d_packed;
    const int bits = ogq_bits_for_levels(s);
    A.words_per_bucket = (int64_t)d * bits / 32;
    const PhiloxKeys pk = philox_round_keys((uint32_t)seed, (uint32_t)(seed >> 32));
    switch (bits) {
        case 1: return bkt_dispatch<1>(A, pk, sm_count, stream);
        case 2: return bkt_dispatch<2>(A, pk, sm_count, stream);
        case 3: return bkt_dispatch<3>(A, pk, sm_count, stream);
        case 4: return bkt_dispatch<4>(A, pk, sm_count, stream);
        case 5: return bkt_dispatch<5>(A, pk, sm_count, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace ogq
