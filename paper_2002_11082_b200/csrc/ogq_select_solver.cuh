// Scalar logic of the exact level solvers (ORQ and BinGrad-pb).
//
// The solvers never sort a large tensor.  Each round builds, for a set of
// disjoint key intervals that are known to contain every unresolved level, a
// histogram of aligned power-of-two key cells with an exact element count and
// an exact integer sum of the low key bits per cell.  Because an aligned cell
// lies inside one binade, the fp32 values in it are an affine function of the
// key, so the exact sum of the cell's values follows from those two integers.
// From the cell prefix counts and sums this file derives, for every level,
//   - its exact value, when the levels it depends on are exact and the cell
//     that holds its rank is a single key, or
//   - a conservative range of cells that must contain it,
// and turns the ranges into the (narrower, finer) intervals of the next round.
//
// Everything here is plain single-threaded code that compiles for the host as
// well, so it can be exercised without a GPU; the kernels call it from one
// thread after building the prefix arrays in parallel.
#pragma once

#include <math.h>
#include <stdint.h>
#include <string.h>

#ifdef __CUDACC__
#define OGQ_HD __host__ __device__ __forceinline__
#else
#define OGQ_HD inline
#endif

namespace ogq {

constexpr int kCells = 6144;   // histogram cells per tensor and round
constexpr int kMaxIv = 64;     // candidate intervals per tensor
constexpr int kMaxLv = 17;     // levels (s <= 17)
constexpr int kSlots = kCells + kMaxIv + 1;

// One candidate interval: keys [klo, khi], split into ncell aligned cells of 2^sh keys.
struct Interval {
    uint32_t klo, khi;
    int sh, ncell;
    int cellbase;       // index of its first cell in the per-tensor histogram
    int pad;
    long long cbefore;  // exact number of elements with key < klo
    double sbefore;     // exact sum of their values
};

// A level whose value is final, with the prefix statistics other solves need.
struct ExactLv {
    int exact;
    uint32_t key;
    long long c_lt, c_le;  // #{v < b}, #{v <= b}
    double s_lt, s_le;     // sums of those elements
};

OGQ_HD float sel_key_to_float(uint32_t k)
{
    uint32_t b = (k & 0x80000000u) ? (k & 0x7fffffffu) : ~k;
    float f;
#ifdef __CUDA_ARCH__
    f = __uint_as_float(b);
#else
    memcpy(&f, &b, 4);
#endif
    return f;
}

// Exact sum of the fp32 values of a cell [kbase, kbase + 2^sh) holding cnt elements whose
// low key bits (key - kbase) add up to lsum.  The cell lies in one binade and one sign.
OGQ_HD double sel_cell_sum(uint32_t kbase, int sh, unsigned long long cnt, unsigned long long lsum)
{
    if (cnt == 0) return 0.0;
    unsigned long long magsum;
    uint32_t mag0;
    double sign;
    if (kbase & 0x80000000u) {  // non-negative values: magnitude bits = key & 0x7fffffff
        mag0 = kbase & 0x7fffffffu;
        magsum = cnt * (unsigned long long)mag0 + lsum;
        sign = 1.0;
    } else {  // negative values: magnitude bits = 0x7fffffff - key
        mag0 = 0x7fffffffu - kbase;
        magsum = cnt * (unsigned long long)mag0 - lsum;
        mag0 -= (sh > 0) ? ((1u << sh) - 1u) : 0u;
        sign = -1.0;
    }
    const int e = (int)(mag0 >> 23);
    // value = mant * 2^(max(e,1) - 150); for e = 0 (subnormals) mant is the plain sum of magnitudes
    const unsigned long long mant = (e == 0) ? magsum : magsum - cnt * ((unsigned long long)(e - 1) << 23);
    const int ee = (e == 0) ? 1 : e;
#ifdef __CUDA_ARCH__
    const double scale = __hiloint2double((ee + 873) << 20, 0);  // 2^(ee - 150), exact
    return sign * (__ull2double_rn(mant) * scale);
#else
    return sign * ldexp((double)mant, ee - 150);
#endif
}

// Prefix arrays over "slots": interval j owns slots [slotbase[j], slotbase[j] + ncell_j]; slot
// slotbase[j] + c is the state before its cell c, the last one the state after its last cell.
struct SolverView {
    const uint8_t* slot_iv;  // optional: interval index of every slot (null: searched)
    const uint32_t* xkeys;  // explicit mode: cell c of the view holds the single key xkeys[c] (else null)
    const uint32_t* cpre;  // #{elements before the slot} (absolute)
    const double* spre;    // their sum
    const Interval* iv;
    int m;
    int slotbase[kMaxIv + 1];
    int nslots;
    long long n;
    double stot;
};

OGQ_HD void sel_init_slots(SolverView& v)
{
    int s = 0;
    for (int j = 0; j < v.m; ++j) {
        v.slotbase[j] = s;
        s += v.iv[j].ncell + 1;
    }
    v.slotbase[v.m] = s;
    v.nslots = s;
}

OGQ_HD int sel_interval_of_slot(const SolverView& v, int slot)
{
    if (v.slot_iv) return v.slot_iv[slot];
    int lo = 0, hi = v.m;  // last interval whose first slot is <= slot
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (v.slotbase[mid] <= slot) lo = mid; else hi = mid;
    }
    return lo;
}

OGQ_HD bool sel_is_end_slot(const SolverView& v, int slot)
{
    const int j = sel_interval_of_slot(v, slot);
    return slot == v.slotbase[j] + v.iv[j].ncell;
}

OGQ_HD uint32_t sel_slot_kbase(const SolverView& v, int slot)
{
    const int j = sel_interval_of_slot(v, slot);
    if (v.xkeys) return v.xkeys[slot - j];  // explicit cells are numbered without the end slots
    return v.iv[j].klo + ((uint32_t)(slot - v.slotbase[j]) << v.iv[j].sh);
}

OGQ_HD int sel_slot_shift(const SolverView& v, int slot)
{
    return v.xkeys ? 0 : v.iv[sel_interval_of_slot(v, slot)].sh;
}

OGQ_HD double sel_slot_vlo(const SolverView& v, int slot) { return (double)sel_key_to_float(sel_slot_kbase(v, slot)); }

OGQ_HD double sel_slot_vhi(const SolverView& v, int slot)
{
    const int sh = sel_slot_shift(v, slot);
    return (double)sel_key_to_float(sel_slot_kbase(v, slot) + ((sh > 0) ? ((1u << sh) - 1u) : 0u));
}

// First slot whose prefix count exceeds pos.
OGQ_HD int sel_upper_bound(const SolverView& v, long long pos)
{
    int lo = 0, hi = v.nslots;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if ((long long)v.cpre[mid] > pos) hi = mid; else lo = mid + 1;
    }
    return lo;
}

// Cell slot that holds the element of ascending rank pos (0-based).  If pos falls between two
// intervals, round_up selects the first cell after the gap, otherwise the last cell before it.
// Returns -1 when there is no such cell.
OGQ_HD int sel_locate(const SolverView& v, long long pos, bool round_up, bool* in_gap)
{
    const int u = sel_upper_bound(v, pos);
    *in_gap = false;
    if (u > 0 && !sel_is_end_slot(v, u - 1)) return u - 1;
    *in_gap = true;
    if (round_up) {
        // u is the first slot of an interval (or nslots)
        return (u < v.nslots) ? u : -1;
    }
    // u - 1 is an end slot: the last cell of that interval
    return (u >= 2) ? u - 2 : -1;
}

// Working description of a level during one solver pass.
struct LvInfo {
    int exact;
    uint32_t key;
    double val;
    long long c_lt, c_le;
    double s_lt, s_le;
    int sa, sb;       // cell-slot range when not exact
    double vlo, vhi;  // value bounds of that range
};

OGQ_HD void sel_make_exact_from_slot(const SolverView& v, int slot, LvInfo& o)
{
    o.exact = 1;
    o.key = sel_slot_kbase(v, slot);
    o.val = (double)sel_key_to_float(o.key);
    o.c_lt = v.cpre[slot];
    o.c_le = v.cpre[slot + 1];
    o.s_lt = v.spre[slot];
    o.s_le = v.spre[slot + 1];
    o.sa = o.sb = slot;
    o.vlo = o.vhi = o.val;
}

OGQ_HD void sel_make_range(const SolverView& v, int sa, int sb, LvInfo& o)
{
    o.exact = 0;
    o.sa = sa;
    o.sb = sb;
    o.vlo = sel_slot_vlo(v, sa);
    o.vhi = sel_slot_vhi(v, sb);
}

// Q*(L, R) on the current cells: exact when both brackets are exact and the target rank sits in
// a single-key cell, otherwise a conservative range of cells.  Returns false on an internal
// inconsistency (the range cannot be placed on any cell).
OGQ_HD bool sel_orq_solve(const SolverView& v, const LvInfo& L, const LvInfo& R, LvInfo& out)
{
    bool gap;
    if (L.exact && R.exact) {
        if (!(R.val > L.val)) {
            out = L;
            return true;
        }
        const long long nseg = R.c_le - L.c_lt;
        const double A = (R.s_le - L.s_lt) - L.val * (double)nseg;
        const double T = A / (R.val - L.val);
        long long k = (long long)floor(T);
        if (k < 0) k = 0;
        if (k > nseg - 1) k = nseg - 1;
        const long long pos = R.c_le - 1 - k;
        const int slot = sel_locate(v, pos, true, &gap);
        if (slot < 0 || gap) return false;
        if (sel_slot_shift(v, slot) == 0) sel_make_exact_from_slot(v, slot, out);
        else sel_make_range(v, slot, slot, out);
        return true;
    }
    // prefix state right after L's part and right before R's part
    const long long Cs = L.exact ? L.c_lt : (long long)v.cpre[L.sb + 1];
    const double Ss = L.exact ? L.s_lt : v.spre[L.sb + 1];
    const long long Ce = R.exact ? R.c_le : (long long)v.cpre[R.sa];
    const double Se = R.exact ? R.s_le : v.spre[R.sa];
    const double Llo = L.exact ? L.val : L.vlo, Lhi = L.exact ? L.val : L.vhi;
    const double Rlo = R.exact ? R.val : R.vlo, Rhi = R.exact ? R.val : R.vhi;
    const long long cntL = L.exact ? 0 : (long long)v.cpre[L.sb + 1] - (long long)v.cpre[L.sa];
    const long long cntR = R.exact ? 0 : (long long)v.cpre[R.sb + 1] - (long long)v.cpre[R.sa];
    const long long floor_pos = L.exact ? L.c_lt : (long long)v.cpre[L.sa];
    const long long ceil_pos = (R.exact ? R.c_le : (long long)v.cpre[R.sb + 1]) - 1;
    long long pos_lo = floor_pos, pos_hi = ceil_pos;
    // With M the elements strictly between L's cells and R's cells (count cntM, sum sumM, all of
    // them inside [Lhi, Rlo]), T = [t_L + (sumM - L cntM) + t_R] / (R - L), where t_L and t_R are
    // the contributions of the elements of L's and R's own cells.  f(L, R) = (sumM - L cntM)/(R - L)
    // decreases in L and in R, so its extremes are taken at matching corners, which stays tight
    // even when a bracket is only known to lie somewhere in a sparse stretch of cells.
    const double den_lo = Rlo - Lhi;
    const long long cntM = Ce - Cs;
    if (cntM >= 0 && den_lo > 0.0) {
        const double sumM = Se - Ss;
        double num_lo = sumM - Lhi * (double)cntM, num_hi = sumM - Llo * (double)cntM;
        if (num_lo < 0.0) num_lo = 0.0;
        if (num_hi < 0.0) num_hi = 0.0;
        const double mid_lo = num_lo / (Rhi - Lhi), mid_hi = num_hi / (Rlo - Llo);
        const double eps_l = (double)cntL * (Lhi - Llo) / (Rlo - Llo);
        const double eps_r = (double)cntR * (Rhi - Rlo) / (Rhi - Lhi);
        const double g_lo = (double)Ce - eps_l - mid_hi;
        const double g_hi = (double)Ce + eps_r - mid_lo;
        const double delta = 2.0 + 1e-9 * (double)v.n;
        const double p_lo = ceil(g_lo - delta) - 1.0, p_hi = ceil(g_hi + delta) - 1.0;
        if (p_lo > (double)pos_lo) pos_lo = (long long)p_lo;
        if (p_hi < (double)pos_hi) pos_hi = (long long)p_hi;
        if (pos_lo > ceil_pos) pos_lo = ceil_pos;
        if (pos_hi < floor_pos) pos_hi = floor_pos;
        if (pos_lo > pos_hi) pos_lo = pos_hi;
    }
    if (pos_lo < 0) pos_lo = 0;
    if (pos_hi > v.n - 1) pos_hi = v.n - 1;
    const int sa = sel_locate(v, pos_lo, true, &gap);
    const int sb = sel_locate(v, pos_hi, false, &gap);
    if (sa < 0 || sb < 0 || sa > sb) return false;
    sel_make_range(v, sa, sb, out);
    return true;
}

// One ORQ solver pass over all levels in the order of Algorithm 1 (a level after its two
// brackets).  lv[0] and lv[s-1] must be exact on entry.  ranges receives the slot ranges of the
// levels that are still open; returns their number, or -1 on an internal inconsistency.
OGQ_HD int sel_orq_pass(const SolverView& v, int s, LvInfo* lv, int* range_a, int* range_b)
{
    int open = 0;
    for (int stride = (s - 1) >> 1; stride >= 1; stride >>= 1) {
        for (int q = stride; q < s - 1; q += 2 * stride) {
            if (lv[q].exact) continue;
            if (!sel_orq_solve(v, lv[q - stride], lv[q + stride], lv[q])) return -1;
            if (!lv[q].exact) {
                range_a[open] = lv[q].sa;
                range_b[open] = lv[q].sb;
                ++open;
            }
        }
    }
    return open;
}

OGQ_HD int sel_floor_log2(long long x)
{
    int r = 0;
    while ((x >> (r + 1)) > 0) ++r;
    return r;
}

// Turns open slot ranges into the intervals of the next round.
//
// The ranges (one per open level) are swept in slot order.  With trim_empty (ORQ: a level is
// always a data value) only populated cells are kept, and a run of cells is cut wherever more
// than `hole` consecutive cells are empty, so that two far-apart populated cells do not drag
// the empty stretch between them along.  Cells that belong to a narrow range (at most kTight
// cells) form intervals of their own even inside a wide range, so that they are refined first
// and their level becomes exact quickly; this is what lets the levels that depend on it tighten
// in the next round.  The spare cell budget is then handed out narrow intervals first.
// Returns the number of new intervals, or a negative code if no refinement is possible.
OGQ_HD int sel_refine(const SolverView& v, int nr, const int* ra_in, const int* rb_in, bool trim_empty,
                      Interval* out, long long* total_elems_out)
{
    constexpr int kTight = 8;
    int ra[kMaxLv], rb[kMaxLv];
    for (int i = 0; i < nr; ++i) { ra[i] = ra_in[i]; rb[i] = rb_in[i]; }
    for (int i = 1; i < nr; ++i) {  // sort by start
        const int a = ra[i], b = rb[i];
        int j = i - 1;
        while (j >= 0 && ra[j] > a) { ra[j + 1] = ra[j]; rb[j + 1] = rb[j]; --j; }
        ra[j + 1] = a;
        rb[j + 1] = b;
    }
    int pa[kMaxIv], pb[kMaxIv];
    int m = 0;
    // Fast path (the usual case): the ranges do not touch each other, so every range is handled on
    // its own -- narrow ones by walking their cells, wide sparse ones by hopping from one populated
    // cell to the next with the prefix counts, wide dense ones by trimming their two ends.
    bool fast = true;
    for (int i = 1; i < nr; ++i)
        if (ra[i] <= rb[i - 1] + 1) fast = false;
    for (int i = 0; i < nr && fast; ++i) {
        const int a = ra[i], b = rb[i];
        int first = a, last = b;
        bool hop = false;
        if (trim_empty) {
            const long long cnt = (long long)v.cpre[b + 1] - (long long)v.cpre[a];
            if (cnt <= 0) continue;
            bool gap;
            first = sel_locate(v, (long long)v.cpre[a], true, &gap);
            last = sel_locate(v, (long long)v.cpre[b + 1] - 1, false, &gap);
            if (first < a || last > b || first > last) { fast = false; break; }
            hop = (last - first + 1 > 12) && cnt <= 32;
        }
        if (hop) {
            // few elements spread over many cells: one piece per populated cell (neighbours joined)
            long long pos = v.cpre[first];
            const long long end = v.cpre[last + 1];
            while (pos < end && fast) {
                bool gap;
                const int c = sel_locate(v, pos, true, &gap);
                if (c < 0 || gap) { fast = false; break; }
                if (m > 0 && c <= pb[m - 1] + 2 && c > pb[m - 1] &&
                    sel_interval_of_slot(v, c) == sel_interval_of_slot(v, pb[m - 1])) {
                    pb[m - 1] = c;
                } else {
                    if (m >= kMaxIv) { fast = false; break; }
                    pa[m] = c; pb[m] = c; ++m;
                }
                pos = v.cpre[c + 1];
            }
        } else if (last - first + 1 <= 12 && trim_empty) {
            // narrow: walk the cells, cut at end slots and at more than one empty cell in a row
            int run_a = -1, lastp = -1;
            for (int c = first; c <= last + 1 && fast; ++c) {
                const bool boundary = (c > last) || sel_is_end_slot(v, c);
                const bool populated = !boundary && v.cpre[c + 1] != v.cpre[c];
                if (run_a >= 0 && (boundary || (!populated && c - lastp > 1))) {
                    if (m >= kMaxIv) { fast = false; break; }
                    pa[m] = run_a; pb[m] = lastp; ++m;
                    run_a = -1;
                }
                if (populated) { if (run_a < 0) run_a = c; lastp = c; }
            }
        } else {
            // wide and dense (or no trimming wanted): the hull, cut where it crosses into another interval
            int j0 = sel_interval_of_slot(v, first);
            const int j1 = sel_interval_of_slot(v, last);
            for (int j = j0; j <= j1 && fast; ++j) {
                const int lo = v.slotbase[j], hi = v.slotbase[j] + v.iv[j].ncell - 1;
                const int x = first > lo ? first : lo, y = last < hi ? last : hi;
                if (x > y) continue;
                if (m >= kMaxIv) { fast = false; break; }
                pa[m] = x; pb[m] = y; ++m;
            }
        }
    }
    if (!fast) {
        int hole = 1;
        bool use_tight = true;
        for (;;) {
            m = 0;
            bool overflow = false;
            int idx = 0;
            while (idx < nr && !overflow) {
                int hull_b = rb[idx], jn = idx + 1;
                while (jn < nr && ra[jn] <= hull_b + 1) { if (rb[jn] > hull_b) hull_b = rb[jn]; ++jn; }
                int iv_j = sel_interval_of_slot(v, ra[idx]);
                int iv_end = v.slotbase[iv_j] + v.iv[iv_j].ncell;  // end slot of the current interval
                int run_a = -1, last = -1;
                bool run_tight = false;
                for (int c = ra[idx]; c <= hull_b + 1 && !overflow; ++c) {
                    while (c > iv_end && iv_j + 1 < v.m) { ++iv_j; iv_end = v.slotbase[iv_j] + v.iv[iv_j].ncell; }
                    const bool boundary = (c > hull_b) || (c == iv_end);
                    bool populated = false, tight = false;
                    if (!boundary) {
                        populated = !trim_empty || v.cpre[c + 1] != v.cpre[c];
                        if (populated && use_tight)
                            for (int k = idx; k < jn; ++k)
                                if (ra[k] <= c && c <= rb[k] && rb[k] - ra[k] < kTight) tight = true;
                    }
                    const bool cut = run_a >= 0 && (boundary || (populated && tight != run_tight) ||
                                                    (!populated && c - last > hole));
                    if (cut) {
                        if (m >= kMaxIv) overflow = true;
                        else { pa[m] = run_a; pb[m] = last; ++m; }
                        run_a = -1;
                    }
                    if (populated) {
                        if (run_a < 0) { run_a = c; run_tight = tight; }
                        last = c;
                    }
                }
                idx = jn;
            }
            if (!overflow) break;
            if (hole < (1 << 28)) hole *= 8;
            else if (use_tight) use_tight = false;
            else return -11;
        }
    }
    if (m == 0) return -12;
    // cell budget: every interval starts with its current cells (always fits), then the spare
    // cells are handed out one halving of the cell width at a time, narrow intervals first
    int rbits[kMaxIv], order[kMaxIv], psh[kMaxIv];
    {
        int used = 0;
        for (int i = 0; i < m; ++i) {
            rbits[i] = 0;
            order[i] = i;
            psh[i] = sel_slot_shift(v, pa[i]);
            used += pb[i] - pa[i] + 1;
        }
        if (used > kCells) return -14;
        for (int i = 1; i < m; ++i) {  // ascending by cell count
            const int o = order[i], c = pb[o] - pa[o];
            int j = i - 1;
            while (j >= 0 && pb[order[j]] - pa[order[j]] > c) { order[j + 1] = order[j]; --j; }
            order[j + 1] = o;
        }
        for (bool changed = true; changed;) {
            changed = false;
            for (int q = 0; q < m; ++q) {
                const int i = order[q];
                if (rbits[i] >= psh[i]) continue;
                const int cost = (pb[i] - pa[i] + 1) << rbits[i];  // extra cells of one more halving
                if (used + cost > kCells) continue;
                used += cost;
                ++rbits[i];
                changed = true;
            }
        }
    }
    int cellbase = 0;
    bool progress = false, open_shift = false;
    long long total_elems = 0;
    for (int i = 0; i < m; ++i) {
        total_elems += (long long)v.cpre[pb[i] + 1] - (long long)v.cpre[pa[i]];
        const int j = sel_interval_of_slot(v, pa[i]);
        const Interval& o = v.iv[j];
        const int ca = pa[i] - v.slotbase[j], cb = pb[i] - v.slotbase[j];
        const int cells = cb - ca + 1;
        int r = rbits[i];
        if (r > o.sh) r = o.sh;
        Interval& ni = out[i];
        ni.sh = o.sh - r;
        ni.ncell = cells << r;
        ni.klo = o.klo + ((uint32_t)ca << o.sh);
        ni.khi = ni.klo + (uint32_t)((((unsigned long long)ni.ncell) << ni.sh) - 1ull);
        ni.cellbase = cellbase;
        ni.pad = 0;
        ni.cbefore = v.cpre[pa[i]];
        ni.sbefore = v.spre[pa[i]];
        cellbase += ni.ncell;
        if (r > 0) progress = true;
        if (ni.sh > 0) open_shift = true;
    }
    if (total_elems_out) *total_elems_out = total_elems;
    if (cellbase > kCells) return -15;
    if (open_shift && !progress) return -16;
    return m;
}

// ------------------------------------------------------------------ BinGrad-pb
// g(x) = x n - sum_{|v| >= x} |v| at the lower edge of a cell slot (keys are magnitudes here).
OGQ_HD double sel_pb_g(const SolverView& v, int slot, double* x_out)
{
    const double x = sel_slot_vlo(v, slot);
    *x_out = x;
    return x * (double)v.n - (v.stot - v.spre[slot]);
}

// Final BinGrad-pb step on single-key cells.  c is the last key with g(x_c) <= 0, so the sign
// change of g lies in [x_c, next key).  With P_up the sum of all magnitudes above x_c: if the
// zero P_up / n of the piece above x_c is larger than x_c it is the answer, otherwise g jumps
// across zero at the data value x_c itself.
OGQ_HD double sel_pb_final(const SolverView& v, int slot)
{
    const double x = sel_slot_vlo(v, slot);
    const double stat_up = (v.stot - v.spre[slot + 1]) / (double)v.n;
    return stat_up > x ? stat_up : x;
}

}  // namespace ogq
