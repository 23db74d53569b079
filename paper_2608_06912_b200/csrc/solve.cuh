// Threshold solve on sorted data (App. A and App. B of the paper):
//   stabilised prefix/suffix scans of e^{+-s/t} -> node values of the budget
//   curve -> crossing index -> closed-form root of the per-interval quadratic.
// The same block-level routine serves three levels: tiles of a globally sorted
// row (aggregates), the elements of the crossing tile / of a whole short row /
// of the bracket's middle band (in shared memory).
#pragma once
#include "common.cuh"

namespace lapsum {

// Tails that enclose the data a solve looks at (App. B).  L: sum over everything
// below, pivoted at L.pivot (= a_L, or -inf with sum 0 when nothing is below);
// R: sum over everything above, pivoted at R.pivot (= a_R, or +inf); n_R = count above.
struct Seeds {
    Agg L, R;
    long long n_R;
};

struct TileAgg {
    float first, last;  // smallest and largest key of the tile
    float sum_up;       // sum e^{(s - last)/t}
    float sum_down;     // sum e^{-(s - first)/t}
};

struct SolveResult {
    float b;          // fp32 threshold
    RowThreshold th;  // the same threshold as pivot + offset
    int status;       // 0 or LAPSUM_ST_ROOT_LEFT / RIGHT / NO_CROSSING bits
    int jstar;
};

constexpr unsigned ST_ROOT_LEFT = 0x4u, ST_ROOT_RIGHT = 0x8u, ST_NO_CROSSING = 0x20u;

struct ScanShared {
    Agg warp_agg[32];
    double dsum[32];
    int imax[32];
};

// ------------------------------------------------ block scans (monoid) ----
// Exclusive prefix of per-thread aggregates in thread order, `seed` folded in
// below thread 0.  Warp-shuffle scan inside warps, one warp scans the warp totals.
// Only the first `nw` warps hold data (the others pass empty aggregates and skip the arithmetic, but
// every thread of the block must call: the function contains block barriers).
__device__ inline Agg block_exclusive_up(Agg mine, Agg seed, ExpScale sc, ScanShared &sh, int nw)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool on = warp < nw;
    Agg incl = mine;
    if (on) {
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            Agg other;
            other.pivot = __shfl_up_sync(FULL, incl.pivot, o);
            other.sum = __shfl_up_sync(FULL, incl.sum, o);
            if (lane >= o) incl = combine_up(other, incl, sc);
        }
    }
    __syncthreads();
    if (on && lane == 31) sh.warp_agg[warp] = incl;
    __syncthreads();
    if (warp == 0 && nw > 1) {
        Agg w = (lane < nw) ? sh.warp_agg[lane] : empty_up();
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            Agg other;
            other.pivot = __shfl_up_sync(FULL, w.pivot, o);
            other.sum = __shfl_up_sync(FULL, w.sum, o);
            if (lane >= o) w = combine_up(other, w, sc);
        }
        sh.warp_agg[lane] = w;
    }
    __syncthreads();
    if (!on) return seed;
    Agg below;
    below.pivot = __shfl_up_sync(FULL, incl.pivot, 1);
    below.sum = __shfl_up_sync(FULL, incl.sum, 1);
    if (lane == 0) below = empty_up();
    Agg wp = (warp > 0) ? sh.warp_agg[warp - 1] : empty_up();
    return combine_up(seed, combine_up(wp, below, sc), sc);
}

// Exclusive suffix: everything held by higher threads, `seed` folded in above the last thread.
__device__ inline Agg block_exclusive_down(Agg mine, Agg seed, ExpScale sc, ScanShared &sh, int nw)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool on = warp < nw;
    Agg incl = mine;
    if (on) {
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            Agg other;
            other.pivot = __shfl_down_sync(FULL, incl.pivot, o);
            other.sum = __shfl_down_sync(FULL, incl.sum, o);
            if (lane + o < 32) incl = combine_down(incl, other, sc);
        }
    }
    __syncthreads();
    if (on && lane == 0) sh.warp_agg[warp] = incl;
    __syncthreads();
    if (warp == 0 && nw > 1) {
        Agg w = (lane < nw) ? sh.warp_agg[lane] : empty_down();
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            Agg other;
            other.pivot = __shfl_down_sync(FULL, w.pivot, o);
            other.sum = __shfl_down_sync(FULL, w.sum, o);
            if (lane + o < 32) w = combine_down(w, other, sc);
        }
        sh.warp_agg[lane] = w;
    }
    __syncthreads();
    if (!on) return seed;
    Agg above;
    above.pivot = __shfl_down_sync(FULL, incl.pivot, 1);
    above.sum = __shfl_down_sync(FULL, incl.sum, 1);
    if (lane == 31) above = empty_down();
    Agg wp = (warp + 1 < nw) ? sh.warp_agg[warp + 1] : empty_down();
    return combine_down(combine_down(above, wp, sc), seed, sc);
}

// ------------------------------------------------------- item sources ----
// An item is a run of consecutive sorted elements summarised by its first and
// last key and its two pivoted sums.  end(i) = number of elements in items 0..i.
struct ElemItems {
    const float *s;
    __device__ float first(int i) const { return s[i]; }
    __device__ float last(int i) const { return s[i]; }
    __device__ float up(int) const { return 1.f; }
    __device__ float down(int) const { return 1.f; }
    __device__ long long end(int i) const { return i + 1; }
};
struct TileItems {
    const TileAgg *a;
    long long total;
    int tile;
    __device__ float first(int i) const { return a[i].first; }
    __device__ float last(int i) const { return a[i].last; }
    __device__ float up(int i) const { return a[i].sum_up; }
    __device__ float down(int i) const { return a[i].sum_down; }
    __device__ long long end(int i) const
    {
        long long e = (long long)(i + 1) * tile;
        return e < total ? e : total;
    }
};

// Node values at the end of every item and the crossing (App. A: "index lookup"):
// returns J = number of leading items whose end node has Lap >= k, i.e. the
// root lies in item J (J == count: above all items); -1 if even the left end
// a_L has Lap < k.  pref/suf are scratch arrays of `count` floats.
template <typename Items>
__device__ int crossing_item(const Items it, int count, long long total, Seeds sd, double k, ExpScale sc,
                             float *pref, float *suf, ScanShared &sh, bool trust_left)
{
    // a scan round costs every participating warp the same whatever it holds, so no more warps take part
    // than give each thread two items
    const int tid = threadIdx.x;
    int nw = (count + 63) / 64;
    nw = max(1, min(nw, (int)(blockDim.x >> 5)));
    if (blockDim.x < 32) nw = 1;
    const int T = min((int)blockDim.x, nw * 32);
    const int chunk = (count + T - 1) / T;
    const int c0 = (tid < T) ? min(count, tid * chunk) : count, c1 = min(count, c0 + chunk);

    // prefix direction
    Agg a = empty_up();
    for (int i = c0; i < c1; ++i) a = combine_up(a, Agg{it.last(i), it.up(i)}, sc);
    Agg run = block_exclusive_up(a, sd.L, sc, sh, nw);
    for (int i = c0; i < c1; ++i) {
        run = combine_up(run, Agg{it.last(i), it.up(i)}, sc);
        pref[i] = run.sum;
    }
    // suffix direction
    a = empty_down();
    for (int i = c1 - 1; i >= c0; --i) a = combine_down(Agg{it.first(i), it.down(i)}, a, sc);
    run = block_exclusive_down(a, sd.R, sc, sh, nw);
    for (int i = c1 - 1; i >= c0; --i) {
        run = combine_down(Agg{it.first(i), it.down(i)}, run, sc);
        suf[i] = run.sum;
    }
    __syncthreads();

    int cand = INT_MIN;
    for (int i = c0; i < c1; ++i) {
        const float node = it.last(i);
        Agg above = (i + 1 < count) ? Agg{it.first(i + 1), suf[i + 1]} : sd.R;
        const float Bp = fold_down(above, node, sc);
        const double G = 0.5 * ((double)pref[i] - (double)Bp) + ((double)(sd.n_R + total - it.end(i)) - k);
        if (G >= 0.0) cand = i + 1;
    }
    if (tid == 0) {
        if (trust_left || sd.L.pivot == -CUDART_INF_F) {
            cand = max(cand, 0);  // Lap(-inf) = all elements > k, or a coarser level already placed the root here
        } else {
            Agg above = (count > 0) ? Agg{it.first(0), suf[0]} : sd.R;
            const float Bp = fold_down(above, sd.L.pivot, sc);
            const double G = 0.5 * ((double)sd.L.sum - (double)Bp) + ((double)(sd.n_R + total) - k);
            if (G >= 0.0) cand = max(cand, 0);
        }
    }
    int J = block_max(cand, sh.imax);
    return J < 0 ? -1 : J;
}

// Root of the budget equation inside [lo, hi] (the per-interval quadratic):
//   c = N_above - k;  A = sum_{<= lo} e^{(s-lo)/t};  B = sum_{>= hi} e^{-(s-hi)/t}
//   c <= 0: u = e^{(b-lo)/t} = A / (sqrt(c^2 + A B e^{-d/t}) - c)
//   c >  0: w = e^{(hi-b)/t} = B / (c + sqrt(c^2 + A e^{-d/t} B))
//   c == 0: b = (lo+hi)/2 + (t/2) ln(A/B)
// The result is stored as (nearer end, offset) so that the offset is small.
__device__ inline SolveResult interval_root(float lo, float hi, double A, double B, double c, double t)
{
    SolveResult r;
    r.status = 0;
    r.jstar = 0;
    const double d = (double)hi - (double)lo;  // may be +inf
    double off_lo;                             // b - lo (when lo finite)
    double off_hi;                             // b - hi (when hi finite), <= 0
    const bool lo_ok = lo > -CUDART_INF_F, hi_ok = hi < CUDART_INF_F;
    if (c == 0.0 && lo_ok && hi_ok && A > 0.0 && B > 0.0) {
        off_lo = 0.5 * d + 0.5 * t * log(A / B);
    } else if (c <= 0.0 && lo_ok) {
        const double Bp = hi_ok ? B * exp(-d / t) : 0.0;
        const double den = sqrt(c * c + A * Bp) - c;
        off_lo = (den > 0.0 && A > 0.0) ? t * log(A / den) : 0.0;
    } else if (hi_ok) {
        const double Ap = lo_ok ? A * exp(-d / t) : 0.0;
        const double w = B / (c + sqrt(c * c + Ap * B));
        const double back = (w > 1.0) ? t * log(w) : 0.0;  // hi - b >= 0
        off_lo = d - back;
        if (!lo_ok) {
            off_hi = -back;
            r.th.hi = hi;
            r.th.lo = (float)off_hi;
            r.b = (float)((double)hi + off_hi);
            return r;
        }
    } else {
        r.status = (int)ST_NO_CROSSING;
        r.th.hi = lo_ok ? lo : 0.f;
        r.th.lo = 0.f;
        r.b = r.th.hi;
        return r;
    }
    if (!hi_ok) {
        off_lo = fmax(off_lo, 0.0);
        r.th.hi = lo;
        r.th.lo = (float)off_lo;
        r.b = (float)((double)lo + off_lo);
        return r;
    }
    off_lo = fmin(fmax(off_lo, 0.0), d);  // clamp into the interval
    off_hi = off_lo - d;
    if (off_lo <= -off_hi) {
        r.th.hi = lo;
        r.th.lo = (float)off_lo;
    } else {
        r.th.hi = hi;
        r.th.lo = (float)off_hi;
    }
    r.b = (float)((double)lo + off_lo);
    return r;
}

// The same root in fp32, for rows so short (the one-warp-per-row path, n <= 128) that the fp64 log/exp/sqrt
// of interval_root would be a third of the whole row's work.  Every quantity is O(n) or smaller and the
// formulas are the cancellation-free forms, so fp32 keeps u (w) to ~2e-7 relative, i.e. b to ~2e-7 t.
// `side` (nullable) receives -1 / +1 when the unclamped root lies below lo / above hi by more than rounding: the
// crossing index that chose the interval was then off by at least one, and the caller may move it; 0 otherwise.
// (The interval's formula continued beyond its ends is still monotone, so the side is the true one.)
__device__ inline SolveResult interval_root_f32(float lo, float hi, float A, float B, float c, float t, int *side = nullptr)
{
    SolveResult r;
    r.status = 0;
    r.jstar = 0;
    if (side) *side = 0;
    const float d = hi - lo;  // may be +inf
    const bool lo_ok = lo > -CUDART_INF_F, hi_ok = hi < CUDART_INF_F;
    const float slack = 1e-6f * t;
    float off_lo;  // b - lo, not yet clamped into [0, d]
    if (c == 0.f && lo_ok && hi_ok && A > 0.f && B > 0.f) {
        off_lo = 0.5f * d + 0.5f * t * logf(A / B);
    } else if (c <= 0.f && lo_ok) {
        const float Bp = hi_ok ? B * expf(-d / t) : 0.f;
        const float den = sqrtf(fmaf(c, c, A * Bp)) - c;
        off_lo = (den > 0.f && A > 0.f) ? t * logf(A / den) : 0.f;
    } else if (hi_ok) {
        const float Ap = lo_ok ? A * expf(-d / t) : 0.f;
        const float w = B / (c + sqrtf(fmaf(c, c, Ap * B)));
        const float back = (w > 0.f) ? t * logf(w) : 0.f;  // hi - b; negative when the root lies above hi
        if (!lo_ok) {
            if (side && back < -slack) *side = 1;
            r.th.hi = hi;
            r.th.lo = -fmaxf(back, 0.f);
            r.b = hi + r.th.lo;
            return r;
        }
        off_lo = d - back;
    } else {
        r.status = (int)ST_NO_CROSSING;
        r.th.hi = lo_ok ? lo : 0.f;
        r.th.lo = 0.f;
        r.b = r.th.hi;
        return r;
    }
    if (side) *side = (off_lo < -slack) ? -1 : (hi_ok && off_lo > d + slack) ? 1 : 0;
    if (!hi_ok) {
        off_lo = fmaxf(off_lo, 0.f);
        r.th.hi = lo;
        r.th.lo = off_lo;
        r.b = lo + off_lo;
        return r;
    }
    off_lo = fminf(fmaxf(off_lo, 0.f), d);
    const float off_hi = off_lo - d;
    if (off_lo <= -off_hi) {
        r.th.hi = lo;
        r.th.lo = off_lo;
    } else {
        r.th.hi = hi;
        r.th.lo = off_hi;
    }
    r.b = lo + off_lo;
    return r;
}

// Full solve over `count` sorted items (single scores, or runs of equal scores with a multiplicity)
// with tails `sd`.  pref/suf: scratch of `count` floats each.  Every thread returns the same result.
// trust_left: the left end was already certified (an interior tile boundary or -inf), so
// Lap(left end) is not tested; test_right: the right end is a real bracket end a_R whose
// certificate Lap(a_R) <= k must be checked.
template <typename Items>
__device__ inline SolveResult solve_items_block(const Items it, int count, long long total, Seeds sd, double k, double t,
                                                ExpScale sc, float *pref, float *suf, ScanShared &sh,
                                                SolveResult *sh_res, bool trust_left, bool test_right)
{
    const int J = crossing_item(it, count, total, sd, k, sc, pref, suf, sh, trust_left);
    SolveResult res;
    if (J < 0) {
        res.status = (int)ST_ROOT_LEFT;
        res.jstar = -1;
        res.b = sd.L.pivot;
        res.th.hi = sd.L.pivot;
        res.th.lo = 0.f;
        return res;
    }
    const float lo = (J == 0) ? sd.L.pivot : it.last(J - 1);
    const float hi = (J == count) ? sd.R.pivot : it.first(J);
    // direct re-summation about the interval ends: one rounding per term instead of a scan tree
    double accA = 0.0, accB = 0.0;
    for (int i = threadIdx.x; i < count; i += blockDim.x) {
        if (i < J) accA += (double)(it.up(i) * decay(lo - it.last(i), sc));
        else accB += (double)(it.down(i) * decay(it.first(i) - hi, sc));
    }
    double A = block_sum(accA, sh.dsum);
    double B = block_sum(accB, sh.dsum);
    if (threadIdx.x == 0) {
        A += (double)fold_up(sd.L, lo, sc);
        B += (double)fold_down(sd.R, hi, sc);
        const long long at_or_below = (J > 0) ? it.end(J - 1) : 0;
        const double c = (double)(sd.n_R + (total - at_or_below)) - k;
        SolveResult r = interval_root(lo, hi, A, B, c, t);
        r.jstar = J;
        // certificate of the right end (Alg. 1): Lap(a_R) <= k, else the root is right of a_R
        if (test_right && J == count && sd.R.pivot < CUDART_INF_F) {
            const double A_R = A * exp(-((double)hi - (double)lo) / t);
            const double F_R = 0.5 * A_R + (double)sd.n_R - 0.5 * (double)sd.R.sum;
            if (F_R > k) r.status |= (int)ST_ROOT_RIGHT;
        }
        *sh_res = r;
    }
    __syncthreads();
    res = *sh_res;
    __syncthreads();
    return res;
}

// M sorted single scores in shared memory
__device__ inline SolveResult solve_sorted_block(const float *s, int M, Seeds sd, double k, double t, ExpScale sc,
                                                 float *pref, float *suf, ScanShared &sh, SolveResult *sh_res,
                                                 bool trust_left, bool test_right)
{
    return solve_items_block(ElemItems{s}, M, (long long)M, sd, k, t, sc, pref, suf, sh, sh_res, trust_left, test_right);
}

// ------------------------------------ short forms for single-block kernels ----
// A kernel that runs once per call as a single block executes every instruction cold: measured on B200,
// about 40 cycles per instruction of straight-line code that is not in the instruction cache yet, and a
// third of that once it is.  So the routines below keep their loops rolled, share one out-of-line scan and
// take the root in fp32: the shortest code wins, not the fewest executed instructions.

struct WarpScan {
    unsigned cnt;  // inclusive count
    Agg up, down;  // inclusive prefix (pivot = last) and suffix (pivot = first) aggregates
};
// inclusive scans across the lanes of one warp: counts and prefix aggregates upwards, suffix aggregates downwards
__device__ __noinline__ WarpScan warp_scan3(WarpScan v, ExpScale sc)
{
    const int lane = threadIdx.x & 31;
#pragma unroll 1
    for (int o = 1; o < 32; o <<= 1) {
        const unsigned c1 = __shfl_up_sync(FULL, v.cnt, o);
        Agg ou, od;
        ou.pivot = __shfl_up_sync(FULL, v.up.pivot, o);
        ou.sum = __shfl_up_sync(FULL, v.up.sum, o);
        od.pivot = __shfl_down_sync(FULL, v.down.pivot, o);
        od.sum = __shfl_down_sync(FULL, v.down.sum, o);
        if (lane >= o) {
            v.cnt += c1;
            v.up = combine_up(ou, v.up, sc);
        }
        if (lane + o < 32) v.down = combine_down(v.down, od, sc);
    }
    return v;
}

// Exact solve over m <= PAIRS_MAX UNSORTED scores by all pairs: no sort and no scan.
// For a score s_i let "below" be the scores that precede it in sorted order (smaller, or equal with a
// lower list position) plus itself, and "above" the rest plus itself.  Then
//   rank_i = |below|,  P_i = sum_below e^{-(s_i - s_j)/t},  Q_i = sum_above e^{-(s_j - s_i)/t}
// are exactly the prefix and suffix sums of the sorted list at its rank_i-th node (App. A), so the node value is
// 0.5 (P_i - (Q_i - 1)) + (N_above - k), the crossing is the largest rank whose node value is >= k, and the
// interval's two sums are P at that rank and Q at the next one.  g lanes share one score and split the j loop;
// terms are summed as 2^-40 fixed point, so neither the list's order nor the lane split can change a bit.
// Every thread of the block calls (two barriers) and returns the result.  Cost m^2 / 32 warp iterations of a
// loop of a dozen instructions: the shortest code, which is what a once-per-call block is bound by.
constexpr int PAIRS_MAX = 256;
struct PairsShared {
    float sorted[PAIRS_MAX];
    double P[PAIRS_MAX], Q[PAIRS_MAX];
    int jmax;
};

__device__ inline SolveResult solve_list_pairs(uint32_t *list, int m, Seeds sd, double k, double t, ExpScale sc,
                                               PairsShared &ps, bool trust_left, bool test_right)
{
    const int tid = threadIdx.x;
    float *val = reinterpret_cast<float *>(list);
    for (int i = tid; i < m; i += blockDim.x) val[i] = key_to_float(list[i]);
    if (tid == 0) ps.jmax = INT_MIN;
    __syncthreads();
    int g = 32;  // lanes per score
    while (g > 1 && m * g > (int)blockDim.x) g >>= 1;
    const int sub = tid & (g - 1), grp = tid / g, ngrp = (int)blockDim.x / g;
    const double base = (double)(sd.n_R + m) - k;
    constexpr float FX = 1099511627776.f;  // 2^40
#pragma unroll 1
    for (int i0 = 0; i0 < m; i0 += ngrp) {
        const int i = i0 + grp;
        const bool live = i < m;
        const float si = live ? val[i] : 0.f;
        long long P = 0, Q = 0;
        int rank = 0;
        if (live) {
#pragma unroll 1
            for (int j = sub; j < m; j += g) {
                const float sj = val[j];
                const long long e = __float2ll_rn(decay(fabsf(sj - si), sc) * FX);
                if (sj < si || (sj == si && j <= i)) {
                    P += e;
                    ++rank;
                }
                if (sj > si || (sj == si && j >= i)) Q += e;
            }
        }
#pragma unroll 1
        for (int o = g >> 1; o > 0; o >>= 1) {
            P += __shfl_xor_sync(FULL, P, o);
            Q += __shfl_xor_sync(FULL, Q, o);
            rank += __shfl_xor_sync(FULL, rank, o);
        }
        if (live && sub == 0) {
            const double Pd = (double)P * (1.0 / (double)FX) + (double)fold_up(sd.L, si, sc);
            const double Qd = (double)Q * (1.0 / (double)FX) + (double)fold_down(sd.R, si, sc);
            ps.sorted[rank - 1] = si;
            ps.P[rank - 1] = Pd;
            ps.Q[rank - 1] = Qd;
            const double G = 0.5 * (Pd - (Qd - 1.0)) + (base - (double)rank);
            if (G >= 0.0) atomicMax(&ps.jmax, rank);
        }
    }
    __syncthreads();
    int J = ps.jmax;
    if (trust_left || sd.L.pivot == -CUDART_INF_F) {
        J = max(J, 0);  // Lap(-inf) = all elements > k, or a coarser level already placed the root here
    } else {
        const Agg above = (m > 0) ? Agg{ps.sorted[0], (float)ps.Q[0]} : sd.R;
        const double G = 0.5 * ((double)sd.L.sum - (double)fold_down(above, sd.L.pivot, sc)) + base;
        if (G >= 0.0) J = max(J, 0);
    }
    SolveResult res;
    if (J < 0) {
        res.status = (int)ST_ROOT_LEFT;
        res.jstar = -1;
        res.b = sd.L.pivot;
        res.th.hi = sd.L.pivot;
        res.th.lo = 0.f;
        return res;
    }
    const float lo = (J == 0) ? sd.L.pivot : ps.sorted[J - 1];
    const float hi = (J == m) ? sd.R.pivot : ps.sorted[J];
    const double A = (J == 0) ? (double)sd.L.sum : ps.P[J - 1];
    const double B = (J == m) ? (double)sd.R.sum : ps.Q[J];
    const double c = (double)(sd.n_R + (m - J)) - k;
    res = interval_root_f32(lo, hi, (float)A, (float)B, (float)c, (float)t);
    res.jstar = J;
    // certificate of the right end (Alg. 1): Lap(a_R) <= k, else the root is right of a_R
    if (test_right && J == m && sd.R.pivot < CUDART_INF_F) {
        const double F_R = 0.5 * A * (double)decay(hi - lo, sc) + (double)sd.n_R - 0.5 * (double)sd.R.sum;
        if (F_R > k) res.status |= (int)ST_ROOT_RIGHT;
    }
    return res;
}

}  // namespace lapsum
