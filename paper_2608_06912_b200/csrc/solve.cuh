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

constexpr unsigned ST_ROOT_LEFT = 0x4u, ST_ROOT_RIGHT = 0x8u, ST_NO_CROSSING = 0x20u, ST_BAD_BUDGET = 0x80u;

// A row whose budget or temperature is unusable (see RowParams) is solved with harmless stand-ins and void_result()
// then replaces what came out: NaN threshold, hence a NaN mask.
__device__ __forceinline__ void void_result(SolveResult &res)
{
    res.b = __int_as_float(0x7fc00000);
    res.th.hi = res.b;
    res.th.lo = 0.f;
}

struct ScanShared {
    Agg warp_agg[32], warp_agg2[32];
    double dsum[32], dsum2[32];
    int imax[32];
};

// ------------------------------------------------------ scans (monoid) ----
// A kernel that runs once per call as a single block executes every instruction cold: measured on B200,
// about 40 cycles per instruction of straight-line code that is not in the instruction cache yet, and a
// third of that once it is.  So the routines of this file keep their loops rolled, share one out-of-line
// warp scan, use one barrier where three would be natural, and take the root in fp32: the shortest code
// wins, not the fewest executed instructions.
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

// ------------------------------------------------------- item sources ----
// An item is a run of consecutive sorted elements summarised by its first and
// last key and its two pivoted sums.  end(i) = number of elements in items 0..i.
// Index of element i in an array that skips one word after every 32: threads that walk consecutive chunks of such
// an array (stride = chunk length) then hit different shared-memory banks.  PAD = true item sources, and the
// pref / suf scratch used with them, are laid out this way (count + count / 32 words).
template <typename Items>
__device__ __forceinline__ int pidx(int i) { return Items::PAD ? i + (i >> 5) : i; }

struct ElemItems {
    static constexpr bool PAD = false;
    const float *s;
    __device__ float first(int i) const { return s[i]; }
    __device__ float last(int i) const { return s[i]; }
    __device__ float up(int) const { return 1.f; }
    __device__ float down(int) const { return 1.f; }
    __device__ long long end(int i) const { return i + 1; }
};
struct PaddedElemItems {  // single scores stored at s[i + i / 32]
    static constexpr bool PAD = true;
    const float *s;
    __device__ float first(int i) const { return s[i + (i >> 5)]; }
    __device__ float last(int i) const { return s[i + (i >> 5)]; }
    __device__ float up(int) const { return 1.f; }
    __device__ float down(int) const { return 1.f; }
    __device__ long long end(int i) const { return i + 1; }
};
struct TileItems {
    static constexpr bool PAD = false;
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
// What a block's scan of its own items leaves in every thread's registers: the thread's chunk [c0, c1), the inclusive
// scans of the chunk aggregates inside the warp (w) and of the warps' totals (top).  It does not depend on the seeds, so
// a block that first has to tell others what its items add up to (a cluster's part of a row) scans once.
struct LocalScan {
    WarpScan w, top;
    int c0, c1;
    __device__ Agg total_up() const { return shfl_agg(top.up, 31); }     // all items, prefix form (pivot: the last item)
    __device__ Agg total_down() const { return shfl_agg(top.down, 0); }  // all items, suffix form (pivot: the first item)
};

template <typename Items>
__device__ LocalScan scan_items(const Items it, int count, ExpScale sc, ScanShared &sh)
{
    // every thread of the block calls (one barrier).  A scan round costs every participating warp the same
    // whatever it holds, so no more warps take part than give each thread two items.
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = (int)(blockDim.x + 31) >> 5;
    int nw = (count + 63) / 64;
    nw = max(1, min(nw, nwarps));
    const int T = min((int)blockDim.x, nw * 32);
    const int chunk = (count + T - 1) / T;
    const int c0 = (tid < T) ? min(count, tid * chunk) : count, c1 = min(count, c0 + chunk);

    // this thread's chunk in both directions, then the warp's inclusive scans
    WarpScan w{0u, empty_up(), empty_down()};
#pragma unroll 1
    for (int i = c0; i < c1; ++i) w.up = combine_up(w.up, Agg{it.last(i), it.up(i)}, sc);
#pragma unroll 1
    for (int i = c1 - 1; i >= c0; --i) w.down = combine_down(Agg{it.first(i), it.down(i)}, w.down, sc);
    w = warp_scan3(w, sc);
    if (lane == 31) sh.warp_agg[warp] = w.up;
    if (lane == 0) sh.warp_agg2[warp] = w.down;
    __syncthreads();
    // every warp scans the warps' totals for itself
    WarpScan top{0u, lane < nwarps ? sh.warp_agg[lane] : empty_up(), lane < nwarps ? sh.warp_agg2[lane] : empty_down()};
    top = warp_scan3(top, sc);
    return LocalScan{w, top, c0, c1};
}

template <typename Items>
__device__ int crossing_from_scan(const Items it, int count, long long total, Seeds sd, double k, ExpScale sc,
                                  float *pref, float *suf, ScanShared &sh, bool trust_left, const LocalScan &ls)
{
    // every thread of the block calls (three barriers)
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = (int)(blockDim.x + 31) >> 5;
    const WarpScan &w = ls.w, &top = ls.top;
    const int c0 = ls.c0, c1 = ls.c1;
    Agg run = shfl_agg(w.up, max(lane - 1, 0));  // this warp's lanes below
    if (lane == 0) run = empty_up();
    Agg oth = shfl_agg(top.up, max(warp - 1, 0));  // the warps below
    if (warp == 0) oth = empty_up();
    run = combine_up(combine_up(sd.L, oth, sc), run, sc);
#pragma unroll 1
    for (int i = c0; i < c1; ++i) {
        run = combine_up(run, Agg{it.last(i), it.up(i)}, sc);
        pref[pidx<Items>(i)] = run.sum;
    }
    run = shfl_agg(w.down, min(lane + 1, 31));
    if (lane == 31) run = empty_down();
    oth = shfl_agg(top.down, min(warp + 1, 31));
    if (warp + 1 >= nwarps) oth = empty_down();
    run = combine_down(combine_down(run, oth, sc), sd.R, sc);
#pragma unroll 1
    for (int i = c1 - 1; i >= c0; --i) {
        run = combine_down(Agg{it.first(i), it.down(i)}, run, sc);
        suf[pidx<Items>(i)] = run.sum;
    }
    __syncthreads();

    int cand = INT_MIN;
#pragma unroll 1
    for (int i = c0; i < c1; ++i) {
        const float node = it.last(i);
        const Agg above = (i + 1 < count) ? Agg{it.first(i + 1), suf[pidx<Items>(i + 1)]} : sd.R;
        const float Bp = fold_down(above, node, sc);
        const double G = 0.5 * ((double)pref[pidx<Items>(i)] - (double)Bp) + ((double)(sd.n_R + total - it.end(i)) - k);
        if (G >= 0.0) cand = i + 1;
    }
    if (tid == 0) {
        if (trust_left || sd.L.pivot == -CUDART_INF_F) {
            cand = max(cand, 0);  // Lap(-inf) = all elements > k, or a coarser level already placed the root here
        } else {
            const Agg above = (count > 0) ? Agg{it.first(0), suf[0]} : sd.R;
            const float Bp = fold_down(above, sd.L.pivot, sc);
            const double G = 0.5 * ((double)sd.L.sum - (double)Bp) + ((double)(sd.n_R + total) - k);
            if (G >= 0.0) cand = max(cand, 0);
        }
    }
    cand = warp_max(cand);
    __syncthreads();  // sh.imax may still be read by an earlier call's last step
    if (lane == 0) sh.imax[warp] = cand;
    __syncthreads();
    const int J = warp_max(lane < nwarps ? sh.imax[lane] : INT_MIN);
    return J < 0 ? -1 : J;
}

template <typename Items>
__device__ int crossing_item(const Items it, int count, long long total, Seeds sd, double k, ExpScale sc,
                             float *pref, float *suf, ScanShared &sh, bool trust_left)
{
    const LocalScan ls = scan_items(it, count, sc, sh);
    return crossing_from_scan(it, count, total, sd, k, sc, pref, suf, sh, trust_left, ls);
}

// Root of the budget equation inside [lo, hi] (the per-interval quadratic):
//   c = N_above - k;  A = sum_{<= lo} e^{(s-lo)/t};  B = sum_{>= hi} e^{-(s-hi)/t}
//   c <= 0: u = e^{(b-lo)/t} = A / (sqrt(c^2 + A B e^{-d/t}) - c)
//   c >  0: w = e^{(hi-b)/t} = B / (c + sqrt(c^2 + A e^{-d/t} B))
//   c == 0: b = (lo+hi)/2 + (t/2) ln(A/B)
// The result is stored as (pivot of the form used, offset from it).
// Taken in fp32: these are the cancellation-free forms (every sum is of positive terms), A and B arrive as
// correctly rounded fp64 sums and c as the rounded fp64 difference, so u (w) is good to ~2e-7 relative and
// the offset to ~2e-7 t; the fp64 log/exp/sqrt would be several hundred instructions executed once.
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
    // Each form gives the offset from ITS OWN pivot (u: above lo, w: below hi) and the threshold is stored
    // against that pivot: converting between the two (d - offset) would round at ulp(d), which can be many t
    // when the interval is a wide gap.  The form that applies is the one whose pivot the root is near.
    float up = 0.f, down = 0.f;  // b - lo (u form) or hi - b (w form), not yet clamped into [0, d]
    bool from_lo;
    if (c == 0.f && lo_ok && hi_ok && A > 0.f && B > 0.f) {
        const float shift = 0.5f * t * logf(A / B);  // b = (lo + hi)/2 + shift
        from_lo = shift <= 0.f;
        up = 0.5f * d + shift;
        down = 0.5f * d - shift;
    } else if (c <= 0.f && lo_ok) {
        const float Bp = hi_ok ? B * expf(-d / t) : 0.f;
        const float den = sqrtf(fmaf(c, c, A * Bp)) - c;
        from_lo = true;
        up = (den > 0.f && A > 0.f) ? t * logf(A / den) : 0.f;
    } else if (hi_ok) {
        const float Ap = lo_ok ? A * expf(-d / t) : 0.f;
        const float w = B / (c + sqrtf(fmaf(c, c, Ap * B)));
        from_lo = false;
        down = (w > 0.f) ? t * logf(w) : 0.f;
    } else {
        r.status = (int)ST_NO_CROSSING;
        r.th.hi = lo_ok ? lo : 0.f;
        r.th.lo = 0.f;
        r.b = r.th.hi;
        return r;
    }
    if (from_lo) {
        if (side) *side = (up < -slack) ? -1 : (hi_ok && up > d + slack) ? 1 : 0;
        up = fmaxf(up, 0.f);
        if (hi_ok) up = fminf(up, d);
        r.th.hi = lo;
        r.th.lo = up;
        r.b = lo + up;
    } else {
        if (side) *side = (down < -slack) ? 1 : (lo_ok && down > d + slack) ? -1 : 0;
        down = fmaxf(down, 0.f);
        if (lo_ok) down = fminf(down, d);
        r.th.hi = hi;
        r.th.lo = -down;
        r.b = hi - down;
    }
    return r;
}

// Full solve over `count` sorted items (single scores, or runs of equal scores with a multiplicity)
// with tails `sd`.  pref/suf: scratch of `count` floats each.  Every thread returns the same result.
// trust_left: the left end was already certified (an interior tile boundary or -inf), so
// Lap(left end) is not tested; test_right: the right end is a real bracket end a_R whose
// certificate Lap(a_R) <= k must be checked.
template <typename Items>
__device__ inline SolveResult solve_items_block(const Items it, int count, long long total, Seeds sd, double k, double t,
                                                ExpScale sc, float *pref, float *suf, ScanShared &sh, bool trust_left,
                                                bool test_right, const LocalScan *scanned = nullptr)
{
    // scanned: the result of scan_items on the same items, if the caller has it already
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = (int)(blockDim.x + 31) >> 5;
    const int J = scanned ? crossing_from_scan(it, count, total, sd, k, sc, pref, suf, sh, trust_left, *scanned)
                          : crossing_item(it, count, total, sd, k, sc, pref, suf, sh, trust_left);
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
    double A = 0.0, B = 0.0;
#pragma unroll 1
    for (int i = threadIdx.x; i < count; i += blockDim.x) {
        if (i < J) A += (double)(it.up(i) * decay(lo - it.last(i), sc));
        else B += (double)(it.down(i) * decay(it.first(i) - hi, sc));
    }
    A = warp_sum(A);
    B = warp_sum(B);
    if (lane == 0) { sh.dsum[warp] = A; sh.dsum2[warp] = B; }
    __syncthreads();
    A = warp_sum(lane < nwarps ? sh.dsum[lane] : 0.0) + (double)fold_up(sd.L, lo, sc);
    B = warp_sum(lane < nwarps ? sh.dsum2[lane] : 0.0) + (double)fold_down(sd.R, hi, sc);
    const long long at_or_below = (J > 0) ? it.end(J - 1) : 0;
    const double c = (double)(sd.n_R + (total - at_or_below)) - k;
    res = interval_root_f32(lo, hi, (float)A, (float)B, (float)c, (float)t);
    res.jstar = J;
    // certificate of the right end (Alg. 1): Lap(a_R) <= k, else the root is right of a_R
    if (test_right && J == count && sd.R.pivot < CUDART_INF_F) {
        const double F_R = 0.5 * A * (double)decay(hi - lo, sc) + (double)sd.n_R - 0.5 * (double)sd.R.sum;
        if (F_R > k) res.status |= (int)ST_ROOT_RIGHT;
    }
    __syncthreads();  // sh.dsum may be reused by the caller
    return res;
}

// M sorted single scores in shared memory
__device__ inline SolveResult solve_sorted_block(const float *s, int M, Seeds sd, double k, double t, ExpScale sc,
                                                 float *pref, float *suf, ScanShared &sh, bool trust_left, bool test_right)
{
    return solve_items_block(ElemItems{s}, M, (long long)M, sd, k, t, sc, pref, suf, sh, trust_left, test_right);
}
// the same with s, pref and suf in the padded layout (M + M / 32 words each)
__device__ inline SolveResult solve_sorted_block_padded(const float *s, int M, Seeds sd, double k, double t, ExpScale sc,
                                                        float *pref, float *suf, ScanShared &sh, bool trust_left,
                                                        bool test_right)
{
    return solve_items_block(PaddedElemItems{s}, M, (long long)M, sd, k, t, sc, pref, suf, sh, trust_left, test_right);
}

// ------------------------------------ short forms for single-block kernels ----
// A kernel that runs once per call as a single block executes every instruction cold: measured on B200,
// about 40 cycles per instruction of straight-line code that is not in the instruction cache yet, and a
// third of that once it is.  So the routines below keep their loops rolled, share one out-of-line scan and
// take the root in fp32: the shortest code wins, not the fewest executed instructions.

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
                                               PairsShared &ps, bool trust_left, bool test_right, Control *ctl = nullptr)
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
            if (LAPSUM_IN_BOUNDS(rank - 1, PAIRS_MAX, ctl)) {
                ps.sorted[rank - 1] = si;
                ps.P[rank - 1] = Pd;
                ps.Q[rank - 1] = Qd;
            }
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
