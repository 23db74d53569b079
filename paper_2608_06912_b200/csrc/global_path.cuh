// Kernels of the two large-row pipelines.
//   full sort : radix sort -> tile_aggregate -> solve_global -> cdf_map
//   bracket   : sample_hist -> sample_pick -> stream_band -> band_solve -> cdf_map   (bracket_select.cuh),
//               band_solve launching, from the device and only on a failed certificate, a widened
//               stream_band + band_solve or the full-sort chain;
//               with full_sorts = 1: sample_gather -> radix sort of the sample -> stream_band
//               -> radix sort of the band -> tile_aggregate -> solve_global -> (predicated full sort) -> cdf_map
//   backward  : vjp_reduce -> vjp_map
#pragma once
#include "common.cuh"
#include "radix_sort.cuh"
#include "row_block.cuh"
#include "solve.cuh"

namespace lapsum {

constexpr int TILE_S = 2048;      // elements per scan tile
constexpr int AGG_THREADS = 256;  // tile_aggregate block
constexpr int SOLVE_THREADS = 1024;

// ------------------------------------------------------- row parameters ----
// One thread per row: the row's budget and temperature (device vectors; a null vector means the call's scalar) become
// the RowParams every later kernel reads.  The checks are those the host applies to scalar arguments: alpha finite,
// non-zero and |alpha| a normal fp32 number; 0 < k < n.  A row that fails is void: its threshold (and with it its mask)
// is NaN, a status bit is raised, and the kernels of its chain return at once.  Eq. 8 is evaluated without fused
// multiply-adds, so that the ranks are those of the host and of the oracle.
__global__ void row_params_kernel(const double *k_rows, const double *alpha_rows, double k_call, double alpha_call,
                                  long long rows, long long n, long long K, double z, int need_budget, RowParams *out,
                                  float *b_out, RowThreshold *th_out, Control *ctl)
{
    pdl_wait();
    const long long row = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (row >= rows) return;
    const double k = k_rows ? k_rows[row] : k_call;
    const double alpha = alpha_rows ? alpha_rows[row] : alpha_call;
    const double t = fabs(alpha);
    const bool alpha_ok = isfinite(alpha) && t >= 1.1754943508222875e-38 && t <= 3.0e38;
    const bool k_ok = !need_budget || (isfinite(k) && k > 0.0 && k < (double)n);
    RowParams p;
    p.valid = (alpha_ok && k_ok) ? 1 : 0;
    p.pad = 0;
    const double tt = alpha_ok ? t : 1.0;
    const double kk = (need_budget && k_ok) ? k : 0.5 * (double)n;
    p.k = alpha < 0.0 ? kk : (double)n - kk;
    p.t = tt;
    p.inv_t = 1.0 / tt;
    p.sc = make_scale(tt);
    p.c = (float)(1.4426950408889634074 / tt);
    p.c_mask = alpha < 0.0 ? p.c : -p.c;
    p.half_inv_t = (float)(0.5 / tt);
    p.gsign = alpha < 0.0 ? 1.f : -1.f;
    p.j = p.l = 0;
    if (K > 0) {
        const double q = __ddiv_rn(__dsub_rn((double)n, p.k), (double)n);
        const double mu = __dmul_rn((double)K, q);
        const double sd = __dsqrt_rn(__dmul_rn(__dmul_rn((double)K, q), __dsub_rn(1.0, q)));
        p.j = (long long)floor(__dsub_rn(mu, __dmul_rn(z, sd)));
        p.l = (long long)ceil(__dadd_rn(mu, __dmul_rn(z, sd)));
    }
    out[row] = p;
    if (!p.valid) {
        if (b_out) b_out[row] = __int_as_float(0x7fc00000);
        if (th_out) th_out[row] = RowThreshold{__int_as_float(0x7fc00000), 0.f};
        set_status(ctl, (alpha_ok ? 0u : ST_BAD_ALPHA_BIT) | (k_ok ? 0u : (unsigned)ST_BAD_BUDGET));
    }
}

// --------------------------------------------------- tile aggregates ----
// Per tile of the sorted keys: first/last key and the two pivoted exponential
// sums (the (pivot, sum) monoid elements that the tile-level scan combines).
__global__ void __launch_bounds__(AGG_THREADS) tile_aggregate_kernel(const uint32_t *__restrict__ keys, SortCount cnt,
                                                                      TileAgg *aggs, ExpScale sc, const int *run_flag,
                                                                      const RowParams *rp)
{
    pdl_wait();
    if (run_flag && *run_flag == 0) return;
    if (rp) {
        if (!rp->valid) return;
        sc = rp->sc;
    }
    // one warp per tile: 64 keys per lane (128-bit loads where the tile is whole), sums by shuffles, no block barrier
    const int lane = threadIdx.x & 31;
    const unsigned long long n = cnt.get();
    const unsigned long long ntiles = (n + TILE_S - 1) / TILE_S;
    const unsigned long long warps = (unsigned long long)gridDim.x * (AGG_THREADS / 32);
    for (unsigned long long tile = (unsigned long long)blockIdx.x * (AGG_THREADS / 32) + (threadIdx.x >> 5); tile < ntiles;
         tile += warps) {
        const unsigned long long base = tile * TILE_S;
        const int valid = (int)min((unsigned long long)TILE_S, n - base);
        const float first = key_to_float(__ldg(keys + base));
        const float last = key_to_float(__ldg(keys + base + valid - 1));
        float up = 0.f, down = 0.f;
        if (valid == TILE_S && (((uintptr_t)keys) & 15) == 0) {
            const uint4 *k4 = reinterpret_cast<const uint4 *>(keys + base);
#pragma unroll 4
            for (int j = 0; j < TILE_S / 128; ++j) {
                const uint4 q = __ldg(k4 + j * 32 + lane);
                const float s0 = key_to_float(q.x), s1 = key_to_float(q.y), s2 = key_to_float(q.z), s3 = key_to_float(q.w);
                up += (decay(last - s0, sc) + decay(last - s1, sc)) + (decay(last - s2, sc) + decay(last - s3, sc));
                down += (decay(s0 - first, sc) + decay(s1 - first, sc)) + (decay(s2 - first, sc) + decay(s3 - first, sc));
            }
        } else {
            for (int i = lane; i < valid; i += 32) {
                const float s = key_to_float(__ldg(keys + base + i));
                up += decay(last - s, sc);
                down += decay(s - first, sc);
            }
        }
        const double U = warp_sum((double)up), D = warp_sum((double)down);
        if (lane == 0) aggs[tile] = TileAgg{first, last, (float)U, (float)D};
    }
}

// ------------------------------------------------------ global solve ----
struct SolveArgs {
    const uint32_t *keys;  // sorted keys
    SortCount cnt;
    const TileAgg *aggs;
    float *pref, *suf;  // scratch, one float per tile each
    Control *ctl;
    float *b_out;          // threshold of this row
    RowThreshold *th_out;  // threshold pair of this row
    const int *run_flag;   // nullable: run only if *run_flag != 0
    double k, t;
    ExpScale sc;
    int bracket;              // 1: tails come from the stream pass, a failed certificate raises the fallback flag
    unsigned long long cap;   // band capacity (bracket)
    unsigned long long total_n;  // row length (for statistics)
    const RowParams *rp;         // nullable: the row's own budget and temperature replace k, t, sc
};

__global__ void __launch_bounds__(SOLVE_THREADS) solve_global_kernel(SolveArgs a)
{
    pdl_wait();
    if (a.run_flag && *a.run_flag == 0) return;
    if (a.rp) {
        if (!a.rp->valid) return;
        a.k = a.rp->k;
        a.t = a.rp->t;
        a.sc = a.rp->sc;
    }
    __shared__ float s[TILE_S];
    __shared__ float pref2[TILE_S];
    __shared__ float suf2[TILE_S];
    __shared__ ScanShared sh;

    Seeds sd;
    sd.L = empty_up();
    sd.R = empty_down();
    sd.n_R = 0;
    unsigned long long M = 0;
    if (a.bracket) {
        const CallCtl &c = a.ctl->call;
        const unsigned long long raw = c.band_count;
        if (raw > a.cap) {  // band overflow: the whole row goes through the full sort
            if (threadIdx.x == 0) {
                a.ctl->call.fallback = 1;
                set_status(a.ctl, 0x1u | 0x2u);
                atomicAdd(&a.ctl->persist.fallbacks, 1ull);
            }
            return;
        }
        M = raw;
        if (c.a_L > -CUDART_INF_F) sd.L = Agg{c.a_L, (float)c.S_L};
        if (c.a_R < CUDART_INF_F) sd.R = Agg{c.a_R, (float)c.S_R};
        sd.n_R = (long long)c.n_R;
    } else {
        M = a.cnt.get();
    }
    const int ntiles = (int)((M + TILE_S - 1) / TILE_S);
    TileItems it{a.aggs, (long long)M, TILE_S};
    const int J = crossing_item(it, ntiles, (long long)M, sd, a.k, a.sc, a.pref, a.suf, sh, false);
    SolveResult res;
    if (J < 0) {
        res.status = (int)ST_ROOT_LEFT;
        res.b = sd.L.pivot;
        res.th = RowThreshold{sd.L.pivot, 0.f};
    } else {
        // tails of the crossing tile, re-summed directly about its neighbours' keys
        Seeds s2 = sd;
        if (J > 0) {
            const float pv = a.aggs[J - 1].last;
            double acc = 0.0;
            for (int T = threadIdx.x; T < J; T += blockDim.x)
                acc += (double)(a.aggs[T].sum_up * decay(pv - a.aggs[T].last, a.sc));
            acc = block_sum(acc, sh.dsum) + (double)fold_up(sd.L, pv, a.sc);
            s2.L = Agg{pv, (float)acc};
        }
        if (J + 1 < ntiles) {
            const float pv = a.aggs[J + 1].first;
            double acc = 0.0;
            for (int T = J + 1 + threadIdx.x; T < ntiles; T += blockDim.x)
                acc += (double)(a.aggs[T].sum_down * decay(a.aggs[T].first - pv, a.sc));
            acc = block_sum(acc, sh.dsum) + (double)fold_down(sd.R, pv, a.sc);
            s2.R = Agg{pv, (float)acc};
        }
        int M2 = 0;
        if (J < ntiles) {
            const unsigned long long base = (unsigned long long)J * TILE_S;
            M2 = (int)min((unsigned long long)TILE_S, M - base);
            for (int i = threadIdx.x; i < M2; i += blockDim.x) s[i] = key_to_float(__ldg(a.keys + base + i));
            s2.n_R = sd.n_R + (long long)(M - base - M2);
        }
        __syncthreads();
        res = solve_sorted_block(s, M2, s2, a.k, a.t, a.sc, pref2, suf2, sh, /*trust_left=*/J > 0 || !a.bracket,
                                 /*test_right=*/a.bracket && J + 1 >= ntiles);
    }
    if (threadIdx.x == 0) {
        if (a.bracket && (res.status & (int)(ST_ROOT_LEFT | ST_ROOT_RIGHT))) {
            a.ctl->call.fallback = 1;
            set_status(a.ctl, 0x1u | (unsigned)res.status);
            atomicAdd(&a.ctl->persist.fallbacks, 1ull);
        } else {
            if (res.status) set_status(a.ctl, a.bracket ? (unsigned)res.status : 0x20u);
            *a.b_out = res.b;
            *a.th_out = res.th;
        }
    }
}

// ------------------------------------------------- device-side fallback ----
// Everything the full-sort solve of one row needs, prepared by the host.  When the bracket's certificate
// fails (Alg. 1 line 5) the kernel that finds out launches this chain itself, into the tail-launch stream:
// the chain runs after that kernel and before the next kernel of the caller's stream, and a forward whose
// bracket held (all but ~1e-6 of them) launches nothing for it.
struct FallbackPlan {
    int enabled;
    int hist_grid, pass_grid, agg_grid;
    const void *r_in;  // the row's scores
    int in_kind;       // their element type as a radix input kind (RS_IN_F32 / F16 / BF16)
    SortCount cnt;
    SortCtl *sort_ctl;
    PassArgs pass[4];
    TileAgg *aggs;
    ExpScale sc;
    SolveArgs solve;  // solve.rp (nullable) also serves the tile aggregates
};

// the plan of row `g` of a group from the plan of the group's first row (BatchShift)
__device__ inline void shift_plan(FallbackPlan &f, unsigned g, unsigned long long ws, unsigned long long data_bytes)
{
    shift_bytes(f.r_in, data_bytes);
    shift_bytes(f.sort_ctl, ws);
    for (int p = 0; p < 4; ++p) {
        PassArgs &a = f.pass[p];
        shift_bytes(a.keys_in, p == 0 ? data_bytes : ws);  // the first pass reads the scores themselves
        shift_bytes(a.vals_in, ws);
        shift_bytes(a.keys_out, ws);
        shift_bytes(a.vals_out, ws);
        shift_bytes(a.ctl, ws);
        shift_bytes(a.status, ws);
        shift_bytes(a.status_next, ws);
        shift_bytes(a.control, ws);
    }
    shift_bytes(f.aggs, ws);
    SolveArgs &sv = f.solve;
    shift_bytes(sv.keys, ws);
    shift_bytes(sv.aggs, ws);
    shift_bytes(sv.pref, ws);
    shift_bytes(sv.suf, ws);
    shift_bytes(sv.ctl, ws);
    if (sv.b_out) sv.b_out += g;
    if (sv.th_out) sv.th_out += g;
    if (sv.rp) sv.rp += g;
}

template <int IN>
__device__ inline void launch_fullsort_head(const FallbackPlan &f, bool payload)
{   // histogram and first pass read the scores in their own element type
    rs_histogram_kernel<IN><<<f.hist_grid, 512, 0, cudaStreamTailLaunch>>>(f.r_in, f.cnt, f.sort_ctl, f.pass[0].status, nullptr);
    if (payload) rs_onesweep_kernel<IN, true><<<f.pass_grid, RS_THREADS, sizeof(PassShared<true>), cudaStreamTailLaunch>>>(f.pass[0]);
    else rs_onesweep_kernel<IN, false><<<f.pass_grid, RS_THREADS, sizeof(PassShared<false>), cudaStreamTailLaunch>>>(f.pass[0]);
}

__device__ inline void launch_fullsort_fallback(const FallbackPlan &f)
{
    const bool payload = f.pass[0].vals_out != nullptr;
    if (f.in_kind == RS_IN_F16) launch_fullsort_head<RS_IN_F16>(f, payload);
    else if (f.in_kind == RS_IN_BF16) launch_fullsort_head<RS_IN_BF16>(f, payload);
    else launch_fullsort_head<RS_IN_F32>(f, payload);
    for (int p = 1; p < 4; ++p) {
        if (payload) rs_onesweep_kernel<RS_IN_KEYS, true><<<f.pass_grid, RS_THREADS, sizeof(PassShared<true>), cudaStreamTailLaunch>>>(f.pass[p]);
        else rs_onesweep_kernel<RS_IN_KEYS, false><<<f.pass_grid, RS_THREADS, sizeof(PassShared<false>), cudaStreamTailLaunch>>>(f.pass[p]);
    }
    tile_aggregate_kernel<<<f.agg_grid, AGG_THREADS, 0, cudaStreamTailLaunch>>>(static_cast<const uint32_t *>(f.pass[3].keys_out), f.cnt, f.aggs, f.sc, nullptr, f.solve.rp);
    solve_global_kernel<<<1, SOLVE_THREADS, 0, cudaStreamTailLaunch>>>(f.solve);
}

// ------------------------------------------------------------ p map ----
// The three element-wise streams (mask, VJP reduction, VJP map) walk a row in tiles of EW_THREADS * EW_U 16-byte
// vectors; the tiles go to the blocks round-robin, thread t of the block takes vectors t, t + EW_THREADS, ... of the
// tile (constant offsets from one index), and the arithmetic runs on pairs of scores (packed fp32 instructions).
// What is left of the row behind the last full tile, and rows that are not 16-byte aligned, take a plain loop.
constexpr int EW_THREADS = 512;
constexpr int EW_U = 2;
constexpr unsigned EW_TILE = EW_THREADS * EW_U;
// The mask kernel reads one array only: eight vectors per thread keep as many bytes in flight as the vectors of two arrays in
// the VJP kernels (measured at n = 1e8: 2, 4, 8 vectors -> 125, 122.5, 121.8 us).  Rows below CDF_LONG_N keep tiles of two
// vectors per thread, so that a mid-size row still spreads over all SMs.
constexpr int CDF_U_LONG = 8, CDF_U_SHORT = 2;
constexpr long long CDF_LONG_N = 1ll << 23;
#ifndef LAPSUM_VMAP_U
#define LAPSUM_VMAP_U 3
#endif
constexpr int VMAP_U = LAPSUM_VMAP_U;  // (r, v) vector pairs per thread and tile of the VJP map
constexpr unsigned VMAP_TILE = EW_THREADS * VMAP_U;

// p_i = sigma((r_i - b)/t) from the unsorted scores (Eq. 2-3): 128-bit loads and stores.
// The row is walked from its end towards its start: the pass that ran before (the stream pass of
// the bracket path) read the row front to back, so its tail is what the L2 still holds.
// path_note != 0: this launch closes a forward call (bookkeeping for lapsum_status); in a group launch its low byte is
// the note and the bits above name the row + 1 whose blocks write it.
// clean_call != 0: the last block also zeroes the per-call control scalars: every kernel that used them has
// completed by now, and the next forward on this workspace then needs no memset of its own in front of it.
template <typename T, int CDF_U>
__global__ void __launch_bounds__(EW_THREADS, 2) cdf_map_kernel(const T *__restrict__ r, T *__restrict__ p,
                                                              unsigned long long n, const RowThreshold *th_ptr, float c,
                                                              Control *ctl, int path_note, const RowParams *rp, int clean_call,
                                                              BatchShift bs)
{
    pdl_wait();
    if (bs.active) {  // row blockIdx.y of a group; path_note - 1 is then the row that closes the call (0: none)
        const unsigned g = blockIdx.y;
        r += g * bs.row_step;
        p += g * bs.row_step;
        th_ptr += g;
        shift_bytes(ctl, g * bs.ws_step);
        if (rp) rp += g;
        path_note = (path_note >> 8) == (int)g + 1 ? (path_note & 0xff) : 0;
    }
    if (rp) c = rp->c_mask;
    if (clean_call && blockIdx.x == gridDim.x - 1) {
        static_assert(sizeof(CallCtl) % 8 == 0 && offsetof(Control, call) % 8 == 0, "CallCtl is cleared with 64-bit stores");
        unsigned long long *z = reinterpret_cast<unsigned long long *>(&ctl->call);
        for (unsigned i = threadIdx.x; i < sizeof(CallCtl) / 8; i += blockDim.x) z[i] = 0ull;
    }
    constexpr int V = Io<T>::V, P = V / 2;
    constexpr unsigned CDF_TILE = EW_THREADS * CDF_U;
    using Vec = typename Io<T>::Vec;
    const RowThreshold th = *th_ptr;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    const unsigned long long gtid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (gtid == 0 && path_note) {
        ctl->persist.last_path = path_note;
        ctl->persist.forwards += 1;
    }
    unsigned long long nvec = 0;
    if ((((uintptr_t)r | (uintptr_t)p) & 15) == 0 && blockDim.x == EW_THREADS) {
        nvec = n / V;
        const Vec *r4 = reinterpret_cast<const Vec *>(r);
        Vec *p4 = reinterpret_cast<Vec *>(p);
        const float2 nhi = dup2(-th.hi), nlo = dup2(-th.lo), cc = dup2(c);
        auto map_vec = [&](const Vec &xv) {
            float2 x[P], y[P];
            Io<T>::unpack2(xv, x);
#pragma unroll
            for (int w = 0; w < P; ++w) y[w] = laplace_cdf2(x[w], nhi, nlo, cc);
            return Io<T>::pack2(y);
        };
        const long long ntile = (long long)(nvec / CDF_TILE), step = (long long)gridDim.x * CDF_TILE;
        for (long long i = (ntile - 1 - (long long)blockIdx.x) * CDF_TILE + threadIdx.x; i >= 0; i -= step) {
            Vec xv[CDF_U];
#pragma unroll
            for (int u = 0; u < CDF_U; ++u) xv[u] = io_ldg<T>(r4 + i + u * EW_THREADS);  // kept in L2: the backward reads r again
#pragma unroll
            for (int u = 0; u < CDF_U; ++u) io_stcs<T>(p4 + i + u * EW_THREADS, map_vec(xv[u]));
        }
        for (unsigned long long i = (unsigned long long)ntile * CDF_TILE + gtid; i < nvec; i += stride) io_stcs<T>(p4 + i, map_vec(io_ldg<T>(r4 + i)));
    }
    for (unsigned long long i = nvec * V + gtid; i < n; i += stride) Io<T>::store1(p + i, laplace_cdf(Io<T>::load1(r + i), th, c));
}

// -------------------------------------------------------------- VJP ----
// Eq. 5 in two passes: S_f = sum f, S_vf = sum v f (fixed-order reduction),
// then grad_i = f_i (v_i - S_vf/S_f).
struct VjpArgs {
    const void *v, *r;       // upstream gradient and scores of the row, in the workspace's element type
    const float *b;
    const RowThreshold *th;  // nullable: the forward's threshold pair of this row (workspace)
    void *grad;              // gradient out, same element type
    unsigned long long n;
    double *partials;  // 4 doubles per block
    Control *ctl;
    float c, half_inv_t;
    float *grad_k, *grad_alpha;  // nullable: this row's scalar gradients
    double inv_t;
    float gsign;  // +1, or -1 when alpha > 0: sign of the mask's Jacobian (the reduction and the scalar gradients ignore it)
    const RowParams *rp;  // nullable: the row's own temperature replaces c, half_inv_t, inv_t, gsign
    int all_sums;         // 1: the four sums are formed and left in the control block whether or not grad_k / grad_alpha
                          // are asked for (a shard of a row: the sums of all shards are added before they are used)
    BatchShift bs;
};

// moves the arguments to the block's row (group launch), then reads the row's own parameters;
// returns true for a void row (unusable temperature): its gradients are NaN
template <typename T>
__device__ __forceinline__ bool vjp_row_params(VjpArgs &a)
{
    if (a.bs.active) {
        const unsigned g = blockIdx.y;
        const unsigned long long data = g * a.bs.row_step * sizeof(T), ws = g * a.bs.ws_step;
        shift_bytes(a.v, data);
        shift_bytes(a.r, data);
        shift_bytes(a.grad, data);
        a.b += g;
        if (a.th) a.th += g;
        shift_bytes(a.partials, ws);
        shift_bytes(a.ctl, ws);
        if (a.grad_k) a.grad_k += g;
        if (a.grad_alpha) a.grad_alpha += g;
        if (a.rp) a.rp += g;
        a.bs.active = 0;
    }
    if (!a.rp) return false;
    a.c = a.rp->c;
    a.half_inv_t = a.rp->half_inv_t;
    a.inv_t = a.rp->inv_t;
    a.gsign = a.rp->gsign;
    return a.rp->valid == 0;
}

// host side: does a launch with these arguments need the two extra sums of grad_alpha?
inline bool vjp_wants_scalars(const VjpArgs &a) { return a.grad_k || a.grad_alpha || a.all_sums; }

// SCALARS: also sum e (r-b) and v e (r-b), the two sums grad_alpha needs.  The sums are taken of e = e^{-|b-r|/t};
// the common factor 1/(2t) of the densities is applied once per block, in fp64.
template <typename T, bool SCALARS>
__global__ void __launch_bounds__(EW_THREADS, 2) vjp_reduce_kernel(VjpArgs a)
{
    pdl_wait();
    const bool dead = vjp_row_params<T>(a);
    constexpr int V = Io<T>::V, P = V / 2;
    using Vec = typename Io<T>::Vec;
    const T *ar = static_cast<const T *>(a.r), *av = static_cast<const T *>(a.v);
    __shared__ double red[32];
    __shared__ int is_last;
    const RowThreshold b = backward_threshold(a.b, a.th);
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    const unsigned long long gtid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    const float2 nhi = dup2(-b.hi), nlo = dup2(-b.lo), cc = dup2(a.c);
    float2 se = dup2(0.f), sv = dup2(0.f), sd = dup2(0.f), svd = dup2(0.f);
    auto add_pair = [&](float2 x, float2 w) {
        const float2 d = add2(add2(x, nhi), nlo);
        const float2 z = mul2(d, cc);
        const float2 e = make_float2(ex2_approx(-fabsf(z.x)), ex2_approx(-fabsf(z.y)));
        se = add2(se, e);
        const float2 we = mul2(w, e);
        sv = add2(sv, we);
        if (SCALARS) {
            sd = fma2(e, d, sd);
            svd = fma2(we, d, svd);
        }
    };
    auto add_vec = [&](const Vec &xv, const Vec &wv) {
        float2 x[P], w[P];
        Io<T>::unpack2(xv, x);
        Io<T>::unpack2(wv, w);
#pragma unroll
        for (int e = 0; e < P; ++e) add_pair(x[e], w[e]);
    };
    unsigned long long nvec = 0;
    if ((((uintptr_t)ar | (uintptr_t)av) & 15) == 0 && blockDim.x == EW_THREADS) {
        nvec = a.n / V;
        const Vec *r4 = reinterpret_cast<const Vec *>(ar);
        const Vec *v4 = reinterpret_cast<const Vec *>(av);
        // Two tiles per thread are in flight at any time: the loads of the next tile are issued before the current one
        // is summed (the two register sets alternate), so the memory system is never idle while a warp computes.
        const unsigned long long ntile = nvec / EW_TILE, step = (unsigned long long)gridDim.x * EW_TILE, end = ntile * EW_TILE;
        Vec xa[EW_U], wa[EW_U], xb[EW_U], wb[EW_U];
        auto fetch = [&](Vec (&x)[EW_U], Vec (&w)[EW_U], unsigned long long i) {
#pragma unroll
            for (int u = 0; u < EW_U; ++u) {
                x[u] = io_ldg<T>(r4 + i + u * EW_THREADS);
                w[u] = io_ldg<T>(v4 + i + u * EW_THREADS);
            }
        };
        auto consume = [&](const Vec (&x)[EW_U], const Vec (&w)[EW_U]) {
#pragma unroll
            for (int u = 0; u < EW_U; ++u) add_vec(x[u], w[u]);
        };
        unsigned long long i = (unsigned long long)blockIdx.x * EW_TILE + threadIdx.x;
        if (i < end) {
            fetch(xa, wa, i);
            for (;;) {
                i += step;
                if (i < end) fetch(xb, wb, i);
                consume(xa, wa);
                if (i >= end) break;
                i += step;
                if (i < end) fetch(xa, wa, i);
                consume(xb, wb);
                if (i >= end) break;
            }
        }
        for (unsigned long long i = ntile * EW_TILE + gtid; i < nvec; i += stride) add_vec(io_ldg<T>(r4 + i), io_ldg<T>(v4 + i));
    }
    for (unsigned long long i = nvec * V + gtid; i < a.n; i += stride) {  // one score at a time, into the first halves
        const float d = (Io<T>::load1(ar + i) - b.hi) - b.lo;
        const float e = ex2_approx(-fabsf(d * a.c));
        const float we = Io<T>::load1(av + i) * e;
        se.x += e;
        sv.x += we;
        if (SCALARS) {
            sd.x = fmaf(e, d, sd.x);
            svd.x = fmaf(we, d, svd.x);
        }
    }
    const double h = (double)a.half_inv_t;
    const double S_f = block_sum((double)se.x + (double)se.y, red) * h;
    const double S_vf = block_sum((double)sv.x + (double)sv.y, red) * h;
    double S_fd = 0.0, S_vfd = 0.0;
    if (SCALARS) {
        S_fd = block_sum((double)sd.x + (double)sd.y, red) * h;
        S_vfd = block_sum((double)svd.x + (double)svd.y, red) * h;
    }
    if (threadIdx.x == 0) {
        double *o = a.partials + 4 * (size_t)blockIdx.x;
        o[0] = S_f;
        o[1] = S_vf;
        o[2] = S_fd;
        o[3] = S_vfd;
        __threadfence();
        const unsigned t = atomicAdd(&a.ctl->call.vjp_ticket, 1u);
        is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double pf = 0.0, pv = 0.0, pd = 0.0, pvd = 0.0;
    for (unsigned i = threadIdx.x; i < gridDim.x; i += blockDim.x) {
        pf += __ldcg(a.partials + 4 * i);
        pv += __ldcg(a.partials + 4 * i + 1);
        pd += __ldcg(a.partials + 4 * i + 2);
        pvd += __ldcg(a.partials + 4 * i + 3);
    }
    pf = block_sum(pf, red);
    pv = block_sum(pv, red);
    pd = block_sum(pd, red);
    pvd = block_sum(pvd, red);
    if (threadIdx.x == 0) {
        a.ctl->persist.S_f = pf;
        a.ctl->persist.S_vf = pv;
        a.ctl->persist.S_fd = pd;
        a.ctl->persist.S_vfd = pvd;
        a.ctl->call.vjp_ticket = 0;  // ready for the next row / call
        const double mean = (pf > 0.0) ? pv / pf : 0.0;
        const float nanf_ = __int_as_float(0x7fc00000);
        if (a.grad_k) *a.grad_k = dead ? nanf_ : (float)mean;
        if (a.grad_alpha) *a.grad_alpha = dead ? nanf_ : (pf > 0.0) ? (float)((pvd - mean * pd) * a.inv_t) : 0.f;
    }
}

template <typename T>
__global__ void __launch_bounds__(EW_THREADS, 2) vjp_map_kernel(VjpArgs a)
{
    pdl_wait();
    const bool dead = vjp_row_params<T>(a);
    constexpr int V = Io<T>::V, P = V / 2;
    using Vec = typename Io<T>::Vec;
    const T *ar = static_cast<const T *>(a.r), *av = static_cast<const T *>(a.v);
    T *ag = static_cast<T *>(a.grad);
    const RowThreshold b = backward_threshold(a.b, a.th);
    const double S_f = a.ctl->persist.S_f, S_vf = a.ctl->persist.S_vf;
    const bool live = S_f > 0.0;
    const float mean = live ? (float)(S_vf / S_f) : 0.f;
    const float h = dead ? __int_as_float(0x7fc00000) : live ? a.half_inv_t * a.gsign : 0.f;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    const unsigned long long gtid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    unsigned long long nvec = 0;
    if ((((uintptr_t)ar | (uintptr_t)av | (uintptr_t)ag) & 15) == 0 && blockDim.x == EW_THREADS) {
        nvec = a.n / V;
        const Vec *r4 = reinterpret_cast<const Vec *>(ar);
        const Vec *v4 = reinterpret_cast<const Vec *>(av);
        Vec *g4 = reinterpret_cast<Vec *>(ag);
        const float2 nhi = dup2(-b.hi), nlo = dup2(-b.lo), cc = dup2(a.c), hh = dup2(h), nmean = dup2(-mean);
        auto map_vec = [&](const Vec &xv, const Vec &wv) {
            float2 x[P], w[P], g[P];
            Io<T>::unpack2(xv, x);
            Io<T>::unpack2(wv, w);
#pragma unroll
            for (int e = 0; e < P; ++e) g[e] = mul2(laplace_pdf2(x[e], nhi, nlo, cc, hh), add2(w[e], nmean));
            return Io<T>::pack2(g);
        };
        // back to front: the reduction pass left the tail of r and v in L2
        const long long ntile = (long long)(nvec / VMAP_TILE), step = (long long)gridDim.x * VMAP_TILE;
        for (long long i = (ntile - 1 - (long long)blockIdx.x) * VMAP_TILE + threadIdx.x; i >= 0; i -= step) {
            Vec x[VMAP_U], w[VMAP_U];
#pragma unroll
            for (int u = 0; u < VMAP_U; ++u) {
                x[u] = io_ldcs<T>(r4 + i + u * EW_THREADS);
                w[u] = io_ldcs<T>(v4 + i + u * EW_THREADS);
            }
#pragma unroll
            for (int u = 0; u < VMAP_U; ++u) io_stcs<T>(g4 + i + u * EW_THREADS, map_vec(x[u], w[u]));
        }
        for (unsigned long long i = (unsigned long long)ntile * VMAP_TILE + gtid; i < nvec; i += stride)
            io_stcs<T>(g4 + i, map_vec(io_ldcs<T>(r4 + i), io_ldcs<T>(v4 + i)));
    }
    for (unsigned long long i = nvec * V + gtid; i < a.n; i += stride)
        Io<T>::store1(ag + i, laplace_pdf(Io<T>::load1(ar + i), b, a.c, h) * (Io<T>::load1(av + i) - mean));
}

// ------------------------------------------------------------ bracket ----
// 32-bit finaliser of MurmurHash3, used as the counter-based generator of the sampler
__host__ __device__ inline uint32_t mix32(uint32_t h)
{
    h ^= h >> 16;
    h *= 0x85ebca6bu;
    h ^= h >> 13;
    h *= 0xc2b2ae35u;
    h ^= h >> 16;
    return h;
}

// Kernel-noised systematic sample (Alg. 1 line 1; the sampler of Sec. 4 and App. D reads the row at a
// stride and adds noise from a table prepared in advance): one draw per stride-long stratum,
// y_s = fma(t, e_s, r[i_s]) with a single fp32 rounding.
template <typename T>
__global__ void sample_gather_kernel(const T *__restrict__ r, long long K, long long stride, uint32_t seed_lo,
                                     const float *__restrict__ noise, float tf, uint32_t *keys_out, float *y_out,
                                     const RowParams *rp)
{
    pdl_wait();
    if (rp) {
        if (!rp->valid) return;
        tf = (float)rp->t;
    }
    const long long s = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= K) return;
    const uint32_t h = mix32((uint32_t)s * 0x9E3779B9u + seed_lo);
    const long long idx = s * stride + (long long)(h % (uint32_t)stride);
    const float y = fmaf(tf, __ldg(noise + s), Io<T>::load1(r + idx));
    keys_out[s] = float_to_key(y);
    if (y_out) y_out[s] = y;
}

// full_sorts mode: the two order statistics (or, where Eq. 8 gives no rank on a side, the sample's extreme there) from
// the sorted sample, left where the radix selection of the default mode leaves them
__global__ void pick_sorted_kernel(const uint32_t *sorted, long long K, long long j, long long l, const RowParams *rp,
                                   Control *ctl)
{
    pdl_wait();
    if (rp) {
        if (!rp->valid) return;
        j = rp->j;
        l = rp->l;
    }
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        ctl->call.sel_keys[0] = sorted[min(max(j, 1ll), K) - 1];
        ctl->call.sel_keys[1] = sorted[min(max(l, 1ll), K) - 1];
    }
}

// ---- one row sharded over several GPUs: the pieces that differ from the single-GPU chain ----
// A shard draws the strata of the systematic sample whose index falls into it; the other strata stay 0 in its copy of
// the key buffer, so that adding the ranks' buffers (each entry is written by exactly one rank) gives the whole sample.
template <typename T>
__global__ void sample_shard_kernel(const T *__restrict__ r_shard, long long shard_begin, long long shard_len, long long K,
                                    long long stride, uint32_t seed_lo, const float *__restrict__ noise, float tf,
                                    uint32_t *keys_out)
{
    pdl_wait();
    const long long s = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= K) return;
    const uint32_t h = mix32((uint32_t)s * 0x9E3779B9u + seed_lo);
    const long long idx = s * stride + (long long)(h % (uint32_t)stride) - shard_begin;
    uint32_t kv = 0u;
    if (idx >= 0 && idx < shard_len) kv = float_to_key(fmaf(tf, __ldg(noise + s), Io<T>::load1(r_shard + idx)));
    keys_out[s] = kv;
}

// Histogram of the top SEL_BITS = 12 bits of the K sample keys (what sample_hist_kernel builds while it draws them)
__global__ void __launch_bounds__(1024) sample_keys_hist_kernel(const uint32_t *__restrict__ keys, long long K, Control *ctl)
{
    pdl_wait();
    __shared__ uint32_t hist[4096];
    for (int i = threadIdx.x; i < 4096; i += blockDim.x) hist[i] = 0;
    __syncthreads();
    const long long s = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (s < K) atomicAdd(&hist[__ldcg(keys + s) >> 20], 1u);
    __syncthreads();
    for (int i = threadIdx.x; i < 4096; i += blockDim.x)
        if (hist[i]) atomicAdd(&ctl->call.sel_hist[i], hist[i]);
}

// The scalar gradients of a sharded row from the sums of all shards (what the last block of vjp_reduce_kernel does
// for a row that lives on one GPU)
__global__ void vjp_scalars_kernel(Control *ctl, double inv_t, float *grad_k, float *grad_alpha)
{
    pdl_wait();
    if (threadIdx.x != 0 || blockIdx.x != 0) return;
    const double pf = ctl->persist.S_f, pv = ctl->persist.S_vf, pd = ctl->persist.S_fd, pvd = ctl->persist.S_vfd;
    const double mean = (pf > 0.0) ? pv / pf : 0.0;
    if (grad_k) *grad_k = (float)mean;
    if (grad_alpha) *grad_alpha = (pf > 0.0) ? (float)((pvd - mean * pd) * inv_t) : 0.f;
}

struct StreamArgs {
    const void *r;  // the row's scores in the workspace's element type
    unsigned long long n;
    const uint32_t *sel;  // two keys: y_(j) and y_(l), or the sample's extreme on a side where Eq. 8 gives no rank (j < 1, l > K):
                          // that end of the bracket is then open and the extreme is where the band's buckets stop
    float fscale;  // fixed-point scale of the bucket sums: fixed_scale(cap)
    long long K, j, l;              // Eq. 8 ranks (1-indexed): decide which ends are open; recorded for lapsum_status
    const RowParams *rp;            // nullable: the row's own ranks and temperature replace j, l, c, sc
    int use_imm;                    // 1: bracket ends given by the host
    float aL_imm, aR_imm;
    float c;                        // log2(e)/t
    ExpScale sc;                    // the same constant split in two floats (accurate exponentials)
    uint32_t *band_keys;            // middle band out (keys)
    uint32_t *band_idx;             // nullable: original indices of the band
    unsigned long long cap;
    double *partials;               // 4 doubles per block: S_L, S_R, |L|, |R|
    Control *ctl;
    BatchShift bs;
};

// the stream pass of row `g` of a group from the arguments of the group's first row
__device__ inline void shift_stream_args(StreamArgs &a, unsigned g, unsigned long long data_bytes)
{
    const unsigned long long ws = g * a.bs.ws_step;
    shift_bytes(a.r, data_bytes);
    shift_bytes(a.sel, ws);
    shift_bytes(a.band_keys, ws);
    shift_bytes(a.band_idx, ws);
    shift_bytes(a.partials, ws);
    shift_bytes(a.ctl, ws);
    if (a.rp) a.rp += g;
    a.bs.active = 0;
}

// One pass over the row (Alg. 1 line 7, Eq. 7): tail sums and counts of
// L = {r < a_L} and R = {r >= a_R}, and compaction of M = {a_L <= r < a_R}.
//
// A score farther than `reach` = 64 t ln2 below a_L (above a_R) would add less than 2^-64 to its tail
// sum and is left out.  This cannot move any p_i by more than n 2^-65 (< 3e-11 for n <= 2^30):
// with A, B' the two sums of the root's interval, u = e^{(b-lo)/t} >= 1 and the budget equation
// A/(2u) - B'u/2 = -c, one has db = t dA / (A + B'u^2) and |dp_i| = min(p_i, 1-p_i) |db| / t, while
// (A + B'u^2)/(2u) = sum_below p_j + sum_above (1-p_j) >= min(p_i, 1-p_i); hence |dp_i| <= dA/(2u)
// <= dA/2, and dA <= (number of dropped scores) 2^-64 because folding a tail into a higher pivot
// only shrinks it.  So only scores inside [a_L - reach, a_R + reach] need arithmetic.
// The common case costs one maximum per score (half of one for 16-bit scores): a lane looks only at the largest of
// its scores.  |L| is not counted: |L| = n - |M| - |R|.
constexpr int SB_THREADS = 512;
constexpr int SB_U = 4;            // 16-byte vectors per thread and tile: 16 fp32 scores, 32 16-bit scores (64 bytes)
constexpr unsigned SB_QCAP = 128;  // band scores a warp queues before it has to flush
constexpr int SB_DENSE_LANES = 12; // more flagged entries (16 scores of a lane) than this in one tile of a warp: every lane classifies its own scores
constexpr int SB_PEND_CAP = 14;    // pending entries per warp: at most 1 left over + SB_DENSE_LANES new ones

template <typename T>
__device__ __forceinline__ void stream_band_body(StreamArgs a);

template <typename T>
__global__ void __launch_bounds__(SB_THREADS, 2) stream_band_kernel(StreamArgs a)
{
    pdl_wait();
    stream_band_body<T>(a);
}

// a group launch (blockIdx.y = row) works on the row's own copy of the arguments
template <typename T>
__global__ void __launch_bounds__(SB_THREADS, 2) stream_band_group_kernel(StreamArgs a)
{
    pdl_wait();
    StreamArgs mine = a;
    shift_stream_args(mine, blockIdx.y, blockIdx.y * a.bs.row_step * sizeof(T));
    stream_band_body<T>(mine);
}

template <typename T>
__device__ __forceinline__ void stream_band_body(StreamArgs a)
{
    constexpr int V = Io<T>::V;
    constexpr int ELEMS = 16;         // scores of one pending entry: half a warp's worth
    constexpr int EV = ELEMS / V;     // vectors of an entry (4 of fp32, 2 of 16-bit scores)
    constexpr int SUB = SB_U / EV;    // entries a thread holds per tile (1 or 2)
    constexpr int EPC = 32 / ELEMS;   // pending entries the warp works off per round (one score per lane)
    using Vec = typename Io<T>::Vec;
    const T *row = static_cast<const T *>(a.r);
    if (a.rp) {
        if (!a.rp->valid) return;
        a.j = a.rp->j;
        a.l = a.rp->l;
        a.c = a.rp->c;
        a.sc = a.rp->sc;
    }
    __shared__ double red[32];
    __shared__ long long redl[32];
    __shared__ int is_last;
    __shared__ uint32_t wq[SB_THREADS / 32][SB_QCAP];
    __shared__ unsigned wcnt[SB_THREADS / 32], woff[SB_THREADS / 32];
    __shared__ unsigned long long block_base;
    __shared__ Vec pend_buf[SB_THREADS / 32][SB_PEND_CAP][EV];
    if (threadIdx.x < SB_THREADS / 32) wcnt[threadIdx.x] = 0;
    __syncthreads();
    float a_L, a_R;
    unsigned long long gl, gh;
    if (a.use_imm) {
        a_L = a.aL_imm;
        a_R = a.aR_imm;
        gl = float_to_key(a_L);
        gh = float_to_key(a_R);
    } else {
        const uint32_t kL = __ldcg(a.sel), kR = __ldcg(a.sel + 1);
        const bool open_L = a.j < 1, open_R = a.l > a.K;
        a_L = open_L ? -CUDART_INF_F : key_to_float(kL);
        a_R = open_R ? CUDART_INF_F : key_to_float(kR);
        gl = kL;
        gh = open_R ? (unsigned long long)kR + 1ull : (unsigned long long)kR;
    }
    const BandGrid grid = bracket_grid(a_L, a_R, gl, gh);
    const float fscale = a.fscale;
    const float reach = 64.f / a.c;  // terms below 2^-64 are dropped (bound on the effect: see above)
    const float far_L = a_L - reach;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const unsigned lt_mask = (1u << lane) - 1u;
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    const unsigned long long gtid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    float sL = 0.f, sR = 0.f;
    unsigned cR = 0;

    // One score, branch-free: a score outside the band adds its term to the tail on its side (Eq. 7); returns true for
    // a band score.  dL > 0: below the band, dR >= 0: above it; the term is e^{-distance to the band / t}.
    auto tally = [&](float x, bool live) -> bool {
        const float dL = a_L - x, dR = x - a_R;
        const float e = ex2_approx(-fmaxf(dL, dR) * a.c);
        const bool inL = dL > 0.f, inR = dR >= 0.f;
        if (live && inL) sL += e;
        if (live && inR) {
            sR += e;
            ++cR;
        }
        return live && !inL && !inR;
    };
    // Append of at most one band score per lane (all lanes of the warp call this together).  Band
    // scores collect in a per-warp queue in shared memory; the block reserves its share of the band
    // buffer with ONE atomic at the end of the kernel (a full queue is flushed early with its own
    // atomic), so the single band counter sees about one atomic per block instead of one per score.
    auto flush_warp = [&](unsigned cnt) {
        unsigned long long base = 0;
        if (lane == 0) base = atomicAdd(&a.ctl->call.band_count, (unsigned long long)cnt);
        base = __shfl_sync(FULL, base, 0);
        for (unsigned i = lane; i < cnt; i += 32)
            if (base + i < a.cap && LAPSUM_IN_BOUNDS(i, SB_QCAP, a.ctl)) a.band_keys[base + i] = wq[warp][i];
        __syncwarp();
    };
    auto append = [&](float x, bool has) {
        const unsigned votes = __ballot_sync(FULL, has);
        if (!votes) return;
        const unsigned nb = __popc(votes);
        unsigned cnt = wcnt[warp];
        if (cnt + nb > SB_QCAP) {
            flush_warp(cnt);
            cnt = 0;
        }
        if (has) {
            const uint32_t kv = float_to_key(x);
            const unsigned qpos = cnt + __popc(votes & lt_mask);
            if (LAPSUM_IN_BOUNDS(qpos, SB_QCAP, a.ctl)) wq[warp][qpos] = kv;
            // first-level bucket of the band solve: count and the two sums pivoted at the bucket's edges
            const int bkt = grid.bucket(kv);
            if (LAPSUM_IN_BOUNDS(bkt, BAND_BUCKETS, a.ctl)) {
                atomicAdd(&a.ctl->call.band_cnt[bkt], 1u);
                atomicAdd(&a.ctl->call.band_up[bkt], (unsigned long long)__float2ll_rn(decay(grid.edge(bkt + 1) - x, a.sc) * fscale));
                atomicAdd(&a.ctl->call.band_down[bkt], (unsigned long long)__float2ll_rn(decay(x - grid.edge(bkt), a.sc) * fscale));
            }
        }
        __syncwarp();
        if (lane == 0) wcnt[warp] = cnt + nb;
        __syncwarp();
    };

    // The row is walked in tiles of SB_THREADS * SB_U vectors, handed to the blocks round-robin; thread t takes
    // vectors t, t + SB_THREADS, ... of the tile: 64 bytes of scores, in entries of 16 scores.  Nearly all of them lie
    // below far_L and need nothing: a lane finds that out from the maximum of an entry (for 16-bit scores the maximum
    // is taken on packed pairs in the storage type, which commutes with the exact conversion to fp32).  An entry whose
    // maximum reaches far_L is `flagged`.  Few flagged entries: the lane parks the entry's raw bytes in the warp's
    // pending list in shared memory, and the warp works that list off 32 scores at a time, one per lane, with every
    // lane busy.  Many flagged entries (a wide kernel, or a bracket in the bulk of the scores): every lane classifies
    // its own scores from registers, branch-free.
    constexpr unsigned TILE = SB_THREADS * SB_U;
    unsigned pend = 0;  // entries in this warp's pending list (the same in all lanes)
    const T *pend_elems = reinterpret_cast<const T *>(&pend_buf[warp][0][0]);

    // classify + append the scores of `count` <= EPC pending entries from entry e0 on
    auto work_off = [&](unsigned e0, unsigned count) {
        const bool live = (unsigned)(lane / ELEMS) < count;
        // lane / ELEMS selects the entry, lane % ELEMS the score (a read past `count` entries stays inside the list)
        const float x = Io<T>::from_storage(pend_elems[e0 * ELEMS + lane]);
        append(x, tally(x, live));
    };
    auto dense = [&](const Vec (&q)[SB_U], const T *base) {
        unsigned bandbits = 0;
#pragma unroll
        for (int u = 0; u < SB_U; ++u) {
            float x[V];
            Io<T>::unpack(q[u], x);
#pragma unroll
            for (int w = 0; w < V; ++w)
                if (tally(x[w], true)) bandbits |= 1u << (u * V + w);
        }
        while (__any_sync(FULL, bandbits != 0)) {  // append band scores, one per lane and round
            const bool has = bandbits != 0;
            const int e = has ? __ffs(bandbits) - 1 : 0;
            bandbits &= bandbits - 1u;
            const float xb = has ? Io<T>::load1(base + (unsigned)(e / V) * (SB_THREADS * V) + (e % V)) : 0.f;  // L1 hit
            append(xb, has);
        }
    };
    auto body = [&](const Vec (&q)[SB_U], const T *base) {
        bool flag[SUB];
        unsigned votes[SUB], total = 0;
#pragma unroll
        for (int h = 0; h < SUB; ++h) {
            flag[h] = Io<T>::template max_of<EV>(&q[h * EV]) >= far_L;
            votes[h] = __ballot_sync(FULL, flag[h]);
            total += __popc(votes[h]);
        }
        if (!total) return;
        if (total > SB_DENSE_LANES) {
            dense(q, base);
            return;
        }
#pragma unroll
        for (int h = 0; h < SUB; ++h) {
            if (flag[h]) {
                const unsigned slot = pend + __popc(votes[h] & lt_mask);
                if (LAPSUM_IN_BOUNDS(slot, SB_PEND_CAP, a.ctl)) {
#pragma unroll
                    for (int u = 0; u < EV; ++u) pend_buf[warp][slot][u] = q[h * EV + u];
                }
            }
            pend += __popc(votes[h]);
        }
        __syncwarp();
        while (pend >= EPC) {
            pend -= EPC;
            work_off(pend, EPC);
        }
    };

    unsigned long long done = 0;  // scores handled by the tile loop
    if (((uintptr_t)row & 15) == 0) {
        const Vec *r4 = reinterpret_cast<const Vec *>(row);
        const unsigned long long ntile = a.n / V / TILE, step = (unsigned long long)gridDim.x * TILE, end = ntile * TILE;
        done = end * V;
        Vec qa[SB_U], qb[SB_U];
        auto fetch = [&](Vec (&q)[SB_U], unsigned long long i) {
#pragma unroll
            for (int u = 0; u < SB_U; ++u) q[u] = io_ldg<T>(r4 + i + u * SB_THREADS);
        };
        unsigned long long i = (unsigned long long)blockIdx.x * TILE + threadIdx.x;
        if (i < end) {  // two tiles per thread in flight: the next one is requested before this one is looked at
            fetch(qa, i);
            for (;;) {
                const T *base = reinterpret_cast<const T *>(r4 + i);
                i += step;
                if (i < end) fetch(qb, i);
                body(qa, base);
                if (i >= end) break;
                base = reinterpret_cast<const T *>(r4 + i);
                i += step;
                if (i < end) fetch(qa, i);
                body(qb, base);
                if (i >= end) break;
            }
        }
        if (pend) work_off(0, pend);
    }
    {   // what the tiles leave over (less than one tile), or the whole row when it is not 16-byte aligned: one score
        // per lane and round
        const unsigned long long rest = a.n - done;
        const unsigned long long nround = (rest + 31) / 32 * 32;
        for (unsigned long long i = gtid; i < nround; i += stride) {
            const bool live = i < rest;
            const float x = live ? Io<T>::load1(row + done + i) : 0.f;
            append(x, tally(x, live));
        }
    }
    // hand the queued band scores over: one reservation per block
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned tot = 0;
        for (int w = 0; w < SB_THREADS / 32; ++w) { woff[w] = tot; tot += wcnt[w]; }
        block_base = tot ? atomicAdd(&a.ctl->call.band_count, (unsigned long long)tot) : 0ull;
    }
    __syncthreads();
    for (unsigned i = lane; i < wcnt[warp]; i += 32) {
        const unsigned long long pos = block_base + woff[warp] + i;
        if (pos < a.cap && LAPSUM_IN_BOUNDS(i, SB_QCAP, a.ctl)) a.band_keys[pos] = wq[warp][i];
    }
    const double S_L = block_sum((double)sL, red);
    const double S_R = block_sum((double)sR, red);
    const long long N_R = block_sum((long long)cR, redl);
    if (threadIdx.x == 0) {
        double *o = a.partials + 4 * (size_t)blockIdx.x;
        o[0] = S_L;
        o[1] = S_R;
        o[2] = 0.0;
        o[3] = (double)N_R;  // exact: counts stay far below 2^53
        __threadfence();
        const unsigned t = atomicAdd(&a.ctl->call.stream_ticket, 1u);
        is_last = (t == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    double p0 = 0.0, p1 = 0.0, p2 = 0.0, p3 = 0.0;
    for (unsigned i = threadIdx.x; i < gridDim.x; i += blockDim.x) {
        p0 += __ldcg(a.partials + 4 * i);
        p1 += __ldcg(a.partials + 4 * i + 1);
        p2 += __ldcg(a.partials + 4 * i + 2);
        p3 += __ldcg(a.partials + 4 * i + 3);
    }
    p0 = block_sum(p0, red);
    p1 = block_sum(p1, red);
    p2 = block_sum(p2, red);
    p3 = block_sum(p3, red);
    if (threadIdx.x == 0) {
        CallCtl &c = a.ctl->call;
        c.S_L = p0;
        c.S_R = p1;
        const unsigned long long n_M = *((volatile unsigned long long *)&c.band_count);
        c.n_R = (unsigned long long)p3;
        c.n_L = a.n - n_M - c.n_R;
        (void)p2;
        c.a_L = a_L;
        c.a_R = a_R;
        c.grid_klo = grid.klo;
        c.grid_khi = grid.khi;
        PersistCtl &ps = a.ctl->persist;
        ps.S_L = p0;
        ps.S_R = p1;
        ps.n_L = c.n_L;
        ps.n_R = c.n_R;
        ps.n_M = n_M;
        ps.a_L = a_L;
        ps.a_R = a_R;
        ps.K = a.K;
        ps.j = a.j;
        ps.l = a.l;
    }
}

}  // namespace lapsum
