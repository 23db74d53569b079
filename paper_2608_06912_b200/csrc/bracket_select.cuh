// Fast forms of the two small sorts of the bracket path (Alg. 1):
//   sample_select : the bracket needs only two order statistics y_(j), y_(l) of the K noised
//                   samples, so they are found by radix selection instead of sorting the sample;
//   band_solve    : the middle band M is bucketed by key range, the buckets' (pivot, sum)
//                   aggregates give the budget curve at the bucket edges, and only the three
//                   buckets around the root enter the exact interval solve (by all pairs when
//                   they hold at most 256 scores, sorted otherwise).
// Both give exactly the values the full sorts give (same order statistics, same root).
#pragma once
#include "common.cuh"
#include "global_path.cuh"
#include "solve.cuh"

namespace lapsum {

constexpr int SEL_BITS = 12;
constexpr int SEL_BINS = 1 << SEL_BITS;
constexpr int SEL_THREADS = 1024;
constexpr int SEL_SHORT = 256;  // a candidate list this short is ranked by counting; longer ones descend another digit

struct SelectArgs {
    const void *r;  // the row's scores in the workspace's element type
    long long K, stride;
    uint32_t seed_lo;
    const float *noise;
    float tf;
    uint32_t *keys;  // K keys of the noised sample (draw order)
    float *y_out;    // nullable
    long long j, l;  // 1-indexed ranks wanted (ignored when < 1 / > K)
    Control *ctl;
    const RowParams *rp;  // nullable: the row's own temperature replaces tf
    BatchShift bs;
};

// Smallest bin whose inclusive count reaches `want` (1-indexed rank) in hist[0..SEL_BINS); returns the bin and
// the count before it through out[1], out[2].  One block of SEL_THREADS threads, four bins per thread.
__device__ inline void find_bin(const uint32_t *hist, long long want, uint32_t *out, uint32_t *warp_tot /*32*/)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint32_t h[4], c = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) { h[q] = hist[4 * tid + q]; c += h[q]; }
    uint32_t incl = c;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const uint32_t t1 = __shfl_up_sync(FULL, incl, o);
        if (lane >= o) incl += t1;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    uint32_t off = 0;
    for (int w = 0; w < warp; ++w) off += warp_tot[w];
    const long long hi = (long long)off + incl, lo = hi - c;
    if (lo < want && want <= hi) {
        long long acc = lo;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            if (acc + h[q] >= want) { out[1] = 4 * tid + q; out[2] = (uint32_t)acc; break; }
            acc += h[q];
        }
    }
    __syncthreads();
}

// Rank `want` (1-indexed) among the keys of `keys[0..K)` whose top `known_bits` bits equal `prefix`;
// `cnt` = how many such keys there are.  One block; re-reads the key buffer (L2 resident) once per level:
// while there are more candidates than SEL_SHORT, histogram their next digit and descend into the bin that holds
// the rank (its count is the next level's `cnt`); then collect them and pick the rank by counting.
__device__ inline uint32_t select_refine(const uint32_t *keys, long long K, uint32_t prefix, int known_bits,
                                         long long want, long long cnt, uint32_t *hist /*SEL_BINS*/,
                                         uint32_t *list /*SEL_SHORT*/, uint32_t *sh_scalar /*4*/, uint32_t *warp_tot /*32*/)
{
    const int tid = threadIdx.x;
    while (cnt > SEL_SHORT) {
        if (known_bits >= 32) return prefix;  // more equal keys than the list holds: the key is fully known
        const int d = min(SEL_BITS, 32 - known_bits);
        for (int i = tid; i < SEL_BINS; i += blockDim.x) hist[i] = 0;
        __syncthreads();
        for (long long i = tid; i < K; i += blockDim.x) {
            const uint32_t kv = __ldcg(keys + i);
            if (known_bits == 0 || (kv >> (32 - known_bits)) == prefix)
                atomicAdd(&hist[(kv >> (32 - known_bits - d)) & ((1u << d) - 1)], 1u);
        }
        __syncthreads();
        find_bin(hist, want, sh_scalar, warp_tot);
        prefix = (prefix << d) | sh_scalar[1];
        want -= sh_scalar[2];
        cnt = hist[sh_scalar[1]];
        known_bits += d;
        __syncthreads();
    }
    if (tid == 0) sh_scalar[0] = 0;
    __syncthreads();
    for (long long i = tid; i < K; i += blockDim.x) {
        const uint32_t kv = __ldcg(keys + i);
        if (known_bits == 0 || (kv >> (32 - known_bits)) == prefix) {
            const uint32_t pos = atomicAdd(&sh_scalar[0], 1u);
            if (pos < SEL_SHORT) list[pos] = kv;
        }
    }
    __syncthreads();
    const int m = (int)min(sh_scalar[0], (uint32_t)SEL_SHORT);
    __syncthreads();
    if (tid < m) {  // thread i takes candidate i and counts the candidates that order before it
        const uint32_t mine = list[tid];
        int before = 0;
#pragma unroll 1
        for (int j = 0; j < m; ++j) {
            const uint32_t o = list[j];
            before += (o < mine || (o == mine && j < tid)) ? 1 : 0;
        }
        if (before == (int)want - 1) sh_scalar[3] = mine;
    }
    __syncthreads();
    const uint32_t out = sh_scalar[3];
    __syncthreads();
    return out;
}

// Step 1 of the selection: draw the K kernel-noised samples (one per stratum,
// y_s = fma(t, e_s, r[i_s])), store their keys and histogram the keys' top 12 bits.
// GROUP: a launch for a group of rows (BatchShift; blockIdx.y = row); a kernel of its own so that the one-row launch
// does not pay for the moved pointers
template <typename T, bool GROUP>
__global__ void __launch_bounds__(SEL_THREADS) sample_hist_kernel(SelectArgs a)
{
    pdl_wait();
    if (GROUP) {
        const unsigned g = blockIdx.y;
        const unsigned long long ws = g * a.bs.ws_step;
        shift_bytes(a.r, g * a.bs.row_step * sizeof(T));
        shift_bytes(a.noise, ws);
        shift_bytes(a.keys, ws);
        shift_bytes(a.ctl, ws);
        if (a.rp) a.rp += g;
    }
    if (a.rp) {
        if (!a.rp->valid) return;
        a.tf = (float)a.rp->t;
    }
    __shared__ uint32_t hist[SEL_BINS];
    const int tid = threadIdx.x, lane = tid & 31;
    for (int i = tid; i < SEL_BINS; i += SEL_THREADS) hist[i] = 0;
    __syncthreads();
    const long long s = (long long)blockIdx.x * SEL_THREADS + tid;
    uint32_t bin = 0xffffffffu;
    if (s < a.K) {
        const uint32_t h = mix32((uint32_t)s * 0x9E3779B9u + a.seed_lo);
        const long long idx = s * a.stride + (long long)(h % (uint32_t)a.stride);
        const float y = fmaf(a.tf, __ldg(a.noise + s), Io<T>::load1(static_cast<const T *>(a.r) + idx));
        const uint32_t kv = float_to_key(y);
        a.keys[s] = kv;
        if (a.y_out) a.y_out[s] = y;
        bin = kv >> (32 - SEL_BITS);
    }
    // sample values cluster in a few top-bit bins: one shared-memory atomic per distinct bin and warp
    const unsigned peers = match_bits<13>(bin & 0x1fffu);  // bit 12 is set only for the padding lanes
    if (bin != 0xffffffffu && (peers & ((1u << lane) - 1u)) == 0) atomicAdd(&hist[bin], (uint32_t)__popc(peers));
    __syncthreads();
    for (int i = tid; i < SEL_BINS; i += SEL_THREADS)
        if (hist[i]) atomicAdd(&a.ctl->call.sel_hist[i], hist[i]);
}

// Step 2: every block finds the two histogram bins that hold ranks j and l (Eq. 8), filters its share of
// the keys into two candidate lists in global memory; the last block to finish picks the two ranks among the
// candidates (by counting, after further digits if a list is long) and leaves the keys of y_(j) and y_(l) in
// ctl->call.sel_keys.  A rank that Eq. 8 puts outside 1..K is replaced by the sample's extreme on that side.
struct PickArgs {
    const uint32_t *keys;
    uint32_t *cand;   // 2 x cand_cap candidate keys
    long long K, j, l, cand_cap;
    Control *ctl;
    const RowParams *rp;  // nullable: the row's own ranks replace j, l
    BatchShift bs;
};

template <bool GROUP>
__global__ void __launch_bounds__(SEL_THREADS) sample_pick_kernel(PickArgs a)
{
    pdl_wait();
    if (GROUP) {
        const unsigned g = blockIdx.y;
        const unsigned long long ws = g * a.bs.ws_step;
        shift_bytes(a.keys, ws);
        shift_bytes(a.cand, ws);
        shift_bytes(a.ctl, ws);
        if (a.rp) a.rp += g;
    }
    if (a.rp) {
        if (!a.rp->valid) return;
        a.j = a.rp->j;
        a.l = a.rp->l;
    }
    __shared__ uint32_t hist[SEL_BINS];
    __shared__ uint32_t list[2 * SEL_SHORT];
    __shared__ uint32_t scal[4];
    __shared__ uint32_t warp_tot[32];
    __shared__ int is_last;
    const int tid = threadIdx.x;
    for (int i = tid; i < SEL_BINS; i += SEL_THREADS) hist[i] = __ldcg(&a.ctl->call.sel_hist[i]);
    __syncthreads();
    // a rank outside 1..K means that end of the bracket is open; the sample's extreme is found in its place
    // (it bounds the key range that the band's buckets have to cover)
    const long long ranks[2] = {min(max(a.j, 1ll), a.K), min(max(a.l, 1ll), a.K)};
    uint32_t bin0[2];
    long long rest[2];
    {   // both bins from one scan of the histogram (four bins per thread)
        const int lane = tid & 31, warp = tid >> 5;
        uint32_t h[4], csum = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) { h[q] = hist[4 * tid + q]; csum += h[q]; }
        uint32_t incl = csum;
#pragma unroll 1
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t1 = __shfl_up_sync(FULL, incl, o);
            if (lane >= o) incl += t1;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        uint32_t off = 0;
        for (int w = 0; w < warp; ++w) off += warp_tot[w];
        const long long hi = (long long)off + incl, lo = hi - csum;
#pragma unroll
        for (int which = 0; which < 2; ++which) {
            const long long want = ranks[which];
            if (lo < want && want <= hi) {
                long long acc = lo;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    if (acc + h[q] >= want) { scal[2 * which] = 4 * tid + q; scal[2 * which + 1] = (uint32_t)acc; break; }
                    acc += h[q];
                }
            }
        }
        __syncthreads();
#pragma unroll
        for (int which = 0; which < 2; ++which) {
            bin0[which] = scal[2 * which];
            rest[which] = ranks[which] - (long long)scal[2 * which + 1];
        }
        __syncthreads();  // scal is reused below
    }
    // this block's contiguous share of the keys, 128-bit loads
    auto push = [&](uint32_t kv) {
        const uint32_t top = kv >> (32 - SEL_BITS);
#pragma unroll
        for (int which = 0; which < 2; ++which) {
            if (top == bin0[which]) {
                const uint32_t pos = atomicAdd(&a.ctl->call.sel_cand[which], 1u);
                if ((long long)pos < a.cand_cap && LAPSUM_IN_BOUNDS((long long)which * a.cand_cap + pos, 2 * a.cand_cap, a.ctl))
                    a.cand[(long long)which * a.cand_cap + pos] = kv;
            }
        }
    };
    {
        const long long nvec = a.K / 4;
        const long long per = (nvec + gridDim.x - 1) / gridDim.x;
        const long long v0 = (long long)blockIdx.x * per, v1 = min(nvec, v0 + per);
        const uint4 *k4 = reinterpret_cast<const uint4 *>(a.keys);
        constexpr int U = 4;
        for (long long base = v0; base < v1; base += (long long)SEL_THREADS * U) {
            uint4 q[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long i = base + (long long)u * SEL_THREADS + tid;
                q[u] = (i < v1) ? __ldcg(k4 + i) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (base + (long long)u * SEL_THREADS + tid >= v1) continue;
                push(q[u].x); push(q[u].y); push(q[u].z); push(q[u].w);
            }
        }
        if (blockIdx.x == 0)
            for (long long i = nvec * 4 + tid; i < a.K; i += SEL_THREADS) push(__ldcg(a.keys + i));
    }
    __syncthreads();
    if (tid == 0) {
        __threadfence();
        is_last = (atomicAdd(&a.ctl->call.sel_ticket, 1u) == gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    uint32_t *lists[2] = {list, list + SEL_SHORT};
    const uint32_t cnts[2] = {*((volatile uint32_t *)&a.ctl->call.sel_cand[0]), *((volatile uint32_t *)&a.ctl->call.sel_cand[1])};
    if (max(cnts[0], cnts[1]) <= SEL_SHORT && (long long)max(cnts[0], cnts[1]) <= a.cand_cap) {
        // short candidate lists (the usual case): the wanted rank by counting, both lists at once, no sort.
        // Thread i of each half takes candidate i and counts the candidates that order before it.
        const int which = tid / SEL_SHORT, i = tid % SEL_SHORT;
        const int cnt = (tid < 2 * SEL_SHORT) ? (int)(which ? cnts[1] : cnts[0]) : 0;
        uint32_t *mylist = list + which * SEL_SHORT;
        if (i < cnt) mylist[i] = __ldcg(a.cand + (long long)which * a.cand_cap + i);
        __syncthreads();
        if (i < cnt) {
            const uint32_t mine = mylist[i];
            int before = 0;
#pragma unroll 1
            for (int j = 0; j < cnt; ++j) {
                const uint32_t o = mylist[j];
                before += (o < mine || (o == mine && j < i)) ? 1 : 0;
            }
            if (before == (int)(which ? rest[1] : rest[0]) - 1) a.ctl->call.sel_keys[which] = mine;
        }
        return;
    }
    for (int which = 0; which < 2; ++which) {
        uint32_t kv;
        const uint32_t cnt = cnts[which];
        if ((long long)cnt <= a.cand_cap) {
            // more candidates than the shared-memory list holds: descend digit by digit over the candidate list
            kv = select_refine(a.cand + (long long)which * a.cand_cap, (long long)cnt, bin0[which], SEL_BITS, rest[which],
                               (long long)cnt, hist, lists[which], scal, warp_tot);
        } else {
            // the candidate list itself overflowed (nearly all keys share their top bits): descend over all keys
            kv = select_refine(a.keys, a.K, bin0[which], SEL_BITS, rest[which], (long long)cnt, hist, lists[which], scal,
                               warp_tot);
        }
        if (tid == 0) a.ctl->call.sel_keys[which] = kv;
        __syncthreads();
    }
}

// ------------------------------------------------------------ band solve ----
constexpr int BAND_LIST = 2048;
constexpr int BAND_LEVELS = 5;

struct BandArgs {
    const uint32_t *band;  // |M| keys in arbitrary order
    Control *ctl;
    float *b_out;
    RowThreshold *th_out;
    unsigned long long cap;
    double k, t;
    ExpScale sc;
    float c;  // log2(e)/t for the coarse (bucket-level) sums of the deeper levels
    float fscale;  // fixed-point scale of the stream pass's bucket sums (a power of two)
    uint32_t *glist;  // BAND_LIST keys in global memory: where the blocks of a multi-block launch gather to
    FallbackPlan fb;  // the full-sort chain to launch if the certificate fails
    // validated widening (App. C): another stream pass over a bracket doubled on the failing side
    StreamArgs stream;  // the stream pass as the host launched it
    int stream_grid, solve_blocks;
    int attempt, max_widen;
    const RowParams *rp;  // nullable: the row's own budget and temperature replace k, t, sc, c
    int io;               // element type of the scores (lapsum_io_dtype): which stream pass a widened attempt launches
    BatchShift bs;
};

struct BucketItems {
    static constexpr bool PAD = false;
    const float *edge;               // BAND_BUCKETS + 1 edges (values)
    const float *sum_up, *sum_down;  // pivoted sums of each bucket (upper edge / lower edge)
    const unsigned *cum;             // inclusive cumulative counts
    __device__ float first(int i) const { return edge[i]; }
    __device__ float last(int i) const { return edge[i + 1]; }
    __device__ float up(int i) const { return sum_up[i]; }
    __device__ float down(int i) const { return sum_down[i]; }
    __device__ long long end(int i) const { return cum[i]; }
};

// Buckets one key wide: every bucket is a run of equal scores (value = its edge, multiplicity = its count)
struct TieItems {
    static constexpr bool PAD = false;
    const float *edge;
    const unsigned *cum;
    __device__ float first(int i) const { return edge[i]; }
    __device__ float last(int i) const { return edge[i]; }
    __device__ float up(int i) const { return (float)(cum[i] - (i ? cum[i - 1] : 0u)); }
    __device__ float down(int i) const { return up(i); }
    __device__ long long end(int i) const { return cum[i]; }
};

// Apply f to every key of part `part` of `nparts` of band[0..M): 128-bit loads, four in flight per thread.
template <typename F>
__device__ __forceinline__ void for_each_band_key(const uint32_t *band, long long M, F f, int part = 0, int nparts = 1)
{
    const int tid = threadIdx.x, T = blockDim.x;
    const long long nvec = (((uintptr_t)band & 15) == 0) ? M / 4 : 0;
    const long long per = (nvec + nparts - 1) / nparts;
    const long long v0 = min(nvec, (long long)part * per), v1 = min(nvec, v0 + per);
    const uint4 *b4 = reinterpret_cast<const uint4 *>(band);
    constexpr int U = 4;
    for (long long base = v0; base < v1; base += (long long)T * U) {
        uint4 q[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long i = base + (long long)u * T + tid;
            q[u] = (i < v1) ? __ldg(b4 + i) : make_uint4(0xffffffffu, 0xffffffffu, 0xffffffffu, 0xffffffffu);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (base + (long long)u * T + tid >= v1) continue;
            f(q[u].x); f(q[u].y); f(q[u].z); f(q[u].w);
        }
    }
    if (part == nparts - 1)
        for (long long i = nvec * 4 + tid; i < M; i += T) f(__ldg(band + i));
}

struct __align__(16) BandShared {
    unsigned fx_up[BAND_BUCKETS], fx_down[BAND_BUCKETS];  // coarse sums of the deeper levels, 32-bit fixed point
    unsigned cnt[BAND_BUCKETS];
    float edge[BAND_BUCKETS + 1];
    float up[BAND_BUCKETS], down[BAND_BUCKETS];
    float pref[BAND_BUCKETS], suf[BAND_BUCKETS];
    uint32_t list[BAND_LIST], list2[BAND_LIST];
    float pref2[BAND_LIST], suf2[BAND_LIST];
    ScanShared sh;
    long long sh_fx[2][32];
    unsigned sh_cnt;
    // first level, one bucket per thread: warp totals of the three scans, of the crossing and of the tails
    Agg w_up[32], w_down[32];
    unsigned w_cnt[32];
    int w_j[32];
    double w_tail[2][32];
    long long cum_at[2];  // scores below bucket lo_i / up to bucket hi_i - 1
    int is_last;
    PairsShared pairs;
};

// Exact solve over the middle band without sorting all of it.
//  A level cuts the unresolved key range [klo, khi) into <= 1024 buckets of 2^shift keys.  Each bucket
//  has a count and two pivoted exponential sums (pivots = its edges); a block scan of those aggregates
//  gives the budget curve at every edge and the bucket J that holds the root.  Buckets J-1..J+1 stay
//  unresolved (bucket sums are only trusted to +-1 bucket), everything else is folded into the tails,
//  re-summed about the new range ends.  When the unresolved scores fit the list they are gathered
//  and solved exactly (App. B): by all pairs up to 256 scores, after one more bucketing of the list
//  itself in shared memory, or sorted by the block; otherwise the next level cuts the range again;
//  buckets one key wide are runs of equal scores and are solved as they are.
//  The first level's buckets were filled by the stream pass while it found the band; levels that
//  do not fit the list (rare: more than 2048 scores within three buckets) re-read the band.
//  Every sum over band scores is integer fixed point: the band's arbitrary order cannot change a bit.
__global__ void band_solve_kernel(const __grid_constant__ BandArgs a);

// The certificate failed on one side: widen there and run stream pass + band solve once more (from the device).
// Returns false when widening is not possible any more; the caller then launches the full sort.
__device__ inline bool launch_widened_attempt(const BandArgs &a, int status_bits)
{
    if (a.attempt >= a.max_widen) return false;
    CallCtl &c = a.ctl->call;
    const float aL = c.a_L, aR = c.a_R;
    const bool both = aL > -CUDART_INF_F && aR < CUDART_INF_F;
    float w = both ? aR - aL : 0.f;
    if (!(w > 0.f)) w = (float)a.t;  // an empty or open-ended bracket has no width of its own: the temperature stands in
    float nL, nR;
    if (status_bits & (int)ST_ROOT_RIGHT) {
        if (!(aR < CUDART_INF_F)) return false;
        nL = aR;
        nR = aR + 2.f * w;
    } else {
        if (!(aL > -CUDART_INF_F)) return false;
        nR = aL;
        nL = aL - 2.f * w;
    }
    if (!(nL < nR)) return false;
    // fresh per-attempt state (the children start after this grid has completed)
    c.band_count = 0;
    c.stream_ticket = 0;
    c.solve_ticket = 0;
    c.solve_list_cnt = 0;
    for (int i = 0; i < BAND_BUCKETS; ++i) { c.band_cnt[i] = 0; c.band_up[i] = 0; c.band_down[i] = 0; }
    atomicAdd(&a.ctl->persist.widenings, 1ull);
    set_status(a.ctl, 0x40u | (unsigned)status_bits);
    StreamArgs sa = a.stream;
    sa.use_imm = 1;
    sa.aL_imm = nL;
    sa.aR_imm = nR;
    if (a.io == 1) stream_band_kernel<__half><<<a.stream_grid, SB_THREADS, 0, cudaStreamTailLaunch>>>(sa);
    else if (a.io == 2) stream_band_kernel<__nv_bfloat16><<<a.stream_grid, SB_THREADS, 0, cudaStreamTailLaunch>>>(sa);
    else stream_band_kernel<float><<<a.stream_grid, SB_THREADS, 0, cudaStreamTailLaunch>>>(sa);
    if (cudaGetLastError() != cudaSuccess) return false;
    BandArgs next = a;
    next.attempt = a.attempt + 1;
    band_solve_kernel<<<a.solve_blocks, 1024, sizeof(BandShared), cudaStreamTailLaunch>>>(next);
    return cudaGetLastError() == cudaSuccess;  // a refused launch leaves the full sort to the caller
}

// The row a block of the band solve works for: the pointers of the launch arguments, moved to the block's row when the
// launch serves a group of rows (BatchShift).  The launch arguments themselves stay where the launch put them; only
// the rare repairs (widened attempt, full sort) make a row's own copy of all of them.
struct BandRow {
    const uint32_t *band;
    uint32_t *glist;
    Control *ctl;
    float *b_out;
    RowThreshold *th_out;
    const RowParams *rp;
    unsigned g;  // row within the group
};

template <bool GROUP>
__device__ __forceinline__ BandRow band_row(const BandArgs &a)
{
    BandRow w{a.band, a.glist, a.ctl, a.b_out, a.th_out, a.rp, 0u};
    if (GROUP) {
        w.g = blockIdx.y;
        const unsigned long long ws = w.g * a.bs.ws_step;
        shift_bytes(w.band, ws);
        shift_bytes(w.glist, ws);
        shift_bytes(w.ctl, ws);
        if (w.b_out) w.b_out += w.g;
        if (w.th_out) w.th_out += w.g;
        if (w.rp) w.rp += w.g;
    }
    return w;
}

// the row's own copy of all launch arguments (for what the row launches itself)
__device__ inline void band_args_of_row(const BandArgs &a, const BandRow &w, BandArgs *out)
{
    *out = a;
    const unsigned long long ws = w.g * a.bs.ws_step, data = w.g * a.bs.row_step * (a.io == 0 ? 4ull : 2ull);
    out->band = w.band;
    out->glist = w.glist;
    out->ctl = w.ctl;
    out->b_out = w.b_out;
    out->th_out = w.th_out;
    out->rp = w.rp;
    shift_plan(out->fb, w.g, ws, data);
    shift_stream_args(out->stream, w.g, data);
    out->bs.active = 0;
}

// The certificate failed, or the band overflowed (status_bits = 0x2): widen the bracket if that is still allowed, else
// run the full sort.  One thread; `a` holds the row's own arguments.
__device__ inline void band_repair_row(const BandArgs &a, int status_bits, bool may_widen)
{
    if (may_widen && launch_widened_attempt(a, status_bits)) return;
    a.ctl->call.fallback = 1;
    set_status(a.ctl, 0x1u | (unsigned)status_bits);
    atomicAdd(&a.ctl->persist.fallbacks, 1ull);
    if (a.fb.enabled) launch_fullsort_fallback(a.fb);
}
template <bool GROUP>
__device__ inline void band_repair(const BandArgs &a, const BandRow &w, int status_bits, bool may_widen)
{
    if (!GROUP) {  // a launch for one row: its arguments are the row's
        band_repair_row(a, status_bits, may_widen);
        return;
    }
    BandArgs mine;
    band_args_of_row(a, w, &mine);
    band_repair_row(mine, status_bits, may_widen);
}

template <bool GROUP>
__device__ __forceinline__ void band_solve_body(const BandArgs &a);

// One launch for one row ...
__global__ void __launch_bounds__(1024) band_solve_kernel(const __grid_constant__ BandArgs a)
{
    pdl_wait();
    band_solve_body<false>(a);
}

// ... or for a group of rows (BatchShift): blockIdx.y is the row.  A kernel of its own, so that the one-row launch
// keeps reading its arguments from the constant bank instead of holding the row's pointers in registers.
__global__ void __launch_bounds__(1024) band_solve_group_kernel(const __grid_constant__ BandArgs a)
{
    pdl_wait();
    band_solve_body<true>(a);
}

template <bool GROUP>
__device__ __forceinline__ void band_solve_body(const BandArgs &a)
{
    const BandRow w = band_row<GROUP>(a);
    double k = a.k, t = a.t;
    ExpScale sc = a.sc;
    float cexp = a.c;
    if (w.rp) {
        if (!w.rp->valid) return;
        k = w.rp->k;
        t = w.rp->t;
        sc = w.rp->sc;
        cexp = w.rp->c;
    }
    extern __shared__ __align__(16) unsigned char smem_raw[];
    BandShared &S = *reinterpret_cast<BandShared *>(smem_raw);
    ScanShared &sh = S.sh;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    const CallCtl &c = w.ctl->call;
    const unsigned long long raw = c.band_count;
    // Launched with several blocks, every block takes the first level's decisions for itself (same inputs, same
    // arithmetic, same result) and gathers its share of the band; the last one to arrive goes on alone.  Whatever
    // does not go through that level is block 0's.
    const int nblk = gridDim.x;
    if (raw > a.cap) {  // band overflow: the whole row goes through the full sort
        if (tid == 0 && blockIdx.x == 0) band_repair<GROUP>(a, w, 0x2, false);
        return;
    }
    const long long M = (long long)raw;
    Seeds sd;
    sd.L = (c.a_L > -CUDART_INF_F) ? Agg{c.a_L, (float)c.S_L} : empty_up();
    sd.R = (c.a_R < CUDART_INF_F) ? Agg{c.a_R, (float)c.S_R} : empty_down();
    sd.n_R = (long long)c.n_R;
    const float fscale = a.fscale;
    const float inv_fscale_f = 1.f / fscale;  // exact: a power of two
    const double inv_fscale = (double)inv_fscale_f;

    BandGrid g = bracket_grid(c.a_L, c.a_R, c.grid_klo, c.grid_khi);
    bool trust_left = false;       // the left end is a bucket edge that a level already placed below the root
    bool right_is_bracket = true;  // the right end is still the bracket's own a_R
    bool left_failed = false, gathered = false, solved = false;
    long long in_range = M;
    SolveResult res;

    // ---- levels with one bucket per thread and four block barriers each ----
    // Level 0 reads the tables the stream pass filled and gathers from the band in global memory; a further
    // level (only when the three buckets around the crossing still hold more than the all-pairs solve takes)
    // buckets the gathered list itself, in shared memory.  Same aggregates, node values and +-1 bucket rule
    // as the general level loop below, which takes over when three buckets do not fit the list.
    bool first_done = false;
    uint32_t *cur = S.list, *other = S.list2;
    int m_list = 0;
    constexpr float CSCALE = 1048576.f;  // 2^20: at most 2048 list terms of at most 1 inside 32 bits
    for (int lvl = 0; lvl < BAND_LEVELS; ++lvl) {
        if (lvl == 0) {
            if (!(M > PAIRS_MAX && !g.one_key_buckets() && blockDim.x == BAND_BUCKETS)) {
                if (blockIdx.x != 0) return;
                break;
            }
        } else {
            if (!(gathered && m_list > PAIRS_MAX)) break;
            const BandGrid g2 = make_band_grid(g.tlo, g.thi, sd.L.pivot > -CUDART_INF_F ? sd.L.pivot : g.lo_val,
                                               sd.R.pivot < CUDART_INF_F ? sd.R.pivot : g.hi_val);
            if (g2.shift == 0) break;  // one key per bucket: the list is runs of equal scores, the block solve takes it
            g = g2;
        }
        const int bkt = tid;
        const float e0 = g.edge(bkt), e1 = g.edge(bkt + 1);
        unsigned my_cnt;
        float my_up, my_down;
        if (lvl == 0) {
            my_cnt = c.band_cnt[bkt];
            my_up = __ull2float_rn(c.band_up[bkt]) * inv_fscale_f;
            my_down = __ull2float_rn(c.band_down[bkt]) * inv_fscale_f;
        } else {
            S.cnt[tid] = 0;
            S.fx_up[tid] = 0;
            S.fx_down[tid] = 0;
            __syncthreads();
#pragma unroll 1
            for (int i = tid; i < m_list; i += BAND_BUCKETS) {
                const uint32_t kv = cur[i];
                const int bk = g.bucket(kv);
                const float x = key_to_float(kv);
                if (LAPSUM_IN_BOUNDS(bk, BAND_BUCKETS, w.ctl)) {
                    atomicAdd(&S.cnt[bk], 1u);
                    atomicAdd(&S.fx_up[bk], __float2uint_rn(ex2_approx((x - g.edge(bk + 1)) * cexp) * CSCALE));
                    atomicAdd(&S.fx_down[bk], __float2uint_rn(ex2_approx((g.edge(bk) - x) * cexp) * CSCALE));
                }
            }
            __syncthreads();
            my_cnt = S.cnt[tid];
            my_up = (float)S.fx_up[tid] * (1.f / CSCALE);
            my_down = (float)S.fx_down[tid] * (1.f / CSCALE);
        }
        if (tid == 0) { S.sh_cnt = 0; S.cum_at[0] = 0; S.cum_at[1] = 0; }
        // inclusive scans inside the warp: counts, prefix aggregates (pivot = upper edge), suffix aggregates
        WarpScan in = warp_scan3(WarpScan{my_cnt, Agg{e1, my_up}, Agg{e0, my_down}}, sc);
        const unsigned ci = in.cnt;
        const Agg iu = in.up, idn = in.down;
        if (lane == 31) { S.w_up[warp] = iu; S.w_cnt[warp] = ci; }
        if (lane == 0) S.w_down[warp] = idn;
        __syncthreads();
        // every warp scans the 32 warp totals for itself
        const WarpScan top = warp_scan3(WarpScan{S.w_cnt[lane], S.w_up[lane], S.w_down[lane]}, sc);
        const long long total = (long long)__shfl_sync(FULL, top.cnt, 31);
        const unsigned c_below = __shfl_sync(FULL, top.cnt, max(warp - 1, 0));
        Agg u_below = shfl_agg(top.up, max(warp - 1, 0)), d_above = shfl_agg(top.down, min(warp + 1, 31));
        if (warp == 0) u_below = empty_up();
        if (warp == 31) d_above = empty_down();
        const long long cum = (long long)(warp > 0 ? c_below : 0u) + ci;  // scores in buckets 0..bkt
        const Agg pre = combine_up(combine_up(sd.L, u_below, sc), iu, sc);  // everything up to this bucket's end
        Agg above;  // everything above this bucket
        above.pivot = __shfl_down_sync(FULL, idn.pivot, 1);
        above.sum = __shfl_down_sync(FULL, idn.sum, 1);
        if (lane == 31) above = empty_down();
        above = combine_down(combine_down(above, d_above, sc), sd.R, sc);
        // node value at this bucket's upper edge, and the crossing
        int cand = INT_MIN;
        {
            const float Bp = fold_down(above, e1, sc);
            const double G = 0.5 * ((double)pre.sum - (double)Bp) + ((double)(sd.n_R + total - cum) - k);
            if (G >= 0.0) cand = bkt + 1;
        }
        if (tid == 0) {
            if (trust_left || sd.L.pivot == -CUDART_INF_F) {
                cand = max(cand, 0);
            } else {
                const Agg all = combine_down(Agg{e0, my_down}, above, sc);
                const float Bp = fold_down(all, sd.L.pivot, sc);
                const double G = 0.5 * ((double)sd.L.sum - (double)Bp) + ((double)(sd.n_R + total) - k);
                if (G >= 0.0) cand = max(cand, 0);
            }
        }
        cand = warp_max(cand);
        if (lane == 0) S.w_j[warp] = cand;
        __syncthreads();
        const int J = warp_max(S.w_j[lane]);
        if (J < 0) {
            if (lvl == 0 && blockIdx.x != 0) return;
            left_failed = true;
            first_done = true;
            break;
        }
        const int lo_i = max(J - 1, 0), hi_i = min(J + 2, BAND_BUCKETS);
        const float e_lo = g.edge(lo_i), e_hi = g.edge(hi_i);
        const unsigned long long k_lo = g.key_lo(lo_i), k_hi = g.key_hi(hi_i);
        if (bkt == lo_i - 1) S.cum_at[0] = cum;
        if (bkt == hi_i - 1) S.cum_at[1] = cum;
        double tailL, tailR;
        if (lvl == 0) {
            // tails from the bucket sums (accurate exponentials, one more per bucket)
            double accL = 0.0, accR = 0.0;
            if (bkt < lo_i) accL = (double)(my_up * decay(e_lo - e1, sc));
            else if (bkt >= hi_i) accR = (double)(my_down * decay(e0 - e_hi, sc));
            accL = warp_sum(accL);
            accR = warp_sum(accR);
            if (lane == 0) { S.w_tail[0][warp] = accL; S.w_tail[1][warp] = accR; }
            __syncthreads();
            tailL = warp_sum(S.w_tail[0][lane]);
            tailR = warp_sum(S.w_tail[1][lane]);
            if (S.cum_at[1] - S.cum_at[0] > BAND_LIST) {  // the general loop starts over on the band
                if (blockIdx.x != 0) return;
                break;
            }
            if (nblk == 1) {
                for_each_band_key(w.band, M, [&](uint32_t kv) {
                    if (kv >= k_lo && kv < k_hi) {
                        const unsigned pos = atomicAdd(&S.sh_cnt, 1u);
                        if (LAPSUM_IN_BOUNDS(pos, BAND_LIST, w.ctl)) cur[pos] = kv;
                    }
                });
            } else {
                for_each_band_key(w.band, M, [&](uint32_t kv) {
                    if (kv >= k_lo && kv < k_hi) {
                        const unsigned pos = atomicAdd(&w.ctl->call.solve_list_cnt, 1u);
                        if (LAPSUM_IN_BOUNDS(pos, BAND_LIST, w.ctl)) w.glist[pos] = kv;
                    }
                }, blockIdx.x, nblk);
                __syncthreads();
                if (tid == 0) {
                    __threadfence();
                    S.is_last = (atomicAdd(&w.ctl->call.solve_ticket, 1u) == (unsigned)nblk - 1u);
                }
                __syncthreads();
                if (!S.is_last) return;
                __threadfence();
                const unsigned got = *((volatile unsigned *)&w.ctl->call.solve_list_cnt);
                for (unsigned i = tid; i < got; i += blockDim.x)
                    if (LAPSUM_IN_BOUNDS(i, BAND_LIST, w.ctl)) cur[i] = __ldcg(w.glist + i);
                if (tid == 0) S.sh_cnt = got;
            }
        } else {
            // tails of the list's own scores outside the three buckets, exactly (fixed point), and the new list
            long long accL = 0, accR = 0;
#pragma unroll 1
            for (int i = tid; i < m_list; i += BAND_BUCKETS) {
                const uint32_t kv = cur[i];
                if (kv < k_lo) accL += __float2ll_rn(decay(e_lo - key_to_float(kv), sc) * fscale);
                else if (kv >= k_hi) accR += __float2ll_rn(decay(key_to_float(kv) - e_hi, sc) * fscale);
                else {
                    const unsigned pos = atomicAdd(&S.sh_cnt, 1u);
                    if (LAPSUM_IN_BOUNDS(pos, BAND_LIST, w.ctl)) other[pos] = kv;
                }
            }
            accL = warp_sum(accL);
            accR = warp_sum(accR);
            if (lane == 0) { S.sh_fx[0][warp] = accL; S.sh_fx[1][warp] = accR; }
            __syncthreads();
            tailL = (double)warp_sum(S.sh_fx[0][lane]) * inv_fscale;
            tailR = (double)warp_sum(S.sh_fx[1][lane]) * inv_fscale;
            uint32_t *tmp = cur;
            cur = other;
            other = tmp;
        }
        const long long below = S.cum_at[0], upto = S.cum_at[1];
        Seeds s2;
        if (lo_i > 0 || sd.L.pivot > -CUDART_INF_F)
            s2.L = Agg{e_lo, (float)(tailL + (double)fold_up(sd.L, e_lo, sc))};
        else
            s2.L = sd.L;
        if (e_hi < CUDART_INF_F)
            s2.R = Agg{e_hi, (float)(tailR + (double)fold_down(sd.R, e_hi, sc))};
        else
            s2.R = sd.R;
        s2.n_R = sd.n_R + (total - upto);
        if (lo_i > 0) trust_left = true;
        if (k_hi < g.thi) right_is_bracket = false;
        sd = s2;
        g.tlo = g.klo = k_lo;
        g.thi = g.khi = k_hi;
        in_range = upto - below;
        gathered = true;
        first_done = true;
        __syncthreads();
        const int m_new = (int)S.sh_cnt;
        if (lvl > 0 && m_new >= m_list) { m_list = m_new; break; }  // no progress (an open end): the block solve takes it
        m_list = m_new;
    }

    for (int level = 0; !first_done && level < BAND_LEVELS && in_range > BAND_LIST; ++level) {
        if (level > 0) g = make_band_grid(g.tlo, g.thi, sd.L.pivot > -CUDART_INF_F ? sd.L.pivot : g.lo_val,
                                          sd.R.pivot < CUDART_INF_F ? sd.R.pivot : g.hi_val);
        for (int i = tid; i <= BAND_BUCKETS; i += blockDim.x) {
            S.edge[i] = g.edge(i);
            if (i < BAND_BUCKETS) {
                if (level == 0) {  // filled by the stream pass
                    S.cnt[i] = c.band_cnt[i];
                    S.up[i] = __ull2float_rn(c.band_up[i]) * inv_fscale_f;
                    S.down[i] = __ull2float_rn(c.band_down[i]) * inv_fscale_f;
                } else {
                    S.fx_up[i] = 0;
                    S.fx_down[i] = 0;
                    S.cnt[i] = 0;
                }
            }
        }
        __syncthreads();
        int cbits = 31;  // coarse sums of the deeper levels: M terms of at most 1 inside 32 bits
        while (cbits > 0 && ((long long)1 << (31 - cbits)) <= M) --cbits;
        const float cscale = (float)(1u << cbits);
        const float inv_cscale = 1.f / cscale;
        if (level > 0) {
            for_each_band_key(w.band, M, [&](uint32_t kv) {
                if (kv < g.tlo || kv >= g.thi) return;
                const int bkt = g.bucket((uint32_t)kv);
                const float x = key_to_float(kv);
                if (LAPSUM_IN_BOUNDS(bkt, BAND_BUCKETS, w.ctl)) {
                    atomicAdd(&S.cnt[bkt], 1u);
                    atomicAdd(&S.fx_up[bkt], __float2uint_rn(ex2_approx((x - S.edge[bkt + 1]) * cexp) * cscale));
                    atomicAdd(&S.fx_down[bkt], __float2uint_rn(ex2_approx((S.edge[bkt] - x) * cexp) * cscale));
                }
            });
            __syncthreads();
            if (tid < BAND_BUCKETS) {
                S.up[tid] = (float)S.fx_up[tid] * inv_cscale;
                S.down[tid] = (float)S.fx_down[tid] * inv_cscale;
            }
        }
        {   // inclusive cumulative counts
            unsigned v = (tid < BAND_BUCKETS) ? S.cnt[tid] : 0, vi = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const unsigned t1 = __shfl_up_sync(FULL, vi, o);
                if (lane >= o) vi += t1;
            }
            if (lane == 31) sh.imax[warp] = (int)vi;
            __syncthreads();
            unsigned off = 0;
            for (int w = 0; w < warp; ++w) off += (unsigned)sh.imax[w];
            __syncthreads();
            if (tid < BAND_BUCKETS) S.cnt[tid] = off + vi;
        }
        __syncthreads();
        const long long total = (long long)S.cnt[BAND_BUCKETS - 1];
        if (g.one_key_buckets()) {
            // every bucket is one key value: runs of equal scores with multiplicities, solved exactly as they are
            res = solve_items_block(TieItems{S.edge, S.cnt}, BAND_BUCKETS, total, sd, k, t, sc, S.pref, S.suf, sh,
                                    trust_left, right_is_bracket);
            solved = true;
            break;
        }
        BucketItems it{S.edge, S.up, S.down, S.cnt};
        const int J = crossing_item(it, BAND_BUCKETS, total, sd, k, sc, S.pref, S.suf, sh, trust_left);
        if (J < 0) { left_failed = true; break; }
        // keep buckets J-1 .. J+1 unresolved
        const int lo_i = max(J - 1, 0), hi_i = min(J + 2, BAND_BUCKETS);
        const float e_lo = S.edge[lo_i], e_hi = S.edge[hi_i];
        const unsigned long long k_lo = g.key_lo(lo_i), k_hi = g.key_hi(hi_i);
        const long long below = (lo_i > 0) ? (long long)S.cnt[lo_i - 1] : 0;
        const long long upto = (long long)S.cnt[hi_i - 1];
        const bool fits = (upto - below) <= BAND_LIST;
        if (tid == 0) S.sh_cnt = 0;
        __syncthreads();
        double tailL = 0.0, tailR = 0.0;
        if (level == 0) {
            // tails from the first-level bucket sums (accurate exponentials, one more per bucket)
            double accL = 0.0, accR = 0.0;
            for (int b = tid; b < BAND_BUCKETS; b += blockDim.x) {
                if (b < lo_i) accL += (double)(S.up[b] * decay(e_lo - S.edge[b + 1], sc));
                else if (b >= hi_i) accR += (double)(S.down[b] * decay(S.edge[b] - e_hi, sc));
            }
            tailL = block_sum(accL, sh.dsum);
            tailR = block_sum(accR, sh.dsum);
            if (fits)
                for_each_band_key(w.band, M, [&](uint32_t kv) {
                    if (kv >= k_lo && kv < k_hi) {
                        const unsigned pos = atomicAdd(&S.sh_cnt, 1u);
                        if (LAPSUM_IN_BOUNDS(pos, BAND_LIST, w.ctl)) S.list[pos] = kv;
                    }
                });
        } else {
            long long accL = 0, accR = 0;
            for_each_band_key(w.band, M, [&](uint32_t kv) {
                if (kv < g.tlo || kv >= g.thi) return;
                if (kv < k_lo) accL += __float2ll_rn(decay(e_lo - key_to_float(kv), sc) * fscale);
                else if (kv >= k_hi) accR += __float2ll_rn(decay(key_to_float(kv) - e_hi, sc) * fscale);
                else if (fits) {
                    const unsigned pos = atomicAdd(&S.sh_cnt, 1u);
                    if (LAPSUM_IN_BOUNDS(pos, BAND_LIST, w.ctl)) S.list[pos] = kv;
                }
            });
            accL = warp_sum(accL);
            accR = warp_sum(accR);
            if (lane == 0) { S.sh_fx[0][warp] = accL; S.sh_fx[1][warp] = accR; }
            __syncthreads();
            long long totL = 0, totR = 0;
            for (int w = 0; w < 32; ++w) { totL += S.sh_fx[0][w]; totR += S.sh_fx[1][w]; }
            tailL = (double)totL * inv_fscale;
            tailR = (double)totR * inv_fscale;
        }
        Seeds s2;
        if (lo_i > 0 || sd.L.pivot > -CUDART_INF_F)
            s2.L = Agg{e_lo, (float)(tailL + (double)fold_up(sd.L, e_lo, sc))};
        else
            s2.L = sd.L;
        if (e_hi < CUDART_INF_F)
            s2.R = Agg{e_hi, (float)(tailR + (double)fold_down(sd.R, e_hi, sc))};
        else
            s2.R = sd.R;
        s2.n_R = sd.n_R + (total - upto);
        if (lo_i > 0) trust_left = true;
        if (k_hi < g.thi) right_is_bracket = false;
        sd = s2;
        g.tlo = g.klo = k_lo;
        g.thi = g.khi = k_hi;
        in_range = upto - below;
        gathered = fits;
        __syncthreads();
    }

    if (solved) {
        // done inside the level loop
    } else if (left_failed) {
        res.status = (int)ST_ROOT_LEFT;
        res.b = sd.L.pivot;
        res.th = RowThreshold{sd.L.pivot, 0.f};
    } else if (in_range > BAND_LIST) {
        // the levels always end with a list that fits or with one-key buckets; if they ever did not,
        // let the full sort take over rather than solve on a truncated list
        res.status = (int)ST_ROOT_LEFT;
        res.b = sd.L.pivot;
        res.th = RowThreshold{sd.L.pivot, 0.f};
    } else {
        if (!gathered) {  // small band: no level ran
            if (tid == 0) S.sh_cnt = 0;
            __syncthreads();
            for_each_band_key(w.band, M, [&](uint32_t kv) {
                if (kv < g.tlo || kv >= g.thi) return;
                const unsigned pos = atomicAdd(&S.sh_cnt, 1u);
                if (pos < BAND_LIST) cur[pos] = kv;
            });
            __syncthreads();
        }
        const int m = (int)min(S.sh_cnt, (unsigned)BAND_LIST);
        if (m <= PAIRS_MAX) {
            // a short list (the usual case): all pairs, neither sort nor scan
            res = solve_list_pairs(cur, m, sd, k, t, sc, S.pairs, trust_left, right_is_bracket, w.ctl);
        } else {
            int pad = 1;
            while (pad < m) pad <<= 1;
            float *s = reinterpret_cast<float *>(cur);
            __syncthreads();
            for (int i = m + tid; i < pad; i += blockDim.x) cur[i] = 0xffffffffu;
            __syncthreads();
            bitonic_sort_shared(cur, pad);
            for (int i = tid; i < m; i += blockDim.x) s[i] = key_to_float(cur[i]);
            __syncthreads();
            res = solve_sorted_block(s, m, sd, k, t, sc, S.pref2, S.suf2, sh, trust_left,
                                     right_is_bracket);
        }
    }
    if (tid == 0) {
        if (res.status & (int)(ST_ROOT_LEFT | ST_ROOT_RIGHT)) {
            band_repair<GROUP>(a, w, res.status, true);
        } else {
            if (res.status) set_status(w.ctl, (unsigned)res.status);
            *w.b_out = res.b;
            *w.th_out = res.th;
        }
    }
}

}  // namespace lapsum
