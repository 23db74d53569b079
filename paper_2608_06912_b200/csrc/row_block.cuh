// Short rows.  Up to 128 scores: 16 lanes per row (two rows per warp), everything in registers.  Up to 16384: one thread
// block per row; the row is sorted by a bitonic network with the keys in registers (exchanged through
// shared memory only for the index bits that neither registers nor lanes hold), scanned and solved
// in shared memory (App. A).  The mask is evaluated from the unsorted scores so that no scatter is
// needed (the fused CDF of the paper's implementation notes, App. D).  The backward is the fused
// single-reduction VJP of Eq. 5.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"
#include "solve.cuh"

namespace lapsum {

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Laplace CDF at (x - b)/t with b = th.hi + th.lo and c = log2(e)/t  (Eq. 3).  A negative c = -log2(e)/t gives
// the CDF at (b - x)/t instead: the mask of Eq. 1 for alpha > 0.
__device__ __forceinline__ float laplace_cdf(float x, RowThreshold th, float c)
{
    const float z = ((x - th.hi) - th.lo) * c;
    const float e = 0.5f * ex2_approx(-fabsf(z));
    return z <= 0.f ? e : 1.f - e;
}

// Laplace density at b = th.hi + th.lo (Eq. 5): e^{-|b-x|/t}/(2t), half_inv_t = 1/(2t)
__device__ __forceinline__ float laplace_pdf(float x, RowThreshold th, float c, float half_inv_t)
{
    return ex2_approx(-fabsf((x - th.hi) - th.lo) * c) * half_inv_t;
}

// The same two functions on a pair of scores (packed arithmetic; each half equals the scalar function's result)
__device__ __forceinline__ float2 laplace_cdf2(float2 x, float2 neg_hi, float2 neg_lo, float2 c)
{
    const float2 z = mul2(add2(add2(x, neg_hi), neg_lo), c);
    const float2 e = mul2(make_float2(ex2_approx(-fabsf(z.x)), ex2_approx(-fabsf(z.y))), dup2(0.5f));
    const float2 u = fma2(e, dup2(-1.f), dup2(1.f));  // 1 - e, exactly rounded like the subtraction
    return make_float2(z.x <= 0.f ? e.x : u.x, z.y <= 0.f ? e.y : u.y);
}

__device__ __forceinline__ float2 laplace_pdf2(float2 x, float2 neg_hi, float2 neg_lo, float2 c, float2 half_inv_t)
{
    const float2 z = mul2(add2(add2(x, neg_hi), neg_lo), c);
    return mul2(make_float2(ex2_approx(-fabsf(z.x)), ex2_approx(-fabsf(z.y))), half_inv_t);
}

// The threshold the backward works with.  The caller passes the forward's fp32 b; when the workspace still
// holds that forward's (pivot, offset) pair for this row - i.e. the pair rounds to exactly that b - the pair
// is used instead, which keeps |r_i - b| accurate to ~1e-7 t rather than to half an ulp of b.
__device__ __forceinline__ RowThreshold backward_threshold(const float *b_ptr, const RowThreshold *th_ptr)
{
    const float b = __ldg(b_ptr);
    RowThreshold out{b, 0.f};
    if (th_ptr) {
        const RowThreshold th = *th_ptr;
        if ((float)((double)th.hi + (double)th.lo) == b) out = th;
    }
    return out;
}

// Short arrays: one warp sorts with warp barriers only, the rest of the block waits at one block barrier.
template <typename T>
__device__ inline void bitonic_sort_warp(T *a, int n_pad)
{
    if (threadIdx.x < 32) {
        for (int k = 2; k <= n_pad; k <<= 1) {
            for (int j = k >> 1; j > 0; j >>= 1) {
                for (int p = threadIdx.x; p < (n_pad >> 1); p += 32) {
                    const int lo = ((p & ~(j - 1)) << 1) | (p & (j - 1));
                    const int hi = lo | j;
                    const bool asc = (lo & k) == 0;
                    const T x = a[lo], y = a[hi];
                    if ((x > y) == asc) {
                        a[lo] = y;
                        a[hi] = x;
                    }
                }
                __syncwarp();
            }
        }
    }
    __syncthreads();
}

template <typename T>
__device__ inline void bitonic_sort_shared(T *a, int n_pad)
{
    if (n_pad <= 256 && blockDim.x >= 256) {  // many idle warps would otherwise meet at every block barrier
        bitonic_sort_warp(a, n_pad);
        return;
    }
    for (int k = 2; k <= n_pad; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int p = threadIdx.x; p < (n_pad >> 1); p += blockDim.x) {
                const int lo = ((p & ~(j - 1)) << 1) | (p & (j - 1));
                const int hi = lo | j;
                const bool asc = (lo & k) == 0;
                const T x = a[lo], y = a[hi];
                if ((x > y) == asc) {
                    a[lo] = y;
                    a[hi] = x;
                }
            }
            __syncthreads();
        }
    }
}

// ---- block sort with the keys in registers ----
// Bitonic network over n_pad = blockDim * E keys, E per thread.  A compare-exchange step pairs elements whose
// indices differ in one bit q; it costs nothing but arithmetic when that bit is a register index, one shuffle
// when it is a lane bit, and needs another thread block-wide otherwise.  Two assignments of index bits make every
// step one of the first two kinds:
//   layout 1: e = thread * E + i            (bits: registers, then lanes, then warps)      covers q < log2(E) + 5
//   layout 2: e = i * T + lane * W + warp   (bits: warps, then lanes, then registers)      covers q >= log2(W)
// (T threads, W = T / 32 warps).  A stage that reaches bits above layout 1's goes through shared memory into
// layout 2 for those steps and back: two exchanges per stage instead of a block barrier per step (for 4096
// keys 10 exchanges instead of 78 barrier steps).  The exchange buffer is indexed e + e / 32, which keeps both
// layouts free of bank conflicts; it holds n_pad + n_pad / 32 words.
template <int E>
__device__ __forceinline__ void sort_regs_step_regs(uint32_t (&v)[E], int rb_limit, int k, int e_base, int e_stride)
{   // every register-bit step rb <= rb_limit, highest bit first; element i has index e_base + i * e_stride
#pragma unroll
    for (int rb = 4; rb >= 0; --rb) {
        if ((1 << rb) >= E || rb > rb_limit) continue;
#pragma unroll
        for (int i = 0; i < E; ++i) {
            if (i & (1 << rb)) continue;
            const int ip = i | (1 << rb);
            const bool asc = ((e_base + i * e_stride) & k) == 0;
            const uint32_t x = v[i], y = v[ip];
            const bool swap = (x > y) == asc;
            v[i] = swap ? y : x;
            v[ip] = swap ? x : y;
        }
    }
}
template <int E>
__device__ __forceinline__ void sort_regs_step_lanes(uint32_t (&v)[E], int d, int k, int e_base, int e_stride)
{   // partner = lane ^ d; this lane holds the lower element of each pair when (lane & d) == 0
    const bool lower = ((threadIdx.x & 31) & d) == 0;
#pragma unroll
    for (int i = 0; i < E; ++i) {
        const uint32_t other = __shfl_xor_sync(FULL, v[i], d);
        const bool asc = ((e_base + i * e_stride) & k) == 0;
        v[i] = (asc == lower) ? min(v[i], other) : max(v[i], other);
    }
}
template <int E>
__device__ inline void bitonic_sort_regs(uint32_t *buf, int n_pad, bool padded_out)
{
    const int T = blockDim.x, t = threadIdx.x, lane = t & 31, warp = t >> 5, W = T >> 5;
    constexpr int LE = (E == 2) ? 1 : (E == 4) ? 2 : (E == 8) ? 3 : 4;
    const int LT = 31 - __clz(T), LW = LT - 5;
    auto pad = [](int e) { return e + (e >> 5); };
    const int e1 = t * E;             // layout 1: e = e1 + i
    const int e2 = lane * W + warp;   // layout 2: e = e2 + i * T
    uint32_t v[E];
#pragma unroll
    for (int i = 0; i < E; ++i) v[i] = buf[e1 + i];
    __syncthreads();  // the buffer is reused with padded indices from here on
#pragma unroll 1
    for (int s = 1; (1 << s) <= n_pad; ++s) {
        const int k = 1 << s;
        int q = s - 1;
        if (q >= LE + 5) {
#pragma unroll
            for (int i = 0; i < E; ++i) buf[pad(e1 + i)] = v[i];
            __syncthreads();
#pragma unroll
            for (int i = 0; i < E; ++i) v[i] = buf[pad(e2 + i * T)];
            __syncthreads();
            if (q >= LT) {
                sort_regs_step_regs<E>(v, q - LT, k, e2, T);
                q = LT - 1;
            }
#pragma unroll 1
            for (; q >= LE + 5; --q) sort_regs_step_lanes<E>(v, 1 << (q - LW), k, e2, T);
#pragma unroll
            for (int i = 0; i < E; ++i) buf[pad(e2 + i * T)] = v[i];
            __syncthreads();
#pragma unroll
            for (int i = 0; i < E; ++i) v[i] = buf[pad(e1 + i)];
            __syncthreads();
        }
#pragma unroll 1
        for (; q >= LE; --q) sort_regs_step_lanes<E>(v, 1 << (q - LE), k, e1, 1);
        sort_regs_step_regs<E>(v, q, k, e1, 1);
    }
#pragma unroll
    for (int i = 0; i < E; ++i) buf[padded_out ? pad(e1 + i) : e1 + i] = v[i];
    __syncthreads();
}

// Sort n_pad keys held in `buf` (n_pad + n_pad / 32 words) by the whole block; with padded_out the sorted key e
// ends up at buf[e + e / 32]
__device__ inline void block_sort_keys(uint32_t *buf, int n_pad, bool padded_out)
{
    const int T = blockDim.x;
    if (T >= 32 && (T & (T - 1)) == 0 && n_pad == 2 * T) bitonic_sort_regs<2>(buf, n_pad, padded_out);
    else if (T >= 32 && (T & (T - 1)) == 0 && n_pad == 4 * T) bitonic_sort_regs<4>(buf, n_pad, padded_out);
    else if (T >= 32 && (T & (T - 1)) == 0 && n_pad == 8 * T) bitonic_sort_regs<8>(buf, n_pad, padded_out);
    else if (T >= 32 && (T & (T - 1)) == 0 && n_pad == 16 * T) bitonic_sort_regs<16>(buf, n_pad, padded_out);
    else {
        bitonic_sort_shared(buf, n_pad);
        if (padded_out) {  // no launch of this library gets here; kept so that any block shape stays correct
            if (threadIdx.x == 0)
                for (int e = n_pad - 1; e >= 32; --e) buf[e + (e >> 5)] = buf[e];  // high to low: in place
            __syncthreads();
        }
    }
}

struct BlockFwdArgs {
    const void *r;  // scores, rows x n, in the workspace's element type
    void *p;        // mask out, same type
    float *b;
    RowThreshold *th;  // nullable: per-row threshold pairs kept in the workspace
    Control *ctl;
    int n, n_pad;
    double k, t;
    ExpScale sc;
    float c;  // log2(e)/t in fp32 for the mask (negated when alpha > 0: see laplace_cdf)
    const RowParams *rp;   // nullable: rows parameter sets, one per row, replace k, t, sc, c
    float *keys_dump;      // nullable (test hook): the sorted row is written here and the kernel stops after its sort
};

// dynamic shared memory: n_pad + n_pad / 32 key words, then pref and suf (n + n / 32 + 1 words each)
template <typename T>
__global__ void __launch_bounds__(1024) row_block_forward_kernel(BlockFwdArgs a)
{
    pdl_wait();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t *keys = reinterpret_cast<uint32_t *>(smem_raw);
    float *pref = reinterpret_cast<float *>(keys + a.n_pad + (a.n_pad >> 5));
    float *suf = pref + a.n + (a.n >> 5) + 1;
    __shared__ ScanShared sh;

    const long long row = blockIdx.x;
    const T *rr = static_cast<const T *>(a.r) + row * a.n;
    for (int i = threadIdx.x; i < a.n_pad; i += blockDim.x)
        keys[i] = (i < a.n) ? float_to_key(Io<T>::load1(rr + i)) : 0xffffffffu;
    __syncthreads();
    block_sort_keys(keys, a.n_pad, true);
    float *s = reinterpret_cast<float *>(keys);  // padded layout: sorted score e at s[e + e / 32]
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) s[i + (i >> 5)] = key_to_float(keys[i + (i >> 5)]);
    __syncthreads();
    if (a.keys_dump) {  // test hook: the row as this kernel's sort left it (App. A "after sorting")
        for (int i = threadIdx.x; i < a.n; i += blockDim.x) a.keys_dump[row * a.n + i] = s[i + (i >> 5)];
        return;
    }

    Seeds sd;
    sd.L = empty_up();
    sd.R = empty_down();
    sd.n_R = 0;
    bool k_ok = true;
    if (a.rp) {
        const RowParams &q = a.rp[row];
        a.k = q.k;
        a.t = q.t;
        a.sc = q.sc;
        a.c = q.c_mask;
        k_ok = q.valid != 0;
    }
    SolveResult res = solve_sorted_block_padded(s, a.n, sd, a.k, a.t, a.sc, pref, suf, sh, true, false);
    if (!k_ok) void_result(res);
    if (threadIdx.x == 0) {
        a.b[row] = res.b;
        if (a.th) a.th[row] = res.th;
        if (res.status) set_status(a.ctl, (unsigned)res.status);
        if (row == 0) {
            a.ctl->persist.last_path = 1;
            a.ctl->persist.forwards += 1;
        }
    }
    T *pp = static_cast<T *>(a.p) + row * a.n;
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) Io<T>::store1(pp + i, laplace_cdf(Io<T>::load1(rr + i), res.th, a.c));
}

// ---- one row per cluster of four thread blocks (rows of 8192 / 16384 padded scores, few rows) ----
// A row that long keeps one block busy for ~100 us while most SMs idle when the batch is small.  Four blocks of a
// cluster take a quarter of the row each: the bitonic network runs over all four (the two highest index bits are the
// block's rank in the cluster: those three steps exchange keys through distributed shared memory), every block then
// holds one sorted quarter, the quarters' (pivot, sum) aggregates are exchanged, and each block solves its quarter with
// the other quarters as tails (App. B's seeded solve): exactly one of them holds the root.
namespace cg = cooperative_groups;
constexpr int ROW_CLUSTER = 4;      // blocks per row by default
constexpr int ROW_CLUSTER_MAX = 8;  // for the longest rows when the batch is small enough (the portable cluster limit)

template <int E>
__device__ inline void cluster_sort_regs(uint32_t *buf, int n_local, cg::cluster_group &cluster, Control *ctl)
{
    const int T = blockDim.x, t = threadIdx.x, lane = t & 31, warp = t >> 5, W = T >> 5;
    constexpr int LE = (E == 2) ? 1 : (E == 4) ? 2 : (E == 8) ? 3 : 4;
    const int LT = 31 - __clz(T), LW = LT - 5, LN = 31 - __clz(n_local);
    const int rank = (int)cluster.block_rank(), n_total = n_local * (int)cluster.num_blocks();
    auto pad = [](int e) { return e + (e >> 5); };
    const int e1 = t * E, e2 = lane * W + warp;  // the two layouts of bitonic_sort_regs, inside this block's quarter
    const int g0 = rank * n_local;               // index of the quarter's first element in the whole row
    uint32_t v[E];
#pragma unroll
    for (int i = 0; i < E; ++i) v[i] = buf[e1 + i];
    __syncthreads();
#pragma unroll 1
    for (int s = 1; (1 << s) <= n_total; ++s) {
        const int k = 1 << s;
        int q = s - 1;
#pragma unroll 1
        for (; q >= LN; --q) {  // partner = the same position in another block of the cluster
            const int bit = 1 << (q - LN);
#pragma unroll
            for (int i = 0; i < E; ++i) buf[pad(e1 + i)] = v[i];
            cluster.sync();
            const uint32_t *remote = cluster.map_shared_rank(buf, rank ^ bit);
            const bool lower = (rank & bit) == 0;
#pragma unroll
            for (int i = 0; i < E; ++i) {
                const uint32_t other = LAPSUM_IN_BOUNDS(pad(e1 + i), n_local + (n_local >> 5), ctl) ? remote[pad(e1 + i)] : v[i];
                const bool asc = ((g0 + e1 + i) & k) == 0;
                v[i] = (asc == lower) ? min(v[i], other) : max(v[i], other);
            }
            cluster.sync();  // no block overwrites its buffer before its partner has read it
        }
        if (q >= LE + 5) {
#pragma unroll
            for (int i = 0; i < E; ++i) buf[pad(e1 + i)] = v[i];
            __syncthreads();
#pragma unroll
            for (int i = 0; i < E; ++i) v[i] = buf[pad(e2 + i * T)];
            __syncthreads();
            if (q >= LT) {
                sort_regs_step_regs<E>(v, q - LT, k, g0 + e2, T);
                q = LT - 1;
            }
#pragma unroll 1
            for (; q >= LE + 5; --q) sort_regs_step_lanes<E>(v, 1 << (q - LW), k, g0 + e2, T);
#pragma unroll
            for (int i = 0; i < E; ++i) buf[pad(e2 + i * T)] = v[i];
            __syncthreads();
#pragma unroll
            for (int i = 0; i < E; ++i) v[i] = buf[pad(e1 + i)];
            __syncthreads();
        }
#pragma unroll 1
        for (; q >= LE; --q) sort_regs_step_lanes<E>(v, 1 << (q - LE), k, g0 + e1, 1);
        sort_regs_step_regs<E>(v, q, k, g0 + e1, 1);
    }
#pragma unroll
    for (int i = 0; i < E; ++i) buf[pad(e1 + i)] = v[i];
    __syncthreads();
}

// What a block tells the other blocks of its cluster
struct ClusterNote {
    Agg up, down;   // the quarter's aggregates: prefix form (pivot = its last score), suffix form (pivot = its first)
    int count;      // scores in the quarter (the row's padding lies in the last quarters)
    int left_ok;    // the root is not left of this quarter
    int status;
    float b;
    RowThreshold th;
};

// launched with the cluster size as a launch attribute (4 or 8 blocks per row)
template <typename T>
__global__ void __launch_bounds__(1024) row_cluster_forward_kernel(BlockFwdArgs a)
{
    pdl_wait();
    cg::cluster_group cluster = cg::this_cluster();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int CL = (int)cluster.num_blocks();
    const int n_local = a.n_pad / CL, rank = (int)cluster.block_rank();
    uint32_t *keys = reinterpret_cast<uint32_t *>(smem_raw);
    float *pref = reinterpret_cast<float *>(keys + n_local + (n_local >> 5));
    float *suf = pref + n_local + (n_local >> 5) + 1;
    __shared__ ScanShared sh;
    __shared__ ClusterNote note;

    const long long row = blockIdx.x / CL;
    const T *rr = static_cast<const T *>(a.r) + row * a.n;
    const int g0 = rank * n_local;
    for (int i = threadIdx.x; i < n_local; i += blockDim.x) keys[i] = (g0 + i < a.n) ? float_to_key(Io<T>::load1(rr + g0 + i)) : 0xffffffffu;
    __syncthreads();
    if (n_local == 2 * (int)blockDim.x) cluster_sort_regs<2>(keys, n_local, cluster, a.ctl);
    else cluster_sort_regs<4>(keys, n_local, cluster, a.ctl);
    const int count = max(0, min(n_local, a.n - g0));
    float *s = reinterpret_cast<float *>(keys);  // padded layout: sorted score e of the quarter at s[e + e / 32]
    for (int i = threadIdx.x; i < count; i += blockDim.x) s[i + (i >> 5)] = key_to_float(keys[i + (i >> 5)]);
    __syncthreads();
    if (a.keys_dump) {  // test hook: every block writes its sorted part of the row (the sort's last step ended with a cluster barrier)
        for (int i = threadIdx.x; i < count; i += blockDim.x) a.keys_dump[row * a.n + g0 + i] = s[i + (i >> 5)];
        return;
    }

    bool k_ok = true;
    if (a.rp) {
        const RowParams &q = a.rp[row];
        a.k = q.k;
        a.t = q.t;
        a.sc = q.sc;
        a.c = q.c_mask;
        k_ok = q.valid != 0;
    }
    // the quarter's two aggregates, for the other quarters' tails
    const PaddedElemItems it{s};
    const LocalScan ls = scan_items(it, count, a.sc, sh);  // scanned once: the totals now, the crossing below
    const Agg tot_up = ls.total_up(), tot_down = ls.total_down();
    if (threadIdx.x == 0) {
        note.up = tot_up;
        note.down = tot_down;
        note.count = count;
    }
    cluster.sync();
    Seeds sd;
    sd.L = empty_up();
    sd.R = empty_down();
    sd.n_R = 0;
    for (int c = 0; c < rank; ++c) sd.L = combine_up(sd.L, cluster.map_shared_rank(&note, c)->up, a.sc);
    for (int c = CL - 1; c > rank; --c) {
        const ClusterNote *o = cluster.map_shared_rank(&note, c);
        sd.R = combine_down(o->down, sd.R, a.sc);
        sd.n_R += o->count;
    }
    const SolveResult res = solve_items_block(it, count, (long long)count, sd, a.k, a.t, a.sc, pref, suf, sh,
                                              /*trust_left=*/rank == 0, /*test_right=*/true, &ls);
    if (threadIdx.x == 0) {
        note.left_ok = (rank == 0) || !(res.status & (int)ST_ROOT_LEFT);
        note.status = res.status & ~(int)(ST_ROOT_LEFT | ST_ROOT_RIGHT);
        note.b = res.b;
        note.th = res.th;
    }
    cluster.sync();
    // the root's quarter is the highest one that does not see it on its left
    int owner = 0;
    for (int c = CL - 1; c > 0; --c)
        if (cluster.map_shared_rank(&note, c)->left_ok) { owner = c; break; }
    const ClusterNote *won = cluster.map_shared_rank(&note, owner);
    SolveResult out;
    out.b = won->b;
    out.th = won->th;
    out.status = won->status;
    if (!k_ok) void_result(out);
    const RowThreshold th = out.th;
    if (rank == 0 && threadIdx.x == 0) {
        a.b[row] = out.b;
        if (a.th) a.th[row] = th;
        if (out.status) set_status(a.ctl, (unsigned)out.status);
        if (row == 0) {
            a.ctl->persist.last_path = 1;
            a.ctl->persist.forwards += 1;
        }
    }
    T *pp = static_cast<T *>(a.p) + row * a.n;
    for (int i = g0 + threadIdx.x; i < min(a.n, g0 + n_local); i += blockDim.x) Io<T>::store1(pp + i, laplace_cdf(Io<T>::load1(rr + i), th, a.c));
    cluster.sync();  // a block's shared memory stays alive until the others have read its note
}

// (key, index) pairs of every row, sorted as 64-bit composites: equal keys come out by ascending index
__global__ void row_block_sort_pairs_kernel(const float *r, int n, int n_pad, float *keys_out, uint32_t *idx_out)
{
    pdl_wait();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    unsigned long long *a = reinterpret_cast<unsigned long long *>(smem_raw);
    const long long row = blockIdx.x;
    for (int i = threadIdx.x; i < n_pad; i += blockDim.x)
        a[i] = (i < n) ? (((unsigned long long)float_to_key(__ldg(r + row * n + i)) << 32) | (unsigned)i)
                       : 0xffffffffffffffffull;
    __syncthreads();
    bitonic_sort_shared(a, n_pad);
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        keys_out[row * n + i] = key_to_float((uint32_t)(a[i] >> 32));
        idx_out[row * n + i] = (uint32_t)(a[i] & 0xffffffffu);
    }
}

struct BlockBwdArgs {
    const void *v, *r;       // upstream gradient and scores in the workspace's element type
    const float *b;
    const RowThreshold *th;  // nullable: the forward's threshold pairs (workspace)
    void *grad;              // gradient out, same type
    Control *ctl;
    int n;
    float c, half_inv_t;
    float *grad_k, *grad_alpha;  // nullable, one value per row
    double inv_t;
    float gsign;  // +1, or -1 when alpha > 0 (the Jacobian of Eq. 1 changes sign with alpha; the scalar gradients do not)
    const RowParams *rp;  // nullable: one parameter set per row replaces c, half_inv_t, inv_t, gsign
};

template <typename T>
__global__ void row_block_backward_kernel(BlockBwdArgs a)
{
    pdl_wait();
    __shared__ double red[32];
    const long long row = blockIdx.x;
    bool dead = false;  // a void row (unusable temperature) gets NaN gradients
    if (a.rp) {
        const RowParams &q = a.rp[row];
        dead = q.valid == 0;
        a.c = q.c;
        a.half_inv_t = q.half_inv_t;
        a.inv_t = q.inv_t;
        a.gsign = q.gsign;
    }
    const float nanf_ = __int_as_float(0x7fc00000);
    const T *rr = static_cast<const T *>(a.r) + row * a.n, *vv = static_cast<const T *>(a.v) + row * a.n;
    const RowThreshold b = backward_threshold(a.b + row, a.th ? a.th + row : nullptr);
    const bool scalars = a.grad_k || a.grad_alpha;
    float sf = 0.f, svf = 0.f, sd = 0.f, svd = 0.f;
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) {
        const float x = Io<T>::load1(rr + i), w = Io<T>::load1(vv + i);
        const float f = laplace_pdf(x, b, a.c, a.half_inv_t);
        sf += f;
        svf = fmaf(w, f, svf);
        if (scalars) {
            const float d = (x - b.hi) - b.lo;
            sd = fmaf(f, d, sd);
            svd = fmaf(w * f, d, svd);
        }
    }
    const double S_f = block_sum((double)sf, red);
    const double S_vf = block_sum((double)svf, red);
    if (scalars) {
        const double S_fd = block_sum((double)sd, red), S_vfd = block_sum((double)svd, red);
        if (threadIdx.x == 0) {
            const double m = (S_f > 0.0) ? S_vf / S_f : 0.0;
            if (a.grad_k) a.grad_k[row] = dead ? nanf_ : (float)m;
            if (a.grad_alpha) a.grad_alpha[row] = dead ? nanf_ : (S_f > 0.0) ? (float)((S_vfd - m * S_fd) * a.inv_t) : 0.f;
        }
    }
    const float mean = (S_f > 0.0) ? (float)(S_vf / S_f) : 0.f;
    T *gg = static_cast<T *>(a.grad) + row * a.n;
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) {
        const float f = laplace_pdf(Io<T>::load1(rr + i), b, a.c, a.half_inv_t * a.gsign);
        Io<T>::store1(gg + i, dead ? nanf_ : (S_f > 0.0) ? f * (Io<T>::load1(vv + i) - mean) : 0.f);
    }
    if (threadIdx.x == 0 && row == (long long)gridDim.x - 1) {
        a.ctl->persist.S_f = S_f;
        a.ctl->persist.S_vf = S_vf;
    }
}

}  // namespace lapsum

namespace lapsum {

// ---------------------------------------------------------------- warp path ----
// Rows of at most 128 scores: LANES lanes per row, the row lives in registers (ITEMS consecutive
// sorted positions per lane), every step is warp shuffles; several rows per block.
// The routing-shaped batch (65536 rows x 128 expert logits) runs here.
constexpr int WP_WARPS = 8;  // warps per block
#ifndef LAPSUM_WARP_ROW_LANES
#define LAPSUM_WARP_ROW_LANES 16
#endif
constexpr int WARP_ROW_LANES = LAPSUM_WARP_ROW_LANES;  // lanes that share a row: 16 (two rows per warp) or 32

struct WarpFwdArgs {
    const void *r;  // scores, rows x n, in the workspace's element type
    void *p;        // mask out, same type
    float *b;
    RowThreshold *th;
    Control *ctl;
    long long rows;
    int n;
    double k, t;
    ExpScale sc;
    float c;
    float c_mask;  // c for the mask: -c when alpha > 0 (see laplace_cdf)
    const RowParams *rp;   // ROW_P instantiations only: one parameter set per row replaces k, t, sc, c, c_mask
    float *keys_dump;      // DUMP instantiations only (test hook): the sorted rows are written here
};

// One compare-exchange of ITEMS keys with the partner lane's: a lane that holds the lower position of its pairs keeps
// the smaller key of every pair, the other lane the larger one.  The two predicated forms cost two issue slots per
// key where minimum, maximum and select cost three.
template <int ITEMS>
__device__ __forceinline__ void keep_min_or_max(uint32_t (&key)[ITEMS], const uint32_t (&other)[ITEMS], bool keep_min)
{
    static_assert(ITEMS == 1 || ITEMS == 2 || ITEMS == 4 || ITEMS == 8, "one predicate, then ITEMS predicated pairs");
    const unsigned flag = keep_min ? 1u : 0u;
    if constexpr (ITEMS == 1) {
        asm("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %2, 0;\n\t"
            "@p min.u32 %0, %0, %1;\n\t@!p max.u32 %0, %0, %1;\n\t"
            "}"
            : "+r"(key[0])
            : "r"(other[0]), "r"(flag));
    } else if constexpr (ITEMS == 2) {
        asm("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %4, 0;\n\t"
            "@p min.u32 %0, %0, %2;\n\t@!p max.u32 %0, %0, %2;\n\t"
            "@p min.u32 %1, %1, %3;\n\t@!p max.u32 %1, %1, %3;\n\t"
            "}"
            : "+r"(key[0]), "+r"(key[1])
            : "r"(other[0]), "r"(other[1]), "r"(flag));
    } else if constexpr (ITEMS == 4) {
        asm("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %8, 0;\n\t"
            "@p min.u32 %0, %0, %4;\n\t@!p max.u32 %0, %0, %4;\n\t"
            "@p min.u32 %1, %1, %5;\n\t@!p max.u32 %1, %1, %5;\n\t"
            "@p min.u32 %2, %2, %6;\n\t@!p max.u32 %2, %2, %6;\n\t"
            "@p min.u32 %3, %3, %7;\n\t@!p max.u32 %3, %3, %7;\n\t"
            "}"
            : "+r"(key[0]), "+r"(key[1]), "+r"(key[2]), "+r"(key[3])
            : "r"(other[0]), "r"(other[1]), "r"(other[2]), "r"(other[3]), "r"(flag));
    } else {
        asm("{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %16, 0;\n\t"
            "@p min.u32 %0, %0, %8;\n\t@!p max.u32 %0, %0, %8;\n\t"
            "@p min.u32 %1, %1, %9;\n\t@!p max.u32 %1, %1, %9;\n\t"
            "@p min.u32 %2, %2, %10;\n\t@!p max.u32 %2, %2, %10;\n\t"
            "@p min.u32 %3, %3, %11;\n\t@!p max.u32 %3, %3, %11;\n\t"
            "@p min.u32 %4, %4, %12;\n\t@!p max.u32 %4, %4, %12;\n\t"
            "@p min.u32 %5, %5, %13;\n\t@!p max.u32 %5, %5, %13;\n\t"
            "@p min.u32 %6, %6, %14;\n\t@!p max.u32 %6, %6, %14;\n\t"
            "@p min.u32 %7, %7, %15;\n\t@!p max.u32 %7, %7, %15;\n\t"
            "}"
            : "+r"(key[0]), "+r"(key[1]), "+r"(key[2]), "+r"(key[3]), "+r"(key[4]), "+r"(key[5]), "+r"(key[6]), "+r"(key[7])
            : "r"(other[0]), "r"(other[1]), "r"(other[2]), "r"(other[3]), "r"(other[4]), "r"(other[5]), "r"(other[6]), "r"(other[7]), "r"(flag));
    }
}

// ROW_P: the rows carry their own budgets and temperatures (a.rp); a separate instantiation, so that the common case
// keeps its register count.  DUMP: test hook, the kernel stops after its sort and writes the sorted row to a.keys_dump.
// LANES (32 or 16) lanes share a row, ITEMS consecutive sorted positions per lane: with 16 lanes a warp works on two
// rows at once, so every warp-level step (shuffle rounds, the root) is paid once for two rows and more of the sorting
// network runs inside the lanes' registers.
// WHOLE: the rows fill all LANES * ITEMS positions (n = 16, 32, 64, 128): no padding to keep track of.
template <int ITEMS, int LANES, bool ROW_P, bool DUMP = false, typename T = float, bool WHOLE = false>
__global__ void __launch_bounds__(WP_WARPS * 32) row_warp_forward_kernel(WarpFwdArgs a)
{
    pdl_wait();
    constexpr int RPW = 32 / LANES;  // rows per warp
    constexpr int N = LANES * ITEMS;
    const int lane = threadIdx.x & (LANES - 1);  // lane within the row's group of lanes
    const long long row_w = ((long long)blockIdx.x * WP_WARPS + (threadIdx.x >> 5)) * RPW;
    if (row_w >= a.rows) return;  // whole warps leave together
    long long row = row_w + ((threadIdx.x & 31) / LANES);
    const bool row_ok = row < a.rows;
    if (!row_ok) row = a.rows - 1;  // a group of lanes without a row of its own shadows the last row and writes nothing
    const int n = WHOLE ? N : a.n;
    const T *rr = static_cast<const T *>(a.r) + row * n;

    // load: lane holds positions lane*ITEMS .. lane*ITEMS+ITEMS-1 of the unsorted row
    float ux[ITEMS];
    constexpr bool F32 = sizeof(T) == 4;  // the vector forms below are those of fp32 rows; 16-bit rows load element-wise
    const bool vec = F32 && (n == N) && ITEMS >= 2 && ((((uintptr_t)rr) & (4 * (ITEMS < 4 ? ITEMS : 4) - 1)) == 0);
    if (vec && ITEMS >= 4) {
#pragma unroll
        for (int q4 = 0; q4 < ITEMS / 4; ++q4) {
            const float4 q = __ldg(reinterpret_cast<const float4 *>(rr) + lane * (ITEMS / 4) + q4);
            ux[(4 * q4) % ITEMS] = q.x; ux[(4 * q4 + 1) % ITEMS] = q.y; ux[(4 * q4 + 2) % ITEMS] = q.z; ux[(4 * q4 + 3) % ITEMS] = q.w;
        }
    } else if (vec && ITEMS == 2) {
        const float2 q = __ldg(reinterpret_cast<const float2 *>(rr) + lane);
        ux[0] = q.x; ux[1 % ITEMS] = q.y;
    } else {
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            const int e = lane * ITEMS + i;
            ux[i] = (e < n) ? Io<T>::load1(rr + e) : 0.f;
        }
    }
    uint32_t key[ITEMS];
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) key[i] = (WHOLE || lane * ITEMS + i < n) ? float_to_key(ux[i]) : 0xffffffffu;

    // Bitonic sort of the N positions e = lane*ITEMS + i.  Merge phase k sorts runs of k positions, ascending where
    // (e & k) == 0.  While k >= ITEMS that direction is the same for all of a lane's keys, and the lane keeps them
    // complemented during a descending phase: every compare-exchange is then "lower position takes the minimum".
    uint32_t flip = 0u;  // 0xffffffff while this lane's keys are held complemented
#pragma unroll
    for (int k = 2; k <= N; k <<= 1) {
        if (k >= ITEMS) {
            const uint32_t want = ((lane * ITEMS) & k) ? 0xffffffffu : 0u;  // k == N: no position has that bit, all ascending
            const uint32_t x = flip ^ want;
#pragma unroll
            for (int i = 0; i < ITEMS; ++i) key[i] ^= x;
            flip = want;
        }
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            if (j >= ITEMS) {
                uint32_t other[ITEMS];
#pragma unroll
                for (int i = 0; i < ITEMS; ++i) other[i] = __shfl_xor_sync(FULL, key[i], j / ITEMS, LANES);
                keep_min_or_max<ITEMS>(key, other, ((lane * ITEMS) & j) == 0);
            } else {
#pragma unroll
                for (int i = 0; i < ITEMS; ++i) {
                    if ((i & j) == 0) {
                        // inside a lane: k < ITEMS means the direction depends on the position within the lane only
                        const bool asc = (k >= ITEMS) || ((i & k) == 0);
                        const uint32_t x = key[i], y = key[i | j];
                        const uint32_t mn = min(x, y), mx = max(x, y);
                        key[i] = asc ? mn : mx;
                        key[i | j] = asc ? mx : mn;
                    }
                }
            }
        }
    }
    float s[ITEMS];
    bool ok[ITEMS];  // sorted position holds a real score (padding sorts last)
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        ok[i] = WHOLE || lane * ITEMS + i < n;
        s[i] = ok[i] ? key_to_float(key[i]) : CUDART_INF_F;
    }
    if (DUMP) {
#pragma unroll
        for (int i = 0; i < ITEMS; ++i)
            if (ok[i] && row_ok) a.keys_dump[row * n + lane * ITEMS + i] = s[i];
        return;
    }

    // The scans only LOCATE the crossing, so they run the affine recurrence of App. A as it stands, in fp32 with
    // the hardware exponential: x_e = w_e x_{e-1} + 1 with w_e = e^{-(s_e - s_{e-1})/t} in (0, 1] gives the prefix
    // sum A_e = sum_{j<=e} e^{-(s_e - s_j)/t}, and the mirror image y_e = w_{e+1} y_{e+1} + 1 the suffix sum;
    // both use the same n gaps, so the row costs n exponentials and the scan steps are two multiply-adds (no
    // pivots: every factor is at most 1, so products only underflow towards 0, the exact limit).  The index they
    // give is then CHECKED: the two sums that enter the root are re-summed about the interval's ends with the
    // accurate exponential, and a root that falls outside its interval moves the index by one and repeats.
    bool k_ok = true;
    double k_row = a.k;
    if (ROW_P) {
        const RowParams &q = a.rp[row];
        k_row = q.k;
        a.t = q.t;
        a.sc = q.sc;
        a.c = q.c;
        a.c_mask = q.c_mask;
        k_ok = q.valid != 0;
    }
    const float kf = (float)k_row;
    float w[ITEMS];  // gap factor to the previous sorted score (0 for position 0 and for padding)
    {
        const float prev_last = __shfl_up_sync(FULL, s[ITEMS - 1], 1, LANES);
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            const float below = (i == 0) ? prev_last : s[i - 1];
            const bool first = (i == 0) && (lane == 0);
            w[i] = (ok[i] && !first) ? ex2_approx((below - s[i]) * a.c) : 0.f;
        }
    }
    // prefix: lane-local recurrence, scan of the lanes' affine maps x -> W x + C over the row's lanes, prefix applied
    float A[ITEMS];
    {
        float W = 1.f, C = 0.f;
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            W *= w[i];
            C = fmaf(C, w[i], ok[i] ? 1.f : 0.f);
        }
#pragma unroll
        for (int o = 1; o < LANES; o <<= 1) {
            const float Wo = __shfl_up_sync(FULL, W, o, LANES), Co = __shfl_up_sync(FULL, C, o, LANES);
            if (lane >= o) {
                C = fmaf(Co, W, C);
                W *= Wo;
            }
        }
        float x = __shfl_up_sync(FULL, C, 1, LANES);  // value at the end of the previous lane
        if (lane == 0) x = 0.f;
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            x = fmaf(x, w[i], ok[i] ? 1.f : 0.f);
            A[i] = x;
        }
    }
    // suffix: the factor between e and e + 1 is w of e + 1
    int cand = 0;  // number of leading positions whose node value is >= k
    {
        const float next_w0 = __shfl_down_sync(FULL, w[0], 1, LANES);
        float wn[ITEMS];
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) wn[i] = (i == ITEMS - 1) ? (lane == LANES - 1 ? 0.f : next_w0) : w[(i + 1) % ITEMS];
        float W = 1.f, C = 0.f;
#pragma unroll
        for (int i = ITEMS - 1; i >= 0; --i) {
            W *= wn[i];
            C = fmaf(C, wn[i], ok[i] ? 1.f : 0.f);
        }
#pragma unroll
        for (int o = 1; o < LANES; o <<= 1) {
            const float Wo = __shfl_down_sync(FULL, W, o, LANES), Co = __shfl_down_sync(FULL, C, o, LANES);
            if (lane + o < LANES) {
                C = fmaf(Co, W, C);
                W *= Wo;
            }
        }
        float y = __shfl_down_sync(FULL, C, 1, LANES);  // value at the start of the next lane
        if (lane == LANES - 1) y = 0.f;
        // node values: Lap(s_e) = A_e/2 + (n - 1 - e) - B'_e/2, B'_e = y_e - 1 = everything above e folded down to s_e
#pragma unroll
        for (int i = ITEMS - 1; i >= 0; --i) {
            const int e = lane * ITEMS + i;
            y = fmaf(y, wn[i], ok[i] ? 1.f : 0.f);
            const float G = 0.5f * (A[i] - (y - 1.f)) + ((float)(n - 1 - e) - kf);
            if (ok[i] && G >= 0.f) cand = max(cand, e + 1);
        }
    }
#pragma unroll
    for (int o = LANES / 2; o > 0; o >>= 1) cand = max(cand, __shfl_xor_sync(FULL, cand, o, LANES));
    int J = cand;

    // the rows of a warp finish their checks independently: a row that is done keeps its result while the other goes on
    SolveResult res;
    bool done = false;
#pragma unroll 1
    for (int attempt = 0; attempt < 4; ++attempt) {
        // interval ends s_{J-1}, s_J (fetched from the lane that holds them)
        float lo = -CUDART_INF_F, hi = CUDART_INF_F;
        {
            float pick_lo = 0.f, pick_hi = 0.f;
#pragma unroll
            for (int i = 0; i < ITEMS; ++i) {
                if (((J - 1) & (ITEMS - 1)) == i) pick_lo = s[i];
                if ((J & (ITEMS - 1)) == i) pick_hi = s[i];
            }
            const float l2 = __shfl_sync(FULL, pick_lo, ((J - 1) / ITEMS) & (LANES - 1), LANES);
            const float h2 = __shfl_sync(FULL, pick_hi, (J / ITEMS) & (LANES - 1), LANES);
            if (J > 0) lo = l2;
            if (J < n) hi = h2;
        }
        // direct re-summation about the interval ends
        float Asum = 0.f, Bsum = 0.f;
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            const int e = lane * ITEMS + i;
            const float d = (e < J) ? lo - s[i] : s[i] - hi;
            // d >= 0 and finite for a real score; the product is formed with the two-float scale, the hardware
            // exponential's own error (2^-22) is far inside what the root needs
            const float ex = ok[i] ? ex2_approx(fmaf(-d, a.sc.hi, -d * a.sc.lo)) : 0.f;
            if (e < J) Asum += ex;
            else Bsum += ex;
        }
#pragma unroll
        for (int o = LANES / 2; o > 0; o >>= 1) {
            Asum += __shfl_xor_sync(FULL, Asum, o, LANES);
            Bsum += __shfl_xor_sync(FULL, Bsum, o, LANES);
        }
        const float c = (float)((double)(n - J) - k_row);
        int side = 0;
        const SolveResult r1 = interval_root_f32(lo, hi, Asum, Bsum, c, (float)a.t, &side);
        if (!done) {
            res = r1;
            // side < 0: the unclamped root lies below lo, so the crossing is at least one position lower; > 0: higher
            if (side == 0 || attempt >= 3 || (side < 0 && J == 0) || (side > 0 && J == n)) done = true;
            else J += side;
        }
        if (__all_sync(FULL, done)) break;
    }
    if (ROW_P && !k_ok) void_result(res);
    if (lane == 0 && row_ok) {
        a.b[row] = res.b;
        if (a.th) a.th[row] = res.th;
        if (res.status) set_status(a.ctl, (unsigned)res.status);
        if (row == 0) {
            a.ctl->persist.last_path = 1;
            a.ctl->persist.forwards += 1;
        }
    }
    if (!row_ok) return;
    // mask from the unsorted scores still held in registers
    T *pp = static_cast<T *>(a.p) + row * n;
    float pv[ITEMS];
    if constexpr (ITEMS >= 2) {
        const float2 nhi = dup2(-res.th.hi), nlo = dup2(-res.th.lo), cc = dup2(a.c_mask);
#pragma unroll
        for (int i = 0; i < ITEMS; i += 2) {
            const float2 q = laplace_cdf2(make_float2(ux[i], ux[i + 1]), nhi, nlo, cc);
            pv[i] = q.x;
            pv[i + 1] = q.y;
        }
    } else {
        pv[0] = laplace_cdf(ux[0], res.th, a.c_mask);
    }
    if (vec && ITEMS >= 4) {
#pragma unroll
        for (int q4 = 0; q4 < ITEMS / 4; ++q4)
            reinterpret_cast<float4 *>(pp)[lane * (ITEMS / 4) + q4] =
                make_float4(pv[(4 * q4) % ITEMS], pv[(4 * q4 + 1) % ITEMS], pv[(4 * q4 + 2) % ITEMS], pv[(4 * q4 + 3) % ITEMS]);
    } else if (vec && ITEMS == 2) {
        reinterpret_cast<float2 *>(pp)[lane] = make_float2(pv[0], pv[1 % ITEMS]);
    } else {
#pragma unroll
        for (int i = 0; i < ITEMS; ++i)
            if (lane * ITEMS + i < n) Io<T>::store1(pp + lane * ITEMS + i, pv[i]);
    }
}

struct WarpBwdArgs {
    const void *v, *r;  // upstream gradient and scores in the workspace's element type
    const float *b;
    const RowThreshold *th;
    void *grad;         // gradient out, same type
    Control *ctl;
    long long rows;
    int n;
    float c, half_inv_t;
    float *grad_k, *grad_alpha;  // nullable, one value per row
    double inv_t;
    float gsign;  // +1, or -1 when alpha > 0 (the Jacobian of Eq. 1 changes sign with alpha; the scalar gradients do not)
    const RowParams *rp;  // nullable: one parameter set per row replaces c, half_inv_t, inv_t, gsign
};

// Eq. 5 for rows of at most 128 scores: LANES (32 or 16) lanes share a row, r and v are read once and stay in registers
template <int ITEMS, int LANES, typename T = float>
__global__ void __launch_bounds__(WP_WARPS * 32) row_warp_backward_kernel(WarpBwdArgs a)
{
    pdl_wait();
    constexpr int RPW = 32 / LANES;
    constexpr int N = LANES * ITEMS;
    const int lane = threadIdx.x & (LANES - 1);
    const long long row_w = ((long long)blockIdx.x * WP_WARPS + (threadIdx.x >> 5)) * RPW;
    if (row_w >= a.rows) return;  // whole warps leave together
    long long row = row_w + ((threadIdx.x & 31) / LANES);
    const bool row_ok = row < a.rows;
    if (!row_ok) row = a.rows - 1;  // a group of lanes without a row of its own shadows the last row and writes nothing
    bool dead = false;  // a void row (unusable temperature) gets NaN gradients
    if (a.rp) {
        const RowParams &q = a.rp[row];
        dead = q.valid == 0;
        a.c = q.c;
        a.half_inv_t = q.half_inv_t;
        a.inv_t = q.inv_t;
        a.gsign = q.gsign;
    }
    const float nanf_ = __int_as_float(0x7fc00000);
    const int n = a.n;
    const T *rr = static_cast<const T *>(a.r) + row * n, *vv = static_cast<const T *>(a.v) + row * n;
    T *gg = static_cast<T *>(a.grad) + row * n;
    const RowThreshold b = backward_threshold(a.b + row, a.th ? a.th + row : nullptr);
    float x[ITEMS], w[ITEMS];
    const bool vec = sizeof(T) == 4 && ITEMS >= 4 && (n == N) && (((((uintptr_t)rr) | ((uintptr_t)vv) | ((uintptr_t)gg)) & 15) == 0);
    if (vec) {
#pragma unroll
        for (int q4 = 0; q4 < ITEMS / 4; ++q4) {
            const float4 q = __ldg(reinterpret_cast<const float4 *>(rr) + lane * (ITEMS / 4) + q4);
            const float4 u = __ldg(reinterpret_cast<const float4 *>(vv) + lane * (ITEMS / 4) + q4);
            x[(4 * q4) % ITEMS] = q.x; x[(4 * q4 + 1) % ITEMS] = q.y; x[(4 * q4 + 2) % ITEMS] = q.z; x[(4 * q4 + 3) % ITEMS] = q.w;
            w[(4 * q4) % ITEMS] = u.x; w[(4 * q4 + 1) % ITEMS] = u.y; w[(4 * q4 + 2) % ITEMS] = u.z; w[(4 * q4 + 3) % ITEMS] = u.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            const int e = lane * ITEMS + i;
            x[i] = (e < n) ? Io<T>::load1(rr + e) : CUDART_INF_F;  // padding: density 0
            w[i] = (e < n) ? Io<T>::load1(vv + e) : 0.f;
        }
    }
    // sums over the row's lanes: at most 128 terms each, so fp32 (and one fp32 division) keeps 1e-6 of the gradient's scale
    auto row_sum = [&](float v) {
#pragma unroll
        for (int o = LANES / 2; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o, LANES);
        return v;
    };
    float f[ITEMS], sf = 0.f, svf = 0.f;
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) {
        f[i] = laplace_pdf(x[i], b, a.c, a.half_inv_t);
        sf += f[i];
        svf = fmaf(w[i], f[i], svf);
    }
    const float S_f = row_sum(sf), S_vf = row_sum(svf);
    const float mean = (S_f > 0.f) ? S_vf / S_f : 0.f;
    if (a.grad_k || a.grad_alpha) {
        float sd = 0.f, svd = 0.f;
#pragma unroll
        for (int i = 0; i < ITEMS; ++i) {
            const float d = (lane * ITEMS + i < n) ? (x[i] - b.hi) - b.lo : 0.f;
            sd = fmaf(f[i], d, sd);
            svd = fmaf(w[i] * f[i], d, svd);
        }
        const double S_fd = (double)row_sum(sd), S_vfd = (double)row_sum(svd);
        if (lane == 0 && row_ok) {
            const double m = (S_f > 0.f) ? (double)S_vf / (double)S_f : 0.0;
            if (a.grad_k) a.grad_k[row] = dead ? nanf_ : (float)m;
            if (a.grad_alpha) a.grad_alpha[row] = dead ? nanf_ : (S_f > 0.f) ? (float)((S_vfd - m * S_fd) * a.inv_t) : 0.f;
        }
    }
    if (!row_ok) return;
    float g[ITEMS];
#pragma unroll
    for (int i = 0; i < ITEMS; ++i) g[i] = dead ? nanf_ : (S_f > 0.f) ? a.gsign * f[i] * (w[i] - mean) : 0.f;
    if (vec) {
#pragma unroll
        for (int q4 = 0; q4 < ITEMS / 4; ++q4)
            reinterpret_cast<float4 *>(gg)[lane * (ITEMS / 4) + q4] =
                make_float4(g[(4 * q4) % ITEMS], g[(4 * q4 + 1) % ITEMS], g[(4 * q4 + 2) % ITEMS], g[(4 * q4 + 3) % ITEMS]);
    } else {
#pragma unroll
        for (int i = 0; i < ITEMS; ++i)
            if (lane * ITEMS + i < n) Io<T>::store1(gg + lane * ITEMS + i, g[i]);
    }
    if (lane == 0 && row == a.rows - 1) {
        a.ctl->persist.S_f = (double)S_f;
        a.ctl->persist.S_vf = (double)S_vf;
    }
}

}  // namespace lapsum
