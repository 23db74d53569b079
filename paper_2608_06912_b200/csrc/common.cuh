// Shared device helpers: order-preserving key transform, the (pivot, sum)
// monoid of the stabilised exponential scan, warp/block reductions, the
// device-resident control block of a workspace.
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

namespace lapsum {

constexpr unsigned FULL = 0xffffffffu;

// First statement of every kernel: with programmatic stream serialisation a kernel's blocks may start
// while the previous kernel of the stream is still draining; this holds them until that kernel has
// completed and its writes are visible.  (A no-op for kernels launched the ordinary way.)  Every
// kernel must execute it, early-exit paths included, so that completion stays transitive.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------- keys ----
// Ascending total order on fp32 bit patterns: flip all bits of negatives, set
// the sign bit of non-negatives.  -0.0 < +0.0.
__device__ __forceinline__ uint32_t float_to_key(float x)
{
    uint32_t b = __float_as_uint(x);
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float key_to_float(uint32_t u)
{
    return __uint_as_float((u & 0x80000000u) ? (u & 0x7fffffffu) : ~u);
}

// Lanes of the warp that hold the same `bits`-bit value as this lane (all 32 lanes must call).
// Built from one ballot per bit: a fixed cost, unlike the match instruction whose time grows with
// the number of distinct values in the warp (radix digits are nearly all distinct).
template <int BITS>
__device__ __forceinline__ unsigned match_bits(uint32_t v)
{
    unsigned peers = FULL;
#pragma unroll
    for (int b = 0; b < BITS; ++b) {
        const bool bit = (v >> b) & 1u;
        const unsigned bal = __ballot_sync(FULL, bit);
        peers &= bit ? bal : ~bal;
    }
    return peers;
}

// ------------------------------------------------------------ element I/O ----
// Scores, upstream gradients, masks and gradients travel as fp32, fp16 or bf16 (lapsum_params.io_dtype); all
// arithmetic is fp32 (fp64 where sums are combined) whatever the storage type.  Io<T> gives the 16-byte vector of
// the type (4 floats, or 8 halves), its unpacking to floats and packing back (round to nearest even).
template <typename T>
struct Io;

template <>
struct Io<float> {
    static constexpr int V = 4;  // elements per 16-byte vector
    using Vec = float4;
    static __device__ __forceinline__ void unpack(const Vec &q, float (&x)[4]) { x[0] = q.x; x[1] = q.y; x[2] = q.z; x[3] = q.w; }
    static __device__ __forceinline__ Vec pack(const float (&x)[4]) { return make_float4(x[0], x[1], x[2], x[3]); }
    static __device__ __forceinline__ void unpack2(const Vec &q, float2 (&x)[2]) { x[0] = make_float2(q.x, q.y); x[1] = make_float2(q.z, q.w); }
    static __device__ __forceinline__ Vec pack2(const float2 (&x)[2]) { return make_float4(x[0].x, x[0].y, x[1].x, x[1].y); }
    static __device__ __forceinline__ float from_storage(float x) { return x; }
    template <int N>
    static __device__ __forceinline__ float max_of(const Vec *q)
    {   // largest of the 4 N scores
        float m = fmaxf(fmaxf(q[0].x, q[0].y), fmaxf(q[0].z, q[0].w));
#pragma unroll
        for (int u = 1; u < N; ++u) m = fmaxf(fmaxf(m, fmaxf(q[u].x, q[u].y)), fmaxf(q[u].z, q[u].w));
        return m;
    }
    static __device__ __forceinline__ float load1(const float *p) { return __ldg(p); }
    static __device__ __forceinline__ void store1(float *p, float x) { *p = x; }
    static __device__ __forceinline__ Vec zero() { return make_float4(0.f, 0.f, 0.f, 0.f); }
};

template <>
struct Io<__half> {
    static constexpr int V = 8;
    using Vec = uint4;
    static __device__ __forceinline__ void unpack(const Vec &q, float (&x)[8])
    {
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
            x[2 * i] = f.x;
            x[2 * i + 1] = f.y;
        }
    }
    static __device__ __forceinline__ Vec pack(const float (&x)[8])
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __half2 h = __floats2half2_rn(x[2 * i], x[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t *>(&h);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
    static __device__ __forceinline__ void unpack2(const Vec &q, float2 (&x)[4])
    {
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) x[i] = __half22float2(*reinterpret_cast<const __half2 *>(&w[i]));
    }
    static __device__ __forceinline__ Vec pack2(const float2 (&x)[4])
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __half2 h = __float22half2_rn(x[i]);
            w[i] = *reinterpret_cast<const uint32_t *>(&h);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
    static __device__ __forceinline__ float from_storage(__half x) { return __half2float(x); }
    template <int N>
    static __device__ __forceinline__ float max_of(const Vec *q)
    {   // largest of the 8 N scores: maxima of packed pairs in fp16 (exact), widened at the end
        auto h2 = [](uint32_t w) { return *reinterpret_cast<const __half2 *>(&w); };
        __half2 m = __hmax2(__hmax2(h2(q[0].x), h2(q[0].y)), __hmax2(h2(q[0].z), h2(q[0].w)));
#pragma unroll
        for (int u = 1; u < N; ++u) m = __hmax2(__hmax2(m, __hmax2(h2(q[u].x), h2(q[u].y))), __hmax2(h2(q[u].z), h2(q[u].w)));
        const float2 f = __half22float2(m);
        return fmaxf(f.x, f.y);
    }
    static __device__ __forceinline__ float load1(const __half *p) { return __half2float(__ldg(p)); }
    static __device__ __forceinline__ void store1(__half *p, float x) { *p = __float2half_rn(x); }
    static __device__ __forceinline__ Vec zero() { return make_uint4(0, 0, 0, 0); }
};

template <>
struct Io<__nv_bfloat16> {
    static constexpr int V = 8;
    using Vec = uint4;
    static __device__ __forceinline__ void unpack(const Vec &q, float (&x)[8])
    {   // a bf16 is the upper half of the fp32 with the same value
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ Vec pack(const float (&x)[8])
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
            w[i] = *reinterpret_cast<const uint32_t *>(&h);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
    static __device__ __forceinline__ void unpack2(const Vec &q, float2 (&x)[4])
    {
        const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) x[i] = make_float2(__uint_as_float(w[i] << 16), __uint_as_float(w[i] & 0xffff0000u));
    }
    static __device__ __forceinline__ Vec pack2(const float2 (&x)[4])
    {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const __nv_bfloat162 h = __float22bfloat162_rn(x[i]);
            w[i] = *reinterpret_cast<const uint32_t *>(&h);
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
    static __device__ __forceinline__ float from_storage(__nv_bfloat16 x) { return __bfloat162float(x); }
    template <int N>
    static __device__ __forceinline__ float max_of(const Vec *q)
    {   // largest of the 8 N scores: maxima of packed pairs in bf16 (exact), widened at the end
        auto b2 = [](uint32_t w) { return *reinterpret_cast<const __nv_bfloat162 *>(&w); };
        __nv_bfloat162 m = __hmax2(__hmax2(b2(q[0].x), b2(q[0].y)), __hmax2(b2(q[0].z), b2(q[0].w)));
#pragma unroll
        for (int u = 1; u < N; ++u) m = __hmax2(__hmax2(m, __hmax2(b2(q[u].x), b2(q[u].y))), __hmax2(b2(q[u].z), b2(q[u].w)));
        const float2 f = __bfloat1622float2(m);
        return fmaxf(f.x, f.y);
    }
    static __device__ __forceinline__ float load1(const __nv_bfloat16 *p) { return __bfloat162float(__ldg(p)); }
    static __device__ __forceinline__ void store1(__nv_bfloat16 *p, float x) { *p = __float2bfloat16_rn(x); }
    static __device__ __forceinline__ Vec zero() { return make_uint4(0, 0, 0, 0); }
};

// Two floats per instruction: the packed fp32 add / multiply / fused multiply-add of sm_100 (each half is the IEEE
// round-to-nearest result of the scalar operation).  The element-wise streams are bound by instruction issue once the
// scores are 16-bit, so they do their arithmetic on pairs.
__device__ __forceinline__ float2 dup2(float a) { return make_float2(a, a); }
__device__ __forceinline__ float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float2 mul2(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }

// 16-byte vector load through the read-only path / streaming variants
template <typename T>
__device__ __forceinline__ typename Io<T>::Vec io_ldg(const typename Io<T>::Vec *p) { return __ldg(p); }
template <typename T>
__device__ __forceinline__ typename Io<T>::Vec io_ldcs(const typename Io<T>::Vec *p) { return __ldcs(p); }
template <typename T>
__device__ __forceinline__ void io_stcs(typename Io<T>::Vec *p, const typename Io<T>::Vec &v) { __stcs(p, v); }

// ------------------------------------------------------------- monoid ----
// Stabilised exponential prefix (App. A: the affine recurrence
// x_i = w_i x_{i-1} + 1 is associative): an aggregate is the sum of
// e^{(s - pivot)/t} over its elements, all exponents <= 0.  Combining a left
// aggregate into a right one rescales it by e^{-(pivot_r - pivot_l)/t}.
// The suffix direction is the mirror image (pivot = smallest element).
struct Agg {
    float pivot;
    float sum;
};

struct ExpScale {
    float hi, lo;  // log2(e)/t split in two floats: x*hi + x*lo keeps the product exact to ~2^-45
};

__host__ __device__ inline ExpScale make_scale(double t)
{
    double c = 1.4426950408889634074 / t;
    ExpScale s;
    s.hi = (float)c;
    s.lo = (float)(c - (double)s.hi);
    return s;
}

// e^{-d/t} for d >= 0 (d may be +inf), accurate path (exp2f, <= 2 ulp)
__device__ __forceinline__ float decay(float d, ExpScale sc)
{
    // e^{-d/t} < 2^-256 is below every fp32.  The test also covers d = +inf and distances so large (a bucket edge
    // of a grid that reaches to +-inf) that d * lo would overflow: with lo < 0 the fma would then return +inf.
    if (!(d * sc.hi < 256.f)) return 0.f;
    float x = fmaf(-d, sc.hi, -d * sc.lo);
    return exp2f(x);
}

// left aggregate folded into pivot `p` (p >= a.pivot): a.sum * e^{-(p - a.pivot)/t}
__device__ __forceinline__ float fold_up(Agg a, float p, ExpScale sc)
{
    return (a.sum == 0.f) ? 0.f : a.sum * decay(p - a.pivot, sc);
}
// right aggregate folded into pivot `p` (p <= a.pivot)
__device__ __forceinline__ float fold_down(Agg a, float p, ExpScale sc)
{
    return (a.sum == 0.f) ? 0.f : a.sum * decay(a.pivot - p, sc);
}
__device__ __forceinline__ Agg combine_up(Agg l, Agg r, ExpScale sc)
{   // l lies below r; result pivoted at r.pivot.  An empty r (sum 0, pivot -inf) returns l.
    if (r.sum == 0.f && r.pivot == -CUDART_INF_F) return l;
    Agg o;
    o.pivot = r.pivot;
    o.sum = fold_up(l, r.pivot, sc) + r.sum;
    return o;
}
__device__ __forceinline__ Agg combine_down(Agg l, Agg r, ExpScale sc)
{   // suffix direction: l lies below r; result pivoted at l.pivot.  An empty l returns r.
    if (l.sum == 0.f && l.pivot == CUDART_INF_F) return r;
    Agg o;
    o.pivot = l.pivot;
    o.sum = l.sum + fold_down(r, l.pivot, sc);
    return o;
}
__device__ __forceinline__ Agg empty_up() { return Agg{-CUDART_INF_F, 0.f}; }
__device__ __forceinline__ Agg empty_down() { return Agg{CUDART_INF_F, 0.f}; }

__device__ __forceinline__ Agg shfl_agg(Agg a, int src)
{
    Agg o;
    o.pivot = __shfl_sync(FULL, a.pivot, src);
    o.sum = __shfl_sync(FULL, a.sum, src);
    return o;
}

// --------------------------------------------------------- reductions ----
__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    return v;
}
__device__ __forceinline__ long long warp_sum(long long v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    return v;
}
__device__ __forceinline__ int warp_max(int v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(FULL, v, o));
    return v;
}

// Block-wide sum in a fixed order; `scratch` holds >= 32 elements.  All threads get the result.
template <typename T>
__device__ __forceinline__ T block_sum(T v, T *scratch)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    T r = (lane < nw) ? scratch[lane] : T(0);
    r = warp_sum(r);
    return r;
}
// ------------------------------------------------------ control block ----
// Device-resident scalars of one workspace.  `call` is zeroed by one memset at
// the start of every forward; `persist` lives from workspace_init on.
constexpr int MAX_SORT_SLOTS = 3;  // sample sort, band sort, full sort

struct SortCtl {
    uint32_t hist[4][256];  // digit histograms of the four 8-bit passes
    uint32_t ticket[4];     // dynamic tile ids, one counter per pass
};

struct CallCtl {
    SortCtl sort[MAX_SORT_SLOTS];
    // bracket
    unsigned long long band_count;  // |M| (keeps counting past capacity)
    unsigned int stream_ticket;
    unsigned int vjp_ticket;
    int fallback;                   // 1: certificate failed or band overflow -> full sort runs
    int pad0;
    unsigned long long n_L, n_R;
    double S_L, S_R;
    float a_L, a_R;
    // radix selection of the two sample order statistics
    unsigned int sel_ticket;
    unsigned int solve_ticket, solve_list_cnt;  // band solve run by several blocks: arrivals, scores gathered so far
    uint32_t sel_keys[2];  // keys of y_(j) and y_(l) (of y_(1) / y_(K) where Eq. 8 leaves that end open)
    unsigned long long grid_klo, grid_khi;  // bucketed key range the stream pass used
    uint32_t sel_cand[2];  // candidates collected for each of the two ranks
    int pad1;
    uint32_t sel_hist[4096];
    // first-level buckets of the middle band, filled by the stream pass as it finds band scores
    unsigned int band_cnt[1024];
    unsigned long long band_up[1024], band_down[1024];  // fixed-point pivoted sums (upper / lower bucket edge)
};

struct PersistCtl {
    unsigned int status_bits;
    int last_path;
    unsigned long long forwards, fallbacks, lookback_timeouts, widenings;
    long long K, j, l;
    double S_f, S_vf, S_fd, S_vfd;  // last backward: sum f, sum v f, sum f (r - b), sum v f (r - b)
    // last bracket, copied from CallCtl when the stream pass finishes
    unsigned long long n_L, n_M, n_R;
    double S_L, S_R;
    float a_L, a_R;
};

struct Control {
    CallCtl call;
    PersistCtl persist;
};

// threshold of one row as a two-float sum: hi is an input value (the nearer
// end of the root's interval), lo the offset t*ln(.) from it
struct RowThreshold {
    float hi, lo;
};

// Per-row problem parameters for calls that carry one budget and / or one temperature per row (the paper's
// applications learn both, Sec. 6).  A prologue kernel derives them on the device from the caller's vectors; every
// kernel of the row's chain then reads them here instead of taking the call's scalars.
struct RowParams {
    double k;         // the budget the solve runs with (n - k for alpha > 0: the complementary problem)
    double t, inv_t;  // |alpha| and its reciprocal
    ExpScale sc;      // log2(e)/t split in two floats
    float c, c_mask;  // log2(e)/t in fp32; the same with the sign of -alpha (the mask's argument, see laplace_cdf)
    float half_inv_t, gsign;  // 1/(2t); +1, or -1 when alpha > 0 (sign of the mask's Jacobian)
    long long j, l;   // Eq. 8 ranks of the bracket path
    int valid;        // 0: the row's budget or temperature is unusable; the row is void (NaN outputs) and nothing runs for it
    int pad;
};

// A launch that serves several long rows of a batch at once: blockIdx.y is the row within the group.  The arguments
// describe the group's first row; a block moves every pointer to its own row first: pointers into the workspace by the
// distance between two rows' copies of the per-call buffers ("slots"), score arrays by the row length, per-row arrays
// (thresholds, parameters, scalar gradients) by one entry.
struct BatchShift {
    unsigned long long ws_step;   // bytes between the slots of two consecutive rows
    unsigned long long row_step;  // scores per row
    int active;                   // 0: the arguments already are those of the block's row
};
template <typename P>
__device__ __forceinline__ void shift_bytes(P *&p, unsigned long long bytes)
{
    if (p) p = reinterpret_cast<P *>(reinterpret_cast<uintptr_t>(p) + bytes);
}

// Key-range buckets of the middle band [a_L, a_R): at most BAND_BUCKETS buckets of 2^shift keys each.
// Stream pass and band solve derive the same grid from the same numbers.
// [klo, khi) is the key range that is cut into buckets; [tlo, thi) the key range the band really covers.
// They differ only for a bracket with an open end (Eq. 8 gave no order statistic there): cutting a range
// that reaches to +-inf would waste nearly all buckets, so the buckets stop at the sample's extreme value
// and the outermost bucket also takes whatever lies beyond it (its outer edge stays +-inf).
constexpr int BAND_BUCKETS = 1024;
struct BandGrid {
    unsigned long long klo, khi;  // bucketed key range
    unsigned long long tlo, thi;  // key range of the band
    int shift, nb;                // bucket width 2^shift keys, nb >= 1 buckets in use
    float lo_val, hi_val;         // values at the two ends of the band (the bracket ends, or -inf / +inf)
    __device__ float edge(int i) const
    {
        if (i == 0) return lo_val;
        const unsigned long long e = klo + ((unsigned long long)i << shift);
        return (e >= khi) ? hi_val : key_to_float((uint32_t)e);
    }
    // every bucket holds one key value (a run of equal scores): only a grid that does not clamp anything into its
    // outermost buckets can say so
    __device__ bool one_key_buckets() const { return shift == 0 && klo == tlo && khi == thi; }
    __device__ int bucket(uint32_t kv) const
    {
        if (kv < klo) return 0;
        return (int)min((unsigned long long)(nb - 1), ((unsigned long long)kv - klo) >> shift);
    }
    // key range [key_lo(i), key_hi(j)) = buckets i .. j-1
    __device__ unsigned long long key_lo(int i) const { return i <= 0 ? tlo : min(klo + ((unsigned long long)i << shift), khi); }
    __device__ unsigned long long key_hi(int i) const
    {
        const unsigned long long e = klo + ((unsigned long long)i << shift);
        return (i >= nb || e >= khi) ? thi : e;
    }
};
__device__ __forceinline__ BandGrid make_band_grid(unsigned long long klo, unsigned long long khi, float lo_val, float hi_val)
{
    BandGrid g;
    g.klo = g.tlo = klo;
    g.khi = g.thi = khi;
    g.lo_val = lo_val;
    g.hi_val = hi_val;
    // smallest shift with ceil((khi - klo) / 2^shift) <= BAND_BUCKETS (= 2^10)
    const unsigned long long span = khi - klo;
    const int shift = (span > (unsigned long long)BAND_BUCKETS) ? max(0, 54 - __clzll((long long)(span - 1))) : 0;
    g.shift = shift;
    g.nb = max(1, (int)((khi - klo + (1ull << shift) - 1) >> shift));
    return g;
}
// The bracket's grid: [gl, gh) is the bucketed key range (the bracket's own ends where they are finite)
__device__ __forceinline__ BandGrid bracket_grid(float a_L, float a_R, unsigned long long gl, unsigned long long gh)
{
    const unsigned long long tlo = float_to_key(a_L), thi = float_to_key(a_R);  // -inf / +inf ends included
    gl = min(max(gl, tlo), thi);
    gh = max(min(gh, thi), gl);
    BandGrid g = make_band_grid(gl, gh, a_L, a_R);
    g.tlo = tlo;
    g.thi = thi;
    return g;
}
// 2^e with e chosen so that `count` terms of at most 1 stay inside 62 bits (capped at 2^44)
__host__ __device__ inline float fixed_scale(unsigned long long count)
{
    int bits = 0;
    while (bits < 62 && (1ull << bits) <= count) ++bits;
    int e = 62 - bits;
    if (e > 44) e = 44;
    return (float)(1ull << e);
}

constexpr unsigned ST_BAD_ALPHA_BIT = 0x100u;
__device__ __forceinline__ void set_status(Control *ctl, unsigned bits) { atomicOr(&ctl->persist.status_bits, bits); }

// Check build (-DLAPSUM_CHECK_BOUNDS; the stand-in for a memory checker where none can be run): every store or
// remote load at a COMPUTED index - radix scatter, band queue and list appends, candidate lists, bucket tables,
// distributed-shared-memory reads - is compared with its limit first.  A violation raises LAPSUM_ST_BOUNDS in the
// status word and the access is skipped; nothing traps.  In the normal build the test is the constant `true`.
constexpr unsigned ST_BOUNDS_BIT = 0x200u;
#ifdef LAPSUM_CHECK_BOUNDS
__device__ __forceinline__ bool index_in_bounds(unsigned long long idx, unsigned long long limit, Control *ctl)
{
    if (idx < limit) return true;
    if (ctl) atomicOr(&ctl->persist.status_bits, ST_BOUNDS_BIT);
    return false;
}
#define LAPSUM_IN_BOUNDS(idx, limit, ctl) lapsum::index_in_bounds((unsigned long long)(idx), (unsigned long long)(limit), (ctl))
#else
#define LAPSUM_IN_BOUNDS(idx, limit, ctl) (true)
#endif

}  // namespace lapsum
