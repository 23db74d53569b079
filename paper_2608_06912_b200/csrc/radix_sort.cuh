// Least-significant-digit radix sort of 32-bit keys (optionally with a 32-bit
// payload): one up-front histogram kernel for all four 8-bit digits, then four
// single-pass ("onesweep") scatter kernels chained by decoupled look-back over
// per-tile, per-digit status words.  Stable, so equal keys keep input order.
//
// The element count may live on the device (count_ptr) so that the band of the
// bracket path can be sorted without a host round trip; a run_flag lets a whole
// sort be skipped on the device (the full-sort fallback of the bracket path).
#pragma once
#include "common.cuh"

namespace lapsum {

constexpr int RS_THREADS = 512;
constexpr int RS_ITEMS = 16;
constexpr int RS_TILE = RS_THREADS * RS_ITEMS;  // 8192 keys per tile
constexpr int RS_WARPS = RS_THREADS / 32;
constexpr int RS_WARP_KEYS = 32 * RS_ITEMS;     // every warp owns 512 consecutive keys of the tile
constexpr int RS_SPIN_LIMIT = 1 << 16;  // bounded look-back wait: polls of one predecessor word (~1 us each) before giving up
constexpr int RS_WINDOW = 16;           // predecessor words fetched per look-back round

// Look-back status word of one (tile, digit): [31:30] flag, [29:0] count.  Two arrays of tiles x 256 words are used
// alternately by the four passes: the histogram kernel zeroes the first for pass 0 and every pass zeroes the other
// array for its successor, so a word with flag 0 always means "not published yet in THIS pass".
constexpr uint32_t RS_FLAG_AGG = 1u, RS_FLAG_PREFIX = 2u;
__device__ __forceinline__ uint32_t rs_pack(uint32_t flag, uint32_t v) { return (flag << 30) | v; }
__device__ __forceinline__ uint32_t rs_poll(const uint32_t *p)
{
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void rs_publish(uint32_t *p, uint32_t v)
{
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

struct SortCount {
    const unsigned long long *ptr;  // device count (nullable)
    unsigned long long imm;         // used when ptr == nullptr
    unsigned long long cap;         // clamp for device counts
    __device__ unsigned long long get() const
    {
        if (!ptr) return imm;
        unsigned long long v = *ptr;
        return v < cap ? v : cap;
    }
};

// What the first pass of a sort reads: keys as they are, or scores (fp32 / fp16 / bf16) that are converted to
// order-preserving 32-bit keys on the fly (a 16-bit score sorts as the fp32 of the same value)
enum : int { RS_IN_KEYS = 0, RS_IN_F32 = 1, RS_IN_F16 = 2, RS_IN_BF16 = 3 };
template <int IN>
struct RsIn { using T = float; };  // element type behind the input pointer (keys and fp32 scores: 32-bit words)
template <>
struct RsIn<RS_IN_F16> { using T = __half; };
template <>
struct RsIn<RS_IN_BF16> { using T = __nv_bfloat16; };

// ------------------------------------------------------------ histogram ----
// Also clears the look-back words that pass 0 of this sort will use (status0: tiles x 256 words).
template <int IN>
__global__ void __launch_bounds__(512) rs_histogram_kernel(const void *__restrict__ in_raw, SortCount cnt,
                                                            SortCtl *ctl, uint32_t *status0, const int *run_flag)
{
    constexpr bool IS_FLOAT = IN == RS_IN_F32;
    constexpr bool IS_16 = IN == RS_IN_F16 || IN == RS_IN_BF16;
    using T16 = typename RsIn<IN>::T;
    const uint32_t *in = static_cast<const uint32_t *>(in_raw);
    pdl_wait();
    if (run_flag && *run_flag == 0) return;
    __shared__ uint32_t h[4][256];
    for (int i = threadIdx.x; i < 1024; i += blockDim.x) (&h[0][0])[i] = 0;
    __syncthreads();
    const unsigned long long n = cnt.get();
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    const unsigned long long gtid = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    {
        const unsigned long long words = (n + RS_TILE - 1) / RS_TILE * 256ull;
        for (unsigned long long i = gtid; i < words; i += stride) status0[i] = 0u;
    }
    const unsigned long long nvec = (((uintptr_t)in & 15) == 0) ? n / 4 : 0;
    const int lane = threadIdx.x & 31;
    // every lane of a warp runs the same number of iterations (dead lanes carry live = false), so the warp-wide
    // match below always sees the whole warp
    auto add = [&](uint32_t key, bool live) {
        if (IS_FLOAT) key = float_to_key(__uint_as_float(key));
        if (live) {
            atomicAdd(&h[0][key & 255u], 1u);
            atomicAdd(&h[1][(key >> 8) & 255u], 1u);
            atomicAdd(&h[2][(key >> 16) & 255u], 1u);
        }
        // the top digit of floating-point data sits in a few bins: one atomic per distinct value and warp
        const uint32_t d = live ? (key >> 24) : 0xffffffffu;
        const unsigned peers = __match_any_sync(FULL, d);
        if (live && (peers & ((1u << lane) - 1u)) == 0) atomicAdd(&h[3][d], (uint32_t)__popc(peers));
    };
    if constexpr (IS_16) {  // 16-bit scores: eight per 128-bit load, each sorted as the fp32 of the same value
        const T16 *in16 = static_cast<const T16 *>(in_raw);
        const unsigned long long nv8 = (((uintptr_t)in_raw & 15) == 0) ? n / 8 : 0;
        const uint4 *in4 = reinterpret_cast<const uint4 *>(in_raw);
        for (unsigned long long ib = gtid - lane; ib < nv8; ib += stride) {
            const bool live = ib + lane < nv8;
            const uint4 q = live ? __ldg(in4 + ib + lane) : make_uint4(0, 0, 0, 0);
            float x[8];
            Io<T16>::unpack(q, x);
#pragma unroll
            for (int e = 0; e < 8; ++e) add(float_to_key(x[e]), live);
        }
        for (unsigned long long ib = nv8 * 8 + gtid - lane; ib < n; ib += stride) {
            const bool live = ib + lane < n;
            add(live ? float_to_key(Io<T16>::load1(in16 + ib + lane)) : 0u, live);
        }
    } else {
    const uint4 *in4 = reinterpret_cast<const uint4 *>(in);
    for (unsigned long long ib = gtid - lane; ib < nvec; ib += stride) {
        const bool live = ib + lane < nvec;
        uint4 q = live ? __ldg(in4 + ib + lane) : make_uint4(0, 0, 0, 0);
        add(q.x, live); add(q.y, live); add(q.z, live); add(q.w, live);
    }
    for (unsigned long long ib = nvec * 4 + gtid - lane; ib < n; ib += stride) {
        const bool live = ib + lane < n;
        add(live ? __ldg(in + ib + lane) : 0u, live);
    }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 1024; i += blockDim.x) {
        const uint32_t v = (&h[0][0])[i];
        if (v) atomicAdd(&ctl->hist[0][0] + i, v);
    }
}

// ------------------------------------------------------- onesweep pass ----
struct PassArgs {
    const void *keys_in;      // keys, or (first pass) the scores in the element type the kernel is instantiated for
    const uint32_t *vals_in;  // nullptr on the first pass of a pair sort: payload = position
    uint32_t *keys_out;
    uint32_t *vals_out;
    SortCount cnt;
    SortCtl *ctl;
    uint32_t *status;       // look-back words of this pass (tiles x 256)
    uint32_t *status_next;  // the other array, cleared here for the next pass
    Control *control;
    const int *run_flag;
    int spin_limit;  // polls of one predecessor word before the wait gives up (RS_SPIN_LIMIT; the time-out test passes less)
    int pass;        // 0..3, digit = bits [8*pass, 8*pass+8)
};

template <bool PAYLOAD>
struct __align__(16) PassShared {
    uint32_t keys[RS_TILE];                      // staging of the 128-bit loads, then the tile in digit order
    uint32_t vals[PAYLOAD ? RS_TILE : 4];        // the payload in the same order
    uint32_t warp_hist[RS_WARPS][256];
    uint32_t gstart[256];                        // start of every digit's bin in the output (the same for all tiles)
    uint32_t gbase[256];
    uint32_t scan_tmp[2 * RS_WARPS];
    uint32_t tile_id;
};

// One pass over one digit.  Persistent blocks take tiles of 8192 keys in ticket order (so a tile only ever waits for
// tiles that running blocks already hold).  Per tile:
//   1. 128-bit loads: every warp owns 512 consecutive keys, a lane loads four consecutive keys at a time; the keys go
//      through the warp's slice of shared memory so that lane l then holds keys l, 32 + l, 64 + l, ... of the slice;
//   2. stable rank among the warp's equal digits (item by item, lane order inside an item = input order): lanes
//      with the same digit find each other by ballots; per-warp running digit counts in shared memory;
//   3. per digit: the warps' exclusive offsets and the tile's count, PUBLISHED at once as this tile's aggregate;
//   4. the keys (and payload) are scattered into digit order inside shared memory: the registers are free again;
//   5. decoupled look-back: 256 threads, one per digit, sum the counts of the preceding tiles, 32 words per round
//      (independent loads), until a tile that already knows its inclusive prefix; the wait for a word is bounded;
//   6. coalesced write-out: consecutive slots of one digit are consecutive in the output.
template <int IN, bool PAYLOAD>
__global__ void __launch_bounds__(RS_THREADS, 2) rs_onesweep_kernel(PassArgs a)
{
    constexpr bool IS_FLOAT = IN == RS_IN_F32;
    constexpr bool IS_16 = IN == RS_IN_F16 || IN == RS_IN_BF16;
    using T16 = typename RsIn<IN>::T;
    pdl_wait();
    if (a.run_flag && *a.run_flag == 0) return;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    PassShared<PAYLOAD> &sh = *reinterpret_cast<PassShared<PAYLOAD> *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned long long n = a.cnt.get();
    const int shift = 8 * a.pass;
    const bool aligned = !IS_16 && (((uintptr_t)a.keys_in) & 15) == 0;
    const uint32_t *keys_in = static_cast<const uint32_t *>(a.keys_in);
    const int wbase = warp * RS_WARP_KEYS;
    {   // bin starts in the output: exclusive scan of the digit's global histogram, once per block
        const uint32_t g = (tid < 256) ? a.ctl->hist[a.pass][tid] : 0;
        uint32_t gi = g;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t2 = __shfl_up_sync(FULL, gi, o);
            if (lane >= o) gi += t2;
        }
        if (tid < 256 && lane == 31) sh.scan_tmp[RS_WARPS + warp] = gi;
        __syncthreads();
        if (tid < 256) {
            uint32_t go = 0;
            for (int w = 0; w < warp; ++w) go += sh.scan_tmp[RS_WARPS + w];
            sh.gstart[tid] = go + gi - g;
        }
    }

  for (;;) {
    __syncthreads();  // the previous tile's shared state is no longer needed
    if (tid == 0) sh.tile_id = atomicAdd(&a.ctl->ticket[a.pass], 1u);
    for (int i = tid; i < RS_WARPS * 256; i += RS_THREADS) (&sh.warp_hist[0][0])[i] = 0;
    __syncthreads();
    const uint32_t tile = sh.tile_id;
    const unsigned long long tile_base = (unsigned long long)tile * RS_TILE;
    if (tile_base >= n) return;
    const int valid = (int)min((unsigned long long)RS_TILE, n - tile_base);
    const bool full = valid == RS_TILE;
    if (tid < 256) a.status_next[(unsigned long long)tile * 256 + tid] = 0u;

    // 1. load
    uint32_t key[RS_ITEMS];
    if (full && aligned) {
        const uint4 *src = reinterpret_cast<const uint4 *>(keys_in + tile_base + wbase);
        uint4 *stage = reinterpret_cast<uint4 *>(sh.keys + wbase);
        uint4 q[RS_ITEMS / 4];
#pragma unroll
        for (int j = 0; j < RS_ITEMS / 4; ++j) q[j] = __ldg(src + j * 32 + lane);
#pragma unroll
        for (int j = 0; j < RS_ITEMS / 4; ++j) stage[j * 32 + lane] = q[j];
        __syncwarp();
#pragma unroll
        for (int i = 0; i < RS_ITEMS; ++i) key[i] = sh.keys[wbase + i * 32 + lane];
        __syncwarp();
    } else {
#pragma unroll
        for (int i = 0; i < RS_ITEMS; ++i) {
            const int local = wbase + i * 32 + lane;
            if constexpr (IS_16) key[i] = (local < valid) ? float_to_key(Io<T16>::load1(static_cast<const T16 *>(a.keys_in) + tile_base + local)) : 0u;
            else key[i] = (local < valid) ? __ldg(keys_in + tile_base + local) : 0u;
        }
    }
    if (IS_FLOAT) {
#pragma unroll
        for (int i = 0; i < RS_ITEMS; ++i) key[i] = float_to_key(__uint_as_float(key[i]));
    }

    // 2. rank inside the warp among equal digits (stable: earlier item first, lower lane first inside an item).
    // Lanes with the same digit find each other by ballots (one per digit bit; independent across items, so they
    // overlap); the lowest lane of every group advances the warp's running count of the digit with ONE shared-memory
    // atomic whose return value is the group's base.  The warp barrier orders an item's update before the next
    // item's, where another lane may lead the same digit.  The bases travel to the other lanes afterwards, so the
    // atomics of eight items are in flight together instead of one round trip per item.
    uint32_t rank[RS_ITEMS];
    const unsigned lt_mask = (1u << lane) - 1u;
#pragma unroll
    for (int h = 0; h < RS_ITEMS; h += 8) {  // eight items at a time
        uint32_t who[8];  // leader lane and number of group members in lower lanes
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int i = h + j;
            const bool ok = full || (wbase + i * 32 + lane < valid);
            const uint32_t d = ok ? ((key[i] >> shift) & 255u) : 256u;
            const unsigned peers = full ? match_bits<8>(d) : match_bits<9>(d);  // bit 8 separates the last tile's padding
            const unsigned below = peers & lt_mask;
            rank[i] = 0;
            if (ok && below == 0) rank[i] = atomicAdd(&sh.warp_hist[warp][d], (uint32_t)__popc(peers));
            who[j] = ((uint32_t)(__ffs(peers) - 1) << 8) | (uint32_t)__popc(below);
            __syncwarp();
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) rank[h + j] = __shfl_sync(FULL, rank[h + j], who[j] >> 8) + (who[j] & 255u);
    }
    __syncthreads();

    // 3. per digit: exclusive offsets of the warps inside the tile, the tile's count, published at once
    uint32_t tile_count = 0;
    if (tid < 256) {
        uint32_t acc = 0;
#pragma unroll
        for (int w = 0; w < RS_WARPS; ++w) {
            const uint32_t c = sh.warp_hist[w][tid];
            sh.warp_hist[w][tid] = acc;
            acc += c;
        }
        tile_count = acc;
        // tile 0's aggregate is its inclusive prefix already
        rs_publish(a.status + (unsigned long long)tile * 256 + tid, rs_pack(tile == 0 ? RS_FLAG_PREFIX : RS_FLAG_AGG, tile_count));
    }
    // exclusive scan over the 256 digits: the first slot of every digit inside the tile
    {
        const uint32_t v = (tid < 256) ? tile_count : 0;
        uint32_t vi = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const uint32_t t1 = __shfl_up_sync(FULL, vi, o);
            if (lane >= o) vi += t1;
        }
        if (tid < 256 && lane == 31) sh.scan_tmp[warp] = vi;
        __syncthreads();
        if (tid < 256) {
            uint32_t vo = 0;
            for (int w = 0; w < warp; ++w) vo += sh.scan_tmp[w];
            const uint32_t te = vo + vi - v;
            sh.gbase[tid] = sh.gstart[tid] - te;  // out index of slot q of this digit = gbase + q (+ earlier tiles, below)
#pragma unroll
            for (int w = 0; w < RS_WARPS; ++w) sh.warp_hist[w][tid] += te;  // slot of a key = this + its rank
        }
    }
    __syncthreads();

    // 4. scatter into digit order inside shared memory (from here on the keys live there, not in registers)
#pragma unroll
    for (int i = 0; i < RS_ITEMS; ++i) {
        const int local = wbase + i * 32 + lane;
        if (local < valid) {
            const uint32_t d = (key[i] >> shift) & 255u;
            const uint32_t slot = sh.warp_hist[warp][d] + rank[i];
            if (LAPSUM_IN_BOUNDS(slot, RS_TILE, a.control)) {
                sh.keys[slot] = key[i];
                if (PAYLOAD) sh.vals[slot] = a.vals_in ? __ldg(a.vals_in + tile_base + local) : (uint32_t)(tile_base + local);
            }
        }
    }

    // 5. decoupled look-back: counts of all earlier tiles for this thread's digit
    if (tid < 256 && tile > 0) {
        uint32_t excl = 0;
        bool timed_out = false, done = false;
        long long t = (long long)tile - 1;
        while (t >= 0 && !done) {
            const int wlen = (int)min((long long)RS_WINDOW, t + 1);
            const uint32_t *w0 = a.status + (unsigned long long)t * 256 + tid;  // word of tile t - i: w0 - 256 i
            uint32_t s[RS_WINDOW];
#pragma unroll
            for (int i = 0; i < RS_WINDOW; ++i)
                if (i < wlen) s[i] = rs_poll(w0 - 256 * i);
#pragma unroll
            for (int i = 0; i < RS_WINDOW; ++i) {
                if (i >= wlen || done) continue;
                uint32_t sv = s[i];
                int spins = 0;
                while ((sv >> 30) == 0u && spins < a.spin_limit) {
                    __nanosleep(20);
                    sv = rs_poll(w0 - 256 * i);
                    ++spins;
                }
                if ((sv >> 30) == 0u) { timed_out = true; done = true; continue; }
                excl += sv & 0x3fffffffu;
                if ((sv >> 30) == RS_FLAG_PREFIX) done = true;
            }
            t -= wlen;
        }
        if (timed_out) {  // the result is invalid; say so and carry on so that nothing waits on this tile for ever
            set_status(a.control, 0x10u);
            atomicAdd(&a.control->persist.lookback_timeouts, 1ull);
        }
        rs_publish(a.status + (unsigned long long)tile * 256 + tid, rs_pack(RS_FLAG_PREFIX, (excl + tile_count) & 0x3fffffffu));
        sh.gbase[tid] += excl;
    }
    __syncthreads();

    // 6. coalesced write-out: consecutive slots of one digit are consecutive in the output
#pragma unroll 4
    for (int i = 0; i < RS_ITEMS; ++i) {
        const int q = tid + i * RS_THREADS;
        if (q < valid) {
            const uint32_t kv = sh.keys[q];
            const uint32_t d = (kv >> shift) & 255u;
            const uint32_t dst = sh.gbase[d] + (uint32_t)q;
            if (LAPSUM_IN_BOUNDS(dst, n, a.control)) {
                a.keys_out[dst] = kv;
                if (PAYLOAD) a.vals_out[dst] = sh.vals[q];
            }
        }
    }
  }  // next tile
}

}  // namespace lapsum
