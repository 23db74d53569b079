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
constexpr int RS_SPIN_LIMIT = 1 << 22;  // bounded look-back wait (iterations per predecessor)
constexpr int RS_WINDOW = 8;            // predecessor words fetched per look-back round

// status word: [63:32] epoch, [31:30] flag, [29:0] count
constexpr uint32_t RS_FLAG_AGG = 1u, RS_FLAG_PREFIX = 2u;
__device__ __forceinline__ unsigned long long rs_pack(uint32_t epoch, uint32_t flag, uint32_t v)
{
    return ((unsigned long long)epoch << 32) | ((unsigned long long)flag << 30) | (unsigned long long)v;
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

// ------------------------------------------------------------ histogram ----
// IS_FLOAT: input holds fp32 scores, converted to order-preserving keys on the fly.
template <bool IS_FLOAT>
__global__ void __launch_bounds__(512) rs_histogram_kernel(const uint32_t *__restrict__ in, SortCount cnt,
                                                            SortCtl *ctl, const int *run_flag)
{
    pdl_wait();
    if (run_flag && *run_flag == 0) return;
    __shared__ uint32_t h[4][256];
    for (int i = threadIdx.x; i < 1024; i += blockDim.x) (&h[0][0])[i] = 0;
    __syncthreads();
    const unsigned long long n = cnt.get();
    const unsigned long long nvec = (((uintptr_t)in & 15) == 0) ? n / 4 : 0;
    auto add = [&](uint32_t key) {
        if (IS_FLOAT) key = float_to_key(__uint_as_float(key));
        atomicAdd(&h[0][key & 255], 1u);
        atomicAdd(&h[1][(key >> 8) & 255], 1u);
        atomicAdd(&h[2][(key >> 16) & 255], 1u);
        // the top digit of floating-point data is concentrated in a few bins: aggregate per warp
        const uint32_t d = key >> 24;
        atomicAdd(&h[3][d], 1u);
    };
    const uint4 *in4 = reinterpret_cast<const uint4 *>(in);
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    const unsigned long long nvec_round = (nvec + 31) / 32 * 32;
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < nvec_round; i += stride) {
        if (i < nvec) {
            uint4 q = __ldg(in4 + i);
            add(q.x); add(q.y); add(q.z); add(q.w);
        }
    }
    for (unsigned long long i = nvec * 4 + (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
        add(__ldg(in + i));
    __syncthreads();
    for (int i = threadIdx.x; i < 1024; i += blockDim.x) {
        const uint32_t v = (&h[0][0])[i];
        if (v) atomicAdd(&ctl->hist[0][0] + i, v);
    }
}

// ------------------------------------------------------- onesweep pass ----
struct PassArgs {
    const uint32_t *keys_in;
    const uint32_t *vals_in;  // nullptr on the first pass of a pair sort: payload = position
    uint32_t *keys_out;
    uint32_t *vals_out;
    SortCount cnt;
    SortCtl *ctl;
    unsigned long long *status;  // tiles x 256 look-back words
    Control *control;
    const int *run_flag;
    uint32_t epoch;
    int pass;  // 0..3, digit = bits [8*pass, 8*pass+8)
};

struct __align__(16) PassShared {
    uint32_t warp_hist[RS_WARPS][256];
    uint32_t keys[RS_TILE];
    uint32_t tile_excl[256];
    int64_t gbase[256];
    uint32_t scan_tmp[RS_WARPS];
    uint32_t tile_id;
};

template <bool IS_FLOAT, bool PAYLOAD>
__global__ void __launch_bounds__(RS_THREADS, 2) rs_onesweep_kernel(PassArgs a)
{
    pdl_wait();
    if (a.run_flag && *a.run_flag == 0) return;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    PassShared &sh = *reinterpret_cast<PassShared *>(smem_raw);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const unsigned long long n = a.cnt.get();
    const int shift = 8 * a.pass;

  // persistent blocks: tiles are handed out in order by a ticket counter, so a tile only ever waits
  // for tiles that were taken earlier by blocks that are already running
  for (;;) {
    __syncthreads();  // the previous tile's shared state is no longer needed
    if (tid == 0) sh.tile_id = atomicAdd(&a.ctl->ticket[a.pass], 1u);
    for (int i = tid; i < RS_WARPS * 256; i += RS_THREADS) (&sh.warp_hist[0][0])[i] = 0;
    __syncthreads();
    const uint32_t tile = sh.tile_id;
    const unsigned long long tile_base = (unsigned long long)tile * RS_TILE;
    if (tile_base >= n) return;
    const int valid = (int)min((unsigned long long)RS_TILE, n - tile_base);
    // load: warp-striped, so that (item, lane) order is the input order inside a warp's slice
    uint32_t key[RS_ITEMS];
    const int wbase = warp * (32 * RS_ITEMS);
#pragma unroll
    for (int i = 0; i < RS_ITEMS; ++i) {
        const int local = wbase + i * 32 + lane;
        uint32_t kv = 0xffffffffu;
        if (local < valid) {
            kv = __ldg(a.keys_in + tile_base + local);
            if (IS_FLOAT) kv = float_to_key(__uint_as_float(kv));
        }
        key[i] = kv;
    }

    // rank inside the warp by matching digits (stable: earlier item, lower lane first)
    uint32_t rank[RS_ITEMS];
#pragma unroll
    for (int i = 0; i < RS_ITEMS; ++i) {
        const int local = wbase + i * 32 + lane;
        const bool ok = local < valid;
        const uint32_t d = ok ? ((key[i] >> shift) & 255u) : 256u;
        const unsigned peers = match_bits<9>(d);  // bit 8 separates the padding of the last tile
        const unsigned below = peers & ((1u << lane) - 1u);
        const int leader = __ffs(peers) - 1;
        uint32_t prev = 0;
        if (ok && below == 0) {
            prev = sh.warp_hist[warp][d];
            sh.warp_hist[warp][d] = prev + __popc(peers);
        }
        prev = __shfl_sync(FULL, prev, leader);
        rank[i] = prev + __popc(below);
        __syncwarp();
    }
    __syncthreads();

    // per digit: exclusive offsets of the warps inside the tile, tile count
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
        // publish the tile's aggregate (tile 0: already an inclusive prefix)
        const uint32_t flag = (tile == 0) ? RS_FLAG_PREFIX : RS_FLAG_AGG;
        atomicExch(a.status + (unsigned long long)tile * 256 + tid, rs_pack(a.epoch, flag, tile_count));
    }
    // exclusive scan over the 256 digits: tile-local bin starts and global bin starts
    {
        uint32_t v = (tid < 256) ? tile_count : 0;
        uint32_t g = (tid < 256) ? a.ctl->hist[a.pass][tid] : 0;
        uint32_t vi = v, gi = g;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t t1 = __shfl_up_sync(FULL, vi, o), t2 = __shfl_up_sync(FULL, gi, o);
            if (lane >= o) { vi += t1; gi += t2; }
        }
        if (tid < 256 && lane == 31) { sh.scan_tmp[warp] = vi; sh.scan_tmp[8 + warp] = gi; }
        __syncthreads();
        if (tid < 256) {
            uint32_t vo = 0, go = 0;
            for (int w = 0; w < warp; ++w) { vo += sh.scan_tmp[w]; go += sh.scan_tmp[8 + w]; }
            sh.tile_excl[tid] = vo + vi - v;
            sh.gbase[tid] = (int64_t)(go + gi - g);  // start of the digit's bin in the output
        }
    }
    // decoupled look-back: sum the counts of all earlier tiles for this digit.  Predecessor words are
    // fetched RS_WINDOW at a time (independent loads) so that a run of tiles that all started together
    // costs one memory round trip per window instead of one per tile.
    if (tid < 256 && tile > 0) {
        uint32_t excl = 0;
        bool timed_out = false, done = false;
        long long t = (long long)tile - 1;
        while (t >= 0 && !done && !timed_out) {
            const int wlen = (int)min((long long)RS_WINDOW, t + 1);
            unsigned long long s[RS_WINDOW];
#pragma unroll
            for (int i = 0; i < RS_WINDOW; ++i)
                if (i < wlen) s[i] = *((const volatile unsigned long long *)(a.status + (unsigned long long)(t - i) * 256 + tid));
#pragma unroll
            for (int i = 0; i < RS_WINDOW; ++i) {
                if (i >= wlen || done || timed_out) continue;
                unsigned long long sv = s[i];
                int spins = 0;
                while (((uint32_t)(sv >> 32) != a.epoch || ((sv >> 30) & 3u) == 0u) && spins < RS_SPIN_LIMIT) {
                    __nanosleep(20);
                    sv = *((const volatile unsigned long long *)(a.status + (unsigned long long)(t - i) * 256 + tid));
                    ++spins;
                }
                if ((uint32_t)(sv >> 32) != a.epoch || ((sv >> 30) & 3u) == 0u) { timed_out = true; continue; }
                excl += (uint32_t)(sv & 0x3fffffffu);
                if (((sv >> 30) & 3u) == RS_FLAG_PREFIX) done = true;
            }
            t -= wlen;
        }
        if (timed_out) {
            set_status(a.control, 0x10u);
            atomicAdd(&a.control->persist.lookback_timeouts, 1ull);
        }
        atomicExch(a.status + (unsigned long long)tile * 256 + tid, rs_pack(a.epoch, RS_FLAG_PREFIX, excl + tile_count));
        sh.gbase[tid] += (int64_t)excl;
    }
    __syncthreads();
    if (tid < 256) sh.gbase[tid] -= (int64_t)sh.tile_excl[tid];  // out index = gbase[d] + slot
    // scatter into tile order
    uint32_t slot[RS_ITEMS];
#pragma unroll
    for (int i = 0; i < RS_ITEMS; ++i) {
        const int local = wbase + i * 32 + lane;
        if (local < valid) {
            const uint32_t d = (key[i] >> shift) & 255u;
            slot[i] = sh.tile_excl[d] + sh.warp_hist[warp][d] + rank[i];
            sh.keys[slot[i]] = key[i];
        }
    }
    __syncthreads();
    // coalesced write-out: consecutive slots of one digit are consecutive in the output
    int64_t dst[RS_ITEMS];
#pragma unroll
    for (int i = 0; i < RS_ITEMS; ++i) {
        const int q = tid + i * RS_THREADS;
        dst[i] = -1;
        if (q < valid) {
            const uint32_t kv = sh.keys[q];
            dst[i] = sh.gbase[(kv >> shift) & 255u] + q;
            a.keys_out[dst[i]] = kv;
        }
    }
    if (PAYLOAD) {
        __syncthreads();
#pragma unroll
        for (int i = 0; i < RS_ITEMS; ++i) {
            const int local = wbase + i * 32 + lane;
            if (local < valid)
                sh.keys[slot[i]] = a.vals_in ? __ldg(a.vals_in + tile_base + local) : (uint32_t)(tile_base + local);
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < RS_ITEMS; ++i) {
            const int q = tid + i * RS_THREADS;
            if (q < valid) a.vals_out[dst[i]] = sh.keys[q];
        }
    }
  }  // next tile
}

}  // namespace lapsum
