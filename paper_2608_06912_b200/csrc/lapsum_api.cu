// C ABI of the LapSum solver: argument checks, workspace layout, path dispatch
// and kernel launches.  No allocation, no host synchronisation in
// forward/backward; everything is enqueued on the caller's stream.
#include <cmath>
#include <cstdio>
#include <cstring>
#include <atomic>
#include <memory>
#include <mutex>
#include <unordered_map>
#include <vector>

#include "../../include/lapsum.h"
#include "common.cuh"
#include "bracket_select.cuh"
#include "global_path.cuh"
#include "radix_sort.cuh"
#include "row_block.cuh"
#include "solve.cuh"

using namespace lapsum;

namespace {

std::atomic<int64_t> g_launches{0};
thread_local int g_last_cuda = 0;

constexpr int BLOCK_MAX_N = 16384;
constexpr int SOLVE_BLOCKS = 8;  // blocks that share the band solve's one pass over the band
constexpr int64_t BRACKET_FLOOR_N = 4096;  // below this the sample (256 scores) is too small to be worth a bracket
constexpr int STREAM_THREADS = 512;

inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

struct Layout {
    int64_t rows = 0, n = 0;
    lapsum_params prm{};
    int path = 0;
    int64_t K = 0, stride = 0, cap = 0;
    int grid_stream = 0;
    int64_t rs_tiles = 0, scan_tiles = 0;
    size_t off_control = 0, off_th = 0, off_rowparams = 0, off_noise = 0, off_sample[2] = {0, 0}, off_band_keys[2] = {0, 0},
           off_full_keys[2] = {0, 0}, off_full_idx[2] = {0, 0}, off_aggs = 0, off_pref = 0,
           off_suf = 0, off_status = 0, off_partials = 0, total = 0;
    // A batch of long rows works on up to MAX_ROW_SLOTS rows at a time, each in its own copy ("slot") of everything
    // above: slot s starts at s * slot_bytes.  The bracket path serves a group of `slots` rows with one launch per kernel
    // (blockIdx.y = the row within the group); the full-sort path loops over the rows, slot by slot, on up to
    // ROW_STREAMS streams.  Thresholds and parameters of all rows live in slot 0.
    int slots = 1;
    size_t slot_bytes = 0;
    bool sharded = false;  // workspace of one shard of a row that is spread over several GPUs: no full-sort buffers
};
constexpr int MAX_ROW_SLOTS = 16;  // rows of a batch of long rows that one launch serves (bracket path)
constexpr int ROW_STREAMS = 4;     // streams of the row-by-row loop (full-sort path, full_sorts mode)

struct Profile {
    bool on = false;
    uint32_t mask = 0;
    int used = 0;
    std::vector<cudaEvent_t> ev0, ev1;
    std::vector<int> kid;
};

// Side streams and events of the host-buffer entry point (created on its first call, destroyed with the
// workspace's registration)
struct HostPipe {
    cudaStream_t h2d = nullptr, d2h = nullptr;
    cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    bool ready = false;
};

// Side streams of a batch of long rows (created on the first such call, destroyed with the registration)
struct RowPipe {
    cudaStream_t side[ROW_STREAMS - 1] = {};
    cudaEvent_t fork = nullptr, done[ROW_STREAMS - 1] = {};
    bool ready = false;
};

struct WsInfo {
    std::mutex mu;  // held while a call enqueues work for this workspace: calls on different workspaces do not wait for each other
    Layout lay;
    Profile prof;
    HostPipe pipe;
    RowPipe rowpipe;
    size_t bytes = 0;
    void *base = nullptr;  // the workspace itself (slot 0)
    uint64_t seed = 0;
    int device = 0;
    int sm_count = 148;
    // per slot: the per-call control scalars are zero (workspace_init, or a bracket forward whose mask kernel cleared
    // them behind itself); whoever dirties them without clearing resets the flag
    bool call_clean[MAX_ROW_SLOTS] = {};
};

std::mutex g_mu;  // guards the registry only (lookup, insert, erase)
std::unordered_map<void *, std::shared_ptr<WsInfo>> g_ws;

// A registered workspace, kept alive and locked for the duration of one call
struct WsHandle {
    std::shared_ptr<WsInfo> keep;
    std::unique_lock<std::mutex> lock;
    WsInfo *W = nullptr;
};

int cuda_fail(cudaError_t e)
{
    g_last_cuda = (int)e;
    return LAPSUM_ERR_CUDA;
}
#define CU(x)                                   \
    do {                                        \
        cudaError_t e__ = (x);                  \
        if (e__ != cudaSuccess) return cuda_fail(e__); \
    } while (0)

int64_t sample_count(int64_t n)
{   // least K with K^3 >= n^2  (K = ceil(n^(2/3)), Alg. 1 line 1)
    unsigned __int128 n2 = (unsigned __int128)n * (unsigned __int128)n;
    int64_t K = (int64_t)std::cbrt((long double)n * (long double)n);
    if (K < 1) K = 1;
    while (K > 1 && (unsigned __int128)(K - 1) * (K - 1) * (K - 1) >= n2) --K;
    while ((unsigned __int128)K * K * K < n2) ++K;
    return K;
}

int check_params(const lapsum_params &p)
{
    if (!(p.z > 0.0) || !std::isfinite(p.z)) return LAPSUM_ERR_PARAM;
    if (p.force_path < 0 || p.force_path > 3) return LAPSUM_ERR_PARAM;
    if (p.block_max_n < 1 || p.block_max_n > BLOCK_MAX_N) return LAPSUM_ERR_PARAM;
    if (p.band_capacity < 0 || p.bracket_min_n < 1) return LAPSUM_ERR_PARAM;
    if (p.full_sorts != 0 && p.full_sorts != 1) return LAPSUM_ERR_PARAM;
    if (p.max_widenings < 0 || p.max_widenings > 8) return LAPSUM_ERR_PARAM;
    if (p.io_dtype < LAPSUM_IO_F32 || p.io_dtype > LAPSUM_IO_BF16) return LAPSUM_ERR_PARAM;
    return LAPSUM_OK;
}

int choose_path(int64_t rows, int64_t n, const lapsum_params &p, int *path)
{
    int want = p.force_path;
    if (want == LAPSUM_PATH_AUTO) {
        // a single row of more than 8192 scores is faster on the bracket path than in one thread block
        // (n = 16384: 62 us against 108 us per forward + backward); batches keep the block path, which runs all rows at once
        const bool lone_long_row = rows == 1 && n > 8192 && n >= BRACKET_FLOOR_N && n >= p.bracket_min_n / 2;
        if (n <= p.block_max_n && !lone_long_row) want = LAPSUM_PATH_BLOCK;
        else if ((n >= p.bracket_min_n || lone_long_row) && n >= BRACKET_FLOOR_N) want = LAPSUM_PATH_BRACKET;
        else want = LAPSUM_PATH_FULLSORT;
    }
    if (want == LAPSUM_PATH_BLOCK && n > BLOCK_MAX_N) return LAPSUM_ERR_PARAM;
    if (want == LAPSUM_PATH_BRACKET && n < BRACKET_FLOOR_N) return LAPSUM_ERR_PARAM;
    *path = want;
    return LAPSUM_OK;
}

int make_layout(int64_t rows, int64_t n, const lapsum_params *prm_in, int sm_count, Layout *out, bool sharded = false)
{
    if (rows < 1 || n < 1 || n > LAPSUM_MAX_N) return LAPSUM_ERR_SHAPE;
    Layout L;
    L.rows = rows;
    L.n = n;
    L.sharded = sharded;
    if (prm_in) L.prm = *prm_in;
    else lapsum_default_params(&L.prm);
    int rc = check_params(L.prm);
    if (rc) return rc;
    if (sharded) {
        // a sharded row is solved on the bracket path (radix selection, bucketed band solve), fp32 storage
        if (L.prm.full_sorts || L.prm.io_dtype != LAPSUM_IO_F32 || rows != 1) return LAPSUM_ERR_PARAM;
        L.prm.force_path = LAPSUM_PATH_BRACKET;
    }
    rc = choose_path(rows, n, L.prm, &L.path);
    if (rc) return rc;

    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off = align_up(off + bytes);
        return o;
    };
    L.off_control = take(sizeof(Control));
    L.off_th = take(sizeof(RowThreshold) * (size_t)rows);
    L.off_rowparams = take(sizeof(RowParams) * (size_t)rows);
    L.grid_stream = sm_count * 4;
    L.off_partials = take(sizeof(double) * 8 * (size_t)L.grid_stream);
    const bool global = L.path != LAPSUM_PATH_BLOCK && !sharded;
    const bool payload = L.prm.sort_payload != 0;
    int64_t sort_max = 0;
    if (L.path == LAPSUM_PATH_BRACKET) {
        L.K = sample_count(n);
        L.stride = n / L.K;
        L.cap = L.prm.band_capacity > 0
                    ? L.prm.band_capacity
                    : std::max<int64_t>(8192, (int64_t)std::ceil(8.0 * L.prm.z * (double)n / std::sqrt((double)L.K)));
        if (L.cap > n) L.cap = n;
        L.off_noise = take(sizeof(float) * (size_t)L.K);
        for (int i = 0; i < 2; ++i) L.off_sample[i] = take(4 * (size_t)L.K);
        for (int i = 0; i < 2; ++i) L.off_band_keys[i] = take(4 * (size_t)L.cap);
    }
    if (global) {
        for (int i = 0; i < 2; ++i) L.off_full_keys[i] = take(4 * (size_t)n);
        if (payload)
            for (int i = 0; i < 2; ++i) L.off_full_idx[i] = take(4 * (size_t)n);
        sort_max = n;
        L.rs_tiles = (sort_max + RS_TILE - 1) / RS_TILE;
        L.scan_tiles = (sort_max + TILE_S - 1) / TILE_S;
        L.off_aggs = take(sizeof(TileAgg) * (size_t)L.scan_tiles);
        L.off_pref = take(4 * (size_t)L.scan_tiles);
        L.off_suf = take(4 * (size_t)L.scan_tiles);
        L.off_status = take(8 * 256 * (size_t)L.rs_tiles);
    }
    L.slot_bytes = off;
    L.slots = 1;
    if (global && rows > 1) {
        L.slots = (int)std::min<int64_t>(rows, MAX_ROW_SLOTS);
        while (L.slots > 1 && (double)L.slots * (double)L.slot_bytes > 8e9) --L.slots;  // long rows: fewer at a time
    }
    L.total = L.slot_bytes * (size_t)L.slots;
    *out = L;
    return LAPSUM_OK;
}

template <typename T>
T *at(void *ws, size_t off) { return reinterpret_cast<T *>(reinterpret_cast<unsigned char *>(ws) + off); }

int lock_ws(void *ws, WsHandle &h)
{
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_ws.find(ws);
        if (it == g_ws.end()) return LAPSUM_ERR_WORKSPACE;
        h.keep = it->second;
    }
    h.lock = std::unique_lock<std::mutex>(h.keep->mu);
    h.W = h.keep.get();
    return LAPSUM_OK;
}

int post_launch()
{
    g_launches.fetch_add(1, std::memory_order_relaxed);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e);
    return LAPSUM_OK;
}
int prof_begin(WsInfo &W, int kid, cudaStream_t st);
void prof_end(WsInfo &W, int slot, cudaStream_t st);
// launch `...` as kernel `kid` of workspace W on stream st, optionally bracketed by profiling events
// Every kernel is launched with programmatic stream serialisation: its blocks may be scheduled while
// the previous kernel of the stream drains, and its first instruction (pdl_wait) holds it until that
// kernel's memory operations are complete and visible.  This hides most of the launch latency of the
// short dependent kernels that make up a forward call.
thread_local int g_cluster_blocks = 0;  // > 0: the next launch_kernel groups that many blocks into a cluster
// true: the next launch_kernel is an ordinary launch, fully ordered behind the stream's previous kernel AND behind
// whatever that kernel put into its tail-launch stream.  Used for the kernel that follows band_solve_kernel, which
// may launch a widened attempt or the full-sort chain from the device: CUDA orders tail launches before the next
// kernel of the parent's stream, but nothing documents that griddepcontrol.wait of a programmatically launched
// successor also waits for them.
thread_local bool g_plain_launch = false;
template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = g_plain_launch ? 0 : 1;
    g_plain_launch = false;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (g_cluster_blocks > 0) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)g_cluster_blocks;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.numAttrs = 2;
        g_cluster_blocks = 0;
    }
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
// launch kernel `kern` as kernel `kid` of workspace W on stream st, optionally bracketed by profiling events
#define LAUNCH(W, kid, st, kern, grid, block, smem, ...)                                   \
    do {                                                                                   \
        const int slot__ = prof_begin(W, kid, st);                                         \
        cudaError_t le__ = launch_kernel(kern, dim3(grid), dim3(block), (size_t)(smem), st, __VA_ARGS__); \
        prof_end(W, slot__, st);                                                           \
        if (le__ != cudaSuccess) return cuda_fail(le__);                                   \
        int rc__ = post_launch();                                                          \
        if (rc__) return rc__;                                                             \
    } while (0)

int prof_begin(WsInfo &W, int kid, cudaStream_t st)
{
    Profile &P = W.prof;
    if (!P.on || !((P.mask >> kid) & 1u) || P.used >= (int)P.ev0.size()) return -1;
    const int slot = P.used++;
    P.kid[(size_t)slot] = kid;
    cudaEventRecord(P.ev0[(size_t)slot], st);
    return slot;
}
void prof_end(WsInfo &W, int slot, cudaStream_t st)
{
    if (slot >= 0) cudaEventRecord(W.prof.ev1[(size_t)slot], st);
}
void prof_destroy(Profile &P)
{
    for (auto e : P.ev0) cudaEventDestroy(e);
    for (auto e : P.ev1) cudaEventDestroy(e);
    P = Profile{};
}

std::once_flag g_attr_once[16];
int g_attr_rc[16];

int set_kernel_attributes(int device)
{
    if (device < 0 || device >= 16) device = 0;
    std::call_once(g_attr_once[device], [device]() {
        int rc = 0;
        auto set = [&](const void *f, size_t bytes) {
            if (cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) rc = 1;
        };
        set((const void *)rs_onesweep_kernel<RS_IN_KEYS, false>, sizeof(PassShared<false>));
        set((const void *)rs_onesweep_kernel<RS_IN_KEYS, true>, sizeof(PassShared<true>));
        set((const void *)rs_onesweep_kernel<RS_IN_F32, false>, sizeof(PassShared<false>));
        set((const void *)rs_onesweep_kernel<RS_IN_F32, true>, sizeof(PassShared<true>));
        set((const void *)rs_onesweep_kernel<RS_IN_F16, false>, sizeof(PassShared<false>));
        set((const void *)rs_onesweep_kernel<RS_IN_F16, true>, sizeof(PassShared<true>));
        set((const void *)rs_onesweep_kernel<RS_IN_BF16, false>, sizeof(PassShared<false>));
        set((const void *)rs_onesweep_kernel<RS_IN_BF16, true>, sizeof(PassShared<true>));
        const size_t fwd_smem = (3 * 4 * (size_t)BLOCK_MAX_N) / 32 * 33 + 8;
        set((const void *)row_block_forward_kernel<float>, fwd_smem);
        set((const void *)row_block_forward_kernel<__half>, fwd_smem);
        set((const void *)row_block_forward_kernel<__nv_bfloat16>, fwd_smem);
        set((const void *)row_cluster_forward_kernel<float>, fwd_smem / ROW_CLUSTER + 8);
        set((const void *)row_cluster_forward_kernel<__half>, fwd_smem / ROW_CLUSTER + 8);
        set((const void *)row_cluster_forward_kernel<__nv_bfloat16>, fwd_smem / ROW_CLUSTER + 8);
        set((const void *)row_block_sort_pairs_kernel, 8 * (size_t)BLOCK_MAX_N);
        set((const void *)band_solve_kernel, sizeof(BandShared));
        set((const void *)band_solve_group_kernel, sizeof(BandShared));
        g_attr_rc[device] = rc;
    });
    return g_attr_rc[device] ? LAPSUM_ERR_CUDA : LAPSUM_OK;
}

int next_pow2(int x)
{
    int p = 1;
    while (p < x) p <<= 1;
    return p;
}

int block_threads(int n_pad, int64_t rows = 1 << 30, int sm_count = 148)
{
    if (rows <= sm_count) {
        // fewer rows than SMs: a row's latency is all that counts, so one thread per pair of the sort
        if (n_pad <= 64) return 32;
        return std::min(1024, n_pad / 2);
    }
    if (n_pad <= 64) return 32;
    if (n_pad <= 256) return 64;
    if (n_pad <= 1024) return 128;
    if (n_pad <= 4096) return 512;
    return 1024;
}

// ------------------------------------------------------------ sort ----
struct SortJob {
    const void *in;           // first-pass input: keys, or scores of the kind in_kind
    int in_kind;              // RS_IN_KEYS / RS_IN_F32 / RS_IN_F16 / RS_IN_BF16
    uint32_t *keys[2];        // ping-pong
    uint32_t *vals[2];        // payload ping-pong (nullptr: keys only)
    uint32_t *final_keys;     // nullable: last pass writes here instead of the ping-pong buffer
    uint32_t *final_vals;
    SortCount cnt;
    int64_t max_n;            // host bound on the count (grid sizing)
    int slot;
    const int *run_flag;
    int spin_limit = 0;  // 0: RS_SPIN_LIMIT
    int passes = 4;      // the time-out test runs the first pass only
};

// Returns (through *sorted) which buffer holds the sorted keys.
int run_sort(WsInfo &W, void *ws, const SortJob &J, cudaStream_t st, uint32_t **sorted, uint32_t **sorted_vals)
{
    Control *ctl = at<Control>(ws, W.lay.off_control);
    SortCtl *sc = &ctl->call.sort[J.slot];
    uint32_t *status = at<uint32_t>(ws, W.lay.off_status);  // two arrays of rs_tiles x 256 words, used alternately
    const size_t status_words = 256 * (size_t)W.lay.rs_tiles;
    // persistent blocks (two fit on an SM) pull tiles from a ticket counter
    const int tiles = (int)std::min<int64_t>((J.max_n + RS_TILE - 1) / RS_TILE, (int64_t)W.sm_count * 2);
    const int hgrid = (int)std::min<int64_t>((J.max_n + 512 * 16 - 1) / (512 * 16), (int64_t)W.sm_count * 4);
    if (J.in_kind == RS_IN_F32)
        LAUNCH(W, LAPSUM_K_HISTOGRAM, st, rs_histogram_kernel<RS_IN_F32>, std::max(hgrid, 1), 512, 0, J.in, J.cnt, sc, status, J.run_flag);
    else if (J.in_kind == RS_IN_F16)
        LAUNCH(W, LAPSUM_K_HISTOGRAM, st, rs_histogram_kernel<RS_IN_F16>, std::max(hgrid, 1), 512, 0, J.in, J.cnt, sc, status, J.run_flag);
    else if (J.in_kind == RS_IN_BF16)
        LAUNCH(W, LAPSUM_K_HISTOGRAM, st, rs_histogram_kernel<RS_IN_BF16>, std::max(hgrid, 1), 512, 0, J.in, J.cnt, sc, status, J.run_flag);
    else
        LAUNCH(W, LAPSUM_K_HISTOGRAM, st, rs_histogram_kernel<RS_IN_KEYS>, std::max(hgrid, 1), 512, 0, J.in, J.cnt, sc, status, J.run_flag);
    const bool payload = J.vals[0] != nullptr;
    const void *kin = J.in;
    const uint32_t *vin = nullptr;
    int dst = 0;
    // keys-only sorts that start in keys[0] must not overwrite their own input
    if (J.in == J.keys[0]) dst = 1;
    for (int pass = 0; pass < 4; ++pass) {
        PassArgs a;
        a.keys_in = kin;
        a.vals_in = vin;
        a.keys_out = (pass == 3 && J.final_keys) ? J.final_keys : J.keys[dst];
        a.vals_out = payload ? ((pass == 3 && J.final_vals) ? J.final_vals : J.vals[dst]) : nullptr;
        a.cnt = J.cnt;
        a.ctl = sc;
        a.status = status + (size_t)(pass & 1) * status_words;
        a.status_next = status + (size_t)((pass + 1) & 1) * status_words;
        a.control = ctl;
        a.run_flag = J.run_flag;
        a.spin_limit = J.spin_limit > 0 ? J.spin_limit : RS_SPIN_LIMIT;
        a.pass = pass;
        if (pass >= J.passes) break;
        const int kind = (pass == 0) ? J.in_kind : RS_IN_KEYS;
        const size_t smem = payload ? sizeof(PassShared<true>) : sizeof(PassShared<false>);
        if (payload) {
            if (kind == RS_IN_F32) LAUNCH(W, LAPSUM_K_ONESWEEP, st, (rs_onesweep_kernel<RS_IN_F32, true>), tiles, RS_THREADS, smem, a);
            else if (kind == RS_IN_F16) LAUNCH(W, LAPSUM_K_ONESWEEP, st, (rs_onesweep_kernel<RS_IN_F16, true>), tiles, RS_THREADS, smem, a);
            else if (kind == RS_IN_BF16) LAUNCH(W, LAPSUM_K_ONESWEEP, st, (rs_onesweep_kernel<RS_IN_BF16, true>), tiles, RS_THREADS, smem, a);
            else LAUNCH(W, LAPSUM_K_ONESWEEP, st, (rs_onesweep_kernel<RS_IN_KEYS, true>), tiles, RS_THREADS, smem, a);
        } else {
            if (kind == RS_IN_F32) LAUNCH(W, LAPSUM_K_ONESWEEP, st, (rs_onesweep_kernel<RS_IN_F32, false>), tiles, RS_THREADS, smem, a);
            else if (kind == RS_IN_F16) LAUNCH(W, LAPSUM_K_ONESWEEP, st, (rs_onesweep_kernel<RS_IN_F16, false>), tiles, RS_THREADS, smem, a);
            else if (kind == RS_IN_BF16) LAUNCH(W, LAPSUM_K_ONESWEEP, st, (rs_onesweep_kernel<RS_IN_BF16, false>), tiles, RS_THREADS, smem, a);
            else LAUNCH(W, LAPSUM_K_ONESWEEP, st, (rs_onesweep_kernel<RS_IN_KEYS, false>), tiles, RS_THREADS, smem, a);
        }
        kin = a.keys_out;
        vin = a.vals_out;
        dst ^= 1;
    }
    *sorted = static_cast<uint32_t *>(const_cast<void *>(kin));
    if (sorted_vals) *sorted_vals = const_cast<uint32_t *>(vin);
    return LAPSUM_OK;
}

__global__ void keys_to_float_kernel(const uint32_t *keys, float *out, unsigned long long n, const unsigned long long *cnt,
                                     unsigned long long cap)
{
    pdl_wait();
    unsigned long long m = n;
    if (cnt) m = min(*cnt, cap);
    for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < m;
         i += (unsigned long long)gridDim.x * blockDim.x)
        out[i] = key_to_float(keys[i]);
}

struct Scalars {
    double k, t;
    ExpScale sc;
    float c, half_inv_t;
    float c_mask;  // c, negated when alpha > 0
    float gsign;   // +1, or -1 when alpha > 0
};

// alpha > 0 (Eq. 1 as printed: p_i = sigma((b - r_i)/alpha), the k smallest scores) is solved through the identity
// sigma(-u) = 1 - sigma(u): sum_i sigma((b - r_i)/alpha) = k  <=>  sum_i sigma((r_i - b)/alpha) = n - k, i.e. the
// threshold is that of the alpha' = -alpha problem with budget n - k.  Every solve kernel therefore runs unchanged on
// (n - k, t = alpha); only the mask (sigma at (b - r_i)/t: c_mask) and the sign of grad_r (gsign) differ.
Scalars make_scalars(double k, double alpha, int64_t n)
{
    Scalars s;
    s.k = alpha < 0.0 ? k : (double)n - k;
    s.t = std::fabs(alpha);
    s.sc = make_scale(s.t);
    s.c = (float)(1.4426950408889634074 / s.t);
    s.half_inv_t = (float)(0.5 / s.t);
    s.c_mask = alpha < 0.0 ? s.c : -s.c;
    s.gsign = alpha < 0.0 ? 1.f : -1.f;
    return s;
}

// alpha finite, not zero, and a temperature |alpha| that fp32 holds as a normal number (the kernels compute in fp32:
// a smaller one would turn into 0 and 1/t into infinity)
bool alpha_ok(double alpha)
{
    const double t = std::fabs(alpha);
    return std::isfinite(alpha) && t >= 1.1754943508222875e-38 && t <= 3.0e38;
}

int check_problem(int64_t rows, int64_t n, double k, double alpha)
{
    if (rows < 1 || n < 1 || n > LAPSUM_MAX_N) return LAPSUM_ERR_SHAPE;
    if (!alpha_ok(alpha)) return LAPSUM_ERR_ALPHA;
    if (!std::isfinite(k) || !(k > 0.0) || !(k < (double)n)) return LAPSUM_ERR_BUDGET;
    return LAPSUM_OK;
}

// tile_aggregate_kernel: one warp per scan tile, eight tiles per block at a time
int agg_grid(int64_t tiles, int sm_count)
{
    const int64_t per_block = AGG_THREADS / 32;
    return (int)std::max<int64_t>(1, std::min<int64_t>((tiles + per_block - 1) / per_block, (int64_t)sm_count * 8));
}

// element type of scores / masks / gradients (lapsum_io_dtype) as a type, and as the radix sort's input kind
template <typename T> struct IoOf;
template <> struct IoOf<float> { static constexpr int io = LAPSUM_IO_F32, kind = RS_IN_F32; };
template <> struct IoOf<__half> { static constexpr int io = LAPSUM_IO_F16, kind = RS_IN_F16; };
template <> struct IoOf<__nv_bfloat16> { static constexpr int io = LAPSUM_IO_BF16, kind = RS_IN_BF16; };

// blocks of the stream pass: two per SM, but no more than the row has tiles (+ 1 for what the tiles leave over)
int stream_blocks(const WsInfo &W)
{
    const int64_t tiles = W.lay.n / ((int64_t)SB_THREADS * SB_U * 4) + 1;
    return (int)std::min<int64_t>(std::min(W.lay.grid_stream, W.sm_count * 2), tiles);
}

// blocks of 512 threads per SM for the element-wise maps and for the VJP reduction (grid-stride loops)
#ifndef LAPSUM_MAP_BLOCKS_PER_SM
#define LAPSUM_MAP_BLOCKS_PER_SM 8
#endif
#ifndef LAPSUM_REDUCE_BLOCKS_PER_SM
#define LAPSUM_REDUCE_BLOCKS_PER_SM 8
#endif
int map_grid(const WsInfo &W, int64_t n, int per_sm = LAPSUM_MAP_BLOCKS_PER_SM)
{
    const int64_t want = n / (4 * (int64_t)EW_TILE) + 1;  // one block per tile of the row (+ 1 for what the tiles leave over)
    return (int)std::max<int64_t>(1, std::min<int64_t>(want, (int64_t)W.sm_count * per_sm));
}

// full sort of one row + tile scan + solve (App. A); run_flag predicates the whole chain on the device
int enqueue_fullsort_solve(WsInfo &W, void *ws, const void *r_row, int in_kind, const Scalars &S, float *b_row,
                           RowThreshold *th_row, const int *run_flag, const RowParams *rp, cudaStream_t st)
{
    const Layout &L = W.lay;
    Control *ctl = at<Control>(ws, L.off_control);
    SortJob J{};
    J.in = r_row;
    J.in_kind = in_kind;
    J.keys[0] = at<uint32_t>(ws, L.off_full_keys[0]);
    J.keys[1] = at<uint32_t>(ws, L.off_full_keys[1]);
    const bool payload = L.prm.sort_payload != 0;
    J.vals[0] = payload ? at<uint32_t>(ws, L.off_full_idx[0]) : nullptr;
    J.vals[1] = payload ? at<uint32_t>(ws, L.off_full_idx[1]) : nullptr;
    J.cnt = SortCount{nullptr, (unsigned long long)L.n, (unsigned long long)L.n};
    J.max_n = L.n;
    J.slot = 2;
    J.run_flag = run_flag;
    uint32_t *sorted = nullptr;
    int rc = run_sort(W, ws, J, st, &sorted, nullptr);
    if (rc) return rc;
    TileAgg *aggs = at<TileAgg>(ws, L.off_aggs);
    const int agrid = agg_grid(L.scan_tiles, W.sm_count);
    LAUNCH(W, LAPSUM_K_TILE_AGG, st, tile_aggregate_kernel, agrid, AGG_THREADS, 0, sorted, J.cnt, aggs, S.sc, run_flag, rp);
    SolveArgs a{};
    a.keys = sorted;
    a.cnt = J.cnt;
    a.aggs = aggs;
    a.pref = at<float>(ws, L.off_pref);
    a.suf = at<float>(ws, L.off_suf);
    a.ctl = ctl;
    a.b_out = b_row;
    a.th_out = th_row;
    a.run_flag = run_flag;
    a.k = S.k;
    a.t = S.t;
    a.sc = S.sc;
    a.bracket = 0;
    a.cap = 0;
    a.total_n = (unsigned long long)L.n;
    a.rp = rp;
    LAUNCH(W, LAPSUM_K_SOLVE, st, solve_global_kernel, 1, SOLVE_THREADS, 0, a);
    return LAPSUM_OK;
}

// the same chain as enqueue_fullsort_solve, but only described: the device launches it if it is needed
void fill_fullsort_plan(WsInfo &W, void *ws, const void *r_row, int in_kind, const Scalars &S, float *b_row,
                        RowThreshold *th_row, const RowParams *rp, FallbackPlan *f)
{
    const Layout &L = W.lay;
    Control *ctl = at<Control>(ws, L.off_control);
    const bool payload = L.prm.sort_payload != 0;
    uint32_t *keys[2] = {at<uint32_t>(ws, L.off_full_keys[0]), at<uint32_t>(ws, L.off_full_keys[1])};
    uint32_t *vals[2] = {payload ? at<uint32_t>(ws, L.off_full_idx[0]) : nullptr,
                         payload ? at<uint32_t>(ws, L.off_full_idx[1]) : nullptr};
    f->enabled = 1;
    f->hist_grid = (int)std::max<int64_t>(1, std::min<int64_t>((L.n + 512 * 16 - 1) / (512 * 16), (int64_t)W.sm_count * 4));
    f->pass_grid = (int)std::min<int64_t>((L.n + RS_TILE - 1) / RS_TILE, (int64_t)W.sm_count * 2);
    f->agg_grid = agg_grid(L.scan_tiles, W.sm_count);
    f->r_in = r_row;
    f->in_kind = in_kind;
    f->cnt = SortCount{nullptr, (unsigned long long)L.n, (unsigned long long)L.n};
    f->sort_ctl = &ctl->call.sort[2];
    const void *kin = f->r_in;
    const uint32_t *vin = nullptr;
    int dst = 0;
    for (int pass = 0; pass < 4; ++pass) {
        PassArgs &a = f->pass[pass];
        a.keys_in = kin;
        a.vals_in = vin;
        a.keys_out = keys[dst];
        a.vals_out = vals[dst];
        a.cnt = f->cnt;
        a.ctl = f->sort_ctl;
        a.status = at<uint32_t>(ws, L.off_status) + (size_t)(pass & 1) * 256 * (size_t)L.rs_tiles;
        a.status_next = at<uint32_t>(ws, L.off_status) + (size_t)((pass + 1) & 1) * 256 * (size_t)L.rs_tiles;
        a.control = ctl;
        a.run_flag = nullptr;
        a.spin_limit = RS_SPIN_LIMIT;
        a.pass = pass;
        kin = a.keys_out;
        vin = a.vals_out;
        dst ^= 1;
    }
    f->aggs = at<TileAgg>(ws, L.off_aggs);
    f->sc = S.sc;
    SolveArgs &sv = f->solve;
    sv = SolveArgs{};
    sv.keys = static_cast<const uint32_t *>(kin);
    sv.cnt = f->cnt;
    sv.aggs = f->aggs;
    sv.pref = at<float>(ws, L.off_pref);
    sv.suf = at<float>(ws, L.off_suf);
    sv.ctl = ctl;
    sv.b_out = b_row;
    sv.th_out = th_row;
    sv.run_flag = nullptr;
    sv.k = S.k;
    sv.t = S.t;
    sv.sc = S.sc;
    sv.bracket = 0;
    sv.cap = 0;
    sv.total_n = (unsigned long long)L.n;
    sv.rp = rp;
}

void bracket_ranks(int64_t n, int64_t K, double k, double z, int64_t *j, int64_t *l)
{   // Eq. 8
    const double q = ((double)n - k) / (double)n;
    const double mu = (double)K * q;
    const double sd = std::sqrt((double)K * q * (1.0 - q));
    *j = (int64_t)std::floor(mu - z * sd);
    *l = (int64_t)std::ceil(mu + z * sd);
}

// sampling + order statistics + stream pass (Alg. 1 lines 1-3 and 7)
template <typename T>
int enqueue_bracket_stream(WsInfo &W, void *ws, const T *r_row, const Scalars &S, const RowParams *rp, int use_imm,
                           float aL, float aR, float *y_out, cudaStream_t st, StreamArgs *launched = nullptr, int group = 1)
{
    // group > 1: the arguments are those of the group's first row (slot 0); the kernels serve rows 0 .. group-1 at once
    const Layout &L = W.lay;
    Control *ctl = at<Control>(ws, L.off_control);
    const BatchShift bs{(unsigned long long)L.slot_bytes, (unsigned long long)L.n, group > 1 ? 1 : 0};
    const unsigned G = (unsigned)group;
    int64_t j = 0, l = 0;
    bracket_ranks(L.n, L.K, S.k, L.prm.z, &j, &l);  // with rp the kernels read the row's own ranks instead
    if (!use_imm || y_out) {
        uint32_t *sa = at<uint32_t>(ws, L.off_sample[0]);
        if (L.prm.full_sorts) {
            const int g = (int)((L.K + 255) / 256);
            LAUNCH(W, LAPSUM_K_SAMPLE, st, sample_gather_kernel<T>, g, 256, 0, r_row, L.K, L.stride, (uint32_t)(W.seed & 0xffffffffu), at<float>(ws, L.off_noise), (float)S.t, sa, y_out, rp);
            SortJob J{};
            J.in = sa;
            J.in_kind = RS_IN_KEYS;
            J.keys[0] = sa;
            J.keys[1] = at<uint32_t>(ws, L.off_sample[1]);
            J.cnt = SortCount{nullptr, (unsigned long long)L.K, (unsigned long long)L.K};
            J.max_n = L.K;
            J.slot = 0;
            uint32_t *sorted_sample = nullptr;
            int rc = run_sort(W, ws, J, st, &sorted_sample, nullptr);
            if (rc) return rc;
            LAUNCH(W, LAPSUM_K_SAMPLE, st, pick_sorted_kernel, 1, 32, 0, sorted_sample, L.K, j, l, rp, ctl);
        } else {
            SelectArgs sa_args{};
            sa_args.r = r_row;
            sa_args.K = L.K;
            sa_args.stride = L.stride;
            sa_args.seed_lo = (uint32_t)(W.seed & 0xffffffffu);
            sa_args.noise = at<float>(ws, L.off_noise);
            sa_args.tf = (float)S.t;
            sa_args.keys = sa;
            sa_args.y_out = y_out;
            sa_args.j = j;
            sa_args.l = l;
            sa_args.ctl = ctl;
            sa_args.rp = rp;
            PickArgs pk{};
            pk.keys = sa;
            pk.cand = at<uint32_t>(ws, L.off_sample[1]);  // the second sample buffer is free in this mode
            pk.K = L.K;
            pk.j = j;
            pk.l = l;
            pk.cand_cap = L.K / 2;
            pk.ctl = ctl;
            pk.rp = rp;
            pk.bs = bs;
            sa_args.bs = bs;
            const int g = (int)((L.K + SEL_THREADS - 1) / SEL_THREADS);
            if (group > 1) LAUNCH(W, LAPSUM_K_SAMPLE, st, (sample_hist_kernel<T, true>), dim3((unsigned)g, G), SEL_THREADS, 0, sa_args);
            else LAUNCH(W, LAPSUM_K_SAMPLE, st, (sample_hist_kernel<T, false>), g, SEL_THREADS, 0, sa_args);
            const int gp = (int)std::max<int64_t>(1, std::min<int64_t>(64, L.K / 4 / (SEL_THREADS * 2) + 1));
            if (group > 1) LAUNCH(W, LAPSUM_K_SAMPLE, st, sample_pick_kernel<true>, dim3((unsigned)gp, G), SEL_THREADS, 0, pk);
            else LAUNCH(W, LAPSUM_K_SAMPLE, st, sample_pick_kernel<false>, gp, SEL_THREADS, 0, pk);
        }
    }
    StreamArgs a{};
    a.r = r_row;
    a.n = (unsigned long long)L.n;
    a.sel = &ctl->call.sel_keys[0];
    a.fscale = fixed_scale((unsigned long long)L.cap);
    a.K = L.K;
    a.j = j;
    a.l = l;
    a.rp = rp;
    a.use_imm = use_imm;
    a.aL_imm = aL;
    a.aR_imm = aR;
    a.c = S.c;
    a.sc = S.sc;
    a.band_keys = at<uint32_t>(ws, L.off_band_keys[0]);
    a.band_idx = nullptr;  // the solve needs only the band's keys
    a.cap = (unsigned long long)L.cap;
    a.partials = at<double>(ws, L.off_partials);
    a.ctl = ctl;
    a.bs = bs;
    // one generation of blocks (two resident per SM): the block epilogue (queue flush, three block sums) is paid once
    if (group > 1) LAUNCH(W, LAPSUM_K_STREAM_BAND, st, stream_band_group_kernel<T>, dim3((unsigned)stream_blocks(W), G), STREAM_THREADS, 0, a);
    else LAUNCH(W, LAPSUM_K_STREAM_BAND, st, stream_band_kernel<T>, stream_blocks(W), STREAM_THREADS, 0, a);
    if (launched) *launched = a;
    return LAPSUM_OK;
}

template <typename T>
int enqueue_bracket_forward(WsInfo &W, void *ws, const T *r_row, const Scalars &S, const RowParams *rp, T *p_row,
                            float *b_row, RowThreshold *th_row, int use_imm, float aL, float aR, bool last_row,
                            cudaStream_t st, int group = 1)
{
    // group > 1 (default mode only): rows 0 .. group-1 from r_row on, in slots 0 .. group-1 from ws on, one launch per
    // kernel; p_row, b_row, th_row and rp are those of the group's first row
    const Layout &L = W.lay;
    Control *ctl = at<Control>(ws, L.off_control);
    const int slot = L.slot_bytes ? (int)(((unsigned char *)ws - (unsigned char *)W.base) / L.slot_bytes) : 0;
    const BatchShift bs{(unsigned long long)L.slot_bytes, (unsigned long long)L.n, group > 1 ? 1 : 0};
    const unsigned G = (unsigned)group;
    if (group > 1 && (L.prm.full_sorts || use_imm || slot + group > L.slots)) return LAPSUM_ERR_UNSUPPORTED;
    for (int g = 0; g < group; ++g) {
        if (!W.call_clean[slot + g]) CU(cudaMemsetAsync(&at<Control>(ws, (size_t)g * L.slot_bytes + L.off_control)->call, 0, sizeof(CallCtl), st));
        W.call_clean[slot + g] = false;  // until this forward's last kernel is enqueued
    }
    StreamArgs launched{};
    int rc = enqueue_bracket_stream(W, ws, r_row, S, rp, use_imm, aL, aR, nullptr, st, &launched, group);
    if (rc) return rc;
    if (!L.prm.full_sorts) {
        // bucket the band by key range and sort only the bucket that holds the root
        BandArgs ba{};
        ba.band = at<uint32_t>(ws, L.off_band_keys[0]);
        ba.glist = at<uint32_t>(ws, L.off_band_keys[1]);  // the second band buffer is free in this mode (cap >= 8192 keys)
        ba.ctl = ctl;
        ba.b_out = b_row;
        ba.th_out = th_row;
        ba.cap = (unsigned long long)L.cap;
        ba.fscale = fixed_scale((unsigned long long)L.cap);
        ba.k = S.k;
        ba.t = S.t;
        ba.sc = S.sc;
        ba.c = S.c;
        fill_fullsort_plan(W, ws, r_row, IoOf<T>::kind, S, b_row, th_row, rp, &ba.fb);
        ba.rp = rp;
        ba.io = IoOf<T>::io;
        ba.stream = launched;
        ba.stream_grid = stream_blocks(W);
        // several blocks share the pass over the band only when the band is expected to be long: for a short one
        // the hand-over (ticket, fence, re-read of the gathered list) costs more than the pass
        int solve_blocks = 1;
        if (rp) {
            // the rows' budgets live on the device: go by the longest band Eq. 8 can give (the buffer's size)
            if (!use_imm && L.cap >= 65536) solve_blocks = SOLVE_BLOCKS;
        } else if (!use_imm) {
            int64_t j = 0, l = 0;
            bracket_ranks(L.n, L.K, S.k, L.prm.z, &j, &l);
            const double expected_band = (double)(std::min(l, L.K) - std::max<int64_t>(j, 1)) / (double)L.K * (double)L.n;
            if (expected_band >= 65536.0) solve_blocks = SOLVE_BLOCKS;
        }
        ba.solve_blocks = solve_blocks;
        ba.attempt = 0;
        ba.max_widen = L.prm.max_widenings;
        ba.bs = bs;
        if (group > 1) LAUNCH(W, LAPSUM_K_SOLVE, st, band_solve_group_kernel, dim3((unsigned)solve_blocks, G), 1024, sizeof(BandShared), ba);
        else LAUNCH(W, LAPSUM_K_SOLVE, st, band_solve_kernel, solve_blocks, 1024, sizeof(BandShared), ba);
    } else {
    // sort the middle band (its size is known only on the device)
    SortJob J{};
    J.in = at<uint32_t>(ws, L.off_band_keys[0]);
    J.in_kind = RS_IN_KEYS;
    J.keys[0] = at<uint32_t>(ws, L.off_band_keys[0]);
    J.keys[1] = at<uint32_t>(ws, L.off_band_keys[1]);
    J.cnt = SortCount{&ctl->call.band_count, 0, (unsigned long long)L.cap};
    J.max_n = L.cap;
    J.slot = 1;
    uint32_t *sorted = nullptr;
    rc = run_sort(W, ws, J, st, &sorted, nullptr);
    if (rc) return rc;
    TileAgg *aggs = at<TileAgg>(ws, L.off_aggs);
    const int64_t band_tiles = (L.cap + TILE_S - 1) / TILE_S;
    const int agrid = agg_grid(band_tiles, W.sm_count);
    LAUNCH(W, LAPSUM_K_TILE_AGG, st, tile_aggregate_kernel, agrid, AGG_THREADS, 0, sorted, J.cnt, aggs, S.sc, nullptr, rp);
    SolveArgs a{};
    a.keys = sorted;
    a.cnt = J.cnt;
    a.aggs = aggs;
    a.pref = at<float>(ws, L.off_pref);
    a.suf = at<float>(ws, L.off_suf);
    a.ctl = ctl;
    a.b_out = b_row;
    a.th_out = th_row;
    a.run_flag = nullptr;
    a.k = S.k;
    a.t = S.t;
    a.sc = S.sc;
    a.bracket = 1;
    a.cap = (unsigned long long)L.cap;
    a.total_n = (unsigned long long)L.n;
    a.rp = rp;
    LAUNCH(W, LAPSUM_K_SOLVE, st, solve_global_kernel, 1, SOLVE_THREADS, 0, a);
    }
    // Alg. 1 line 5: if the certificate failed, fall back to the exact full-sort solve.  The default mode lets
    // band_solve launch that chain from the device; full_sorts keeps the host-enqueued, device-predicated chain.
    if (L.prm.full_sorts) {
        rc = enqueue_fullsort_solve(W, ws, r_row, IoOf<T>::kind, S, b_row, th_row, &ctl->call.fallback, rp, st);
        if (rc) return rc;
    }
    // band_solve_kernel may have tail-launched a widened attempt or the full sort: its successor is an ordinary launch
    if (!L.prm.full_sorts) g_plain_launch = true;
    const int note = !last_row ? 0 : group > 1 ? (L.path | (group << 8)) : L.path;  // the group's last row closes the call
    if (L.n >= CDF_LONG_N) LAUNCH(W, LAPSUM_K_CDF_MAP, st, (cdf_map_kernel<T, CDF_U_LONG>), dim3((unsigned)map_grid(W, L.n), G), 512, 0, r_row, p_row, (unsigned long long)L.n, th_row, S.c_mask, ctl, note, rp, 1, bs);
    else LAUNCH(W, LAPSUM_K_CDF_MAP, st, (cdf_map_kernel<T, CDF_U_SHORT>), dim3((unsigned)map_grid(W, L.n), G), 512, 0, r_row, p_row, (unsigned long long)L.n, th_row, S.c_mask, ctl, note, rp, 1, bs);
    for (int g = 0; g < group; ++g) W.call_clean[slot + g] = true;
    return LAPSUM_OK;
}

// ---- scratch of lapsum_backward_static: lives in the library image, one copy per GPU that loads it ----
// Layout: a Control block (only its VJP ticket and row sums are used) followed by 4 doubles per block.
constexpr int STATIC_MAX_BLOCKS = 148 * 8;
constexpr size_t STATIC_PARTIALS_OFF = (sizeof(Control) + 255) / 256 * 256;
static_assert(STATIC_PARTIALS_OFF + sizeof(double) * 4 * STATIC_MAX_BLOCKS <= LAPSUM_STATIC_SCRATCH_BYTES,
              "static scratch too small");
static __device__ __align__(256) unsigned char g_static_scratch[LAPSUM_STATIC_SCRATCH_BYTES];

std::mutex g_static_mu;
void *g_static_ptr[16] = {nullptr};  // device address of g_static_scratch, per device

// streams, events and profiling records that belong to a workspace's registration
void release_host_objects(WsInfo &W)
{
    prof_destroy(W.prof);
    HostPipe &hp = W.pipe;
    if (hp.ready) {
        for (cudaEvent_t e : hp.ev)
            if (e) cudaEventDestroy(e);
        if (hp.h2d) cudaStreamDestroy(hp.h2d);
        if (hp.d2h) cudaStreamDestroy(hp.d2h);
    }
    RowPipe &rp = W.rowpipe;
    if (rp.ready) {
        if (rp.fork) cudaEventDestroy(rp.fork);
        for (cudaEvent_t e : rp.done)
            if (e) cudaEventDestroy(e);
        for (cudaStream_t q : rp.side)
            if (q) cudaStreamDestroy(q);
    }
    W.pipe = HostPipe{};
    W.rowpipe = RowPipe{};
}

}  // namespace

// =================================================================== API ===
extern "C" {

void lapsum_default_params(lapsum_params *prm)
{
    if (!prm) return;
    std::memset(prm, 0, sizeof(*prm));
    prm->z = 5.16;
    prm->bracket_min_n = 16385;
    prm->band_capacity = 0;
    prm->force_path = LAPSUM_PATH_AUTO;
    prm->sort_payload = 0;
    prm->block_max_n = BLOCK_MAX_N;
    prm->full_sorts = 0;
    prm->max_widenings = 2;
    prm->io_dtype = LAPSUM_IO_F32;
}

int lapsum_workspace_bytes(int64_t rows, int64_t n, const lapsum_params *prm, size_t *bytes)
{
    if (!bytes) return LAPSUM_ERR_NULL;
    Layout L;
    int rc = make_layout(rows, n, prm, 148, &L);
    if (rc) return rc;
    *bytes = L.total;
    return LAPSUM_OK;
}

int lapsum_describe(int64_t rows, int64_t n, double k, const lapsum_params *prm, lapsum_plan *out)
{
    if (!out) return LAPSUM_ERR_NULL;
    Layout L;
    int rc = make_layout(rows, n, prm, 148, &L);
    if (rc) return rc;
    if (k != 0.0 && (!std::isfinite(k) || !(k > 0.0) || !(k < (double)n))) return LAPSUM_ERR_BUDGET;
    *out = lapsum_plan{};
    out->path = L.path;
    out->workspace_bytes = L.total;
    if (L.path == LAPSUM_PATH_BRACKET) {
        out->K = L.K;
        out->stride = L.stride;
        out->band_capacity = L.cap;
        if (k != 0.0) bracket_ranks(L.n, L.K, k, L.prm.z, &out->j, &out->l);
    }
    return LAPSUM_OK;
}

static int workspace_init_impl(void *ws, size_t bytes, int64_t rows, int64_t n, const lapsum_params *prm, uint64_t seed,
                               void *stream, bool sharded)
{
    if (!ws) return LAPSUM_ERR_NULL;
    if (((uintptr_t)ws & 255) != 0) return LAPSUM_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    std::shared_ptr<WsInfo> fresh = std::make_shared<WsInfo>();
    WsInfo &W = *fresh;
    int rc = make_layout(rows, n, prm, 148, &W.lay, sharded);
    if (rc) return rc;
    if (bytes < W.lay.total) return LAPSUM_ERR_WORKSPACE;
    CU(cudaGetDevice(&W.device));
    int sms = 0;
    CU(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, W.device));
    W.sm_count = sms > 0 ? sms : 148;
    // the layout is sized with 148 SMs per grid; never launch wider than that sizing
    if (W.sm_count > 148) W.sm_count = 148;
    W.lay.grid_stream = std::min(W.lay.grid_stream, W.sm_count * 4);
    W.bytes = bytes;
    W.base = ws;
    W.seed = seed;
    rc = set_kernel_attributes(W.device);
    if (rc) return rc;
    const Layout &L = W.lay;
    std::vector<float> noise;
    if (L.path == LAPSUM_PATH_BRACKET) {
        // unit-Laplace kernel noise by inverse CDF of a hashed counter, fp64 on the host, one rounding to fp32
        noise.resize((size_t)L.K);
        const uint32_t seed_hi = (uint32_t)(seed >> 32);
        for (int64_t s = 0; s < L.K; ++s) {
            const uint32_t h = mix32((uint32_t)s * 0x9E3779B9u + (seed_hi ^ 0x68E31DA4u));
            const double U = ((double)h + 0.5) / 4294967296.0;
            const double e = (U < 0.5) ? std::log(2.0 * U) : -std::log(2.0 * (1.0 - U));
            noise[(size_t)s] = (float)e;
        }
    }
    for (int slot = 0; slot < L.slots; ++slot) {
        void *wsS = at<unsigned char>(ws, (size_t)slot * L.slot_bytes);
        CU(cudaMemsetAsync(at<unsigned char>(wsS, L.off_control), 0, sizeof(Control), st));
        CU(cudaMemsetAsync(at<unsigned char>(wsS, L.off_th), 0, sizeof(RowThreshold) * (size_t)rows, st));
        if (L.off_status) CU(cudaMemsetAsync(at<unsigned char>(wsS, L.off_status), 0, 8 * 256 * (size_t)L.rs_tiles, st));
        if (L.path == LAPSUM_PATH_BRACKET)
            CU(cudaMemcpyAsync(at<float>(wsS, L.off_noise), noise.data(), sizeof(float) * (size_t)L.K, cudaMemcpyHostToDevice, st));
    }
    CU(cudaStreamSynchronize(st));
    for (bool &c : W.call_clean) c = true;  // every slot's control block was just zeroed
    std::shared_ptr<WsInfo> old;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_ws.find(ws);
        if (it != g_ws.end()) old = it->second;
        g_ws[ws] = fresh;
    }
    if (old) {  // re-initialised in place: the earlier registration's streams and events go (once no call holds it)
        std::lock_guard<std::mutex> lk(old->mu);
        release_host_objects(*old);
    }
    return LAPSUM_OK;
}

int lapsum_workspace_init(void *ws, size_t bytes, int64_t rows, int64_t n, const lapsum_params *prm, uint64_t seed,
                          void *stream)
{
    return workspace_init_impl(ws, bytes, rows, n, prm, seed, stream, false);
}

int lapsum_workspace_release(void *ws)
{
    std::shared_ptr<WsInfo> gone;
    {
        std::lock_guard<std::mutex> lk(g_mu);
        auto it = g_ws.find(ws);
        if (it == g_ws.end()) return LAPSUM_ERR_WORKSPACE;
        gone = it->second;
        g_ws.erase(it);
    }
    std::lock_guard<std::mutex> lk(gone->mu);  // a call that is still enqueueing for this workspace finishes first
    release_host_objects(*gone);
    return LAPSUM_OK;
}

extern "C++" {
namespace {
// A batch of long rows: row i runs in slot i % slots, slot 0 on the caller's stream and the others on side streams that
// start behind what the caller's stream holds (fork) and that the caller's stream waits for at the end (join).
int rows_fork(WsInfo &W, cudaStream_t st)
{
    RowPipe &rp = W.rowpipe;
    const int sides = std::min(W.lay.slots, ROW_STREAMS) - 1;
    if (sides <= 0) return LAPSUM_OK;
    if (!rp.ready) {
        CU(cudaEventCreateWithFlags(&rp.fork, cudaEventDisableTiming));
        for (int i = 0; i < sides; ++i) {
            CU(cudaStreamCreateWithFlags(&rp.side[i], cudaStreamNonBlocking));
            CU(cudaEventCreateWithFlags(&rp.done[i], cudaEventDisableTiming));
        }
        rp.ready = true;
    }
    CU(cudaEventRecord(rp.fork, st));
    for (int i = 0; i < sides; ++i) CU(cudaStreamWaitEvent(rp.side[i], rp.fork, 0));
    return LAPSUM_OK;
}
int rows_join(WsInfo &W, cudaStream_t st)
{
    RowPipe &rp = W.rowpipe;
    for (int i = 0; i < std::min(W.lay.slots, ROW_STREAMS) - 1; ++i) {
        CU(cudaEventRecord(rp.done[i], rp.side[i]));
        CU(cudaStreamWaitEvent(st, rp.done[i], 0));
    }
    return LAPSUM_OK;
}
// a slot always runs on the same stream, so that the rows that share it follow one another
cudaStream_t row_stream(WsInfo &W, cudaStream_t st, int64_t row) { const int s = (int)(row % W.lay.slots) % ROW_STREAMS; return s == 0 ? st : W.rowpipe.side[s - 1]; }
void *row_slot(const WsInfo &W, void *ws, int64_t row) { return at<unsigned char>(ws, (size_t)(row % W.lay.slots) * W.lay.slot_bytes); }


// Forward of a batch of short rows (block path): one warp per row up to 128 scores, one thread block per row, or one
// cluster of 4 / 8 blocks per row when the rows are long and few.  keys_dump != nullptr (test hook) runs the same
// kernel in the same launch shape, but it stops after its sort and writes the sorted rows there.
template <typename T>
int launch_block_path_forward(WsInfo &Wi, const T *r, int64_t rows, int64_t n, const Scalars &S, const RowParams *rp, T *p,
                              float *b, RowThreshold *th, Control *ctl, float *keys_dump, cudaStream_t st)
{
    WsInfo *W = &Wi;
    if (n <= 128) {
        // short rows: a group of 16 lanes per row (two rows per warp), the row in registers
        WarpFwdArgs a{r, p, b, th, ctl, (long long)rows, (int)n, S.k, S.t, S.sc, S.c, S.c_mask, rp, keys_dump};
        constexpr int WL = WARP_ROW_LANES;
        const unsigned grid = (unsigned)((rows + WP_WARPS * (32 / WL) - 1) / (WP_WARPS * (32 / WL)));
#define LAPSUM_WARP_FWD1(ITEMS, ROW_P, DUMP)                                                                                       \
    do {                                                                                                                      \
        if (n == (ITEMS) * WL && !(DUMP)) LAUNCH(*W, LAPSUM_K_BLOCK_FWD, st, (row_warp_forward_kernel<ITEMS, WL, ROW_P, false, T, true>), grid, WP_WARPS * 32, 0, a); \
        else LAUNCH(*W, LAPSUM_K_BLOCK_FWD, st, (row_warp_forward_kernel<ITEMS, WL, ROW_P, DUMP, T, false>), grid, WP_WARPS * 32, 0, a); \
    } while (0)
#define LAPSUM_WARP_FWD(ROW_P, DUMP)                                                                                              \
    do {                                                                                                                      \
        if (n <= WL) LAPSUM_WARP_FWD1(1, ROW_P, DUMP);                                                                         \
        else if (n <= 2 * WL) LAPSUM_WARP_FWD1(2, ROW_P, DUMP);                                                                \
        else if (n <= 4 * WL) LAPSUM_WARP_FWD1(4, ROW_P, DUMP);                                                                \
        else LAPSUM_WARP_FWD1(128 / WL, ROW_P, DUMP);                                                                          \
    } while (0)
        if (keys_dump) LAPSUM_WARP_FWD(false, true);
        else if (rp) LAPSUM_WARP_FWD(true, false);
        else LAPSUM_WARP_FWD(false, false);
#undef LAPSUM_WARP_FWD1
#undef LAPSUM_WARP_FWD
        return LAPSUM_OK;
    }
    BlockFwdArgs a{};
    a.r = r;
    a.p = p;
    a.b = b;
    a.th = th;
    a.ctl = ctl;
    a.n = (int)n;
    a.n_pad = next_pow2((int)n);
    a.k = S.k;
    a.t = S.t;
    a.sc = S.sc;
    a.c = S.c_mask;
    a.rp = rp;
    a.keys_dump = keys_dump;
    const size_t smem = 4 * ((size_t)a.n_pad + (size_t)a.n_pad / 32) + 8 * ((size_t)n + (size_t)n / 32 + 1);
    if (a.n_pad >= 4096 && rows * ROW_CLUSTER <= W->sm_count) {
        // few long rows: the blocks of a cluster share a row (eight for the longest rows while they all fit at once)
        const int cl = (a.n_pad >= 8192 && rows * ROW_CLUSTER_MAX <= W->sm_count) ? ROW_CLUSTER_MAX : ROW_CLUSTER;
        const size_t nl = (size_t)a.n_pad / (size_t)cl;
        const size_t csmem = 4 * (nl + nl / 32) + 8 * (nl + nl / 32 + 1);
        const int cthreads = (int)std::min<size_t>(1024, nl / 2);
        g_cluster_blocks = cl;
        LAUNCH(*W, LAPSUM_K_BLOCK_FWD, st, row_cluster_forward_kernel<T>, (unsigned)(rows * cl), cthreads, csmem, a);
    } else {
        LAUNCH(*W, LAPSUM_K_BLOCK_FWD, st, row_block_forward_kernel<T>, (unsigned)rows, block_threads(a.n_pad, rows, W->sm_count), smem, a);
    }
    return LAPSUM_OK;
}

// Launch the prologue that turns per-row budgets / temperatures into RowParams (in slot 0 of the workspace)
int enqueue_row_params(WsInfo &W, void *ws, const double *k_rows, const double *alpha_rows, double k, double alpha,
                              int need_budget, float *b, RowThreshold *th, cudaStream_t st, const RowParams **out)
{
    const Layout &L = W.lay;
    RowParams *rp = at<RowParams>(ws, L.off_rowparams);
    const unsigned grid = (unsigned)((L.rows + 255) / 256);
    LAUNCH(W, LAPSUM_K_MISC, st, row_params_kernel, grid, 256, 0, k_rows, alpha_rows, k, alpha, (long long)L.rows, (long long)L.n,
           (long long)(L.path == LAPSUM_PATH_BRACKET ? L.K : 0), L.prm.z, need_budget, rp, b, th, at<Control>(ws, L.off_control));
    *out = rp;
    return LAPSUM_OK;
}

// forward with the call's budget k and temperature alpha, or (k_rows / alpha_rows != nullptr) one of either per row;
// T is the workspace's element type (the caller has looked it up)
template <typename T>
int forward_impl(const T *r, int64_t rows, int64_t n, double k, const double *k_rows, double alpha,
                 const double *alpha_rows, T *p, float *b, void *ws, void *stream)
{
    if (!r || !p || !b || !ws) return LAPSUM_ERR_NULL;
    int rc = check_problem(rows, n, k, alpha);
    if (rc) return rc;
    WsHandle wsh;
    rc = lock_ws(ws, wsh);
    WsInfo *W = wsh.W;
    if (rc) return rc;
    const Layout &L = W->lay;
    if (L.rows != rows || L.n != n || L.prm.io_dtype != IoOf<T>::io) return LAPSUM_ERR_WORKSPACE;
    if (L.sharded) return LAPSUM_ERR_UNSUPPORTED;  // a shard's workspace serves the lapsum_shard_* calls only
    cudaStream_t st = (cudaStream_t)stream;
    const Scalars S = make_scalars(k, alpha, n);
    Control *ctl = at<Control>(ws, L.off_control);
    RowThreshold *th = at<RowThreshold>(ws, L.off_th);
    const RowParams *rp = nullptr;
    if (k_rows || alpha_rows) {
        rc = enqueue_row_params(*W, ws, k_rows, alpha_rows, k, alpha, 1, b, th, st, &rp);
        if (rc) return rc;
    }
    if (L.path == LAPSUM_PATH_BLOCK) {
        rc = launch_block_path_forward<T>(*W, r, rows, n, S, rp, p, b, th, ctl, nullptr, st);
        if (rc) return rc;
    } else if (L.path == LAPSUM_PATH_BRACKET && !L.prm.full_sorts) {
        // groups of up to `slots` rows, one launch per kernel and group, all on the caller's stream
        for (int64_t row0 = 0; row0 < rows; row0 += L.slots) {
            const int group = (int)std::min<int64_t>(L.slots, rows - row0);
            rc = enqueue_bracket_forward<T>(*W, ws, r + row0 * n, S, rp ? rp + row0 : nullptr, p + row0 * n, b + row0, th + row0, 0,
                                            0.f, 0.f, row0 + group == rows, st, group);
            if (rc) return rc;
        }
    } else {
        rc = rows_fork(*W, st);
        if (rc) return rc;
        for (int64_t row = 0; row < rows; ++row) {
            const T *rr = r + row * n;
            void *wsS = row_slot(*W, ws, row);
            cudaStream_t sr = row_stream(*W, st, row);
            Control *ctlS = at<Control>(wsS, L.off_control);
            const RowParams *rpr = rp ? rp + row : nullptr;
            if (L.path == LAPSUM_PATH_FULLSORT) {
                CU(cudaMemsetAsync(&ctlS->call, 0, sizeof(CallCtl), sr));
                W->call_clean[row % L.slots] = false;
                // a void row (unusable budget or temperature) skips the whole chain: its kernels are predicated on rp->valid
                rc = enqueue_fullsort_solve(*W, wsS, rr, IoOf<T>::kind, S, b + row, th + row, rpr ? &rpr->valid : nullptr, rpr, sr);
                if (rc) return rc;
                if (n >= CDF_LONG_N) LAUNCH(*W, LAPSUM_K_CDF_MAP, sr, (cdf_map_kernel<T, CDF_U_LONG>), map_grid(*W, n), 512, 0, rr, p + row * n, (unsigned long long)n, th + row, S.c_mask, ctlS, row + 1 == rows ? L.path : 0, rpr, 0, BatchShift{});
                else LAUNCH(*W, LAPSUM_K_CDF_MAP, sr, (cdf_map_kernel<T, CDF_U_SHORT>), map_grid(*W, n), 512, 0, rr, p + row * n, (unsigned long long)n, th + row, S.c_mask, ctlS, row + 1 == rows ? L.path : 0, rpr, 0, BatchShift{});
            } else {
                rc = enqueue_bracket_forward<T>(*W, wsS, rr, S, rpr, p + row * n, b + row, th + row, 0, 0.f, 0.f, row + 1 == rows, sr);
                if (rc) return rc;
            }
        }
        rc = rows_join(*W, st);
        if (rc) return rc;
    }
    return LAPSUM_OK;
}

template <typename T>
int backward_impl(const T *v, const T *r, const float *b, double alpha, const double *alpha_rows, T *grad_r,
                  float *grad_k, float *grad_alpha, void *ws, void *stream)
{
    if (!v || !r || !b || !grad_r || !ws) return LAPSUM_ERR_NULL;
    if (!alpha_ok(alpha)) return LAPSUM_ERR_ALPHA;
    WsHandle wsh;
    int rc = lock_ws(ws, wsh);
    WsInfo *W = wsh.W;
    if (rc) return rc;
    const Layout &L = W->lay;
    if (L.prm.io_dtype != IoOf<T>::io) return LAPSUM_ERR_WORKSPACE;
    if (L.sharded) return LAPSUM_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const Scalars S = make_scalars(1.0, alpha, 2);
    Control *ctl = at<Control>(ws, L.off_control);
    const RowParams *rp = nullptr;
    if (alpha_rows) {
        rc = enqueue_row_params(*W, ws, nullptr, alpha_rows, 1.0, alpha, 0, nullptr, nullptr, st, &rp);
        if (rc) return rc;
    }
    if (L.path == LAPSUM_PATH_BLOCK && L.n <= 128) {
        WarpBwdArgs a{v, r, b, at<RowThreshold>(ws, L.off_th), grad_r, ctl, (long long)L.rows, (int)L.n, S.c, S.half_inv_t,
                      grad_k, grad_alpha, 1.0 / S.t, S.gsign, rp};
        constexpr int WL = WARP_ROW_LANES;
        const unsigned grid = (unsigned)((L.rows + WP_WARPS * (32 / WL) - 1) / (WP_WARPS * (32 / WL)));
        if (L.n <= WL) LAUNCH(*W, LAPSUM_K_BLOCK_BWD, st, (row_warp_backward_kernel<1, WL, T>), grid, WP_WARPS * 32, 0, a);
        else if (L.n <= 2 * WL) LAUNCH(*W, LAPSUM_K_BLOCK_BWD, st, (row_warp_backward_kernel<2, WL, T>), grid, WP_WARPS * 32, 0, a);
        else if (L.n <= 4 * WL) LAUNCH(*W, LAPSUM_K_BLOCK_BWD, st, (row_warp_backward_kernel<4, WL, T>), grid, WP_WARPS * 32, 0, a);
        else LAUNCH(*W, LAPSUM_K_BLOCK_BWD, st, (row_warp_backward_kernel<128 / WL, WL, T>), grid, WP_WARPS * 32, 0, a);
    } else if (L.path == LAPSUM_PATH_BLOCK) {
        BlockBwdArgs a{v, r, b, at<RowThreshold>(ws, L.off_th), grad_r, ctl, (int)L.n, S.c, S.half_inv_t, grad_k, grad_alpha, 1.0 / S.t, S.gsign, rp};
        const int threads = (int)std::min<int64_t>(1024, std::max<int64_t>(32, (L.n + 3) / 4 / 32 * 32));
        LAUNCH(*W, LAPSUM_K_BLOCK_BWD, st, row_block_backward_kernel<T>, (unsigned)L.rows, threads, 0, a);
    } else {
        // long rows: groups of up to `slots` rows (each row has its own partial sums and ticket in its slot), two
        // launches per group
        for (int64_t row0 = 0; row0 < L.rows; row0 += L.slots) {
            const int group = (int)std::min<int64_t>(L.slots, L.rows - row0);
            VjpArgs a{};
            a.v = v + row0 * L.n;
            a.r = r + row0 * L.n;
            a.b = b + row0;
            a.th = at<RowThreshold>(ws, L.off_th) + row0;
            a.grad = grad_r + row0 * L.n;
            a.n = (unsigned long long)L.n;
            a.partials = at<double>(ws, L.off_partials);
            a.ctl = ctl;
            a.c = S.c;
            a.half_inv_t = S.half_inv_t;
            a.grad_k = grad_k ? grad_k + row0 : nullptr;
            a.grad_alpha = grad_alpha ? grad_alpha + row0 : nullptr;
            a.inv_t = 1.0 / S.t;
            a.gsign = S.gsign;
            a.rp = rp ? rp + row0 : nullptr;
            a.bs = BatchShift{(unsigned long long)L.slot_bytes, (unsigned long long)L.n, group > 1 ? 1 : 0};
            const unsigned G = (unsigned)group;
            const int g = std::min(map_grid(*W, L.n, LAPSUM_REDUCE_BLOCKS_PER_SM), L.grid_stream * 2);
            if (vjp_wants_scalars(a)) LAUNCH(*W, LAPSUM_K_VJP_REDUCE, st, (vjp_reduce_kernel<T, true>), dim3((unsigned)g, G), EW_THREADS, 0, a);
            else LAUNCH(*W, LAPSUM_K_VJP_REDUCE, st, (vjp_reduce_kernel<T, false>), dim3((unsigned)g, G), EW_THREADS, 0, a);
            LAUNCH(*W, LAPSUM_K_VJP_MAP, st, vjp_map_kernel<T>, dim3((unsigned)map_grid(*W, L.n), G), 512, 0, a);
        }
    }
    return LAPSUM_OK;
}

// the element type a workspace was built for (LAPSUM_ERR_WORKSPACE if it is not registered)
int workspace_io(void *ws, int *io)
{
    if (!ws) return LAPSUM_ERR_NULL;
    WsHandle wsh;
    int rc = lock_ws(ws, wsh);
    WsInfo *W = wsh.W;
    if (rc) return rc;
    *io = W->lay.prm.io_dtype;
    return LAPSUM_OK;
}
}  // namespace
}  // extern "C++"

int lapsum_forward(const float *r, int64_t rows, int64_t n, double k, double alpha, float *p, float *b, void *ws,
                   void *stream)
{
    return forward_impl(r, rows, n, k, nullptr, alpha, nullptr, p, b, ws, stream);
}

int lapsum_forward_row_budgets(const float *r, int64_t rows, int64_t n, const double *k_rows, double alpha, float *p,
                               float *b, void *ws, void *stream)
{
    if (!k_rows) return LAPSUM_ERR_NULL;
    // the budgets live on the device: the host checks the rest with a budget that is valid for every n
    return forward_impl(r, rows, n, 0.5 * (double)std::max<int64_t>(n, 1), k_rows, alpha, nullptr, p, b, ws, stream);
}

int lapsum_forward_rows(const float *r, int64_t rows, int64_t n, const double *k_rows, const double *alpha_rows, double k,
                        double alpha, float *p, float *b, void *ws, void *stream)
{
    // a vector that is given lives on the device and is checked there, row by row; the scalar it replaces only has to
    // pass the host's checks, so a stand-in that is valid for every n is put in its place
    if (k_rows) k = 0.5 * (double)std::max<int64_t>(n, 1);
    if (alpha_rows) alpha = -1.0;
    return forward_impl(r, rows, n, k, k_rows, alpha, alpha_rows, p, b, ws, stream);
}

int lapsum_forward_io(const void *r, int64_t rows, int64_t n, const double *k_rows, const double *alpha_rows, double k,
                      double alpha, void *p, float *b, void *ws, void *stream)
{
    int io = 0;
    int rc = workspace_io(ws, &io);
    if (rc) return rc;
    if (k_rows) k = 0.5 * (double)std::max<int64_t>(n, 1);
    if (alpha_rows) alpha = -1.0;
    if (io == LAPSUM_IO_F16)
        return forward_impl<__half>(static_cast<const __half *>(r), rows, n, k, k_rows, alpha, alpha_rows, static_cast<__half *>(p), b, ws, stream);
    if (io == LAPSUM_IO_BF16)
        return forward_impl<__nv_bfloat16>(static_cast<const __nv_bfloat16 *>(r), rows, n, k, k_rows, alpha, alpha_rows,
                                           static_cast<__nv_bfloat16 *>(p), b, ws, stream);
    return forward_impl<float>(static_cast<const float *>(r), rows, n, k, k_rows, alpha, alpha_rows, static_cast<float *>(p), b, ws, stream);
}

int lapsum_backward_io(const void *v, const void *r, const float *b, const double *alpha_rows, double alpha, void *grad_r,
                       float *grad_k, float *grad_alpha, void *ws, void *stream)
{
    int io = 0;
    int rc = workspace_io(ws, &io);
    if (rc) return rc;
    if (alpha_rows) alpha = -1.0;
    if (io == LAPSUM_IO_F16)
        return backward_impl<__half>(static_cast<const __half *>(v), static_cast<const __half *>(r), b, alpha, alpha_rows,
                                     static_cast<__half *>(grad_r), grad_k, grad_alpha, ws, stream);
    if (io == LAPSUM_IO_BF16)
        return backward_impl<__nv_bfloat16>(static_cast<const __nv_bfloat16 *>(v), static_cast<const __nv_bfloat16 *>(r), b, alpha,
                                            alpha_rows, static_cast<__nv_bfloat16 *>(grad_r), grad_k, grad_alpha, ws, stream);
    return backward_impl<float>(static_cast<const float *>(v), static_cast<const float *>(r), b, alpha, alpha_rows,
                                static_cast<float *>(grad_r), grad_k, grad_alpha, ws, stream);
}

// ---- one row sharded over several GPUs (every call works on THIS rank's shard; the caller's collectives merge) ----
int lapsum_shard_workspace_bytes(int64_t n_total, const lapsum_params *prm, size_t *bytes)
{
    if (!bytes) return LAPSUM_ERR_NULL;
    Layout L;
    int rc = make_layout(1, n_total, prm, 148, &L, true);
    if (rc) return rc;
    *bytes = L.total;
    return LAPSUM_OK;
}

int lapsum_shard_workspace_init(void *ws, size_t bytes, int64_t n_total, const lapsum_params *prm, uint64_t seed, void *stream)
{
    return workspace_init_impl(ws, bytes, 1, n_total, prm, seed, stream, true);
}

int lapsum_shard_describe(void *ws, lapsum_shard_layout *out)
{
    if (!ws || !out) return LAPSUM_ERR_NULL;
    WsHandle wsh;
    int rc = lock_ws(ws, wsh);
    if (rc) return rc;
    const Layout &L = wsh.W->lay;
    if (!L.sharded) return LAPSUM_ERR_UNSUPPORTED;
    *out = lapsum_shard_layout{};
    out->K = L.K;
    out->band_capacity = L.cap;
    out->off_sample_keys = L.off_sample[0];
    out->off_band_count = L.off_control + offsetof(Control, call) + offsetof(CallCtl, band_count);
    out->off_n_R = L.off_control + offsetof(Control, call) + offsetof(CallCtl, n_R);
    out->off_tails = L.off_control + offsetof(Control, call) + offsetof(CallCtl, S_L);
    out->off_bucket_counts = L.off_control + offsetof(Control, call) + offsetof(CallCtl, band_cnt);
    out->off_bucket_sums = L.off_control + offsetof(Control, call) + offsetof(CallCtl, band_up);
    out->off_band_keys = L.off_band_keys[0];
    out->off_vjp_sums = L.off_control + offsetof(Control, persist) + offsetof(PersistCtl, S_f);
    static_assert(offsetof(CallCtl, S_R) == offsetof(CallCtl, S_L) + 8, "the two tails are exchanged as one pair of doubles");
    static_assert(offsetof(CallCtl, band_down) == offsetof(CallCtl, band_up) + 8 * BAND_BUCKETS, "the two bucket sums are exchanged as one array");
    static_assert(offsetof(PersistCtl, S_vfd) == offsetof(PersistCtl, S_f) + 24, "the four VJP sums are exchanged as one array");
    return LAPSUM_OK;
}

static int shard_ws(void *ws, WsHandle &wsh, int64_t n_total)
{
    int rc = lock_ws(ws, wsh);
    if (rc) return rc;
    const Layout &L = wsh.W->lay;
    if (!L.sharded) return LAPSUM_ERR_UNSUPPORTED;
    if (L.n != n_total) return LAPSUM_ERR_WORKSPACE;
    return LAPSUM_OK;
}

int lapsum_shard_sample(const float *r_shard, int64_t shard_begin, int64_t shard_len, int64_t n_total, double alpha, void *ws,
                        void *stream)
{
    if (!r_shard || !ws) return LAPSUM_ERR_NULL;
    if (shard_begin < 0 || shard_len < 1 || shard_begin + shard_len > n_total) return LAPSUM_ERR_SHAPE;
    if (!alpha_ok(alpha)) return LAPSUM_ERR_ALPHA;
    WsHandle wsh;
    int rc = shard_ws(ws, wsh, n_total);
    if (rc) return rc;
    WsInfo *W = wsh.W;
    const Layout &L = W->lay;
    cudaStream_t st = (cudaStream_t)stream;
    Control *ctl = at<Control>(ws, L.off_control);
    if (!W->call_clean[0]) CU(cudaMemsetAsync(&ctl->call, 0, sizeof(CallCtl), st));
    W->call_clean[0] = false;
    const int g = (int)((L.K + 255) / 256);
    LAUNCH(*W, LAPSUM_K_SAMPLE, st, sample_shard_kernel<float>, g, 256, 0, r_shard, (long long)shard_begin, (long long)shard_len,
           (long long)L.K, (long long)L.stride, (uint32_t)(W->seed & 0xffffffffu), at<float>(ws, L.off_noise), (float)std::fabs(alpha),
           at<uint32_t>(ws, L.off_sample[0]));
    return LAPSUM_OK;
}

int lapsum_shard_stream(const float *r_shard, int64_t shard_len, int64_t n_total, double k, double alpha, void *ws, void *stream)
{
    if (!r_shard || !ws) return LAPSUM_ERR_NULL;
    if (shard_len < 1 || shard_len > n_total) return LAPSUM_ERR_SHAPE;
    int rc = check_problem(1, n_total, k, alpha);
    if (rc) return rc;
    WsHandle wsh;
    rc = shard_ws(ws, wsh, n_total);
    if (rc) return rc;
    WsInfo *W = wsh.W;
    const Layout &L = W->lay;
    cudaStream_t st = (cudaStream_t)stream;
    Control *ctl = at<Control>(ws, L.off_control);
    const Scalars S = make_scalars(k, alpha, n_total);
    int64_t j = 0, l = 0;
    bracket_ranks(L.n, L.K, S.k, L.prm.z, &j, &l);
    uint32_t *sa = at<uint32_t>(ws, L.off_sample[0]);
    // the whole sample is in the key buffer now (the caller added the ranks' buffers): histogram, then the two order statistics
    LAUNCH(*W, LAPSUM_K_SAMPLE, st, sample_keys_hist_kernel, (int)((L.K + 1023) / 1024), 1024, 0, sa, (long long)L.K, ctl);
    PickArgs pk{};
    pk.keys = sa;
    pk.cand = at<uint32_t>(ws, L.off_sample[1]);
    pk.K = L.K;
    pk.j = j;
    pk.l = l;
    pk.cand_cap = L.K / 2;
    pk.ctl = ctl;
    const int gp = (int)std::max<int64_t>(1, std::min<int64_t>(64, L.K / 4 / (SEL_THREADS * 2) + 1));
    LAUNCH(*W, LAPSUM_K_SAMPLE, st, sample_pick_kernel<false>, gp, SEL_THREADS, 0, pk);
    StreamArgs a{};
    a.r = r_shard;
    a.n = (unsigned long long)shard_len;
    a.sel = &ctl->call.sel_keys[0];
    a.fscale = fixed_scale((unsigned long long)L.cap);
    a.K = L.K;
    a.j = j;
    a.l = l;
    a.c = S.c;
    a.sc = S.sc;
    a.band_keys = at<uint32_t>(ws, L.off_band_keys[0]);
    a.cap = (unsigned long long)L.cap;
    a.partials = at<double>(ws, L.off_partials);
    a.ctl = ctl;
    LAUNCH(*W, LAPSUM_K_STREAM_BAND, st, stream_band_kernel<float>, stream_blocks(*W), STREAM_THREADS, 0, a);
    return LAPSUM_OK;
}

int lapsum_shard_solve(int64_t n_total, double k, double alpha, float *b, void *ws, void *stream)
{
    if (!b || !ws) return LAPSUM_ERR_NULL;
    int rc = check_problem(1, n_total, k, alpha);
    if (rc) return rc;
    WsHandle wsh;
    rc = shard_ws(ws, wsh, n_total);
    if (rc) return rc;
    WsInfo *W = wsh.W;
    const Layout &L = W->lay;
    cudaStream_t st = (cudaStream_t)stream;
    Control *ctl = at<Control>(ws, L.off_control);
    RowThreshold *th = at<RowThreshold>(ws, L.off_th);
    const Scalars S = make_scalars(k, alpha, n_total);
    // a failed certificate leaves the threshold as it is set here: NaN (all bits one)
    CU(cudaMemsetAsync(b, 0xff, sizeof(float), st));
    CU(cudaMemsetAsync(th, 0xff, sizeof(RowThreshold), st));
    BandArgs ba{};
    ba.band = at<uint32_t>(ws, L.off_band_keys[0]);
    ba.glist = at<uint32_t>(ws, L.off_band_keys[1]);
    ba.ctl = ctl;
    ba.b_out = b;
    ba.th_out = th;
    ba.cap = (unsigned long long)L.cap;
    ba.fscale = fixed_scale((unsigned long long)L.cap);
    ba.k = S.k;
    ba.t = S.t;
    ba.sc = S.sc;
    ba.c = S.c;
    ba.fb.enabled = 0;  // no fallback from the device: the full sort of a sharded row is the caller's to arrange
    ba.solve_blocks = 1;
    ba.attempt = 0;
    ba.max_widen = 0;
    ba.io = LAPSUM_IO_F32;
    LAUNCH(*W, LAPSUM_K_SOLVE, st, band_solve_kernel, 1, 1024, sizeof(BandShared), ba);
    return LAPSUM_OK;
}

int lapsum_shard_mask(const float *r_shard, int64_t shard_len, int64_t n_total, double alpha, float *p_shard, void *ws,
                      void *stream)
{
    if (!r_shard || !p_shard || !ws) return LAPSUM_ERR_NULL;
    if (shard_len < 1 || shard_len > n_total) return LAPSUM_ERR_SHAPE;
    if (!alpha_ok(alpha)) return LAPSUM_ERR_ALPHA;
    WsHandle wsh;
    int rc = shard_ws(ws, wsh, n_total);
    if (rc) return rc;
    WsInfo *W = wsh.W;
    const Layout &L = W->lay;
    cudaStream_t st = (cudaStream_t)stream;
    const Scalars S = make_scalars(1.0, alpha, 2);
    LAUNCH(*W, LAPSUM_K_CDF_MAP, st, (cdf_map_kernel<float, CDF_U_LONG>), map_grid(*W, shard_len), 512, 0, r_shard, p_shard,
           (unsigned long long)shard_len, at<RowThreshold>(ws, L.off_th), S.c_mask, at<Control>(ws, L.off_control), L.path,
           (const RowParams *)nullptr, 1, BatchShift{});
    W->call_clean[0] = true;
    return LAPSUM_OK;
}

static int shard_vjp_args(WsInfo *W, void *ws, const float *v_shard, const float *r_shard, int64_t shard_len, const float *b,
                          double alpha, float *grad_shard, VjpArgs *a)
{
    const Layout &L = W->lay;
    const Scalars S = make_scalars(1.0, alpha, 2);
    *a = VjpArgs{};
    a->v = v_shard;
    a->r = r_shard;
    a->b = b;
    a->th = at<RowThreshold>(ws, L.off_th);
    a->grad = grad_shard;
    a->n = (unsigned long long)shard_len;
    a->partials = at<double>(ws, L.off_partials);
    a->ctl = at<Control>(ws, L.off_control);
    a->c = S.c;
    a->half_inv_t = S.half_inv_t;
    a->inv_t = 1.0 / S.t;
    a->gsign = S.gsign;
    a->all_sums = 1;
    return LAPSUM_OK;
}

int lapsum_shard_vjp_partial(const float *v_shard, const float *r_shard, int64_t shard_len, int64_t n_total, const float *b,
                             double alpha, void *ws, void *stream)
{
    if (!v_shard || !r_shard || !b || !ws) return LAPSUM_ERR_NULL;
    if (shard_len < 1 || shard_len > n_total) return LAPSUM_ERR_SHAPE;
    if (!alpha_ok(alpha)) return LAPSUM_ERR_ALPHA;
    WsHandle wsh;
    int rc = shard_ws(ws, wsh, n_total);
    if (rc) return rc;
    WsInfo *W = wsh.W;
    VjpArgs a;
    shard_vjp_args(W, ws, v_shard, r_shard, shard_len, b, alpha, nullptr, &a);
    const int g = std::min(map_grid(*W, shard_len, LAPSUM_REDUCE_BLOCKS_PER_SM), W->lay.grid_stream * 2);
    LAUNCH(*W, LAPSUM_K_VJP_REDUCE, (cudaStream_t)stream, (vjp_reduce_kernel<float, true>), g, EW_THREADS, 0, a);
    return LAPSUM_OK;
}

int lapsum_shard_vjp_apply(const float *v_shard, const float *r_shard, int64_t shard_len, int64_t n_total, const float *b,
                           double alpha, float *grad_shard, float *grad_k, float *grad_alpha, void *ws, void *stream)
{
    if (!v_shard || !r_shard || !b || !grad_shard || !ws) return LAPSUM_ERR_NULL;
    if (shard_len < 1 || shard_len > n_total) return LAPSUM_ERR_SHAPE;
    if (!alpha_ok(alpha)) return LAPSUM_ERR_ALPHA;
    WsHandle wsh;
    int rc = shard_ws(ws, wsh, n_total);
    if (rc) return rc;
    WsInfo *W = wsh.W;
    cudaStream_t st = (cudaStream_t)stream;
    VjpArgs a;
    shard_vjp_args(W, ws, v_shard, r_shard, shard_len, b, alpha, grad_shard, &a);
    if (grad_k || grad_alpha) LAUNCH(*W, LAPSUM_K_MISC, st, vjp_scalars_kernel, 1, 32, 0, a.ctl, a.inv_t, grad_k, grad_alpha);
    LAUNCH(*W, LAPSUM_K_VJP_MAP, st, vjp_map_kernel<float>, map_grid(*W, shard_len), 512, 0, a);
    return LAPSUM_OK;
}

int lapsum_forward_with_bracket(const float *r, int64_t n, double k, double alpha, float a_L, float a_R, float *p,
                                float *b, void *ws, void *stream)
{
    if (!r || !p || !b || !ws) return LAPSUM_ERR_NULL;
    int rc = check_problem(1, n, k, alpha);
    if (rc) return rc;
    WsHandle wsh;
    rc = lock_ws(ws, wsh);
    WsInfo *W = wsh.W;
    if (rc) return rc;
    const Layout &L = W->lay;
    if (L.rows != 1 || L.n != n || L.prm.io_dtype != LAPSUM_IO_F32) return LAPSUM_ERR_WORKSPACE;
    if (L.path != LAPSUM_PATH_BRACKET || L.sharded) return LAPSUM_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const Scalars S = make_scalars(k, alpha, n);
    rc = enqueue_bracket_forward<float>(*W, ws, r, S, nullptr, p, b, at<RowThreshold>(ws, L.off_th), 1, a_L, a_R, true, st);
    if (rc) return rc;
    return LAPSUM_OK;
}

int lapsum_backward(const float *v, const float *r, const float *b, double k, double alpha, float *grad_r, void *ws,
                    void *stream)
{
    return lapsum_backward_scalars(v, r, b, k, alpha, grad_r, nullptr, nullptr, ws, stream);
}

int lapsum_backward_scalars(const float *v, const float *r, const float *b, double k, double alpha, float *grad_r,
                            float *grad_k, float *grad_alpha, void *ws, void *stream)
{
    (void)k;
    return backward_impl(v, r, b, alpha, nullptr, grad_r, grad_k, grad_alpha, ws, stream);
}

int lapsum_backward_rows(const float *v, const float *r, const float *b, const double *alpha_rows, double alpha,
                         float *grad_r, float *grad_k, float *grad_alpha, void *ws, void *stream)
{
    if (alpha_rows) alpha = -1.0;  // checked on the device, row by row
    return backward_impl(v, r, b, alpha, alpha_rows, grad_r, grad_k, grad_alpha, ws, stream);
}

int lapsum_backward_static(const float *v, const float *r, const float *b, int64_t rows, int64_t n, double alpha,
                           float *grad_r, void *stream)
{
    if (!v || !r || !b || !grad_r) return LAPSUM_ERR_NULL;
    if (rows < 1 || rows > LAPSUM_STATIC_MAX_ROWS || n < 1 || n > LAPSUM_MAX_N) return LAPSUM_ERR_SHAPE;
    if (!alpha_ok(alpha)) return LAPSUM_ERR_ALPHA;
    cudaStream_t st = (cudaStream_t)stream;
    int device = 0;
    CU(cudaGetDevice(&device));
    if (device < 0 || device >= 16) return LAPSUM_ERR_UNSUPPORTED;
    void *scratch = nullptr;
    {
        // In host code the array's name is only a handle; the address a kernel can use has to be asked for,
        // once per device and with that device current.
        std::lock_guard<std::mutex> lk(g_static_mu);
        if (!g_static_ptr[device]) {
            void *ptr = nullptr;
            CU(cudaGetSymbolAddress(&ptr, g_static_scratch));
            if (!ptr) return LAPSUM_ERR_CUDA;
            g_static_ptr[device] = ptr;
        }
        scratch = g_static_ptr[device];
    }
    Control *ctl = reinterpret_cast<Control *>(scratch);
    double *partials = reinterpret_cast<double *>(static_cast<unsigned char *>(scratch) + STATIC_PARTIALS_OFF);
    // the array keeps whatever the last call left: the ticket of the last-block reduction must start at zero
    CU(cudaMemsetAsync(&ctl->call.vjp_ticket, 0, sizeof(ctl->call.vjp_ticket), st));
    const Scalars S = make_scalars(1.0, alpha, 2);
    int sms = 0;
    CU(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device));
    const int max_blocks = std::min(STATIC_MAX_BLOCKS, std::max(1, sms) * 8);
    const int grid = (int)std::max<int64_t>(1, std::min<int64_t>((n / 4 + 511) / 512, (int64_t)max_blocks));
    WsInfo none;  // no workspace: profiling hooks stay off
    for (int64_t row = 0; row < rows; ++row) {
        VjpArgs a{};
        a.v = v + row * n;
        a.r = r + row * n;
        a.b = b + row;
        a.grad = grad_r + row * n;
        a.n = (unsigned long long)n;
        a.partials = partials;
        a.ctl = ctl;
        a.c = S.c;
        a.half_inv_t = S.half_inv_t;
        a.gsign = S.gsign;
        LAUNCH(none, LAPSUM_K_VJP_REDUCE, st, (vjp_reduce_kernel<float, false>), grid, EW_THREADS, 0, a);
        LAUNCH(none, LAPSUM_K_VJP_MAP, st, vjp_map_kernel<float>, grid, 512, 0, a);
    }
    return LAPSUM_OK;
}

int lapsum_forward_backward_host(const float *r_host, const float *v_host, int64_t rows, int64_t n, double k, double alpha,
                                 float *p_host, float *grad_host, float *b_host, float *staging, void *ws, void *stream)
{
    if (!r_host || !v_host || !p_host || !grad_host || !b_host || !staging || !ws) return LAPSUM_ERR_NULL;
    int rc = check_problem(rows, n, k, alpha);
    if (rc) return rc;
    HostPipe hp;
    {
        WsHandle wsh;
        rc = lock_ws(ws, wsh);
        if (rc) return rc;
        WsInfo *W = wsh.W;
        if (W->lay.rows != rows || W->lay.n != n) return LAPSUM_ERR_WORKSPACE;
        if (!W->pipe.ready) {
            CU(cudaStreamCreateWithFlags(&W->pipe.h2d, cudaStreamNonBlocking));
            CU(cudaStreamCreateWithFlags(&W->pipe.d2h, cudaStreamNonBlocking));
            for (cudaEvent_t &e : W->pipe.ev) CU(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
            W->pipe.ready = true;
        }
        hp = W->pipe;
    }
    cudaStream_t st = (cudaStream_t)stream;
    const size_t N = (size_t)rows * (size_t)n, bytes = N * sizeof(float);
    float *r_d = staging, *v_d = r_d + N, *p_d = v_d + N, *g_d = p_d + N, *b_d = g_d + N;
    cudaEvent_t ev_start = hp.ev[0], ev_r = hp.ev[1], ev_v = hp.ev[2], ev_f = hp.ev[3], ev_p = hp.ev[4];
    // the side streams start behind whatever the caller's stream holds already
    CU(cudaEventRecord(ev_start, st));
    CU(cudaStreamWaitEvent(hp.h2d, ev_start, 0));
    CU(cudaStreamWaitEvent(hp.d2h, ev_start, 0));
    // host -> device: r first (the forward needs all of it), v behind it on the same link direction
    CU(cudaMemcpyAsync(r_d, r_host, bytes, cudaMemcpyHostToDevice, st));
    CU(cudaEventRecord(ev_r, st));
    CU(cudaStreamWaitEvent(hp.h2d, ev_r, 0));
    CU(cudaMemcpyAsync(v_d, v_host, bytes, cudaMemcpyHostToDevice, hp.h2d));
    CU(cudaEventRecord(ev_v, hp.h2d));
    rc = lapsum_forward(r_d, rows, n, k, alpha, p_d, b_d, ws, stream);
    if (rc) return rc;
    // device -> host of the mask runs in the other link direction while v is still arriving
    CU(cudaEventRecord(ev_f, st));
    CU(cudaStreamWaitEvent(hp.d2h, ev_f, 0));
    CU(cudaMemcpyAsync(p_host, p_d, bytes, cudaMemcpyDeviceToHost, hp.d2h));
    CU(cudaMemcpyAsync(b_host, b_d, (size_t)rows * sizeof(float), cudaMemcpyDeviceToHost, hp.d2h));
    CU(cudaEventRecord(ev_p, hp.d2h));
    CU(cudaStreamWaitEvent(st, ev_v, 0));
    rc = lapsum_backward(v_d, r_d, b_d, k, alpha, g_d, ws, stream);
    if (rc) return rc;
    CU(cudaMemcpyAsync(grad_host, g_d, bytes, cudaMemcpyDeviceToHost, st));
    CU(cudaStreamWaitEvent(st, ev_p, 0));  // the caller's stream is through only when every copy is
    return LAPSUM_OK;
}

int lapsum_status(void *ws, void *stream, lapsum_stats *out)
{
    if (!ws || !out) return LAPSUM_ERR_NULL;
    struct { Layout lay; } W;
    {
        WsHandle wsh;
        int rc = lock_ws(ws, wsh);
        if (rc) return rc;
        W.lay = wsh.W->lay;
    }
    cudaStream_t st = (cudaStream_t)stream;
    CU(cudaStreamSynchronize(st));
    // the last row's slot holds the last bracket and the path note; counters and status bits add up over the slots
    PersistCtl ps;
    const int last_slot = (int)((W.lay.rows - 1) % W.lay.slots);
    CU(cudaMemcpy(&ps, &at<Control>(ws, (size_t)last_slot * W.lay.slot_bytes + W.lay.off_control)->persist, sizeof(ps), cudaMemcpyDeviceToHost));
    for (int slot = 0; slot < W.lay.slots; ++slot) {
        if (slot == last_slot) continue;
        PersistCtl q;
        CU(cudaMemcpy(&q, &at<Control>(ws, (size_t)slot * W.lay.slot_bytes + W.lay.off_control)->persist, sizeof(q), cudaMemcpyDeviceToHost));
        ps.status_bits |= q.status_bits;
        ps.fallbacks += q.fallbacks;
        ps.widenings += q.widenings;
        ps.lookback_timeouts += q.lookback_timeouts;
    }
    std::memset(out, 0, sizeof(*out));
    out->status_bits = ps.status_bits;
    out->path = ps.last_path;
    out->forwards = (int64_t)ps.forwards;
    out->fallbacks = (int64_t)ps.fallbacks;
    out->widenings = (int64_t)ps.widenings;
    out->lookback_timeouts = (int64_t)ps.lookback_timeouts;
    out->K = ps.K;
    out->j = ps.j;
    out->l = ps.l;
    out->a_L = ps.a_L;
    out->a_R = ps.a_R;
    out->n_L = (int64_t)ps.n_L;
    out->n_M = (int64_t)ps.n_M;
    out->n_R = (int64_t)ps.n_R;
    out->S_L = ps.S_L;
    out->S_R = ps.S_R;
    out->S_f = ps.S_f;
    out->S_vf = ps.S_vf;
    return LAPSUM_OK;
}

int lapsum_debug_sort_pairs(const float *keys, int64_t rows, int64_t n, float *keys_out, uint32_t *idx_out, void *ws,
                            void *stream)
{
    if (!keys || !keys_out || !ws) return LAPSUM_ERR_NULL;
    if (rows < 1 || n < 1 || n > LAPSUM_MAX_N) return LAPSUM_ERR_SHAPE;
    WsHandle wsh;
    int rc = lock_ws(ws, wsh);
    WsInfo *W = wsh.W;
    if (rc) return rc;
    const Layout &L = W->lay;
    if (L.rows != rows || L.n != n || L.prm.io_dtype != LAPSUM_IO_F32) return LAPSUM_ERR_WORKSPACE;
    if (L.sharded) return LAPSUM_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    if (L.path == LAPSUM_PATH_BLOCK) {
        if (!idx_out) {
            // the forward's own kernel for this shape (warp / block / cluster), stopped after its sort
            const Scalars S = make_scalars(0.5 * (double)n, -1.0, n);
            return launch_block_path_forward<float>(*W, keys, rows, n, S, nullptr, nullptr, nullptr, nullptr,
                                                    at<Control>(ws, L.off_control), keys_out, st);
        }
        const int n_pad = next_pow2((int)n);
        LAUNCH(*W, LAPSUM_K_MISC, st, row_block_sort_pairs_kernel, (unsigned)rows, block_threads(n_pad), 8 * (size_t)n_pad, keys, (int)n, n_pad, keys_out, idx_out);
        return LAPSUM_OK;
    }
    const bool payload = L.prm.sort_payload != 0;
    if (idx_out && !payload) return LAPSUM_ERR_UNSUPPORTED;
    Control *ctl = at<Control>(ws, L.off_control);
    for (int64_t row = 0; row < rows; ++row) {
        // the sort job of the forward's full-sort chain (keys only unless the workspace carries the payload)
        CU(cudaMemsetAsync(&ctl->call, 0, sizeof(CallCtl), st));
        W->call_clean[0] = false;
        SortJob J{};
        J.in = keys + row * n;
        J.in_kind = RS_IN_F32;
        J.keys[0] = at<uint32_t>(ws, L.off_full_keys[0]);
        J.keys[1] = at<uint32_t>(ws, L.off_full_keys[1]);
        J.vals[0] = payload ? at<uint32_t>(ws, L.off_full_idx[0]) : nullptr;
        J.vals[1] = payload ? at<uint32_t>(ws, L.off_full_idx[1]) : nullptr;
        J.final_vals = idx_out ? idx_out + row * n : nullptr;
        J.cnt = SortCount{nullptr, (unsigned long long)n, (unsigned long long)n};
        J.max_n = n;
        J.slot = 2;
        uint32_t *sorted = nullptr;
        rc = run_sort(*W, ws, J, st, &sorted, nullptr);
        if (rc) return rc;
        LAUNCH(*W, LAPSUM_K_MISC, st, keys_to_float_kernel, map_grid(*W, n), 512, 0, sorted, keys_out + row * n, (unsigned long long)n, nullptr, 0);
    }
    return LAPSUM_OK;
}

int lapsum_debug_lookback_timeout(const float *keys, int64_t n, int spin_limit, void *ws, void *stream)
{
    if (!keys || !ws) return LAPSUM_ERR_NULL;
    if (n < 1 || n > LAPSUM_MAX_N) return LAPSUM_ERR_SHAPE;
    if (spin_limit < 1 || spin_limit > RS_SPIN_LIMIT) return LAPSUM_ERR_PARAM;
    WsHandle wsh;
    int rc = lock_ws(ws, wsh);
    WsInfo *W = wsh.W;
    if (rc) return rc;
    const Layout &L = W->lay;
    if (L.rows != 1 || L.n != n) return LAPSUM_ERR_WORKSPACE;
    if (L.path == LAPSUM_PATH_BLOCK || n <= RS_TILE || L.sharded) return LAPSUM_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    Control *ctl = at<Control>(ws, L.off_control);
    CU(cudaMemsetAsync(&ctl->call, 0, sizeof(CallCtl), st));
    W->call_clean[0] = false;
    // the ticket counter of the first pass starts at 1: no block ever takes tile 0, so its look-back words stay
    // unpublished and every tile that has to read them waits until its bounded wait runs out
    CU(cudaMemsetAsync(&ctl->call.sort[2].ticket[0], 1, 1, st));
    SortJob J{};
    J.in = keys;
    J.in_kind = RS_IN_F32;
    J.keys[0] = at<uint32_t>(ws, L.off_full_keys[0]);
    J.keys[1] = at<uint32_t>(ws, L.off_full_keys[1]);
    J.cnt = SortCount{nullptr, (unsigned long long)n, (unsigned long long)n};
    J.max_n = n;
    J.slot = 2;
    J.spin_limit = spin_limit;
    J.passes = 1;
    uint32_t *sorted = nullptr;
    return run_sort(*W, ws, J, st, &sorted, nullptr);
}

int lapsum_debug_bracket(const float *r, int64_t n, double k, double alpha, void *ws, void *stream, int use_override,
                         float a_L, float a_R, float *y_out, float *band_out)
{
    if (!r || !ws) return LAPSUM_ERR_NULL;
    int rc = check_problem(1, n, k, alpha);
    if (rc) return rc;
    WsHandle wsh;
    rc = lock_ws(ws, wsh);
    WsInfo *W = wsh.W;
    if (rc) return rc;
    const Layout &L = W->lay;
    if (L.rows != 1 || L.n != n || L.prm.io_dtype != LAPSUM_IO_F32) return LAPSUM_ERR_WORKSPACE;
    if (L.path != LAPSUM_PATH_BRACKET || L.sharded) return LAPSUM_ERR_UNSUPPORTED;
    cudaStream_t st = (cudaStream_t)stream;
    const Scalars S = make_scalars(k, alpha, n);
    Control *ctl = at<Control>(ws, L.off_control);
    CU(cudaMemsetAsync(&ctl->call, 0, sizeof(CallCtl), st));
    W->call_clean[0] = false;
    rc = enqueue_bracket_stream<float>(*W, ws, r, S, nullptr, use_override, a_L, a_R, y_out, st);
    if (rc) return rc;
    if (band_out)
        LAUNCH(*W, LAPSUM_K_MISC, st, keys_to_float_kernel, map_grid(*W, L.cap), 512, 0, at<uint32_t>(ws, L.off_band_keys[0]), band_out, 0, &ctl->call.band_count, (unsigned long long)L.cap);
    return LAPSUM_OK;
}

int lapsum_profile_enable(void *ws, uint32_t kernel_mask, int max_records)
{
    if (!ws) return LAPSUM_ERR_NULL;
    if (max_records < 1 || max_records > (1 << 20)) return LAPSUM_ERR_PARAM;
    WsHandle wsh;
    int rc = lock_ws(ws, wsh);
    WsInfo *W = wsh.W;
    if (rc) return rc;
    prof_destroy(W->prof);
    Profile &P = W->prof;
    P.ev0.resize((size_t)max_records);
    P.ev1.resize((size_t)max_records);
    P.kid.assign((size_t)max_records, -1);
    for (int i = 0; i < max_records; ++i) {
        CU(cudaEventCreate(&P.ev0[(size_t)i]));
        CU(cudaEventCreate(&P.ev1[(size_t)i]));
    }
    P.mask = kernel_mask;
    P.used = 0;
    P.on = true;
    return LAPSUM_OK;
}

int lapsum_profile_read(void *ws, void *stream, int kernel_id, int64_t *launches, double *total_ms)
{
    if (!ws || !launches || !total_ms) return LAPSUM_ERR_NULL;
    WsHandle wsh;
    int rc = lock_ws(ws, wsh);
    WsInfo *W = wsh.W;
    if (rc) return rc;
    CU(cudaStreamSynchronize((cudaStream_t)stream));
    int64_t cnt = 0;
    double ms = 0.0;
    const Profile &P = W->prof;
    for (int i = 0; i < P.used; ++i) {
        if (P.kid[(size_t)i] != kernel_id) continue;
        float e = 0.f;
        CU(cudaEventElapsedTime(&e, P.ev0[(size_t)i], P.ev1[(size_t)i]));
        ms += (double)e;
        ++cnt;
    }
    *launches = cnt;
    *total_ms = ms;
    return LAPSUM_OK;
}

int lapsum_profile_disable(void *ws)
{
    if (!ws) return LAPSUM_ERR_NULL;
    WsHandle wsh;
    int rc = lock_ws(ws, wsh);
    WsInfo *W = wsh.W;
    if (rc) return rc;
    prof_destroy(W->prof);
    return LAPSUM_OK;
}

const char *lapsum_kernel_name(int kernel_id)
{
    static const char *names[LAPSUM_K_COUNT] = {"row_block_forward", "row_block_backward", "rs_histogram", "rs_onesweep",
                                                "tile_aggregate", "solve_global", "cdf_map", "vjp_reduce", "vjp_map",
                                                "sample_gather", "stream_band", "misc"};
    return (kernel_id >= 0 && kernel_id < LAPSUM_K_COUNT) ? names[kernel_id] : "?";
}

int64_t lapsum_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

const char *lapsum_error_string(int err)
{
    switch (err) {
    case LAPSUM_OK: return "ok";
    case LAPSUM_ERR_NULL: return "a required pointer is NULL";
    case LAPSUM_ERR_SHAPE: return "rows/n out of range";
    case LAPSUM_ERR_BUDGET: return "budget k must satisfy 0 < k < n";
    case LAPSUM_ERR_ALPHA: return "alpha must be a finite non-zero number whose magnitude fp32 holds as a normal number";
    case LAPSUM_ERR_WORKSPACE: return "workspace unknown, misaligned, too small or built for other dimensions";
    case LAPSUM_ERR_CUDA: return "CUDA runtime error";
    case LAPSUM_ERR_PARAM: return "lapsum_params field out of range";
    case LAPSUM_ERR_UNSUPPORTED: return "entry point not available for this workspace configuration";
    default: return "unknown error";
    }
}

int lapsum_last_cuda_error(void) { return g_last_cuda; }

}  // extern "C"
