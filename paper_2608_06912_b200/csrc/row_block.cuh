// Block path: one thread block per row.  The row is sorted in shared memory
// with a bitonic network, scanned and solved there (App. A), and the mask is
// evaluated from the unsorted scores so that no scatter is needed (the fused
// CDF of the paper's implementation notes, App. D).  The backward is the
// fused single-reduction VJP of Eq. 5.
#pragma once
#include "common.cuh"
#include "solve.cuh"

namespace lapsum {

__device__ __forceinline__ float ex2_approx(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Laplace CDF at (x - b)/t with b = th.hi + th.lo and c = log2(e)/t  (Eq. 3)
__device__ __forceinline__ float laplace_cdf(float x, RowThreshold th, float c)
{
    const float d = (x - th.hi) - th.lo;
    const float e = 0.5f * ex2_approx(-fabsf(d) * c);
    return d <= 0.f ? e : 1.f - e;
}

// Laplace density at b (Eq. 5): e^{-|b-x|/t}/(2t), half_inv_t = 1/(2t)
__device__ __forceinline__ float laplace_pdf(float x, float b, float c, float half_inv_t)
{
    return ex2_approx(-fabsf(x - b) * c) * half_inv_t;
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

struct BlockFwdArgs {
    const float *r;
    float *p;
    float *b;
    RowThreshold *th;  // nullable: per-row threshold pairs kept in the workspace
    Control *ctl;
    int n, n_pad;
    double k, t;
    ExpScale sc;
    float c;  // log2(e)/t in fp32 for the mask
};

// dynamic shared memory: n_pad keys, then pref[n], suf[n]
__global__ void row_block_forward_kernel(BlockFwdArgs a)
{
    pdl_wait();
    extern __shared__ __align__(16) unsigned char smem_raw[];
    uint32_t *keys = reinterpret_cast<uint32_t *>(smem_raw);
    float *pref = reinterpret_cast<float *>(keys + a.n_pad);
    float *suf = pref + a.n;
    __shared__ ScanShared sh;
    __shared__ SolveResult sh_res;

    const long long row = blockIdx.x;
    const float *rr = a.r + row * a.n;
    for (int i = threadIdx.x; i < a.n_pad; i += blockDim.x)
        keys[i] = (i < a.n) ? float_to_key(__ldg(rr + i)) : 0xffffffffu;
    __syncthreads();
    bitonic_sort_shared(keys, a.n_pad);
    float *s = reinterpret_cast<float *>(keys);
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) s[i] = key_to_float(keys[i]);
    __syncthreads();

    Seeds sd;
    sd.L = empty_up();
    sd.R = empty_down();
    sd.n_R = 0;
    SolveResult res = solve_sorted_block(s, a.n, sd, a.k, a.t, a.sc, pref, suf, sh, &sh_res, true, false);
    if (threadIdx.x == 0) {
        a.b[row] = res.b;
        if (a.th) a.th[row] = res.th;
        if (res.status) set_status(a.ctl, (unsigned)res.status);
        if (row == 0) {
            a.ctl->persist.last_path = 1;
            a.ctl->persist.forwards += 1;
        }
    }
    float *pp = a.p + row * a.n;
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) pp[i] = laplace_cdf(__ldg(rr + i), res.th, a.c);
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
    const float *v, *r, *b;
    float *grad;
    Control *ctl;
    int n;
    float c, half_inv_t;
};

__global__ void row_block_backward_kernel(BlockBwdArgs a)
{
    pdl_wait();
    __shared__ double red[32];
    const long long row = blockIdx.x;
    const float *rr = a.r + row * a.n, *vv = a.v + row * a.n;
    const float b = __ldg(a.b + row);
    float sf = 0.f, svf = 0.f;
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) {
        const float f = laplace_pdf(__ldg(rr + i), b, a.c, a.half_inv_t);
        sf += f;
        svf = fmaf(__ldg(vv + i), f, svf);
    }
    const double S_f = block_sum((double)sf, red);
    const double S_vf = block_sum((double)svf, red);
    const float mean = (S_f > 0.0) ? (float)(S_vf / S_f) : 0.f;
    float *gg = a.grad + row * a.n;
    for (int i = threadIdx.x; i < a.n; i += blockDim.x) {
        const float f = laplace_pdf(__ldg(rr + i), b, a.c, a.half_inv_t);
        gg[i] = (S_f > 0.0) ? f * (__ldg(vv + i) - mean) : 0.f;
    }
    if (threadIdx.x == 0 && row == (long long)gridDim.x - 1) {
        a.ctl->persist.S_f = S_f;
        a.ctl->persist.S_vf = S_vf;
    }
}

}  // namespace lapsum
