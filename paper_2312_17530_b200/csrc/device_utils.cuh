// Block-level helpers used by several kernels (256-thread CTAs).
#pragma once

#include "rsdgc_internal.cuh"

namespace rsdgc {

// Exclusive prefix sum of one value per thread over the CTA, in thread order.
// `warp_tot` points to NTHREADS/32 words of shared memory.  Every thread receives the CTA
// total in *total.  Contains two barriers; all threads must call it.
template <typename T, int NTHREADS = kThreads>
__device__ __forceinline__ T block_exclusive_scan(T x, T *warp_tot, T *total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    T incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        T y = __shfl_up_sync(0xFFFFFFFFu, incl, d);
        if (lane >= d) incl += y;
    }
    if (lane == 31) warp_tot[warp] = incl;
    __syncthreads();
    T offset = 0, sum = 0;
#pragma unroll
    for (int w = 0; w < NTHREADS / 32; ++w) {
        T t = warp_tot[w];
        if (w < warp) offset += t;
        sum += t;
    }
    __syncthreads();
    *total = sum;
    return offset + incl - x;
}

// Walks a histogram in shared memory from its highest bin downwards and finds the bin in
// which the running count reaches `need` (need >= 1): out[0] = bin, out[1] = how many
// entries of that bin are still needed (need minus the count of all higher bins).
// If the histogram holds fewer than `need` entries, bin 0 is returned with what is missing.
// `out` and `warp_tot` are shared memory; all threads must call; ends with a barrier.
template <int NBINS, int NTHREADS = kThreads>
__device__ __forceinline__ void find_bin_from_top(const unsigned int *h, unsigned long long need,
                                                  unsigned long long *out, unsigned long long *warp_tot)
{
    constexpr int PER = NBINS / NTHREADS;
    static_assert(NBINS % NTHREADS == 0, "histogram size must be a multiple of the CTA size");
    unsigned long long local = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) local += h[NBINS - 1 - (threadIdx.x * PER + j)];
    unsigned long long total;
    unsigned long long excl = block_exclusive_scan<unsigned long long, NTHREADS>(local, warp_tot, &total);
    if (threadIdx.x == 0 && total < need) {
        out[0] = 0;
        out[1] = need - (total - h[0]);
    }
    if (excl < need && need <= excl + local) {
        unsigned long long run = excl;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int b = NBINS - 1 - (threadIdx.x * PER + j);
            const unsigned long long c = h[b];
            if (run < need && need <= run + c) {
                out[0] = (unsigned long long)b;
                out[1] = need - run;
            }
            run += c;
        }
    }
    __syncthreads();
}

// Bounds-checked build (-DRSDGC_DEBUG): every index a kernel forms into a caller's buffer or a plan
// table is tested against the extents recorded in the status block; a failure raises
// RSDGC_STATUS_BOUNDS and the access is skipped.  In the normal build the test is not compiled.
#ifdef RSDGC_DEBUG
__device__ __forceinline__ bool debug_in_bounds(bool ok, StatusDev *st)
{
    if (!ok) atomicOr(&st->flags, RSDGC_STATUS_BOUNDS);
    return ok;
}
#define RSDGC_CHECKED(cond, st) debug_in_bounds((cond), (st))
#else
#define RSDGC_CHECKED(cond, st) true
#endif

// Programmatic dependent launch: a kernel launched with the "programmatic stream
// serialization" attribute may start while its predecessor in the stream is still draining.
// grid_dependency_wait() returns once the predecessor has completed and its writes are visible;
// everything before it may only touch data that no earlier kernel of the same call writes
// (plan tables, shared memory).  grid_dependency_launch_next() lets the successor start; it is
// called after the wait so that completion stays transitive along the chain of kernels.
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dependency_launch_next()
{
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// floor(x / d) for x < 8192 and d <= 8192 by a multiply-high with inv = ceil(2^32 / d)
// (inv = 0 encodes d = 1).
__device__ __forceinline__ int fast_div(int x, unsigned int inv)
{
    return inv ? (int)__umulhi((unsigned int)x, inv) : x;
}

// x / d and x % d for 0 <= x < 2^31, d >= 1, with the common divisors (3, 9) as compile-time
// constants (multiply + shift instead of the generic division sequence).
__device__ __forceinline__ void divmod_small(int x, int d, int *q, int *r)
{
    int qq;
    if (d == 9) qq = x / 9;
    else if (d == 3) qq = x / 3;
    else if (d == 1) qq = x;
    else qq = x / d;
    *q = qq;
    *r = x - qq * d;
}

// Number of tiles to keep, k = ceil(K * ratio) (Eq. 11) limited to [0 or 1, K]; the product
// is taken in binary64 on the binary32 ratio.
__device__ __forceinline__ int keep_count(int K, float ratio, unsigned int flags)
{
    const double x = ceil((double)K * (double)ratio);
    int k = (x > 0.0) ? ((x >= (double)K) ? K : (int)x) : 0;
    if ((flags & RSDGC_KEEP_AT_LEAST_ONE) && k < 1) k = 1;
    return k < K ? k : K;
}

}  // namespace rsdgc
