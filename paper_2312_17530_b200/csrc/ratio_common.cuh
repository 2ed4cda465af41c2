// The two halves of one level of the ratio rule's radix selection (Eq. 3-5), shared by the
// plan-based kernels (ratio.cu) and the ones that allocate nothing (ratio_noalloc.cu): the
// histogram of one chunk of weight magnitudes, and what the last CTA to arrive does with the
// layers' histograms.  The callers differ only in where the layer table and the scratch live.
#pragma once

#include "device_utils.cuh"

namespace rsdgc {

template <int LEVEL>
struct RatioLevel {
    static constexpr int kBins = (LEVEL == 1) ? kL1Bins : (LEVEL == 2 ? kL2Bins : kL3Bins);
    static constexpr int kShiftHi = (LEVEL == 1) ? 31 : (LEVEL == 2 ? kL1Shift : kL2Shift);  // bit 31 of |w| is 0
    static constexpr int kShiftLo = (LEVEL == 1) ? kL1Shift : (LEVEL == 2 ? kL2Shift : 0);
};

struct RatioShared {
    unsigned int hist[kHistStride];
    unsigned long long gh64[kHistStride];  // per-bin totals over all layers (last CTA)
    unsigned long long scan_tmp[kThreads / 32];
    unsigned long long found[2];
    int is_last;
};

// Histogram (into sh.hist, cleared here) of the level's bits of the n magnitudes at wp that carry
// `prefix` in the bits above; wp is 16-byte aligned.  Ends with a barrier.
template <int LEVEL>
__device__ __forceinline__ void ratio_histogram_chunk(RatioShared &sh, const uint32_t *__restrict__ wp, int n,
                                                      uint32_t prefix, bool in_bounds)
{
    constexpr int NBINS = RatioLevel<LEVEL>::kBins, SHIFT_HI = RatioLevel<LEVEL>::kShiftHi,
                  SHIFT_LO = RatioLevel<LEVEL>::kShiftLo;
    constexpr int BATCH = 8;
    const int tid = threadIdx.x;
    for (int b = tid; b < NBINS; b += kThreads) sh.hist[b] = 0;
    __syncthreads();
    auto tally = [&](uint32_t w) {
        const uint32_t k = w & 0x7FFFFFFFu;
        if ((k >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(k >> SHIFT_LO) & (NBINS - 1)], 1u);
    };
    if (prefix != kTakeNone && in_bounds) {
        const int nvec = n >> 2;
        for (int base = 0; base < nvec; base += kThreads * BATCH) {
            uint4 q[BATCH];  // all loads of a batch are issued before any is consumed
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int i = base + u * kThreads + tid;
                q[u] = (i < nvec) ? __ldcs(reinterpret_cast<const uint4 *>(wp) + i) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < BATCH; ++u) {
                const int i = base + u * kThreads + tid;
                if (i < nvec) {
                    tally(q[u].x);
                    tally(q[u].y);
                    tally(q[u].z);
                    tally(q[u].w);
                }
            }
        }
        const int i = (nvec << 2) + tid;
        if (i < n) tally(wp[i]);
    }
    __syncthreads();
}

// Adds sh.hist to the layer's global histogram gh and takes a ticket; true in every thread of the
// CTA that arrived last of n_ctas.
template <int LEVEL>
__device__ __forceinline__ bool ratio_flush_and_ticket(RatioShared &sh, unsigned int *gh, RatioState *rs, int n_ctas)
{
    constexpr int NBINS = RatioLevel<LEVEL>::kBins;
    const int tid = threadIdx.x;
    for (int b = tid; b < NBINS; b += kThreads) {
        const unsigned int n = sh.hist[b];
        if (n) atomicAdd(gh + b, n);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned int t = atomicAdd(&rs->ticket, 1u);
        sh.is_last = (t + 1u == (unsigned int)n_ctas);
    }
    __syncthreads();
    if (!sh.is_last) return false;
    __threadfence();
    return true;
}

// The last CTA of a level: sums the layers' histograms in 64 bits (Eq. 4 ranks across the whole
// network), finds the bin that holds the n_keep-th largest magnitude, credits every layer with its
// entries above that bin, after level 3 hands the entries equal to the threshold to the layers in
// arena order and writes the ratios (Eq. 5), and clears the histograms and the ticket.
// hist_of(l): the layer's histogram (kHistStride words); size_of(l): its number of elements.
template <int LEVEL, typename HistOf, typename SizeOf>
__device__ __forceinline__ void ratio_resolve_level(RatioShared &sh, int n_layers, HistOf hist_of, SizeOf size_of,
                                                    RatioState *rs, long long *survivors, float *ratios,
                                                    long long n_keep, uint32_t prefix)
{
    constexpr int NBINS = RatioLevel<LEVEL>::kBins;
    constexpr int PER = NBINS / kThreads;
    const int tid = threadIdx.x;
    const long long remaining = (LEVEL == 1) ? n_keep : rs->remaining;
    const bool active = (LEVEL == 1) ? (n_keep > 0) : (prefix != kTakeNone);
    unsigned long long gsum[PER];
#pragma unroll
    for (int j = 0; j < PER; ++j) gsum[j] = 0;
    for (int l = 0; l < n_layers; ++l) {
        const unsigned int *lh = hist_of(l);
#pragma unroll
        for (int j = 0; j < PER; ++j) gsum[j] += __ldcg(lh + j * kThreads + tid);
    }
#pragma unroll
    for (int j = 0; j < PER; ++j) sh.gh64[j * kThreads + tid] = gsum[j];
    if (tid == 0) {
        sh.found[0] = 0;
        sh.found[1] = 0;
    }
    __syncthreads();
    // the bin from the top with 64-bit running sums: thread t owns bins NBINS-1-t*PER downwards
    unsigned long long local = 0;
#pragma unroll
    for (int j = 0; j < PER; ++j) local += sh.gh64[NBINS - 1 - (tid * PER + j)];
    unsigned long long total;
    const unsigned long long excl = block_exclusive_scan<unsigned long long>(local, sh.scan_tmp, &total);
    if (active && excl < (unsigned long long)remaining && (unsigned long long)remaining <= excl + local) {
        unsigned long long run = excl;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int b = NBINS - 1 - (tid * PER + j);
            const unsigned long long n = sh.gh64[b];
            if (run < (unsigned long long)remaining && (unsigned long long)remaining <= run + n) {
                sh.found[0] = (unsigned long long)b;
                sh.found[1] = (unsigned long long)remaining - run;
            }
            run += n;
        }
    }
    __syncthreads();
    const int bin = (int)sh.found[0];
    const long long rem_next = (long long)sh.found[1];

    // ---- every layer is credited with its entries above the bin (one warp per layer at a time)
    const int lane = tid & 31, warp = tid >> 5;
    for (int l = warp; l < n_layers; l += kThreads / 32) {
        const unsigned int *lh = hist_of(l);
        long long above = 0;
        if (active)
            for (int b = bin + 1 + lane; b < NBINS; b += 32) above += __ldcg(lh + b);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) above += __shfl_xor_sync(0xFFFFFFFFu, above, d);
        if (lane == 0) survivors[l] = (LEVEL == 1 ? 0 : survivors[l]) + above;
    }
    __syncthreads();
    if (LEVEL == 3 && tid == 0) {
        // entries equal to the threshold magnitude: lower arena position first (Eq. 4)
        long long left = active ? rem_next : 0;
        for (int l = 0; l < n_layers; ++l) {
            long long take = active ? (long long)__ldcg(hist_of(l) + bin) : 0;
            if (take > left) take = left;
            left -= take;
            const long long cl = survivors[l] + take;
            ratios[l] = (float)((double)cl / (double)size_of(l));  // Eq. 5
            survivors[l] = cl;
        }
    }
    __syncthreads();
    // ---- the histograms and the ticket start the next level / the next call from zero
    for (int l = 0; l < n_layers; ++l) {
        unsigned int *lh = hist_of(l);
        for (int b = tid; b < NBINS; b += kThreads) lh[b] = 0;
    }
    if (tid == 0) {
        rs->ticket = 0;
        if (LEVEL == 1) {
            rs->prefix = active ? (uint32_t)bin : kTakeNone;
            rs->remaining = rem_next;
            rs->n_keep = n_keep;
        } else if (LEVEL == 2) {
            if (active) rs->prefix = (prefix << kL2Bits) | (uint32_t)bin;
            rs->remaining = rem_next;
        }
    }
}

}  // namespace rsdgc
