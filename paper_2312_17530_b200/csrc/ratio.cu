// Kernels of rsdgc_update_ratios(): layer-wise dynamic compression ratio (Eq. 3-5).
//
// The cross-layer ranking of |w| (Eq. 3-4) is done as a three-level radix selection on the
// magnitude bit patterns (sign bit cleared): per-layer histograms are accumulated by all
// CTAs; the last CTA to arrive sums them over the layers, finds the bin that holds the
// n_keep-th largest magnitude, and credits every layer with its entries above that bin.
// After the third level the threshold magnitude is exact; entries equal to it are credited
// to the layers in arena order (lower position first), so the survivors sum to n_keep.
#include "device_utils.cuh"

namespace rsdgc {

struct RatioShared {
    unsigned int hist[kHistStride];
    unsigned long long scan_tmp[kThreads / 32];
    unsigned long long found[2];
    int is_last;
};

template <int LEVEL>
__global__ void __launch_bounds__(kThreads)
k_ratio_level(const float *__restrict__ weights, const LayerDev *__restrict__ layers,
              const EChunk *__restrict__ echunks, int n_echunks, int n_layers, unsigned int *hist,
              RatioState *rs, long long *survivors, float *ratios, long long n_keep, StatusDev *status)
{
    __shared__ RatioShared sh;
    constexpr int NBINS = (LEVEL == 1) ? kL1Bins : (LEVEL == 2 ? kL2Bins : kL3Bins);
    constexpr int SHIFT_HI = (LEVEL == 1) ? 31 : (LEVEL == 2 ? kL1Shift : kL2Shift);
    constexpr int SHIFT_LO = (LEVEL == 1) ? kL1Shift : (LEVEL == 2 ? kL2Shift : 0);
    const int tid = threadIdx.x;
    const EChunk c = echunks[blockIdx.x];
    const uint32_t prefix = (LEVEL == 1) ? 0u : rs->prefix;  // bit 31 of |w| is 0
    for (int b = tid; b < NBINS; b += kThreads) sh.hist[b] = 0;
    __syncthreads();
    if (prefix != kTakeNone &&
        RSDGC_CHECKED((int)blockIdx.x < status->n_echunks && c.layer >= 0 && c.layer < status->n_layers && c.start >= 0 &&
                          layers[c.layer].elem_off + c.start + c.n <= status->arena_elems, status)) {
        const uint32_t *wp = reinterpret_cast<const uint32_t *>(weights) + layers[c.layer].elem_off + c.start;
        const int nvec = c.n >> 2;  // layer starts and chunk starts are multiples of 4 elements
        constexpr int BATCH = 8;
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
                    const uint32_t k0 = q[u].x & 0x7FFFFFFFu, k1 = q[u].y & 0x7FFFFFFFu;
                    const uint32_t k2 = q[u].z & 0x7FFFFFFFu, k3 = q[u].w & 0x7FFFFFFFu;
                    if ((k0 >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(k0 >> SHIFT_LO) & (NBINS - 1)], 1u);
                    if ((k1 >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(k1 >> SHIFT_LO) & (NBINS - 1)], 1u);
                    if ((k2 >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(k2 >> SHIFT_LO) & (NBINS - 1)], 1u);
                    if ((k3 >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(k3 >> SHIFT_LO) & (NBINS - 1)], 1u);
                }
            }
        }
        const int i = (nvec << 2) + tid;
        if (i < c.n) {
            const uint32_t q = wp[i] & 0x7FFFFFFFu;
            if ((q >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(q >> SHIFT_LO) & (NBINS - 1)], 1u);
        }
    }
    __syncthreads();
    unsigned int *gh = hist + (size_t)c.layer * kHistStride;
    for (int b = tid; b < NBINS; b += kThreads) {
        const unsigned int n = sh.hist[b];
        if (n) atomicAdd(gh + b, n);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned int t = atomicAdd(&rs->ticket, 1u);
        sh.is_last = (t + 1u == (unsigned int)n_echunks);
    }
    __syncthreads();
    if (!sh.is_last) return;
    __threadfence();

    // ---- last CTA: histogram summed over the layers in 64 bits (Eq. 4 ranks across the whole network)
    const long long remaining = (LEVEL == 1) ? n_keep : rs->remaining;
    const bool active = (LEVEL == 1) ? (n_keep > 0) : (prefix != kTakeNone);
    unsigned long long gsum[NBINS / kThreads];
#pragma unroll
    for (int j = 0; j < NBINS / kThreads; ++j) gsum[j] = 0;
    for (int l = 0; l < n_layers; ++l) {
        const unsigned int *lh = hist + (size_t)l * kHistStride;
#pragma unroll
        for (int j = 0; j < NBINS / kThreads; ++j) gsum[j] += __ldcg(lh + j * kThreads + tid);
    }
    // find the bin from the top with 64-bit running sums: bins are owned top-down by thread
    // order in find_bin_from_top, so redo it here on 64-bit per-bin totals kept in registers
    __shared__ unsigned long long gh64[NBINS];  // per-bin totals over all layers
#pragma unroll
    for (int j = 0; j < NBINS / kThreads; ++j) gh64[j * kThreads + tid] = gsum[j];
    __syncthreads();
    unsigned long long local = 0;
    constexpr int PER = NBINS / kThreads;
#pragma unroll
    for (int j = 0; j < PER; ++j) local += gh64[NBINS - 1 - (tid * PER + j)];
    unsigned long long total;
    const unsigned long long excl = block_exclusive_scan<unsigned long long>(local, sh.scan_tmp, &total);
    if (tid == 0) {
        sh.found[0] = 0;
        sh.found[1] = 0;
    }
    __syncthreads();
    if (active && excl < (unsigned long long)remaining && (unsigned long long)remaining <= excl + local) {
        unsigned long long run = excl;
#pragma unroll
        for (int j = 0; j < PER; ++j) {
            const int b = NBINS - 1 - (tid * PER + j);
            const unsigned long long n = gh64[b];
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

    // ---- credit every layer with its entries above the bin (one warp per layer at a time)
    const int lane = tid & 31, warp = tid >> 5;
    for (int l = warp; l < n_layers; l += kThreads / 32) {
        const unsigned int *lh = hist + (size_t)l * kHistStride;
        long long above = 0;
        if (active)
            for (int b = bin + 1 + lane; b < NBINS; b += 32) above += __ldcg(lh + b);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) above += __shfl_xor_sync(0xFFFFFFFFu, above, d);
        if (lane == 0) survivors[l] = (LEVEL == 1 ? 0 : survivors[l]) + above;
    }
    __syncthreads();
    if (LEVEL == 3 && tid == 0) {
        // entries equal to the threshold magnitude: lower arena position first
        long long left = active ? rem_next : 0;
        for (int l = 0; l < n_layers; ++l) {
            long long take = active ? (long long)__ldcg(hist + (size_t)l * kHistStride + bin) : 0;
            if (take > left) take = left;
            left -= take;
            const long long cl = survivors[l] + take;
            const double G = (double)(layers[l].rows * layers[l].cols);
            ratios[l] = (float)((double)cl / G);  // Eq. 5
            survivors[l] = cl;
        }
    }
    __syncthreads();
    // ---- reset the histograms and the ticket for the next level / next call
    for (int l = 0; l < n_layers; ++l) {
        unsigned int *lh = hist + (size_t)l * kHistStride;
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

cudaError_t launch_update_ratios(rsdgc_plan *p, const float *weights, long long n_keep, float *ratios,
                                 cudaStream_t s)
{
    const int n = (int)p->echunks.size();
    k_ratio_level<1><<<n, kThreads, 0, s>>>(weights, p->d_layers, p->d_echunks, n, p->n_layers, p->d_hist,
                                            p->d_rstate, p->d_survivors, ratios, n_keep, p->d_status);
    k_ratio_level<2><<<n, kThreads, 0, s>>>(weights, p->d_layers, p->d_echunks, n, p->n_layers, p->d_hist,
                                            p->d_rstate, p->d_survivors, ratios, n_keep, p->d_status);
    k_ratio_level<3><<<n, kThreads, 0, s>>>(weights, p->d_layers, p->d_echunks, n, p->n_layers, p->d_hist,
                                            p->d_rstate, p->d_survivors, ratios, n_keep, p->d_status);
    count_launch(3);
    return cudaGetLastError();
}

}  // namespace rsdgc
