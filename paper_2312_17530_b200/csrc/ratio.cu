// Kernels of rsdgc_update_ratios(): layer-wise dynamic compression ratio (Eq. 3-5).
//
// The cross-layer ranking of |w| (Eq. 3-4) is done as a three-level radix selection on the
// magnitude bit patterns (sign bit cleared): per-layer histograms are accumulated by all
// CTAs; the last CTA to arrive sums them over the layers, finds the bin that holds the
// n_keep-th largest magnitude, and credits every layer with its entries above that bin.
// After the third level the threshold magnitude is exact; entries equal to it are credited
// to the layers in arena order (lower position first), so the survivors sum to n_keep.
#include "ratio_common.cuh"

namespace rsdgc {

template <int LEVEL>
__global__ void __launch_bounds__(kThreads)
k_ratio_level(const float *__restrict__ weights, const LayerDev *__restrict__ layers,
              const EChunk *__restrict__ echunks, int n_echunks, int n_layers, unsigned int *hist,
              RatioState *rs, long long *survivors, float *ratios, long long n_keep, StatusDev *status)
{
    __shared__ RatioShared sh;
    const EChunk c = echunks[blockIdx.x];
    const uint32_t prefix = (LEVEL == 1) ? 0u : rs->prefix;
    const bool ok = RSDGC_CHECKED((int)blockIdx.x < status->n_echunks && c.layer >= 0 && c.layer < status->n_layers &&
                                      c.start >= 0 && layers[c.layer].elem_off + c.start + c.n <= status->arena_elems,
                                  status);
    // layer starts and chunk starts are multiples of 4 elements
    ratio_histogram_chunk<LEVEL>(sh, reinterpret_cast<const uint32_t *>(weights) + layers[c.layer].elem_off + c.start,
                                 c.n, prefix, ok);
    if (!ratio_flush_and_ticket<LEVEL>(sh, hist + (size_t)c.layer * kHistStride, rs, n_echunks)) return;
    ratio_resolve_level<LEVEL>(
        sh, n_layers, [&](int l) { return hist + (size_t)l * kHistStride; },
        [&](int l) { return layers[l].rows * layers[l].cols; }, rs, survivors, ratios, n_keep, prefix);
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
