// rsdgc_update_ratios_noalloc(): the layer-wise ratio rule for callers that must not
// allocate device memory.  Same computation as rsdgc_update_ratios() (three-level radix
// selection on the weight magnitudes), but it needs no plan: the layer table travels in the
// kernel parameters and every byte of scratch lives in one file-scope device array.
#include <climits>
#include <cmath>
#include <mutex>

#include "ratio_common.cuh"

namespace rsdgc {

constexpr int kNoAllocMaxLayers = RSDGC_NOALLOC_MAX_LAYERS;
constexpr int kNoAllocMaxDevices = 64;

// Layer table passed by value in the kernel parameters (about 1.3 KB).
struct NoAllocLayers {
    long long off[kNoAllocMaxLayers];        // first element of the layer in the weight arena
    long long size[kNoAllocMaxLayers];       // elements of the layer
    int chunk_begin[kNoAllocMaxLayers + 1];  // first 16384-element chunk of the layer; [n_layers] = total
    int n_layers;
};

struct NoAllocScratch {
    unsigned int hist[kNoAllocMaxLayers][kHistStride];  // per-layer histogram of the current level
    long long survivors[kNoAllocMaxLayers];
    RatioState rs;
};

// The scratch itself: about 513 KB of device memory on every GPU that loads the library, held
// until the process exits.  All calls on a device share it.
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoAllocScratch)];

template <int LEVEL>
__global__ void __launch_bounds__(kThreads)
k_ratio_noalloc(const float *__restrict__ weights, const __grid_constant__ NoAllocLayers t, NoAllocScratch *sc,
                float *ratios, long long n_keep)
{
    __shared__ RatioShared sh;
    const int n_layers = t.n_layers;
    const int n_chunks = t.chunk_begin[n_layers];

    // the layer this CTA's chunk belongs to
    int lo = 0, hi = n_layers;
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (t.chunk_begin[mid] <= (int)blockIdx.x) lo = mid; else hi = mid;
    }
    const int layer = lo;
    const long long start = (long long)((int)blockIdx.x - t.chunk_begin[layer]) * kChunkKeys;
    const int n = (int)min((long long)kChunkKeys, t.size[layer] - start);

    const uint32_t prefix = (LEVEL == 1) ? 0u : sc->rs.prefix;
    ratio_histogram_chunk<LEVEL>(sh, reinterpret_cast<const uint32_t *>(weights) + t.off[layer] + start, n, prefix, true);
    if (!ratio_flush_and_ticket<LEVEL>(sh, sc->hist[layer], &sc->rs, n_chunks)) return;
    ratio_resolve_level<LEVEL>(
        sh, n_layers, [&](int l) { return sc->hist[l]; }, [&](int l) { return t.size[l]; }, &sc->rs, sc->survivors,
        ratios, n_keep, prefix);
}

// Device address of the scratch array on the current device, looked up once per device.
static cudaError_t noalloc_scratch_ptr(NoAllocScratch **out)
{
    static std::mutex mu;
    static void *ptrs[kNoAllocMaxDevices] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kNoAllocMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!ptrs[dev]) {
        // In host code the array's name is only a handle: the address a kernel can use has
        // to be asked for, with the device current.
        void *p = nullptr;
        e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
        if (e != cudaSuccess) return e;
        ptrs[dev] = p;
    }
    *out = reinterpret_cast<NoAllocScratch *>(ptrs[dev]);
    return cudaSuccess;
}

}  // namespace rsdgc

using namespace rsdgc;

extern "C" int rsdgc_update_ratios_noalloc(const float *weights_dev, const int64_t *layer_offsets_host,
                                           const int64_t *layer_sizes_host, int32_t n_layers, float global_keep,
                                           float *ratios_dev, void *stream)
{
    if (!weights_dev || !layer_offsets_host || !layer_sizes_host || !ratios_dev || n_layers < 1)
        return RSDGC_ERR_INVALID;
    if (!(global_keep >= 0.0f && global_keep <= 1.0f)) return RSDGC_ERR_INVALID;
    if (n_layers > kNoAllocMaxLayers) return RSDGC_ERR_CAPACITY;  // beyond the fixed scratch
    if (reinterpret_cast<uintptr_t>(weights_dev) & 15u) return RSDGC_ERR_ALIGNMENT;
    NoAllocLayers t{};
    t.n_layers = n_layers;
    long long chunks = 0, G = 0;
    for (int l = 0; l < n_layers; ++l) {
        const int64_t off = layer_offsets_host[l], size = layer_sizes_host[l];
        if (off < 0 || size < 1) return RSDGC_ERR_INVALID;
        if (size > (int64_t)INT32_MAX) return RSDGC_ERR_CAPACITY;
        if (off & 3) return RSDGC_ERR_ALIGNMENT;
        t.off[l] = off;
        t.size[l] = size;
        t.chunk_begin[l] = (int)chunks;
        chunks += (size + kChunkKeys - 1) / kChunkKeys;
        if (chunks > (long long)INT32_MAX) return RSDGC_ERR_CAPACITY;
        G += size;
    }
    t.chunk_begin[n_layers] = (int)chunks;
    const double x = std::ceil((double)global_keep * (double)G);
    const long long n_keep = x <= 0.0 ? 0 : (x >= (double)G ? G : (long long)x);

    NoAllocScratch *sc = nullptr;
    cudaError_t e = noalloc_scratch_ptr(&sc);
    cudaStream_t s = (cudaStream_t)stream;
    // the array keeps whatever the previous call (or an interrupted one) left behind
    if (e == cudaSuccess) e = cudaMemsetAsync(sc, 0, sizeof(NoAllocScratch), s);
    if (e == cudaSuccess) {
        k_ratio_noalloc<1><<<(unsigned)chunks, kThreads, 0, s>>>(weights_dev, t, sc, ratios_dev, n_keep);
        k_ratio_noalloc<2><<<(unsigned)chunks, kThreads, 0, s>>>(weights_dev, t, sc, ratios_dev, n_keep);
        k_ratio_noalloc<3><<<(unsigned)chunks, kThreads, 0, s>>>(weights_dev, t, sc, ratios_dev, n_keep);
        count_launch(3);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) {
        set_last_cuda_error((int)e);
        return RSDGC_ERR_CUDA;
    }
    return RSDGC_OK;
}
