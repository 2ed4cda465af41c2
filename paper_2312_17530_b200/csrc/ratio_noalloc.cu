// rsdgc_update_ratios_noalloc(): the layer-wise ratio rule for callers that must not
// allocate device memory.  Same computation as rsdgc_update_ratios() (three-level radix
// selection on the weight magnitudes), but it needs no plan: the layer table travels in the
// kernel parameters and every byte of scratch lives in one file-scope device array.
#include <climits>
#include <cmath>
#include <mutex>

#include "device_utils.cuh"

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

struct NoAllocShared {
    unsigned int hist[kHistStride];
    unsigned long long gh64[kHistStride];
    unsigned long long scan_tmp[kThreads / 32];
    unsigned long long found[2];
    int is_last;
};

template <int LEVEL>
__global__ void __launch_bounds__(kThreads)
k_ratio_noalloc(const float *__restrict__ weights, const __grid_constant__ NoAllocLayers t, NoAllocScratch *sc,
                float *ratios, long long n_keep)
{
    __shared__ NoAllocShared sh;
    constexpr int NBINS = (LEVEL == 1) ? kL1Bins : (LEVEL == 2 ? kL2Bins : kL3Bins);
    constexpr int SHIFT_HI = (LEVEL == 1) ? 31 : (LEVEL == 2 ? kL1Shift : kL2Shift);
    constexpr int SHIFT_LO = (LEVEL == 1) ? kL1Shift : (LEVEL == 2 ? kL2Shift : 0);
    constexpr int BATCH = 8;
    const int tid = threadIdx.x;
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

    const uint32_t prefix = (LEVEL == 1) ? 0u : sc->rs.prefix;  // bit 31 of |w| is 0
    for (int b = tid; b < NBINS; b += kThreads) sh.hist[b] = 0;
    __syncthreads();
    if (prefix != kTakeNone) {
        const uint32_t *wp = reinterpret_cast<const uint32_t *>(weights) + t.off[layer] + start;
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
        if (i < n) {
            const uint32_t q = wp[i] & 0x7FFFFFFFu;
            if ((q >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(q >> SHIFT_LO) & (NBINS - 1)], 1u);
        }
    }
    __syncthreads();
    unsigned int *gh = sc->hist[layer];
    for (int b = tid; b < NBINS; b += kThreads) {
        const unsigned int c = sh.hist[b];
        if (c) atomicAdd(gh + b, c);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned int ticket = atomicAdd(&sc->rs.ticket, 1u);
        sh.is_last = (ticket + 1u == (unsigned int)n_chunks);
    }
    __syncthreads();
    if (!sh.is_last) return;
    __threadfence();

    // ---- last CTA to arrive: totals over the layers, the bin holding the n_keep-th magnitude
    const long long remaining = (LEVEL == 1) ? n_keep : sc->rs.remaining;
    const bool active = (LEVEL == 1) ? (n_keep > 0) : (prefix != kTakeNone);
    constexpr int PER = NBINS / kThreads;
    unsigned long long gsum[PER];
#pragma unroll
    for (int j = 0; j < PER; ++j) gsum[j] = 0;
    for (int l = 0; l < n_layers; ++l) {
#pragma unroll
        for (int j = 0; j < PER; ++j) gsum[j] += __ldcg(&sc->hist[l][j * kThreads + tid]);
    }
#pragma unroll
    for (int j = 0; j < PER; ++j) sh.gh64[j * kThreads + tid] = gsum[j];
    if (tid == 0) {
        sh.found[0] = 0;
        sh.found[1] = 0;
    }
    __syncthreads();
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
            const unsigned long long c = sh.gh64[b];
            if (run < (unsigned long long)remaining && (unsigned long long)remaining <= run + c) {
                sh.found[0] = (unsigned long long)b;
                sh.found[1] = (unsigned long long)remaining - run;
            }
            run += c;
        }
    }
    __syncthreads();
    const int bin = (int)sh.found[0];
    const long long rem_next = (long long)sh.found[1];

    // ---- every layer is credited with its entries above the bin
    const int lane = tid & 31, warp = tid >> 5;
    for (int l = warp; l < n_layers; l += kThreads / 32) {
        long long above = 0;
        if (active)
            for (int b = bin + 1 + lane; b < NBINS; b += 32) above += __ldcg(&sc->hist[l][b]);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) above += __shfl_xor_sync(0xFFFFFFFFu, above, d);
        if (lane == 0) sc->survivors[l] = (LEVEL == 1 ? 0 : sc->survivors[l]) + above;
    }
    __syncthreads();
    if (LEVEL == 3 && tid == 0) {
        // entries equal to the threshold magnitude go to the layers in arena order (Eq. 4)
        long long left = active ? rem_next : 0;
        for (int l = 0; l < n_layers; ++l) {
            long long take = active ? (long long)__ldcg(&sc->hist[l][bin]) : 0;
            if (take > left) take = left;
            left -= take;
            const long long cl = sc->survivors[l] + take;
            ratios[l] = (float)((double)cl / (double)t.size[l]);  // Eq. 5
        }
    }
    __syncthreads();
    // ---- the histograms and the ticket start the next level from zero
    for (int l = 0; l < n_layers; ++l)
        for (int b = tid; b < NBINS; b += kThreads) sc->hist[l][b] = 0;
    if (tid == 0) {
        sc->rs.ticket = 0;
        if (LEVEL == 1) {
            sc->rs.prefix = active ? (uint32_t)bin : kTakeNone;
            sc->rs.remaining = rem_next;
        } else if (LEVEL == 2) {
            if (active) sc->rs.prefix = (prefix << kL2Bits) | (uint32_t)bin;
            sc->rs.remaining = rem_next;
        }
    }
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
