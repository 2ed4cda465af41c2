// Kernel of rsdgc_decompress_accumulate(): scatter-add of one worker's payload into the dense
// gradient arena (Eq. 12 third line / Eq. 2 Sync).  One launch per worker; inside a launch
// every dense element is touched by at most one thread, so plain read-modify-write is enough
// and the order of the binary32 additions across workers is the launch order.
#include "device_utils.cuh"

namespace rsdgc {

__global__ void __launch_bounds__(kThreads)
k_decompress(const int32_t *__restrict__ idx, const float *__restrict__ val,
             const int32_t *__restrict__ counts, const LayerDev *__restrict__ layers, int n_layers,
             float scale, float *__restrict__ dense)
{
    // exclusive prefix sums over the layers of k_l * slot_l (values) and k_l (tiles)
    __shared__ long long val_off[kMaxLayers + 1];
    __shared__ long long idx_off[kMaxLayers + 1];
    __shared__ unsigned long long scan_tmp[kThreads / 32];
    const int tid = threadIdx.x;
    unsigned long long carry_v = 0, carry_i = 0;
    for (int base = 0; base < n_layers; base += kThreads) {
        const int l = base + tid;
        long long k = 0, kv = 0;
        if (l < n_layers) {
            k = counts[l];
            if (k < 0) k = 0;
            kv = k * layers[l].slot;
        }
        unsigned long long tv, ti;
        const unsigned long long ev = block_exclusive_scan<unsigned long long>((unsigned long long)kv, scan_tmp, &tv);
        const unsigned long long ei = block_exclusive_scan<unsigned long long>((unsigned long long)k, scan_tmp, &ti);
        if (l < n_layers) {
            val_off[l] = (long long)(carry_v + ev);
            idx_off[l] = (long long)(carry_i + ei);
        }
        carry_v += tv;
        carry_i += ti;
    }
    if (tid == 0) {
        val_off[n_layers] = (long long)carry_v;
        idx_off[n_layers] = (long long)carry_i;
    }
    __syncthreads();
    const long long total = val_off[n_layers];

    constexpr int B = 4;  // independent entries per thread: index loads, then dense loads, then stores
    const long long stride = (long long)gridDim.x * kThreads;
    for (long long j0 = (long long)blockIdx.x * kThreads + tid; j0 < total; j0 += stride * B) {
        long long ga[B];
        float pv[B], dv[B];
        int tile[B], lay[B], el[B];
#pragma unroll
        for (int u = 0; u < B; ++u) {
            const long long j = j0 + u * stride;
            ga[u] = -1;
            tile[u] = -1;
            if (j < total) {
                int lo = 0, hi = n_layers;  // layer with val_off[lo] <= j < val_off[lo + 1]
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (val_off[mid] <= j) lo = mid; else hi = mid;
                }
                const int slot = layers[lo].slot;
                const long long jl = j - val_off[lo];
                const long long s = jl / slot;
                lay[u] = lo;
                el[u] = (int)(jl - s * slot);
                tile[u] = __ldg(idx + idx_off[lo] + s);
                pv[u] = __ldg(val + j);
            }
        }
#pragma unroll
        for (int u = 0; u < B; ++u) {
            if (tile[u] >= 0) {
                const LayerDev &L = layers[lay[u]];
                if (tile[u] < L.K) {
                    const int tr = tile[u] / L.TC, tc = tile[u] - tr * L.TC;
                    const int a = el[u] / L.nw, b = el[u] - a * L.nw;
                    const long long i = (long long)tr * L.nh + a, jj = (long long)tc * L.nw + b;
                    if (i < L.rows && jj < L.cols) ga[u] = L.elem_off + i * L.cols + jj;
                }
            }
        }
#pragma unroll
        for (int u = 0; u < B; ++u) dv[u] = (ga[u] >= 0) ? dense[ga[u]] : 0.0f;
#pragma unroll
        for (int u = 0; u < B; ++u)
            if (ga[u] >= 0) dense[ga[u]] = __fadd_rn(dv[u], __fmul_rn(scale, pv[u]));
    }
}

cudaError_t launch_decompress(rsdgc_plan *p, const int32_t *idx, const float *val, const int32_t *counts,
                              float scale, float *dense, cudaStream_t s)
{
    k_decompress<<<p->n_sm * 8, kThreads, 0, s>>>(idx, val, counts, p->d_layers, p->n_layers, scale, dense);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace rsdgc
