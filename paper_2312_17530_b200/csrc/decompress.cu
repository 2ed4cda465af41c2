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

    for (long long j = (long long)blockIdx.x * kThreads + tid; j < total; j += (long long)gridDim.x * kThreads) {
        int lo = 0, hi = n_layers;  // layer with val_off[lo] <= j < val_off[lo + 1]
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (val_off[mid] <= j) lo = mid; else hi = mid;
        }
        const LayerDev &L = layers[lo];
        const long long jl = j - val_off[lo];
        const long long s = jl / L.slot;
        const int el = (int)(jl - s * L.slot);
        const int tile = idx[idx_off[lo] + s];
        if (tile < 0 || tile >= L.K) continue;
        const int tr = tile / L.TC, tc = tile - tr * L.TC;
        const int a = el / L.nw, b = el - a * L.nw;
        const long long i = (long long)tr * L.nh + a, jj = (long long)tc * L.nw + b;
        if (i < L.rows && jj < L.cols) {
            const long long g = L.elem_off + i * L.cols + jj;
            dense[g] = __fadd_rn(dense[g], __fmul_rn(scale, val[j]));
        }
    }
}

cudaError_t launch_decompress(rsdgc_plan *p, const int32_t *idx, const float *val, const int32_t *counts,
                              float scale, float *dense, cudaStream_t s)
{
    k_decompress<<<p->n_sm * 4, kThreads, 0, s>>>(idx, val, counts, p->d_layers, p->n_layers, scale, dense);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace rsdgc
