// Kernel of rsdgc_payload_to_coo(): the per-element (coordinate) view of a payload.
//
// The payload names neighborhoods (Sec. III-C: a neighborhood index plus all the values of
// the neighborhood).  Receivers that want one position per value get it here: for payload
// value j, coo[j] is the arena position of the element it belongs to, or -1 for the +0 padding
// of a tile clipped by the layer's edge.  The values themselves stay where they are.
#include "device_utils.cuh"

namespace rsdgc {

constexpr int kCooBatch = 4;
constexpr int kLayersPerThread = kMaxLayers / kThreads;

struct CooShared {
    long long val_off[kMaxLayers + 1];
    long long idx_off[kMaxLayers];
    unsigned long long scan_tmp[kThreads / 32];
};

__global__ void __launch_bounds__(kThreads)
k_payload_to_coo(const int32_t *__restrict__ idx, const int32_t *__restrict__ counts,
                 const LayerDev *__restrict__ layers, int n_layers, long long *__restrict__ coo, long long coo_cap,
                 StatusDev *status)
{
    __shared__ CooShared sh;
    const int tid = threadIdx.x;
    // payload offsets of every layer: prefix sums of k_l and k_l * slot_l (thread t owns the
    // layers [t * kLayersPerThread, (t + 1) * kLayersPerThread))
    long long ki[kLayersPerThread], kv[kLayersPerThread];
    long long si = 0, sv = 0;
#pragma unroll
    for (int j = 0; j < kLayersPerThread; ++j) {
        const int l = tid * kLayersPerThread + j;
        long long k = (l < n_layers) ? (long long)counts[l] : 0;
        if (k < 0) k = 0;
        ki[j] = k;
        kv[j] = (l < n_layers) ? k * layers[l].slot : 0;
        si += ki[j];
        sv += kv[j];
    }
    unsigned long long tot_i, tot_v;
    long long bi = (long long)block_exclusive_scan<unsigned long long>((unsigned long long)si, sh.scan_tmp, &tot_i);
    long long bv = (long long)block_exclusive_scan<unsigned long long>((unsigned long long)sv, sh.scan_tmp, &tot_v);
#pragma unroll
    for (int j = 0; j < kLayersPerThread; ++j) {
        const int l = tid * kLayersPerThread + j;
        if (l < n_layers) {
            sh.idx_off[l] = bi;
            sh.val_off[l] = bv;
        }
        bi += ki[j];
        bv += kv[j];
    }
    if (tid == 0) sh.val_off[n_layers] = (long long)tot_v;
    __syncthreads();
    const long long total = min((long long)tot_v, coo_cap);
    const long long stride = (long long)gridDim.x * kThreads * kCooBatch;
    for (long long jb = (long long)blockIdx.x * kThreads * kCooBatch; jb < total; jb += stride) {
#pragma unroll
        for (int u = 0; u < kCooBatch; ++u) {
            const long long j = jb + u * kThreads + tid;
            if (j >= total) continue;
            int lo = 0, hi = n_layers;  // layer with val_off[lo] <= j < val_off[lo + 1]
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (sh.val_off[mid] <= j) lo = mid; else hi = mid;
            }
            const LayerDev &L = layers[lo];
            const long long jl = j - sh.val_off[lo];
            const long long s = jl / L.slot;
            const int el = (int)(jl - s * L.slot);
            const int tile = __ldg(idx + sh.idx_off[lo] + s);
            long long pos = -1;
            if (tile >= 0 && tile < L.K) {
                const int tr = tile / L.TC, tc = tile - tr * L.TC;
                const int a = el / L.nw, b = el - a * L.nw;
                const long long i = (long long)tr * L.nh + a, jj = (long long)tc * L.nw + b;
                if (i < L.rows && jj < L.cols) pos = L.elem_off + i * L.cols + jj;
                if (!RSDGC_CHECKED(pos < status->arena_elems, status)) pos = -1;
            }
            coo[j] = pos;
        }
    }
}

cudaError_t launch_payload_to_coo(rsdgc_plan *p, const int32_t *idx, const int32_t *counts, long long *coo,
                                  long long coo_cap, cudaStream_t s)
{
    k_payload_to_coo<<<p->n_sm * 4, kThreads, 0, s>>>(idx, counts, p->d_layers, p->n_layers, coo, coo_cap, p->d_status);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace rsdgc
