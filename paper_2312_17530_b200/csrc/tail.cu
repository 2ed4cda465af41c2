// Everything after the accumulate+NSI pass in ONE kernel per layer-size class, for plans whose layers
// are small enough to keep a layer's keys on chip: keep count (Eq. 11), the three-level radix
// selection of the threshold (Algorithm 1's ranking), the payload indices, the gather of the kept
// values and the clearing of the accumulator (Sec. III-C, Eq. 12).
//
// Why: the chained kernels (two refinement passes, count, mark, gather) each cost a chain of
// dependent global round trips (table, layer state, keys, histogram flush, ticket, last CTA), about
// 7 us per kernel whatever the data, which is most of a call on network-sized layer sets.  Here a
// layer's keys are read from global memory once, into shared memory, and every later step works
// from there.
//
//  * k_tail<kTailCluster, ...>: a layer of up to kTailCluster * kTailKeysBig tiles is cut into slices
//    of kTailKeysBig keys, one slice per CTA, all CTAs of a layer in one thread-block cluster.  The
//    slices' histograms are added into the first CTA's ("leader") shared memory through distributed
//    shared memory; the leader resolves the level and the others read the result back.  Hardware
//    cluster barriers separate the steps (all CTAs of a cluster are co-scheduled; no flag is polled).
//    Several layers share a cluster when their slices fit; ranks without a slice only take part in
//    the barriers.
//  * k_tail<1, ...>: layers of at most kTailKeysSmall tiles, one CTA per layer, no cluster.
//
// The payload offsets of a layer need nothing but the ratios (k_l = ceil(K_l * ratio_l) of the
// preceding layers), so every CTA computes its own before it waits for the first pass.
#include <cooperative_groups.h>
#include <cuda_bf16.h>

#include "device_utils.cuh"

namespace cg = cooperative_groups;

namespace rsdgc {

template <int NT>
struct TailShared {
    unsigned int hist[kL2Bins];              // this CTA's histogram; the leader's also receives the others'
    unsigned long long scan_tmp[NT / 32];
    unsigned long long found[2];
    unsigned int res[2];                     // leader: what the level resolved (bin / prefix, remaining)
    unsigned int cnt[kTailCluster][2];       // leader: per rank, keys above the threshold / equal to it
    unsigned int warp_cnt[NT / 32][2];       // per warp of this CTA: the same counts over the warp's keys
    long long idx_off, val_off;              // payload offsets of the layer
    int k;                                   // tiles to keep (Eq. 11)
};

// Block-wide sum of one value per thread (every thread gets it).  Two barriers.
template <int NT>
__device__ __forceinline__ unsigned long long block_sum(unsigned long long x, unsigned long long *tmp)
{
    unsigned long long total;
    (void)block_exclusive_scan<unsigned long long, NT>(x, tmp, &total);
    return total;
}

template <int CS, int KEYS, int NT, bool BF16VAL>
__global__ void __launch_bounds__(NT, 1)
k_tail(const __grid_constant__ LaneTable lanes, const LayerDev *__restrict__ layers,
       const TailSlice *__restrict__ slices, const float *__restrict__ ratios, int n_layers, long long idx_cap,
       long long val_cap, StatusDev *status, unsigned int flags, int wait_late)
{
    extern __shared__ __align__(16) unsigned char tail_smem_raw[];
    uint32_t *skeys = reinterpret_cast<uint32_t *>(tail_smem_raw);  // KEYS words
    __shared__ TailShared<NT> sh;
    const Lane &ln = lanes.l[blockIdx.y];
    const TailSlice sl = slices[blockIdx.x];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NW = NT / 32;
    const bool active = sl.n > 0;  // a rank without a slice only takes part in the cluster's barriers
    const bool leader = active && sl.rank == 0;

    // every CTA of a cluster runs the same sequence of barriers
    auto sync_all = [&]() {
        if constexpr (CS > 1) cg::this_cluster().sync();
        else __syncthreads();
    };
    // the leader's copy of a shared-memory object (this CTA's own when it is the leader)
    auto at_leader = [&](auto *p) {
        if constexpr (CS > 1) return cg::this_cluster().map_shared_rank(p, (unsigned int)sl.leader);
        else return p;
    };

    // ---- what needs only the plan and the ratios: k_l and the layer's payload offsets
    for (int b = tid; b < kL2Bins; b += NT) sh.hist[b] = 0;
    if (active) {
        long long si = 0, sv = 0;
        for (int l = tid; l < sl.layer; l += NT) {
            const long long kk = keep_count(layers[l].K, ratios[l], flags);
            si += kk;
            sv += kk * layers[l].slot;
        }
        const unsigned long long ti = block_sum<NT>((unsigned long long)si, sh.scan_tmp);
        const unsigned long long tv = block_sum<NT>((unsigned long long)sv, sh.scan_tmp);
        if (tid == 0) {
            sh.idx_off = (long long)ti;
            sh.val_off = (long long)tv;
            sh.k = keep_count(layers[sl.layer].K, ratios[sl.layer], flags);
        }
    }
    // ---- the first pass has written the keys (a kernel launched right behind a sibling of this one
    // starts only after that sibling's CTAs have passed this wait, and waits itself before it exits)
    if (!wait_late) grid_dependency_wait();
    grid_dependency_launch_next();
    const LayerDev L = layers[active ? sl.layer : 0];
    if (active) {
        const uint32_t *kp = ln.keys + L.tile_off + sl.start;  // 16-byte aligned: offsets are multiples of 64 keys
        const int nvec = sl.n >> 2;
        for (int i = tid; i < nvec; i += NT)
            reinterpret_cast<uint4 *>(skeys)[i] = __ldcg(reinterpret_cast<const uint4 *>(kp) + i);
        for (int i = (nvec << 2) + tid; i < sl.n; i += NT) skeys[i] = __ldcg(kp + i);
    }
    __syncthreads();
    sync_all();  // every histogram of the cluster is zero before anything is added to a leader's
    const int k = active ? sh.k : 0;

    // ---- three radix levels on the key bits 30..21, 20..10, 9..0
    uint32_t prefix = (k > 0) ? 0u : kTakeNone;  // key bits resolved so far
    unsigned int remaining = (unsigned int)k;    // tiles still to take among the keys that carry the prefix
#pragma unroll
    for (int level = 1; level <= 3; ++level) {
        const int shift_hi = level == 1 ? 31 : (level == 2 ? kL1Shift : kL2Shift);
        const int shift_lo = level == 1 ? kL1Shift : (level == 2 ? kL2Shift : 0);
        const int nbins = level == 2 ? kL2Bins : kL1Bins;
        if (active && prefix != kTakeNone) {
            for (int i = tid; i < sl.n; i += NT) {
                const uint32_t key = skeys[i];
                if ((key >> shift_hi) == prefix) atomicAdd(&sh.hist[(key >> shift_lo) & (nbins - 1)], 1u);
            }
            if (CS > 1 && !leader) {
                __syncthreads();
                unsigned int *lh = at_leader(&sh.hist[0]);
                for (int b = tid; b < nbins; b += NT) {
                    const unsigned int c = sh.hist[b];
                    if (c) {
                        atomicAdd(lh + b, c);
                        sh.hist[b] = 0;
                    }
                }
            }
        }
        sync_all();
        if (leader && prefix != kTakeNone) {
            if (level == 2) find_bin_from_top<kL2Bins, NT>(sh.hist, (unsigned long long)remaining, sh.found, sh.scan_tmp);
            else find_bin_from_top<kL1Bins, NT>(sh.hist, (unsigned long long)remaining, sh.found, sh.scan_tmp);
            if (tid == 0) {
                sh.res[0] = (unsigned int)sh.found[0];
                sh.res[1] = (unsigned int)sh.found[1];
            }
            for (int b = tid; b < nbins; b += NT) sh.hist[b] = 0;
        }
        sync_all();
        if (active && prefix != kTakeNone) {
            const unsigned int *res = at_leader(&sh.res[0]);
            prefix = (prefix << (level == 2 ? kL2Bits : kL1Bits)) | res[0];
            remaining = res[1];
        }
    }
    const uint32_t T = prefix;                 // the threshold key, or kTakeNone
    const long long e = (long long)remaining;  // keys equal to T that are taken, lowest tile index first

    // ---- per warp, per CTA, per layer: how many keys lie above T and how many equal it
    // warp w owns the keys [w * per_warp, (w + 1) * per_warp) of the slice
    constexpr int per_warp = KEYS / NW;
    const int w0 = warp * per_warp;
    {
        unsigned int gt = 0, eq = 0;
        if (active && T != kTakeNone)
            for (int i = w0 + lane; i < min(sl.n, w0 + per_warp); i += 32) {
                const uint32_t key = skeys[i];
                gt += key > T;
                eq += key == T;
            }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            gt += __shfl_xor_sync(0xFFFFFFFFu, gt, d);
            eq += __shfl_xor_sync(0xFFFFFFFFu, eq, d);
        }
        if (lane == 0) {
            sh.warp_cnt[warp][0] = gt;
            sh.warp_cnt[warp][1] = eq;
        }
    }
    __syncthreads();
    if (active && tid == 0) {
        unsigned int a = 0, b = 0;
        for (int w = 0; w < NW; ++w) {
            a += sh.warp_cnt[w][0];
            b += sh.warp_cnt[w][1];
        }
        unsigned int *c = at_leader(&sh.cnt[0][0]);
        c[2 * sl.rank] = a;
        c[2 * sl.rank + 1] = b;
    }
    sync_all();
    long long lay_gt0 = 0, lay_eq0 = 0;  // keys above / equal in the slices of the layer before this one
    if (active) {
        const unsigned int *c = at_leader(&sh.cnt[0][0]);
        for (int r = 0; r < sl.rank; ++r) {
            lay_gt0 += c[2 * r];
            lay_eq0 += c[2 * r + 1];
        }
    }
    sync_all();  // nothing of another CTA's shared memory is touched from here on
    if (!active) {
        if (wait_late) grid_dependency_wait();
        return;
    }

    const long long idx_off = sh.idx_off, val_off = sh.val_off;
    if (leader && tid == 0) {
        ln.counts[sl.layer] = k;
        if (sl.layer == n_layers - 1) {
            const long long need_i = idx_off + k, need_v = val_off + (long long)k * L.slot;
            status->idx_needed = need_i;
            status->val_needed = need_v;
            if (need_i > idx_cap || need_v > val_cap) atomicOr(&status->flags, RSDGC_STATUS_PAYLOAD_OVERFLOW);
        }
    }
    if (T == kTakeNone) {
        if (wait_late) grid_dependency_wait();
        return;
    }

    // ---- payload indices: a tile is kept if its key is above T, or equals T with fewer than e equal
    // keys before it in the layer; its slot is the number of kept tiles before it
    long long gt_before = lay_gt0, eq_before = lay_eq0, cta_gt = 0, cta_eq = 0;
    for (int w = 0; w < NW; ++w) {
        if (w < warp) {
            gt_before += sh.warp_cnt[w][0];
            eq_before += sh.warp_cnt[w][1];
        }
        cta_gt += sh.warp_cnt[w][0];
        cta_eq += sh.warp_cnt[w][1];
    }
    int32_t *__restrict__ idx = ln.idx;
    for (int base = w0; base < min(sl.n, w0 + per_warp); base += 32) {
        const int i = base + lane;
        const uint32_t key = (i < sl.n) ? skeys[i] : 0u;
        const bool above = (i < sl.n) && key > T, equal = (i < sl.n) && key == T;
        const unsigned int ma = __ballot_sync(0xFFFFFFFFu, above), me = __ballot_sync(0xFFFFFFFFu, equal);
        const unsigned int lower = (1u << lane) - 1u;
        const long long g_rank = gt_before + __popc(ma & lower), e_rank = eq_before + __popc(me & lower);
        if (above || (equal && e_rank < e)) {
            const long long s = idx_off + g_rank + min(e_rank, e);
            if (s < idx_cap) idx[s] = sl.start + i;
        }
        gt_before += __popc(ma);
        eq_before += __popc(me);
    }
    __syncthreads();  // the gather below reads the indices this CTA has just written

    // ---- gather: the values of the kept tiles leave the accumulator (Eq. 12)
    // kept tiles of this CTA: payload slots [s_first, s_first + n_kept) of the call
    const long long s_first = idx_off + lay_gt0 + min(lay_eq0, e);
    const long long n_kept = cta_gt + (min(lay_eq0 + cta_eq, e) - min(lay_eq0, e));
    const int slot = L.slot;
    float *__restrict__ resid = ln.resid;
    float *__restrict__ val = reinterpret_cast<float *>(ln.val);
    __nv_bfloat16 *__restrict__ val16 = reinterpret_cast<__nv_bfloat16 *>(ln.val);
    constexpr int kBatch = 4;
    const long long n_vals = n_kept * slot;
    for (long long j0 = 0; j0 < n_vals; j0 += (long long)NT * kBatch) {
        long long ga[kBatch], vo[kBatch];
        float xv[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const long long j = j0 + u * NT + tid;
            ga[u] = -1;
            vo[u] = -1;
            if (j < n_vals) {
                long long q;
                int el;
                if (j < 0x7FFFFFFFll) {
                    int qq;
                    divmod_small((int)j, slot, &qq, &el);
                    q = qq;
                } else {
                    q = j / slot;
                    el = (int)(j - q * slot);
                }
                const long long s = s_first + q;
                // tiles that do not fit the payload buffers are not sent and stay in the accumulator
                if (s < idx_cap && val_off + (s - idx_off + 1) * slot <= val_cap) {
                    const int tile = __ldcg(idx + s);
                    const int tr = tile / L.TC, tc = tile - tr * L.TC;
                    int a, b;
                    divmod_small(el, L.nw, &a, &b);
                    const long long i = (long long)tr * L.nh + a, jj = (long long)tc * L.nw + b;
                    if (i < L.rows && jj < L.cols) ga[u] = L.elem_off + i * L.cols + jj;
                    vo[u] = val_off + (s - idx_off) * slot + el;
                }
            }
        }
        if (BF16VAL) {  // q = bfloat16(v) is sent, v - q stays (exact in binary32)
#pragma unroll
            for (int u = 0; u < kBatch; ++u) xv[u] = (ga[u] >= 0) ? resid[ga[u]] : 0.0f;
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const __nv_bfloat16 q = __float2bfloat16_rn(xv[u]);
                if (ga[u] >= 0) resid[ga[u]] = __fsub_rn(xv[u], __bfloat162float(q));
                if (vo[u] >= 0) val16[vo[u]] = q;
            }
        } else {  // read v and leave +0 in one exchange (see k_gather)
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                xv[u] = (ga[u] >= 0) ? __uint_as_float(atomicExch(reinterpret_cast<unsigned int *>(resid) + ga[u], 0u))
                                     : 0.0f;
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                if (vo[u] >= 0) val[vo[u]] = xv[u];
        }
    }
    if (wait_late) grid_dependency_wait();
}

// ------------------------------------------------------------------------------------------

constexpr size_t kTailSmemBig = (size_t)kTailKeysBig * sizeof(uint32_t);
constexpr size_t kTailSmemSmall = (size_t)kTailKeysSmall * sizeof(uint32_t);

template <bool BF16VAL>
static cudaError_t tail_configure()
{
    cudaError_t e = cudaFuncSetAttribute(k_tail<kTailCluster, kTailKeysBig, kTailThreadsBig, BF16VAL>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTailSmemBig);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(k_tail<1, kTailKeysSmall, kTailThreadsSmall, BF16VAL>,
                                 cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTailSmemSmall);
    return e;
}

// How many clusters of the big variant the current device can hold at a time (0 on failure).
int tail_max_active_clusters()
{
    if (tail_configure<false>() != cudaSuccess || tail_configure<true>() != cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kTailCluster * 64);
    cfg.blockDim = dim3(kTailThreadsBig);
    cfg.dynamicSmemBytes = kTailSmemBig;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kTailCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, k_tail<kTailCluster, kTailKeysBig, kTailThreadsBig, false>, &cfg) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return 0;
    }
    return n;
}

template <bool BF16VAL>
static cudaError_t launch_tail_typed(rsdgc_plan *p, const LaneTable &lanes, int n_lanes, const float *ratios,
                                     long long idx_cap, long long val_cap, int prof, cudaStream_t s,
                                     cudaError_t (*mark)(rsdgc_plan *, cudaStream_t))
{
    cudaError_t e = cudaSuccess;
    const LayerDev *layers = p->d_layers;
    const bool have_big = p->n_tail_big > 0, have_small = p->n_tail_small > 0;
    if (have_big) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)p->n_tail_big, (unsigned)n_lanes);
        cfg.blockDim = dim3(kTailThreadsBig);
        cfg.dynamicSmemBytes = kTailSmemBig;
        cfg.stream = s;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = kTailCluster;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 2;
        const TailSlice *slices = p->d_tail_slices;
        e = cudaLaunchKernelEx(&cfg, k_tail<kTailCluster, kTailKeysBig, kTailThreadsBig, BF16VAL>, lanes, layers, slices,
                               ratios, p->n_layers, idx_cap, val_cap, p->d_status, (unsigned int)p->flags, 0);
        count_launch(1);
    }
    if (prof >= 2 && e == cudaSuccess) e = mark(p, s);
    if (have_small && e == cudaSuccess) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)p->n_tail_small, (unsigned)n_lanes);
        cfg.blockDim = dim3(kTailThreadsSmall);
        cfg.dynamicSmemBytes = kTailSmemSmall;
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const TailSlice *slices = p->d_tail_slices + p->n_tail_big;
        // behind the cluster kernel it may start as soon as that kernel's CTAs have seen the first pass
        // complete (the layers of the two kernels are disjoint); with event records in between it may not
        const int wait_late = (have_big && prof < 2) ? 1 : 0;
        e = cudaLaunchKernelEx(&cfg, k_tail<1, kTailKeysSmall, kTailThreadsSmall, BF16VAL>, lanes, layers, slices, ratios,
                               p->n_layers, idx_cap, val_cap, p->d_status, (unsigned int)p->flags, wait_late);
        count_launch(1);
    }
    if (prof >= 2 && e == cudaSuccess) e = mark(p, s);
    return e;
}

cudaError_t launch_tail(rsdgc_plan *p, const LaneTable &lanes, int n_lanes, const float *ratios, long long idx_cap,
                        long long val_cap, int prof, cudaStream_t s, cudaError_t (*mark)(rsdgc_plan *, cudaStream_t))
{
    return (p->flags & RSDGC_PAYLOAD_BF16)
               ? launch_tail_typed<true>(p, lanes, n_lanes, ratios, idx_cap, val_cap, prof, s, mark)
               : launch_tail_typed<false>(p, lanes, n_lanes, ratios, idx_cap, val_cap, prof, s, mark);
}

}  // namespace rsdgc
