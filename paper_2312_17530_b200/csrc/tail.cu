// Everything after the accumulate+NSI pass in ONE kernel per layer-size class, for plans whose layers
// are small enough to keep a layer's keys on chip: levels 2 and 3 of the radix selection of the
// threshold (Algorithm 1's ranking; level 1 and the keep count of Eq. 11 come with the first pass,
// whose histogram work is spread over all SMs), the payload indices, the gather of the kept values
// and the clearing of the accumulator (Sec. III-C, Eq. 12).
//
// Why: the chained kernels (two refinement passes, count, mark, gather) each cost a chain of
// dependent global round trips (table, layer state, keys, histogram flush, ticket, last CTA), about
// 7 us per kernel whatever the data, which is most of a call on network-sized layer sets.  Here a
// layer's keys are read from global memory once, into shared memory, and every later step works
// from there.  (Keys held in registers would need fully unrolled passes: measured, the instruction
// fetches of the straight-line code, cold after every call, cost more than the shared-memory reads.)
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

constexpr int kTailCand = 1024;  // candidates a CTA can list (keys that share the threshold's upper 21 bits)

template <int NT, int KEYS>
struct TailShared {
    unsigned int hist[kL2Bins];              // this CTA's histogram; the leader's also receives the others'
    unsigned long long scan_tmp[NT / 32];
    unsigned long long found[2];
    unsigned int res[3];                     // leader: what a level resolved (bin, remaining), fallback flag
    unsigned int cnt[kTailCluster][2];       // leader: per rank, keys above the threshold / equal to it
    unsigned int overflow[kTailCluster];     // leader: per rank, its candidate list did not hold its candidates
    unsigned int warp_cnt[NT / 32][2];       // per warp of this CTA: kept-for-sure / equal keys in the warp's range
    unsigned int warp_pre[NT / 32 + 1][2];   // the counts of the warps before each warp; last entry: the CTA's totals
    unsigned int above[KEYS / 32];           // one bit per key of the slice: above the threshold
    unsigned int equal[KEYS / 32];           // ... equal to the threshold
    unsigned int cand[kTailCand];            // candidates: key bits 9..0 << 15 | position in the slice
    unsigned int n_cand;
    long long idx_off, val_off;              // payload offsets of the layer
};

// Block-wide sum of one value per thread (every thread gets it).  Not inlined: these kernels run
// once per call, so their code is kept small (loops with a little unrolling for memory-level
// parallelism, one copy of every helper).
template <int NT>
__device__ __noinline__ unsigned long long block_sum(unsigned long long x, unsigned long long *tmp)
{
    unsigned long long total;
    (void)block_exclusive_scan<unsigned long long, NT>(x, tmp, &total);
    return total;
}

template <int NT>
__device__ __noinline__ void tail_find_bin(const unsigned int *h, unsigned long long need, unsigned long long *out,
                                           unsigned long long *tmp)
{
    find_bin_from_top<kL2Bins, NT>(h, need, out, tmp);
}

// How the passes over a slice are kept few: a CTA is one SM, and every pass over up to 32768 keys costs
// it 2 to 3 us.  Level 2 is histogrammed while the keys arrive.  After level 2 the upper 21 bits of
// the threshold are known: a key above them is kept, a key below is not, and the few keys that share
// them ("candidates") decide the rest.  ONE pass writes a bit per key (above) and lists the
// candidates; level 3, the equal keys and all ranks then come from the list and the bit masks.  If some
// CTA of the layer has more candidates than its list holds (many equal indicators: constant layers),
// the layer takes one more pass: level 3 over all its keys, then the masks from the full threshold.
template <int CS, int KEYS, int NT, bool BF16VAL>
__global__ void __launch_bounds__(NT, 1)
k_tail(const __grid_constant__ LaneTable lanes, const LayerDev *__restrict__ layers,
       const TailSlice *__restrict__ slices, const float *__restrict__ ratios, int n_layers, long long idx_cap,
       long long val_cap, StatusDev *status, unsigned int flags, int wait_late)
{
    extern __shared__ __align__(16) unsigned char tail_smem_raw[];
    uint32_t *skeys = reinterpret_cast<uint32_t *>(tail_smem_raw);  // KEYS words
    __shared__ TailShared<NT, KEYS> sh;
    const Lane &ln = lanes.l[blockIdx.y];
    const TailSlice sl = slices[blockIdx.x];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int NW = NT / 32;
    constexpr int WPW = KEYS / 32 / NW;  // mask words per warp (a warp owns KEYS / NW consecutive keys)
    static_assert(WPW >= 1 && WPW <= 32 * 2 && (KEYS / 32) % NW == 0, "a lane handles at most two mask words");
    // a rank without a slice only takes part in the cluster's barriers (so does, in the bounds-checked
    // build, a slice that does not lie inside its layer and the key array)
    const bool active = sl.n > 0 &&
                        RSDGC_CHECKED(sl.n <= KEYS && sl.layer >= 0 && sl.layer < status->n_layers && sl.start >= 0 &&
                                          sl.start + sl.n <= layers[sl.layer].K &&
                                          layers[sl.layer].tile_off + sl.start + sl.n <= status->keys_len, status);
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
    // adds this CTA's histogram (bins 0 .. nbins - 1) to the leader's and clears it
    auto push_hist = [&](int nbins) {
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
    };
    // the leader finds the bin in which the running count from the top reaches `need`, publishes it and
    // clears its histogram (level 3 fills the lower 1024 of the 2048 bins; the upper ones are zero)
    auto resolve = [&](unsigned int need, int nbins) {
        tail_find_bin<NT>(sh.hist, (unsigned long long)need, sh.found, sh.scan_tmp);
        if (tid == 0) {
            sh.res[0] = (unsigned int)sh.found[0];
            sh.res[1] = (unsigned int)sh.found[1];
        }
        for (int b = tid; b < nbins; b += NT) sh.hist[b] = 0;
    };

    // ---- what needs only the plan and the ratios: the layer's payload offsets (sums of the k_l of the
    // preceding layers, Eq. 11)
    for (int b = tid; b < kL2Bins; b += NT) sh.hist[b] = 0;
    for (int b = tid; b < KEYS / 32; b += NT) sh.above[b] = sh.equal[b] = 0;
    if (tid == 0) sh.n_cand = 0;
    if (tid < kTailCluster) sh.overflow[tid] = 0;
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
        }
    }
    // every CTA's tables are cleared before anything is added to a leader's: this barrier still runs
    // while the first pass does
    sync_all();
    // ---- the first pass has written the keys (a kernel launched right behind a sibling of this one
    // starts only after that sibling's CTAs have passed this wait, and waits itself before it exits)
    if (!wait_late) grid_dependency_wait();
    grid_dependency_launch_next();
    const LayerDev L = layers[active ? sl.layer : 0];
    // it also left k_l and level 1 (key bits 30..21) of the layer's selection in the layer's state
    int k = 0;
    uint32_t prefix = kTakeNone;   // key bits resolved so far
    unsigned int remaining = 0;    // tiles still to take among the keys that carry the prefix
    const int n4 = (sl.n + 3) >> 2;  // the slice as 128-bit words (the last one padded)
    if (active) {
        const LayerState &st = ln.state[sl.layer];
        k = __ldcg(&st.k);
        prefix = __ldcg(&st.prefix);
        remaining = (unsigned int)__ldcg(&st.remaining);
        // keys: global -> shared memory, and level 2 (bits 20..10 of the keys that carry the level-1
        // prefix) histogrammed on the way
        const uint32_t *kp = ln.keys + L.tile_off + sl.start;  // 16-byte aligned: offsets are multiples of 64 keys
        const int nvec = sl.n >> 2;
        constexpr int kLoadBatch = 8;  // 128-bit loads in flight per thread: the slice arrives in one or two round trips
#pragma unroll 1
        for (int base = 0; base < n4; base += NT * kLoadBatch) {
            uint4 q[kLoadBatch];
#pragma unroll
            for (int u = 0; u < kLoadBatch; ++u) {
                const int i = base + u * NT + tid;
                q[u] = (i < nvec) ? __ldcg(reinterpret_cast<const uint4 *>(kp) + i) : make_uint4(~0u, ~0u, ~0u, ~0u);
                if (i == nvec && (sl.n & 3)) {  // the last, partial word: keys beyond the slice stay all ones,
                    q[u].x = __ldcg(kp + 4 * i);  // which no prefix or threshold matches
                    if ((sl.n & 3) > 1) q[u].y = __ldcg(kp + 4 * i + 1);
                    if ((sl.n & 3) > 2) q[u].z = __ldcg(kp + 4 * i + 2);
                }
            }
#pragma unroll
            for (int u = 0; u < kLoadBatch; ++u) {
                const int i = base + u * NT + tid;
                if (i < n4) {
                    reinterpret_cast<uint4 *>(skeys)[i] = q[u];
                    if ((q[u].x >> kL1Shift) == prefix) atomicAdd(&sh.hist[(q[u].x >> kL2Shift) & (kL2Bins - 1)], 1u);
                    if ((q[u].y >> kL1Shift) == prefix) atomicAdd(&sh.hist[(q[u].y >> kL2Shift) & (kL2Bins - 1)], 1u);
                    if ((q[u].z >> kL1Shift) == prefix) atomicAdd(&sh.hist[(q[u].z >> kL2Shift) & (kL2Bins - 1)], 1u);
                    if ((q[u].w >> kL1Shift) == prefix) atomicAdd(&sh.hist[(q[u].w >> kL2Shift) & (kL2Bins - 1)], 1u);
                }
            }
        }
    }
    if (active && prefix != kTakeNone) push_hist(kL2Bins);
    sync_all();
    if (leader && prefix != kTakeNone) resolve(remaining, kL2Bins);
    sync_all();
    if (active && prefix != kTakeNone) {
        const unsigned int *res = at_leader(&sh.res[0]);
        prefix = (prefix << kL2Bits) | res[0];   // the upper 21 bits of the threshold
        remaining = res[1];
    }

    // ---- one pass: a bit per key above the upper 21 bits, the candidates that share them into the list
    // (a group of 32 keys is one mask word; the warps take four groups at a time, round robin, so a
    // short slice is spread over all of them)
    const int n_groups = (sl.n + 31) >> 5;
    if (active && prefix != kTakeNone) {
#pragma unroll 1
        for (int g0 = warp * 4; g0 < n_groups; g0 += NW * 4) {
            uint32_t key[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = (g0 + u) * 32 + lane;
                key[u] = (i < sl.n) ? skeys[i] : 0xFFFFFFFFu;
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int i = (g0 + u) * 32 + lane;
                const uint32_t hi = key[u] >> kL2Shift;
                const unsigned int ma = __ballot_sync(0xFFFFFFFFu, key[u] != 0xFFFFFFFFu && hi > prefix);
                if (lane == 0 && g0 + u < n_groups) sh.above[g0 + u] = ma;
                if (hi == prefix) {
                    const unsigned int pos = atomicAdd(&sh.n_cand, 1u);
                    if (pos < (unsigned int)kTailCand) sh.cand[pos] = ((key[u] & (kL3Bins - 1)) << 15) | (unsigned int)i;
                }
            }
        }
    }
    __syncthreads();
    const unsigned int n_cand_all = sh.n_cand;  // may exceed the list
    const int n_cand = (int)min(n_cand_all, (unsigned int)kTailCand);
    if (active && prefix != kTakeNone) {
        // level 3 (key bits 9..0) over the candidates; an overflowing list is reported to the leader
        for (int c = tid; c < n_cand; c += NT) atomicAdd(&sh.hist[sh.cand[c] >> 15], 1u);
        if (tid == 0 && n_cand_all > (unsigned int)kTailCand) at_leader(&sh.overflow[0])[sl.rank] = 1u;
        push_hist(kL3Bins);
    }
    sync_all();
    if (leader && prefix != kTakeNone) {
        unsigned int any = 0;
        for (int r = 0; r < sl.n_ranks; ++r) any |= sh.overflow[r];
        if (any) {  // some list is incomplete: its histogram is worthless
            for (int b = tid; b < kL3Bins; b += NT) sh.hist[b] = 0;
            if (tid == 0) sh.res[2] = 1u;
        } else {
            resolve(remaining, kL3Bins);
            if (tid == 0) sh.res[2] = 0u;
        }
    }
    sync_all();
    bool fallback = false;
    uint32_t T = kTakeNone;  // the threshold key
    int e = 0;               // keys equal to T that are taken, lowest tile index first
    if (active && prefix != kTakeNone) {
        const unsigned int *res = at_leader(&sh.res[0]);
        fallback = res[2] != 0u;
        if (!fallback) {
            T = (prefix << kL3Bits) | res[0];
            e = (int)res[1];
        }
    }
    // ---- the layer's extra pass when a candidate list overflowed: level 3 over all the keys
    if (fallback) {
#pragma unroll 1
        for (int base = 0; base < n4; base += NT * 2) {
            uint4 q[2];
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                const int i = base + u * NT + tid;
                q[u] = (i < n4) ? reinterpret_cast<const uint4 *>(skeys)[i] : make_uint4(~0u, ~0u, ~0u, ~0u);
            }
#pragma unroll
            for (int u = 0; u < 2; ++u) {
                if ((q[u].x >> kL2Shift) == prefix) atomicAdd(&sh.hist[q[u].x & (kL3Bins - 1)], 1u);
                if ((q[u].y >> kL2Shift) == prefix) atomicAdd(&sh.hist[q[u].y & (kL3Bins - 1)], 1u);
                if ((q[u].z >> kL2Shift) == prefix) atomicAdd(&sh.hist[q[u].z & (kL3Bins - 1)], 1u);
                if ((q[u].w >> kL2Shift) == prefix) atomicAdd(&sh.hist[q[u].w & (kL3Bins - 1)], 1u);
            }
        }
        push_hist(kL3Bins);
    }
    sync_all();
    if (leader && fallback) resolve(remaining, kL3Bins);
    sync_all();
    if (fallback) {
        const unsigned int *res = at_leader(&sh.res[0]);
        T = (prefix << kL3Bits) | res[0];
        e = (int)res[1];
    }

    // ---- the bit masks of the keys above and equal to the full threshold
    if (active && T != kTakeNone) {
        if (!fallback) {  // only the candidates can still change a bit
            const uint32_t t_low = T & (kL3Bins - 1);
            for (int c = tid; c < n_cand; c += NT) {
                const unsigned int v = sh.cand[c], low = v >> 15, i = v & 0x7FFFu;
                if (low > t_low) atomicOr(&sh.above[i >> 5], 1u << (i & 31));
                else if (low == t_low) atomicOr(&sh.equal[i >> 5], 1u << (i & 31));
            }
        } else {
#pragma unroll 1
            for (int g0 = warp * 4; g0 < n_groups; g0 += NW * 4) {
                uint32_t key[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int i = (g0 + u) * 32 + lane;
                    key[u] = (i < sl.n) ? skeys[i] : 0xFFFFFFFFu;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const unsigned int ma = __ballot_sync(0xFFFFFFFFu, key[u] != 0xFFFFFFFFu && key[u] > T);
                    const unsigned int me = __ballot_sync(0xFFFFFFFFu, key[u] == T);
                    if (lane == 0 && g0 + u < n_groups) {
                        sh.above[g0 + u] = ma;
                        sh.equal[g0 + u] = me;
                    }
                }
            }
        }
    }
    __syncthreads();

    // ---- per warp, per CTA, per layer: how many keys lie above T and how many equal it.  A lane holds
    // the mask words lane * WPL .. of its warp's range.
    constexpr int WPL = (WPW + 31) / 32;  // mask words per lane (1 or 2)
    unsigned int ab[WPL], eq[WPL];
    unsigned int my_gt = 0, my_eq = 0;
#pragma unroll
    for (int j = 0; j < WPL; ++j) {
        const int wl = lane * WPL + j;  // word within the warp's range
        ab[j] = (wl < WPW) ? sh.above[warp * WPW + wl] : 0u;
        eq[j] = (wl < WPW) ? sh.equal[warp * WPW + wl] : 0u;
        my_gt += __popc(ab[j]);
        my_eq += __popc(eq[j]);
    }
    // exclusive prefix over the lanes of the warp, and the warp's totals
    unsigned int pg = my_gt, pe = my_eq;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const unsigned int yg = __shfl_up_sync(0xFFFFFFFFu, pg, d), ye = __shfl_up_sync(0xFFFFFFFFu, pe, d);
        if (lane >= d) {
            pg += yg;
            pe += ye;
        }
    }
    if (lane == 31) {
        sh.warp_cnt[warp][0] = pg;
        sh.warp_cnt[warp][1] = pe;
    }
    pg -= my_gt;
    pe -= my_eq;
    __syncthreads();
    // exclusive prefix of the warps' counts (warp 0, by shuffles); the CTA's totals end up in entry NW
    if (warp == 0) {
        unsigned int a = (lane < NW) ? sh.warp_cnt[lane][0] : 0u, b2 = (lane < NW) ? sh.warp_cnt[lane][1] : 0u;
        const unsigned int a0 = a, b0 = b2;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned int ya = __shfl_up_sync(0xFFFFFFFFu, a, d), yb = __shfl_up_sync(0xFFFFFFFFu, b2, d);
            if (lane >= d) {
                a += ya;
                b2 += yb;
            }
        }
        if (lane < NW) {
            sh.warp_pre[lane][0] = a - a0;
            sh.warp_pre[lane][1] = b2 - b0;
        }
        if (lane == NW - 1) {
            sh.warp_pre[NW][0] = a;
            sh.warp_pre[NW][1] = b2;
        }
    }
    __syncthreads();
    const int cta_gt = (int)sh.warp_pre[NW][0], cta_eq = (int)sh.warp_pre[NW][1];
    if (active && tid == 0) {
        unsigned int *c = at_leader(&sh.cnt[0][0]);
        c[2 * sl.rank] = (unsigned int)cta_gt;
        c[2 * sl.rank + 1] = (unsigned int)cta_eq;
    }
    sync_all();
    int lay_gt0 = 0, lay_eq0 = 0;  // keys above / equal in the slices of the layer before this one (< K_l < 2^31)
    if (active) {
        const unsigned int *c = at_leader(&sh.cnt[0][0]);
        for (int r = 0; r < sl.rank; ++r) {
            lay_gt0 += (int)c[2 * r];
            lay_eq0 += (int)c[2 * r + 1];
        }
    }
    sync_all();  // nothing of another CTA's shared memory is touched from here on
    if (!active) {
        if (wait_late) grid_dependency_wait();
        return;
    }

    const long long idx_off = sh.idx_off, val_off = sh.val_off;
    if (leader && tid == 0 && sl.layer == n_layers - 1) {
        const long long need_i = idx_off + k, need_v = val_off + (long long)k * L.slot;
        status->idx_needed = need_i;
        status->val_needed = need_v;
        if (need_i > idx_cap || need_v > val_cap) atomicOr(&status->flags, RSDGC_STATUS_PAYLOAD_OVERFLOW);
    }
    if (T == kTakeNone) {
        if (wait_late) grid_dependency_wait();
        return;
    }

    // ---- payload indices: a tile is kept if its key is above T, or equals T with fewer than e equal
    // keys before it in the layer; its slot is the number of kept tiles before it.  Only the set bits
    // are visited.
    int32_t *__restrict__ idx = ln.idx;
    // kept tiles of this CTA: payload slots [s_first, s_first + n_kept) of the call; their indices also
    // stay in shared memory (the keys are no longer needed), where the gather below finds them
    const long long s_first = idx_off + lay_gt0 + min(lay_eq0, e);
    const long long n_kept = cta_gt + (min(lay_eq0 + cta_eq, e) - min(lay_eq0, e));
    int32_t *sidx = reinterpret_cast<int32_t *>(skeys);
    {
        int g_rank = lay_gt0 + (int)sh.warp_pre[warp][0] + (int)pg, e_rank = lay_eq0 + (int)sh.warp_pre[warp][1] + (int)pe;
#pragma unroll
        for (int j = 0; j < WPL; ++j) {
            const int tile0 = sl.start + (warp * WPW + lane * WPL + j) * 32;
            unsigned int todo = ab[j] | eq[j];
            while (todo) {
                const int bit = __ffs((int)todo) - 1;
                todo &= todo - 1;
                const unsigned int below = (1u << bit) - 1u;
                const int gr = g_rank + __popc(ab[j] & below), er = e_rank + __popc(eq[j] & below);
                if (((ab[j] >> bit) & 1u) || er < e) {
                    const long long s = idx_off + (gr + min(er, e));
                    sidx[s - s_first] = tile0 + bit;
                    if (s < idx_cap) idx[s] = tile0 + bit;
                }
            }
            g_rank += __popc(ab[j]);
            e_rank += __popc(eq[j]);
        }
    }
    __syncthreads();  // the gather below reads the indices this CTA has just left in shared memory

    // ---- gather: the values of the kept tiles leave the accumulator (Eq. 12)
    const int slot = L.slot;
    // positions relative to the layer's start in the arena / in the payload fit 32 bits (a layer has
    // fewer than 2^31 elements)
    float *__restrict__ resid_l = ln.resid + L.elem_off;
    float *__restrict__ val_l = reinterpret_cast<float *>(ln.val) + val_off;
    __nv_bfloat16 *__restrict__ val16_l = reinterpret_cast<__nv_bfloat16 *>(ln.val) + val_off;
    constexpr int kBatch = 4;
    const long long n_vals = n_kept * slot;
    const int cols = (int)L.cols;
#pragma unroll 1
    for (long long j0 = 0; j0 < n_vals; j0 += (long long)NT * kBatch) {
        int ga[kBatch], vo[kBatch];
        float xv[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const long long j = j0 + u * NT + tid;
            ga[u] = -1;
            vo[u] = -1;
            if (j < n_vals) {
                int q, el;
                divmod_small((int)j, slot, &q, &el);  // n_vals <= the layer's elements < 2^31
                const long long s = s_first + q;
                // tiles that do not fit the payload buffers are not sent and stay in the accumulator
                if (s < idx_cap && val_off + (s - idx_off + 1) * slot <= val_cap) {
                    const int tile = sidx[q];
                    const int tr = tile / L.TC, tc = tile - tr * L.TC;
                    int a, b;
                    divmod_small(el, L.nw, &a, &b);
                    const int i = tr * L.nh + a, jj = tc * L.nw + b;
                    if (i < (int)L.rows && jj < cols) ga[u] = i * cols + jj;
                    vo[u] = (int)(s - idx_off) * slot + el;
                    if (!RSDGC_CHECKED(tile >= 0 && tile < L.K && L.elem_off + ga[u] < status->arena_elems, status))
                        ga[u] = -1, vo[u] = -1;
                }
            }
        }
        if (BF16VAL) {  // q = bfloat16(v) is sent, v - q stays (exact in binary32)
#pragma unroll
            for (int u = 0; u < kBatch; ++u) xv[u] = (ga[u] >= 0) ? resid_l[ga[u]] : 0.0f;
#pragma unroll
            for (int u = 0; u < kBatch; ++u) {
                const __nv_bfloat16 q = __float2bfloat16_rn(xv[u]);
                if (ga[u] >= 0) resid_l[ga[u]] = __fsub_rn(xv[u], __bfloat162float(q));
                if (vo[u] >= 0) val16_l[vo[u]] = q;
            }
        } else {  // read v and leave +0 in one exchange (see k_gather)
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                xv[u] = (ga[u] >= 0) ? __uint_as_float(atomicExch(reinterpret_cast<unsigned int *>(resid_l) + ga[u], 0u))
                                     : 0.0f;
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                if (vo[u] >= 0) val_l[vo[u]] = xv[u];
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
