// Kernels of rsdgc_compress() after the accumulate+NSI pass: two refinement passes of the
// per-layer radix selection (the second leaves the per-chunk counts and their scan), the payload
// indices and the gather.
//
// Ordering between CTAs comes only from kernel boundaries and from "last arriver finishes
// the job" tickets (an atomic counter per layer and phase); no thread ever waits on another
// CTA.  The per-layer histograms and tickets are reset by the CTA that consumes them, so the
// plan's tables are all-zero again when a compress call has run to completion.

#include <cuda_bf16.h>

#include <algorithm>

#include "device_utils.cuh"

namespace rsdgc {

// ------------------------------------------------------------------------------------------
// K2: level 2 of the radix selection, a histogram pass over the keys
// ------------------------------------------------------------------------------------------

constexpr int kKeyVecBatch = 8;  // 128-bit key loads in flight per thread in the key passes
constexpr int kRefineCtasPerSm = 6;  // resident CTAs per SM of k_refine2 (40 registers, 8 KB of shared memory)

struct RefineShared {
    unsigned int hist[kL2Bins];
    unsigned long long scan_tmp[kThreads / 32];
    unsigned long long found[2];
    int is_last;
};

// Adds the CTA's histogram of `layer` (it covers n_done chunks of the layer) to the layer's
// global one and clears it; the CTA that accounts for the layer's last chunk finds the bin the
// threshold falls into and extends the layer's prefix to 21 bits.
__device__ __forceinline__ void refine2_flush(RefineShared &sh, const Lane &ln, const LayerDev *__restrict__ layers,
                                              int layer, int n_done)
{
    const int tid = threadIdx.x;
    LayerState &st = ln.state[layer];
    unsigned int *gh = ln.hist + (size_t)layer * kHistStride;
    __syncthreads();
    for (int b = tid; b < kL2Bins; b += kThreads) {
        const unsigned int n = sh.hist[b];
        if (n) {
            atomicAdd(gh + b, n);
            sh.hist[b] = 0;
        }
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned int t = atomicAdd(&st.ticket[1], (unsigned int)n_done);
        sh.is_last = (t + (unsigned int)n_done == (unsigned int)layers[layer].n_chunks);
    }
    __syncthreads();
    if (!sh.is_last) return;
    __threadfence();
    {
        unsigned int h[kL2Bins / kThreads];
#pragma unroll
        for (int j = 0; j < kL2Bins / kThreads; ++j) h[j] = __ldcg(gh + j * kThreads + tid);
#pragma unroll
        for (int j = 0; j < kL2Bins / kThreads; ++j) {
            sh.hist[j * kThreads + tid] = h[j];
            gh[j * kThreads + tid] = 0;
        }
    }
    __syncthreads();
    const uint32_t prefix = st.prefix;
    const int remaining = st.remaining;
    if (prefix != kTakeNone)
        find_bin_from_top<kL2Bins>(sh.hist, (unsigned long long)remaining, sh.found, sh.scan_tmp);
    if (tid == 0) {
        st.ticket[1] = 0;
        if (prefix != kTakeNone) {
            st.prefix = (prefix << kL2Bits) | (uint32_t)sh.found[0];
            st.remaining = (int32_t)sh.found[1];
        }
    }
    __syncthreads();
    for (int b = tid; b < kL2Bins; b += kThreads) sh.hist[b] = 0;  // it held the layer's totals
    __syncthreads();
}

// Among the keys whose bits 30..21 equal the layer's prefix (level 1, resolved by the first pass),
// histogram bits 20..10.  Every CTA takes a contiguous range of the key chunks (one chunk when the
// grid is as large as the chunk list) and keeps one shared-memory histogram per layer it passes through.
__global__ void __launch_bounds__(kThreads, kRefineCtasPerSm)
k_refine2(const __grid_constant__ LaneTable lanes, const LayerDev *__restrict__ layers,
          const Chunk *__restrict__ chunks, int n_chunks_all, StatusDev *status)
{
    __shared__ RefineShared sh;
    const Lane &ln = lanes.l[blockIdx.y];
    const uint32_t *__restrict__ keys = ln.keys;
    const int tid = threadIdx.x;
    const int chunk_begin = (int)((long long)blockIdx.x * n_chunks_all / gridDim.x);
    const int chunk_end = (int)((long long)(blockIdx.x + 1) * n_chunks_all / gridDim.x);
    for (int b = tid; b < kL2Bins; b += kThreads) sh.hist[b] = 0;
    grid_dependency_wait();
    grid_dependency_launch_next();
    __syncthreads();
    int cur_layer = -1, n_done = 0;
    uint32_t prefix = kTakeNone;
    auto tally = [&](uint32_t key) {
        if ((key >> kL1Shift) == prefix) atomicAdd(&sh.hist[(key >> kL2Shift) & (kL2Bins - 1)], 1u);
    };
    for (int chunk_id = chunk_begin; chunk_id < chunk_end; ++chunk_id) {
        const Chunk c = chunks[chunk_id];
        if (c.layer != cur_layer) {
            if (n_done) refine2_flush(sh, ln, layers, cur_layer, n_done);
            cur_layer = c.layer;
            n_done = 0;
            // not yet extended by this pass: this CTA still owes the layer a chunk
            prefix = ln.state[c.layer].prefix;
        }
        ++n_done;
        if (prefix == kTakeNone) continue;
        if (!RSDGC_CHECKED(chunk_id < status->n_chunks && c.layer < status->n_layers && c.start >= 0 && c.n >= 0 &&
                               layers[c.layer].tile_off + c.start + c.n <= status->keys_len, status))
            continue;
        const uint32_t *kp = keys + layers[c.layer].tile_off + c.start;
        const int nvec = c.n >> 2;
        for (int base = 0; base < nvec; base += kThreads * kKeyVecBatch) {
            uint4 q[kKeyVecBatch];  // all loads of a batch are issued before any is consumed
#pragma unroll
            for (int u = 0; u < kKeyVecBatch; ++u) {
                const int i = base + u * kThreads + tid;
                q[u] = (i < nvec) ? __ldg(reinterpret_cast<const uint4 *>(kp) + i) : make_uint4(~0u, ~0u, ~0u, ~0u);
            }
#pragma unroll
            for (int u = 0; u < kKeyVecBatch; ++u) {  // the all-ones filler never matches a prefix
                tally(q[u].x);
                tally(q[u].y);
                tally(q[u].z);
                tally(q[u].w);
            }
        }
        const int i = (nvec << 2) + tid;
        if (i < c.n) tally(kp[i]);
    }
    if (n_done) refine2_flush(sh, ln, layers, cur_layer, n_done);
}

// ------------------------------------------------------------------------------------------
// K3: level 3 of the selection AND everything the index pass needs, in one pass over the keys.
// When this pass runs, the upper 21 bits of a layer's threshold are known.  A key above them is kept
// whatever level 3 finds, a key below them is not; only the keys that share them ("in the bin") depend
// on the low 10 bits.  Per chunk the pass therefore leaves
//   * one code byte per four keys (bit c: key c above the bin, bit 4 + c: key c in the bin),
//   * the number of keys above the bin,
//   * the suffix sums of the chunk's histogram of the low 10 bits of its in-bin keys
//     (sfx[b] = in-bin keys of the chunk whose low bits are >= b),
// and adds the chunk's histogram to the layer's.  The CTA that accounts for a layer's last chunk
// resolves level 3 (T and e), reads two suffix sums per chunk to get every chunk's count of keys
// above T and equal to T, turns them into exclusive bases and computes the layer's payload offsets:
// no separate counting pass over the keys.
// ------------------------------------------------------------------------------------------

struct Refine3Shared {
    unsigned int hist[kL3Bins];   // level-3 histogram of the current layer over the chunks this CTA took
    unsigned int chist[kL3Bins];  // ... of the current chunk
    unsigned long long scan_tmp[kThreads / 32];
    unsigned long long found[2];
    unsigned int red[kThreads / 32];
    int is_last;
};

// Layer `layer` is complete in this CTA (n_done of its chunks): add to the layer's global histogram;
// the last CTA to do so finishes the layer.
__device__ __forceinline__ void refine3_flush(Refine3Shared &sh, const Lane &ln, const LayerDev *__restrict__ layers,
                                              int layer, int n_done, int n_layers, long long idx_cap,
                                              long long val_cap, StatusDev *status)
{
    const int tid = threadIdx.x;
    LayerState &st = ln.state[layer];
    const LayerDev &L = layers[layer];
    unsigned int *gh = ln.hist + (size_t)layer * kHistStride;
    __syncthreads();
    for (int b = tid; b < kL3Bins; b += kThreads) {
        const unsigned int n = sh.hist[b];
        if (n) {
            atomicAdd(gh + b, n);
            sh.hist[b] = 0;
        }
    }
    __threadfence();  // also orders this CTA's per-chunk counts and suffix sums before its ticket
    __syncthreads();
    if (tid == 0) {
        const unsigned int t = atomicAdd(&st.ticket[2], (unsigned int)n_done);
        sh.is_last = (t + (unsigned int)n_done == (unsigned int)L.n_chunks);
    }
    __syncthreads();
    if (!sh.is_last) return;
    __threadfence();
    {
        unsigned int h[kL3Bins / kThreads];
#pragma unroll
        for (int j = 0; j < kL3Bins / kThreads; ++j) h[j] = __ldcg(gh + j * kThreads + tid);
#pragma unroll
        for (int j = 0; j < kL3Bins / kThreads; ++j) {
            sh.hist[j * kThreads + tid] = h[j];
            gh[j * kThreads + tid] = 0;
        }
    }
    __syncthreads();
    const uint32_t prefix = st.prefix;
    const int remaining = st.remaining;
    int bin = 0;
    if (prefix != kTakeNone) {
        find_bin_from_top<kL3Bins>(sh.hist, (unsigned long long)remaining, sh.found, sh.scan_tmp);
        bin = (int)sh.found[0];
    }
    if (tid == 0) {
        st.ticket[2] = 0;
        st.T = prefix != kTakeNone ? ((prefix << kL3Bits) | (uint32_t)bin) : kTakeNone;
        st.e = prefix != kTakeNone ? (int32_t)sh.found[1] : 0;
    }
    __syncthreads();
    for (int b = tid; b < kL3Bins; b += kThreads) sh.hist[b] = 0;  // it held the layer's totals

    // per chunk: keys above T = keys above the bin + in-bin keys with low bits > bin; equal = low bits == bin;
    // then the exclusive scan over the layer's chunks, in chunk order
    uint2 *cc = ln.chunk_cnt + L.first_chunk;
    const unsigned short *sfx = ln.chunk_sfx + (size_t)L.first_chunk * kL3Bins;
    unsigned long long carry = 0;  // above in the low 32 bits, equal in the high 32 bits
    for (int base = 0; base < L.n_chunks; base += kThreads) {
        const int i = base + tid;
        unsigned long long x = 0;
        if (i < L.n_chunks && prefix != kTakeNone) {
            const uint2 a = __ldcg(cc + i);  // (keys above the 21 bits, keys sharing them)
            unsigned int ge = 0, gt = 0;
            if (a.y) {
                ge = __ldcg(sfx + (size_t)i * kL3Bins + bin);
                if (bin + 1 < kL3Bins) gt = __ldcg(sfx + (size_t)i * kL3Bins + bin + 1);
            }
            x = ((unsigned long long)(ge - gt) << 32) | (unsigned long long)(a.x + gt);
        }
        unsigned long long total;
        const unsigned long long ex = block_exclusive_scan<unsigned long long>(x, sh.scan_tmp, &total) + carry;
        if (i < L.n_chunks) cc[i] = make_uint2((unsigned int)(ex & 0xFFFFFFFFull), (unsigned int)(ex >> 32));
        carry += total;
    }

    // payload offsets of this layer: sums over the preceding layers of k and k * slot
    long long si = 0, sv = 0;
    for (int l = tid; l < layer; l += kThreads) {
        const long long k = ln.state[l].k;
        si += k;
        sv += k * layers[l].slot;
    }
    unsigned long long tot_i, tot_v;
    (void)block_exclusive_scan<unsigned long long>((unsigned long long)si, sh.scan_tmp, &tot_i);
    (void)block_exclusive_scan<unsigned long long>((unsigned long long)sv, sh.scan_tmp, &tot_v);
    if (tid == 0) {
        st.idx_off = (long long)tot_i;
        st.val_off = (long long)tot_v;
        if (layer == n_layers - 1) {
            const long long need_i = (long long)tot_i + st.k;
            const long long need_v = (long long)tot_v + (long long)st.k * L.slot;
            status->idx_needed = need_i;
            status->val_needed = need_v;
            if (need_i > idx_cap || need_v > val_cap) atomicOr(&status->flags, RSDGC_STATUS_PAYLOAD_OVERFLOW);
        }
    }
    __syncthreads();
}

constexpr int kRefine3CtasPerSm = 4;  // 64 registers per thread

__global__ void __launch_bounds__(kThreads, kRefine3CtasPerSm)
k_refine3_count(const __grid_constant__ LaneTable lanes, const LayerDev *__restrict__ layers,
                const Chunk *__restrict__ chunks, int n_chunks_all, int n_layers, long long idx_cap, long long val_cap,
                StatusDev *status)
{
    __shared__ Refine3Shared sh;
    const Lane &ln = lanes.l[blockIdx.y];
    const uint32_t *__restrict__ keys = ln.keys;
    unsigned char *__restrict__ codes = ln.codes;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int chunk_begin = (int)((long long)blockIdx.x * n_chunks_all / gridDim.x);
    const int chunk_end = (int)((long long)(blockIdx.x + 1) * n_chunks_all / gridDim.x);
    for (int b = tid; b < kL3Bins; b += kThreads) sh.hist[b] = sh.chist[b] = 0;
    grid_dependency_wait();
    grid_dependency_launch_next();
    __syncthreads();
    int cur_layer = -1, n_done = 0;
    uint32_t prefix = kTakeNone;
    // (the CTA walks its range backwards: the level-2 pass walked it forwards, so what that pass read last
    // - about half of the keys when they exceed the L2 - is read first here and still found there)
    for (int chunk_id = chunk_end - 1; chunk_id >= chunk_begin; --chunk_id) {
        const Chunk c = chunks[chunk_id];
        if (c.layer != cur_layer) {
            if (n_done) refine3_flush(sh, ln, layers, cur_layer, n_done, n_layers, idx_cap, val_cap, status);
            cur_layer = c.layer;
            n_done = 0;
            prefix = ln.state[c.layer].prefix;  // the upper 21 bits, left by the level-2 pass
        }
        ++n_done;
        if (prefix == kTakeNone) continue;  // nothing of this layer is kept: no code, no count is read
        const LayerDev &L = layers[c.layer];
        if (!RSDGC_CHECKED(chunk_id < status->n_chunks && c.layer < status->n_layers && c.start >= 0 && c.n >= 0 &&
                               L.tile_off + c.start + c.n <= status->keys_len, status))
            continue;
        const uint32_t *kp = keys + L.tile_off + c.start;
        unsigned char *cp = codes + ((L.tile_off + c.start) >> 2);
        const int nvec = c.n >> 2;
        // keys in [lo_key, hi_key) share the threshold's upper 21 bits, keys >= hi_key lie above them
        // (prefix < 2^21, so hi_key <= 2^31 does not wrap)
        const uint32_t lo_key = prefix << kL3Bits, hi_key = lo_key + (uint32_t)kL3Bins;
        unsigned int above = 0, sharing = 0;
        auto code_of = [&](uint32_t k0, uint32_t k1, uint32_t k2, uint32_t k3) {
            unsigned int code = (unsigned int)(k0 >= hi_key) | ((unsigned int)(k1 >= hi_key) << 1) |
                                ((unsigned int)(k2 >= hi_key) << 2) | ((unsigned int)(k3 >= hi_key) << 3);
            const bool s0 = (k0 - lo_key) < (uint32_t)kL3Bins, s1 = (k1 - lo_key) < (uint32_t)kL3Bins;
            const bool s2 = (k2 - lo_key) < (uint32_t)kL3Bins, s3 = (k3 - lo_key) < (uint32_t)kL3Bins;
            if (s0 | s1 | s2 | s3) {  // rare: a layer has few keys that close to its threshold
                if (s0) atomicAdd(&sh.chist[k0 & (kL3Bins - 1)], 1u);
                if (s1) atomicAdd(&sh.chist[k1 & (kL3Bins - 1)], 1u);
                if (s2) atomicAdd(&sh.chist[k2 & (kL3Bins - 1)], 1u);
                if (s3) atomicAdd(&sh.chist[k3 & (kL3Bins - 1)], 1u);
                code |= ((unsigned int)s0 << 4) | ((unsigned int)s1 << 5) | ((unsigned int)s2 << 6) | ((unsigned int)s3 << 7);
                sharing += (unsigned int)s0 + (unsigned int)s1 + (unsigned int)s2 + (unsigned int)s3;
            }
            above += __popc(code & 0x0Fu);
            return (unsigned char)code;
        };
        for (int base = 0; base < nvec; base += kThreads * kKeyVecBatch) {
            uint4 q[kKeyVecBatch];  // all loads of a batch are issued before any is consumed
#pragma unroll
            for (int u = 0; u < kKeyVecBatch; ++u) {
                const int i = base + u * kThreads + tid;
                q[u] = (i < nvec) ? __ldg(reinterpret_cast<const uint4 *>(kp) + i) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < kKeyVecBatch; ++u) {
                const int i = base + u * kThreads + tid;
                if (i < nvec) cp[i] = code_of(q[u].x, q[u].y, q[u].z, q[u].w);
            }
        }
        if ((c.n & 3) && tid == 0) {  // the last, partial word of the chunk; absent keys get no flag
            unsigned int code = 0;
            for (int j = 0; j < (c.n & 3); ++j) {
                const uint32_t k = kp[4 * nvec + j];
                if (k >= hi_key) {
                    code |= 1u << j;
                    ++above;
                } else if (k - lo_key < (uint32_t)kL3Bins) {
                    code |= 16u << j;
                    atomicAdd(&sh.chist[k & (kL3Bins - 1)], 1u);
                    ++sharing;
                }
            }
            cp[nvec] = (unsigned char)code;
        }
        // ---- the chunk's count of keys above the bin; when it has keys that share the 21 bits, the suffix
        // sums of its histogram, and the histogram into the layer's
        const int any_sharing = __syncthreads_or((int)sharing);  // also: the chunk's histogram is complete
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) above += __shfl_xor_sync(0xFFFFFFFFu, above, d);
        if (lane == 0) sh.red[warp] = above;
        unsigned long long total = 0;
        if (any_sharing) {
            constexpr int PER = kL3Bins / kThreads;  // thread t owns bins [t * PER, (t + 1) * PER)
            unsigned int h[PER];
            unsigned long long mine = 0;
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                h[j] = sh.chist[tid * PER + j];
                mine += h[j];
            }
            unsigned long long below = block_exclusive_scan<unsigned long long>(mine, sh.scan_tmp, &total);
            unsigned short *out = ln.chunk_sfx + (size_t)chunk_id * kL3Bins + tid * PER;
#pragma unroll
            for (int j = 0; j < PER; ++j) {
                out[j] = (unsigned short)(total - below);  // sharing keys with low bits >= this bin (<= 16384)
                below += h[j];
                if (h[j]) {
                    sh.hist[tid * PER + j] += h[j];
                    sh.chist[tid * PER + j] = 0;
                }
            }
        }
        __syncthreads();
        if (tid == 0) {
            unsigned int a = 0;
            for (int w = 0; w < kThreads / 32; ++w) a += sh.red[w];
            ln.chunk_cnt[chunk_id] = make_uint2(a, (unsigned int)total);  // (keys above the 21 bits, keys sharing them)
        }
    }
    if (n_done) refine3_flush(sh, ln, layers, cur_layer, n_done, n_layers, idx_cap, val_cap, status);
}

// ------------------------------------------------------------------------------------------
// K4: mark.  A tile is kept if its key is above T, or equals T and fewer than e equal keys
// precede it in the layer.  Its payload slot is its rank among the kept tiles of the layer
// (ascending tile index).  This kernel writes the tile indices of the payload; the values are
// moved by k_gather, whose work is spread evenly whatever the spatial pattern of the kept tiles.
// ------------------------------------------------------------------------------------------

constexpr int kKeysPerThread = kChunkKeys / kThreads;  // 64 consecutive keys per thread

struct MarkShared {
    unsigned long long scan_tmp[kThreads / 32];
};

__global__ void __launch_bounds__(kThreads)
k_mark(const __grid_constant__ LaneTable lanes, const LayerDev *__restrict__ layers,
       const Chunk *__restrict__ chunks, long long idx_cap, StatusDev *status)
{
    __shared__ MarkShared sh;
    const Lane &ln = lanes.l[blockIdx.y];
    const unsigned char *__restrict__ codes = ln.codes;
    const LayerState *__restrict__ state = ln.state;
    const uint2 *__restrict__ chunk_cnt = ln.chunk_cnt;
    const uint32_t *__restrict__ keys = ln.keys;
    int32_t *__restrict__ idx = ln.idx;
    const Chunk c = chunks[blockIdx.x];
    const int tid = threadIdx.x;
    grid_dependency_wait();
    grid_dependency_launch_next();
    const LayerState st = state[c.layer];
    if (st.k == 0) return;
    if (!RSDGC_CHECKED((int)blockIdx.x < status->n_chunks && c.layer < status->n_layers &&
                           layers[c.layer].tile_off + c.start + c.n <= status->keys_len, status))
        return;
    const uint2 base = chunk_cnt[blockIdx.x];  // tiles above T / equal to T in earlier chunks
    // equal keys of this chunk that are still taken: those with layer-wide equal-rank < e
    const long long eq_room = max(0ll, (long long)st.e - (long long)base.y);

    // ---- the code bytes the level-3 pass left: thread t owns keys [64 t, 64 t + 64) = 16 bytes; bytes
    // beyond the chunk's last word belong to whatever follows in the array and are masked off
    const unsigned char *cp = codes + ((layers[c.layer].tile_off + c.start) >> 2);
    const int nvec_all = (c.n + 3) >> 2;
    unsigned int w[4] = {0u, 0u, 0u, 0u};
    if (tid * 16 < nvec_all) {
        const uint4 cw = __ldg(reinterpret_cast<const uint4 *>(cp) + tid);
        w[0] = cw.x, w[1] = cw.y, w[2] = cw.z, w[3] = cw.w;
        const int valid = nvec_all - tid * 16;  // code bytes of this thread that are inside the chunk
        if (valid < 16) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int vb = valid - 4 * j;  // valid bytes of word j
                if (vb <= 0) w[j] = 0;
                else if (vb < 4) w[j] &= (1u << (8 * vb)) - 1u;
            }
        }
    }
    // 64-bit masks in key order: bit 4 * byte + c of `above` (`inbin`) is set when key c of that
    // code byte lies above (shares) the upper 21 bits of the threshold
    unsigned long long above = 0, inbin = 0, equal = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const unsigned int lo = w[j] & 0x0F0F0F0Fu, hi = (w[j] >> 4) & 0x0F0F0F0Fu;
        const unsigned int a16 = (lo & 0xFu) | ((lo >> 4) & 0xF0u) | ((lo >> 8) & 0xF00u) | ((lo >> 12) & 0xF000u);
        const unsigned int e16 = (hi & 0xFu) | ((hi >> 4) & 0xF0u) | ((hi >> 8) & 0xF00u) | ((hi >> 12) & 0xF000u);
        above |= (unsigned long long)a16 << (16 * j);
        inbin |= (unsigned long long)e16 << (16 * j);
    }
    // the few keys in the bin are looked at themselves: their low 10 bits against the threshold's
    {
        const uint32_t t_low = st.T & (kL3Bins - 1);
        const uint32_t *kp = keys + layers[c.layer].tile_off + c.start + tid * kKeysPerThread;
        while (inbin) {
            const int p = __ffsll((long long)inbin) - 1;
            inbin &= inbin - 1;
            const uint32_t low = __ldg(kp + p) & (kL3Bins - 1);
            if (low > t_low) above |= 1ull << p;
            else if (low == t_low) equal |= 1ull << p;
        }
    }
    const unsigned int gt = __popcll(above), eq = __popcll(equal);
    unsigned long long total;
    const unsigned long long ex =
        block_exclusive_scan<unsigned long long>(((unsigned long long)eq << 32) | gt, sh.scan_tmp, &total);
    const unsigned int gt_before = (unsigned int)(ex & 0xFFFFFFFFull), eq_before = (unsigned int)(ex >> 32);
    // equal keys from this thread on are no longer taken once eq_room is used up
    unsigned long long todo = above | (((long long)eq_before < eq_room) ? equal : 0ull);
    if (todo == 0) return;
    // payload position of this chunk's first kept tile
    const long long slot0 = st.idx_off + (long long)base.x + min((long long)base.y, (long long)st.e);
    const int p0 = c.start + tid * kKeysPerThread;
    // only the set bits are visited: a warp takes as many rounds as its busiest lane has kept tiles
    while (todo) {
        const int p = __ffsll((long long)todo) - 1;
        todo &= todo - 1;
        const unsigned long long below = (1ull << p) - 1ull;
        const long long g_rank = (long long)gt_before + __popcll(above & below);
        const long long e_rank = (long long)eq_before + __popcll(equal & below);
        long long s;
        if ((above >> p) & 1ull) s = slot0 + g_rank + min(e_rank, eq_room);
        else if (e_rank < eq_room) s = slot0 + g_rank + e_rank;
        else continue;
        if (s < idx_cap) idx[s] = p0 + p;
    }
}

// ------------------------------------------------------------------------------------------
// K5: gather.  Payload value j of the whole call belongs to layer l (val_off_l <= j <
// val_off_l + k_l * slot_l), payload slot s = (j - val_off_l) / slot_l, element el of the tile
// idx[idx_off_l + s].  The value is moved from the residual to val and the residual entry
// becomes +0 (Eq. 12: what is sent leaves the accumulator); with 16-bit payload values
// q = bfloat16(v) is sent and v - q stays.  Grid-stride over blocks of consecutive payload values
// (so the work is even whatever the spatial pattern of the kept tiles, and the payload stores are
// contiguous) with kCopyBatch independent entries in flight per thread.
//
// "Read v, leave +0" is ONE atomic exchange per element, executed where the line lives (L2): a
// plain load followed by a store of 0 to the same sector is 3x slower on this memory system (the
// store meets the sector while its fill is still in flight) and fetches twice the bytes from DRAM
// (127 against 84 bytes per 12-byte row segment of a 3x3 tile).  No two threads touch the same
// element, so the exchange is only a fused read-and-clear, not a synchronisation.
// ------------------------------------------------------------------------------------------

#ifndef RSDGC_COPY_BATCH
#define RSDGC_COPY_BATCH 4
#endif
constexpr int kCopyBatch = RSDGC_COPY_BATCH;

template <bool BF16VAL>
__global__ void __launch_bounds__(kThreads)
k_gather(const __grid_constant__ LaneTable lanes, int n_lanes, const LayerDev *__restrict__ layers, int n_layers,
         long long idx_cap, long long val_cap, StatusDev *status)
{
    extern __shared__ __align__(16) unsigned char gather_smem_raw[];
    long long *val_off = reinterpret_cast<long long *>(gather_smem_raw);  // n_layers + 1
    long long *idx_off = val_off + n_layers + 1;                          // n_layers
    const int tid = threadIdx.x;
    grid_dependency_wait();
    // the workers one after the other: the scattered accesses of the CTAs that run at the same
    // time then fall into one worker's arena
    for (int lane = 0; lane < n_lanes; ++lane) {
        const Lane &ln = lanes.l[lane];
        float *__restrict__ resid = ln.resid;
        const LayerState *__restrict__ state = ln.state;
        const int32_t *__restrict__ idx = ln.idx;
        float *__restrict__ val = reinterpret_cast<float *>(ln.val);
        __nv_bfloat16 *__restrict__ val16 = reinterpret_cast<__nv_bfloat16 *>(ln.val);
        if (lane) __syncthreads();  // everyone is done with the previous worker's tables
        for (int l = tid; l < n_layers; l += kThreads) {
            val_off[l] = state[l].val_off;
            idx_off[l] = state[l].idx_off;
        }
        if (tid == 0) {
            const LayerState &last = state[n_layers - 1];
            val_off[n_layers] = last.val_off + (long long)last.k * layers[n_layers - 1].slot;
        }
        __syncthreads();
        const long long total = val_off[n_layers];
        // a CTA takes blocks of kThreads * kCopyBatch consecutive payload values: almost always one
        // layer per block, so the layer search is done once per block, not once per value
        constexpr long long kBlock = (long long)kThreads * kCopyBatch;
        auto find_layer = [&](long long j) {
            int lo = 0, hi = n_layers;  // layer with val_off[lo] <= j < val_off[lo + 1]
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (val_off[mid] <= j) lo = mid; else hi = mid;
            }
            return lo;
        };
        for (long long jb = (long long)blockIdx.x * kBlock; jb < total; jb += (long long)gridDim.x * kBlock) {
            const long long jend = min(total, jb + kBlock) - 1;
            const int l_first = find_layer(jb);
            const bool one_layer = val_off[l_first + 1] > jend;
            long long ga[kCopyBatch], vo[kCopyBatch];
            int tile[kCopyBatch], lay[kCopyBatch], el[kCopyBatch];
            float xv[kCopyBatch];
#pragma unroll
            for (int u = 0; u < kCopyBatch; ++u) {
                const long long j = jb + u * kThreads + tid;
                ga[u] = -1;
                vo[u] = -1;
                tile[u] = -1;
                if (j < total) {
                    const int lo = one_layer ? l_first : find_layer(j);
                    const int slot = layers[lo].slot;
                    const long long jl = j - val_off[lo];
                    // 32-bit division whenever the layer's payload is below 2^31 values (the usual case)
                    long long s;
                    if (jl < 0x7FFFFFFFll) {
                        int q, r;
                        divmod_small((int)jl, slot, &q, &r);
                        s = q;
                        el[u] = r;
                    } else {
                        s = jl / slot;
                        el[u] = (int)(jl - s * slot);
                    }
                    lay[u] = lo;
                    // tiles that do not fit the payload buffers are not sent and stay in the residual
                    if (idx_off[lo] + s < idx_cap && val_off[lo] + (s + 1) * slot <= val_cap) {
                        tile[u] = __ldg(idx + idx_off[lo] + s);
                        vo[u] = j;
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < kCopyBatch; ++u) {
                if (tile[u] >= 0) {
                    const LayerDev &L = layers[lay[u]];
                    const int tr = tile[u] / L.TC, tc = tile[u] - tr * L.TC;
                    int a, b;
                    divmod_small(el[u], L.nw, &a, &b);
                    const long long i = (long long)tr * L.nh + a, jj = (long long)tc * L.nw + b;
                    if (i < L.rows && jj < L.cols) ga[u] = L.elem_off + i * L.cols + jj;
                    if (!RSDGC_CHECKED(tile[u] < L.K && ga[u] < status->arena_elems, status)) ga[u] = -1, vo[u] = -1;
                }
            }
            if (BF16VAL) {  // q = bfloat16(v) is sent, v - q stays (exact in binary32)
#pragma unroll
                for (int u = 0; u < kCopyBatch; ++u) xv[u] = (ga[u] >= 0) ? resid[ga[u]] : 0.0f;
#pragma unroll
                for (int u = 0; u < kCopyBatch; ++u) {
                    const __nv_bfloat16 q = __float2bfloat16_rn(xv[u]);
                    if (ga[u] >= 0) resid[ga[u]] = __fsub_rn(xv[u], __bfloat162float(q));
                    if (vo[u] >= 0) val16[vo[u]] = q;
                }
            } else {
#pragma unroll
                for (int u = 0; u < kCopyBatch; ++u)
                    xv[u] = (ga[u] >= 0) ? __uint_as_float(atomicExch(reinterpret_cast<unsigned int *>(resid) + ga[u], 0u))
                                         : 0.0f;
#pragma unroll
                for (int u = 0; u < kCopyBatch; ++u)
                    if (vo[u] >= 0) val[vo[u]] = xv[u];
            }
        }
    }
}

// ------------------------------------------------------------------------------------------

// Next event of the plan's pool (created on demand), recorded on the stream.
static cudaError_t record_event(rsdgc_plan *p, cudaStream_t s)
{
    if (p->events_used == p->events.size()) {
        cudaEvent_t ev;
        cudaError_t e = cudaEventCreate(&ev);
        if (e != cudaSuccess) return e;
        p->events.push_back(ev);
    }
    return cudaEventRecord(p->events[p->events_used++], s);
}

// Launch with the programmatic-stream-serialization attribute: the kernel may be scheduled
// while its predecessor drains; it calls grid_dependency_wait() before touching that kernel's
// results.
template <typename... KArgs, typename... Args>
static cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, size_t smem, cudaStream_t s, Args... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// The four kernels after the accumulate+NSI pass, one launch each for all the lanes of the call.
static cudaError_t launch_selection(rsdgc_plan *p, const LaneTable &lanes, int n_lanes, int64_t idx_cap,
                                    int64_t val_cap, int prof, cudaStream_t s)
{
    const dim3 grid((unsigned)p->chunks.size(), (unsigned)n_lanes);
    const dim3 grid_gather((unsigned)(p->n_sm * 8));  // grid-stride loops over each lane's payload
    cudaError_t e = cudaSuccess;
#define RSDGC_MARK(level)                              \
    if (prof >= (level) && e == cudaSuccess) e = record_event(p, s)
    const int n_chunks = (int)p->chunks.size();
    // The two key passes.  Contiguous ranges of chunks of EQUAL length (the last CTAs one chunk less) when the list is
    // longer than the CTAs that fit on the device at once: with ceil(n / resident) chunks per CTA
    // and only as many CTAs as that takes, nobody is still working on an extra chunk while the
    // others are done.
    auto refine_grid = [&](int ctas_per_sm) {
        const int at_once = std::max(1, p->n_sm * ctas_per_sm / n_lanes);
        const int per_cta = (n_chunks + at_once - 1) / at_once;
        return dim3((unsigned)std::max(1, (n_chunks + per_cta - 1) / per_cta), (unsigned)n_lanes);
    };
    const dim3 grid_refine = refine_grid(kRefineCtasPerSm), grid_refine3 = refine_grid(kRefine3CtasPerSm);
    if (e == cudaSuccess)
        e = launch_chained(k_refine2, grid_refine, 0, s, lanes, p->d_layers, p->d_chunks, n_chunks, p->d_status);
    RSDGC_MARK(2);
    if (e == cudaSuccess)
        e = launch_chained(k_refine3_count, grid_refine3, 0, s, lanes, p->d_layers, p->d_chunks, n_chunks, p->n_layers,
                           (long long)idx_cap, (long long)val_cap, p->d_status);
    RSDGC_MARK(2);
    if (e == cudaSuccess)
        e = launch_chained(k_mark, grid, 0, s, lanes, p->d_layers, p->d_chunks, (long long)idx_cap, p->d_status);
    RSDGC_MARK(2);
    const size_t gather_smem = (size_t)(2 * p->n_layers + 1) * sizeof(long long);  // val_off, idx_off tables
    if (e == cudaSuccess)
        e = (p->flags & RSDGC_PAYLOAD_BF16)
                ? launch_chained(k_gather<true>, grid_gather, gather_smem, s, lanes, n_lanes, p->d_layers, p->n_layers,
                                 (long long)idx_cap, (long long)val_cap, p->d_status)
                : launch_chained(k_gather<false>, grid_gather, gather_smem, s, lanes, n_lanes, p->d_layers,
                                 p->n_layers, (long long)idx_cap, (long long)val_cap, p->d_status);
    RSDGC_MARK(2);
#undef RSDGC_MARK
    count_launch(4);
    return e;
}

// Plans whose layers all fit the single-kernel tail take it when the call's clusters (one set per
// worker) can all be resident at once; otherwise the chained kernels.
static bool use_fused_tail(const rsdgc_plan *p, int n_lanes)
{
    if (p->n_tail_big + p->n_tail_small == 0) return false;
    return (long long)p->n_tail_clusters * n_lanes <= p->tail_max_clusters;
}

// The single-kernel tail in the event layout of the chained path: stage 1 = the cluster kernel,
// stage 2 = the one-CTA kernel, stages 3..5 empty.
static cudaError_t launch_fused_tail(rsdgc_plan *p, const LaneTable &lanes, int n_lanes, const float *ratios,
                                     int64_t idx_cap, int64_t val_cap, int prof, cudaStream_t s)
{
    cudaError_t e = launch_tail(p, lanes, n_lanes, ratios, (long long)idx_cap, (long long)val_cap, prof, s, record_event);
    for (int k = 0; k < 2 && prof >= 2 && e == cudaSuccess; ++k) e = record_event(p, s);
    return e;
}

cudaError_t launch_compress(rsdgc_plan *p, const void *grads, float *resid, float *vel, float mom,
                            const float *ratios, int32_t *idx, int64_t idx_cap, void *val, int64_t val_cap,
                            int32_t *counts, uint32_t *keys, cudaStream_t s)
{
    const int prof = p->profile;
    cudaError_t e = cudaSuccess;
    if (prof) p->profile_recorded = prof;
    if (prof >= 1) e = record_event(p, s);
    const bool fused = use_fused_tail(p, 1);
    if (e == cudaSuccess)
        // ahead of the single-kernel tail the first pass lets its successor be scheduled as its CTAs leave:
        // that kernel touches only plan tables and the ratios before its own dependency wait
        e = launch_accumulate_nsi(p, p->d_hist, p->d_state, grads, resid, vel, mom, ratios, counts, keys, s, false,
                                  fused);
    if (prof >= 1 && e == cudaSuccess) e = record_event(p, s);
    LaneTable lanes{};
    lanes.l[0] = Lane{keys, p->d_hist, p->d_state, p->d_chunk_cnt, p->d_chunk_sfx, p->d_codes, resid, idx, val};
    if (e == cudaSuccess)
        e = fused ? launch_fused_tail(p, lanes, 1, ratios, idx_cap, val_cap, prof, s)
                  : launch_selection(p, lanes, 1, idx_cap, val_cap, prof, s);
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

// Several workers' gradients in one call (the data-parallel replicas that share a GPU): one
// accumulate+NSI launch per worker, back to back, then ONE launch of each selection kernel and of
// the gather for all the workers (blockIdx.y = worker).  The short, latency-bound kernels so
// serve several workers at a time.  With profiling on, stage 0 of a record covers the first
// passes of all the workers of a group (up to kMaxLanes workers form a group).
cudaError_t launch_compress_workers(rsdgc_plan *p, int n_workers, const void *const *grads, float *const *resid,
                                    const float *ratios, int32_t *const *idx, int64_t idx_cap, void *const *val,
                                    int64_t val_cap, int32_t *const *counts, uint32_t *keys_all, cudaStream_t s)
{
    const size_t key_stride = (size_t)p->info.workspace_bytes / sizeof(uint32_t);
    const int prof = p->profile;
    if (prof) p->profile_recorded = prof;
    cudaError_t e = cudaSuccess;
    for (int w0 = 0; w0 < n_workers && e == cudaSuccess; w0 += kMaxLanes) {
        const int n = n_workers - w0 < kMaxLanes ? n_workers - w0 : kMaxLanes;
        const bool fused = use_fused_tail(p, n);
        LaneTable lanes{};
        if (prof >= 1) e = record_event(p, s);
        for (int j = 0; j < n && e == cudaSuccess; ++j) {
            const int w = w0 + j;
            Lane &ln = lanes.l[j];
            if (w == 0) {
                ln = Lane{keys_all, p->d_hist, p->d_state, p->d_chunk_cnt, p->d_chunk_sfx, p->d_codes, resid[0], idx[0], val[0]};
            } else {
                const rsdgc_plan::LaneScratch &x = p->extra_lanes[(size_t)w - 1];
                ln = Lane{keys_all + (size_t)w * key_stride, x.hist, x.state, x.chunk_cnt, x.chunk_sfx, x.codes, resid[w], idx[w],
                          val[w]};
            }
            // the first passes of a group's workers share nothing: all but the first start without waiting
            e = launch_accumulate_nsi(p, ln.hist, ln.state, grads[w], ln.resid, nullptr, 0.0f, ratios, counts[w],
                                      ln.keys, s, j > 0, j + 1 < n);
        }
        if (prof >= 1 && e == cudaSuccess) e = record_event(p, s);
        if (e == cudaSuccess)
            e = fused ? launch_fused_tail(p, lanes, n, ratios, idx_cap, val_cap, prof, s)
                      : launch_selection(p, lanes, n, idx_cap, val_cap, prof, s);
    }
    if (e != cudaSuccess) return e;
    return cudaGetLastError();
}

}  // namespace rsdgc
