// Kernels of rsdgc_compress(): accumulate + NSI (+ level-1 histogram), two refinement
// passes of the per-layer radix selection, the per-chunk count/scan and the pack.
//
// Ordering between CTAs comes only from kernel boundaries and from "last arriver finishes
// the job" tickets (an atomic counter per layer and phase); no thread ever waits on another
// CTA.  The per-layer histograms and tickets are reset by the CTA that consumes them, so the
// plan's tables are all-zero again when a compress call has run to completion.
#include <cfloat>
#include <cuda_bf16.h>

#include "device_utils.cuh"

namespace rsdgc {

// ------------------------------------------------------------------------------------------
// K1: v = g + r in place, NSI key of every tile, level-1 histogram of the keys
// ------------------------------------------------------------------------------------------

constexpr int kVecPerThread = 6;  // 128-bit loads of g and of r in flight per thread

__device__ __forceinline__ float4 load_grad4(const float *g, long long i4)
{
    return __ldcs(reinterpret_cast<const float4 *>(g) + i4);
}
__device__ __forceinline__ float4 load_grad4(const __nv_bfloat16 *g, long long i4)
{
    const uint2 u = __ldcs(reinterpret_cast<const uint2 *>(g) + i4);
    float4 f;
    f.x = __uint_as_float(u.x << 16);
    f.y = __uint_as_float(u.x & 0xFFFF0000u);
    f.z = __uint_as_float(u.y << 16);
    f.w = __uint_as_float(u.y & 0xFFFF0000u);
    return f;
}
__device__ __forceinline__ float load_grad1(const float *g, long long i) { return __ldcs(g + i); }
__device__ __forceinline__ float load_grad1(const __nv_bfloat16 *g, long long i)
{
    return __uint_as_float(((unsigned int)__ldcs(reinterpret_cast<const unsigned short *>(g) + i)) << 16);
}

// NSI of one tile held in shared memory (Eq. 8-10), binary32, elements visited row-major,
// plain running sums, mean first and squared deviations in a second sweep; every operation
// is an explicitly rounded single operation (no fused multiply-add).
__device__ __forceinline__ float tile_nsi(const float *p, int pitch, int hh, int ww, float alpha)
{
    float sa = 0.0f, sv = 0.0f;
    for (int a = 0; a < hh; ++a)
        for (int b = 0; b < ww; ++b) {
            const float x = p[a * pitch + b];
            sa = __fadd_rn(sa, fabsf(x));
            sv = __fadd_rn(sv, x);
        }
    const float fn = (float)(hh * ww);
    const float mean_abs = __fdiv_rn(sa, fn);
    const float m = __fdiv_rn(sv, fn);
    float sq = 0.0f;
    for (int a = 0; a < hh; ++a)
        for (int b = 0; b < ww; ++b) {
            const float d = __fsub_rn(p[a * pitch + b], m);
            sq = __fadd_rn(sq, __fmul_rn(d, d));
        }
    const float s = __fsqrt_rn(__fdiv_rn(sq, fn));
    return __fadd_rn(__fmul_rn(alpha, mean_abs), __fmul_rn(__fsub_rn(1.0f, alpha), s));
}

template <int HH, int WW>
__device__ __forceinline__ float tile_nsi_fixed(const float *p, int pitch, float alpha)
{
    float x[HH * WW];
#pragma unroll
    for (int a = 0; a < HH; ++a)
#pragma unroll
        for (int b = 0; b < WW; ++b) x[a * WW + b] = p[a * pitch + b];
    float sa = 0.0f, sv = 0.0f;
#pragma unroll
    for (int i = 0; i < HH * WW; ++i) {
        sa = __fadd_rn(sa, fabsf(x[i]));
        sv = __fadd_rn(sv, x[i]);
    }
    const float fn = (float)(HH * WW);
    const float mean_abs = __fdiv_rn(sa, fn);
    const float m = __fdiv_rn(sv, fn);
    float sq = 0.0f;
#pragma unroll
    for (int i = 0; i < HH * WW; ++i) {
        const float d = __fsub_rn(x[i], m);
        sq = __fadd_rn(sq, __fmul_rn(d, d));
    }
    const float s = __fsqrt_rn(__fdiv_rn(sq, fn));
    return __fadd_rn(__fmul_rn(alpha, mean_abs), __fmul_rn(__fsub_rn(1.0f, alpha), s));
}

struct K1Shared {
    float v[kItemElems];
    unsigned int hist[kL1Bins];
    unsigned long long scan_tmp[kThreads / 32];
    unsigned long long found[2];
    int is_last;
};

// Adds this CTA's level-1 histogram to the layer's global histogram; the last CTA to do so
// for the layer computes k_l (Eq. 11) and resolves the first 11 key bits of the threshold.
__device__ void k1_flush_layer(K1Shared &sh, int layer, const LayerDev *layers, unsigned int *hist,
                               LayerState *state, const float *ratios, int32_t *counts, unsigned int flags)
{
    __syncthreads();
    unsigned int *gh = hist + (size_t)layer * kHistStride;
    for (int b = threadIdx.x; b < kL1Bins; b += kThreads) {
        const unsigned int c = sh.hist[b];
        if (c) {
            atomicAdd(gh + b, c);
            sh.hist[b] = 0;
        }
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int t = atomicAdd(&state[layer].ticket[0], 1u);
        sh.is_last = (t + 1u == (unsigned int)layers[layer].n_flush1);
    }
    __syncthreads();
    if (!sh.is_last) return;  // uniform for the CTA
    __threadfence();
    for (int b = threadIdx.x; b < kL1Bins; b += kThreads) {
        sh.hist[b] = __ldcg(gh + b);
        gh[b] = 0;
    }
    __syncthreads();
    const int K = layers[layer].K;
    const int k = keep_count(K, ratios[layer], flags);
    if (k > 0) find_bin_from_top<kL1Bins>(sh.hist, (unsigned long long)k, sh.found, sh.scan_tmp);
    if (threadIdx.x == 0) {
        LayerState &st = state[layer];
        st.k = k;
        st.prefix = k > 0 ? (uint32_t)sh.found[0] : kTakeNone;
        st.remaining = k > 0 ? (int32_t)sh.found[1] : 0;
        st.ticket[0] = 0;
        counts[layer] = k;
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kL1Bins; b += kThreads) sh.hist[b] = 0;
    __syncthreads();
}

template <typename G>
__global__ void __launch_bounds__(kThreads)
k1_accumulate_nsi(const G *__restrict__ grads, float *__restrict__ resid, uint32_t *__restrict__ keys,
                  const LayerDev *__restrict__ layers, const Item *__restrict__ items,
                  const int32_t *__restrict__ cta_begin, unsigned int *hist, LayerState *state,
                  const float *__restrict__ ratios, int32_t *counts, StatusDev *status, float alpha,
                  unsigned int flags)
{
    __shared__ K1Shared sh;
    const int begin = cta_begin[blockIdx.x], end = cta_begin[blockIdx.x + 1];
    if (begin >= end) return;
    const int tid = threadIdx.x;
    for (int b = tid; b < kL1Bins; b += kThreads) sh.hist[b] = 0;
    unsigned int nonfinite = 0;
    int cur_layer = items[begin].layer;
    __syncthreads();

    for (int it = begin; it < end; ++it) {
        const Item im = items[it];
        if (im.layer != cur_layer) {
            k1_flush_layer(sh, cur_layer, layers, hist, state, ratios, counts, flags);
            cur_layer = im.layer;
        }
        const LayerDev L = layers[im.layer];
        const int nh = L.nh, nw = L.nw;
        const long long row0 = (long long)im.tr0 * nh;
        const int R = (int)min((long long)im.ntr * nh, L.rows - row0);     // rows held
        const long long col0 = (long long)im.tc0 * nw;
        const int W = (int)min((long long)im.ntc * nw, L.cols - col0);     // cols held = smem pitch
        const bool full = (W == L.cols);
        const int nseg = full ? 1 : R;              // contiguous global runs
        const int seglen = full ? R * W : W;
        const long long gbase = L.elem_off + row0 * L.cols + col0;

        // ---- v = g + r : global -> registers -> global (in place) and shared memory
        const bool vec = ((gbase & 3) == 0) && (nseg == 1 || ((L.cols & 3) == 0 && (W & 3) == 0));
        if (vec) {
            const int wv = seglen >> 2;            // 128-bit vectors per run
            const int nvec = wv * nseg;
            for (int base = 0; base < nvec; base += kThreads * kVecPerThread) {
                float4 g[kVecPerThread], r[kVecPerThread];
                long long gi[kVecPerThread];
                int si[kVecPerThread];
#pragma unroll
                for (int u = 0; u < kVecPerThread; ++u) {
                    const int i = base + u * kThreads + tid;
                    if (i < nvec) {
                        const int seg = (nseg == 1) ? 0 : i / wv;
                        const int j = i - seg * wv;
                        gi[u] = ((gbase + (long long)seg * L.cols) >> 2) + j;
                        si[u] = ((seg * W) >> 2) + j;
                        g[u] = load_grad4(grads, gi[u]);
                        r[u] = __ldcs(reinterpret_cast<const float4 *>(resid) + gi[u]);
                    }
                }
#pragma unroll
                for (int u = 0; u < kVecPerThread; ++u) {
                    const int i = base + u * kThreads + tid;
                    if (i < nvec) {
                        float4 v;
                        v.x = __fadd_rn(g[u].x, r[u].x);
                        v.y = __fadd_rn(g[u].y, r[u].y);
                        v.z = __fadd_rn(g[u].z, r[u].z);
                        v.w = __fadd_rn(g[u].w, r[u].w);
                        reinterpret_cast<float4 *>(resid)[gi[u]] = v;
                        reinterpret_cast<float4 *>(sh.v)[si[u]] = v;
                    }
                }
            }
            if (nseg == 1) {  // scalar tail of a run whose length is not a multiple of 4
                const int i = (wv << 2) + tid;
                if (i < seglen) {
                    const float v = __fadd_rn(load_grad1(grads, gbase + i), resid[gbase + i]);
                    resid[gbase + i] = v;
                    sh.v[i] = v;
                }
            }
        } else {
            const int n = nseg * seglen;
            for (int i = tid; i < n; i += kThreads) {
                const int seg = (nseg == 1) ? 0 : i / seglen;
                const int j = i - seg * seglen;
                const long long gidx = gbase + (long long)seg * L.cols + j;
                const float v = __fadd_rn(load_grad1(grads, gidx), resid[gidx]);
                resid[gidx] = v;
                sh.v[seg * W + j] = v;
            }
        }
        __syncthreads();

        // ---- NSI of every tile of the item, one thread per tile
        const int ntr = (R + nh - 1) / nh;
        const int ntc = im.ntc;
        const int ntile = ntr * ntc;
        uint32_t *kout = keys + L.tile_off + (long long)im.tr0 * L.TC + im.tc0;
        for (int t = tid; t < ntile; t += kThreads) {
            const int ti = (ntr == 1) ? 0 : t / ntc;
            const int tj = t - ti * ntc;
            const int hh = min(nh, R - ti * nh);
            const int ww = min(nw, W - tj * nw);
            const float *p = sh.v + (ti * nh) * W + tj * nw;
            float nsi;
            if (hh == 3 && ww == 3 && nh == 3 && nw == 3)
                nsi = tile_nsi_fixed<3, 3>(p, W, alpha);
            else if (hh == 1 && ww == 9 && nw == 9)
                nsi = tile_nsi_fixed<1, 9>(p, W, alpha);
            else
                nsi = tile_nsi(p, W, hh, ww, alpha);
            uint32_t key = __float_as_uint(nsi);
            if (!(nsi <= FLT_MAX)) {  // NaN or infinity: ranks first, deterministically
                key = 0x7F800000u;
                ++nonfinite;
            }
            kout[(long long)ti * L.TC + tj] = key;
            atomicAdd(&sh.hist[key >> kL1Shift], 1u);
        }
        __syncthreads();
    }
    k1_flush_layer(sh, cur_layer, layers, hist, state, ratios, counts, flags);
    if (nonfinite) {
        atomicAdd(&status->nonfinite, (unsigned long long)nonfinite);
        atomicOr(&status->flags, RSDGC_STATUS_NONFINITE);
    }
}

// ------------------------------------------------------------------------------------------
// K2 / K3: refinement passes over the keys (levels 2 and 3 of the radix selection)
// ------------------------------------------------------------------------------------------

struct RefineShared {
    unsigned int hist[kL2Bins];
    unsigned long long scan_tmp[kThreads / 32];
    unsigned long long found[2];
    int is_last;
};

// LEVEL 2: among keys whose bits 30..20 equal the layer's prefix, histogram bits 19..10.
// LEVEL 3: among keys whose bits 30..10 equal the prefix, histogram bits 9..0; the last CTA
// of the layer then knows the threshold key T and how many keys equal to T are taken.
template <int LEVEL>
__global__ void __launch_bounds__(kThreads)
k_refine(const uint32_t *__restrict__ keys, const LayerDev *__restrict__ layers,
         const Chunk *__restrict__ chunks, unsigned int *hist, LayerState *state)
{
    __shared__ RefineShared sh;
    constexpr int SHIFT_HI = (LEVEL == 2) ? kL1Shift : kL2Shift;
    constexpr int SHIFT_LO = (LEVEL == 2) ? kL2Shift : 0;
    const Chunk c = chunks[blockIdx.x];
    const int tid = threadIdx.x;
    LayerState &st = state[c.layer];
    const uint32_t prefix = st.prefix;
    for (int b = tid; b < kL2Bins; b += kThreads) sh.hist[b] = 0;
    __syncthreads();
    if (prefix != kTakeNone) {
        const uint32_t *kp = keys + layers[c.layer].tile_off + c.start;
        const int nvec = c.n >> 2;
        for (int i = tid; i < nvec; i += kThreads) {
            const uint4 q = __ldg(reinterpret_cast<const uint4 *>(kp) + i);
            if ((q.x >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(q.x >> SHIFT_LO) & (kL2Bins - 1)], 1u);
            if ((q.y >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(q.y >> SHIFT_LO) & (kL2Bins - 1)], 1u);
            if ((q.z >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(q.z >> SHIFT_LO) & (kL2Bins - 1)], 1u);
            if ((q.w >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(q.w >> SHIFT_LO) & (kL2Bins - 1)], 1u);
        }
        const int i = (nvec << 2) + tid;
        if (i < c.n) {
            const uint32_t q = kp[i];
            if ((q >> SHIFT_HI) == prefix) atomicAdd(&sh.hist[(q >> SHIFT_LO) & (kL2Bins - 1)], 1u);
        }
    }
    __syncthreads();
    unsigned int *gh = hist + (size_t)c.layer * kHistStride;
    for (int b = tid; b < kL2Bins; b += kThreads) {
        const unsigned int n = sh.hist[b];
        if (n) atomicAdd(gh + b, n);
    }
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned int t = atomicAdd(&st.ticket[LEVEL - 1], 1u);
        sh.is_last = (t + 1u == (unsigned int)layers[c.layer].n_chunks);
    }
    __syncthreads();
    if (!sh.is_last) return;
    __threadfence();
    for (int b = tid; b < kL2Bins; b += kThreads) {
        sh.hist[b] = __ldcg(gh + b);
        gh[b] = 0;
    }
    __syncthreads();
    const int remaining = st.remaining;
    if (prefix != kTakeNone)
        find_bin_from_top<kL2Bins>(sh.hist, (unsigned long long)remaining, sh.found, sh.scan_tmp);
    if (tid == 0) {
        st.ticket[LEVEL - 1] = 0;
        if (prefix != kTakeNone) {
            const uint32_t next = (prefix << 10) | (uint32_t)sh.found[0];
            if (LEVEL == 2) {
                st.prefix = next;
                st.remaining = (int32_t)sh.found[1];
            } else {
                st.T = next;
                st.e = (int32_t)sh.found[1];
            }
        } else if (LEVEL == 3) {
            st.T = kTakeNone;
            st.e = 0;
        }
    }
}

// ------------------------------------------------------------------------------------------
// K4: per chunk, how many keys lie above the threshold and how many equal it; the last CTA
// of a layer turns the layer's chunk counts into exclusive bases and computes the layer's
// payload offsets (prefix sums of k_l' over the preceding layers).
// ------------------------------------------------------------------------------------------

struct CountShared {
    unsigned long long scan_tmp[kThreads / 32];
    unsigned int red[2][kThreads / 32];
    int is_last;
};

__global__ void __launch_bounds__(kThreads)
k_count(const uint32_t *__restrict__ keys, const LayerDev *__restrict__ layers,
        const Chunk *__restrict__ chunks, LayerState *state, uint2 *chunk_cnt, int n_layers,
        long long idx_cap, long long val_cap, StatusDev *status)
{
    __shared__ CountShared sh;
    const Chunk c = chunks[blockIdx.x];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    LayerState &st = state[c.layer];
    const LayerDev &L = layers[c.layer];
    const uint32_t T = st.T;
    unsigned int gt = 0, eq = 0;
    {
        const uint32_t *kp = keys + L.tile_off + c.start;
        const int nvec = c.n >> 2;
        for (int i = tid; i < nvec; i += kThreads) {
            const uint4 q = __ldg(reinterpret_cast<const uint4 *>(kp) + i);
            gt += (q.x > T) + (q.y > T) + (q.z > T) + (q.w > T);
            eq += (q.x == T) + (q.y == T) + (q.z == T) + (q.w == T);
        }
        const int i = (nvec << 2) + tid;
        if (i < c.n) {
            const uint32_t q = kp[i];
            gt += (q > T);
            eq += (q == T);
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        gt += __shfl_xor_sync(0xFFFFFFFFu, gt, d);
        eq += __shfl_xor_sync(0xFFFFFFFFu, eq, d);
    }
    if (lane == 0) {
        sh.red[0][warp] = gt;
        sh.red[1][warp] = eq;
    }
    __syncthreads();
    if (tid == 0) {
        unsigned int a = 0, b = 0;
        for (int w = 0; w < kThreads / 32; ++w) {
            a += sh.red[0][w];
            b += sh.red[1][w];
        }
        chunk_cnt[blockIdx.x] = make_uint2(a, b);
        __threadfence();
        const unsigned int t = atomicAdd(&st.ticket[3], 1u);
        sh.is_last = (t + 1u == (unsigned int)L.n_chunks);
    }
    __syncthreads();
    if (!sh.is_last) return;
    __threadfence();

    // exclusive scan of (gt, eq) over the layer's chunks, in chunk order
    uint2 *cc = chunk_cnt + L.first_chunk;
    unsigned long long carry = 0;  // gt in the low 32 bits, eq in the high 32 bits
    for (int base = 0; base < L.n_chunks; base += kThreads) {
        const int i = base + tid;
        unsigned long long x = 0;
        if (i < L.n_chunks) {
            const unsigned long long raw = __ldcg(reinterpret_cast<const unsigned long long *>(cc + i));
            x = raw;  // uint2 {x = gt, y = eq} is little-endian: low word gt, high word eq
        }
        unsigned long long total;
        const unsigned long long ex = block_exclusive_scan<unsigned long long>(x, sh.scan_tmp, &total) + carry;
        if (i < L.n_chunks) cc[i] = make_uint2((unsigned int)(ex & 0xFFFFFFFFull), (unsigned int)(ex >> 32));
        carry += total;
    }

    // payload offsets of this layer: sums over the preceding layers of k and k * slot
    long long si = 0, sv = 0;
    for (int l = tid; l < c.layer; l += kThreads) {
        const long long k = state[l].k;
        si += k;
        sv += k * layers[l].slot;
    }
    unsigned long long tot_i, tot_v;
    (void)block_exclusive_scan<unsigned long long>((unsigned long long)si, sh.scan_tmp, &tot_i);
    (void)block_exclusive_scan<unsigned long long>((unsigned long long)sv, sh.scan_tmp, &tot_v);
    if (tid == 0) {
        st.idx_off = (long long)tot_i;
        st.val_off = (long long)tot_v;
        st.ticket[3] = 0;
        if (c.layer == n_layers - 1) {
            const long long need_i = (long long)tot_i + st.k;
            const long long need_v = (long long)tot_v + (long long)st.k * L.slot;
            status->idx_needed = need_i;
            status->val_needed = need_v;
            if (need_i > idx_cap || need_v > val_cap) atomicOr(&status->flags, RSDGC_STATUS_PAYLOAD_OVERFLOW);
        }
    }
}

// ------------------------------------------------------------------------------------------
// K5: pack.  A tile is kept if its key is above T, or equals T and fewer than e equal keys
// precede it in the layer.  Its payload slot is its rank among the kept tiles of the layer
// (ascending tile index).  Kept tiles are copied out of the residual and zeroed there.
// ------------------------------------------------------------------------------------------

constexpr int kKeysPerThread = kChunkKeys / kThreads;  // 64 consecutive keys per thread

struct PackShared {
    unsigned short pos[kChunkKeys];  // position in the chunk of the r-th kept tile
    unsigned long long scan_tmp[kThreads / 32];
};

__global__ void __launch_bounds__(kThreads)
k_pack(const uint32_t *__restrict__ keys, float *__restrict__ resid, const LayerDev *__restrict__ layers,
       const Chunk *__restrict__ chunks, const LayerState *__restrict__ state,
       const uint2 *__restrict__ chunk_cnt, int32_t *__restrict__ idx, long long idx_cap,
       float *__restrict__ val, long long val_cap)
{
    __shared__ PackShared sh;
    const Chunk c = chunks[blockIdx.x];
    const int tid = threadIdx.x;
    const LayerState st = state[c.layer];
    if (st.k == 0) return;
    const LayerDev L = layers[c.layer];
    const uint32_t T = st.T;
    const uint2 base = chunk_cnt[blockIdx.x];  // tiles above T / equal to T in earlier chunks
    // equal keys of this chunk that are still taken: those with layer-wide equal-rank < e
    const long long eq_room = max(0ll, (long long)st.e - (long long)base.y);

    const uint32_t *kp = keys + L.tile_off + c.start;
    const int p0 = tid * kKeysPerThread;
    const int p1 = min(c.n, p0 + kKeysPerThread);
    unsigned int gt = 0, eq = 0;
    for (int p = p0; p < p1; p += 4) {  // chunk starts and p0 are multiples of 4
        if (p + 4 <= c.n) {
            const uint4 q = __ldg(reinterpret_cast<const uint4 *>(kp + p));
            gt += (q.x > T) + (q.y > T) + (q.z > T) + (q.w > T);
            eq += (q.x == T) + (q.y == T) + (q.z == T) + (q.w == T);
        } else {
            for (int j = p; j < c.n; ++j) {
                const uint32_t q = kp[j];
                gt += (q > T);
                eq += (q == T);
            }
        }
    }
    unsigned long long total;
    const unsigned long long ex =
        block_exclusive_scan<unsigned long long>(((unsigned long long)eq << 32) | gt, sh.scan_tmp, &total);
    unsigned int gt_before = (unsigned int)(ex & 0xFFFFFFFFull), eq_before = (unsigned int)(ex >> 32);
    for (int p = p0; p < p1; ++p) {
        const uint32_t q = __ldg(kp + p);
        if (q > T) {
            sh.pos[gt_before + (unsigned int)min((long long)eq_before, eq_room)] = (unsigned short)p;
            ++gt_before;
        } else if (q == T) {
            if ((long long)eq_before < eq_room)
                sh.pos[gt_before + eq_before] = (unsigned short)p;
            ++eq_before;
        }
    }
    __syncthreads();
    const unsigned int tot_gt = (unsigned int)(total & 0xFFFFFFFFull), tot_eq = (unsigned int)(total >> 32);
    const int n_kept = (int)(tot_gt + (unsigned int)min((long long)tot_eq, eq_room));
    // rank in the layer of this chunk's first kept tile
    const long long rank0 = (long long)base.x + min((long long)base.y, (long long)st.e);

    const int slot = L.slot;
    const long long n_copy = (long long)n_kept * slot;
    for (long long j = tid; j < n_copy; j += kThreads) {
        const int r = (int)(j / slot);
        const int el = (int)(j - (long long)r * slot);
        const int tile = c.start + sh.pos[r];
        const long long s = st.idx_off + rank0 + r;           // payload slot (tiles)
        const long long vbase = st.val_off + (rank0 + r) * slot;
        if (s >= idx_cap || vbase + slot > val_cap) continue;  // does not fit: not sent
        const int tr = tile / L.TC, tc = tile - tr * L.TC;
        const int a = el / L.nw, b = el - a * L.nw;
        const long long i = (long long)tr * L.nh + a, jj = (long long)tc * L.nw + b;
        float x = 0.0f;
        if (i < L.rows && jj < L.cols) {
            const long long g = L.elem_off + i * L.cols + jj;
            x = resid[g];
            resid[g] = 0.0f;
        }
        val[vbase + el] = x;
        if (el == 0) idx[s] = tile;
    }
}

// ------------------------------------------------------------------------------------------

cudaError_t launch_compress(rsdgc_plan *p, const void *grads, float *resid, const float *ratios, int32_t *idx,
                            int64_t idx_cap, float *val, int64_t val_cap, int32_t *counts, uint32_t *keys,
                            cudaStream_t s)
{
    const int n_chunks = (int)p->chunks.size();
    if (p->dtype == RSDGC_BF16)
        k1_accumulate_nsi<__nv_bfloat16><<<p->grid1, kThreads, 0, s>>>(
            reinterpret_cast<const __nv_bfloat16 *>(grads), resid, keys, p->d_layers, p->d_items, p->d_cta_begin,
            p->d_hist, p->d_state, ratios, counts, p->d_status, p->alpha, p->flags);
    else
        k1_accumulate_nsi<float><<<p->grid1, kThreads, 0, s>>>(
            reinterpret_cast<const float *>(grads), resid, keys, p->d_layers, p->d_items, p->d_cta_begin,
            p->d_hist, p->d_state, ratios, counts, p->d_status, p->alpha, p->flags);
    k_refine<2><<<n_chunks, kThreads, 0, s>>>(keys, p->d_layers, p->d_chunks, p->d_hist, p->d_state);
    k_refine<3><<<n_chunks, kThreads, 0, s>>>(keys, p->d_layers, p->d_chunks, p->d_hist, p->d_state);
    k_count<<<n_chunks, kThreads, 0, s>>>(keys, p->d_layers, p->d_chunks, p->d_state, p->d_chunk_cnt,
                                          p->n_layers, idx_cap, val_cap, p->d_status);
    k_pack<<<n_chunks, kThreads, 0, s>>>(keys, resid, p->d_layers, p->d_chunks, p->d_state, p->d_chunk_cnt, idx,
                                         idx_cap, val, val_cap);
    count_launch(5);
    return cudaGetLastError();
}

}  // namespace rsdgc
