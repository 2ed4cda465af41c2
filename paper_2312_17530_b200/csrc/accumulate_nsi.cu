// First pass of rsdgc_compress(): v = g + r in place (Eq. 12), the NSI key of every tile
// (Eq. 8-10), and the level-1 histogram of the keys per layer.
//
// Two kernels share the work list:
//  * k1_bulk: three persistent 256-thread CTAs per SM (two with momentum correction).  The g and
//    r blocks of an item are brought into shared memory by the bulk-copy engine (cp.async.bulk +
//    mbarrier) one item ahead of their use, v is formed in shared memory and written back with a
//    bulk store, and the tiles are reduced from shared memory.  Bytes in flight do not occupy
//    registers.  It takes every item whose rows are 16-byte aligned in memory (all the usual
//    shapes).
//  * k1_reg: 256-thread CTAs that stage an item in registers (128-bit loads where possible,
//    scalar otherwise).  It takes the remaining items (odd pitches, unaligned starts).
//
// Ordering between CTAs comes only from kernel boundaries and from "last arriver finishes the
// job" tickets; the only waits are on a CTA's own mbarriers and every such wait is bounded.
#include <cfloat>
#include <cuda_bf16.h>

#include "device_utils.cuh"

namespace rsdgc {

// ------------------------------------------------------------------------------------------
// NSI of one tile
// ------------------------------------------------------------------------------------------

// NSI of one tile held in shared memory (Eq. 8-10) in binary32: elements visited row-major,
// plain running sums, mean first and squared deviations in a second sweep; the three
// "(1/n) sum" of Eq. 9-10 multiply the sum by inv_n = 1/n (rounded once).  Every operation is
// an explicitly rounded single operation (no fused multiply-add).
__device__ float tile_nsi_generic(const float *p, int pitch, int hh, int ww, float alpha)
{
    float sa = 0.0f, sv = 0.0f;
    for (int a = 0; a < hh; ++a)
        for (int b = 0; b < ww; ++b) {
            const float x = p[a * pitch + b];
            sa = __fadd_rn(sa, fabsf(x));
            sv = __fadd_rn(sv, x);
        }
    const float inv_n = __fdiv_rn(1.0f, (float)(hh * ww));
    const float mean_abs = __fmul_rn(sa, inv_n);
    const float m = __fmul_rn(sv, inv_n);
    float sq = 0.0f;
    for (int a = 0; a < hh; ++a)
        for (int b = 0; b < ww; ++b) {
            const float d = __fsub_rn(p[a * pitch + b], m);
            sq = __fadd_rn(sq, __fmul_rn(d, d));
        }
    const float s = __fsqrt_rn(__fmul_rn(sq, inv_n));
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
    const float inv_n = __fdiv_rn(1.0f, (float)(HH * WW));  // folded at compile time
    const float mean_abs = __fmul_rn(sa, inv_n);
    const float m = __fmul_rn(sv, inv_n);
    float sq = 0.0f;
#pragma unroll
    for (int i = 0; i < HH * WW; ++i) {
        const float d = __fsub_rn(x[i], m);
        sq = __fadd_rn(sq, __fmul_rn(d, d));
    }
    const float s = __fsqrt_rn(__fmul_rn(sq, inv_n));
    return __fadd_rn(__fmul_rn(alpha, mean_abs), __fmul_rn(__fsub_rn(1.0f, alpha), s));
}

// Key of one indicator value; counts it in the CTA's level-1 histogram.
__device__ __forceinline__ void emit_key(float nsi, uint32_t *dst, unsigned int *hist_smem, unsigned int &nonfinite)
{
    uint32_t key = __float_as_uint(nsi);
    if (!(nsi <= FLT_MAX)) {  // NaN or infinity: ranks first, deterministically
        key = 0x7F800000u;
        ++nonfinite;
    }
    *dst = key;
    atomicAdd(&hist_smem[key >> kL1Shift], 1u);
}

// Keys of all tiles of an item none of whose tiles is clipped, for a tile shape known at compile
// time: two tiles per thread and round, so that the two chains of dependent additions (every sum is
// sequential by definition) overlap instead of following each other.
template <int NTHREADS, int HH, int WW>
__device__ __forceinline__ unsigned int item_tile_keys_fixed(const ItemDev &d, const float *sv,
                                                             uint32_t *__restrict__ keys, unsigned int *hist_smem,
                                                             float alpha)
{
    const int P = d.P, ntc = d.ntc;
    const int ntr = d.R / HH;
    const int ntile = ntr * ntc;
    uint32_t *kout = keys + d.kbase;
    unsigned int nonfinite = 0;
    int t = threadIdx.x;
    for (; t + NTHREADS < ntile; t += 2 * NTHREADS) {
        const int ti0 = (ntr == 1) ? 0 : fast_div(t, d.inv_ntc), ti1 = (ntr == 1) ? 0 : fast_div(t + NTHREADS, d.inv_ntc);
        const int tj0 = t - ti0 * ntc, tj1 = t + NTHREADS - ti1 * ntc;
        const float nsi0 = tile_nsi_fixed<HH, WW>(sv + (ti0 * HH) * P + tj0 * WW, P, alpha);
        const float nsi1 = tile_nsi_fixed<HH, WW>(sv + (ti1 * HH) * P + tj1 * WW, P, alpha);
        emit_key(nsi0, kout + ti0 * d.TC + tj0, hist_smem, nonfinite);
        emit_key(nsi1, kout + ti1 * d.TC + tj1, hist_smem, nonfinite);
    }
    if (t < ntile) {
        const int ti = (ntr == 1) ? 0 : fast_div(t, d.inv_ntc);
        const int tj = t - ti * ntc;
        emit_key(tile_nsi_fixed<HH, WW>(sv + (ti * HH) * P + tj * WW, P, alpha), kout + ti * d.TC + tj, hist_smem,
                 nonfinite);
    }
    return nonfinite;
}

// Keys of all tiles of one item from its v block in shared memory (row pitch d.P).
// Returns the number of non-finite indicators this thread saw.
template <int NTHREADS>
__device__ __forceinline__ unsigned int item_tile_keys(const ItemDev &d, const float *sv, uint32_t *__restrict__ keys,
                                                       unsigned int *hist_smem, float alpha)
{
    const int nh = d.nh, nw = d.nw, R = d.R, W = d.W, P = d.P;
    if (d.flags & kItemNoClip) {  // the two usual shapes, every tile whole
        if (nh == 3 && nw == 3) return item_tile_keys_fixed<NTHREADS, 3, 3>(d, sv, keys, hist_smem, alpha);
        if (nh == 1 && nw == 9) return item_tile_keys_fixed<NTHREADS, 1, 9>(d, sv, keys, hist_smem, alpha);
    }
    const int ntr = (R + nh - 1) / nh;
    const int ntc = d.ntc;
    const int ntile = ntr * ntc;
    uint32_t *kout = keys + d.kbase;
    unsigned int nonfinite = 0;
    for (int t = threadIdx.x; t < ntile; t += NTHREADS) {
        const int ti = (ntr == 1) ? 0 : fast_div(t, d.inv_ntc);
        const int tj = t - ti * ntc;
        const int hh = min(nh, R - ti * nh);
        const int ww = min(nw, W - tj * nw);
        const float *pt = sv + (ti * nh) * P + tj * nw;
        const float nsi = (hh == 3 && ww == 3) ? tile_nsi_fixed<3, 3>(pt, P, alpha)
                          : (hh == 1 && ww == 9) ? tile_nsi_fixed<1, 9>(pt, P, alpha)
                                                 : tile_nsi_generic(pt, P, hh, ww, alpha);
        emit_key(nsi, kout + ti * d.TC + tj, hist_smem, nonfinite);
    }
    return nonfinite;
}

// ------------------------------------------------------------------------------------------
// level-1 histogram flush and the first step of the per-layer selection
// ------------------------------------------------------------------------------------------

struct FlushShared {
    unsigned long long scan_tmp[32];
    unsigned long long found[2];
    int is_last;
};

// Adds this CTA's level-1 histogram to the layer's global histogram; the last CTA to do so
// for the layer computes k_l (Eq. 11) and resolves the first 11 key bits of the threshold.
// Called by all threads of the CTA.
// What the flush of a layer needs from the plan's tables and the ratios: loaded when a CTA enters the
// layer, so that the loads (cold: every layer's entries are read only here) are long complete when the
// CTA leaves it.
struct FlushInfo {
    int K, n_flush1;
    float ratio;
};
__device__ __forceinline__ FlushInfo load_flush_info(const LayerDev *__restrict__ layers,
                                                     const float *__restrict__ ratios, int layer)
{
    FlushInfo f;
    f.K = __ldg(&layers[layer].K);
    f.n_flush1 = __ldg(&layers[layer].n_flush1);
    f.ratio = __ldg(&ratios[layer]);
    return f;
}

template <int NTHREADS>
__device__ void k1_flush_layer(unsigned int *hist_smem, FlushShared &fs, int layer, const FlushInfo info,
                               unsigned int *hist, LayerState *state, int32_t *counts, unsigned int flags)
{
    __syncthreads();
    unsigned int *gh = hist + (size_t)layer * kHistStride;
    const bool sole_owner = info.n_flush1 == 1;  // the whole layer went through this CTA
    if (!sole_owner) {
        for (int b = threadIdx.x; b < kL1Bins; b += NTHREADS) {
            const unsigned int c = hist_smem[b];
            if (c) {
                atomicAdd(gh + b, c);
                hist_smem[b] = 0;
            }
        }
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) {
            const unsigned int t = atomicAdd(&state[layer].ticket[0], 1u);
            fs.is_last = (t + 1u == (unsigned int)info.n_flush1);
        }
        __syncthreads();
        if (!fs.is_last) return;  // uniform for the CTA
        __threadfence();
    }
    if (!sole_owner) {  // otherwise the shared-memory histogram already is the layer's histogram
        unsigned int h[kL1Bins / NTHREADS];
#pragma unroll
        for (int j = 0; j < kL1Bins / NTHREADS; ++j) h[j] = __ldcg(gh + j * NTHREADS + threadIdx.x);
#pragma unroll
        for (int j = 0; j < kL1Bins / NTHREADS; ++j) {
            hist_smem[j * NTHREADS + threadIdx.x] = h[j];
            gh[j * NTHREADS + threadIdx.x] = 0;
        }
    }
    __syncthreads();
    const int k = keep_count(info.K, info.ratio, flags);
    if (k > 0) find_bin_from_top<kL1Bins, NTHREADS>(hist_smem, (unsigned long long)k, fs.found, fs.scan_tmp);
    if (threadIdx.x == 0) {
        LayerState &st = state[layer];
        st.k = k;
        st.prefix = k > 0 ? (uint32_t)fs.found[0] : kTakeNone;
        st.remaining = k > 0 ? (int32_t)fs.found[1] : 0;
        if (!sole_owner) st.ticket[0] = 0;
        counts[layer] = k;
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kL1Bins; b += NTHREADS) hist_smem[b] = 0;
    __syncthreads();
}

// ------------------------------------------------------------------------------------------
// gradient element access (binary32 or bfloat16 widened exactly)
// ------------------------------------------------------------------------------------------

__device__ __forceinline__ float4 load_grad4(const float *g, long long i4)
{
    return __ldcs(reinterpret_cast<const float4 *>(g) + i4);
}
__device__ __forceinline__ float4 bf16x4_to_f32(uint2 u)
{
    float4 f;
    f.x = __uint_as_float(u.x << 16);
    f.y = __uint_as_float(u.x & 0xFFFF0000u);
    f.z = __uint_as_float(u.y << 16);
    f.w = __uint_as_float(u.y & 0xFFFF0000u);
    return f;
}
__device__ __forceinline__ float4 load_grad4(const __nv_bfloat16 *g, long long i4)
{
    return bf16x4_to_f32(__ldcs(reinterpret_cast<const uint2 *>(g) + i4));
}
__device__ __forceinline__ float load_grad1(const float *g, long long i) { return __ldcs(g + i); }
__device__ __forceinline__ float load_grad1(const __nv_bfloat16 *g, long long i)
{
    return __uint_as_float(((unsigned int)__ldcs(reinterpret_cast<const unsigned short *>(g) + i)) << 16);
}
__device__ __forceinline__ float4 smem_grad4(const float *g, int i4) { return reinterpret_cast<const float4 *>(g)[i4]; }
__device__ __forceinline__ float4 smem_grad4(const __nv_bfloat16 *g, int i4)
{
    return bf16x4_to_f32(reinterpret_cast<const uint2 *>(g)[i4]);
}

__device__ __forceinline__ ItemDev load_item(const ItemDev *items, int i)
{
    const uint4 *p = reinterpret_cast<const uint4 *>(items + i);
    union {
        uint4 q[4];
        ItemDev d;
    } u;
    u.q[0] = __ldg(p);
    u.q[1] = __ldg(p + 1);
    u.q[2] = __ldg(p + 2);
    u.q[3] = __ldg(p + 3);
    return u.d;
}

#ifdef RSDGC_DEBUG
// Bounds-checked build: every item of the CTA's range must lie inside the arenas, the key array and
// the layer table; called by all threads, the same answer in every thread.
template <int NTHREADS>
__device__ bool debug_items_ok(const ItemDev *items, int begin, int end, StatusDev *status)
{
    bool ok = begin >= 0 && end <= status->n_items;
    for (int i = begin + (int)threadIdx.x; ok && i < end; i += NTHREADS) {
        const ItemDev d = load_item(items, i);
        const int ntr = (d.R + d.nh - 1) / d.nh;
        ok = d.R >= 1 && d.W >= 1 && d.gbase >= 0 && d.gbase + (long long)(d.R - 1) * d.cols + d.W <= status->arena_elems &&
             d.kbase >= 0 && d.kbase + (long long)(ntr - 1) * d.TC + d.ntc <= status->keys_len && d.layer >= 0 &&
             d.layer < status->n_layers && (long long)d.R * d.P <= kItemElemsMax;  // (no variant's stage holds more)
    }
    return !__syncthreads_or(!debug_in_bounds(ok, status));
}
#endif

// Momentum correction (Eq. 12, first line): u = m * u_prev + g, product then sum, each rounded.
__device__ __forceinline__ float momentum_step(float m, float u_prev, float g)
{
    return __fadd_rn(__fmul_rn(m, u_prev), g);
}
__device__ __forceinline__ float4 momentum_step4(float m, float4 u, float4 g)
{
    return make_float4(momentum_step(m, u.x, g.x), momentum_step(m, u.y, g.y), momentum_step(m, u.z, g.z),
                       momentum_step(m, u.w, g.w));
}
__device__ __forceinline__ float4 add4_rn(float4 a, float4 b)
{
    return make_float4(__fadd_rn(a.x, b.x), __fadd_rn(a.y, b.y), __fadd_rn(a.z, b.z), __fadd_rn(a.w, b.w));
}

// The elements of a contiguous item beyond its last full group of `gran` elements (gran = 4
// or 8): plain loads and stores, results also placed in the shared-memory block.  With MOM the
// velocity u = m * u + g is updated in place and takes the gradient's role in v = r + u.
template <typename G, bool MOM>
__device__ __forceinline__ void k1_tail(const ItemDev &d, int gran, const G *__restrict__ grads,
                                        float *__restrict__ resid, float *sv, float *__restrict__ vel, float mom)
{
    const int n = d.R * d.W;
    const int e = (n / gran) * gran + threadIdx.x;
    if (e < n) {
        float g = load_grad1(grads, d.gbase + e);
        if (MOM) {
            g = momentum_step(mom, vel[d.gbase + e], g);
            vel[d.gbase + e] = g;
        }
        const float v = __fadd_rn(g, resid[d.gbase + e]);
        resid[d.gbase + e] = v;
        sv[e] = v;
    }
}

// ------------------------------------------------------------------------------------------
// k1_reg: register-staged variant (any alignment)
// ------------------------------------------------------------------------------------------

constexpr int kVecPerThread = (kItemElemsMax + 4 * kThreads - 1) / (4 * kThreads);  // 128-bit loads of g and of r per thread

struct K1RegShared {
    float v[2][kItemElemsMax];  // double buffer: tiles of item i are reduced while item i+1 streams in
    unsigned int hist[kL1Bins];
    FlushShared fs;
};

template <bool MOM>
struct K1Regs {
    float4 g[kVecPerThread], r[kVecPerThread];
    float4 u[MOM ? kVecPerThread : 1];  // velocity (momentum correction), staged like g and r
};

// Where each of a thread's kVecPerThread vector slots falls inside an item whose rows are
// separate in memory.  Slot u of thread t is vector i = u * kThreads + t of the shared-memory
// block (row pitch P / 4 vectors): row = i / (P/4), j = i % (P/4).  All items of a layer share
// P and the row stride, so the map is recomputed only when those change.
struct K1Map {
    int rel[kVecPerThread];           // row * (cols / 4) + j: vector offset from the item's start
    unsigned int rowj[kVecPerThread]; // row << 16 | j
    int P = -1, cols = -1;
};

__device__ __forceinline__ void k1_update_map(const ItemDev &d, K1Map &m)
{
    if (d.P == m.P && d.cols == m.cols) return;
    m.P = d.P;
    m.cols = d.cols;
    const int pv = d.P >> 2;
#pragma unroll
    for (int u = 0; u < kVecPerThread; ++u) {
        const int i = u * kThreads + threadIdx.x;
        const int row = fast_div(i, d.inv_pv), j = i - row * pv;
        m.rel[u] = row * (d.cols >> 2) + j;
        m.rowj[u] = ((unsigned int)row << 16) | (unsigned int)j;
    }
}

// Arena index of element e (0 <= e < R * P) of an item whose rows are not contiguous; the
// caller checks that the column lies inside the item.
__device__ __forceinline__ long long item_elem_index(const ItemDev &d, int e, bool *valid)
{
    const int row = fast_div(e, d.inv_p), col = e - row * d.P;
    *valid = col < d.W;
    return d.gbase + (long long)row * d.cols + col;
}

template <typename G, bool MOM>
__device__ __forceinline__ void k1_issue_loads(const ItemDev &d, const G *__restrict__ grads,
                                               const float *__restrict__ resid, const float *__restrict__ vel,
                                               K1Regs<MOM> &x, K1Map &m)
{
    const int tid = threadIdx.x;
    if (d.flags & kItemVec) {
        const long long base4 = d.gbase >> 2;
        if (d.flags & kItemFull) {
            const int nvec = (d.R * d.W) >> 2;
#pragma unroll
            for (int u = 0; u < kVecPerThread; ++u) {
                const int i = u * kThreads + tid;
                if (i < nvec) {
                    x.g[u] = load_grad4(grads, base4 + i);
                    x.r[u] = __ldcs(reinterpret_cast<const float4 *>(resid) + base4 + i);
                    if (MOM) x.u[u] = __ldcs(reinterpret_cast<const float4 *>(vel) + base4 + i);
                }
            }
        } else {
            k1_update_map(d, m);
            const unsigned int wv = (unsigned int)d.W >> 2, R = (unsigned int)d.R;
#pragma unroll
            for (int u = 0; u < kVecPerThread; ++u) {
                if ((m.rowj[u] >> 16) < R && (m.rowj[u] & 0xFFFFu) < wv) {
                    x.g[u] = load_grad4(grads, base4 + m.rel[u]);
                    x.r[u] = __ldcs(reinterpret_cast<const float4 *>(resid) + base4 + m.rel[u]);
                    if (MOM) x.u[u] = __ldcs(reinterpret_cast<const float4 *>(vel) + base4 + m.rel[u]);
                }
            }
        }
    } else {
        float *gs = reinterpret_cast<float *>(x.g), *rs = reinterpret_cast<float *>(x.r);
        float *us = reinterpret_cast<float *>(x.u);
        const int n = d.R * d.P;
#pragma unroll
        for (int u = 0; u < 4 * kVecPerThread; ++u) {
            const int e = u * kThreads + tid;
            if (e < n) {
                bool valid = true;
                const long long gi = (d.flags & kItemFull) ? d.gbase + e : item_elem_index(d, e, &valid);
                if (valid) {
                    gs[u] = load_grad1(grads, gi);
                    rs[u] = __ldcs(resid + gi);
                    if (MOM) us[u] = __ldcs(vel + gi);
                }
            }
        }
    }
}

template <bool MOM>
__device__ __forceinline__ void k1_add_store(const ItemDev &d, float *__restrict__ resid, float *__restrict__ vel,
                                             float mom, float *sv, K1Regs<MOM> &x, K1Map &m)
{
    const int tid = threadIdx.x;
    if (d.flags & kItemVec) {
        const long long base4 = d.gbase >> 2;
        const bool full = (d.flags & kItemFull) != 0;
        if (!full) k1_update_map(d, m);
        const int nvec = (d.R * d.W) >> 2;
        const unsigned int wv = (unsigned int)d.W >> 2, R = (unsigned int)d.R;
#pragma unroll
        for (int u = 0; u < kVecPerThread; ++u) {
            const int i = u * kThreads + tid;
            const bool valid = full ? (i < nvec) : ((m.rowj[u] >> 16) < R && (m.rowj[u] & 0xFFFFu) < wv);
            if (valid) {
                const long long gi = base4 + (full ? i : m.rel[u]);
                float4 g = x.g[u];
                if (MOM) {
                    g = momentum_step4(mom, x.u[u], g);
                    __stcs(reinterpret_cast<float4 *>(vel) + gi, g);
                }
                const float4 v = add4_rn(g, x.r[u]);
                __stcs(reinterpret_cast<float4 *>(resid) + gi, v);
                reinterpret_cast<float4 *>(sv)[i] = v;
            }
        }
    } else {
        const float *gs = reinterpret_cast<const float *>(x.g), *rs = reinterpret_cast<const float *>(x.r);
        const float *us = reinterpret_cast<const float *>(x.u);
        const int n = d.R * d.P;
#pragma unroll
        for (int u = 0; u < 4 * kVecPerThread; ++u) {
            const int e = u * kThreads + tid;
            if (e < n) {
                bool valid = true;
                const long long gi = (d.flags & kItemFull) ? d.gbase + e : item_elem_index(d, e, &valid);
                if (valid) {
                    float g = gs[u];
                    if (MOM) {
                        g = momentum_step(mom, us[u], g);
                        __stcs(vel + gi, g);
                    }
                    const float v = __fadd_rn(g, rs[u]);
                    __stcs(resid + gi, v);
                    sv[e] = v;
                }
            }
        }
    }
}

template <typename G, bool MOM>
__global__ void __launch_bounds__(kThreads)
k1_reg(const G *__restrict__ grads, float *__restrict__ resid, float *__restrict__ vel, float mom,
       uint32_t *__restrict__ keys, const LayerDev *__restrict__ layers, const ItemDev *__restrict__ items,
       const int32_t *__restrict__ cta_begin, unsigned int *hist, LayerState *state,
       const float *__restrict__ ratios, int32_t *counts, StatusDev *status, float alpha, unsigned int flags)
{
    extern __shared__ __align__(16) unsigned char k1_smem_raw[];
    K1RegShared &sh = *reinterpret_cast<K1RegShared *>(k1_smem_raw);
    const int begin = cta_begin[blockIdx.x], end = cta_begin[blockIdx.x + 1];
    if (begin >= end) return;
    const int tid = threadIdx.x;
#ifdef RSDGC_DEBUG
    if (!debug_items_ok<kThreads>(items, begin, end, status)) return;
#endif
    for (int b = tid; b < kL1Bins; b += kThreads) sh.hist[b] = 0;
    unsigned int nonfinite = 0;

    K1Regs<MOM> x;
    K1Map map;
    ItemDev cur = load_item(items, begin);
    FlushInfo finfo = load_flush_info(layers, ratios, cur.layer);
    k1_issue_loads<G, MOM>(cur, grads, resid, vel, x, map);
    int buf = 0;

    for (int it = begin; it < end; ++it) {
        const bool has_next = (it + 1 < end);
        ItemDev nxt = cur;
        if (has_next) nxt = load_item(items, it + 1);
        // v = g + r for the current item (its loads were issued one iteration ago)
        float *sv = sh.v[buf];
        k1_add_store<MOM>(cur, resid, vel, mom, sv, x, map);
        if ((cur.flags & (kItemVec | kItemFull)) == (kItemVec | kItemFull))
            k1_tail<G, MOM>(cur, 4, grads, resid, sv, vel, mom);
        // the next item's g and r stream in while this item's tiles are reduced
        if (has_next) k1_issue_loads<G, MOM>(nxt, grads, resid, vel, x, map);
        __syncthreads();
        nonfinite += item_tile_keys<kThreads>(cur, sv, keys, sh.hist, alpha);
        if (!has_next || nxt.layer != cur.layer) {
            k1_flush_layer<kThreads>(sh.hist, sh.fs, cur.layer, finfo, hist, state, counts, flags);
            if (has_next) finfo = load_flush_info(layers, ratios, nxt.layer);
        }
        cur = nxt;
        buf ^= 1;
    }
    if (nonfinite) {
        atomicAdd(&status->nonfinite, (unsigned long long)nonfinite);
        atomicOr(&status->flags, RSDGC_STATUS_NONFINITE);
    }
}

// ------------------------------------------------------------------------------------------
// k1_bulk: bulk-copy (TMA) pipelined variant
// ------------------------------------------------------------------------------------------

#ifndef RSDGC_BULK_STAGES
#define RSDGC_BULK_STAGES 2
#endif
#ifndef RSDGC_BULK_CTAS
#define RSDGC_BULK_CTAS 3
#endif
#ifndef RSDGC_BULK_THREADS
#define RSDGC_BULK_THREADS 256
#endif
constexpr int kBulkThreads = RSDGC_BULK_THREADS;
constexpr int kBulkCtasPerSm = RSDGC_BULK_CTAS;
constexpr int kBulkCtasPerSmMomentum = 2;  // a third block per stage: 110 KB of shared memory per CTA
// Shared-memory stages and elements per stage of a (gradient type, momentum) variant; loads run
// kStages - 1 items ahead.  The pass is bound by the bytes it keeps in flight, and an item costs a CTA
// about one memory round trip whatever it carries: with 2-byte gradients a stage of the same number of
// elements is a quarter smaller, so that variant may take more elements per stage within the same
// shared memory.  The plan cuts its items to bulk_item_elems().
template <typename G, bool MOM>
struct BulkCfg {
    static constexpr int kStages = RSDGC_BULK_STAGES;
    static constexpr int kElems = kItemElems;
};
template <>
struct BulkCfg<__nv_bfloat16, false> {
    static constexpr int kStages = RSDGC_BF16_STAGES;
    static constexpr int kElems = kItemElemsBf16;
};
constexpr unsigned int kSpinLimit = 1u << 22;  // bounded mbarrier waits
constexpr int kOverlapPrev = 1;  // k1_bulk: the previous kernel in the stream is another worker's first pass
constexpr int kOverlapNext = 2;  // k1_bulk: the next one is

template <typename G, bool MOM>
struct K1BulkShared {
    static constexpr int kStages = BulkCfg<G, MOM>::kStages, kElems = BulkCfg<G, MOM>::kElems;
    __align__(128) float r[kStages][kElems];  // residual block; becomes v in place
    __align__(128) G g[kStages][kElems];      // gradient block
    __align__(128) float u[MOM ? kStages : 1][MOM ? kElems : 4];  // velocity block, updated in place
    unsigned int hist[kL1Bins];
    __align__(8) unsigned long long full[kStages];  // mbarriers: stage loaded
    FlushShared fs;
    int dead_at;  // first item whose loads did not arrive within the bound (see k1_bulk)
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(unsigned long long *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait; returns false if the barrier did not complete within `limit` polls.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned long long *bar, uint32_t parity,
                                                  unsigned int limit = kSpinLimit)
{
    for (unsigned int i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_load(void *dst_smem, const void *src_gmem, uint32_t bytes, unsigned long long *bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst_smem)),
                 "l"(__cvta_generic_to_global(src_gmem)), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void bulk_store(void *dst_gmem, const void *src_smem, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(__cvta_generic_to_global(dst_gmem)),
                 "r"(smem_u32(src_smem)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
template <int N>
__device__ __forceinline__ void bulk_wait_all()
{
    asm volatile("cp.async.bulk.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Elements of the shared-memory block covered by bulk copies: R rows of pitch P for separate
// rows (the columns W..P of a narrower last chunk hold stale values that are never stored),
// the largest multiple of the 16-byte granule for a contiguous run (the rest goes through
// k1_tail).
template <typename G>
__device__ __forceinline__ int bulk_elems(const ItemDev &d)
{
    constexpr int gran = (sizeof(G) == 2) ? 8 : 4;
    return (d.flags & kItemFull) ? ((d.R * d.W) / gran) * gran : d.R * d.P;
}

// One thread: arm the stage's barrier and start the copies of g and r (and u) for an item.
template <typename G, bool MOM>
__device__ __forceinline__ void bulk_issue_item(const ItemDev &d, const G *grads, const float *resid,
                                                const float *vel, float *sr, G *sg, float *su,
                                                unsigned long long *bar)
{
    constexpr uint32_t per_elem = sizeof(float) + sizeof(G) + (MOM ? sizeof(float) : 0);
    if (d.flags & kItemFull) {
        const int n = bulk_elems<G>(d);
        if (n > 0) {
            mbar_arrive_expect_tx(bar, (uint32_t)n * per_elem);
            bulk_load(sr, resid + d.gbase, (uint32_t)(n * sizeof(float)), bar);
            bulk_load(sg, grads + d.gbase, (uint32_t)(n * sizeof(G)), bar);
            if (MOM) bulk_load(su, vel + d.gbase, (uint32_t)(n * sizeof(float)), bar);
        } else {
            mbar_arrive_expect_tx(bar, 0);
        }
    } else {
        mbar_arrive_expect_tx(bar, (uint32_t)(d.R * d.W) * per_elem);
        for (int row = 0; row < d.R; ++row) {
            const long long gi = d.gbase + (long long)row * d.cols;
            bulk_load(sr + row * d.P, resid + gi, (uint32_t)(d.W * sizeof(float)), bar);
            bulk_load(sg + row * d.P, grads + gi, (uint32_t)(d.W * sizeof(G)), bar);
            if (MOM) bulk_load(su + row * d.P, vel + gi, (uint32_t)(d.W * sizeof(float)), bar);
        }
    }
}

template <typename G, bool MOM>
__global__ void __launch_bounds__(kBulkThreads, MOM ? kBulkCtasPerSmMomentum : kBulkCtasPerSm)
k1_bulk(const G *__restrict__ grads, float *__restrict__ resid, float *__restrict__ vel, float mom,
        uint32_t *__restrict__ keys, const LayerDev *__restrict__ layers, const ItemDev *__restrict__ items,
        const int32_t *__restrict__ cta_begin, unsigned int *hist, LayerState *state,
        const float *__restrict__ ratios, int32_t *counts, StatusDev *status, float alpha, unsigned int flags,
        int overlap)
{
    extern __shared__ __align__(128) unsigned char k1_bulk_smem_raw[];
    K1BulkShared<G, MOM> &sh = *reinterpret_cast<K1BulkShared<G, MOM> *>(k1_bulk_smem_raw);
    constexpr int kStages = BulkCfg<G, MOM>::kStages, kLookahead = kStages - 1;
    const int begin = cta_begin[blockIdx.x], end = cta_begin[blockIdx.x + 1];
    const bool wait_late = (overlap & kOverlapPrev) != 0;
    if (begin >= end) {
        if (wait_late) grid_dependency_wait();
        return;
    }
    const int tid = threadIdx.x;
#ifdef RSDGC_DEBUG
    if (!debug_items_ok<kBulkThreads>(items, begin, end, status)) {  // nothing is loaded or stored
        if (wait_late) grid_dependency_wait();
        return;
    }
#endif
    for (int b = tid; b < kL1Bins; b += kBulkThreads) sh.hist[b] = 0;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) mbar_init(&sh.full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    __syncthreads();
    // Launched with programmatic stream serialization: everything above overlapped the tail of the
    // previous kernel in the stream.  Normally nothing below may run before that kernel has
    // completed.  kOverlapPrev: the previous kernel is the first pass of another worker of the same
    // call, which touches none of this worker's buffers or tables and has itself passed its own wait
    // (so everything older is complete): this launch runs alongside that kernel's last CTAs, and
    // waits for it only before it exits, which keeps completion transitive along the stream.
    // kOverlapNext: the next kernel is such a first pass; it may be scheduled as soon as CTAs of
    // this one leave.  (Other successors are not released early: their few CTAs would crowd onto
    // the first SMs that become free.)
    if (!wait_late) grid_dependency_wait();
    if (overlap & kOverlapNext) grid_dependency_launch_next();
    // prologue: the first kLookahead items start loading
    if (tid == 0) {
        for (int j = 0; j < kLookahead && begin + j < end; ++j) {
            const ItemDev d = load_item(items, begin + j);
            bulk_issue_item<G, MOM>(d, grads, resid, vel, sh.r[j % kStages], sh.g[j % kStages],
                                    sh.u[MOM ? j % kStages : 0], &sh.full[j % kStages]);
        }
    }
    unsigned int nonfinite = 0;
    // `dead` (the same value in every thread): a bounded wait gave up.  From then on the CTA moves no
    // more data: the items it has not finished keep their old accumulator (v is not stored), no further
    // loads are issued, no keys are written; it still takes part in the layers' histogram tickets so
    // that the plan's tables are left consistent, and raises RSDGC_STATUS_TIMEOUT (the payload of this
    // call is then invalid).
    bool dead = false;
    ItemDev cur = load_item(items, begin);
    FlushInfo finfo = load_flush_info(layers, ratios, cur.layer);
    // the producer thread keeps the descriptor of the next item to load one iteration ahead
    ItemDev ahead = cur;
    if (tid == 0 && begin + kLookahead < end) ahead = load_item(items, begin + kLookahead);

    for (int it = begin; it < end; ++it) {
        const int rel = it - begin;
        const int stage = rel % kStages;
        const bool has_next = (it + 1 < end);
        ItemDev nxt = cur;
        if (has_next) nxt = load_item(items, it + 1);

        // ---- wait for this item's blocks (bounded), form v in place
        float *sr = sh.r[stage];
        const G *sg = sh.g[stage];
        float *su = sh.u[MOM ? stage : 0];
        const int nb = bulk_elems<G>(cur);
        bool arrived = true;
        if (!dead) {
            arrived = mbar_wait_bounded(&sh.full[stage], (uint32_t)((rel / kStages) & 1));
            const int nvec = nb >> 2;
            for (int i = tid; i < nvec; i += kBulkThreads) {
                float4 g = smem_grad4(sg, i);
                if (MOM) {  // u = m * u + g takes the gradient's place (Eq. 12, first line)
                    g = momentum_step4(mom, reinterpret_cast<const float4 *>(su)[i], g);
                    reinterpret_cast<float4 *>(su)[i] = g;
                }
                reinterpret_cast<float4 *>(sr)[i] = add4_rn(g, reinterpret_cast<const float4 *>(sr)[i]);
            }
            fence_async_smem();  // the bulk stores below read what the threads just wrote
            // the elements beyond the last 16-byte group of a contiguous item: plain loads and stores of
            // g and r themselves, so they are right whether or not the bulk copies arrived
            if (cur.flags & kItemFull) k1_tail<G, MOM>(cur, (sizeof(G) == 2) ? 8 : 4, grads, resid, sr, vel, mom);
        }
        // the barrier that orders the threads' writes before the bulk store also tells every thread
        // whether some thread's wait ran out (nothing of the item has left shared memory yet)
        if (__syncthreads_or(!arrived)) {
            if (!dead && tid == 0) sh.dead_at = it;
            dead = true;
        }
        if (!dead) {
            if (tid == 0) {
                if (cur.flags & kItemFull) {
                    if (nb > 0) {
                        bulk_store(resid + cur.gbase, sr, (uint32_t)(nb * sizeof(float)));
                        if (MOM) bulk_store(vel + cur.gbase, su, (uint32_t)(nb * sizeof(float)));
                    }
                } else {
                    for (int row = 0; row < cur.R; ++row) {
                        const long long gi = cur.gbase + (long long)row * cur.cols;
                        bulk_store(resid + gi, sr + row * cur.P, (uint32_t)(cur.W * sizeof(float)));
                        if (MOM) bulk_store(vel + gi, su + row * cur.P, (uint32_t)(cur.W * sizeof(float)));
                    }
                }
                bulk_commit();
                // ---- producer: item it + kLookahead goes into the stage item it - 1 used.  Every
                // thread finished that item's tiles before the barrier above, and its bulk store
                // has finished reading shared memory once only the store just committed is pending.
                // (Issued earlier, before this item is waited for, so that a CTA has two items in flight:
                // measured 7 % slower; the memory system is already saturated by one item per CTA.)
                if (it + kLookahead < end) {
                    bulk_wait_read<1>();
                    const int ps = (rel + kLookahead) % kStages;
                    bulk_issue_item<G, MOM>(ahead, grads, resid, vel, sh.r[ps], sh.g[ps], sh.u[MOM ? ps : 0],
                                            &sh.full[ps]);
                    if (it + 1 + kLookahead < end) ahead = load_item(items, it + 1 + kLookahead);
                }
            }
            // ---- NSI of every tile of the item
            nonfinite += item_tile_keys<kBulkThreads>(cur, sr, keys, sh.hist, alpha);
        }
        if (!has_next || nxt.layer != cur.layer) {
            k1_flush_layer<kBulkThreads>(sh.hist, sh.fs, cur.layer, finfo, hist, state, counts, flags);
            if (has_next) finfo = load_flush_info(layers, ratios, nxt.layer);
        }
        cur = nxt;
    }
    if (dead && tid == 0) {
        // the loads already started still target this CTA's shared memory: give them the same bounded
        // chance to land before the CTA leaves
        // (when the CTA gave up at item d, items d .. d + kLookahead - 1 had been started)
        for (int j = sh.dead_at; j < sh.dead_at + kLookahead && j < end; ++j)
            (void)mbar_wait_bounded(&sh.full[(j - begin) % kStages], (uint32_t)(((j - begin) / kStages) & 1));
    }
    if (tid == 0) bulk_wait_all<0>();  // all stores of this CTA have landed before it exits
    if (nonfinite) {
        atomicAdd(&status->nonfinite, (unsigned long long)nonfinite);
        atomicOr(&status->flags, RSDGC_STATUS_NONFINITE);
    }
    if (dead && tid == 0) atomicOr(&status->flags, RSDGC_STATUS_TIMEOUT);
    if (wait_late) grid_dependency_wait();
}

// ------------------------------------------------------------------------------------------
// Self-test of the bounded wait: one warp arms a barrier for 16 bytes that no copy will ever
// deliver (nothing is in flight, before or after), polls it `polls` times with the same helper the
// first pass uses, and reports the give-up through the status word like the first pass does.
// ------------------------------------------------------------------------------------------

__global__ void k_selftest_bounded_wait(StatusDev *status, unsigned int polls)
{
    __shared__ __align__(8) unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    if (threadIdx.x == 0) mbar_arrive_expect_tx(&bar, 16);
    __syncwarp();
    const bool arrived = mbar_wait_bounded(&bar, 0, polls);
    if (__syncthreads_or(!arrived) && threadIdx.x == 0) atomicOr(&status->flags, RSDGC_STATUS_TIMEOUT);
    __syncthreads();
    if (threadIdx.x == 0) asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_u32(&bar)) : "memory");
}

cudaError_t launch_selftest_bounded_wait(rsdgc_plan *p, unsigned int polls, cudaStream_t s)
{
    k_selftest_bounded_wait<<<1, 32, 0, s>>>(p->d_status, polls);
    count_launch(1);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------

template <typename K>
static cudaError_t allow_smem(K kernel, size_t bytes)
{
    return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
}

// Raises the kernels' dynamic shared-memory limits, once per device (the attribute belongs to the
// device's context); a failure is not cached, so a later call tries again instead of silently
// launching nothing.  The caller has made the plan's device current.
static cudaError_t configure_once()
{
    constexpr int kMaxDevices = 64;
    static bool done[kMaxDevices] = {};
    int dev = 0;
    cudaError_t ed = cudaGetDevice(&dev);
    if (ed != cudaSuccess) return ed;
    const bool tracked = dev >= 0 && dev < kMaxDevices;
    if (tracked && done[dev]) return cudaSuccess;
    const cudaError_t result = [] {
        cudaError_t e = allow_smem(k1_reg<float, false>, sizeof(K1RegShared));
        if (e == cudaSuccess) e = allow_smem(k1_reg<float, true>, sizeof(K1RegShared));
        if (e == cudaSuccess) e = allow_smem(k1_reg<__nv_bfloat16, false>, sizeof(K1RegShared));
        if (e == cudaSuccess) e = allow_smem(k1_reg<__nv_bfloat16, true>, sizeof(K1RegShared));
        if (e == cudaSuccess) e = allow_smem(k1_bulk<float, false>, sizeof(K1BulkShared<float, false>));
        if (e == cudaSuccess) e = allow_smem(k1_bulk<float, true>, sizeof(K1BulkShared<float, true>));
        if (e == cudaSuccess) e = allow_smem(k1_bulk<__nv_bfloat16, false>, sizeof(K1BulkShared<__nv_bfloat16, false>));
        if (e == cudaSuccess) e = allow_smem(k1_bulk<__nv_bfloat16, true>, sizeof(K1BulkShared<__nv_bfloat16, true>));
        return e;
    }();
    if (tracked) done[dev] = (result == cudaSuccess);
    return result;
}

int k1_bulk_ctas_per_sm(bool momentum) { return momentum ? kBulkCtasPerSmMomentum : kBulkCtasPerSm; }

// Elements an item of the first pass may hold for this gradient type (one stage of the variant's
// shared memory).
int bulk_item_elems(int dtype, bool momentum)
{
    return (dtype == RSDGC_BF16 && !momentum) ? BulkCfg<__nv_bfloat16, false>::kElems : kItemElems;
}

// Resident CTAs per SM of the register-staged kernel on the current device.
int k1_reg_ctas_per_sm(int dtype, bool momentum)
{
    int n = 0;
    cudaError_t e = configure_once();
    const size_t smem = sizeof(K1RegShared);
    if (e == cudaSuccess) {
        if (dtype == RSDGC_BF16)
            e = momentum ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k1_reg<__nv_bfloat16, true>, kThreads, smem)
                         : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k1_reg<__nv_bfloat16, false>, kThreads, smem);
        else
            e = momentum ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k1_reg<float, true>, kThreads, smem)
                         : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, k1_reg<float, false>, kThreads, smem);
    }
    if (e != cudaSuccess || n < 1) {
        (void)cudaGetLastError();
        n = 2;
    }
    return n;
}

template <typename G, bool MOM>
static cudaError_t launch_k1_typed(rsdgc_plan *p, uint32_t *hist, LayerState *state, const void *grads, float *resid,
                                   float *vel, float mom, const float *ratios, int32_t *counts, uint32_t *keys,
                                   cudaStream_t s, int *launches, int overlap)
{
    const G *g = reinterpret_cast<const G *>(grads);
    cudaError_t e = cudaSuccess;
    if (p->n_items_bulk > 0) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)p->grid_bulk);
        cfg.blockDim = dim3(kBulkThreads);
        cfg.dynamicSmemBytes = sizeof(K1BulkShared<G, MOM>);
        cfg.stream = s;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        const LayerDev *layers = p->d_layers;
        const ItemDev *items = p->d_items;
        const int32_t *cta_begin = p->d_cta_begin_bulk;
        e = cudaLaunchKernelEx(&cfg, k1_bulk<G, MOM>, g, resid, vel, mom, keys, layers, items, cta_begin, hist,
                               state, ratios, counts, p->d_status, p->alpha, (unsigned int)p->flags, overlap);
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    if (p->n_items_reg > 0) {
        k1_reg<G, MOM><<<p->grid_reg, kThreads, sizeof(K1RegShared), s>>>(
            g, resid, vel, mom, keys, p->d_layers, p->d_items + p->n_items_bulk, p->d_cta_begin_reg, hist,
            state, ratios, counts, p->d_status, p->alpha, p->flags);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
        ++*launches;
    }
    return e;
}

// vel == nullptr: plain accumulation v = g + r; otherwise u = mom * u + g, v = r + u.
// after_sibling / before_sibling: the kernel launched just before / next on this stream is the first
// pass of another worker of the same call (see k1_bulk); only honoured when a first pass is a
// single bulk-copy kernel.
// Returns the first error of the kernel configuration or of a launch: the selection kernels must
// not run on keys no first pass has written.
cudaError_t launch_accumulate_nsi(rsdgc_plan *p, uint32_t *hist, LayerState *state, const void *grads, float *resid,
                                  float *vel, float mom, const float *ratios, int32_t *counts, uint32_t *keys,
                                  cudaStream_t s, bool after_sibling, bool before_sibling)
{
    int overlap = 0;
    if (p->n_items_reg == 0)  // the register-staged kernel is launched without overlap
        overlap = (after_sibling ? kOverlapPrev : 0) | (before_sibling ? kOverlapNext : 0);
    int launches = 0;
    cudaError_t e = configure_once();
    if (e != cudaSuccess) return e;
    if (p->dtype == RSDGC_BF16) {
        if (vel) e = launch_k1_typed<__nv_bfloat16, true>(p, hist, state, grads, resid, vel, mom, ratios, counts, keys, s, &launches, overlap);
        else e = launch_k1_typed<__nv_bfloat16, false>(p, hist, state, grads, resid, vel, mom, ratios, counts, keys, s, &launches, overlap);
    } else {
        if (vel) e = launch_k1_typed<float, true>(p, hist, state, grads, resid, vel, mom, ratios, counts, keys, s, &launches, overlap);
        else e = launch_k1_typed<float, false>(p, hist, state, grads, resid, vel, mom, ratios, counts, keys, s, &launches, overlap);
    }
    count_launch(launches);
    return e;
}

}  // namespace rsdgc
