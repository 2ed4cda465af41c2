// Kernel of rsdgc_decompress_accumulate(): scatter-add of several workers' payloads into the
// dense gradient arena (Eq. 12 third line / Eq. 2 Sync).
//
// One launch handles up to kMaxWorkersPerLaunch workers.  A CTA owns one chunk of 16384
// consecutive tile indices of one layer.  Every worker's index list is ascending inside a
// layer (rsdgc_compress() writes it that way), so the entries of a worker that fall into the
// chunk are one contiguous run, found with a 32-way search by one warp per worker.  The CTA
// then applies the workers one after the other, with a barrier in between: every element of the
// dense arena is only ever touched by the CTA that owns its tile, in worker order, with plain
// read-modify-write, so the binary32 sums are reproducible (no atomics) although all workers
// are processed by one launch.
//
// The ASSIGN variant first stores +0 to every element of the chunk's tiles (the dense arena then
// needs no separate zero fill, and the read-modify-writes that follow find their lines in L2),
// so that dense = scale * sum of the workers' payloads.
#include <cuda_bf16.h>

#include "device_utils.cuh"

namespace rsdgc {

constexpr int kMaxWorkersPerLaunch = 16;
constexpr int kScatterBatch = 9;  // independent entries in flight per thread (one 3x3 tile's worth)

struct WorkerPayloads {
    const int32_t *idx[kMaxWorkersPerLaunch];
    const void *val[kMaxWorkersPerLaunch];  // binary32 or bfloat16 values
    const int32_t *counts[kMaxWorkersPerLaunch];
    long long idx_cap, val_cap;  // entries every worker's idx / val buffer holds
    int n_workers;
};

struct DecompressShared {
    long long idx_off[kMaxWorkersPerLaunch];  // payload offsets of the chunk's layer, per worker
    long long val_off[kMaxWorkersPerLaunch];
    int lo[kMaxWorkersPerLaunch], hi[kMaxWorkersPerLaunch];  // the worker's entries inside the chunk
    long long gbase[kThreads];  // per tile of the current block: arena position of its element (0, 0), or -1
    int hw[kThreads];           // rows << 16 | columns of the tile inside the layer (clipped)
};

// First position in a[0, n) whose value is >= key (a ascending); all 32 lanes of the warp take
// part and return the same result.  Each step probes 32 positions, shrinking the range 33-fold.
__device__ __forceinline__ int warp_lower_bound(const int32_t *a, int n, int key)
{
    const int lane = threadIdx.x & 31;
    int lo = 0, hi = n;  // answer in [lo, hi]
    while (hi - lo > 0) {
        const int span = hi - lo;
        const int step = (span + 32) / 33;  // >= 1
        const int pos = lo + (lane + 1) * step - 1;  // probe positions lo+step-1, lo+2step-1, ...
        const bool below = (pos < hi) ? (__ldg(a + pos) < key) : false;  // a[pos] < key
        const unsigned int m = __ballot_sync(0xFFFFFFFFu, below);
        const int nb = __popc(m);  // ascending array: the lanes with a[pos] < key are a prefix
        const int new_lo = lo + nb * step;
        const int new_hi = (nb < 32) ? min(hi, lo + (nb + 1) * step - 1) : hi;
        lo = min(new_lo, hi);
        hi = max(new_hi, lo);
    }
    return lo;
}

// Stores +0 to dense[begin, end): scalar stores up to the first 16-byte boundary and after the
// last one, 128-bit stores in between; all threads of the CTA take part.
__device__ __forceinline__ void zero_span(float *__restrict__ dense, long long begin, long long end)
{
    if (end <= begin) return;
    const int tid = threadIdx.x;
    const long long body0 = min(end, (begin + 3) & ~3ll), body1 = max(body0, end & ~3ll);
    if (begin + tid < body0) dense[begin + tid] = 0.0f;
    if (body1 + tid < end) dense[body1 + tid] = 0.0f;
    float4 *d4 = reinterpret_cast<float4 *>(dense + body0);
    const long long n4 = (body1 - body0) >> 2;
    for (long long i = tid; i < n4; i += kThreads) d4[i] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
}

// +0 to every element of the tiles [c.start, c.start + c.n) of layer L: a partial first tile
// row, a contiguous run of whole tile rows, a partial last tile row.
__device__ __forceinline__ void zero_chunk(float *__restrict__ dense, const LayerDev &L, const Chunk &c)
{
    const int t_last = c.start + c.n - 1;
    const int tr0 = c.start / L.TC, tc0 = c.start - tr0 * L.TC;
    const int tr1 = t_last / L.TC, tc1 = t_last - tr1 * L.TC;
    const bool head_partial = tc0 != 0, tail_partial = tc1 != L.TC - 1;
    auto rows_of = [&](int tr, long long cb, long long ce) {  // columns [cb, ce) of the rows of tile row tr
        const long long r_end = min((long long)L.rows, ((long long)tr + 1) * L.nh);
        for (long long r = (long long)tr * L.nh; r < r_end; ++r)
            zero_span(dense, L.elem_off + r * L.cols + cb, L.elem_off + r * L.cols + ce);
    };
    if (tr0 == tr1 && (head_partial || tail_partial)) {
        rows_of(tr0, (long long)tc0 * L.nw, min((long long)L.cols, ((long long)tc1 + 1) * L.nw));
        return;
    }
    if (head_partial) rows_of(tr0, (long long)tc0 * L.nw, L.cols);
    if (tail_partial) rows_of(tr1, 0, min((long long)L.cols, ((long long)tc1 + 1) * L.nw));
    const long long full0 = tr0 + (head_partial ? 1 : 0), full1 = tr1 - (tail_partial ? 1 : 0);  // inclusive
    if (full1 >= full0)
        zero_span(dense, L.elem_off + full0 * L.nh * L.cols,
                  L.elem_off + min((long long)L.rows, (full1 + 1) * L.nh) * L.cols);
}

template <bool ASSIGN, bool BF16VAL>
__global__ void __launch_bounds__(kThreads)
k_decompress(const __grid_constant__ WorkerPayloads wp, const LayerDev *__restrict__ layers,
             const Chunk *__restrict__ chunks, float scale, float *__restrict__ dense, StatusDev *status)
{
    __shared__ DecompressShared sh;
    const Chunk c = chunks[blockIdx.x];
    const LayerDev L = layers[c.layer];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int W = wp.n_workers;
    if (!RSDGC_CHECKED((int)blockIdx.x < status->n_chunks && c.layer >= 0 && c.layer < status->n_layers && c.start >= 0 &&
                           c.start + c.n <= L.K && L.elem_off + L.rows * L.cols <= status->arena_elems, status))
        return;
    if (ASSIGN) zero_chunk(dense, L, c);  // made visible to the whole CTA by the barrier below

    // ---- per worker (one warp each, round-robin): payload offsets of this layer = sums of the
    // counts of the preceding layers, and the run of entries that falls into the chunk
    for (int w = warp; w < W; w += kThreads / 32) {
        long long si = 0, sv = 0;
        for (int l = lane; l < c.layer; l += 32) {
            long long k = wp.counts[w][l];
            if (k < 0) k = 0;
            si += k;
            sv += k * layers[l].slot;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            si += __shfl_xor_sync(0xFFFFFFFFu, si, d);
            sv += __shfl_xor_sync(0xFFFFFFFFu, sv, d);
        }
        long long kk = wp.counts[w][c.layer];
        if (kk < 0) kk = 0;
        // a payload cut short by its buffers (RSDGC_STATUS_PAYLOAD_OVERFLOW) holds, of this layer,
        // only the tiles that fit both of them: the rest was neither written nor sent
        kk = min(kk, max(0ll, wp.idx_cap - si));
        kk = min(kk, max(0ll, (wp.val_cap - sv) / layers[c.layer].slot));
        const int k = (int)kk;
        const int32_t *a = wp.idx[w] + si;
        const int lo = warp_lower_bound(a, k, c.start);
        const int hi = lo + warp_lower_bound(a + lo, k - lo, c.start + c.n);
        if (lane == 0) {
            sh.idx_off[w] = si;
            sh.val_off[w] = sv;
            sh.lo[w] = lo;
            sh.hi[w] = hi;
        }
    }
    __syncthreads();

    const int slot = L.slot, nw = L.nw;
    const long long cols = L.cols;
    for (int w = 0; w < W; ++w) {
        const int lo = sh.lo[w];
        const int n_run = sh.hi[w] - lo;  // the worker's tiles inside this chunk
        const int32_t *idx = wp.idx[w] + sh.idx_off[w] + lo;
        const long long v_first = sh.val_off[w] + (long long)lo * slot;
        const float *val = reinterpret_cast<const float *>(wp.val[w]) + v_first;
        const __nv_bfloat16 *val16 = reinterpret_cast<const __nv_bfloat16 *>(wp.val[w]) + v_first;
        // blocks of kThreads tiles: every thread first resolves one tile (index load, tile row / column,
        // clipping) into shared memory; the value loop then needs one division by the slot size per
        // value and its loads do not depend on the index list
        for (int t0 = 0; t0 < n_run; t0 += kThreads) {
            long long gb = -1;
            int hw = 0;
            if (t0 + tid < n_run) {
                const int tile = __ldg(idx + t0 + tid);
                if (tile >= c.start && tile < c.start + c.n) {  // always true for ascending lists
                    const int tr = tile / L.TC, tc = tile - tr * L.TC;
                    const long long i0 = (long long)tr * L.nh, j0 = (long long)tc * L.nw;
                    gb = L.elem_off + i0 * cols + j0;
                    hw = ((int)min((long long)L.nh, L.rows - i0) << 16) | (int)min((long long)L.nw, cols - j0);
                }
            }
            sh.gbase[tid] = gb;
            sh.hw[tid] = hw;
            __syncthreads();
            const int n_vals = min(kThreads, n_run - t0) * slot;
            const long long v0 = (long long)t0 * slot;
            for (int j0 = 0; j0 < n_vals; j0 += kThreads * kScatterBatch) {
                long long ga[kScatterBatch];
                float pv[kScatterBatch], dv[kScatterBatch];
#pragma unroll
                for (int u = 0; u < kScatterBatch; ++u) {
                    const int j = j0 + u * kThreads + tid;
                    ga[u] = -1;
                    pv[u] = 0.0f;
                    if (j < n_vals) {
                        int q, el, a, b;
                        divmod_small(j, slot, &q, &el);
                        divmod_small(el, nw, &a, &b);
                        const long long g0 = sh.gbase[q];
                        const int thw = sh.hw[q];
                        if (g0 >= 0 && a < (thw >> 16) && b < (thw & 0xFFFF) &&
                            RSDGC_CHECKED(g0 + a * cols + b < status->arena_elems, status)) {
                            ga[u] = g0 + a * cols + b;
                            pv[u] = BF16VAL ? __bfloat162float(val16[v0 + j]) : __ldg(val + v0 + j);
                        }
                    }
                }
#pragma unroll
                for (int u = 0; u < kScatterBatch; ++u) dv[u] = (ga[u] >= 0) ? dense[ga[u]] : 0.0f;
#pragma unroll
                for (int u = 0; u < kScatterBatch; ++u)
                    if (ga[u] >= 0) dense[ga[u]] = __fadd_rn(dv[u], __fmul_rn(scale, pv[u]));
            }
            __syncthreads();  // the tables are reused; the next worker may touch the same elements
        }
    }
}

// Applies workers [0, n_workers) in order (after the zero fill of the ASSIGN variant); groups of kMaxWorkersPerLaunch go into one launch
// each, and the stream orders the groups.
cudaError_t launch_decompress(rsdgc_plan *p, int n_workers, const int32_t *const *idx, const void *const *val,
                              const int32_t *const *counts, long long idx_cap, long long val_cap, float scale,
                              float *dense, bool assign, cudaStream_t s)
{
    const int n_chunks = (int)p->chunks.size();
    const bool half = (p->flags & RSDGC_PAYLOAD_BF16) != 0;
    if (assign && n_workers == 0) {  // nothing was sent: the result is all +0
        k_decompress<true, false><<<n_chunks, kThreads, 0, s>>>(WorkerPayloads{}, p->d_layers, p->d_chunks, scale, dense,
                                                                p->d_status);
        count_launch(1);
    }
    for (int w0 = 0; w0 < n_workers; w0 += kMaxWorkersPerLaunch) {
        WorkerPayloads wp{};
        wp.n_workers = n_workers - w0 < kMaxWorkersPerLaunch ? n_workers - w0 : kMaxWorkersPerLaunch;
        wp.idx_cap = idx_cap;
        wp.val_cap = val_cap;
        for (int w = 0; w < wp.n_workers; ++w) {
            wp.idx[w] = idx[w0 + w];
            wp.val[w] = val[w0 + w];
            wp.counts[w] = counts[w0 + w];
        }
        const bool zero_first = assign && w0 == 0;
        auto kernel = zero_first ? (half ? k_decompress<true, true> : k_decompress<true, false>)
                                 : (half ? k_decompress<false, true> : k_decompress<false, false>);
        kernel<<<n_chunks, kThreads, 0, s>>>(wp, p->d_layers, p->d_chunks, scale, dense, p->d_status);
        count_launch(1);
    }
    return cudaGetLastError();
}

}  // namespace rsdgc
