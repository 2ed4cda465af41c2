// Host side of the RS-DGC library: plan tables, argument checks, the C entry points.
#include <algorithm>
#include <atomic>
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "rsdgc_internal.cuh"

// NVTX ranges around the entry points that enqueue device work (visible in Nsight timelines; without
// a profiler attached a range costs a pointer check).  Compiled out without RSDGC_NVTX.
#ifdef RSDGC_NVTX
#include <nvtx3/nvToolsExt.h>
namespace {
struct NvtxRange {
    explicit NvtxRange(const char *name) { nvtxRangePushA(name); }
    ~NvtxRange() { nvtxRangePop(); }
};
}  // namespace
#define RSDGC_RANGE(name) NvtxRange rsdgc_nvtx_range_(name)
#else
#define RSDGC_RANGE(name) ((void)0)
#endif

using namespace rsdgc;

namespace {

thread_local int g_last_cuda_error = 0;
std::atomic<long long> g_launches{0};

int cuda_fail(cudaError_t e)
{
    g_last_cuda_error = (int)e;
    return RSDGC_ERR_CUDA;
}

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    cudaError_t err = cudaSuccess;
    explicit DeviceGuard(int dev)
    {
        err = cudaGetDevice(&prev);
        if (err == cudaSuccess && prev != dev) {
            err = cudaSetDevice(dev);
            switched = (err == cudaSuccess);
        }
    }
    ~DeviceGuard()
    {
        if (switched) cudaSetDevice(prev);
    }
};

inline int64_t ceil_div64(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline int64_t round_up64(int64_t a, int64_t b) { return ceil_div64(a, b) * b; }
inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

template <typename T>
cudaError_t upload(T **dst, const std::vector<T> &src)
{
    size_t bytes = (src.empty() ? 1 : src.size()) * sizeof(T);
    cudaError_t e = cudaMalloc((void **)dst, bytes);
    if (e != cudaSuccess) return e;
    if (!src.empty()) e = cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice);
    return e;
}

template <typename T>
cudaError_t alloc_zero(T **dst, size_t count)
{
    size_t bytes = (count ? count : 1) * sizeof(T);
    cudaError_t e = cudaMalloc((void **)dst, bytes);
    if (e != cudaSuccess) return e;
    return cudaMemset(*dst, 0, bytes);
}

void free_device_tables(rsdgc_plan *p)
{
    cudaFree(p->d_layers);
    cudaFree(p->d_items);
    cudaFree(p->d_cta_begin_bulk);
    cudaFree(p->d_cta_begin_reg);
    cudaFree(p->d_chunks);
    cudaFree(p->d_tail_slices);
    cudaFree(p->d_echunks);
    cudaFree(p->d_state);
    cudaFree(p->d_hist);
    cudaFree(p->d_chunk_cnt);
    cudaFree(p->d_chunk_sfx);
    cudaFree(p->d_codes);
    cudaFree(p->d_survivors);
    cudaFree(p->d_rstate);
    cudaFree(p->d_status);
    for (rsdgc_plan::LaneScratch &x : p->extra_lanes) {
        cudaFree(x.state);
        cudaFree(x.hist);
        cudaFree(x.codes);
        cudaFree(x.chunk_cnt);
        cudaFree(x.chunk_sfx);
    }
    p->extra_lanes.clear();
    for (cudaEvent_t ev : p->events) cudaEventDestroy(ev);
    p->events.clear();
    for (cudaEvent_t ev : p->order_events) cudaEventDestroy(ev);
    p->order_events.clear();
    if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
    p->copy_stream = nullptr;
}

}  // namespace

namespace rsdgc {

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }
void set_last_cuda_error(int e) { g_last_cuda_error = e; }

// Splits every layer into work items for the accumulate+NSI kernel and into key / element
// chunks for the selection passes, and assigns contiguous item ranges of equal cost to the
// CTAs of the accumulate+NSI kernel.
int build_plan_tables(rsdgc_plan *p, const rsdgc_layer_desc *descs, int n_layers)
{
    p->layers.clear();
    p->items.clear();
    p->chunks.clear();
    p->echunks.clear();
    std::vector<int64_t> chunk_w(n_layers, 0);  // columns of a regular (not last) column chunk
    const int64_t item_elems = p->item_elems;
    int64_t elem_off = 0, tile_off = 0, total_elems = 0, total_tiles = 0;
    int max_slot = 0;
    for (int l = 0; l < n_layers; ++l) {
        const rsdgc_layer_desc &d = descs[l];
        if (d.rows < 1 || d.cols < 1 || d.nh < 1 || d.nw < 1) return RSDGC_ERR_INVALID;
        if ((int64_t)d.nh * d.nw > kMaxSlot || d.nh > INT16_MAX || d.nw > INT16_MAX) return RSDGC_ERR_CAPACITY;
        if (d.rows > INT32_MAX || d.cols > INT32_MAX) return RSDGC_ERR_CAPACITY;
        if (d.rows * d.cols > (int64_t)INT32_MAX) return RSDGC_ERR_CAPACITY;
        LayerDev L{};
        L.elem_off = elem_off;
        L.tile_off = tile_off;
        L.rows = d.rows;
        L.cols = d.cols;
        L.nh = d.nh;
        L.nw = d.nw;
        L.TR = (int32_t)ceil_div64(d.rows, d.nh);
        L.TC = (int32_t)ceil_div64(d.cols, d.nw);
        L.K = L.TR * L.TC;
        L.slot = d.nh * d.nw;
        if (L.slot > max_slot) max_slot = L.slot;

        // --- accumulate+NSI items: rectangles of tiles holding at most kItemElems elements
        const int64_t band = (int64_t)d.nh * d.cols;  // one full-width row of tiles
        if (band <= item_elems) {
            int64_t ntr_max = item_elems / band;
            int64_t n_items = ceil_div64(L.TR, ntr_max);
            int64_t ntr = ceil_div64(L.TR, n_items);
            // every item start must be 16-byte aligned in both arenas (8 bfloat16 or 4 binary32 elements)
            // for 128-bit loads and bulk copies: a band of a multiple of 8 elements gives that for any
            // number of tile rows, otherwise multiples of 8 tile rows do
            if (band % 8 != 0) {
                if (round_up64(ntr, 8) <= ntr_max) ntr = round_up64(ntr, 8);
                else if (ntr_max >= 8) ntr = ntr_max & ~(int64_t)7;
            }
            for (int64_t tr0 = 0; tr0 < L.TR; tr0 += ntr) {
                Item it{l, (int32_t)tr0, (int32_t)std::min<int64_t>(ntr, L.TR - tr0), 0, L.TC};
                p->items.push_back(it);
            }
        } else {
            int64_t ntc_max = item_elems / L.slot;
            int64_t n_items = ceil_div64(L.TC, ntc_max);
            int64_t ntc = ceil_div64(L.TC, n_items);
            if (round_up64(ntc, 8) <= ntc_max) ntc = round_up64(ntc, 8);
            else if (ntc_max >= 8) ntc = ntc_max & ~(int64_t)7;
            chunk_w[l] = std::min<int64_t>(ntc * d.nw, d.cols);
            // the chunk width is also the row pitch of the block in shared memory: a multiple of 8
            // elements keeps every row of the block 16-byte aligned there for both element sizes
            // (neighborhoods of more than 550 elements leave fewer than 8 tile columns per item, so
            // the width itself need not be one)
            if (round_up64(chunk_w[l], 8) * d.nh <= item_elems) chunk_w[l] = round_up64(chunk_w[l], 8);
            for (int64_t tr = 0; tr < L.TR; ++tr)
                for (int64_t tc0 = 0; tc0 < L.TC; tc0 += ntc) {
                    Item it{l, (int32_t)tr, 1, (int32_t)tc0, (int32_t)std::min<int64_t>(ntc, L.TC - tc0)};
                    p->items.push_back(it);
                }
        }

        // --- key chunks and element chunks
        L.first_chunk = (int32_t)p->chunks.size();
        L.n_chunks = (int32_t)ceil_div64(L.K, kChunkKeys);
        for (int32_t c = 0; c < L.n_chunks; ++c) {
            int32_t start = c * kChunkKeys;
            p->chunks.push_back(Chunk{l, start, std::min<int32_t>(kChunkKeys, L.K - start)});
        }
        L.first_echunk = (int32_t)p->echunks.size();
        const int64_t n = d.rows * d.cols;
        for (int64_t s = 0; s < n; s += kChunkKeys)
            p->echunks.push_back(EChunk{s, l, (int32_t)std::min<int64_t>(kChunkKeys, n - s)});

        p->layers.push_back(L);
        total_elems += n;
        total_tiles += L.K;
        elem_off += round_up64(n, kArenaAlign);
        tile_off += round_up64(L.K, kArenaAlign);
    }
    if (p->items.size() > (size_t)INT32_MAX || p->echunks.size() > (size_t)INT32_MAX) return RSDGC_ERR_CAPACITY;

    // --- device form of the items; choice of kernel per item
    const size_t n_items = p->items.size();
    auto magic = [](int64_t d) -> uint32_t { return d <= 1 ? 0u : (uint32_t)(((1ll << 32) + d - 1) / d); };
    const int64_t gran = (p->dtype == RSDGC_BF16) ? 8 : 4;  // elements per 16 bytes of the gradient arena
    std::vector<ItemDev> all(n_items);
    p->item_path.assign(n_items, 0);
    p->item_cta.assign(n_items, 0);
    p->item_pitch.assign(n_items, 0);
    p->item_flags.assign(n_items, 0);
    std::vector<double> cost(n_items);
    for (size_t i = 0; i < n_items; ++i) {
        const Item &it = p->items[i];
        const LayerDev &L = p->layers[it.layer];
        ItemDev d{};
        const int64_t row0 = (int64_t)it.tr0 * L.nh, col0 = (int64_t)it.tc0 * L.nw;
        d.R = (int32_t)std::min<int64_t>((int64_t)it.ntr * L.nh, L.rows - row0);
        d.W = (int32_t)std::min<int64_t>((int64_t)it.ntc * L.nw, L.cols - col0);
        d.gbase = L.elem_off + row0 * L.cols + col0;
        d.kbase = L.tile_off + (int64_t)it.tr0 * L.TC + it.tc0;
        d.cols = (int32_t)L.cols;
        d.ntc = it.ntc;
        d.TC = L.TC;
        d.nh = (int16_t)L.nh;
        d.nw = (int16_t)L.nw;
        d.layer = it.layer;
        const bool full = (d.W == L.cols) || d.R == 1;  // one contiguous run
        // shared-memory pitch: the width of the layer's regular column chunk, so that every item
        // of a layer maps threads to elements the same way (the last chunk of a row is narrower)
        d.P = full ? d.W : (int32_t)chunk_w[it.layer];
        // 128-bit accesses / bulk copies need every row of the item 16-byte aligned in global
        // memory (start, row stride, width) AND in the shared-memory block (pitch)
        const bool vec = (d.gbase % 4 == 0) && (full || (L.cols % 4 == 0 && d.W % 4 == 0 && d.P % 4 == 0));
        const bool bulk = !(p->flags & RSDGC_NO_BULK_COPY) && (d.gbase % gran == 0) &&
                          (full || (L.cols % gran == 0 && d.W % gran == 0 && d.P % gran == 0));
        const bool noclip = (d.R % L.nh == 0) && (d.W % L.nw == 0);
        d.flags = (full ? kItemFull : 0) | (vec ? kItemVec : 0) | (bulk ? kItemBulk : 0) | (noclip ? kItemNoClip : 0);
        d.inv_ntc = magic(d.ntc);
        d.inv_p = magic(d.P);
        d.inv_pv = magic(d.P / 4);
        all[i] = d;
        p->item_path[i] = bulk ? 0 : 1;
        p->item_pitch[i] = d.P;
        p->item_flags[i] = d.flags;
        // elements + a fixed cost per item: an item takes a CTA about one memory round trip under load
        // whatever its size (measured: 3.7 us for 4400 elements, hardly less for 3000), the streaming of
        // its bytes adds to that
        cost[i] = (double)d.R * d.W + 8000.0;
        // the first item of a layer pays for the previous layer's histogram flush in its CTA (about 2.5 us)
        if (i > 0 && p->items[i - 1].layer != it.layer) cost[i] += 12000.0;
    }

    // --- each kernel's items in layer order, split into contiguous ranges of equal cost, one
    // range per CTA (all CTAs of a kernel are resident at once)
    p->items_dev.clear();
    p->grid_bulk = p->n_sm * k1_bulk_ctas_per_sm((p->flags & RSDGC_MOMENTUM) != 0);
    p->grid_reg = p->n_sm * p->reg_ctas_per_sm;
    for (auto &L : p->layers) L.n_flush1 = 0;
    for (int path = 0; path < 2; ++path) {
        std::vector<size_t> mine;
        for (size_t i = 0; i < n_items; ++i)
            if (p->item_path[i] == path) mine.push_back(i);
        const int G = path == 0 ? p->grid_bulk : p->grid_reg;
        std::vector<int32_t> &cta_begin = path == 0 ? p->cta_begin_bulk : p->cta_begin_reg;
        (path == 0 ? p->n_items_bulk : p->n_items_reg) = (int)mine.size();
        double total = 0.0;
        for (size_t i : mine) total += cost[i];
        cta_begin.assign(G + 1, (int32_t)mine.size());
        double cum = 0.0;
        size_t next_cta = 0;
        int prev_layer = -1, prev_cta = -1;
        for (size_t j = 0; j < mine.size(); ++j) {
            int g = total > 0.0 ? (int)std::floor(cum * G / total) : 0;
            if (g >= G) g = G - 1;
            while (next_cta <= (size_t)g) cta_begin[next_cta++] = (int32_t)j;
            const size_t i = mine[j];
            p->item_cta[i] = g;
            if (all[i].layer != prev_layer || g != prev_cta) p->layers[all[i].layer].n_flush1 += 1;
            prev_layer = all[i].layer;
            prev_cta = g;
            cum += cost[i];
            p->items_dev.push_back(all[i]);
        }
        while (next_cta <= (size_t)G) cta_begin[next_cta++] = (int32_t)mine.size();
    }

    // --- single-kernel tail (tail.cu): possible when every layer's keys fit one cluster's shared memory
    p->tail_slices.clear();
    p->n_tail_big = p->n_tail_small = p->n_tail_clusters = 0;
    bool tail_ok = !(p->flags & RSDGC_NO_FUSED_TAIL);
    for (const LayerDev &L : p->layers)
        if ((int64_t)L.K > (int64_t)kTailCluster * kTailKeysBig) tail_ok = false;
    if (tail_ok) {
        // layers above the one-CTA size: m slices each, all in one cluster; first fit, largest first.
        // A layer needs ceil(K / 32768) slices; it gets more (a pass over a slice is a CTA's time, so
        // the layer that decides the kernel's duration should be spread over the whole cluster) as long
        // as the plan then takes no more clusters than with the fewest slices.
        struct Big {
            int layer, m;
        };
        std::vector<std::vector<Big>> clusters;
        auto pack = [&](int64_t slice_keys) {
            std::vector<Big> big;
            for (int l = 0; l < n_layers; ++l)
                if (p->layers[l].K > kTailKeysSmall) {
                    const int64_t K = p->layers[l].K;
                    const int m = (int)std::max<int64_t>(ceil_div64(K, kTailKeysBig),
                                                         std::min<int64_t>(kTailCluster, ceil_div64(K, slice_keys)));
                    big.push_back(Big{l, m});
                }
            std::stable_sort(big.begin(), big.end(), [](const Big &a, const Big &b) { return a.m > b.m; });
            std::vector<std::vector<Big>> cl;
            std::vector<int> used;
            for (const Big &b : big) {
                size_t c = 0;
                while (c < cl.size() && used[c] + b.m > kTailCluster) ++c;
                if (c == cl.size()) {
                    cl.emplace_back();
                    used.push_back(0);
                }
                cl[c].push_back(b);
                used[c] += b.m;
            }
            return cl;
        };
        clusters = pack(kTailKeysBig);
        for (int64_t slice_keys = kTailKeysBig / 8; slice_keys < kTailKeysBig; slice_keys *= 2) {
            std::vector<std::vector<Big>> finer = pack(slice_keys);
            if (finer.size() <= clusters.size()) {
                clusters = std::move(finer);
                break;
            }
        }
        for (const std::vector<Big> &cl : clusters) {
            int rank = 0;
            for (const Big &b : cl) {
                const int32_t K = p->layers[b.layer].K;
                // equal slices, starts on multiples of 64 keys (16-byte aligned loads)
                const int32_t per = (int32_t)round_up64(ceil_div64(K, b.m), 64);
                for (int j = 0; j < b.m; ++j) {
                    const int32_t start = j * per;
                    const int32_t n = std::max<int32_t>(0, std::min<int32_t>(per, K - start));
                    p->tail_slices.push_back(TailSlice{b.layer, start, n, b.m, j, rank, {0, 0}});
                }
                rank += b.m;
            }
            for (; rank < kTailCluster; ++rank) p->tail_slices.push_back(TailSlice{0, 0, 0, 0, 0, 0, {0, 0}});
        }
        p->n_tail_clusters = (int)clusters.size();
        p->n_tail_big = p->n_tail_clusters * kTailCluster;
        for (int l = 0; l < n_layers; ++l)
            if (p->layers[l].K <= kTailKeysSmall) {
                p->tail_slices.push_back(TailSlice{l, 0, p->layers[l].K, 1, 0, 0, {0, 0}});
                ++p->n_tail_small;
            }
        if (p->n_tail_clusters > p->tail_max_clusters) {  // more than one wave of clusters: the chained kernels do better
            p->tail_slices.clear();
            p->n_tail_big = p->n_tail_small = p->n_tail_clusters = 0;
        }
    }

    rsdgc_info &I = p->info;
    I.n_layers = n_layers;
    I.grad_dtype = p->dtype;
    I.arena_elems = elem_off;
    I.total_elems = total_elems;
    I.total_tiles = total_tiles;
    I.total_tiles_padded = tile_off;
    I.workspace_bytes = tile_off * (int64_t)sizeof(uint32_t);
    I.max_slot = max_slot;
    I.reserved = 0;
    return RSDGC_OK;
}

}  // namespace rsdgc

// ------------------------------------------------------------------------------------------
// C entry points
// ------------------------------------------------------------------------------------------

extern "C" int rsdgc_plan_create(const rsdgc_layer_desc *layers_host, int32_t n_layers, int32_t grad_dtype,
                                 float alpha, uint32_t flags, int32_t device, rsdgc_plan **out)
{
    if (!layers_host || !out || n_layers < 1) return RSDGC_ERR_INVALID;
    *out = nullptr;
    if (n_layers > kMaxLayers) return RSDGC_ERR_CAPACITY;
    if (grad_dtype != RSDGC_F32 && grad_dtype != RSDGC_BF16) return RSDGC_ERR_INVALID;
    if (!(alpha >= 0.0f && alpha <= 1.0f)) return RSDGC_ERR_INVALID;
    if (flags & ~(RSDGC_KEEP_AT_LEAST_ONE | RSDGC_NO_BULK_COPY | RSDGC_MOMENTUM | RSDGC_PAYLOAD_BF16 |
                  RSDGC_NO_FUSED_TAIL))
        return RSDGC_ERR_INVALID;

    rsdgc_plan *p = new (std::nothrow) rsdgc_plan();
    if (!p) return RSDGC_ERR_NOMEM;
    p->device = device;
    p->n_layers = n_layers;
    p->dtype = grad_dtype;
    p->alpha = alpha;
    p->flags = flags;
    p->item_elems = bulk_item_elems(grad_dtype, (flags & RSDGC_MOMENTUM) != 0);

    if (device >= 0) {
        int n_sm = 0;
        cudaError_t e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, device);
        if (e != cudaSuccess) {
            delete p;
            return cuda_fail(e);
        }
        p->n_sm = n_sm;
        DeviceGuard guard(device);
        // one CTA per resident slot: the static partitions assume all CTAs run concurrently
        p->reg_ctas_per_sm = k1_reg_ctas_per_sm(grad_dtype, (flags & RSDGC_MOMENTUM) != 0);
        p->tail_max_clusters = tail_max_active_clusters();
    }

    int rc;
    try {
        rc = build_plan_tables(p, layers_host, n_layers);
    } catch (const std::bad_alloc &) {
        rc = RSDGC_ERR_NOMEM;
    }
    if (rc != RSDGC_OK) {
        delete p;
        return rc;
    }

    if (device >= 0) {
        DeviceGuard guard(device);
        cudaError_t e = guard.err;
        if (e == cudaSuccess) e = upload(&p->d_layers, p->layers);
        if (e == cudaSuccess) e = upload(&p->d_items, p->items_dev);
        if (e == cudaSuccess) e = upload(&p->d_cta_begin_bulk, p->cta_begin_bulk);
        if (e == cudaSuccess) e = upload(&p->d_cta_begin_reg, p->cta_begin_reg);
        if (e == cudaSuccess) e = upload(&p->d_chunks, p->chunks);
        if (e == cudaSuccess) e = upload(&p->d_tail_slices, p->tail_slices);
        if (e == cudaSuccess) e = upload(&p->d_echunks, p->echunks);
        if (e == cudaSuccess) e = alloc_zero(&p->d_state, (size_t)n_layers);
        if (e == cudaSuccess) e = alloc_zero(&p->d_hist, (size_t)n_layers * kHistStride);
        if (e == cudaSuccess) e = alloc_zero(&p->d_chunk_cnt, p->chunks.size());
        if (e == cudaSuccess) e = alloc_zero(&p->d_chunk_sfx, p->chunks.size() * (size_t)kL3Bins);
        if (e == cudaSuccess) e = alloc_zero(&p->d_codes, (size_t)p->info.total_tiles_padded / 4 + kChunkKeys / 4 + 16);
        if (e == cudaSuccess) e = alloc_zero(&p->d_survivors, (size_t)n_layers);
        if (e == cudaSuccess) e = alloc_zero(&p->d_rstate, 1);
        if (e == cudaSuccess) e = alloc_zero(&p->d_status, 1);
        if (e == cudaSuccess) {
            StatusDev st{};
            st.arena_elems = p->info.arena_elems;
            st.keys_len = p->info.total_tiles_padded;
            st.n_layers = n_layers;
            st.n_chunks = (int)p->chunks.size();
            st.n_echunks = (int)p->echunks.size();
            st.n_items = (int)p->items_dev.size();
            e = cudaMemcpy(p->d_status, &st, sizeof st, cudaMemcpyHostToDevice);
        }
        if (e == cudaSuccess) e = cudaDeviceSynchronize();
        if (e != cudaSuccess) {
            free_device_tables(p);
            delete p;
            return e == cudaErrorMemoryAllocation ? RSDGC_ERR_NOMEM : cuda_fail(e);
        }
    }
    *out = p;
    return RSDGC_OK;
}

extern "C" int rsdgc_plan_destroy(rsdgc_plan *plan)
{
    if (!plan) return RSDGC_ERR_INVALID;
    if (plan->device >= 0) {
        DeviceGuard guard(plan->device);
        free_device_tables(plan);
    }
    delete plan;
    return RSDGC_OK;
}

extern "C" int rsdgc_plan_info(const rsdgc_plan *plan, rsdgc_info *out_host)
{
    if (!plan || !out_host) return RSDGC_ERR_INVALID;
    *out_host = plan->info;
    return RSDGC_OK;
}

extern "C" int rsdgc_plan_layer_info(const rsdgc_plan *plan, int32_t layer, rsdgc_layer_info *out_host)
{
    if (!plan || !out_host || layer < 0 || layer >= plan->n_layers) return RSDGC_ERR_INVALID;
    const LayerDev &L = plan->layers[layer];
    out_host->elem_offset = L.elem_off;
    out_host->tile_offset = L.tile_off;
    out_host->rows = L.rows;
    out_host->cols = L.cols;
    out_host->nh = L.nh;
    out_host->nw = L.nw;
    out_host->n_tiles = L.K;
    return RSDGC_OK;
}

extern "C" int rsdgc_plan_payload_bound(const rsdgc_plan *plan, float max_ratio, int64_t *idx_capacity_host,
                                        int64_t *val_capacity_host)
{
    if (!plan || !idx_capacity_host || !val_capacity_host || !(max_ratio >= 0.0f)) return RSDGC_ERR_INVALID;
    int64_t ni = 0, nv = 0;
    for (const LayerDev &L : plan->layers) {
        double x = std::ceil((double)L.K * (double)max_ratio) + 1.0;
        int64_t k = (x >= (double)L.K) ? (int64_t)L.K : (int64_t)x;
        ni += k;
        nv += k * L.slot;
    }
    *idx_capacity_host = ni;
    *val_capacity_host = nv;
    return RSDGC_OK;
}

// Diagnostic: the accumulate+NSI work list (9 int32 per item: layer, tr0, ntr, tc0, ntc, kernel,
// CTA, shared-memory pitch, item flags), the two grid sizes and the per-layer flush counts; used by
// the host-logic tests.
extern "C" int64_t rsdgc_plan_worklist(const rsdgc_plan *plan, int32_t *items_host, int64_t items_capacity,
                                       int32_t *grids_host, int32_t *n_flush_host)
{
    if (!plan) return RSDGC_ERR_INVALID;
    int64_t n = (int64_t)plan->items.size();
    if (items_host)
        for (int64_t i = 0; i < n && i < items_capacity; ++i) {
            const Item &it = plan->items[i];
            int32_t *o = items_host + 9 * i;
            o[0] = it.layer, o[1] = it.tr0, o[2] = it.ntr, o[3] = it.tc0, o[4] = it.ntc;
            o[5] = plan->item_path[i], o[6] = plan->item_cta[i];
            o[7] = plan->item_pitch[i], o[8] = plan->item_flags[i];
        }
    if (grids_host) grids_host[0] = plan->grid_bulk, grids_host[1] = plan->grid_reg;
    if (n_flush_host)
        for (int l = 0; l < plan->n_layers; ++l) n_flush_host[l] = plan->layers[l].n_flush1;
    return n;
}

// Diagnostic: the slices of the single-kernel tail (6 int32 per slice: layer, first tile, tiles,
// CTAs of the layer, rank among them, cluster rank of the first), cluster slices first; info_host
// receives their number, the number of one-CTA slices and the number of clusters.
extern "C" int64_t rsdgc_plan_tail_slices(const rsdgc_plan *plan, int32_t *slices_host, int64_t capacity,
                                          int32_t *info_host)
{
    if (!plan) return RSDGC_ERR_INVALID;
    const int64_t n = (int64_t)plan->tail_slices.size();
    if (slices_host)
        for (int64_t i = 0; i < n && i < capacity; ++i) {
            const TailSlice &t = plan->tail_slices[i];
            int32_t *o = slices_host + 6 * i;
            o[0] = t.layer, o[1] = t.start, o[2] = t.n, o[3] = t.n_ranks, o[4] = t.rank, o[5] = t.leader;
        }
    if (info_host) info_host[0] = plan->n_tail_big, info_host[1] = plan->n_tail_small, info_host[2] = plan->n_tail_clusters;
    return n;
}

namespace {

int check_plan_device(const rsdgc_plan *plan)
{
    if (!plan) return RSDGC_ERR_INVALID;
    if (plan->device < 0) return RSDGC_ERR_INVALID;  // host-only plan: sizing queries only
    return RSDGC_OK;
}

}  // namespace

extern "C" int rsdgc_update_ratios(rsdgc_plan *plan, const float *weights_dev, float global_keep,
                                   float *ratios_dev, void *stream)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (!weights_dev || !ratios_dev || !(global_keep >= 0.0f && global_keep <= 1.0f)) return RSDGC_ERR_INVALID;
    if (!aligned16(weights_dev)) return RSDGC_ERR_ALIGNMENT;
    // n_keep = ceil(rho * G), product in binary64 of the binary32 ratio (Eq. 4 read as "keep")
    const double G = (double)plan->info.total_elems;
    double x = std::ceil((double)global_keep * G);
    long long n_keep = x <= 0.0 ? 0 : (x >= G ? plan->info.total_elems : (long long)x);
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    RSDGC_RANGE("rsdgc_update_ratios");
    cudaError_t e = launch_update_ratios(plan, weights_dev, n_keep, ratios_dev, (cudaStream_t)stream);
    return e == cudaSuccess ? RSDGC_OK : cuda_fail(e);
}

namespace {

int compress_common(rsdgc_plan *plan, const void *grads_dev, float *velocity_dev, float momentum, float *residual_dev,
                    const float *ratios_dev, int32_t *idx_dev, int64_t idx_capacity, void *val_dev,
                    int64_t val_capacity, int32_t *counts_dev, float *nsi_dev, void *workspace_dev, void *stream)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (!grads_dev || !residual_dev || !ratios_dev || !counts_dev) return RSDGC_ERR_INVALID;
    if (idx_capacity < 0 || val_capacity < 0) return RSDGC_ERR_INVALID;
    if ((idx_capacity > 0 && !idx_dev) || (val_capacity > 0 && !val_dev)) return RSDGC_ERR_INVALID;
    if (!nsi_dev && !workspace_dev) return RSDGC_ERR_INVALID;
    if (!aligned16(grads_dev) || !aligned16(residual_dev) || !aligned16(idx_dev) || !aligned16(val_dev) ||
        !aligned16(nsi_dev) || !aligned16(workspace_dev) || !aligned16(velocity_dev))
        return RSDGC_ERR_ALIGNMENT;
    uint32_t *keys = nsi_dev ? reinterpret_cast<uint32_t *>(nsi_dev) : reinterpret_cast<uint32_t *>(workspace_dev);
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    RSDGC_RANGE(velocity_dev ? "rsdgc_compress_momentum" : "rsdgc_compress");
    cudaError_t e = launch_compress(plan, grads_dev, residual_dev, velocity_dev, momentum, ratios_dev, idx_dev,
                                    idx_capacity, val_dev, val_capacity, counts_dev, keys, (cudaStream_t)stream);
    return e == cudaSuccess ? RSDGC_OK : cuda_fail(e);
}

}  // namespace

extern "C" int rsdgc_compress(rsdgc_plan *plan, const void *grads_dev, float *residual_dev,
                              const float *ratios_dev, int32_t *idx_dev, int64_t idx_capacity, void *val_dev,
                              int64_t val_capacity, int32_t *counts_dev, float *nsi_dev, void *workspace_dev,
                              void *stream)
{
    if (plan && (plan->flags & RSDGC_MOMENTUM)) return RSDGC_ERR_INVALID;  // use rsdgc_compress_momentum()
    return compress_common(plan, grads_dev, nullptr, 0.0f, residual_dev, ratios_dev, idx_dev, idx_capacity, val_dev,
                           val_capacity, counts_dev, nsi_dev, workspace_dev, stream);
}

extern "C" int rsdgc_compress_momentum(rsdgc_plan *plan, const void *grads_dev, float *velocity_dev, float momentum,
                                       float *residual_dev, const float *ratios_dev, int32_t *idx_dev,
                                       int64_t idx_capacity, void *val_dev, int64_t val_capacity,
                                       int32_t *counts_dev, float *nsi_dev, void *workspace_dev, void *stream)
{
    if (!plan || !(plan->flags & RSDGC_MOMENTUM) || !velocity_dev) return RSDGC_ERR_INVALID;
    if (!(momentum >= 0.0f && momentum <= 1.0f)) return RSDGC_ERR_INVALID;
    return compress_common(plan, grads_dev, velocity_dev, momentum, residual_dev, ratios_dev, idx_dev, idx_capacity,
                           val_dev, val_capacity, counts_dev, nsi_dev, workspace_dev, stream);
}

extern "C" int rsdgc_plan_reserve_workers(rsdgc_plan *plan, int32_t n_workers)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (n_workers < 1) return RSDGC_ERR_INVALID;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    while ((int)plan->extra_lanes.size() + 1 < n_workers) {
        rsdgc_plan::LaneScratch x;
        cudaError_t e = alloc_zero(&x.state, (size_t)plan->n_layers);
        if (e == cudaSuccess) e = alloc_zero(&x.hist, (size_t)plan->n_layers * kHistStride);
        if (e == cudaSuccess) e = alloc_zero(&x.chunk_cnt, plan->chunks.size());
        if (e == cudaSuccess) e = alloc_zero(&x.chunk_sfx, plan->chunks.size() * (size_t)kL3Bins);
        if (e == cudaSuccess)
            e = alloc_zero(&x.codes, (size_t)plan->info.total_tiles_padded / 4 + kChunkKeys / 4 + 16);
        if (e == cudaSuccess) e = cudaDeviceSynchronize();
        if (e != cudaSuccess) {
            cudaFree(x.state);
            cudaFree(x.hist);
            cudaFree(x.chunk_cnt);
            cudaFree(x.chunk_sfx);
            cudaFree(x.codes);
            return e == cudaErrorMemoryAllocation ? RSDGC_ERR_NOMEM : cuda_fail(e);
        }
        plan->extra_lanes.push_back(x);
    }
    return RSDGC_OK;
}

extern "C" int rsdgc_compress_workers(rsdgc_plan *plan, int32_t n_workers, const void *const *grads_dev_host,
                                      float *const *residual_dev_host, const float *ratios_dev,
                                      int32_t *const *idx_dev_host, int64_t idx_capacity,
                                      void *const *val_dev_host, int64_t val_capacity,
                                      int32_t *const *counts_dev_host, void *workspace_dev, void *stream)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (plan->flags & RSDGC_MOMENTUM) return RSDGC_ERR_INVALID;
    if (n_workers < 1 || !grads_dev_host || !residual_dev_host || !ratios_dev || !counts_dev_host || !workspace_dev)
        return RSDGC_ERR_INVALID;
    if (idx_capacity < 0 || val_capacity < 0) return RSDGC_ERR_INVALID;
    if ((idx_capacity > 0 && !idx_dev_host) || (val_capacity > 0 && !val_dev_host)) return RSDGC_ERR_INVALID;
    if ((int)plan->extra_lanes.size() + 1 < n_workers) return RSDGC_ERR_CAPACITY;  // rsdgc_plan_reserve_workers()
    if (!aligned16(workspace_dev)) return RSDGC_ERR_ALIGNMENT;
    std::vector<int32_t *> idx((size_t)n_workers, nullptr);
    std::vector<void *> val((size_t)n_workers, nullptr);
    for (int w = 0; w < n_workers; ++w) {
        if (!grads_dev_host[w] || !residual_dev_host[w] || !counts_dev_host[w]) return RSDGC_ERR_INVALID;
        if (idx_capacity > 0) idx[w] = idx_dev_host[w];
        if (val_capacity > 0) val[w] = val_dev_host[w];
        if ((idx_capacity > 0 && !idx[w]) || (val_capacity > 0 && !val[w])) return RSDGC_ERR_INVALID;
        if (!aligned16(grads_dev_host[w]) || !aligned16(residual_dev_host[w]) || !aligned16(idx[w]) ||
            !aligned16(val[w]))
            return RSDGC_ERR_ALIGNMENT;
        for (int v = 0; v < w; ++v)  // every worker has its own accumulator and payload
            if (residual_dev_host[v] == residual_dev_host[w] || counts_dev_host[v] == counts_dev_host[w] ||
                (idx[w] && idx[v] == idx[w]) || (val[w] && val[v] == val[w]))
                return RSDGC_ERR_INVALID;
    }
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    RSDGC_RANGE("rsdgc_compress_workers");
    cudaError_t e = launch_compress_workers(plan, n_workers, grads_dev_host, residual_dev_host, ratios_dev, idx.data(),
                                            idx_capacity, val.data(), val_capacity, counts_dev_host,
                                            reinterpret_cast<uint32_t *>(workspace_dev), (cudaStream_t)stream);
    return e == cudaSuccess ? RSDGC_OK : cuda_fail(e);
}

extern "C" int rsdgc_compress_host(rsdgc_plan *plan, const void *grads_host, void *grads_dev, float *residual_dev,
                                   const float *ratios_dev, int32_t *idx_dev, int64_t idx_capacity, void *val_dev,
                                   int64_t val_capacity, int32_t *counts_dev, void *workspace_dev,
                                   int32_t *idx_host, void *val_host, int32_t *counts_host,
                                   int64_t *idx_used_host, int64_t *val_used_host, void *stream)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (!grads_host || !grads_dev || !counts_host || !idx_used_host || !val_used_host) return RSDGC_ERR_INVALID;
    if ((idx_capacity > 0 && !idx_host) || (val_capacity > 0 && !val_host)) return RSDGC_ERR_INVALID;
    cudaStream_t s = (cudaStream_t)stream;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    const size_t esz = plan->dtype == RSDGC_BF16 ? 2 : 4;
    RSDGC_RANGE("rsdgc_compress_host");
    cudaError_t e = cudaMemcpyAsync(grads_dev, grads_host, (size_t)plan->info.arena_elems * esz,
                                    cudaMemcpyHostToDevice, s);
    if (e != cudaSuccess) return cuda_fail(e);
    rc = rsdgc_compress(plan, grads_dev, residual_dev, ratios_dev, idx_dev, idx_capacity, val_dev, val_capacity,
                        counts_dev, nullptr, workspace_dev, stream);
    if (rc) return rc;
    e = cudaMemcpyAsync(counts_host, counts_dev, (size_t)plan->n_layers * sizeof(int32_t), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e);
    int64_t ni = 0, nv = 0;
    for (int l = 0; l < plan->n_layers; ++l) {
        ni += counts_host[l];
        nv += (int64_t)counts_host[l] * plan->layers[l].slot;
    }
    if (ni > idx_capacity) ni = idx_capacity;
    if (nv > val_capacity) nv = val_capacity;
    if (ni > 0) e = cudaMemcpyAsync(idx_host, idx_dev, (size_t)ni * sizeof(int32_t), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess && nv > 0)
        e = cudaMemcpyAsync(val_host, val_dev, (size_t)nv * ((plan->flags & RSDGC_PAYLOAD_BF16) ? 2 : 4),
                            cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e);
    *idx_used_host = ni;
    *val_used_host = nv;
    return RSDGC_OK;
}

// The host-buffer path for all the workers of a GPU, pipelined over two staging arenas: while
// worker w is compressed on the caller's stream, worker w + 1's gradient is already on its way into
// the other arena on the plan's copy stream, and worker w's payload leaves right behind its
// compress.  One synchronisation, at the end.
extern "C" int rsdgc_compress_workers_host(rsdgc_plan *plan, int32_t n_workers, const void *const *grads_host,
                                           void *const *staging_dev_host, float *const *residual_dev_host,
                                           const float *ratios_dev, int32_t *const *idx_dev_host,
                                           int64_t idx_capacity, void *const *val_dev_host, int64_t val_capacity,
                                           int32_t *const *counts_dev_host, void *workspace_dev,
                                           int32_t *const *idx_host, void *const *val_host,
                                           int32_t *const *counts_host, int64_t *idx_used_host,
                                           int64_t *val_used_host, void *stream)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (n_workers < 1 || !grads_host || !staging_dev_host || !residual_dev_host || !idx_dev_host || !val_dev_host ||
        !counts_dev_host || !idx_host || !val_host || !counts_host || !idx_used_host || !val_used_host)
        return RSDGC_ERR_INVALID;
    if (!staging_dev_host[0] || !staging_dev_host[1] || staging_dev_host[0] == staging_dev_host[1])
        return RSDGC_ERR_INVALID;
    if (idx_capacity < 0 || val_capacity < 0) return RSDGC_ERR_INVALID;
    for (int w = 0; w < n_workers; ++w)
        if (!grads_host[w] || !counts_host[w] || (idx_capacity > 0 && !idx_host[w]) || (val_capacity > 0 && !val_host[w]))
            return RSDGC_ERR_INVALID;
    cudaStream_t s = (cudaStream_t)stream;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    RSDGC_RANGE("rsdgc_compress_workers_host");
    cudaError_t e = cudaSuccess;
    if (!plan->copy_stream) e = cudaStreamCreateWithFlags(&plan->copy_stream, cudaStreamNonBlocking);
    while (e == cudaSuccess && plan->order_events.size() < (size_t)(2 * n_workers + 1)) {
        cudaEvent_t ev;
        e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e == cudaSuccess) plan->order_events.push_back(ev);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    cudaEvent_t *copied = plan->order_events.data();                 // [w]: worker w's gradient has arrived
    cudaEvent_t *consumed = plan->order_events.data() + n_workers;   // [w]: worker w's compress has run
    cudaEvent_t begin = plan->order_events[2 * (size_t)n_workers];
    const size_t esz = plan->dtype == RSDGC_BF16 ? 2 : 4, vsz = (plan->flags & RSDGC_PAYLOAD_BF16) ? 2 : 4;
    const size_t arena_bytes = (size_t)plan->info.arena_elems * esz;
    // the staging arenas may still be read by work the caller queued before this call
    e = cudaEventRecord(begin, s);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(plan->copy_stream, begin, 0);
    for (int w = 0; w < n_workers && e == cudaSuccess; ++w) {
        void *stage = staging_dev_host[w & 1];
        if (w >= 2) e = cudaStreamWaitEvent(plan->copy_stream, consumed[w - 2], 0);  // the arena is free again
        if (e == cudaSuccess) e = cudaMemcpyAsync(stage, grads_host[w], arena_bytes, cudaMemcpyHostToDevice, plan->copy_stream);
        if (e == cudaSuccess) e = cudaEventRecord(copied[w], plan->copy_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s, copied[w], 0);
        if (e != cudaSuccess) break;
        rc = rsdgc_compress(plan, stage, residual_dev_host[w], ratios_dev, idx_dev_host[w], idx_capacity,
                            val_dev_host[w], val_capacity, counts_dev_host[w], nullptr, workspace_dev, stream);
        if (rc) break;
        e = cudaEventRecord(consumed[w], s);
        // the payload sizes are only known on the device: the buffers travel whole (their capacity is
        // the payload bound, a few tiles per layer above the payload itself)
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(counts_host[w], counts_dev_host[w], (size_t)plan->n_layers * sizeof(int32_t),
                                cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess && idx_capacity > 0)
            e = cudaMemcpyAsync(idx_host[w], idx_dev_host[w], (size_t)idx_capacity * sizeof(int32_t),
                                cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess && val_capacity > 0)
            e = cudaMemcpyAsync(val_host[w], val_dev_host[w], (size_t)val_capacity * vsz, cudaMemcpyDeviceToHost, s);
    }
    // whatever happened, nothing of this call is left in flight when it returns
    cudaError_t e2 = cudaStreamSynchronize(plan->copy_stream);
    cudaError_t e3 = cudaStreamSynchronize(s);
    if (rc) return rc;
    if (e == cudaSuccess) e = e2;
    if (e == cudaSuccess) e = e3;
    if (e != cudaSuccess) return cuda_fail(e);
    for (int w = 0; w < n_workers; ++w) {
        int64_t ni = 0, nv = 0;
        for (int l = 0; l < plan->n_layers; ++l) {
            ni += counts_host[w][l];
            nv += (int64_t)counts_host[w][l] * plan->layers[l].slot;
        }
        idx_used_host[w] = ni < idx_capacity ? ni : idx_capacity;
        val_used_host[w] = nv < val_capacity ? nv : val_capacity;
    }
    return RSDGC_OK;
}

namespace {

int decompress_common(rsdgc_plan *plan, int32_t n_workers, const int32_t *const *idx_dev_host,
                      const void *const *val_dev_host, const int32_t *const *counts_dev_host, int64_t idx_capacity,
                      int64_t val_capacity, float scale, float *dense_dev, bool assign, void *stream)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (n_workers < 0 || !dense_dev || idx_capacity < 0 || val_capacity < 0) return RSDGC_ERR_INVALID;
    if (n_workers > 0 && (!idx_dev_host || !val_dev_host || !counts_dev_host)) return RSDGC_ERR_INVALID;
    if (!aligned16(dense_dev)) return RSDGC_ERR_ALIGNMENT;
    for (int w = 0; w < n_workers; ++w) {
        if (!idx_dev_host[w] || !val_dev_host[w] || !counts_dev_host[w]) return RSDGC_ERR_INVALID;
        if (!aligned16(idx_dev_host[w]) || !aligned16(val_dev_host[w])) return RSDGC_ERR_ALIGNMENT;
    }
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    // every dense element is updated by one CTA, worker after worker: reproducible binary32 sums
    if (n_workers > 0 || assign) {
        RSDGC_RANGE(assign ? "rsdgc_decompress_assign" : "rsdgc_decompress_accumulate");
        cudaError_t e = launch_decompress(plan, n_workers, idx_dev_host, val_dev_host, counts_dev_host,
                                          (long long)idx_capacity, (long long)val_capacity, scale, dense_dev, assign,
                                          (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(e);
    }
    return RSDGC_OK;
}

}  // namespace

extern "C" int rsdgc_decompress_accumulate(rsdgc_plan *plan, int32_t n_workers, const int32_t *const *idx_dev_host,
                                           const void *const *val_dev_host,
                                           const int32_t *const *counts_dev_host, int64_t idx_capacity,
                                           int64_t val_capacity, float scale, float *dense_dev, void *stream)
{
    return decompress_common(plan, n_workers, idx_dev_host, val_dev_host, counts_dev_host, idx_capacity,
                             val_capacity, scale, dense_dev, false, stream);
}

extern "C" int rsdgc_decompress_assign(rsdgc_plan *plan, int32_t n_workers, const int32_t *const *idx_dev_host,
                                       const void *const *val_dev_host, const int32_t *const *counts_dev_host,
                                       int64_t idx_capacity, int64_t val_capacity, float scale, float *dense_dev,
                                       void *stream)
{
    return decompress_common(plan, n_workers, idx_dev_host, val_dev_host, counts_dev_host, idx_capacity,
                             val_capacity, scale, dense_dev, true, stream);
}

extern "C" int rsdgc_payload_to_coo(rsdgc_plan *plan, const int32_t *idx_dev, const int32_t *counts_dev,
                                    int64_t *coo_index_dev, int64_t coo_capacity, void *stream)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (!idx_dev || !counts_dev || coo_capacity < 0 || (coo_capacity > 0 && !coo_index_dev)) return RSDGC_ERR_INVALID;
    if (!aligned16(idx_dev) || !aligned16(coo_index_dev)) return RSDGC_ERR_ALIGNMENT;
    if (coo_capacity == 0) return RSDGC_OK;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    static_assert(sizeof(long long) == sizeof(int64_t), "coordinate entries are 64-bit");
    RSDGC_RANGE("rsdgc_payload_to_coo");
    cudaError_t e = launch_payload_to_coo(plan, idx_dev, counts_dev, reinterpret_cast<long long *>(coo_index_dev),
                                          (long long)coo_capacity, (cudaStream_t)stream);
    return e == cudaSuccess ? RSDGC_OK : cuda_fail(e);
}

extern "C" int rsdgc_get_status(rsdgc_plan *plan, void *stream, rsdgc_status *out_host)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (!out_host) return RSDGC_ERR_INVALID;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    cudaStream_t s = (cudaStream_t)stream;
    StatusDev h{};
    cudaError_t e = cudaMemcpyAsync(&h, plan->d_status, sizeof h, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaMemsetAsync(plan->d_status, 0, kStatusResetBytes, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(e);
    out_host->flags = h.flags;
    out_host->reserved = 0;
    out_host->nonfinite = (int64_t)h.nonfinite;
    out_host->idx_needed = h.idx_needed;
    out_host->val_needed = h.val_needed;
    return RSDGC_OK;
}

extern "C" int rsdgc_profile_enable(rsdgc_plan *plan, int32_t level)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (level < 0 || level > 2) return RSDGC_ERR_INVALID;
    if (plan->events_used && level != plan->profile_recorded && level != 0)
        return RSDGC_ERR_INVALID;  // read the recorded calls before switching level
    plan->profile = level;
    return RSDGC_OK;
}

extern "C" int rsdgc_profile_read(rsdgc_plan *plan, double *ms_per_kernel_host, int64_t *n_calls_host)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (!ms_per_kernel_host || !n_calls_host) return RSDGC_ERR_INVALID;
    const size_t stages = plan->profile_recorded == 2 ? RSDGC_N_COMPRESS_KERNELS : 1;
    const size_t per_call = stages + 1;
    const size_t n_calls = plan->events_used / per_call;
    for (int k = 0; k < RSDGC_N_COMPRESS_KERNELS; ++k) ms_per_kernel_host[k] = 0.0;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    for (size_t c = 0; c < n_calls; ++c) {
        const cudaEvent_t *ev = plan->events.data() + c * per_call;
        cudaError_t e = cudaEventSynchronize(ev[per_call - 1]);
        for (size_t k = 0; k < stages && e == cudaSuccess; ++k) {
            float ms = 0.0f;
            e = cudaEventElapsedTime(&ms, ev[k], ev[k + 1]);
            ms_per_kernel_host[k] += ms;
        }
        if (e != cudaSuccess) return cuda_fail(e);
    }
    *n_calls_host = (int64_t)n_calls;
    plan->events_used = 0;
    return RSDGC_OK;
}

extern "C" int rsdgc_selftest_bounded_wait(rsdgc_plan *plan, int32_t polls, void *stream)
{
    int rc = check_plan_device(plan);
    if (rc) return rc;
    if (polls < 1 || polls > (1 << 20)) return RSDGC_ERR_INVALID;
    DeviceGuard guard(plan->device);
    if (guard.err != cudaSuccess) return cuda_fail(guard.err);
    RSDGC_RANGE("rsdgc_selftest_bounded_wait");
    cudaError_t e = launch_selftest_bounded_wait(plan, (unsigned int)polls, (cudaStream_t)stream);
    return e == cudaSuccess ? RSDGC_OK : cuda_fail(e);
}

extern "C" int64_t rsdgc_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

extern "C" const char *rsdgc_strerror(int code)
{
    switch (code) {
        case RSDGC_OK: return "ok";
        case RSDGC_ERR_INVALID: return "invalid argument";
        case RSDGC_ERR_ALIGNMENT: return "device pointer not 16-byte aligned";
        case RSDGC_ERR_CAPACITY: return "size beyond what the library supports";
        case RSDGC_ERR_CUDA: return "CUDA runtime error";
        case RSDGC_ERR_NOMEM: return "out of memory";
        default: return "unknown error";
    }
}

extern "C" int rsdgc_last_cuda_error(void) { return g_last_cuda_error; }
