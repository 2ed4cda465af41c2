// Internal declarations shared by the host code and the kernels of the RS-DGC library.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "rsdgc.h"

namespace rsdgc {

// ---- compile-time geometry -------------------------------------------------------------
constexpr int kThreads = 256;        // threads per CTA, every kernel
#ifndef RSDGC_ITEM_ELEMS
#define RSDGC_ITEM_ELEMS 4400
#endif
constexpr int kItemElems = RSDGC_ITEM_ELEMS;  // elements of one accumulate+NSI work item (the most any variant takes)
#ifndef RSDGC_BF16_STAGES
#define RSDGC_BF16_STAGES 2
#endif
#ifndef RSDGC_BF16_ITEM_ELEMS
#define RSDGC_BF16_ITEM_ELEMS 5600
#endif
constexpr int kItemElemsBf16 = RSDGC_BF16_ITEM_ELEMS;  // ... with bfloat16 gradients and no momentum
constexpr int kItemElemsMax = kItemElems > kItemElemsBf16 ? kItemElems : kItemElemsBf16;  // what the register-staged kernel holds
constexpr int kL1Bits = 10;          // radix level 1: key bits 30..21 (8 exponent + 2 mantissa)
constexpr int kL1Bins = 1 << kL1Bits;
constexpr int kL1Shift = 21;
constexpr int kL2Bits = 11;          // level 2: key bits 20..10
constexpr int kL2Bins = 1 << kL2Bits;
constexpr int kL2Shift = 10;
constexpr int kL3Bits = 10;          // level 3: key bits 9..0
constexpr int kL3Bins = 1 << kL3Bits;
constexpr int kHistStride = kL2Bins; // words of histogram per layer (the largest level)
constexpr int kChunkKeys = 16384;    // keys (or weights) per CTA in the key passes
constexpr int kMaxLayers = 2048;
constexpr int kMaxSlot = 4096;
constexpr int kArenaAlign = 64;      // elements; also the alignment of tile offsets
constexpr uint32_t kTakeNone = 0xFFFFFFFFu;  // prefix / threshold marker: keep nothing
// the single-kernel selection + pack for plans of small layers (tail.cu)
constexpr int kTailCluster = 8;        // CTAs per thread-block cluster = slices a layer may have
constexpr int kTailKeysBig = 32768;    // keys a CTA of the cluster variant holds in shared memory
constexpr int kTailThreadsBig = 512;
constexpr int kTailKeysSmall = 8192;   // layers up to this many tiles take the one-CTA variant
constexpr int kTailThreadsSmall = 256;

// ---- tables ----------------------------------------------------------------------------
struct LayerDev {
    int64_t elem_off;   // start in the element arenas
    int64_t tile_off;   // start in the key array
    int64_t rows, cols;
    int32_t nh, nw;
    int32_t TR, TC;     // tile grid; K = TR * TC
    int32_t K, slot;    // tiles, values per tile (nh * nw)
    int32_t first_chunk, n_chunks;    // key chunks of this layer
    int32_t n_flush1;                 // CTAs of the accumulate+NSI kernel that touch the layer
    int32_t first_echunk;             // first element chunk (ratio rule)
};

// Work item of the accumulate+NSI kernel: tile rows [tr0, tr0+ntr) x tile cols [tc0, tc0+ntc).
struct Item {
    int32_t layer, tr0, ntr, tc0, ntc;
};

// The same item resolved for the device: everything the accumulate+NSI kernels need, so that
// one 64-byte load per item replaces the chain item -> layer table -> data.
struct __align__(16) ItemDev {
    long long gbase;  // arena index of the first element held
    long long kbase;  // key-array index of the first tile
    int32_t R, W;     // rows and columns held
    int32_t cols;     // row stride in global memory
    int32_t ntc;      // tile columns in the item
    int32_t TC;       // tile columns of the layer = key stride between tile rows
    int16_t nh, nw;
    int32_t layer;
    int32_t flags;    // kItem* bits
    uint32_t inv_ntc; // ceil(2^32 / d) for d = ntc, P, P / 4 (0 when d = 1): see fast_div()
    uint32_t inv_p;
    uint32_t inv_pv;
    int32_t P;        // row pitch of the block in shared memory (elements, >= W)
};
static_assert(sizeof(ItemDev) == 64, "ItemDev is loaded as four 16-byte words");
constexpr int kItemFull = 1;    // the rows held are one contiguous run in memory
constexpr int kItemVec = 2;     // every row starts on a 16-byte boundary of the binary32 arenas
constexpr int kItemBulk = 4;    // eligible for the bulk-copy kernel (16-byte rule for g as well)
constexpr int kItemNoClip = 8;  // no tile of the item is clipped by the layer's edge

// Key chunk: keys [start, start + n) of a layer (layer-local tile indices).
struct Chunk {
    int32_t layer, start, n;
};

// Element chunk: elements [start, start + n) of a layer (layer-local flat positions).
struct EChunk {
    int64_t start;
    int32_t layer, n;
};

// One CTA's share of the single-kernel selection + pack: keys [start, start + n) of a layer.  The
// n_ranks CTAs of a layer sit in one cluster, `rank` counts them, `leader` is the cluster rank of
// the first.  n = 0: a rank of a cluster that holds no slice.
struct TailSlice {
    int32_t layer, start, n;
    int32_t n_ranks, rank, leader;
    int32_t pad[2];
};

// Per-layer selection state carried from kernel to kernel (device memory, plan-owned).
struct LayerState {
    unsigned int ticket[4];  // arrival counters of the four phases; each resets itself
    int32_t k;               // tiles to keep (Eq. 11)
    uint32_t prefix;         // key bits resolved so far, or kTakeNone
    int32_t remaining;       // tiles still to take among keys that carry `prefix`
    uint32_t T;              // threshold key
    int32_t e;               // keys equal to T to take, lowest tile index first
    int32_t pad;
    int64_t idx_off, val_off;  // payload offsets of the layer
};

// One worker of a compress call: its buffers and its own copy of the selection tables.  The
// selection and gather kernels of a call that serves several workers take one launch each;
// blockIdx.y picks the lane.
constexpr int kMaxLanes = 16;
struct Lane {
    uint32_t *keys;
    unsigned int *hist;        // n_layers * kHistStride
    LayerState *state;         // n_layers
    uint2 *chunk_cnt;          // one entry per key chunk
    unsigned short *chunk_sfx; // kL3Bins entries per key chunk
    unsigned char *codes;      // one byte per 4 tiles
    float *resid;
    int32_t *idx;
    void *val;                 // binary32 or bfloat16 payload values
};
struct LaneTable {
    Lane l[kMaxLanes];
};

struct RatioState {
    unsigned int ticket;
    uint32_t prefix;
    long long remaining;
    long long n_keep;
};

struct StatusDev {
    unsigned int flags, pad;
    unsigned long long nonfinite;
    long long idx_needed, val_needed;
    // extents of the plan's arenas and tables (constant after plan creation; rsdgc_get_status() resets
    // only what lies before them): what the bounds-checked build tests every index against
    long long arena_elems, keys_len;
    int n_layers, n_chunks, n_echunks, n_items;
};
constexpr size_t kStatusResetBytes = 32;  // flags .. val_needed

}  // namespace rsdgc

struct rsdgc_plan {
    int device = -1;  // < 0: host-only plan (sizing queries only)
    int n_layers = 0;
    int dtype = 0;
    float alpha = 0.5f;
    uint32_t flags = 0;
    int n_sm = 148;
    int reg_ctas_per_sm = 2;
    int item_elems = rsdgc::kItemElems;     // elements an item of the first pass may hold (depends on the gradient type)
    int grid_bulk = 0, grid_reg = 0;        // CTAs of the two accumulate+NSI kernels
    int n_items_bulk = 0, n_items_reg = 0;  // items_dev = [bulk items..., register items...]

    std::vector<rsdgc::LayerDev> layers;
    std::vector<rsdgc::Item> items;
    std::vector<rsdgc::ItemDev> items_dev;
    std::vector<int32_t> item_path, item_cta;          // per host item: kernel (0 bulk, 1 reg) and CTA
    std::vector<int32_t> item_pitch, item_flags;       // per host item: shared-memory row pitch, kItem* bits
    std::vector<int32_t> cta_begin_bulk, cta_begin_reg;  // grid + 1 indices into each kernel's item list
    std::vector<rsdgc::Chunk> chunks;
    std::vector<rsdgc::EChunk> echunks;
    // single-kernel tail (plans of small layers): slices of the cluster variant (n_tail_big of them, a
    // multiple of the cluster size), then those of the one-CTA variant; n_tail_clusters = 0: not eligible
    std::vector<rsdgc::TailSlice> tail_slices;
    int n_tail_big = 0, n_tail_small = 0, n_tail_clusters = 0;
    int tail_max_clusters = 16;  // clusters of the big variant the device holds at a time

    rsdgc_info info{};

    // device tables
    rsdgc::LayerDev *d_layers = nullptr;
    rsdgc::ItemDev *d_items = nullptr;
    int32_t *d_cta_begin_bulk = nullptr, *d_cta_begin_reg = nullptr;
    rsdgc::TailSlice *d_tail_slices = nullptr;
    rsdgc::Chunk *d_chunks = nullptr;
    rsdgc::EChunk *d_echunks = nullptr;
    rsdgc::LayerState *d_state = nullptr;
    uint32_t *d_hist = nullptr;        // n_layers * kHistStride
    unsigned char *d_codes = nullptr;  // one byte per 4 tiles: "above the threshold's bin" / "in it" flags for k_mark
    uint2 *d_chunk_cnt = nullptr;      // per key chunk: #keys above the bin, then exclusive bases (#key > T, #key == T)
    unsigned short *d_chunk_sfx = nullptr;  // per key chunk: suffix sums of its level-3 histogram (kL3Bins entries)
    // the same five tables for workers 1.. of rsdgc_compress_workers() (worker 0 uses the ones above)
    struct LaneScratch {
        rsdgc::LayerState *state = nullptr;
        uint32_t *hist = nullptr;
        unsigned char *codes = nullptr;
        uint2 *chunk_cnt = nullptr;
        unsigned short *chunk_sfx = nullptr;
    };
    std::vector<LaneScratch> extra_lanes;
    long long *d_survivors = nullptr;  // ratio rule: per-layer survivor counts
    rsdgc::RatioState *d_rstate = nullptr;
    rsdgc::StatusDev *d_status = nullptr;

    // rsdgc_compress_workers_host(): a second stream for the host-to-device copies and the events that
    // order it against the caller's stream (created on first use)
    cudaStream_t copy_stream = nullptr;
    std::vector<cudaEvent_t> order_events;

    // optional per-kernel timing of compress calls
    int profile = 0;                  // 0 off, 1 first pass only, 2 every stage
    int profile_recorded = 0;         // level of the calls recorded since the last read
    std::vector<cudaEvent_t> events;  // pool; 2 (level 1) or RSDGC_N_COMPRESS_KERNELS + 1 (level 2) per call
    size_t events_used = 0;
};

namespace rsdgc {

// host: builds every table of the plan from the layer descriptors (no CUDA calls)
int build_plan_tables(rsdgc_plan *p, const rsdgc_layer_desc *layers, int n_layers);

// launches (defined in the .cu files); each returns a cudaError_t
cudaError_t launch_compress(rsdgc_plan *p, const void *grads, float *resid, float *vel, float mom,
                            const float *ratios, int32_t *idx, int64_t idx_cap, void *val, int64_t val_cap,
                            int32_t *counts, uint32_t *keys, cudaStream_t s);
cudaError_t launch_compress_workers(rsdgc_plan *p, int n_workers, const void *const *grads, float *const *resid,
                                    const float *ratios, int32_t *const *idx, int64_t idx_cap, void *const *val,
                                    int64_t val_cap, int32_t *const *counts, uint32_t *keys_all, cudaStream_t s);
cudaError_t launch_update_ratios(rsdgc_plan *p, const float *weights, long long n_keep,
                                 float *ratios, cudaStream_t s);
cudaError_t launch_decompress(rsdgc_plan *p, int n_workers, const int32_t *const *idx, const void *const *val,
                              const int32_t *const *counts, long long idx_cap, long long val_cap, float scale,
                              float *dense, bool assign, cudaStream_t s);
cudaError_t launch_payload_to_coo(rsdgc_plan *p, const int32_t *idx, const int32_t *counts, long long *coo,
                                  long long coo_cap, cudaStream_t s);
cudaError_t launch_selftest_bounded_wait(rsdgc_plan *p, unsigned int polls, cudaStream_t s);
cudaError_t launch_tail(rsdgc_plan *p, const LaneTable &lanes, int n_lanes, const float *ratios, long long idx_cap,
                        long long val_cap, int prof, cudaStream_t s, cudaError_t (*mark)(rsdgc_plan *, cudaStream_t));
int tail_max_active_clusters();
void count_launch(int n);
void set_last_cuda_error(int e);
int k1_reg_ctas_per_sm(int dtype, bool momentum);
int k1_bulk_ctas_per_sm(bool momentum);
int bulk_item_elems(int dtype, bool momentum);
cudaError_t launch_accumulate_nsi(rsdgc_plan *p, uint32_t *hist, LayerState *state, const void *grads, float *resid,
                          float *vel, float mom, const float *ratios, int32_t *counts, uint32_t *keys,
                          cudaStream_t s, bool after_sibling = false, bool before_sibling = false);

}  // namespace rsdgc
