// Batch assembler and ROI crop-resize for one downstream branch, in one kernel.
//
// Assembler (integer work only).  Every CTA scans the per-frame class-filtered detection
// counts of the branch (at most 512 integers) into shared memory: offsets[n+1], total and
// the number of items packed into the caller's window.  CTA 0 writes offsets / n_items.  An
// item is resolved where it is needed: slot -> frame by binary search in the offsets, ->
// detection through the branch's index list, -> outward-rounded integer rectangle.  The item
// table entry of a slot is written by the CTA that processes the slot's first row band.
//
// Crop-resize: bound by instruction issue and shared-memory wavefronts, then HBM (the fp16
// output is as large as the source rectangles).  A persistent grid works through (slot, row
// band) tiles (whole crops where there are many; the last crops of a launch are cut finer so
// that the grid ends together).  A CTA's first two tiles are fixed, the others come from an
// atomic counter, so no host synchronisation sits between NMS and cropping.  Inside a CTA one producer warp walks its tiles: it resolves the
// item, builds the table of horizontal taps (byte offset + exact integer weights per output
// column) and has the bulk-copy engine stage the source rows a pass taps into one of two
// shared-memory buffers (mbarrier "full" / "empty" ring, every wait bounded).  Every tapped
// source row is staged ONCE per pass: output rows that share a source row (always when the
// vertical scale is below 2) point at the same staged copy, so a pass covers as many output
// rows as its distinct source rows fit the buffer.
//
// Consumers own columns.  A consumer thread keeps two pairs of neighbouring output columns, half
// a tile apart (its four tap-table entries live in registers), and walks a run of consecutive
// output rows of the pass: the per-row work that does not depend on the column (row record,
// reuse decision, weights, addresses) is paid once for four pixels, and because the lanes of a
// warp hold neighbouring pairs in both halves, a warp's taps still fall on neighbouring bytes.
// The horizontal integer lerp of a staged row (an exact two-way dot product per channel) is
// kept in registers and reused by the next output row whenever that row taps the same source
// row: per output row only the NEW source rows cost a horizontal pass, i.e. about min(2,
// vertical scale) instead of 2.  The vertical lerp and all scaling are two packed fp32
// operations per channel, and a warp writes 128 contiguous bytes per plane, row and pair
// straight into the downstream slot.
#include "octo_common.cuh"
#include <cstring>

#include "octo_kernels.h"

namespace octo {

// Shared memory for staged source rows.  A row segment longer than kCropMaxStride - 16 bytes
// (a rectangle wider than about 5300 pixels) is split into column tiles, so two rows always
// fit.  Two buffers form a ring between the producer warp and the consumer warps.
constexpr int kCropStages = 2;         // ring depth (row buffers)
constexpr int kCropTables = kCropStages + 1;  // tap tables, one more than ring slots
constexpr int kCropRowBudget = 32768;  // bytes per ring buffer
constexpr int kCropMaxStride = kCropRowBudget / 2;
constexpr int kCropTilePx = 5300;
constexpr int kCropMaxPassRows = 32;   // one producer lane per output row of a pass
constexpr int kCropCtasPerSm = 3;
constexpr int kCropConsumerWarps = 7;   // with the producer warp 8 warps: 80 registers a thread at 3 CTAs per SM
constexpr int kCropConsumers = 32 * kCropConsumerWarps;
constexpr int kCropTailBands = 4;     // finer tiles for the last crops of a launch
constexpr int kCropTilesAhead = 2;   // tiles of a CTA that are fixed in advance and resolved side by side
constexpr int kCropTilesPerCta = 4;  // measured: 4 > 8 > 16 > 1 for small batches; a tile switch costs about 1 us
constexpr unsigned kCropProducerSleepNs = 200;  // between the producer's polls of an "empty" barrier
constexpr int kCropKernelThreads = kCropConsumers + 32;  // + one producer warp

// One pass of a CTA: output rows [r0, r0 + nr) x columns [c0, c0 + ncols) of one item.  The
// producer warp walks the CTA's sequence of passes and publishes each one for the consumers.
struct __align__(16) CropPass {
    int32_t valid;  // 0: no more passes
    int32_t table;  // which tap table the pass uses
    int32_t slot, r0, nr, c0, ncols;
    uint32_t magic;  // floor(2^32 / units per run) + 1: unit index -> row run by one multiplication
    int32_t run_rows;  // the pass is cut into runs of this many consecutive rows ...
    int32_t units;     // ... and (run, two column pairs) units are dealt to the consumer threads
    int32_t _pad[2];
};

// Per output row of a staged pass (RowInfo): row0 = byte offset of the staged copy of the top
// tap row, relative to the ring buffer and to the tap table's offsets; step = kRowStep bits:
// distance to the staged bottom tap row (0: the row has a single tap row) | reuse code << 16,
// or negative for a canvas row (nothing staged).  The reuse code tells a consumer that comes
// from the previous output row what it already holds:
//   0 both tap rows, 1 its bottom row is this row's top row, 2 nothing, 3 the top row only.
constexpr uint32_t kRowStepMask = 0xffffu;

// Horizontal integer lerp of one staged row for a pair of output columns, as exact binary32
// integers (the 2^23 offset of hsample is taken off again).
__device__ __forceinline__ void hpair(uint32_t addra, uint32_t sha, uint32_t wtsa, uint32_t addrb, uint32_t shb,
                                      uint32_t wtsb, unsigned long long& q0, unsigned long long& q1,
                                      unsigned long long& q2) {
    float a0, a1, a2, b0, b1, b2;
    hsample(addra, sha, wtsa, a0, a1, a2);
    hsample(addrb, shb, wtsb, b0, b1, b2);
    const unsigned long long m2 = f32x2(-kF32IntValue, -kF32IntValue);
    q0 = add_f32x2(f32x2(a0, b0), m2);
    q1 = add_f32x2(f32x2(a1, b1), m2);
    q2 = add_f32x2(f32x2(a2, b2), m2);
}

__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}

// QUEUE = false: items come from the stage's current batch through the assembler above.
// QUEUE = true: items are self-contained records popped from a device queue (qrec[0, *qpacked));
// the assembler is skipped and nothing but the crops is written.
//
// GENERAL = true adds the branch options: aspect-preserving fit (per item: fitted size nw x nh and
// offsets inside the slot, canvas columns marked by zero weights in the tap table, canvas rows by a
// negative row step) and per-plane normalisation (one fused multiply-add per value).  The plain
// form carries none of that code.
//
// The frame table comes either by value in kernel parameter space (`tab`, first-level stages:
// no table copy on the critical path) or from device memory (`gtab`, chained stages whose
// table an upstream stage's items define on the device).
template <int CAP, bool QUEUE, bool GENERAL>
__global__ void __launch_bounds__(kCropKernelThreads, kCropCtasPerSm)
crop_kernel(const __grid_constant__ FrameTable<CAP> tab, const FrameDesc* __restrict__ gtab, int n, int max_det,
            int first_item, int max_items,
            const int* __restrict__ bcount, const int* __restrict__ bidx, const octo_det_t* __restrict__ dets,
            int* __restrict__ offsets, int* __restrict__ n_items, octo_item_t* __restrict__ items,
            __half* __restrict__ out, int ow, int oh, int swap_rb, StageCounters* __restrict__ ctr,
            const QRecord* __restrict__ qrec, const int* __restrict__ qpacked, unsigned int* __restrict__ qstatus,
            int* __restrict__ sched, const CropOpts opts, int pdl) {
    extern __shared__ __align__(128) unsigned char smem[];
    pdl_enter(pdl);
    __shared__ __align__(8) uint64_t full[kCropStages], empty[kCropStages];
    __shared__ CropPass s_pass[kCropStages];
    __shared__ __align__(16) RowInfo s_row[kCropStages][kCropMaxPassRows];  // per-row data of the staged passes
    __shared__ int s_off[CAP + 1];                                // exclusive scan of the frame counts

    unsigned char* const s_rows0 = smem;
    XEntry* const s_xtab0 = reinterpret_cast<XEntry*>(smem + kCropStages * kCropRowBudget);  // kCropTables tables of ow entries
    unsigned int* const status = QUEUE ? qstatus : &ctr->status;

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // ---- assembler: offsets of the branch's items per frame ------------------------------------
    if (!QUEUE && warp == 0) {
        int run = 0;
        for (int base = 0; base < n; base += 32) {
            const int i = base + lane;
            const int v = i < n ? bcount[i] : 0;
            int inc = v;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, inc, off);
                if (lane >= off) inc += t;
            }
            if (i < n) s_off[i] = run + inc - v;
            run += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) s_off[n] = run;
    }
    if (threadIdx.x == 0) {
        for (int b = 0; b < kCropStages; ++b) {
            mbar_init(&full[b], 1);
            mbar_init(&empty[b], kCropConsumerWarps);
        }
        mbar_fence_init();
    }
    __syncthreads();
    const int total = QUEUE ? 0 : s_off[n];
    const long long rest = (long long)total - (long long)first_item;
    const int packed = QUEUE ? min(*qpacked, max_items) : (rest < 0 ? 0 : (rest > max_items ? max_items : (int)rest));
    if (!QUEUE && blockIdx.x == 0) {
        for (int i = threadIdx.x; i <= n; i += kCropKernelThreads) offsets[i] = s_off[i];
        if (threadIdx.x == 0) {
            n_items[0] = packed;
            n_items[1] = total;
            ctr->packed = packed;
            ctr->total_items = total;
            if ((long long)total > (long long)first_item + (long long)max_items) atomicOr(status, 0x2u);
        }
    }

    // Tiles are (slot, row band).  One band per crop amortises the per-tile work (item lookup, tap
    // table) best; crops are cut into bands (multiples of 8 rows) only as far as needed to give
    // every CTA about kCropTilesPerCta tiles, which keeps the end of the grid short.
    const int bands_want = packed > 0 ? (kCropTilesPerCta * (int)gridDim.x + packed - 1) / packed : 1;
    const int bands_req = min(max(bands_want, 1), (oh + 7) >> 3);
    const int band_rows = min(((oh + bands_req - 1) / bands_req + 7) & ~7, oh);
    const int bands = (oh + band_rows - 1) / band_rows;
    // The CTAs would end up to one tile apart, so the last crops (about one tile of the coarse cut
    // per CTA) are cut finer and even the end out: into kCropTailBands bands where a whole crop is a
    // tile, into twice as many bands as the others where crops are cut already.
    const int tail_req = min(bands == 1 ? kCropTailBands : 2 * bands, (oh + 7) >> 3);
    const int tail_rows = min(((oh + tail_req - 1) / tail_req + 7) & ~7, oh);
    const int tail_bands = (oh + tail_rows - 1) / tail_rows;
    const int tail_crops = tail_bands > bands ? min(packed, max((int)gridDim.x / bands, 1)) : 0;
    const long long coarse_tiles = (long long)(packed - tail_crops) * bands;
    const long long all_tiles = coarse_tiles + (long long)tail_crops * tail_bands;
    const size_t plane = (size_t)ow * (size_t)oh;

    if (warp == kCropConsumerWarps) {
        // =============================== producer warp ===================================
        const float inv_dx = 1.0f / (float)(2 * ow), inv_dy = 1.0f / (float)(2 * oh);
        // every scale factor folded into the vertical weights: 1 / (255 * den_x * den_y)
        const float inv_all = 1.0f / (255.0f * (float)(2 * ow) * (float)(2 * oh));
        // Tiles (index = slot * bands + band) are handed out dynamically: the first tiles of a CTA
        // are fixed, every further one comes from an atomic counter, so CTAs that drew cheap crops
        // (small source rectangles) take more of them and the grid finishes together.  The round
        // trips of a tile's resolution (counter -> detection index -> detection) are hidden behind
        // the passes that are already staged in the ring.
        int w_tiles = 0;  // tiles opened so far
        int w_slot = 0, w_band = 0, w_band_rows = band_rows;
        int w_pitch = 0, w_rx0 = 0, w_ry0 = 0, w_cw = 1, w_ch = 1;
        const uint8_t* w_data = nullptr;
        int w_row_lo = 0, w_row_hi = 0, w_tile_cols = ow;
        int w_c0 = 0, w_ncols = 0, w_r0 = 0;
        int w_seg_lo = 0, w_seg = 0, w_stride = 16, w_cap_slots = 2;
        int w_runs = 1;           // row runs that fit the consumer threads side by side
        uint32_t w_run_magic = 0, w_unit_magic = 0;  // divisions by w_runs / by the units of a run, as multiplications
        bool w_valid = false, w_new = false;
        // size and offset of the resized rectangle inside the slot: the whole slot unless the
        // branch keeps the aspect ratio
        int w_nw = ow, w_nh = oh, w_pl = 0, w_pt = 0;
        float w_inv_dx = inv_dx, w_inv_dy = inv_dy, w_inv_all = inv_all;
#ifdef OCTO_BOUNDS_CHECK
        int w_fh = 0;  // frame height, for the range check of the staged rows
#endif

        // geometry of the column tile starting at w_c0
        auto set_tile = [&]() {
            w_ncols = min(w_tile_cols, ow - w_c0);
            const int full_lo = (3 * w_rx0) & ~15;
            const int full_hi = (3 * (w_rx0 + w_cw) + 15) & ~15;
            int lo = full_lo, hi = full_hi;
            if (w_tile_cols != ow) {
                int xa, xb, rem;
                // canvas columns count as the nearest image column
                const int ia = min(max(w_c0 - w_pl, 0), w_nw - 1);
                const int ib = min(max(w_c0 + w_ncols - 1 - w_pl, 0), w_nw - 1);
                src_coord(ia, w_cw, w_nw, w_inv_dx, xa, rem);
                src_coord(ib, w_cw, w_nw, w_inv_dx, xb, rem);
                lo = (3 * (w_rx0 + xa)) & ~15;
                hi = min((3 * (w_rx0 + xb) + 6 + 15) & ~15, full_hi);
            }
            w_seg_lo = lo;
            w_seg = hi - lo;
            w_stride = w_seg + 16;
            w_cap_slots = kCropRowBudget / w_stride;  // >= 2
            // Work units of a pass: (run of consecutive rows, two column pairs half a tile apart).
            // A pass is cut into as many runs as fit the consumer threads side by side (224
            // columns: 4 runs x 56 units = the 224 consumer threads).
            const uint32_t quads = (uint32_t)max(w_ncols >> 2, 1);
            w_runs = max(1, min(kCropConsumers / (int)quads, kCropMaxPassRows));
            w_run_magic = w_runs > 1 ? 0xffffffffu / (uint32_t)w_runs + 1u : 0u;
            w_unit_magic = quads > 1u ? 0xffffffffu / quads + 1u : 0u;
        };
        // A tile resolved: (slot, band) -> item -> detection -> outward-rounded rectangle in its frame.
        // Three dependent global round trips when the tile number comes from the counter; no warp
        // collectives inside, so that the lanes may resolve different tiles side by side.
        struct Tile {
            int ok, slot, band, band_rows, f, det, rx0, ry0, rx1, ry1, pitch, fh;
            const uint8_t* data;
        };
        auto resolve = [&](long long tile) {
            Tile t;
            t.ok = tile < all_tiles ? 1 : 0;
            t.slot = 0; t.band = 0; t.band_rows = band_rows; t.f = 0; t.det = 0;
            t.rx0 = 0; t.ry0 = 0; t.rx1 = 1; t.ry1 = 1; t.pitch = 0; t.fh = 1; t.data = nullptr;
            if (!t.ok) return t;
            if (tile < coarse_tiles) {
                t.slot = (int)(tile / bands);
                t.band = (int)(tile - (long long)t.slot * bands);
            } else {
                const long long u = tile - coarse_tiles;
                t.slot = (packed - tail_crops) + (int)(u / tail_bands);
                t.band = (int)(u % tail_bands);
                t.band_rows = tail_rows;
            }
            if (QUEUE) {
                const QRecord rec = qrec[t.slot];
                t.data = rec.data; t.pitch = rec.pitch; t.fh = rec.h;
                t.rx0 = rec.rx0; t.ry0 = rec.ry0; t.rx1 = rec.rx1; t.ry1 = rec.ry1;
            } else {
                const int item = first_item + t.slot;
                int lo = 0, hi = n;  // largest f with s_off[f] <= item (frames without items are skipped)
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (s_off[mid] <= item) lo = mid; else hi = mid;
                }
                t.f = lo;
                if (OCTO_IN_RANGE(item - s_off[t.f] >= 0 && item - s_off[t.f] < max_det, status))
                    t.det = bidx[(size_t)t.f * max_det + (item - s_off[t.f])];
                if (!OCTO_IN_RANGE(t.det >= 0 && t.det < max_det, status)) t.det = 0;
                const octo_det_t d = dets[(size_t)t.f * max_det + t.det];
                const FrameDesc fd = gtab ? gtab[t.f] : tab.f[t.f];
                // outward-rounded rectangle, clamped so that it is never empty
                t.rx0 = (int)floorf(d.x1); t.ry0 = (int)floorf(d.y1);
                t.rx1 = (int)ceilf(d.x2); t.ry1 = (int)ceilf(d.y2);
                t.rx0 = min(max(t.rx0, 0), fd.w - 1);
                t.ry0 = min(max(t.ry0, 0), fd.h - 1);
                t.rx1 = min(max(t.rx1, t.rx0 + 1), fd.w);
                t.ry1 = min(max(t.ry1, t.ry0 + 1), fd.h);
                t.data = fd.data; t.pitch = fd.pitch; t.fh = fd.h;
            }
            return t;
        };
        // The first kCropTilesAhead tiles of a CTA are fixed (block index + j * grid size) and
        // resolved up front, lane j resolving tile j, so that their round trips overlap: with few
        // tiles per CTA (small batches) the chain is paid once, not once per tile.
        const Tile ahead = resolve(lane < kCropTilesAhead ? (long long)blockIdx.x + (long long)lane * (long long)gridDim.x
                                                          : all_tiles);
        // first pass of the next tile, if there is one
        auto open_tile = [&]() {
            Tile t;
            if (w_tiles < kCropTilesAhead) {
                const int src = w_tiles;
                t.ok = __shfl_sync(0xffffffffu, ahead.ok, src);
                t.slot = __shfl_sync(0xffffffffu, ahead.slot, src);
                t.band = __shfl_sync(0xffffffffu, ahead.band, src);
                t.band_rows = __shfl_sync(0xffffffffu, ahead.band_rows, src);
                t.f = __shfl_sync(0xffffffffu, ahead.f, src);
                t.det = __shfl_sync(0xffffffffu, ahead.det, src);
                t.rx0 = __shfl_sync(0xffffffffu, ahead.rx0, src);
                t.ry0 = __shfl_sync(0xffffffffu, ahead.ry0, src);
                t.rx1 = __shfl_sync(0xffffffffu, ahead.rx1, src);
                t.ry1 = __shfl_sync(0xffffffffu, ahead.ry1, src);
                t.pitch = __shfl_sync(0xffffffffu, ahead.pitch, src);
                t.fh = __shfl_sync(0xffffffffu, ahead.fh, src);
                t.data = reinterpret_cast<const uint8_t*>(
                    __shfl_sync(0xffffffffu, (unsigned long long)reinterpret_cast<uintptr_t>(ahead.data), src));
            } else {
                int c = 0;
                if (lane == 0) c = atomicAdd(sched, 1);
                t = resolve((long long)kCropTilesAhead * (long long)gridDim.x +
                            (long long)__shfl_sync(0xffffffffu, c, 0));
            }
            w_tiles += 1;
            w_valid = t.ok != 0;
            if (!w_valid) return;
            w_slot = t.slot; w_band = t.band; w_band_rows = t.band_rows;
            const int rx0 = t.rx0, ry0 = t.ry0, rx1 = t.rx1, ry1 = t.ry1;
            if (!QUEUE && w_band == 0 && lane == 0 && OCTO_IN_RANGE(w_slot >= 0 && w_slot < max_items, status)) {
                // the tile of a slot's first band records the item
                octo_item_t it;
                it.frame = t.f; it.det = t.det;
                it.rx0 = rx0; it.ry0 = ry0; it.rx1 = rx1; it.ry1 = ry1;
                it._pad[0] = 0; it._pad[1] = 0;
                items[w_slot] = it;
            }
            w_data = t.data; w_pitch = t.pitch;
#ifdef OCTO_BOUNDS_CHECK
            w_fh = t.fh;
#endif
            w_rx0 = rx0; w_ry0 = ry0; w_cw = rx1 - rx0; w_ch = ry1 - ry0;
            if (GENERAL && opts.keep_aspect) {
                // the side with the larger ratio fills the slot, the other is the exact quotient
                // rounded half-up (at least 1); centred, odd remainder right / bottom
                if ((long long)ow * w_ch <= (long long)oh * w_cw) {
                    w_nw = ow;
                    w_nh = max(1, (int)((2ll * w_ch * ow + w_cw) / (2ll * w_cw)));
                } else {
                    w_nh = oh;
                    w_nw = max(1, (int)((2ll * w_cw * oh + w_ch) / (2ll * w_ch)));
                }
                w_pl = (ow - w_nw) >> 1;
                w_pt = (oh - w_nh) >> 1;
                w_inv_dx = 1.0f / (float)(2 * w_nw);
                w_inv_dy = 1.0f / (float)(2 * w_nh);
                w_inv_all = 1.0f / (255.0f * (float)(2 * w_nw) * (float)(2 * w_nh));
            }
            const int full_seg = ((3 * rx1 + 15) & ~15) - ((3 * rx0) & ~15);
            w_tile_cols =
                (full_seg + 16 > kCropMaxStride) ? max(4, (int)((long long)kCropTilePx * w_nw / w_cw) & ~3) : ow;
            w_c0 = 0;
            set_tile();
            w_row_lo = w_band * w_band_rows;
            w_row_hi = min(w_row_lo + w_band_rows, oh);
            w_r0 = w_row_lo;
            w_new = true;
        };
        // the pass that was just published covered nr rows
        auto advance = [&](int nr) {
            w_new = false;
            if (w_r0 + nr < w_row_hi) {
                w_r0 += nr;
            } else if (w_c0 + w_ncols < ow) {
                w_c0 += w_ncols;
                set_tile();
                w_r0 = w_row_lo;
            } else {
                open_tile();
            }
        };

        open_tile();
        uint32_t ephase = 0u;  // bit b: parity of empty[b] to wait for
        int tb = kCropTables - 1;
        for (int k = 0;; ++k) {
            const int b = k % kCropStages;
            // ---- prepare the pass in registers; nothing of ring slot b is touched yet ----
            if (w_valid && w_new) {
                // taps of every output column: byte offset inside a frame row + integer weights.
                // Tables rotate with the tiles.  There is one more table than ring slots: the
                // passes still in flight (k - kCropStages .. k - 1) belong to at most kCropStages
                // tiles, so the table of the tile before those is free before this pass's wait.
                tb = (tb + 1) % kCropTables;
                XEntry* const xt = s_xtab0 + (size_t)tb * ow;
                for (int dx = lane; dx < ow; dx += 32) {
                    if (GENERAL) {
                        // a canvas column keeps the (valid) offset of the nearest image column
                        // and gets zero weights, which mark it for the consumers
                        const int ix = dx - w_pl, ixc = min(max(ix, 0), w_nw - 1);
                        XEntry e = make_xentry(ixc, w_cw, w_nw, w_inv_dx, 3 * w_rx0);
                        if (ix != ixc) e.wts = 0u;
                        xt[dx] = e;
                    } else {
                        xt[dx] = make_xentry(dx, w_cw, ow, inv_dx, 3 * w_rx0);
                    }
                }
            }
            // lane r stands for output row w_r0 + r; the pass takes the first nr of them
            const bool cand = w_valid && (w_r0 + lane < w_row_hi);
            const int iy = w_r0 + lane - w_pt;  // row inside the resized rectangle
            const bool has_row = cand && (!GENERAL || (iy >= 0 && iy < w_nh));
            int y0 = 0, ry = 0;
            if (has_row) src_coord(iy, w_ch, w_nh, w_inv_dy, y0, ry);
            const int need2 = ry != 0 ? 1 : 0;
            // Which of this row's tap rows (y0, and y0 + 1 if need2) did the row before it not
            // tap already?  Source rows never decrease from one output row to the next, so the
            // row before is the only one that can share them.
            const int maxrow = y0 + need2;
            int p_has = __shfl_up_sync(0xffffffffu, has_row ? 1 : 0, 1);
            const int p_max = __shfl_up_sync(0xffffffffu, maxrow, 1);
            const int p_need2 = __shfl_up_sync(0xffffffffu, need2, 1);
            if (lane == 0) p_has = 0;
            int newrows = 0, back = 0;
            uint32_t code = 2u;
            if (has_row) {
                if (!p_has || y0 > p_max) { newrows = 1 + need2; }
                else if (y0 == p_max) { newrows = need2; back = 1; code = p_need2 ? 1u : (need2 ? 3u : 0u); }
                else { back = 2; code = 0u; }  // y0 == p_max - 1: both rows are staged
            }
            // inclusive scan (staged rows up to and including this output row) from two votes: a row
            // brings 0, 1 or 2 new rows
            const unsigned upto = 0xffffffffu >> (31 - lane);
            const int incl = __popc(__ballot_sync(0xffffffffu, newrows & 1) & upto) +
                             2 * __popc(__ballot_sync(0xffffffffu, newrows >> 1) & upto);
            const int nr = __popc(__ballot_sync(0xffffffffu, cand && incl <= w_cap_slots));  // >= 1 when valid
            const bool in_pass = lane < nr;
            const int slot_top = incl - newrows - back;
            RowInfo ri;
            ri.row0 = 0; ri.step = 0; ri.wx = 0.0f; ri.wy = 0.0f;
            uint32_t bytes = 0;
            if (in_pass && has_row) {
                bytes = (uint32_t)(newrows * w_seg);
                ri.row0 = slot_top * w_stride - w_seg_lo;  // table offsets are relative to the frame row
                ri.step = (int32_t)((need2 ? (uint32_t)w_stride : 0u) | (code << 16));
                ri.wx = (float)(2 * w_nh - ry) * w_inv_all;
                ri.wy = (float)ry * w_inv_all;
            } else if (GENERAL) {
                ri.step = -1;  // canvas row: nothing is staged for it
            }
            const uint32_t total_tx = __reduce_add_sync(0xffffffffu, bytes);
            CropPass p;
            p.valid = w_valid ? 1 : 0;
            p.table = tb;
            p.slot = w_slot; p.r0 = w_r0; p.nr = nr; p.c0 = w_c0; p.ncols = w_ncols;
            p.magic = w_unit_magic;
            // rows per run = ceil(nr / runs); runs that start past the last row stay empty
            p.run_rows = w_runs > 1 ? (int)__umulhi((uint32_t)(nr + w_runs - 1), w_run_magic) : nr;
            p.units = (w_ncols >> 2) * w_runs;
            p._pad[0] = 0; p._pad[1] = 0;
            // ---- ring slot b: wait until the consumers have finished the pass that used it ----
            if (k >= kCropStages) {
                const uint32_t par = (ephase >> b) & 1u;
                if (!mbar_wait_sleeping(&empty[b], par, kCropProducerSleepNs) && !mbar_wait_sleeping(&empty[b], par, kCropProducerSleepNs)) {
                    if (lane == 0) atomicOr(status, 0x4u);
                    break;
                }
                ephase ^= 1u << b;
            }
            if (lane == 0) s_pass[b] = p;
            if (!w_valid) {
                __syncwarp();
                if (lane == 0) mbar_arrive(&full[b]);  // the end-of-work record
                break;
            }
            if (in_pass) s_row[b][lane] = ri;
            fence_proxy_async();
            __syncwarp();  // table, pass record and row data are written before the barrier is armed
            if (lane == 0) mbar_expect_tx(&full[b], total_tx);
            __syncwarp();
            if (in_pass && newrows > 0) {
                // the new rows are the last `newrows` of {y0, y0 + 1}
                const int first_new = need2 + 1 - newrows;  // 0: y0 is new, 1: only y0 + 1
                const int slot_new = slot_top + first_new;
                const uint8_t* src = w_data + (size_t)(w_ry0 + y0 + first_new) * (size_t)w_pitch + w_seg_lo;
                unsigned char* dst = s_rows0 + (size_t)b * kCropRowBudget + (size_t)slot_new * w_stride;
                bool ok = true;
#ifdef OCTO_BOUNDS_CHECK
                ok = OCTO_IN_RANGE(slot_new >= 0 && slot_new + newrows <= w_cap_slots &&
                                   (slot_new + newrows) * w_stride <= kCropRowBudget &&
                                   w_ry0 + y0 + first_new + newrows <= w_fh && w_seg_lo >= 0 &&
                                   w_seg_lo + w_seg <= w_pitch && (w_seg & 15) == 0, status);
                if (!ok) {  // keep the barrier's byte count right without touching memory
                    asm volatile("mbarrier.complete_tx.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&full[b])),
                                 "r"((uint32_t)(newrows * w_seg)) : "memory");
                }
#endif
                if (ok) {
                    bulk_g2s(dst, src, (uint32_t)w_seg, &full[b]);
                    if (newrows == 2) bulk_g2s(dst + w_stride, src + w_pitch, (uint32_t)w_seg, &full[b]);
                }
            }
            advance(nr);
        }
    } else {
        // =============================== consumer warps ==================================
        __half* const out0 = out + (swap_rb ? 2 : 0) * plane;  // plane of input channel 0
        __half* const out1 = out + plane;
        __half* const out2 = out + (swap_rb ? 0 : 2) * plane;  // plane of input channel 2
        uint32_t fphase = 0u;  // bit b: parity of full[b] to wait for
        for (int k = 0;; ++k) {
            const int b = k % kCropStages;
            const uint32_t par = (fphase >> b) & 1u;
            if (!mbar_wait_bounded(&full[b], par) && !mbar_wait_bounded(&full[b], par)) {
                if (lane == 0) atomicOr(status, 0x4u);
                break;
            }
            fphase ^= 1u << b;
            const CropPass cur = s_pass[b];
            if (!cur.valid) break;
            const uint32_t xt = smem_u32(s_xtab0) + (uint32_t)(cur.table * ow + cur.c0) * (uint32_t)sizeof(XEntry);
            const uint32_t rows = smem_u32(s_rows0) + (uint32_t)b * kCropRowBudget;
            const uint32_t rinfo = smem_u32(&s_row[b][0]);
            const size_t tile_off = (size_t)cur.slot * 3 * plane + (size_t)cur.r0 * ow + cur.c0;
            __half* const t0 = out0 + tile_off;
            __half* const t1 = out1 + tile_off;
            __half* const t2 = out2 + tile_off;
            // Work units (run of rows, two column pairs), laid out by the producer.  The warp that takes
            // the first units rotates from pass to pass: when the units do not fill every warp, a fixed
            // assignment would leave the same warp, hence the same scheduler of the SM (a warp's
            // scheduler follows from its index), idle in every pass of every CTA.  Padding the runs to
            // whole warps instead, so that no warp holds lanes of two runs, costs more (shorter runs
            // reuse fewer rows) than it saves waiting.
            const int quads = cur.ncols >> 2;
            for (int u = (int)((threadIdx.x + 32u * (uint32_t)k) % (uint32_t)kCropConsumers); u < cur.units;
                 u += kCropConsumers) {
                const int run = quads > 1 ? (int)__umulhi((uint32_t)u, cur.magic) : u;
                const int quad = u - run * quads;
                const int ra = run * cur.run_rows, rb = min(ra + cur.run_rows, cur.nr);
                // the unit's two column pairs lie half a tile apart, so that the lanes of a warp tap
                // neighbouring source bytes in both (four neighbouring columns per thread would double
                // the byte span of every load of the warp, and with it its shared-memory wavefronts)
                const uint4 ea = lds128(xt + 16u * (uint32_t)quad);            // XEntry {off, wts} x 2, first pair
                const uint4 eb = lds128(xt + 16u * (uint32_t)(quad + quads));  // ... second pair
                const uint32_t base0 = rows + (ea.x & ~3u), sh0 = ea.x << 3;
                const uint32_t base1 = rows + (ea.z & ~3u), sh1 = ea.z << 3;
                const uint32_t base2 = rows + (eb.x & ~3u), sh2 = eb.x << 3;
                const uint32_t base3 = rows + (eb.z & ~3u), sh3 = eb.z << 3;
                // horizontal lerps of the current top (T) and bottom (B) tap rows: three channels x
                // (columns 0, 1), then three channels x (columns 2, 3)
                unsigned long long T0 = 0ull, T1 = 0ull, T2 = 0ull, T3 = 0ull, T4 = 0ull, T5 = 0ull;
                unsigned long long B0 = 0ull, B1 = 0ull, B2 = 0ull, B3 = 0ull, B4 = 0ull, B5 = 0ull;
                uint32_t o = (uint32_t)(ra * ow + 2 * quad);
                const uint32_t oh2 = 2u * (uint32_t)quads;  // distance to the second pair
                for (int r = ra; r < rb; ++r, o += (uint32_t)ow) {
                    const uint4 rw = lds128(rinfo + 16u * (uint32_t)r);
                    if (GENERAL && (int)rw.y < 0) {  // canvas row
                        const uint32_t f0 = pack_half2(opts.fill[0], opts.fill[0]);
                        const uint32_t f1 = pack_half2(opts.fill[1], opts.fill[1]);
                        const uint32_t f2 = pack_half2(opts.fill[2], opts.fill[2]);
                        *reinterpret_cast<uint32_t*>(t0 + o) = f0;
                        *reinterpret_cast<uint32_t*>(t1 + o) = f1;
                        *reinterpret_cast<uint32_t*>(t2 + o) = f2;
                        *reinterpret_cast<uint32_t*>(t0 + o + oh2) = f0;
                        *reinterpret_cast<uint32_t*>(t1 + o + oh2) = f1;
                        *reinterpret_cast<uint32_t*>(t2 + o + oh2) = f2;
                        continue;
                    }
                    const uint32_t code = r == ra ? 2u : (rw.y >> 16) & 3u;
                    const uint32_t step = rw.y & kRowStepMask;
#ifdef OCTO_BOUNDS_CHECK
                    {
                        // every tap reads 12 bytes from its aligned word: both rows must lie in the buffer
                        const uint32_t omin = min(min(ea.x & ~3u, ea.z & ~3u), min(eb.x & ~3u, eb.z & ~3u));
                        const uint32_t omax = max(max(ea.x & ~3u, ea.z & ~3u), max(eb.x & ~3u, eb.z & ~3u));
                        const long long lo = (long long)(int)rw.x + (long long)omin;
                        const long long hi = (long long)(int)rw.x + (long long)omax + step + 12;
                        if (!OCTO_IN_RANGE(lo >= 0 && hi <= kCropRowBudget && r < kCropMaxPassRows &&
                                           cur.slot >= 0 && cur.slot < max_items && cur.r0 + r < oh &&
                                           cur.c0 + 2 * (quad + quads) + 1 < ow, status))
                            continue;
                    }
#endif
                    if (code == 2u) {
                        hpair(base0 + rw.x, sh0, ea.y, base1 + rw.x, sh1, ea.w, T0, T1, T2);
                        hpair(base2 + rw.x, sh2, eb.y, base3 + rw.x, sh3, eb.w, T3, T4, T5);
                    } else if (code == 1u) {
                        T0 = B0; T1 = B1; T2 = B2; T3 = B3; T4 = B4; T5 = B5;
                    }
                    if (code != 0u && step != 0u) {
                        const uint32_t rb1 = rw.x + step;
                        hpair(base0 + rb1, sh0, ea.y, base1 + rb1, sh1, ea.w, B0, B1, B2);
                        hpair(base2 + rb1, sh2, eb.y, base3 + rb1, sh3, eb.w, B3, B4, B5);
                    }
                    const float wx = __uint_as_float(rw.z), wy = __uint_as_float(rw.w);
                    const unsigned long long wx2 = f32x2(wx, wx), wy2 = f32x2(wy, wy);
                    // fl(fl(v0 * wx) + v1 * wy) per element (B is finite and wy = 0 when the row has one tap row)
                    const unsigned long long p0 = fma_f32x2(B0, wy2, mul_f32x2(T0, wx2));
                    const unsigned long long p1 = fma_f32x2(B1, wy2, mul_f32x2(T1, wx2));
                    const unsigned long long p2 = fma_f32x2(B2, wy2, mul_f32x2(T2, wx2));
                    const unsigned long long p3 = fma_f32x2(B3, wy2, mul_f32x2(T3, wx2));
                    const unsigned long long p4 = fma_f32x2(B4, wy2, mul_f32x2(T4, wx2));
                    const unsigned long long p5 = fma_f32x2(B5, wy2, mul_f32x2(T5, wx2));
                    if (!GENERAL) {
                        *reinterpret_cast<uint32_t*>(t0 + o) = half2_of_f32x2(p0);
                        *reinterpret_cast<uint32_t*>(t1 + o) = half2_of_f32x2(p1);
                        *reinterpret_cast<uint32_t*>(t2 + o) = half2_of_f32x2(p2);
                        *reinterpret_cast<uint32_t*>(t0 + o + oh2) = half2_of_f32x2(p3);
                        *reinterpret_cast<uint32_t*>(t1 + o + oh2) = half2_of_f32x2(p4);
                        *reinterpret_cast<uint32_t*>(t2 + o + oh2) = half2_of_f32x2(p5);
                    } else {
                        // per-plane scale and offset; zero weights mark a canvas column
                        auto finish = [&](unsigned long long lo01, unsigned long long hi23, int c) {
                            float v0, v1, v2, v3;
                            unpack_f32x2(lo01, v0, v1);
                            unpack_f32x2(hi23, v2, v3);
                            v0 = ea.y ? fmaf(v0, opts.sc[c], opts.of[c]) : opts.fill[c];
                            v1 = ea.w ? fmaf(v1, opts.sc[c], opts.of[c]) : opts.fill[c];
                            v2 = eb.y ? fmaf(v2, opts.sc[c], opts.of[c]) : opts.fill[c];
                            v3 = eb.w ? fmaf(v3, opts.sc[c], opts.of[c]) : opts.fill[c];
                            return make_uint2(pack_half2(v0, v1), pack_half2(v2, v3));
                        };
                        const uint2 h0 = finish(p0, p3, 0), h1 = finish(p1, p4, 1), h2 = finish(p2, p5, 2);
                        *reinterpret_cast<uint32_t*>(t0 + o) = h0.x;
                        *reinterpret_cast<uint32_t*>(t1 + o) = h1.x;
                        *reinterpret_cast<uint32_t*>(t2 + o) = h2.x;
                        *reinterpret_cast<uint32_t*>(t0 + o + oh2) = h0.y;
                        *reinterpret_cast<uint32_t*>(t1 + o + oh2) = h1.y;
                        *reinterpret_cast<uint32_t*>(t2 + o + oh2) = h2.y;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[b]);  // this warp is done with ring slot b
        }
    }
    // The last CTA to finish puts the tile counter back to zero for the next launch.
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(sched + 1, 1) == (int)gridDim.x - 1) {
            sched[0] = 0;
            sched[1] = 0;
            __threadfence();
        }
    }
}

static size_t crop_smem_bytes(int out_w) {
    return (size_t)kCropStages * kCropRowBudget + (size_t)kCropTables * sizeof(XEntry) * (size_t)out_w;
}

static int crop_grid(int sm_count, int slots, int out_h) {
    // The kernel cuts crops into row bands itself once it knows how many items there are; the
    // grid only has to be large enough for the finest cut.
    const long long cap = (long long)sm_count * kCropCtasPerSm;
    const long long work = (long long)slots * ((out_h + 7) / 8);
    const int grid = (int)(work < cap ? work : cap);
    return grid < 1 ? 1 : grid;  // a zero-slot window still gets its offsets and totals
}

template <int CAP>
static cudaError_t launch_crop_cap(const CropArgs& a, cudaStream_t stream) {
    FrameTable<CAP> tab;  // built per call (copied into kernel parameter space by the launch)
    if (!a.d_tab)
        for (int i = 0; i < a.n; ++i) tab.f[i] = a.frames[i];
    const int grid = crop_grid(a.sm_count, a.max_items, a.out_h);
    const size_t smem = crop_smem_bytes(a.out_w);
    auto kernel = a.general ? crop_kernel<CAP, false, true> : crop_kernel<CAP, false, false>;
    return launch_kernel(kernel, dim3(grid), dim3(kCropKernelThreads), smem, stream, a.pdl, tab, a.d_tab, a.n,
                         a.max_det, a.first_item, a.max_items, a.d_bcount, a.d_bidx, a.d_dets, a.d_offsets, a.d_n_items,
                         a.d_items, reinterpret_cast<__half*>(a.d_out), a.out_w, a.out_h, a.swap_rb, a.d_ctr,
                         (const QRecord*)nullptr, (const int*)nullptr, (unsigned int*)nullptr, a.d_ctr->sched, a.opts,
                         a.pdl ? 1 : 0);
}

cudaError_t prepare_crop() {
    const int smem = (int)crop_smem_bytes(2048);
    cudaError_t e;
    const void* kernels[] = {
        (const void*)crop_kernel<8, false, false>,   (const void*)crop_kernel<8, false, true>,
        (const void*)crop_kernel<64, false, false>,  (const void*)crop_kernel<64, false, true>,
        (const void*)crop_kernel<512, false, false>, (const void*)crop_kernel<512, false, true>,
        (const void*)crop_kernel<1, true, false>,    (const void*)crop_kernel<1, true, true>,
    };
    for (const void* k : kernels) {
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// Assembler + crop-resize of one branch window (a.max_items may be 0).  The capacity also sizes
// the shared-memory scan of the per-frame counts, so it follows n even when the frame table is
// read from device memory.
cudaError_t launch_crop(const CropArgs& a, cudaStream_t stream) {
    if (a.n <= 8) return launch_crop_cap<8>(a, stream);
    if (a.n <= 64) return launch_crop_cap<64>(a, stream);
    return launch_crop_cap<512>(a, stream);
}

// Crop the records staged by a queue pop (at most bz of them) into the downstream batch.
cudaError_t launch_crop_queue(const QRecord* d_staged, const int* d_qpacked, int bz, void* d_out, int out_w,
                              int out_h, int swap_rb, int sm_count, unsigned int* d_status, int* d_sched,
                              const CropOpts* general, cudaStream_t stream) {
    FrameTable<1> tab;  // unused in queue mode
    memset(&tab, 0, sizeof(tab));
    const int grid = crop_grid(sm_count, bz, out_h);
    const size_t smem = crop_smem_bytes(out_w);
    CropOpts opts;
    memset(&opts, 0, sizeof(opts));
    if (general) opts = *general;
    auto kernel = general ? crop_kernel<1, true, true> : crop_kernel<1, true, false>;
    return launch_kernel(kernel, dim3(grid), dim3(kCropKernelThreads), smem, stream, false, tab,
                         (const FrameDesc*)nullptr, 0, 0, 0, bz, (const int*)nullptr, (const int*)nullptr,
                         (const octo_det_t*)nullptr, (int*)nullptr, (int*)nullptr, (octo_item_t*)nullptr,
                         reinterpret_cast<__half*>(d_out), out_w, out_h, swap_rb, (StageCounters*)nullptr, d_staged,
                         d_qpacked, d_status, d_sched, opts, 0);
}

}  // namespace octo
