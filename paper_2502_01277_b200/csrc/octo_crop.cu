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
// band) tiles that an atomic counter hands out (whole crops, except that the last crops of a
// launch are cut into bands so that the grid ends together), so no host synchronisation sits
// between NMS and cropping.  Inside a CTA one producer warp walks its tiles: it resolves the
// item, builds the table of horizontal taps (byte offset + exact
// integer weights per output column) and has the bulk-copy engine stage the 16-byte aligned
// segments of the source rows a pass taps into one of two shared-memory buffers (mbarrier
// "full" / "empty" ring, every wait bounded).  The 256 threads of the eight consumer warps
// walk a pass as a flat, row-major list of pixel pairs, so every lane is busy and
// neighbouring lanes read neighbouring table entries and row words; the horizontal lerp is
// an exact integer two-way dot product per channel, the vertical lerp and all scaling are two
// fp32 operations, and a warp writes up to 128 contiguous bytes per plane straight into the
// downstream slot.  Measured: large passes matter more than occupancy (2 x 32 KB buffers at
// 3 CTAs/SM beat 2 x 24 KB at 4, 3 x 22 KB at 3 and 4 x 12 KB at 4).
#include "octo_common.cuh"
#include <cstring>

#include "octo_kernels.h"

namespace octo {

// Shared memory for staged source rows.  A pass stages two row segments per output row; a
// segment longer than kCropMaxStride - 16 bytes (a rectangle wider than about 5300 pixels)
// is split into column tiles, so one row pair always fits.  Two buffers form a ring between
// the producer warp and the consumer warps.
constexpr int kCropStages = 2;         // ring depth (row buffers)
constexpr int kCropTables = kCropStages + 1;  // tap tables, one more than ring slots
constexpr int kCropRowBudget = 32768;  // bytes per ring buffer
constexpr int kCropMaxStride = kCropRowBudget / 2;
constexpr int kCropTilePx = 5300;
constexpr int kCropMaxPassRows = 32;
constexpr int kCropCtasPerSm = 3;
constexpr int kCropConsumerWarps = 8;
constexpr int kCropTailBands = 4;     // finer tiles for the last crops of a launch
constexpr int kCropTilesPerCta = 4;  // measured: 4 > 8 > 16 > 1 for small batches; a tile switch costs about 1 us
constexpr unsigned kCropProducerSleepNs = 200;  // between the producer's polls of an "empty" barrier
constexpr int kCropKernelThreads = 32 * (kCropConsumerWarps + 1);  // + one producer warp

// One pass of a CTA: output rows [r0, r0 + nr) x columns [c0, c0 + ncols) of one item.  The
// producer warp walks the CTA's sequence of passes and publishes each one for the consumers.
struct __align__(16) CropPass {
    int32_t valid;  // 0: no more passes
    int32_t table;  // which tap table the pass uses
    int32_t slot, r0, nr, c0, ncols;
    int32_t _pad;
};

// QUEUE = false: items come from the stage's current batch through the assembler above.
// QUEUE = true: items are self-contained records popped from a device queue (qrec[0, *qpacked));
// the assembler is skipped and nothing but the crops is written.
//
// GENERAL = true adds the branch options: aspect-preserving fit (per item: fitted size nw x nh and
// offsets inside the slot, canvas columns marked by zero weights in the tap table, canvas rows by a
// negative row step) and per-plane normalisation (one fused multiply-add per value).  The plain
// form carries none of that code.
template <int CAP, bool QUEUE, bool GENERAL>
__global__ void __launch_bounds__(kCropKernelThreads, kCropCtasPerSm)
crop_kernel(const __grid_constant__ FrameTable<CAP> tab, int n, int max_det, int first_item, int max_items,
            const int* __restrict__ bcount, const int* __restrict__ bidx, const octo_det_t* __restrict__ dets,
            int* __restrict__ offsets, int* __restrict__ n_items, octo_item_t* __restrict__ items,
            __half* __restrict__ out, int ow, int oh, int swap_rb, StageCounters* __restrict__ ctr,
            const QRecord* __restrict__ qrec, const int* __restrict__ qpacked, unsigned int* __restrict__ qstatus,
            int* __restrict__ sched, const CropOpts opts) {
    extern __shared__ __align__(128) unsigned char smem[];
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
    // With whole crops as tiles the grid would end up to one crop apart, so the last crops (one
    // per CTA) are cut into up to kCropTailBands finer tiles that even the end out.
    const int tail_req = min(kCropTailBands, (oh + 7) >> 3);
    const int tail_rows = min(((oh + tail_req - 1) / tail_req + 7) & ~7, oh);
    const int tail_bands = (oh + tail_rows - 1) / tail_rows;
    const int tail_crops = (bands == 1 && tail_bands > 1) ? min(packed, (int)gridDim.x) : 0;
    const long long coarse_tiles = (long long)(packed - tail_crops) * bands;
    const long long all_tiles = coarse_tiles + (long long)tail_crops * tail_bands;
    const size_t plane = (size_t)ow * (size_t)oh;

    if (warp == kCropConsumerWarps) {
        // =============================== producer warp ===================================
        const float inv_dx = 1.0f / (float)(2 * ow), inv_dy = 1.0f / (float)(2 * oh);
        // every scale factor folded into the vertical weights: 1 / (255 * den_x * den_y)
        const float inv_all = 1.0f / (255.0f * (float)(2 * ow) * (float)(2 * oh));
        // Tiles (index = slot * bands + band) are handed out dynamically: the first tile of a CTA
        // is blockIdx.x, every further one comes from an atomic counter, so CTAs that drew cheap
        // crops (small source rectangles) take more of them and the grid finishes together.  The
        // round trips of a tile's resolution (counter -> detection index -> detection) are hidden
        // behind the passes that are already staged in the ring.
        int w_tiles = 0;  // tiles opened so far
        int w_slot = 0, w_band = 0, w_band_rows = band_rows;
        int w_pitch = 0, w_rx0 = 0, w_ry0 = 0, w_cw = 1, w_ch = 1;
        const uint8_t* w_data = nullptr;
        int w_row_lo = 0, w_row_hi = 0, w_tile_cols = ow;
        int w_c0 = 0, w_ncols = 0, w_r0 = 0, w_nr = 0;
        int w_seg_lo = 0, w_seg = 0, w_stride = 16, w_pass_rows = 1;
        bool w_valid = false, w_new = false;
        // size and offset of the resized rectangle inside the slot: the whole slot unless the
        // branch keeps the aspect ratio
        int w_nw = ow, w_nh = oh, w_pl = 0, w_pt = 0;
        float w_inv_dx = inv_dx, w_inv_dy = inv_dy, w_inv_all = inv_all;

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
            w_pass_rows = max(1, min(min(kCropRowBudget / (2 * w_stride), kCropMaxPassRows), w_band_rows));
        };
        // first pass of the next tile, if there is one; every lane resolves the same item
        auto open_tile = [&]() {
            long long tile = blockIdx.x;
            if (w_tiles > 0) {
                int t = 0;
                if (lane == 0) t = atomicAdd(sched, 1);
                tile = (long long)gridDim.x + (long long)__shfl_sync(0xffffffffu, t, 0);
            }
            w_tiles += 1;
            w_valid = tile < all_tiles;
            if (!w_valid) return;
            if (tile < coarse_tiles) {
                w_slot = (int)(tile / bands);
                w_band = (int)(tile - (long long)w_slot * bands);
                w_band_rows = band_rows;
            } else {
                const long long u = tile - coarse_tiles;
                w_slot = (packed - tail_crops) + (int)(u / tail_bands);
                w_band = (int)(u % tail_bands);
                w_band_rows = tail_rows;
            }
            int rx0, ry0, rx1, ry1;
            if (QUEUE) {
                const QRecord rec = qrec[w_slot];
                w_data = rec.data; w_pitch = rec.pitch;
                rx0 = rec.rx0; ry0 = rec.ry0; rx1 = rec.rx1; ry1 = rec.ry1;
            } else {
                const int item = first_item + w_slot;
                int lo = 0, hi = n;  // largest f with s_off[f] <= item (frames without items are skipped)
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (s_off[mid] <= item) lo = mid; else hi = mid;
                }
                const int f = lo;
                const int det = bidx[(size_t)f * max_det + (item - s_off[f])];
                const octo_det_t d = dets[(size_t)f * max_det + det];
                const FrameDesc& fd = tab.f[f];
                // outward-rounded rectangle, clamped so that it is never empty
                rx0 = (int)floorf(d.x1); ry0 = (int)floorf(d.y1);
                rx1 = (int)ceilf(d.x2); ry1 = (int)ceilf(d.y2);
                rx0 = min(max(rx0, 0), fd.w - 1);
                ry0 = min(max(ry0, 0), fd.h - 1);
                rx1 = min(max(rx1, rx0 + 1), fd.w);
                ry1 = min(max(ry1, ry0 + 1), fd.h);
                if (w_band == 0 && lane == 0) {  // the tile of a slot's first band records the item
                    octo_item_t it;
                    it.frame = f; it.det = det;
                    it.rx0 = rx0; it.ry0 = ry0; it.rx1 = rx1; it.ry1 = ry1;
                    it._pad[0] = 0; it._pad[1] = 0;
                    items[w_slot] = it;
                }
                w_data = fd.data; w_pitch = fd.pitch;
            }
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
                (full_seg + 16 > kCropMaxStride) ? max(2, (int)((long long)kCropTilePx * w_nw / w_cw) & ~1) : ow;
            w_c0 = 0;
            set_tile();
            w_row_lo = w_band * w_band_rows;
            w_row_hi = min(w_row_lo + w_band_rows, oh);
            w_r0 = w_row_lo;
            w_nr = min(w_pass_rows, w_row_hi - w_r0);
            w_new = true;
        };
        auto advance = [&]() {
            w_new = false;
            if (w_r0 + w_nr < w_row_hi) {
                w_r0 += w_nr;
            } else if (w_c0 + w_ncols < ow) {
                w_c0 += w_ncols;
                set_tile();
                w_r0 = w_row_lo;
            } else {
                open_tile();
                return;
            }
            w_nr = min(w_pass_rows, w_row_hi - w_r0);
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
            CropPass p;
            p.valid = w_valid ? 1 : 0;
            p.table = tb;
            p.slot = w_slot; p.r0 = w_r0; p.nr = w_nr; p.c0 = w_c0; p.ncols = w_ncols;
            p._pad = 0;
            // lane r owns output row w_r0 + r of the pass
            int ry = 0;
            uint32_t bytes = 0;
            RowInfo ri;
            ri.row0 = 0; ri.step = 0; ri.wx = 0.0f; ri.wy = 0.0f;
            const uint8_t* src = nullptr;
            const bool in_pass = w_valid && lane < w_nr;
            const int iy = w_r0 + lane - w_pt;  // row inside the resized rectangle
            const bool has_row = in_pass && (!GENERAL || (iy >= 0 && iy < w_nh));
            if (has_row) {
                int y0;
                src_coord(iy, w_ch, w_nh, w_inv_dy, y0, ry);
                bytes = (uint32_t)w_seg * (ry != 0 ? 2u : 1u);
                ri.row0 = 2 * lane * w_stride - w_seg_lo;  // table offsets are relative to the frame row
                ri.step = w_stride;
                ri.wx = (float)(2 * w_nh - ry) * w_inv_all;
                ri.wy = (float)ry * w_inv_all;
                src = w_data + (size_t)(w_ry0 + y0) * (size_t)w_pitch + w_seg_lo;
            } else if (GENERAL) {
                ri.step = -1;  // canvas row: nothing is staged for it
            }
            const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
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
            if (lane == 0) mbar_expect_tx(&full[b], total);
            __syncwarp();
            if (has_row) {
                unsigned char* dst = s_rows0 + (size_t)b * kCropRowBudget + (size_t)(2 * lane) * w_stride;
                bulk_g2s(dst, src, (uint32_t)w_seg, &full[b]);
                if (ry != 0) bulk_g2s(dst + w_stride, src + w_pitch, (uint32_t)w_seg, &full[b]);
            }
            advance();
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
            // flat list of pixel pairs (row-major); thread t of the consumers owns pairs t, t+256, ...
            const uint32_t xt = smem_u32(s_xtab0) + (uint32_t)(cur.table * ow + cur.c0) * (uint32_t)sizeof(XEntry);
            const uint32_t rows = smem_u32(s_rows0) + (uint32_t)b * kCropRowBudget;
            const uint32_t rinfo = smem_u32(&s_row[b][0]);
            const size_t tile_off = (size_t)cur.slot * 3 * plane + (size_t)cur.r0 * ow + cur.c0;
            __half* const t0 = out0 + tile_off;
            __half* const t1 = out1 + tile_off;
            __half* const t2 = out2 + tile_off;
            const int pairs = cur.ncols >> 1;
            const int npairs = cur.nr * pairs;
            // (row, pair) of this thread's first element, then advanced by the stride in place
            constexpr int kStride = 32 * kCropConsumerWarps;
            const int dr = kStride / pairs, dp = kStride - dr * pairs;
            int r = (int)threadIdx.x / pairs, pair = (int)threadIdx.x - r * pairs;
            for (int idx = threadIdx.x; idx < npairs; idx += kStride) {
                const uint4 rw = lds128(rinfo + 16u * (uint32_t)r);
                const uint4 ee = lds128(xt + 16u * (uint32_t)pair);
                const float wx = __uint_as_float(rw.z), wy = __uint_as_float(rw.w);
                const float nwx = -kF32IntValue * wx;
                if (!GENERAL) {
                    unsigned long long p0, p1, p2;
                    if (wy != 0.0f) sample_pair<true>(rows + rw.x, rw.y, ee.x, ee.y, ee.z, ee.w, wx, nwx, wy, p0, p1, p2);
                    else sample_pair<false>(rows + rw.x, rw.y, ee.x, ee.y, ee.z, ee.w, wx, nwx, wy, p0, p1, p2);
                    const uint32_t o = (uint32_t)(r * ow + 2 * pair);
                    *reinterpret_cast<uint32_t*>(t0 + o) = half2_of_f32x2(p0);
                    *reinterpret_cast<uint32_t*>(t1 + o) = half2_of_f32x2(p1);
                    *reinterpret_cast<uint32_t*>(t2 + o) = half2_of_f32x2(p2);
                } else {
                    float a0, a1, a2, b0, b1, b2;
                    if (GENERAL && (int)rw.y < 0) {  // canvas row
                        a0 = b0 = opts.fill[0]; a1 = b1 = opts.fill[1]; a2 = b2 = opts.fill[2];
                    } else {
                        if (wy != 0.0f) {
                            sample_px<true>(rows + rw.x, rw.y, ee.x, ee.y, wx, nwx, wy, a0, a1, a2);
                            sample_px<true>(rows + rw.x, rw.y, ee.z, ee.w, wx, nwx, wy, b0, b1, b2);
                        } else {
                            sample_px<false>(rows + rw.x, rw.y, ee.x, ee.y, wx, nwx, wy, a0, a1, a2);
                            sample_px<false>(rows + rw.x, rw.y, ee.z, ee.w, wx, nwx, wy, b0, b1, b2);
                        }
                        if (GENERAL) {
                            a0 = ee.y ? fmaf(a0, opts.sc[0], opts.of[0]) : opts.fill[0];
                            a1 = ee.y ? fmaf(a1, opts.sc[1], opts.of[1]) : opts.fill[1];
                            a2 = ee.y ? fmaf(a2, opts.sc[2], opts.of[2]) : opts.fill[2];
                            b0 = ee.w ? fmaf(b0, opts.sc[0], opts.of[0]) : opts.fill[0];
                            b1 = ee.w ? fmaf(b1, opts.sc[1], opts.of[1]) : opts.fill[1];
                            b2 = ee.w ? fmaf(b2, opts.sc[2], opts.of[2]) : opts.fill[2];
                        }
                    }
                    const uint32_t o = (uint32_t)(r * ow + 2 * pair);
                    *reinterpret_cast<uint32_t*>(t0 + o) = pack_half2(a0, b0);
                    *reinterpret_cast<uint32_t*>(t1 + o) = pack_half2(a1, b1);
                    *reinterpret_cast<uint32_t*>(t2 + o) = pack_half2(a2, b2);
                }
                r += dr;
                pair += dp;
                if (pair >= pairs) { pair -= pairs; ++r; }
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

template <int CAP>
static cudaError_t launch_crop_cap(const CropArgs& a, cudaStream_t stream) {
    static FrameTable<CAP> tab;
    for (int i = 0; i < a.n; ++i) tab.f[i] = a.frames[i];
    // The kernel cuts crops into row bands itself once it knows how many items there are; the
    // grid only has to be large enough for the finest cut.
    const long long cap = (long long)a.sm_count * kCropCtasPerSm;
    const long long work = (long long)a.max_items * ((a.out_h + 7) / 8);
    int grid = (int)(work < cap ? work : cap);
    if (grid < 1) grid = 1;  // a zero-slot window still gets its offsets and totals
    const size_t smem = (size_t)kCropStages * kCropRowBudget + (size_t)kCropTables * sizeof(XEntry) * (size_t)a.out_w;
    if (a.general)
        crop_kernel<CAP, false, true><<<grid, kCropKernelThreads, smem, stream>>>(
            tab, a.n, a.max_det, a.first_item, a.max_items, a.d_bcount, a.d_bidx, a.d_dets, a.d_offsets, a.d_n_items,
            a.d_items, reinterpret_cast<__half*>(a.d_out), a.out_w, a.out_h, a.swap_rb, a.d_ctr, nullptr, nullptr,
            nullptr, a.d_ctr->sched, a.opts);
    else
        crop_kernel<CAP, false, false><<<grid, kCropKernelThreads, smem, stream>>>(
            tab, a.n, a.max_det, a.first_item, a.max_items, a.d_bcount, a.d_bidx, a.d_dets, a.d_offsets, a.d_n_items,
            a.d_items, reinterpret_cast<__half*>(a.d_out), a.out_w, a.out_h, a.swap_rb, a.d_ctr, nullptr, nullptr,
            nullptr, a.d_ctr->sched, a.opts);
    return cudaGetLastError();
}

cudaError_t prepare_crop() {
    const int smem = kCropStages * kCropRowBudget + kCropTables * (int)sizeof(XEntry) * 2048;
    cudaError_t e;
    const void* kernels[] = {
        (const void*)crop_kernel<8, false, false>,   (const void*)crop_kernel<8, false, true>,
        (const void*)crop_kernel<64, false, false>,  (const void*)crop_kernel<64, false, true>,
        (const void*)crop_kernel<512, false, false>, (const void*)crop_kernel<512, false, true>,
        (const void*)crop_kernel<8, true, false>,    (const void*)crop_kernel<8, true, true>,
    };
    for (const void* k : kernels) {
        e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

// Assembler + crop-resize of one branch window (a.max_items may be 0).
cudaError_t launch_crop(const CropArgs& a, cudaStream_t stream) {
    if (a.n <= 8) return launch_crop_cap<8>(a, stream);
    if (a.n <= 64) return launch_crop_cap<64>(a, stream);
    return launch_crop_cap<512>(a, stream);
}

// Crop the records staged by a queue pop (at most bz of them) into the downstream batch.
cudaError_t launch_crop_queue(const QRecord* d_staged, const int* d_qpacked, int bz, void* d_out, int out_w,
                              int out_h, int swap_rb, int sm_count, unsigned int* d_status, int* d_sched,
                              const CropOpts* general, cudaStream_t stream) {
    static FrameTable<8> tab;  // unused in queue mode
    const long long cap = (long long)sm_count * kCropCtasPerSm;
    const long long work = (long long)bz * ((out_h + 7) / 8);
    const int grid = (int)(work < cap ? work : cap);
    const size_t smem = (size_t)kCropStages * kCropRowBudget + (size_t)kCropTables * sizeof(XEntry) * (size_t)out_w;
    CropOpts opts;
    memset(&opts, 0, sizeof(opts));
    if (general)
        crop_kernel<8, true, true><<<grid, kCropKernelThreads, smem, stream>>>(
            tab, 0, 0, 0, bz, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, reinterpret_cast<__half*>(d_out),
            out_w, out_h, swap_rb, nullptr, d_staged, d_qpacked, d_status, d_sched, *general);
    else
        crop_kernel<8, true, false><<<grid, kCropKernelThreads, smem, stream>>>(
            tab, 0, 0, 0, bz, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, reinterpret_cast<__half*>(d_out),
            out_w, out_h, swap_rb, nullptr, d_staged, d_qpacked, d_status, d_sched, opts);
    return cudaGetLastError();
}

}  // namespace octo
