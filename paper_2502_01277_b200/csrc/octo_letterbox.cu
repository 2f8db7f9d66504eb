// Letterbox kernel: n BGR uint8 frames -> fp16 NCHW [n, 3, S, S] detector batch.
//
// HBM-bound gather.  One CTA produces kRows output rows of one frame.  The source rows
// those output rows tap (one row where the vertical weight is zero, e.g. the 3:1 reduction
// of 1080p, else two) are fetched whole into shared memory by the bulk-copy (TMA) engine
// with 16-byte coalesced transactions and an mbarrier; rows that carry no weight are never
// read.  While the copies are in flight the CTA builds a table of horizontal taps (byte
// offset + exact integer weights per canvas column).  Threads then take pixel pairs (lane l
// of a warp owns pixels 2l, 2l+1 of a 64-pixel run): the horizontal lerp is an exact integer
// two-way dot product per channel, the vertical lerp and all scaling are two fp32
// operations, and each warp writes 128 contiguous bytes per colour plane.
#include "octo_common.cuh"
#include "octo_kernels.h"

namespace octo {

constexpr int kLbThreads = 256;
constexpr int kLbRows = 8;  // most output rows a CTA produces; fewer for very wide frames

template <int CAP>
__global__ void __launch_bounds__(kLbThreads)
letterbox_kernel(const __grid_constant__ FrameTable<CAP> tab, __half* __restrict__ out, int S, int band_rows,
                 int slot_bytes, int nslots, uint32_t fill_h2, int swap_rb, unsigned int* __restrict__ status,
                 int pdl) {
    extern __shared__ __align__(128) unsigned char smem[];
    pdl_enter(pdl);
    __shared__ __align__(8) uint64_t bar;
    __shared__ __align__(16) RowInfo s_row[kLbRows];  // per-row data; step < 0 marks a canvas (pad) row

    const FrameDesc& fd = tab.f[blockIdx.y];
    const int dy0 = blockIdx.x * band_rows;
    const int w = fd.w, h = fd.h, nw = fd.nw, nh = fd.nh, pad_l = fd.pad_l, pad_t = fd.pad_t;
    const float inv_dx = 1.0f / (float)(2 * nw), inv_dy = 1.0f / (float)(2 * nh);
    // every scale factor folded into the vertical weights: 1 / (255 * den_x * den_y)
    const float inv_all = 1.0f / (255.0f * (float)(2 * nw) * (float)(2 * nh));
    const int chunks = S >> 3;
    const size_t plane = (size_t)S * (size_t)S;
    __half* const out_img = out + (size_t)blockIdx.y * 3 * plane;
    const uint4 fill4 = make_uint4(fill_h2, fill_h2, fill_h2, fill_h2);
    const int nrows = min(band_rows, S - dy0);
    // the staged rows start after the table of horizontal taps
    XEntry* const s_xtab = reinterpret_cast<XEntry*>(smem);
    unsigned char* const s_rows = smem + (((size_t)S * sizeof(XEntry) + 127) & ~(size_t)127);

    // Does this band touch the image at all?
    const bool any_image = max(dy0, pad_t) < min(dy0 + nrows, pad_t + nh);
    if (!any_image) {
        for (int t = threadIdx.x; t < nrows * chunks; t += kLbThreads) {
            const int r = t / chunks;
            __half* const o0 = out_img + (size_t)(dy0 + r) * S + ((t - r * chunks) << 3);
            *reinterpret_cast<uint4*>(o0) = fill4;
            *reinterpret_cast<uint4*>(o0 + plane) = fill4;
            *reinterpret_cast<uint4*>(o0 + 2 * plane) = fill4;
        }
        return;
    }

    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
        fence_proxy_async();
        const uint32_t row_bytes = (uint32_t)((3 * w + 15) & ~15);
        uint32_t total = 0;
        int slot = 0;
        for (int r = 0; r < nrows; ++r) {
            const int iy = dy0 + r - pad_t;
            RowInfo ri;
            ri.row0 = 0; ri.step = -1; ri.wx = 0.0f; ri.wy = 0.0f;
            if (iy < 0 || iy >= nh) { s_row[r] = ri; continue; }
            int y0, ry;
            src_coord(iy, h, nh, inv_dy, y0, ry);
            ri.row0 = slot * slot_bytes;
            ri.step = slot_bytes;
            ri.wx = (float)(2 * nh - ry) * inv_all;
            ri.wy = (float)ry * inv_all;
            s_row[r] = ri;
            slot += ry != 0 ? 2 : 1;
            total += row_bytes * (ry != 0 ? 2u : 1u);
        }
        mbar_expect_tx(&bar, total);
        slot = 0;
        for (int r = 0; r < nrows; ++r) {
            const int iy = dy0 + r - pad_t;
            if (iy < 0 || iy >= nh) continue;
            int y0, ry;
            src_coord(iy, h, nh, inv_dy, y0, ry);
            const uint8_t* src = fd.data + (size_t)y0 * (size_t)fd.pitch;
#ifdef OCTO_BOUNDS_CHECK
            if (!OCTO_IN_RANGE(slot + (ry != 0 ? 2 : 1) <= nslots && (int)row_bytes + 16 <= slot_bytes &&
                               y0 + (ry != 0 ? 1 : 0) < h && (int)row_bytes <= fd.pitch, status)) {
                // keep the barrier's byte count right without touching memory
                asm volatile("mbarrier.complete_tx.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&bar)),
                             "r"(row_bytes * (ry != 0 ? 2u : 1u)) : "memory");
                slot += ry != 0 ? 2 : 1;
                continue;
            }
#endif
            bulk_g2s(s_rows + (size_t)slot * slot_bytes, src, row_bytes, &bar);
            if (ry != 0) bulk_g2s(s_rows + (size_t)(slot + 1) * slot_bytes, src + fd.pitch, row_bytes, &bar);
            slot += ry != 0 ? 2 : 1;
        }
    }
    // table of horizontal taps, built while the copies are in flight
    for (int dx = threadIdx.x; dx < S; dx += kLbThreads) {
        const int ix = dx - pad_l;
        XEntry e;
        if (ix < 0 || ix >= nw) { e.off = 0; e.wts = 0; }  // zero weights mark a canvas column
        else e = make_xentry(ix, w, nw, inv_dx, 0);
        s_xtab[dx] = e;
    }
    __syncthreads();  // barrier armed, table and row weights visible
    bool copy_ok = mbar_wait_bounded(&bar, 0);
    if (!copy_ok) {
        // Give the copies in flight one more bounded chance to land before leaving.
        copy_ok = mbar_wait_bounded(&bar, 0);
        if (!copy_ok && threadIdx.x == 0) atomicOr(status, 0x4u);
    }

    // one warp per output row of the band
    const int pairs = S >> 1;
    const int lane = threadIdx.x & 31;
    const uint32_t rows_s = smem_u32(s_rows), xtab_s = smem_u32(s_xtab);
    __half* const out0 = out_img + (swap_rb ? 2 : 0) * plane;  // plane of input channel 0
    __half* const out1 = out_img + plane;
    __half* const out2 = out_img + (swap_rb ? 0 : 2) * plane;  // plane of input channel 2
    for (int r = threadIdx.x >> 5; r < nrows; r += kLbThreads / 32) {
        const RowInfo ri = s_row[r];
        const size_t o = (size_t)(dy0 + r) * S;
        if (ri.step < 0 || !copy_ok) {
            for (int pair = lane; pair < pairs; pair += 32) {
                *reinterpret_cast<uint32_t*>(out0 + o + 2 * pair) = fill_h2;
                *reinterpret_cast<uint32_t*>(out1 + o + 2 * pair) = fill_h2;
                *reinterpret_cast<uint32_t*>(out2 + o + 2 * pair) = fill_h2;
            }
        } else if (ri.wy != 0.0f) {
            sample_row<true, true>(rows_s + (uint32_t)ri.row0, (uint32_t)ri.step, ri.wx, ri.wy, xtab_s, pairs, lane,
                                   out0 + o, out1 + o, out2 + o, fill_h2);
        } else {
            sample_row<false, true>(rows_s + (uint32_t)ri.row0, (uint32_t)ri.step, ri.wx, ri.wy, xtab_s, pairs, lane,
                                    out0 + o, out1 + o, out2 + o, fill_h2);
        }
    }
}

// Staging slots an output row needs: one when every row of every frame taps a single source
// row (the vertical ratio is an odd integer, e.g. 1080 -> 360), else two.
static int slots_per_row(const FrameDesc* frames, int n) {
    for (int i = 0; i < n; ++i) {
        const int h = frames[i].h, nh = frames[i].nh;
        const bool single = (h % nh == 0) && ((h / nh) & 1);
        if (!single) return 2;
    }
    return 1;
}

static size_t lb_smem_bytes(int S, int slots, int slot_bytes) {
    return (((size_t)S * sizeof(XEntry) + 127) & ~(size_t)127) + (size_t)slots * slot_bytes;
}

template <int CAP>
static cudaError_t launch_cap(const FrameDesc* frames, int n, void* d_out, int S, int max_w, int pad_value,
                              int swap_rb, unsigned int* d_status, bool pdl, cudaStream_t stream) {
    FrameTable<CAP> tab;  // built per call (copied into kernel parameter space by the launch)
    for (int i = 0; i < n; ++i) tab.f[i] = frames[i];
    const int slot_bytes = ((3 * max_w + 15) & ~15) + 16;  // 16 bytes of slack: a tap reads 12 bytes from its word
    // rows per CTA: as many as fit about 56 KB of shared memory (four CTAs per SM), at most
    // kLbRows, at least one (a single row of the widest supported frame still fits)
    const int per_row = slots_per_row(frames, n) * slot_bytes;
    const long long room = 56 * 1024 - (long long)lb_smem_bytes(S, 0, slot_bytes);
    int band_rows = (int)(room / per_row);
    band_rows = band_rows < 1 ? 1 : (band_rows > kLbRows ? kLbRows : band_rows);
    // small batches: fewer rows per CTA so that the grid still covers the SMs about twice
    while (band_rows > 2 && (long long)n * ((S + band_rows - 1) / band_rows) < 296) band_rows >>= 1;
    const size_t smem = lb_smem_bytes(S, band_rows * slots_per_row(frames, n), slot_bytes);
    const __half hf = __double2half((double)pad_value / 255.0);  // one rounding, nearest even
    const uint32_t fb = *reinterpret_cast<const unsigned short*>(&hf);
    const uint32_t fill_h2 = fb | (fb << 16);
    dim3 grid((S + band_rows - 1) / band_rows, n);
    return launch_kernel(letterbox_kernel<CAP>, grid, dim3(kLbThreads), smem, stream, pdl, tab,
                         reinterpret_cast<__half*>(d_out), S, band_rows, slot_bytes,
                         band_rows * slots_per_row(frames, n), fill_h2, swap_rb, d_status, pdl ? 1 : 0);
}

// largest dynamic shared memory a launch may ask for (see kLetterboxMaxWidth)
constexpr int kLbMaxSmem = 227 * 1024 - 1024;

cudaError_t prepare_letterbox() {
    cudaError_t e;
    e = cudaFuncSetAttribute(letterbox_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLbMaxSmem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(letterbox_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLbMaxSmem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(letterbox_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize, kLbMaxSmem);
}

cudaError_t launch_letterbox(const FrameDesc* frames, int n, void* d_out, int S, int max_w, int pad_value,
                             int swap_rb, unsigned int* d_status, bool pdl, cudaStream_t stream) {
    if (n <= 8) return launch_cap<8>(frames, n, d_out, S, max_w, pad_value, swap_rb, d_status, pdl, stream);
    if (n <= 64) return launch_cap<64>(frames, n, d_out, S, max_w, pad_value, swap_rb, d_status, pdl, stream);
    return launch_cap<512>(frames, n, d_out, S, max_w, pad_value, swap_rb, d_status, pdl, stream);
}

}  // namespace octo
