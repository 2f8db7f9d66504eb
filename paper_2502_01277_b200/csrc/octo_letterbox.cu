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
                 int slot_bytes, uint32_t fill_h2, float fill_f, int swap_rb, unsigned int* __restrict__ status) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ float2 s_roww[kLbRows];  // vertical weights; x < 0 marks a canvas (pad) row
    __shared__ int s_rowslot[kLbRows];  // first staging slot of the row

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
            if (iy < 0 || iy >= nh) { s_roww[r] = make_float2(-1.0f, 0.0f); s_rowslot[r] = 0; continue; }
            int y0, ry;
            src_coord(iy, h, nh, inv_dy, y0, ry);
            s_roww[r] = make_float2((float)(2 * nh - ry) * inv_all, (float)ry * inv_all);
            s_rowslot[r] = slot;
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

    // Lane l of a warp takes the pixel pair 2l, 2l+1 of a 64-pixel run: neighbouring lanes read
    // neighbouring table entries and row words, and the warp writes 128 contiguous bytes per plane.
    const int pairs = S >> 1;
    const size_t pl0 = swap_rb ? 2 : 0, pl2 = swap_rb ? 0 : 2;  // planes of input channels 0 and 2
    int r = 0, pair = threadIdx.x;
    while (pair >= pairs) { pair -= pairs; ++r; }
    for (; r < nrows;) {
        __half* const o0 = out_img + (size_t)(dy0 + r) * S + 2 * pair;
        const float2 wy = s_roww[r];
        if (wy.x < 0.0f || !copy_ok) {
            *reinterpret_cast<uint32_t*>(o0) = fill_h2;
            *reinterpret_cast<uint32_t*>(o0 + plane) = fill_h2;
            *reinterpret_cast<uint32_t*>(o0 + 2 * plane) = fill_h2;
        } else {
            const int slot = s_rowslot[r];
            const uint32_t* row0 = reinterpret_cast<const uint32_t*>(s_rows + (size_t)slot * slot_bytes);
            const uint32_t* row1 = reinterpret_cast<const uint32_t*>(s_rows + (size_t)(slot + 1) * slot_bytes);
            const uint4 ee = *reinterpret_cast<const uint4*>(s_xtab + 2 * pair);
            const XEntry e0 = {ee.x, ee.y}, e1 = {ee.z, ee.w};
            float f[6];
            if (wy.y != 0.0f) {
                sample_px<true>(row0, row1, e0, wy, f[0], f[1], f[2]);
                sample_px<true>(row0, row1, e1, wy, f[3], f[4], f[5]);
            } else {
                sample_px<false>(row0, row1, e0, wy, f[0], f[1], f[2]);
                sample_px<false>(row0, row1, e1, wy, f[3], f[4], f[5]);
            }
            // canvas columns outside the image carry zero weights: replace them by the fill
            // (an exact fp16 value, so it converts back unchanged)
            if (e0.wts == 0u) { f[0] = fill_f; f[1] = fill_f; f[2] = fill_f; }
            if (e1.wts == 0u) { f[3] = fill_f; f[4] = fill_f; f[5] = fill_f; }
            *reinterpret_cast<uint32_t*>(o0 + pl0 * plane) = pack_half2(f[0], f[3]);
            *reinterpret_cast<uint32_t*>(o0 + plane) = pack_half2(f[1], f[4]);
            *reinterpret_cast<uint32_t*>(o0 + pl2 * plane) = pack_half2(f[2], f[5]);
        }
        pair += kLbThreads;
        while (pair >= pairs) { pair -= pairs; ++r; }
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
                              int swap_rb, unsigned int* d_status, cudaStream_t stream) {
    static FrameTable<CAP> tab;  // host staging; a stage is used from one thread at a time
    for (int i = 0; i < n; ++i) tab.f[i] = frames[i];
    const int slot_bytes = ((3 * max_w + 15) & ~15) + 16;
    // rows per CTA: as many as fit about 56 KB of shared memory (four CTAs per SM), at most
    // kLbRows, at least one (a single row of the widest supported frame still fits)
    const int per_row = slots_per_row(frames, n) * slot_bytes;
    const long long room = 56 * 1024 - (long long)lb_smem_bytes(S, 0, slot_bytes);
    int band_rows = (int)(room / per_row);
    band_rows = band_rows < 1 ? 1 : (band_rows > kLbRows ? kLbRows : band_rows);
    const size_t smem = lb_smem_bytes(S, band_rows * slots_per_row(frames, n), slot_bytes);
    const __half hf = __double2half((double)pad_value / 255.0);  // one rounding, nearest even
    const uint32_t fb = *reinterpret_cast<const unsigned short*>(&hf);
    const uint32_t fill_h2 = fb | (fb << 16);
    const float fill_f = __half2float(hf);
    dim3 grid((S + band_rows - 1) / band_rows, n);
    letterbox_kernel<CAP><<<grid, kLbThreads, smem, stream>>>(tab, reinterpret_cast<__half*>(d_out), S, band_rows, slot_bytes,
                                                             fill_h2, fill_f, swap_rb, d_status);
    return cudaGetLastError();
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
                             int swap_rb, unsigned int* d_status, cudaStream_t stream) {
    if (n <= 8) return launch_cap<8>(frames, n, d_out, S, max_w, pad_value, swap_rb, d_status, stream);
    if (n <= 64) return launch_cap<64>(frames, n, d_out, S, max_w, pad_value, swap_rb, d_status, stream);
    return launch_cap<512>(frames, n, d_out, S, max_w, pad_value, swap_rb, d_status, stream);
}

}  // namespace octo
