// Letterbox kernel: n BGR uint8 frames -> fp16 NCHW [n, 3, S, S] detector batch.
//
// HBM-bound gather.  One CTA produces kRows output rows of one frame.  The source rows
// those output rows tap (one row where the vertical weight is zero, e.g. the 3:1 reduction
// of 1080p, else two) are fetched whole into shared memory by the bulk-copy (TMA) engine
// with 16-byte coalesced transactions and an mbarrier; rows that carry no weight are never
// read.  Threads then take 8 consecutive destination pixels each, read the 2x2 taps from
// shared memory as 32-bit words, interpolate in fp32 with exact rational sampling
// coordinates and write one 16-byte store per colour plane.
#include "octo_common.cuh"
#include "octo_kernels.h"

namespace octo {

constexpr int kLbThreads = 256;
constexpr int kLbRows = 8;  // most output rows a CTA produces; fewer for very wide frames
constexpr uint32_t kLbFillOff = 0xffffffffu;  // table entry of a canvas column outside the image

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
        if (ix < 0 || ix >= nw) { e.off = kLbFillOff; e.wts = 0; }
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

    for (int t = threadIdx.x; t < nrows * chunks; t += kLbThreads) {
        const int r = t / chunks;
        const int dx0 = (t - r * chunks) << 3;
        __half* const o0 = out_img + (size_t)(dy0 + r) * S + dx0;
        const float2 wy = s_roww[r];
        if (wy.x < 0.0f || !copy_ok) {
            *reinterpret_cast<uint4*>(o0) = fill4;
            *reinterpret_cast<uint4*>(o0 + plane) = fill4;
            *reinterpret_cast<uint4*>(o0 + 2 * plane) = fill4;
            continue;
        }
        const bool lerp_y = wy.y != 0.0f;
        const int slot = s_rowslot[r];
        const uint32_t* row0 = reinterpret_cast<const uint32_t*>(s_rows + (size_t)slot * slot_bytes);
        const uint32_t* row1 = reinterpret_cast<const uint32_t*>(s_rows + (size_t)(slot + 1) * slot_bytes);

        float v[3][8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const XEntry e = s_xtab[dx0 + i];
            if (e.off == kLbFillOff) {
                v[0][i] = v[1][i] = v[2][i] = fill_f;  // exact fp16 value, converts back unchanged
                continue;
            }
            uint32_t a0, a1, a2;
            hsample(row0, e, a0, a1, a2);
            float f0 = __uint2float_rn(a0) * wy.x, f1 = __uint2float_rn(a1) * wy.x, f2 = __uint2float_rn(a2) * wy.x;
            if (lerp_y) {
                uint32_t b0, b1, b2;
                hsample(row1, e, b0, b1, b2);
                f0 = fmaf(__uint2float_rn(b0), wy.y, f0);
                f1 = fmaf(__uint2float_rn(b1), wy.y, f1);
                f2 = fmaf(__uint2float_rn(b2), wy.y, f2);
            }
            v[0][i] = f0; v[1][i] = f1; v[2][i] = f2;
        }
#pragma unroll
        for (int c = 0; c < 3; ++c) {
            uint32_t p[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) p[i] = pack_half2(v[c][2 * i], v[c][2 * i + 1]);
            const int pl = swap_rb ? 2 - c : c;  // input channel c lands in plane pl
            *reinterpret_cast<uint4*>(o0 + (size_t)pl * plane) = make_uint4(p[0], p[1], p[2], p[3]);
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
