// Batch assembler and ROI crop-resize for one downstream branch.
//
// assemble_kernel (one CTA): exclusive prefix sum of the per-frame class-filtered detection
// counts -> offsets[n+1]; then the item table of the requested window (frame, detection,
// integer crop rectangle).  Integer work only.
//
// crop_kernel: HBM-bound (the fp16 output is as large as the source rectangles).  A
// persistent grid strides over (slot, row band) tiles; the number of packed items is read
// from device memory, so no host synchronisation sits between NMS and cropping.  Per tile the
// CTA builds a table of horizontal taps (byte offset + exact integer weights per column),
// one thread has the bulk-copy engine stage the 16-byte aligned segments of the source rows
// the band taps into shared memory (mbarrier, bounded wait), and every thread then produces
// pixel pairs (lane l of a warp takes pixels 2l, 2l+1 of a 64-pixel run, so table and row
// reads of neighbouring lanes fall into neighbouring banks): the horizontal lerp is an exact
// integer two-way dot product per channel, the vertical lerp and all scaling are two fp32
// operations, and each warp writes 128 contiguous bytes per plane straight into the
// downstream slot.
#include "octo_common.cuh"
#include "octo_kernels.h"

namespace octo {

constexpr int kAsmThreads = 1024;
constexpr int kCropThreads = 256;

template <int CAP>
__global__ void __launch_bounds__(kAsmThreads)
assemble_kernel(const __grid_constant__ FrameTable<CAP> tab, int n, int max_det, int first_item, int max_items,
                const int* __restrict__ bcount, const int* __restrict__ bidx,
                const octo_det_t* __restrict__ dets, int* __restrict__ offsets, int* __restrict__ n_items,
                octo_item_t* __restrict__ items, StageCounters* __restrict__ ctr) {
    __shared__ int s_off[CAP + 1];
    __shared__ int s_warp[kAsmThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // exclusive scan of up to CAP (<= 1024) counts: one element per thread
    static_assert(CAP <= kAsmThreads, "one count per thread");
    {
        const int v = threadIdx.x < n ? bcount[threadIdx.x] : 0;
        int inc = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, inc, off);
            if (lane >= off) inc += t;
        }
        if (lane == 31) s_warp[warp] = inc;
        __syncthreads();
        if (warp == 0) {
            int w = s_warp[lane];
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, w, off);
                if (lane >= off) w += t;
            }
            s_warp[lane] = w;  // inclusive over warps
        }
        __syncthreads();
        const int base = warp > 0 ? s_warp[warp - 1] : 0;
        if (threadIdx.x < n) s_off[threadIdx.x] = base + inc - v;
        if (threadIdx.x == n - 1) s_off[n] = base + inc;
    }
    __syncthreads();
    const int total = s_off[n];
    for (int i = threadIdx.x; i <= n; i += kAsmThreads) offsets[i] = s_off[i];
    if (threadIdx.x == 0) {
        long long rest = (long long)total - (long long)first_item;
        int packed = rest < 0 ? 0 : (rest > max_items ? max_items : (int)rest);
        n_items[0] = packed;
        n_items[1] = total;
        ctr->packed = packed;
        ctr->total_items = total;
        if ((long long)total > (long long)first_item + (long long)max_items) atomicOr(&ctr->status, 0x2u);
    }
    // item table of the window; one warp per frame
    for (int f = warp; f < n; f += kAsmThreads / 32) {
        const int o = s_off[f], m = s_off[f + 1] - o;
        const FrameDesc& fd = tab.f[f];
        for (int j = lane; j < m; j += 32) {
            const long long slot = (long long)o + j - first_item;
            if (slot < 0 || slot >= max_items) continue;
            const int det = bidx[(size_t)f * max_det + j];
            const octo_det_t d = dets[(size_t)f * max_det + det];
            // outward-rounded rectangle, clamped so that it is never empty
            int rx0 = (int)floorf(d.x1), ry0 = (int)floorf(d.y1);
            int rx1 = (int)ceilf(d.x2), ry1 = (int)ceilf(d.y2);
            rx0 = min(max(rx0, 0), fd.w - 1);
            ry0 = min(max(ry0, 0), fd.h - 1);
            rx1 = min(max(rx1, rx0 + 1), fd.w);
            ry1 = min(max(ry1, ry0 + 1), fd.h);
            octo_item_t it;
            it.frame = f; it.det = det;
            it.rx0 = rx0; it.ry0 = ry0; it.rx1 = rx1; it.ry1 = ry1;
            it._pad[0] = 0; it._pad[1] = 0;
            items[slot] = it;
        }
    }
}

// Bytes of shared memory for staged source rows: two rows of the widest supported frame.
constexpr int kCropRowBudget = 2 * (3 * kLetterboxMaxWidth + 64);
constexpr int kCropMaxPassRows = 32;

template <int CAP>
__global__ void __launch_bounds__(kCropThreads, 4)
crop_kernel(const __grid_constant__ FrameTable<CAP> tab, const octo_item_t* __restrict__ items,
            const int* __restrict__ n_items, __half* __restrict__ out, int ow, int oh, int band_rows,
            int swap_rb, unsigned int* __restrict__ status) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ float2 s_roww[kCropMaxPassRows];  // vertical weights of the rows of a pass

    unsigned char* const s_rows = smem;
    XEntry* const s_xtab = reinterpret_cast<XEntry*>(smem + kCropRowBudget);

    const int packed = n_items[0];
    const int bands = (oh + band_rows - 1) / band_rows;
    const int pairs = ow >> 1;
    const size_t plane = (size_t)ow * (size_t)oh;
    const size_t pl0 = swap_rb ? 2 : 0, pl2 = swap_rb ? 0 : 2;  // planes of input channels 0 and 2
    const float inv_dx = 1.0f / (float)(2 * ow), inv_dy = 1.0f / (float)(2 * oh);
    // every scale factor folded into the vertical weights: 1 / (255 * den_x * den_y)
    const float inv_all = 1.0f / (255.0f * (float)(2 * ow) * (float)(2 * oh));
    const long long work = (long long)packed * bands;

    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
    }
    uint32_t phase = 0;
    bool failed = false;

    for (long long wi = blockIdx.x; wi < work; wi += gridDim.x) {
        const int slot = (int)(wi / bands);
        const int band = (int)(wi - (long long)slot * bands);
        const octo_item_t it = items[slot];
        const FrameDesc& fd = tab.f[it.frame];
        const int cw = it.rx1 - it.rx0, ch = it.ry1 - it.ry0;
        // 16-byte aligned byte range of the rectangle's columns inside a frame row
        const int seg_lo = (3 * it.rx0) & ~15;
        const int seg = ((3 * it.rx1 + 15) & ~15) - seg_lo;
        const int stride = seg + 16;
        int pass_rows = kCropRowBudget / (2 * stride);
        pass_rows = min(min(pass_rows, kCropMaxPassRows), band_rows);
        __half* const out_slot = out + (size_t)slot * 3 * plane;
        const int row_lo = band * band_rows;
        const int row_hi = min(row_lo + band_rows, oh);

        __syncthreads();  // everyone is done with the previous tile's table and rows
        for (int dx = threadIdx.x; dx < ow; dx += kCropThreads)
            s_xtab[dx] = make_xentry(dx, cw, ow, inv_dx, 3 * it.rx0 - seg_lo);

        for (int r0 = row_lo; r0 < row_hi; r0 += pass_rows) {
            const int nr = min(pass_rows, row_hi - r0);
            if (r0 != row_lo) __syncthreads();  // previous pass fully consumed
            if (threadIdx.x < 32) {
                // warp 0 stages the pass: lane r owns output row r0 + r
                const int r = threadIdx.x;
                int y0 = 0, ry = 0;
                uint32_t bytes = 0;
                if (r < nr) {
                    src_coord(r0 + r, ch, oh, inv_dy, y0, ry);
                    bytes = (uint32_t)seg * (ry != 0 ? 2u : 1u);
                    s_roww[r] = make_float2((float)(2 * oh - ry) * inv_all, (float)ry * inv_all);
                }
                const uint32_t total = __reduce_add_sync(0xffffffffu, bytes);
                fence_proxy_async();
                if (r == 0) mbar_expect_tx(&bar, total);
                __syncwarp();
                if (r < nr) {
                    const uint8_t* src = fd.data + (size_t)(it.ry0 + y0) * (size_t)fd.pitch + seg_lo;
                    bulk_g2s(s_rows + (size_t)(2 * r) * stride, src, (uint32_t)seg, &bar);
                    if (ry != 0) bulk_g2s(s_rows + (size_t)(2 * r + 1) * stride, src + fd.pitch, (uint32_t)seg, &bar);
                }
            }
            __syncthreads();  // table, row weights and the armed barrier are visible
            if (!failed && !mbar_wait_bounded(&bar, phase)) {
                if (!mbar_wait_bounded(&bar, phase)) failed = true;
            }
            phase ^= 1u;
            if (failed) continue;

            // Lane l of a warp takes the pixel pair 2l, 2l+1 of a 64-pixel run: neighbouring
            // lanes read neighbouring table entries and row words (no bank conflicts) and the
            // warp writes 128 contiguous bytes per plane.
            int r = 0, pair = threadIdx.x;
            while (pair >= pairs) { pair -= pairs; ++r; }
            for (; r < nr;) {
                const float2 wy = s_roww[r];
                const uint32_t* row0 = reinterpret_cast<const uint32_t*>(s_rows + (size_t)(2 * r) * stride);
                const uint32_t* row1 = reinterpret_cast<const uint32_t*>(s_rows + (size_t)(2 * r + 1) * stride);
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
                __half* const o0 = out_slot + (size_t)(r0 + r) * ow + 2 * pair;
                *reinterpret_cast<uint32_t*>(o0 + pl0 * plane) = pack_half2(f[0], f[3]);
                *reinterpret_cast<uint32_t*>(o0 + plane) = pack_half2(f[1], f[4]);
                *reinterpret_cast<uint32_t*>(o0 + pl2 * plane) = pack_half2(f[2], f[5]);
                pair += kCropThreads;
                while (pair >= pairs) { pair -= pairs; ++r; }
            }
        }
    }
    if (failed && threadIdx.x == 0) atomicOr(status, 0x4u);
}

template <int CAP>
static cudaError_t launch_assemble_cap(const CropArgs& a, cudaStream_t stream) {
    static FrameTable<CAP> tab;
    for (int i = 0; i < a.n; ++i) tab.f[i] = a.frames[i];
    assemble_kernel<CAP><<<1, kAsmThreads, 0, stream>>>(tab, a.n, a.max_det, a.first_item, a.max_items, a.d_bcount,
                                                       a.d_bidx, a.d_dets, a.d_offsets, a.d_n_items, a.d_items,
                                                       a.d_ctr);
    return cudaGetLastError();
}

template <int CAP>
static cudaError_t launch_crop_cap(const CropArgs& a, cudaStream_t stream) {
    static FrameTable<CAP> tab;
    for (int i = 0; i < a.n; ++i) tab.f[i] = a.frames[i];
    int band_rows = 4096 / a.out_w;
    band_rows = band_rows < 1 ? 1 : (band_rows > a.out_h ? a.out_h : band_rows);
    const int bands = (a.out_h + band_rows - 1) / band_rows;
    long long work = (long long)a.max_items * bands;
    long long cap = (long long)a.sm_count * 4;
    const int grid = (int)(work < cap ? work : cap);
    const size_t smem = (size_t)kCropRowBudget + sizeof(XEntry) * (size_t)a.out_w;
    crop_kernel<CAP><<<grid, kCropThreads, smem, stream>>>(tab, a.d_items, a.d_n_items,
                                                          reinterpret_cast<__half*>(a.d_out), a.out_w, a.out_h,
                                                          band_rows, a.swap_rb, &a.d_ctr->status);
    return cudaGetLastError();
}

cudaError_t prepare_crop() {
    const int smem = kCropRowBudget + (int)sizeof(XEntry) * 2048;
    cudaError_t e;
    e = cudaFuncSetAttribute(crop_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(crop_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(crop_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
}

cudaError_t launch_assemble(const CropArgs& a, cudaStream_t stream) {
    if (a.n <= 8) return launch_assemble_cap<8>(a, stream);
    if (a.n <= 64) return launch_assemble_cap<64>(a, stream);
    return launch_assemble_cap<512>(a, stream);
}

// Requires a.max_items > 0.
cudaError_t launch_crop(const CropArgs& a, cudaStream_t stream) {
    if (a.n <= 8) return launch_crop_cap<8>(a, stream);
    if (a.n <= 64) return launch_crop_cap<64>(a, stream);
    return launch_crop_cap<512>(a, stream);
}

}  // namespace octo
