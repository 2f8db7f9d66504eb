// Batch assembler and ROI crop-resize for one downstream branch.
//
// assemble_kernel (one CTA): exclusive prefix sum of the per-frame class-filtered detection
// counts -> offsets[n+1]; then the item table of the requested window (frame, detection,
// integer crop rectangle).  Integer work only.
//
// crop_kernel: HBM-write-bound.  A persistent grid strides over (slot, row band) work items;
// the number of packed items is read from device memory, so no host synchronisation sits
// between NMS and cropping.  Each thread produces 8 consecutive pixels of a row for all three
// planes and writes them with 16-byte stores straight into the slot of the downstream batch.
// Source taps are 32-bit words fetched through the read-only path (rectangles are small and
// overlap, so they are served by L1/L2 after first touch).
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

template <int CAP>
__global__ void __launch_bounds__(kCropThreads)
crop_kernel(const __grid_constant__ FrameTable<CAP> tab, const octo_item_t* __restrict__ items,
            const int* __restrict__ n_items, __half* __restrict__ out, int ow, int oh, int band_rows,
            int swap_rb) {
    const int packed = n_items[0];
    const int bands = (oh + band_rows - 1) / band_rows;
    const int chunks = ow >> 3;
    const size_t plane = (size_t)ow * (size_t)oh;
    const float inv_dx = 1.0f / (float)(2 * ow), inv_dy = 1.0f / (float)(2 * oh);
    const long long work = (long long)packed * bands;

    for (long long wi = blockIdx.x; wi < work; wi += gridDim.x) {
        const int slot = (int)(wi / bands);
        const int band = (int)(wi - (long long)slot * bands);
        const octo_item_t it = items[slot];
        const FrameDesc& fd = tab.f[it.frame];
        const int cw = it.rx1 - it.rx0, ch = it.ry1 - it.ry0;
        const int last_word = (fd.pitch >> 2) - 1;
        __half* const out_slot = out + (size_t)slot * 3 * plane;
        const int rows = min(band_rows, oh - band * band_rows);

        for (int t = threadIdx.x; t < rows * chunks; t += kCropThreads) {
            const int r = t / chunks;
            const int dx0 = (t - r * chunks) << 3;
            const int dy = band * band_rows + r;
            int y0, ry;
            src_coord(dy, ch, oh, inv_dy, y0, ry);
            const bool lerp_y = ry != 0;
            const float fy = (float)ry * inv_dy;
            const uint32_t* row0 =
                reinterpret_cast<const uint32_t*>(fd.data + (size_t)(it.ry0 + y0) * (size_t)fd.pitch);
            const uint32_t* row1 = reinterpret_cast<const uint32_t*>(reinterpret_cast<const uint8_t*>(row0) + fd.pitch);
            float v[3][8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                int x0, rx;
                src_coord(dx0 + i, cw, ow, inv_dx, x0, rx);
                const bool lerp_x = rx != 0;
                const float fx = (float)rx * inv_dx;
                const int o = 3 * (it.rx0 + x0);
                uint32_t lo, hi;
                float a0, a1, a2;
                load6(row0, o, last_word, lo, hi);
                row_taps(lo, hi, fx, lerp_x, a0, a1, a2);
                if (lerp_y) {
                    float b0, b1, b2;
                    load6(row1, o, last_word, lo, hi);
                    row_taps(lo, hi, fx, lerp_x, b0, b1, b2);
                    a0 = fmaf(fy, b0 - a0, a0);
                    a1 = fmaf(fy, b1 - a1, a1);
                    a2 = fmaf(fy, b2 - a2, a2);
                }
                v[0][i] = a0 * (1.0f / 255.0f);
                v[1][i] = a1 * (1.0f / 255.0f);
                v[2][i] = a2 * (1.0f / 255.0f);
            }
            __half* const o0 = out_slot + (size_t)dy * ow + dx0;
#pragma unroll
            for (int c = 0; c < 3; ++c) {
                uint32_t p[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) p[i] = pack_half2(v[c][2 * i], v[c][2 * i + 1]);
                const int pl = swap_rb ? 2 - c : c;
                *reinterpret_cast<uint4*>(o0 + (size_t)pl * plane) = make_uint4(p[0], p[1], p[2], p[3]);
            }
        }
    }
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
    int band_rows = 2048 / a.out_w;
    band_rows = band_rows < 1 ? 1 : (band_rows > a.out_h ? a.out_h : band_rows);
    const int bands = (a.out_h + band_rows - 1) / band_rows;
    long long work = (long long)a.max_items * bands;
    long long cap = (long long)a.sm_count * 8;
    const int grid = (int)(work < cap ? work : cap);
    crop_kernel<CAP><<<grid, kCropThreads, 0, stream>>>(tab, a.d_items, a.d_n_items,
                                                       reinterpret_cast<__half*>(a.d_out), a.out_w, a.out_h,
                                                       band_rows, a.swap_rb);
    return cudaGetLastError();
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
