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
constexpr int kLbRows = 4;

template <int CAP>
__global__ void __launch_bounds__(kLbThreads)
letterbox_kernel(const __grid_constant__ FrameTable<CAP> tab, __half* __restrict__ out, int S,
                 int slot_bytes, uint32_t fill_h2, float fill_f, int swap_rb, unsigned int* __restrict__ status) {
    extern __shared__ __align__(128) unsigned char smem[];
    __shared__ __align__(8) uint64_t bar;

    const FrameDesc& fd = tab.f[blockIdx.y];
    const int dy0 = blockIdx.x * kLbRows;
    const int w = fd.w, h = fd.h, nw = fd.nw, nh = fd.nh, pad_l = fd.pad_l, pad_t = fd.pad_t;
    const float inv_dx = 1.0f / (float)(2 * nw), inv_dy = 1.0f / (float)(2 * nh);
    const int chunks = S >> 3;
    const size_t plane = (size_t)S * (size_t)S;
    __half* const out_img = out + (size_t)blockIdx.y * 3 * plane;
    const uint4 fill4 = make_uint4(fill_h2, fill_h2, fill_h2, fill_h2);

    // Does this band touch the image at all?
    const int band_lo = max(dy0, pad_t), band_hi = min(min(dy0 + kLbRows, S), pad_t + nh);
    const bool any_image = band_lo < band_hi;

    bool copy_ok = true;
    if (any_image) {
        if (threadIdx.x == 0) {
            mbar_init(&bar, 1);
            mbar_fence_init();
            fence_proxy_async();
            const uint32_t row_bytes = (uint32_t)((3 * w + 15) & ~15);
            uint32_t total = 0;
            for (int r = 0; r < kLbRows; ++r) {
                const int iy = dy0 + r - pad_t;
                if (iy < 0 || iy >= nh || dy0 + r >= S) continue;
                int y0, ry;
                src_coord(iy, h, nh, inv_dy, y0, ry);
                total += row_bytes * (ry != 0 ? 2u : 1u);
            }
            mbar_expect_tx(&bar, total);
            for (int r = 0; r < kLbRows; ++r) {
                const int iy = dy0 + r - pad_t;
                if (iy < 0 || iy >= nh || dy0 + r >= S) continue;
                int y0, ry;
                src_coord(iy, h, nh, inv_dy, y0, ry);
                const uint8_t* src = fd.data + (size_t)y0 * (size_t)fd.pitch;
                bulk_g2s(smem + (size_t)(2 * r) * slot_bytes, src, row_bytes, &bar);
                if (ry != 0)
                    bulk_g2s(smem + (size_t)(2 * r + 1) * slot_bytes, src + fd.pitch, row_bytes, &bar);
            }
        }
        __syncthreads();  // barrier initialised and visible before anyone polls it
        copy_ok = mbar_wait_bounded(&bar, 0);
        if (!copy_ok) {
            // Give the copies in flight one more bounded chance to land before leaving.
            copy_ok = mbar_wait_bounded(&bar, 0);
            if (!copy_ok && threadIdx.x == 0) atomicOr(status, 0x4u);
        }
    }

    const int last_word = (slot_bytes >> 2) - 1;
    for (int t = threadIdx.x; t < kLbRows * chunks; t += kLbThreads) {
        const int r = t / chunks;
        const int dx0 = (t - r * chunks) << 3;
        const int dy = dy0 + r;
        if (dy >= S) break;
        const int iy = dy - pad_t;
        __half* const o0 = out_img + (size_t)dy * S + dx0;
        if (iy < 0 || iy >= nh || !copy_ok) {
            *reinterpret_cast<uint4*>(o0) = fill4;
            *reinterpret_cast<uint4*>(o0 + plane) = fill4;
            *reinterpret_cast<uint4*>(o0 + 2 * plane) = fill4;
            continue;
        }
        int y0, ry;
        src_coord(iy, h, nh, inv_dy, y0, ry);
        const bool lerp_y = ry != 0;
        const float fy = (float)ry * inv_dy;
        const uint32_t* row0 = reinterpret_cast<const uint32_t*>(smem + (size_t)(2 * r) * slot_bytes);
        const uint32_t* row1 = reinterpret_cast<const uint32_t*>(smem + (size_t)(2 * r + 1) * slot_bytes);

        float v[3][8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int ix = dx0 + i - pad_l;
            if (ix < 0 || ix >= nw) {
                v[0][i] = v[1][i] = v[2][i] = fill_f;  // exact fp16 value, converts back unchanged
                continue;
            }
            int x0, rx;
            src_coord(ix, w, nw, inv_dx, x0, rx);
            const bool lerp_x = rx != 0;
            const float fx = (float)rx * inv_dx;
            uint32_t lo, hi;
            float a0, a1, a2;
            load6(row0, 3 * x0, last_word, lo, hi);
            row_taps(lo, hi, fx, lerp_x, a0, a1, a2);
            if (lerp_y) {
                float b0, b1, b2;
                load6(row1, 3 * x0, last_word, lo, hi);
                row_taps(lo, hi, fx, lerp_x, b0, b1, b2);
                a0 = fmaf(fy, b0 - a0, a0);
                a1 = fmaf(fy, b1 - a1, a1);
                a2 = fmaf(fy, b2 - a2, a2);
            }
            v[0][i] = a0 * (1.0f / 255.0f);
            v[1][i] = a1 * (1.0f / 255.0f);
            v[2][i] = a2 * (1.0f / 255.0f);
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

template <int CAP>
static cudaError_t launch_cap(const FrameDesc* frames, int n, void* d_out, int S, int max_w, int pad_value,
                              int swap_rb, unsigned int* d_status, cudaStream_t stream) {
    static FrameTable<CAP> tab;  // host staging; a stage is used from one thread at a time
    for (int i = 0; i < n; ++i) tab.f[i] = frames[i];
    const int slot_bytes = ((3 * max_w + 15) & ~15) + 16;
    const size_t smem = (size_t)2 * kLbRows * slot_bytes;
    const __half hf = __double2half((double)pad_value / 255.0);  // one rounding, nearest even
    const uint32_t fb = *reinterpret_cast<const unsigned short*>(&hf);
    const uint32_t fill_h2 = fb | (fb << 16);
    const float fill_f = __half2float(hf);
    dim3 grid((S + kLbRows - 1) / kLbRows, n);
    letterbox_kernel<CAP><<<grid, kLbThreads, smem, stream>>>(tab, reinterpret_cast<__half*>(d_out), S, slot_bytes,
                                                             fill_h2, fill_f, swap_rb, d_status);
    return cudaGetLastError();
}

constexpr int kLbMaxSmem = 2 * kLbRows * (((3 * kLetterboxMaxWidth + 15) & ~15) + 16);

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
