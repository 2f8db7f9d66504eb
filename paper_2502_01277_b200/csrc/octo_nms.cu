// Per-image ordering + class-aware greedy NMS + cap + scale-back (one CTA per image).
//
// Latency / shared-memory bound; bytes are negligible.  The candidate keys of an image
// (class | inverted score bits | anchor) are sorted in shared memory with a bitonic network,
// which groups classes and orders each class by score (ties: lower anchor).  Boxes are
// gathered once from the head by anchor.  Classes are independent under class-aware NMS, so
// each warp runs the greedy scan of whole classes: 32 candidates at a time are tested
// against the class's survivors so far (broadcast reads of shared memory), then resolved
// among themselves with ballots and register shuffles.  Survivors are compacted in place,
// re-keyed to (inverted score | anchor | class) and sorted once more to obtain the global
// score order; the first max_det are mapped back to frame pixels and written out, together
// with each downstream branch's class-filtered index list.
//
// Images with more candidates than fit in shared memory take the same code path with the
// arrays in a global-memory workspace.
#include "octo_common.cuh"
#include "octo_kernels.h"

namespace octo {

constexpr int kNmsThreads = 1024;
constexpr int kNmsSmemCap = 8192;  // candidates sorted on chip: 8 B key + 16 B box each

__device__ __forceinline__ void bitonic_sort(unsigned long long* __restrict__ k, int np2) {
    for (int size = 2; size <= np2; size <<= 1) {
        for (int stride = size >> 1; stride > 0; stride >>= 1) {
            __syncthreads();
            for (int t = threadIdx.x; t < (np2 >> 1); t += kNmsThreads) {
                const int lo = 2 * t - (t & (stride - 1));  // index with bit `stride` clear
                const int hi = lo + stride;
                const unsigned long long a = k[lo], b = k[hi];
                const bool up = (lo & size) == 0;
                if ((a > b) == up) { k[lo] = b; k[hi] = a; }
            }
        }
    }
    __syncthreads();
}

__device__ __forceinline__ float4 gather_box(const float* __restrict__ hrow) {
    return box_corners(__ldg(hrow), __ldg(hrow + 1), __ldg(hrow + 2), __ldg(hrow + 3));
}

template <int CAP>
__global__ void __launch_bounds__(kNmsThreads)
nms_kernel(const __grid_constant__ FrameTable<CAP> tab, const float* __restrict__ head, int A, int C,
           float iou_thr, int max_det, int key_stride, unsigned long long* __restrict__ gkeys,
           float4* __restrict__ gboxes, int* __restrict__ cand_count, octo_det_rec* __restrict__ dets,
           int* __restrict__ counts, int num_branches, const __grid_constant__ BranchMasks masks,
           int* __restrict__ bcount, int* __restrict__ bidx, int max_batch, StageCounters* __restrict__ ctr) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ int seg_start[128], seg_end[128];
    __shared__ int s_total;

    const int img = blockIdx.x;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int row_len = 5 + C;
    const float* __restrict__ hbase = head + (size_t)img * (size_t)A * (size_t)row_len;

    int cnt = cand_count[img];
    cnt = min(cnt, min(A, key_stride));
    __syncthreads();
    if (threadIdx.x == 0) {
        cand_count[img] = 0;  // ready for the next batch's decode
        atomicAdd(&ctr->candidates, (unsigned long long)cnt);
        atomicMax(&ctr->max_cand, cnt);
        s_total = 0;
    }
    if (threadIdx.x < 128) { seg_start[threadIdx.x] = 0; seg_end[threadIdx.x] = 0; }

    int np2 = 2;
    while (np2 < cnt) np2 <<= 1;

    unsigned long long* keys;
    float4* boxes;
    unsigned long long* const gk = gkeys + (size_t)img * key_stride;
    if (np2 <= kNmsSmemCap) {
        keys = reinterpret_cast<unsigned long long*>(smem_raw + (size_t)kNmsSmemCap * sizeof(float4));
        boxes = reinterpret_cast<float4*>(smem_raw);
        for (int i = threadIdx.x; i < np2; i += kNmsThreads) keys[i] = i < cnt ? gk[i] : kKeySentinel;
    } else {
        keys = gk;  // key_stride is a power of two >= A, so the padded length fits
        boxes = gboxes + (size_t)img * key_stride;
        for (int i = cnt + threadIdx.x; i < np2; i += kNmsThreads) keys[i] = kKeySentinel;
        if (threadIdx.x == 0) atomicOr(&ctr->status, 0x8u);
    }

    if (cnt > 0) {
        // ---- class-major order: class, then score descending, then anchor ascending ----
        bitonic_sort(keys, np2);

        // ---- class segments and boxes ----
        for (int p = threadIdx.x; p < cnt; p += kNmsThreads) {
            const unsigned long long k = keys[p];
            const int cls = (int)(k >> 57);
            if (p == 0 || (int)(keys[p - 1] >> 57) != cls) seg_start[cls] = p;
            if (p == cnt - 1 || (int)(keys[p + 1] >> 57) != cls) seg_end[cls] = p + 1;
            const int anchor = (int)(k & ((1ull << kKeyAnchorBits) - 1));
            boxes[p] = gather_box(hbase + (size_t)anchor * row_len);
        }
        __syncthreads();

        // ---- greedy NMS, one warp per class ----
        for (int cls = warp; cls < 128; cls += kNmsThreads / 32) {
            const int s = seg_start[cls], e = seg_end[cls];
            int nk = 0;  // survivors of this class, compacted at [s, s + nk)
            for (int c0 = s; c0 < e && nk < max_det; c0 += 32) {
                const int p = c0 + lane;
                const bool valid = p < e;
                float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
                unsigned long long k = kKeySentinel;
                if (valid) { b = boxes[p]; k = keys[p]; }
                bool alive = valid;
                for (int t = 0; t < nk; ++t) {
                    if (!__any_sync(0xffffffffu, alive)) break;
                    const float4 kb = boxes[s + t];
                    if (alive && iou_fixed(kb, b) > iou_thr) alive = false;
                }
                unsigned rem = __ballot_sync(0xffffffffu, alive);
                unsigned keptmask = 0;
                while (rem) {
                    const int l = __ffs(rem) - 1;
                    keptmask |= 1u << l;
                    float4 lb;
                    lb.x = __shfl_sync(0xffffffffu, b.x, l);
                    lb.y = __shfl_sync(0xffffffffu, b.y, l);
                    lb.z = __shfl_sync(0xffffffffu, b.z, l);
                    lb.w = __shfl_sync(0xffffffffu, b.w, l);
                    if (alive && lane > l && iou_fixed(lb, b) > iou_thr) alive = false;
                    rem = __ballot_sync(0xffffffffu, alive) & ~((2u << l) - 1u);
                }
                __syncwarp();
                const int allowed = min(__popc(keptmask), max_det - nk);
                if ((keptmask >> lane) & 1u) {
                    const int r = __popc(keptmask & ((1u << lane) - 1u));
                    if (r < allowed) {
                        boxes[s + nk + r] = b;
                        // re-key for the global order: inverted score | anchor | class
                        keys[s + nk + r] = ((k & ((1ull << 57) - 1)) << 7) | (k >> 57);
                    }
                }
                __syncwarp();
                nk += allowed;
            }
            for (int p = s + nk + lane; p < e; p += 32) keys[p] = kKeySentinel;
            if (lane == 0 && nk > 0) atomicAdd(&s_total, nk);
        }

        // ---- global order of the survivors ----
        bitonic_sort(keys, np2);
    }
    __syncthreads();

    const int nout = min(s_total, max_det);
    const FrameDesc& fd = tab.f[img];
    const float fw = (float)fd.w, fh = (float)fd.h, fpl = (float)fd.pad_l, fpt = (float)fd.pad_t;
    for (int r = threadIdx.x; r < nout; r += kNmsThreads) {
        const unsigned long long g = keys[r];
        const int cls = (int)(g & 127u);
        const int anchor = (int)((g >> 7) & ((1ull << kKeyAnchorBits) - 1));
        const float score = __uint_as_float(~(unsigned)(g >> 32));
        const float4 b = gather_box(hbase + (size_t)anchor * row_len);
        octo_det_rec d;
        d.x1 = fminf(fmaxf(__fmul_rn(__fsub_rn(b.x, fpl), fd.gx), 0.0f), fw);
        d.y1 = fminf(fmaxf(__fmul_rn(__fsub_rn(b.y, fpt), fd.gy), 0.0f), fh);
        d.x2 = fminf(fmaxf(__fmul_rn(__fsub_rn(b.z, fpl), fd.gx), 0.0f), fw);
        d.y2 = fminf(fmaxf(__fmul_rn(__fsub_rn(b.w, fpt), fd.gy), 0.0f), fh);
        d.score = score;
        d.cls = cls;
        d.anchor = anchor;
        d._pad = 0;
        dets[(size_t)img * max_det + r] = d;
    }
    if (threadIdx.x == 0) {
        counts[img] = nout;
        atomicAdd(&ctr->kept, (unsigned long long)nout);
    }
    // ---- per-branch class-filtered index lists (stable), one warp per branch ----
    if (warp < num_branches) {
        int m = 0;
        int* const list = bidx + ((size_t)warp * max_batch + img) * max_det;
        for (int r0 = 0; r0 < nout; r0 += 32) {
            const int r = r0 + lane;
            bool take = false;
            if (r < nout) {
                const unsigned cls = (unsigned)(keys[r] & 127u);
                take = (masks.m[warp][cls >> 5] >> (cls & 31u)) & 1u;
            }
            const unsigned bal = __ballot_sync(0xffffffffu, take);
            if (take) list[m + __popc(bal & ((1u << lane) - 1u))] = r;
            m += __popc(bal);
        }
        if (lane == 0) bcount[warp * max_batch + img] = m;
    }
}

constexpr size_t kNmsSmemBytes = (size_t)kNmsSmemCap * (sizeof(float4) + sizeof(unsigned long long));

cudaError_t prepare_nms() {
    cudaError_t e;
    e = cudaFuncSetAttribute(nms_kernel<8>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kNmsSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(nms_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kNmsSmemBytes);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(nms_kernel<512>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kNmsSmemBytes);
}

template <int CAP>
static cudaError_t launch_cap(const NmsArgs& a, cudaStream_t stream) {
    static FrameTable<CAP> tab;
    for (int i = 0; i < a.n; ++i) tab.f[i] = a.frames[i];
    const size_t smem = kNmsSmemBytes;
    nms_kernel<CAP><<<a.n, kNmsThreads, smem, stream>>>(tab, a.d_head, a.A, a.C, a.iou_thr, a.max_det, a.key_stride,
                                                       a.d_keys, a.d_boxes, a.d_cand_count,
                                                       reinterpret_cast<octo_det_rec*>(a.d_dets), a.d_counts,
                                                       a.num_branches, a.masks, a.d_bcount, a.d_bidx, a.max_batch,
                                                       a.d_ctr);
    return cudaGetLastError();
}

cudaError_t launch_nms(const NmsArgs& a, cudaStream_t stream) {
    if (a.n <= 8) return launch_cap<8>(a, stream);
    if (a.n <= 64) return launch_cap<64>(a, stream);
    return launch_cap<512>(a, stream);
}

}  // namespace octo
