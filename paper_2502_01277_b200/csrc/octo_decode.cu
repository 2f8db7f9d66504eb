// Decode + confidence filter + compaction of a YOLOv5-layout head [n, A, 5 + C] fp32.
//
// HBM-bound scan.  For logit heads sigma <= 1 makes sigma(obj) > conf a necessary condition
// for score = fl(sigma(obj) * sigma(cls)) > conf, so the scan reads only the obj value of
// each 340-byte row (one DRAM sector) and fetches the whole row, 32 bytes at a time by a group
// of eight lanes (four passing rows per warp in flight together), for the few anchors that pass.  Probability heads are read densely.  A passing row is
// reduced by eight lanes (finite check, first-maximum class), scored in the fixed binary32
// sequence and appended to the image's key list with one atomic; the key carries class,
// inverted score bits and anchor, so later steps need nothing else from this kernel and the
// nondeterministic append order is erased by the sort.
//
// Variants.  Multi-label: a passing row yields one key per class whose own score exceeds the
// threshold.  Planes layout [n, 4 + C, A] (anchor-free heads without objectness): consecutive
// anchors are contiguous in every plane, so the scan is a dense, coalesced read of the C class
// planes (the whole head must be read: the maximum over classes needs every value); the four
// box planes are read only for anchors whose score passes.
#include "octo_common.cuh"
#include <cmath>

#include "octo_kernels.h"

namespace octo {

constexpr int kDecThreads = 256;

// Read-only load that asks L2 to fetch 64 bytes around the address instead of the default
// 128: the obj scan touches 4 bytes per 340-byte row, so the smaller fill granularity cuts
// the DRAM traffic of the scan (measured: 27 % less time for the bare scan).  The values are used
// once, so they are kept out of L1 as well (another 3.6 %).
__device__ __forceinline__ float ld_obj(const float* p) {
    float v;
    asm volatile("ld.global.nc.L1::no_allocate.L2::64B.f32 %0, [%1];" : "=f"(v) : "l"(p));
    return v;
}

// Candidate key: class | inverted score bits | anchor (ascending key = descending score, then
// ascending anchor inside a class).
__device__ __forceinline__ unsigned long long make_key(int cls, float score, int anchor) {
    return ((unsigned long long)(unsigned)cls << 57) | ((unsigned long long)(~__float_as_uint(score)) << kKeyAnchorBits) |
           (unsigned long long)(unsigned)anchor;
}

// kDecPerThread anchors per thread: 4 for large batches, 1 when the grid would otherwise be
// too small to cover the SMs.
template <int kDecPerThread>
__global__ void __launch_bounds__(kDecThreads)
decode_kernel(const float* __restrict__ head, int A, int C, int mode, float conf, int key_stride,
              unsigned long long* __restrict__ keys, int* __restrict__ cand_count,
              unsigned int* __restrict__ status, int pdl) {
    pdl_enter(pdl);
    // mode bit 0: obj / class values are logits; bit 1: class-agnostic NMS (key class field 0);
    // bit 2: multi-label candidates
    const int logits = mode & 1;
    const bool agnostic = (mode & 2) != 0;
    const bool multi = (mode & 4) != 0;
    const int img = blockIdx.y;
    const int row_len = 5 + C;
    const float* __restrict__ hbase = head + (size_t)img * (size_t)A * (size_t)row_len;
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int grp = lane >> 3, gl = lane & 7, gbase = lane & 24;  // group of eight lanes, lane in it, its first lane
    const unsigned gmask = 0xffu << gbase;
    // each warp owns kDecPerThread consecutive groups of 32 anchors
    const int a_warp = blockIdx.x * (kDecThreads * kDecPerThread) + warp * (32 * kDecPerThread);

    float obj[kDecPerThread];
#pragma unroll
    for (int u = 0; u < kDecPerThread; ++u) {
        const int a = a_warp + u * 32 + lane;
        obj[u] = (logits && a < A) ? ld_obj(hbase + (size_t)a * row_len + 4) : 0.0f;
    }
    bool nonfinite_seen = false;
#pragma unroll
    for (int u = 0; u < kDecPerThread; ++u) {
        const int a = a_warp + u * 32 + lane;
        bool pass = a < A;
        if (logits && pass) {
            const bool fin = finite_f(obj[u]);
            nonfinite_seen |= !fin;
            pass = fin && sigmoid_fixed(obj[u]) > conf;
        }
        // Passing rows are reduced four at a time, one per group of eight lanes (a row is read in
        // 32-byte pieces, lane g of a group holds elements g, g + 8, ...): the four row fetches are in
        // flight together and a row costs a quarter of the warp's instructions.
        unsigned todo = __ballot_sync(0xffffffffu, pass);
        while (todo) {
            unsigned mine = todo;  // this group's row: the grp-th lowest set bit
            for (int i = 0; i < grp; ++i) mine &= mine - 1;
            const bool have = mine != 0u;
            const int src = have ? __ffs(mine) - 1 : 0;
#pragma unroll
            for (int i = 0; i < 4; ++i) todo &= todo - 1;  // the four lowest rows are taken
            const int ra = a_warp + u * 32 + src;
            const float* __restrict__ row = hbase + (size_t)ra * row_len;
            bool fin = true;
            float best = -INFINITY;
            int best_k = 0x7fffffff;
            float e0 = 0.0f;
            if (have) {
                // the row is requested in batches of kPieces 32-byte pieces (48 values per group), so
                // a row of 85 values takes two round trips and the kernel stays at 32-40 registers
                // (the obj scan of large batches lives on occupancy); the small-grid form asks for
                // the whole row at once (any row of up to 5 + 128 values): one round trip less
                constexpr int kPieces = kDecPerThread == 1 ? 17 : 6;
                for (int e00 = 0; e00 < row_len; e00 += 8 * kPieces) {
                    float v[kPieces];
#pragma unroll
                    for (int j = 0; j < kPieces; ++j) {
                        const int e = e00 + gl + 8 * j;
                        v[j] = e < row_len ? __ldg(row + e) : 0.0f;
                    }
                    if (e00 == 0) e0 = v[0];
#pragma unroll
                    for (int j = 0; j < kPieces; ++j) {
                        const int e = e00 + gl + 8 * j;
                        if (e < row_len) {
                            fin &= finite_f(v[j]);
                            if (e >= 5 && v[j] > best) { best = v[j]; best_k = e - 5; }
                        }
                    }
                }
            }
            const unsigned bad = __ballot_sync(0xffffffffu, !fin) & gmask;
            const float bw = __shfl_sync(0xffffffffu, e0, gbase + 2);
            const float bh = __shfl_sync(0xffffffffu, e0, gbase + 3);
            const float ob = __shfl_sync(0xffffffffu, e0, gbase + 4);
            if (bad) nonfinite_seen = true;
            const bool ok = have && !bad && bw > 0.0f && bh > 0.0f;
            if (!multi) {
#pragma unroll
                for (int off = 4; off > 0; off >>= 1) {  // first maximum over the group's eight lanes
                    const float ov = __shfl_xor_sync(0xffffffffu, best, off);
                    const int ok2 = __shfl_xor_sync(0xffffffffu, best_k, off);
                    if (ov > best || (ov == best && ok2 < best_k)) { best = ov; best_k = ok2; }
                }
                if (ok && gl == 0) {
                    const float score = logits ? __fmul_rn(sigmoid_fixed(ob), sigmoid_fixed(best))
                                               : __fmul_rn(ob, best);
                    if (score > conf) {
                        const int slot = atomicAdd(cand_count + img, 1);
                        if (slot < key_stride)
                            keys[(size_t)img * key_stride + slot] = make_key(agnostic ? 0 : best_k, score, ra);
                        else
                            atomicOr(status, 0x10u);
                    }
                }
            } else {
                // one candidate per class whose own score passes; the keys of a row go out in
                // groups of up to eight with one counter update per group
                const float so = logits ? sigmoid_fixed(ob) : ob;
                for (int e0i = 0; e0i < row_len; e0i += 8) {  // the same trip count in every group
                    const int e = e0i + gl;
                    float score = 0.0f;
                    bool hit = false;
                    if (ok && e >= 5 && e < row_len) {
                        const float v = __ldg(row + e);  // second pass over the row: an L1 hit
                        score = __fmul_rn(so, logits ? sigmoid_fixed(v) : v);
                        hit = score > conf;
                    }
                    const unsigned hits = __ballot_sync(0xffffffffu, hit) & gmask;
                    int base = 0;
                    if (hits != 0u && gl == 0) base = atomicAdd(cand_count + img, __popc(hits));
                    base = __shfl_sync(0xffffffffu, base, gbase);
                    if (hit) {
                        const int slot = base + __popc(hits & ((1u << lane) - 1u));
                        if (slot < key_stride) keys[(size_t)img * key_stride + slot] = make_key(e - 5, score, ra);
                        else atomicOr(status, 0x10u);
                    }
                }
            }
        }
    }
    if (__any_sync(0xffffffffu, nonfinite_seen) && lane == 0) atomicOr(status, 0x1u);
}

// Planes layout [n, 4 + C, A].  A thread owns VEC consecutive anchors (VEC = 4 with 16-byte
// loads when A is a multiple of 4, else 1); the lanes of a warp and kPlaneAnchorWarps warps side
// by side read consecutive addresses of one plane, so a CTA fetches long contiguous runs (DRAM
// pages are used better the longer the run).  kPlaneClassWarps groups of warps split the C class
// planes between them (group g takes classes g, g + groups, ...) and leave their running first
// maxima in shared memory, where one thread per anchor merges them.  For multi-label heads in logit form a value is only run
// through the fixed logistic sequence when it lies above `pre`, a bound placed safely below
// the threshold's logit, so that the common case costs one comparison per value.
// Measured on [256, 84, 8400]: 8 x 1 warps (4 KB contiguous per plane and CTA) 0.141 ms, 4 x 2
// 0.142, 2 x 4 0.156, 1 x 8 0.167; the unroll depth makes no difference from 2 to 16.
constexpr int kPlaneUnroll = 8;
constexpr int kPlaneAnchorWarps = 8;                          // warps side by side along the anchors
constexpr int kPlaneClassWarps = kDecThreads / 32 / kPlaneAnchorWarps;  // warps splitting the classes

template <int VEC>
__global__ void __launch_bounds__(kDecThreads)
decode_planes_kernel(const float* __restrict__ head, int A, int C, int mode, float conf, float pre, int key_stride,
                     unsigned long long* __restrict__ keys, int* __restrict__ cand_count,
                     unsigned int* __restrict__ status, int pdl) {
    pdl_enter(pdl);
    constexpr int kCtaAnchors = kPlaneAnchorWarps * 32 * VEC;
    __shared__ float s_best[kPlaneClassWarps][kCtaAnchors];
    __shared__ int s_k[kPlaneClassWarps][kCtaAnchors];
    __shared__ unsigned s_flags[kPlaneClassWarps][kPlaneAnchorWarps * 32];  // bits 0..3: non-finite, 4..7: above `pre`
    const int logits = mode & 1;
    const bool agnostic = (mode & 2) != 0;
    const bool multi = (mode & 4) != 0;
    const int img = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int aw = warp % kPlaneAnchorWarps, cw = warp / kPlaneAnchorWarps;
    const float* __restrict__ hbase = head + (size_t)img * (size_t)(4 + C) * (size_t)A;
    const int col = aw * 32 + lane;  // this thread's group of VEC anchors inside the CTA
    const int a0 = blockIdx.x * kCtaAnchors + col * VEC;

    float best[VEC];
    int best_k[VEC];
    unsigned flags = 0u;
#pragma unroll
    for (int u = 0; u < VEC; ++u) { best[u] = -INFINITY; best_k[u] = 0x7fffffff; }
    if (a0 < A) {
        const float* __restrict__ cls0 = hbase + (size_t)4 * A + a0;
#pragma unroll kPlaneUnroll
        for (int k = cw; k < C; k += kPlaneClassWarps) {
            float v[VEC];
            if (VEC == 4) {
                const float4 q = __ldg(reinterpret_cast<const float4*>(cls0 + (size_t)k * A));
                v[0] = q.x; v[1 % VEC] = q.y; v[2 % VEC] = q.z; v[3 % VEC] = q.w;
            } else {
                v[0] = __ldg(cls0 + (size_t)k * A);
            }
#pragma unroll
            for (int u = 0; u < VEC; ++u) {
                if (!finite_f(v[u])) flags |= 1u << u;
                if (v[u] > best[u]) { best[u] = v[u]; best_k[u] = k; }
                if (multi && v[u] > pre) flags |= 16u << u;
            }
        }
    }
#pragma unroll
    for (int u = 0; u < VEC; ++u) {
        s_best[cw][col * VEC + u] = best[u];
        s_k[cw][col * VEC + u] = best_k[u];
    }
    s_flags[cw][col] = flags;
    __syncthreads();

    // one thread per anchor of the CTA
    for (int t = threadIdx.x; t < kCtaAnchors; t += kDecThreads) {
        const int u = t % VEC;
        const int anchor = blockIdx.x * kCtaAnchors + t;
        if (anchor >= A) break;
        float bv = -INFINITY;
        int bk = 0x7fffffff;
        unsigned fl = 0u;
#pragma unroll
        for (int w = 0; w < kPlaneClassWarps; ++w) {
            const float v = s_best[w][t];
            const int k = s_k[w][t];
            if (v > bv || (v == bv && k < bk)) { bv = v; bk = k; }  // first maximum over all classes
            fl |= s_flags[w][t / VEC];
        }
        const bool bad = (fl >> u) & 1u;
        if (bad) atomicOr(status, 0x1u);
        const float* __restrict__ bx = hbase + anchor;
        auto box_ok = [&]() {  // finite box with w, h > 0
            const float cx = __ldg(bx), cy = __ldg(bx + A), bw = __ldg(bx + 2 * (size_t)A),
                        bh = __ldg(bx + 3 * (size_t)A);
            if (!(finite_f(cx) && finite_f(cy) && finite_f(bw) && finite_f(bh))) {
                atomicOr(status, 0x1u);
                return false;
            }
            return bw > 0.0f && bh > 0.0f;
        };
        auto emit = [&](int cls, float score) {
            const int slot = atomicAdd(cand_count + img, 1);
            if (slot < key_stride) keys[(size_t)img * key_stride + slot] = make_key(cls, score, anchor);
            else atomicOr(status, 0x10u);
        };
        if (!multi) {
            if (bad || bk == 0x7fffffff) continue;
            const float score = logits ? sigmoid_fixed(bv) : bv;
            if (!(score > conf)) continue;
            if (!box_ok()) continue;
            emit(agnostic ? 0 : bk, score);
        } else {
            // rare: walk the anchor's classes again (the values are in L1 / L2 by now)
            if (bad || !((fl >> (4 + u)) & 1u)) continue;
            if (!box_ok()) continue;
            const float* __restrict__ cv = hbase + (size_t)4 * A + anchor;
            for (int k = 0; k < C; ++k) {
                const float v = __ldg(cv + (size_t)k * A);
                if (!(v > pre)) continue;
                const float score = logits ? sigmoid_fixed(v) : v;
                if (score > conf) emit(k, score);
            }
        }
    }
}

cudaError_t launch_decode(const DecodeArgs& a, cudaStream_t stream) {
    // d_cand_count is zero on entry: zeroed at stage creation and re-zeroed by the NMS kernel.
    const int mode = (a.logits ? 1 : 0) | (a.class_agnostic ? 2 : 0) | (a.multi_label ? 4 : 0);
    const int pdl = a.pdl ? 1 : 0;
    if (a.layout == OCTO_HEAD_PLANES) {
        // Multi-label prefilter in the head's own units: for probabilities the threshold itself;
        // for logits the threshold's logit lowered by a margin that dwarfs the few-ulp error of
        // the fixed logistic sequence (no prefilter where the logistic curve is too flat for that).
        float pre = a.conf;
        if (a.logits) {
            pre = -INFINITY;
            if (a.conf > 0.0f && a.conf <= 0.99f) {
                const double t = log((double)a.conf / (1.0 - (double)a.conf));
                pre = (float)(t - 1e-3 * (1.0 + fabs(t)));
            }
        }
        if ((a.A & 3) == 0 && (reinterpret_cast<uintptr_t>(a.d_head) & 15) == 0) {
            dim3 grid((a.A + 128 * kPlaneAnchorWarps - 1) / (128 * kPlaneAnchorWarps), a.n);
            return launch_kernel(decode_planes_kernel<4>, grid, dim3(kDecThreads), 0, stream, a.pdl, a.d_head, a.A, a.C,
                                 mode, a.conf, pre, a.key_stride, a.d_keys, a.d_cand_count, a.d_status, pdl);
        } else {
            dim3 grid((a.A + 32 * kPlaneAnchorWarps - 1) / (32 * kPlaneAnchorWarps), a.n);
            return launch_kernel(decode_planes_kernel<1>, grid, dim3(kDecThreads), 0, stream, a.pdl, a.d_head, a.A, a.C,
                                 mode, a.conf, pre, a.key_stride, a.d_keys, a.d_cand_count, a.d_status, pdl);
        }
    }
    const int per_cta4 = kDecThreads * 4;
    if ((long long)a.n * ((a.A + per_cta4 - 1) / per_cta4) >= 296) {
        dim3 grid((a.A + per_cta4 - 1) / per_cta4, a.n);
        return launch_kernel(decode_kernel<4>, grid, dim3(kDecThreads), 0, stream, a.pdl, a.d_head, a.A, a.C, mode,
                             a.conf, a.key_stride, a.d_keys, a.d_cand_count, a.d_status, pdl);
    }
    dim3 grid((a.A + kDecThreads - 1) / kDecThreads, a.n);
    return launch_kernel(decode_kernel<1>, grid, dim3(kDecThreads), 0, stream, a.pdl, a.d_head, a.A, a.C, mode, a.conf,
                         a.key_stride, a.d_keys, a.d_cand_count, a.d_status, pdl);
}

}  // namespace octo
