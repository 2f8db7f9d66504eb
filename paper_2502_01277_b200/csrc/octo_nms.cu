// Per-image ordering + class-aware greedy NMS + cap + scale-back (one CTA per image).
//
// Latency / shared-memory bound; bytes are negligible.  Classes are independent under
// class-aware NMS, so the image's candidate keys (class | inverted score bits | anchor) are
// first bucketed by class in shared memory (histogram, scan, scatter).  Each warp then owns
// whole classes: it sorts the class's keys with a warp-level bitonic network (score
// descending, ties by lower anchor), gathers the boxes from the head by anchor and runs the
// greedy scan: 32 candidates at a time are tested against the class's survivors so far
// (broadcast reads of shared memory), then resolved among themselves with ballots and
// register shuffles.  Survivors are compacted in place and re-keyed to (inverted score |
// anchor | class).  The global score order is a merge of the per-class survivor lists: the
// rank of a survivor is its index in its own list plus, for every other class, the number of
// that class's survivors that precede it (binary search).  The first max_det in that order
// are mapped back to frame pixels and written out, together with each downstream branch's
// class-filtered index list.
//
// Images with more candidates than fit in shared memory take the same code path with the
// arrays in a global-memory workspace; classes with more than kWarpSortMax candidates are
// sorted by the whole CTA.
//
// Few images with many candidates each (a crowded scene served at a small batch) leave most SMs
// idle with one CTA per image, so the kernel can be launched with a thread-block cluster per
// image: every CTA of the cluster buckets the image's keys for itself, the classes are handed out
// by one counter in the first CTA's shared memory to the warps of all CTAs, and every finished
// class is written into the first CTA's arrays through distributed shared memory.  The first CTA
// alone merges the classes and writes the image's results.
#include "octo_common.cuh"
#include <cmath>
#include <cooperative_groups.h>
#include <cstring>

#include "octo_kernels.h"

namespace octo {

namespace cg = cooperative_groups;

constexpr int kNmsThreadsFull = 1024;
constexpr int kNmsSmemCap = 8192;   // candidates handled on chip: 8 B key + 16 B box each
// Batches of more images than the GPU has SMs that have held only sparse images lately run two
// smaller CTAs per SM (half the threads, half the on-chip capacity), so that the launch is one
// wave of CTAs instead of two; an image that exceeds the smaller capacity takes the global-memory
// path, and the launches after it are full-sized again.
constexpr int kNmsThreadsHalf = 512;
constexpr int kNmsSmemCapHalf = 4096;
constexpr int kWarpSortMax = 2048;  // largest class segment a single warp sorts
constexpr int kRankSortMax = 512;   // up to here the warp sorts by counting instead of a network
constexpr int kSmallMax = 256;      // images with at most this many candidates take the short path
constexpr int kSmallWords = kSmallMax / 32;
constexpr long long kMergeBySortMin = 8192;  // survivors x live classes above which the merge is a sort
constexpr int kClusterMinCand = 1024;  // an image with more candidates than this makes clusters worth while

__device__ __forceinline__ void cmp_swap(unsigned long long* __restrict__ k, int i, int j) {
    const unsigned long long a = k[i], b = k[j];
    if (a > b) { k[i] = b; k[j] = a; }
}

// Ascending bitonic sort of k[0, m) for any m, by `nthreads` cooperating threads (a warp or
// the whole CTA).  Every comparator puts the smaller key at the lower index (the first stage
// of each merge pairs mirrored positions), so positions >= m can stand for +infinity and are
// simply skipped.
template <bool BLOCK>
__device__ __forceinline__ void bitonic_range(unsigned long long* __restrict__ k, int m, int tid, int nthreads) {
    int np2 = 2;
    while (np2 < m) np2 <<= 1;
    const int half = np2 >> 1;
    for (int size = 2; size <= np2; size <<= 1) {
        if (BLOCK) __syncthreads(); else __syncwarp();
        const int h = size >> 1;
        for (int t = tid; t < half; t += nthreads) {
            const int off = t & (h - 1);
            const int i = 2 * t - off;           // block start + off
            const int j = i + size - 1 - 2 * off;  // mirrored position in the block
            if (j < m) cmp_swap(k, i, j);
        }
        for (int stride = size >> 2; stride > 0; stride >>= 1) {
            if (BLOCK) __syncthreads(); else __syncwarp();
            for (int t = tid; t < half; t += nthreads) {
                const int i = 2 * t - (t & (stride - 1));
                const int j = i + stride;
                if (j < m) cmp_swap(k, i, j);
            }
        }
    }
    if (BLOCK) __syncthreads(); else __syncwarp();
}

// Box of one anchor; es = distance between consecutive values of an anchor (1 in the rows
// layout, A in the planes layout).
__device__ __forceinline__ float4 gather_box(const float* __restrict__ p, size_t es) {
    return box_corners(__ldg(p), __ldg(p + es), __ldg(p + 2 * es), __ldg(p + 3 * es));
}

template <int CAP, int kNmsThreads>
__global__ void __launch_bounds__(kNmsThreads, kNmsThreadsFull / kNmsThreads)
nms_kernel(const __grid_constant__ FrameTable<CAP> tab, const FrameDesc* __restrict__ gtab,
           const float* __restrict__ head, int A, int C, int layout,
           const IouTest iou_test, int max_det, int key_stride, unsigned long long* __restrict__ gkeys,
           float4* __restrict__ gboxes, int* __restrict__ cand_count, octo_det_rec* __restrict__ dets,
           int* __restrict__ counts, int num_branches, int class_agnostic,
           const __grid_constant__ BranchMasks masks,
           int* __restrict__ bcount, int* __restrict__ bidx, int max_batch, StageCounters* __restrict__ ctr,
           int* __restrict__ dense_seen, int launch_seq, int pdl) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    pdl_enter(pdl);
    __shared__ int seg_start[128], seg_cnt[128], cursor[128], nkept[128];
    __shared__ int live[128];  // classes with survivors
    __shared__ int s_total, s_live, s_big, s_nout, s_next;
    unsigned int* const status = &ctr->status;
    (void)status;  // referenced by the range checks of the checked build only

    cg::cluster_group cluster = cg::this_cluster();
    const unsigned csize = cluster.num_blocks();  // 1 unless the launch gave every image a cluster
    const unsigned crank = cluster.block_rank();
    const int img = (int)(blockIdx.x / csize);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // rows layout [A][5 + C] or planes layout [4 + C][A]
    const int nbox = layout == OCTO_HEAD_PLANES ? 4 : 5;
    const size_t es = layout == OCTO_HEAD_PLANES ? (size_t)A : 1;          // value to value
    const size_t as = layout == OCTO_HEAD_PLANES ? 1 : (size_t)(nbox + C);  // anchor to anchor
    const float* __restrict__ hbase = head + (size_t)img * (size_t)A * (size_t)(nbox + C);

    // The frame table comes by value (first-level stages) or from device memory (chained stages,
    // where an entry without a frame stands for an unused slot of the batch: no detections).
    const FrameDesc fd = gtab ? gtab[img] : tab.f[img];
    int cnt = cand_count[img];
    cnt = min(cnt, key_stride);
    if (gtab && fd.data == nullptr) cnt = 0;
    if (threadIdx.x < 128) { seg_cnt[threadIdx.x] = 0; nkept[threadIdx.x] = 0; }
    if (threadIdx.x == 0) {
        s_total = 0;
        s_live = 0;
        s_big = 0;
        s_next = 0;
    }
    // every CTA of the image has read the count, and the first CTA's counters are set, before the
    // count is cleared and before any CTA touches those counters
    if (csize > 1) cluster.sync(); else __syncthreads();
    if (threadIdx.x == 0 && crank == 0) {
        cand_count[img] = 0;  // ready for the next batch's decode
        atomicAdd(&ctr->candidates, (unsigned long long)cnt);
        atomicMax(&ctr->max_cand, cnt);
        // (only crowded images write: a store to host memory delays the end of the kernel by a PCIe
        // round trip, which a sparse launch of ten microseconds would feel)
        if (dense_seen && cnt > kClusterMinCand) *dense_seen = launch_seq;
    }

    unsigned long long* const gk = gkeys + (size_t)img * key_stride;
    // candidates the launch's shared memory holds
    constexpr int smem_cap = kNmsThreads == kNmsThreadsFull ? kNmsSmemCap : kNmsSmemCapHalf;
    const bool on_chip = cnt <= smem_cap;
    unsigned long long* keys;
    float4* boxes;
    if (on_chip) {
        boxes = reinterpret_cast<float4*>(smem_raw);
        keys = reinterpret_cast<unsigned long long*>(smem_raw + (size_t)smem_cap * sizeof(float4));
    } else {
        boxes = gboxes + (size_t)img * key_stride;
        keys = gk;
        if (threadIdx.x == 0 && crank == 0 && cnt > kNmsSmemCap) atomicOr(&ctr->status, 0x8u);
    }
    // the short path and the global-memory path are the first CTA's alone (same count, hence the
    // same decision, in every CTA of the cluster; no cluster barrier follows on those paths)
    if (crank != 0 && (cnt <= kSmallMax || !on_chip)) return;
    // where the other CTAs of the cluster put their finished classes: the first CTA's arrays
    unsigned long long* const keys0 = csize > 1 && on_chip ? cluster.map_shared_rank(keys, 0) : keys;
    int* const nkept0 = csize > 1 ? cluster.map_shared_rank(nkept, 0) : nkept;
    int* const live0 = csize > 1 ? cluster.map_shared_rank(live, 0) : live;
    int* const total0 = csize > 1 ? cluster.map_shared_rank(&s_total, 0) : &s_total;
    int* const nlive0 = csize > 1 ? cluster.map_shared_rank(&s_live, 0) : &s_live;
    int* const next0 = csize > 1 ? cluster.map_shared_rank(&s_next, 0) : &s_next;
    const bool shared_work = csize > 1 && on_chip && cnt > kSmallMax;

    // boxes are dead once NMS is done: their memory holds the ordered survivors (and the ranks)
    unsigned long long* const ordered = reinterpret_cast<unsigned long long*>(boxes);
    int nout;
    if (cnt <= kSmallMax) {
        // ---- short path for images with few candidates (the common case in serving): one
        // thread per candidate and short phases between barriers.  Candidates are bucketed by
        // class, ordered inside their class by counting, tested against the earlier candidates of
        // the class in parallel (one bit each, relative to the class's first position); one
        // thread per class then walks the class in order with the survivor set in a register (a
        // candidate survives iff none of its suppressors did), and the survivors find their place
        // in the global order (score, anchor, class) by counting among themselves. ----
        __shared__ int s_m;
        unsigned long long* const ukey = keys;                   // bucketed by class, unordered inside
        unsigned long long* const skey = keys + kSmallMax;       // ordered inside each class
        unsigned long long* const surv = keys + 2 * kSmallMax;   // global-order keys of the survivors
        float4* const ubox = reinterpret_cast<float4*>(keys + 3 * kSmallMax);
        float4* const sbox = ubox + kSmallMax;
        unsigned int* const sup = reinterpret_cast<unsigned int*>(sbox + kSmallMax);  // [kSmallMax][kSmallWords]
        unsigned char* const alive = reinterpret_cast<unsigned char*>(sup + kSmallMax * kSmallWords);
        const int t = threadIdx.x;
        // Only the first kSmallMax threads work here; they meet at a barrier of their own, so the
        // phases are not paced by the 24 warps that have nothing to do.
        auto bar_small = []() { asm volatile("bar.sync 1, %0;" ::"n"(kSmallMax) : "memory"); };
        if (t < kSmallMax) {
            unsigned long long k = kKeySentinel;
            float4 box = make_float4(0.f, 0.f, 0.f, 0.f);
            int cls = 0;
            if (t == 0) s_m = 0;
            if (t < cnt) {
                k = gk[t];
                cls = (int)(k >> 57);
                atomicAdd(&seg_cnt[cls], 1);
                box = gather_box(hbase + (size_t)(k & ((1ull << kKeyAnchorBits) - 1)) * as, es);
            }
            bar_small();
            if (warp == 0) {
                int run = 0;
    #pragma unroll
                for (int base = 0; base < 128; base += 32) {
                    const int v = seg_cnt[base + lane];
                    int inc = v;
    #pragma unroll
                    for (int off = 1; off < 32; off <<= 1) {
                        const int u = __shfl_up_sync(0xffffffffu, inc, off);
                        if (lane >= off) inc += u;
                    }
                    seg_start[base + lane] = run + inc - v;
                    cursor[base + lane] = run + inc - v;
                    run += __shfl_sync(0xffffffffu, inc, 31);
                }
            }
            bar_small();
            if (t < cnt) {
                const int pos = atomicAdd(&cursor[cls], 1);
                if (OCTO_IN_RANGE(pos >= 0 && pos < kSmallMax, status)) {
                    ukey[pos] = k;
                    ubox[pos] = box;
                }
            }
            bar_small();
            int start = 0;
            if (t < cnt) {  // from here on thread t owns bucket position t
                k = ukey[t];
                box = ubox[t];
                cls = (int)(k >> 57);
                start = seg_start[cls];
                const int m = seg_cnt[cls];
                int r = 0;
                for (int j = start; j < start + m; ++j) r += ukey[j] < k;
                if (OCTO_IN_RANGE(start + r >= 0 && start + r < kSmallMax, status)) {
                    skey[start + r] = k;
                    sbox[start + r] = box;
                }
            }
            bar_small();
            if (t < cnt) {  // ... and ordered position t (same class, hence the same start)
                const float4 bi = sbox[t];
                const int words = (t - start + 31) >> 5;  // words that hold predecessors
                for (int w = 0; w < words; ++w) {
                    unsigned bits = 0u;
                    const int j0 = start + (w << 5), j1 = min(j0 + 32, t);
                    for (int j = j0; j < j1; ++j)
                        if (iou_above(sbox[j], bi, iou_test)) bits |= 1u << (j - j0);
                    sup[t * kSmallWords + w] = bits;
                }
            }
            bar_small();
            if (t < cnt && t == start) {  // first position of a class: walk the class in order
                const int m = seg_cnt[cls];
                if (m <= 32) {
                    unsigned kept = 0u;
                    alive[t] = 1;
                    kept = 1u;
                    for (int i = 1; i < m; ++i) {
                        const bool ok = (sup[(t + i) * kSmallWords] & kept) == 0u;
                        alive[t + i] = ok ? 1 : 0;
                        if (ok) kept |= 1u << i;
                    }
                } else {
                    unsigned kept[kSmallWords];
    #pragma unroll
                    for (int w = 0; w < kSmallWords; ++w) kept[w] = 0u;
                    for (int i = 0; i < m; ++i) {
                        bool ok = true;
    #pragma unroll
                        for (int w = 0; w < kSmallWords; ++w)
                            if (w < ((i + 31) >> 5) && (sup[(t + i) * kSmallWords + w] & kept[w]) != 0u) ok = false;
                        alive[t + i] = ok ? 1 : 0;
    #pragma unroll
                        for (int w = 0; w < kSmallWords; ++w)
                            if (ok && w == (i >> 5)) kept[w] |= 1u << (i & 31);
                    }
                }
            }
            bar_small();
            unsigned long long g = kKeySentinel;
            const bool mine = t < cnt && alive[t] != 0;
            if (mine) {
                const unsigned long long ks = skey[t];
                g = ((ks & ((1ull << 57) - 1)) << 7) | (ks >> 57);  // inverted score | anchor | class
                const int q = atomicAdd(&s_m, 1);
                if (OCTO_IN_RANGE(q >= 0 && q < kSmallMax, status)) surv[q] = g;
            }
            bar_small();
            const int m_all = s_m;
            if (mine) {
                int r = 0;
                for (int j = 0; j < m_all; ++j) r += surv[j] < g;
                if (r < max_det && OCTO_IN_RANGE(r < kSmallMax, status)) ordered[r] = g;
            }
            if (t == 0) s_nout = min(m_all, max_det);
        }
        __syncthreads();
        nout = s_nout;
    } else {
        // ---- bucket the keys by class: histogram, scan, scatter ----
        for (int i = threadIdx.x; i < cnt; i += kNmsThreads) atomicAdd(&seg_cnt[(int)(gk[i] >> 57)], 1);
        __syncthreads();
        if (warp == 0) {
            int run = 0;
    #pragma unroll
            for (int base = 0; base < 128; base += 32) {
                const int v = seg_cnt[base + lane];
                int inc = v;
    #pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const int t = __shfl_up_sync(0xffffffffu, inc, off);
                    if (lane >= off) inc += t;
                }
                seg_start[base + lane] = run + inc - v;
                cursor[base + lane] = run + inc - v;
                run += __shfl_sync(0xffffffffu, inc, 31);
                if (__any_sync(0xffffffffu, v > kWarpSortMax) && lane == 0) s_big = 1;
            }
        }
        __syncthreads();
        {
            // off chip the scatter goes through the box workspace and back into the key array
            unsigned long long* const dst = on_chip ? keys : reinterpret_cast<unsigned long long*>(boxes);
            for (int i = threadIdx.x; i < cnt; i += kNmsThreads) {
                const unsigned long long k = gk[i];
                const int pos = atomicAdd(&cursor[(int)(k >> 57)], 1);
                if (OCTO_IN_RANGE(pos >= 0 && pos < cnt, status)) dst[pos] = k;
            }
            __syncthreads();
            if (!on_chip) {
                for (int i = threadIdx.x; i < cnt; i += kNmsThreads) keys[i] = dst[i];
                __syncthreads();
            }
        }

        // ---- very large classes are sorted by the whole CTA ----
        if (s_big) {
            for (int cls = 0; cls < 128; ++cls) {
                const int m = seg_cnt[cls];
                if (m > kWarpSortMax) bitonic_range<true>(keys + seg_start[cls], m, threadIdx.x, kNmsThreads);
            }
        }

        // The first CTA's bucketing and block-wide sorts are finished before another CTA of the
        // cluster writes a finished class into its arrays.
        if (shared_work) cluster.sync();

        // ---- one warp per class: sort, gather boxes, greedy NMS.  Classes are handed out by a
        // counter, so a warp that drew small classes takes more of them (with a fixed share, 80
        // classes on 32 warps leave half the warps with three classes and half with two). ----
        for (;;) {
            int cls = 0;
            if (lane == 0) cls = atomicAdd(next0, 1);
            cls = __shfl_sync(0xffffffffu, cls, 0);
            if (cls >= 128) break;
            const int m = seg_cnt[cls];
            if (m == 0) continue;
            const int s = seg_start[cls], e = s + m;
            if (m > 1 && m <= kRankSortMax) {
                // small class: every key counts the keys below it and moves to that position, staged
                // in the (not yet used) box slots of the segment
                unsigned long long* const tmp = reinterpret_cast<unsigned long long*>(boxes + s);
                for (int i0 = lane; i0 < m; i0 += 128) {
                    // up to four keys per lane share one pass over the segment
                    const unsigned long long k0 = keys[s + i0];
                    const unsigned long long k1 = i0 + 32 < m ? keys[s + i0 + 32] : kKeySentinel;
                    const unsigned long long k2 = i0 + 64 < m ? keys[s + i0 + 64] : kKeySentinel;
                    const unsigned long long k3 = i0 + 96 < m ? keys[s + i0 + 96] : kKeySentinel;
                    int r0 = 0, r1 = 0, r2 = 0, r3 = 0;
                    for (int j = 0; j < m; ++j) {
                        const unsigned long long kj = keys[s + j];
                        r0 += kj < k0; r1 += kj < k1; r2 += kj < k2; r3 += kj < k3;
                    }
                    tmp[r0] = k0;
                    if (i0 + 32 < m) tmp[r1] = k1;
                    if (i0 + 64 < m) tmp[r2] = k2;
                    if (i0 + 96 < m) tmp[r3] = k3;
                }
                __syncwarp();
                for (int p = lane; p < m; p += 32) keys[s + p] = tmp[p];
                __syncwarp();
            } else if (m > 1 && m <= kWarpSortMax) {
                bitonic_range<false>(keys + s, m, lane, 32);
            }
            // boxes of the class from the head, four per lane in flight (a lone warp pays the full
            // round trip for every load it waits on)
            for (int p0 = s + lane; p0 < e; p0 += 128) {
                float4 b4[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int p = p0 + 32 * u;
                    if (p < e) {
                        const int anchor = (int)(keys[p] & ((1ull << kKeyAnchorBits) - 1));
                        b4[u] = gather_box(hbase + (size_t)anchor * as, es);
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int p = p0 + 32 * u;
                    if (p < e) boxes[p] = b4[u];
                }
            }
            __syncwarp();
            int nk = 0;  // survivors of this class, compacted at [s, s + nk)
            for (int c0 = s; c0 < e && nk < max_det; c0 += 32) {
                const int p = c0 + lane;
                const bool valid = p < e;
                float4 b = make_float4(0.f, 0.f, 0.f, 0.f);
                unsigned long long k = kKeySentinel;
                if (valid) { b = boxes[p]; k = keys[p]; }
                bool alive = valid;
                // four survivors per round: the tests of a round are independent of one another, so
                // their latencies overlap (a lone warp is bound by the dependent chain, not by issue)
                for (int t = 0; t < nk; t += 4) {
                    if (!__any_sync(0xffffffffu, alive)) break;
                    const float4 k0 = boxes[s + t];
                    const float4 k1 = boxes[s + min(t + 1, nk - 1)];
                    const float4 k2 = boxes[s + min(t + 2, nk - 1)];
                    const float4 k3 = boxes[s + min(t + 3, nk - 1)];
                    const bool hit = iou_above(k0, b, iou_test) | iou_above(k1, b, iou_test) |
                                     iou_above(k2, b, iou_test) | iou_above(k3, b, iou_test);
                    if (hit) alive = false;
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
                    if (alive && lane > l && iou_above(lb, b, iou_test)) alive = false;
                    rem = __ballot_sync(0xffffffffu, alive) & ~((2u << l) - 1u);
                }
                __syncwarp();
                const int allowed = min(__popc(keptmask), max_det - nk);
                if ((keptmask >> lane) & 1u) {
                    const int r = __popc(keptmask & ((1u << lane) - 1u));
                    if (r < allowed && OCTO_IN_RANGE(s + nk + r < e, status)) {
                        boxes[s + nk + r] = b;
                        // re-key for the global order: inverted score | anchor | class
                        keys[s + nk + r] = ((k & ((1ull << 57) - 1)) << 7) | (k >> 57);
                    }
                }
                __syncwarp();
                nk += allowed;
            }
            for (int p = s + nk + lane; p < e; p += 32) keys[p] = kKeySentinel;
            if (crank != 0) {  // hand the finished class to the first CTA
                __syncwarp();
                for (int p = s + lane; p < e; p += 32) keys0[p] = keys[p];
            }
            if (lane == 0 && nk > 0) {
                nkept0[cls] = nk;
                atomicAdd(total0, nk);
                const int q = atomicAdd(nlive0, 1);
                if (OCTO_IN_RANGE(q >= 0 && q < 128, status)) live0[q] = cls;
            }
        }
        if (shared_work) {
            cluster.sync();  // every class has arrived in the first CTA's arrays
            if (crank != 0) return;
        } else {
            __syncthreads();
        }

        // ---- global score order: merge of the per-class survivor lists by rank ----
        const int nlive = s_live;
        if ((long long)s_total * nlive > kMergeBySortMin) {
            // Many survivors in many classes: the rank merge below costs survivors x classes binary
            // searches, a sort of the survivors by the whole CTA far less.  Every survivor carries
            // its global-order key (inverted score | anchor | class); the lists are packed into the
            // memory of the (dead) boxes and sorted there.
            if (warp == 0) {
                // exclusive scan of the survivor counts over the classes -> cursor[cls]
                int run = 0;
#pragma unroll
                for (int base = 0; base < 128; base += 32) {
                    const int v = nkept[base + lane];
                    int inc = v;
#pragma unroll
                    for (int off = 1; off < 32; off <<= 1) {
                        const int u = __shfl_up_sync(0xffffffffu, inc, off);
                        if (lane >= off) inc += u;
                    }
                    cursor[base + lane] = run + inc - v;
                    run += __shfl_sync(0xffffffffu, inc, 31);
                }
            }
            __syncthreads();
            const int total = s_total;
            for (int cls = warp; cls < 128; cls += kNmsThreads / 32) {
                const int m = nkept[cls], from = seg_start[cls], to = cursor[cls];
                for (int i = lane; i < m; i += 32)
                    if (OCTO_IN_RANGE(to + i >= 0 && to + i < total && total <= cnt, status)) ordered[to + i] = keys[from + i];
            }
            bitonic_range<true>(ordered, total, threadIdx.x, kNmsThreads);
        } else {
            if (warp == 0) {
                // exclusive scan of the survivor counts over the live classes -> cursor[q]
                int run = 0;
                for (int base = 0; base < nlive; base += 32) {
                    const int q = base + lane;
                    const int v = q < nlive ? nkept[live[q]] : 0;
                    int inc = v;
        #pragma unroll
                    for (int off = 1; off < 32; off <<= 1) {
                        const int t = __shfl_up_sync(0xffffffffu, inc, off);
                        if (lane >= off) inc += t;
                    }
                    if (q < nlive) cursor[q] = run + inc - v;
                    run += __shfl_sync(0xffffffffu, inc, 31);
                }
            }
            __syncthreads();
            // boxes are no longer needed: their memory holds the ordered survivors and the ranks
            int* const rank = reinterpret_cast<int*>(ordered + min(max_det, cnt));
            const int total = s_total;
            // survivor e (dense numbering over the live classes): rank starts as the index in its own list
            for (int e = threadIdx.x; e < total; e += kNmsThreads) {
                int lo = 0, hi = nlive;  // live class q with cursor[q] <= e < cursor[q + 1]
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (cursor[mid] <= e) lo = mid; else hi = mid;
                }
                rank[e] = e - cursor[lo];
            }
            __syncthreads();
            // every (survivor, other live class) pair adds the number of that class's survivors that
            // precede the survivor; pairs are independent, so the searches run in parallel
            // (neighbouring threads take neighbouring survivors against the same class, so the list reads
            // broadcast and the rank updates hit different addresses)
            for (int i = threadIdx.x; i < total * nlive; i += kNmsThreads) {
                const int q = i / total, e = i - q * total;
                int lo = 0, hi = nlive;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (cursor[mid] <= e) lo = mid; else hi = mid;
                }
                if (lo == q) continue;
                const unsigned long long g = keys[seg_start[live[lo]] + (e - cursor[lo])];
                const unsigned long long* const list = keys + seg_start[live[q]];
                int l2 = 0, h2 = nkept[live[q]];
                while (l2 < h2) {
                    const int mid = (l2 + h2) >> 1;
                    if (list[mid] < g) l2 = mid + 1; else h2 = mid;
                }
                if (l2 && OCTO_IN_RANGE(e >= 0 && e < total, status)) atomicAdd(&rank[e], l2);
            }
            __syncthreads();
            for (int e = threadIdx.x; e < total; e += kNmsThreads) {
                const int r = rank[e];
                if (r >= max_det) continue;
                int lo = 0, hi = nlive;
                while (hi - lo > 1) {
                    const int mid = (lo + hi) >> 1;
                    if (cursor[mid] <= e) lo = mid; else hi = mid;
                }
                if (OCTO_IN_RANGE(r >= 0 && r < min(max_det, cnt), status))
                    ordered[r] = keys[seg_start[live[lo]] + (e - cursor[lo])];
            }
            __syncthreads();
        }
        nout = min(s_total, max_det);
    }

    // region of the source frame shown by the detector input: x in [x_lo, x_hi], y likewise
    const float fpl = (float)fd.pad_l, fpt = (float)fd.pad_t;
    const float x_lo = (float)fd.ox, y_lo = (float)fd.oy;
    const float x_hi = (float)(fd.ox + fd.rw), y_hi = (float)(fd.oy + fd.rh);
    for (int r = threadIdx.x; r < nout; r += kNmsThreads) {
        const unsigned long long g = ordered[r];
        int cls = (int)(g & 127u);
        const int anchor = (int)((g >> 7) & ((1ull << kKeyAnchorBits) - 1));
        const float score = __uint_as_float(~(unsigned)(g >> 32));
        const float4 b = gather_box(hbase + (size_t)anchor * as, es);
        if (class_agnostic) {
            // NMS ran with every candidate in class 0: recover the real class (first maximum)
            const float* __restrict__ cv = hbase + (size_t)anchor * as + (size_t)nbox * es;
            float best = __ldg(cv);
            cls = 0;
            for (int k = 1; k < C; ++k) {
                const float v = __ldg(cv + (size_t)k * es);
                if (v > best) { best = v; cls = k; }
            }
        }
        octo_det_rec d;
        // X = fl(fl(fl(x - pad) * gain) + origin), clamped to the region
        d.x1 = fminf(fmaxf(__fadd_rn(__fmul_rn(__fsub_rn(b.x, fpl), fd.gx), x_lo), x_lo), x_hi);
        d.y1 = fminf(fmaxf(__fadd_rn(__fmul_rn(__fsub_rn(b.y, fpt), fd.gy), y_lo), y_lo), y_hi);
        d.x2 = fminf(fmaxf(__fadd_rn(__fmul_rn(__fsub_rn(b.z, fpl), fd.gx), x_lo), x_lo), x_hi);
        d.y2 = fminf(fmaxf(__fadd_rn(__fmul_rn(__fsub_rn(b.w, fpt), fd.gy), y_lo), y_lo), y_hi);
        d.score = score;
        d.cls = cls;
        d.anchor = anchor;
        d._pad = 0;
        dets[(size_t)img * max_det + r] = d;
        if (class_agnostic) ordered[r] = (g & ~127ull) | (unsigned long long)cls;  // for the branch lists
    }
    __syncthreads();
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
                const unsigned cls = (unsigned)(ordered[r] & 127u);
                take = (masks.m[warp][cls >> 5] >> (cls & 31u)) & 1u;
            }
            const unsigned bal = __ballot_sync(0xffffffffu, take);
            if (take && OCTO_IN_RANGE(m + __popc(bal & ((1u << lane) - 1u)) < max_det, status))
                list[m + __popc(bal & ((1u << lane) - 1u))] = r;
            m += __popc(bal);
        }
        if (lane == 0) bcount[warp * max_batch + img] = m;
    }
}

constexpr size_t kNmsSmemBytes = (size_t)kNmsSmemCap * (sizeof(float4) + sizeof(unsigned long long));
constexpr size_t kNmsSmemBytesHalf = (size_t)kNmsSmemCapHalf * (sizeof(float4) + sizeof(unsigned long long));

cudaError_t prepare_nms(int* max_cluster) {
    cudaError_t e;
    e = cudaFuncSetAttribute(nms_kernel<8, kNmsThreadsFull>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kNmsSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(nms_kernel<64, kNmsThreadsFull>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kNmsSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(nms_kernel<512, kNmsThreadsFull>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kNmsSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(nms_kernel<512, kNmsThreadsHalf>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kNmsSmemBytesHalf);
    if (e != cudaSuccess) return e;
    if (max_cluster) {
        // the largest cluster (one CTA per SM: the kernel takes nearly all shared memory of an SM)
        // of which the device can hold at least one
        *max_cluster = 1;
        for (int c = 8; c > 1; c >>= 1) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)c);
            cfg.blockDim = dim3(kNmsThreadsFull);
            cfg.dynamicSmemBytes = kNmsSmemBytes;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)c;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            int active = 0;
            if (cudaOccupancyMaxActiveClusters(&active, nms_kernel<8, kNmsThreadsFull>, &cfg) == cudaSuccess && active > 0) {
                *max_cluster = c;
                break;
            }
            (void)cudaGetLastError();
        }
    }
    return cudaSuccess;
}

template <int CAP>
static cudaError_t launch_cap(const NmsArgs& a, cudaStream_t stream) {
    FrameTable<CAP> tab;  // built per call (copied into kernel parameter space by the launch)
    if (!a.d_tab)
        for (int i = 0; i < a.n; ++i) tab.f[i] = a.frames[i];
    // rounding boundary of the IoU test (see iou_above)
    const float up = nextafterf(a.iou_thr, INFINITY);
    IouTest iou_test;
    iou_test.mid = 0.5 * ((double)a.iou_thr + (double)up);
    unsigned int up_bits;
    memcpy(&up_bits, &up, sizeof(up_bits));
    iou_test.tie_up = (up_bits & 1u) == 0u ? 1 : 0;
    const int cluster = a.cluster == 2 || a.cluster == 4 || a.cluster == 8 ? a.cluster : 1;
    // two half-sized CTAs per SM: only the largest table size has that form (more images than SMs)
    const bool half = CAP == 512 && a.half_ctas && cluster == 1;
    auto kernel = nms_kernel<CAP, kNmsThreadsFull>;
    if constexpr (CAP == 512) {
        if (half) kernel = nms_kernel<512, kNmsThreadsHalf>;
    }
    return launch_kernel_cluster(kernel, dim3((unsigned)(a.n * cluster)), dim3(half ? kNmsThreadsHalf : kNmsThreadsFull),
                                 half ? kNmsSmemBytesHalf : kNmsSmemBytes, stream, a.pdl,
                                 cluster, tab, a.d_tab, a.d_head, a.A, a.C, a.layout, iou_test, a.max_det, a.key_stride,
                                 a.d_keys, a.d_boxes, a.d_cand_count, reinterpret_cast<octo_det_rec*>(a.d_dets),
                                 a.d_counts, a.num_branches, a.class_agnostic, a.masks, a.d_bcount, a.d_bidx,
                                 a.max_batch, a.d_ctr, a.d_dense_seen, a.launch_seq, a.pdl ? 1 : 0);
}

cudaError_t launch_nms(const NmsArgs& a, cudaStream_t stream) {
    if (a.n <= 8) return launch_cap<8>(a, stream);
    if (a.n <= 64) return launch_cap<64>(a, stream);
    return launch_cap<512>(a, stream);
}

}  // namespace octo
