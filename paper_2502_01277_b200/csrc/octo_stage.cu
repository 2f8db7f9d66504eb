// Stage object and the extern "C" boundary (see include/octo.h for the contract).
#include <cstdio>
#include <cstdlib>
#include <cmath>
#include <cstring>
#include <new>

#include <nvtx3/nvToolsExt.h>

#include "octo.h"
#include "octo_kernels.h"
#include "octo_stage_internal.h"

using namespace octo;

static const char* const kKernelRangeNames[OCTO_K_COUNT] = {"octo::letterbox", "octo::decode", "octo::nms",
                                                            "octo::assemble", "octo::crop"};

// Brackets one kernel launch: an NVTX range on the host side (a few nanoseconds when no tool
// listens; profilers show it over the launch) and, while timing is enabled, a CUDA event pair.
struct ScopedKernelTimer {
    octo_stage* st;
    cudaStream_t stream;
    int slot;
    ScopedKernelTimer(octo_stage* s, int kernel, cudaStream_t str) : st(s), stream(str), slot(-1) {
        nvtxRangePushA(kKernelRangeNames[kernel]);
        if (!st->timing) return;
        if (st->ev_used >= kEventPairs) { st->ev_dropped += 1; return; }
        slot = st->ev_used++;
        st->ev_kernel[slot] = kernel;
        cudaEventRecord(st->ev[2 * slot], stream);
    }
    ~ScopedKernelTimer() {
        if (slot >= 0) cudaEventRecord(st->ev[2 * slot + 1], stream);
        nvtxRangePop();
    }
};

static thread_local char g_cuda_err[256] = "";

namespace octo {
// Records the text octo_last_cuda_error returns on this thread; always returns OCTO_E_CUDA.
int report_cuda_error(cudaError_t e, const char* what) {
    snprintf(g_cuda_err, sizeof(g_cuda_err), "%s: %s", what, cudaGetErrorString(e));
    return OCTO_E_CUDA;
}
}  // namespace octo
static int cuda_fail(cudaError_t e, const char* what) { return octo::report_cuda_error(e, what); }
#define OCTO_CUDA(call)                                     \
    do {                                                    \
        cudaError_t e__ = (call);                           \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call); \
    } while (0)

static int validate_config(const octo_stage_config_t* c) {
    if (!c) return OCTO_E_INVALID_ARG;
    if (c->device < 0) return OCTO_E_INVALID_ARG;
    if (c->net_size < 8 || c->net_size > 4096 || (c->net_size & 7)) return OCTO_E_INVALID_ARG;
    if (c->max_batch < 1 || c->max_batch > OCTO_MAX_BATCH) return OCTO_E_INVALID_ARG;
    if (c->num_anchors < 1 || c->num_anchors > (1 << 24)) return OCTO_E_INVALID_ARG;
    if (c->num_classes < 1 || c->num_classes > OCTO_MAX_CLASSES) return OCTO_E_INVALID_ARG;
    if (c->head_is_logits != 0 && c->head_is_logits != 1) return OCTO_E_INVALID_ARG;
    if (!(c->conf_thresh >= 0.0f) || !(c->conf_thresh <= 1.0f)) return OCTO_E_INVALID_ARG;
    if (!(c->iou_thresh >= 0.0f) || !(c->iou_thresh <= 1.0f)) return OCTO_E_INVALID_ARG;
    if (c->max_det < 1 || c->max_det > 65536) return OCTO_E_INVALID_ARG;
    if (c->pad_value < 0 || c->pad_value > 255) return OCTO_E_INVALID_ARG;
    if (c->swap_rb != 0 && c->swap_rb != 1) return OCTO_E_INVALID_ARG;
    if (c->num_branches < 1 || c->num_branches > OCTO_MAX_BRANCHES) return OCTO_E_INVALID_ARG;
    if (c->class_agnostic != 0 && c->class_agnostic != 1) return OCTO_E_INVALID_ARG;
    if (c->head_layout != OCTO_HEAD_ROWS && c->head_layout != OCTO_HEAD_PLANES) return OCTO_E_INVALID_ARG;
    if (c->multi_label != 0 && c->multi_label != 1) return OCTO_E_INVALID_ARG;
    if (c->multi_label && c->class_agnostic) return OCTO_E_INVALID_ARG;
    for (int b = 0; b < c->num_branches; ++b) {
        const octo_branch_cfg_t& br = c->branch[b];
        if (br.out_w < 8 || br.out_w > 2048 || (br.out_w & 7)) return OCTO_E_INVALID_ARG;
        if (br.out_h < 1 || br.out_h > 2048) return OCTO_E_INVALID_ARG;
        if (octo::validate_branch_options(br) != OCTO_OK) return OCTO_E_INVALID_ARG;
    }
    return OCTO_OK;
}

namespace octo {
// branch options, expressed per input channel c (it lands in output plane swap ? 2 - c : c)
void fill_crop_opts(const octo_branch_cfg_t& br, int swap_rb, int pad_value, CropOpts* out) {
    out->keep_aspect = br.keep_aspect;
    for (int ch = 0; ch < 3; ++ch) {
        const int p = swap_rb ? 2 - ch : ch;
        const double m = br.normalize ? (double)br.mean[p] : 0.0, sd = br.normalize ? (double)br.std[p] : 1.0;
        out->sc[ch] = (float)(1.0 / sd);
        out->of[ch] = (float)(-m / sd);
        out->fill[ch] = (float)(((double)pad_value / 255.0 - m) / sd);
    }
}

// shared by octo_stage_create and octo_queue_set_options
int validate_branch_options(const octo_branch_cfg_t& br) {
    if (br.keep_aspect != 0 && br.keep_aspect != 1) return OCTO_E_INVALID_ARG;
    if (br.normalize != 0 && br.normalize != 1) return OCTO_E_INVALID_ARG;
    if (br.normalize) {
        for (int k = 0; k < 3; ++k) {
            if (!(fabsf(br.mean[k]) <= 1e6f)) return OCTO_E_INVALID_ARG;          // finite, sane
            if (!(br.std[k] >= 1e-6f) || !(br.std[k] <= 1e6f)) return OCTO_E_INVALID_ARG;
        }
    }
    return OCTO_OK;
}
}  // namespace octo

template <typename T>
static cudaError_t dev_alloc(T** p, size_t count, int64_t* total) {
    const size_t bytes = sizeof(T) * (count ? count : 1);
    cudaError_t e = cudaMalloc(reinterpret_cast<void**>(p), bytes);
    if (e == cudaSuccess) {
        *total += (int64_t)bytes;
        e = cudaMemset(*p, 0, bytes);
    }
    return e;
}

static void free_all(octo_stage* st) {
    cudaFree(st->d_keys);
    cudaFree(st->d_boxes);
    cudaFree(st->d_cand_count);
    cudaFree(st->d_bcount);
    cudaFree(st->d_bidx);
    for (int b = 0; b < OCTO_MAX_BRANCHES; ++b) cudaFree(st->d_items[b]);
    cudaFree(st->d_ctr);
    cudaFree(st->d_tab);
    if (st->h_dense_seen) cudaFreeHost(st->h_dense_seen);
    for (int i = 0; i < 2 * kEventPairs; ++i)
        if (st->ev[i]) cudaEventDestroy(st->ev[i]);
}

extern "C" int octo_stage_create(const octo_stage_config_t* cfg, octo_stage_t** out) {
    if (!out) return OCTO_E_INVALID_ARG;
    *out = nullptr;
    int rc = validate_config(cfg);
    if (rc != OCTO_OK) return rc;

    int ndev = 0;
    OCTO_CUDA(cudaGetDeviceCount(&ndev));
    if (cfg->device >= ndev) return OCTO_E_INVALID_ARG;
    OCTO_CUDA(cudaSetDevice(cfg->device));

    octo_stage* st = new (std::nothrow) octo_stage();
    if (!st) return OCTO_E_NO_MEMORY;
    memset(st, 0, sizeof(*st));
    st->cfg = *cfg;
    cudaError_t e = cudaDeviceGetAttribute(&st->sm_count, cudaDevAttrMultiProcessorCount, cfg->device);
    if (e != cudaSuccess) {
        delete st;
        return cuda_fail(e, "cudaDeviceGetAttribute");
    }
    int ks = 2;
    while (ks < cfg->num_anchors) ks <<= 1;
    if (cfg->multi_label) ks <<= 1;  // an anchor can yield several candidates
    st->key_stride = ks;

    const size_t mb = (size_t)cfg->max_batch;
    if (e == cudaSuccess) e = dev_alloc(&st->d_keys, mb * ks, &st->workspace_bytes);
    if (e == cudaSuccess) e = dev_alloc(&st->d_boxes, mb * ks, &st->workspace_bytes);
    if (e == cudaSuccess) e = dev_alloc(&st->d_cand_count, mb, &st->workspace_bytes);
    if (e == cudaSuccess) e = dev_alloc(&st->d_bcount, (size_t)OCTO_MAX_BRANCHES * mb, &st->workspace_bytes);
    if (e == cudaSuccess)
        e = dev_alloc(&st->d_bidx, (size_t)OCTO_MAX_BRANCHES * mb * cfg->max_det, &st->workspace_bytes);
    for (int b = 0; b < cfg->num_branches && e == cudaSuccess; ++b)
        e = dev_alloc(&st->d_items[b], mb * cfg->max_det, &st->workspace_bytes);
    if (e == cudaSuccess) e = dev_alloc(&st->d_ctr, 1, &st->workspace_bytes);
    if (e == cudaSuccess) e = dev_alloc(&st->d_tab, mb, &st->workspace_bytes);
    if (e == cudaSuccess) e = prepare_letterbox();
    if (e == cudaSuccess) e = prepare_nms(&st->nms_max_cluster);
    if (e == cudaSuccess) {
        // an integer the NMS kernel writes and the host reads without a copy
        e = cudaHostAlloc(reinterpret_cast<void**>(&st->h_dense_seen), sizeof(int), cudaHostAllocMapped);
        if (e == cudaSuccess) {
            st->h_dense_seen[0] = -(1 << 30);  // no image with many candidates seen yet
            e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&st->d_dense_seen), st->h_dense_seen, 0);
        }
    }
    if (e == cudaSuccess) e = prepare_crop();
    if (e != cudaSuccess) {
        free_all(st);
        delete st;
        cuda_fail(e, "octo_stage_create");
        (void)cudaGetLastError();  // the failure is reported here, not by a later call
        return e == cudaErrorMemoryAllocation ? OCTO_E_NO_MEMORY : OCTO_E_CUDA;
    }
    *out = st;
    return OCTO_OK;
}

extern "C" int octo_stage_destroy(octo_stage_t* st) {
    if (!st) return OCTO_E_INVALID_ARG;
    cudaSetDevice(st->cfg.device);
    free_all(st);
    delete st;
    return OCTO_OK;
}

// Letterbox geometry in exact integer arithmetic: the longer side maps to S, the other to
// round-half-up(short * S / long), at least 1; centred, odd remainder right/bottom.
static void letterbox_geometry(int w, int h, int S, FrameDesc* fd) {
    long long nw, nh;
    if (w >= h) {
        nw = S;
        nh = (2LL * h * S + w) / (2LL * w);
        if (nh < 1) nh = 1;
    } else {
        nh = S;
        nw = (2LL * w * S + h) / (2LL * h);
        if (nw < 1) nw = 1;
    }
    fd->nw = (int)nw;
    fd->nh = (int)nh;
    fd->pad_l = (int)((S - nw) / 2);
    fd->pad_t = (int)((S - nh) / 2);
    fd->gx = (float)w / (float)fd->nw;
    fd->gy = (float)h / (float)fd->nh;
    fd->ox = 0;
    fd->oy = 0;
    fd->rw = (uint16_t)w;
    fd->rh = (uint16_t)h;
}

extern "C" int octo_preprocess_batch(octo_stage_t* st, const octo_frame_t* frames, int32_t n,
                                     void* d_out_f16_nchw, void* cuda_stream) {
    if (!st || !frames || !d_out_f16_nchw || n < 1) return OCTO_E_INVALID_ARG;
    if (n > st->cfg.max_batch) return OCTO_E_CAPACITY;
    if (reinterpret_cast<uintptr_t>(d_out_f16_nchw) & 15) return OCTO_E_ALIGNMENT;
    int max_w = 0;
    for (int i = 0; i < n; ++i) {
        const octo_frame_t& f = frames[i];
        if (!f.d_data || f.width < 1 || f.height < 1) return OCTO_E_INVALID_ARG;
        if (f.width > 16384 || f.height > 16384) return OCTO_E_CAPACITY;
        if (f.width > kLetterboxMaxWidth) return OCTO_E_CAPACITY;
        if ((long long)f.pitch_bytes < 3LL * f.width) return OCTO_E_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(f.d_data) & 15) || (f.pitch_bytes & 15)) return OCTO_E_ALIGNMENT;
        if (f.width > max_w) max_w = f.width;
    }
    st->n_frames = 0;
    st->have_dets = false;
    st->tab_on_device = false;
    for (int i = 0; i < n; ++i) {
        FrameDesc& fd = st->frames[i];
        fd.data = frames[i].d_data;
        fd.w = frames[i].width;
        fd.h = frames[i].height;
        fd.pitch = frames[i].pitch_bytes;
        letterbox_geometry(fd.w, fd.h, st->cfg.net_size, &fd);
    }
    st->max_w = max_w;
    OCTO_CUDA(cudaSetDevice(st->cfg.device));
    {
        ScopedKernelTimer t(st, OCTO_K_LETTERBOX, static_cast<cudaStream_t>(cuda_stream));
        OCTO_CUDA(launch_letterbox(st->frames, n, d_out_f16_nchw, st->cfg.net_size, max_w, st->cfg.pad_value,
                                   st->cfg.swap_rb, &st->d_ctr->status, n <= kPdlMaxBatch,
                                   static_cast<cudaStream_t>(cuda_stream)));
    }
    st->launches += 1;
    st->n_frames = n;
    return OCTO_OK;
}

extern "C" int octo_adopt_regions(octo_stage_t* st, const octo_region_t* regions, int32_t n, void* cuda_stream) {
    (void)cuda_stream;  // nothing is enqueued: the table travels with the next kernel launches
    if (!st || !regions || n < 1) return OCTO_E_INVALID_ARG;
    if (n > st->cfg.max_batch) return OCTO_E_CAPACITY;
    const int S = st->cfg.net_size;
    for (int i = 0; i < n; ++i) {
        const octo_region_t& r = regions[i];
        if (!r.d_data || r.width < 1 || r.height < 1) return OCTO_E_INVALID_ARG;
        if (r.width > 16384 || r.height > 16384) return OCTO_E_CAPACITY;
        if ((long long)r.pitch_bytes < 3LL * r.width) return OCTO_E_INVALID_ARG;
        if ((reinterpret_cast<uintptr_t>(r.d_data) & 15) || (r.pitch_bytes & 15)) return OCTO_E_ALIGNMENT;
        if (r.rx0 < 0 || r.ry0 < 0 || r.rx1 <= r.rx0 || r.ry1 <= r.ry0 || r.rx1 > r.width || r.ry1 > r.height)
            return OCTO_E_INVALID_ARG;
    }
    st->n_frames = 0;
    st->have_dets = false;
    st->tab_on_device = false;
    for (int i = 0; i < n; ++i) {
        const octo_region_t& r = regions[i];
        FrameDesc& fd = st->frames[i];
        fd.data = r.d_data;
        fd.w = r.width;
        fd.h = r.height;
        fd.pitch = r.pitch_bytes;
        fd.nw = S;  // the upstream crop is a plain stretch to S x S: no padding
        fd.nh = S;
        fd.pad_l = 0;
        fd.pad_t = 0;
        fd.ox = (uint16_t)r.rx0;
        fd.oy = (uint16_t)r.ry0;
        fd.rw = (uint16_t)(r.rx1 - r.rx0);
        fd.rh = (uint16_t)(r.ry1 - r.ry0);
        fd.gx = (float)(r.rx1 - r.rx0) / (float)S;
        fd.gy = (float)(r.ry1 - r.ry0) / (float)S;
    }
    st->max_w = 0;
    st->n_frames = n;
    return OCTO_OK;
}

// ---- device-side hand-off between cascade levels ---------------------------------------------
// One thread per entry of the chained stage's batch: entry i becomes item first + i of the
// upstream branch (original frame + rectangle, stretched to S x S, no padding), or an empty
// entry (no frame: the NMS kernel reports no detections for it) when the upstream branch packed
// fewer items.  The arithmetic is the host's (octo_adopt_regions): gains by IEEE division.
namespace octo {
template <int CAP>
__global__ void __launch_bounds__(256)
adopt_items_kernel(const __grid_constant__ FrameTable<CAP> up_tab, const FrameDesc* __restrict__ up_gtab,
                   const octo_item_t* __restrict__ items, const int* __restrict__ up_n_items, int first, int n, int S,
                   FrameDesc* __restrict__ out) {
    pdl_enter(0);
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    FrameDesc fd;
    memset(&fd, 0, sizeof(fd));
    const int slot = first + i;
    if (slot < up_n_items[0]) {
        const octo_item_t it = items[slot];
        const FrameDesc src = up_gtab ? up_gtab[it.frame] : up_tab.f[it.frame];
        fd.data = src.data;
        fd.w = src.w; fd.h = src.h; fd.pitch = src.pitch;
        fd.nw = S; fd.nh = S;
        fd.ox = (uint16_t)it.rx0; fd.oy = (uint16_t)it.ry0;
        fd.rw = (uint16_t)(it.rx1 - it.rx0); fd.rh = (uint16_t)(it.ry1 - it.ry0);
        fd.gx = __fdiv_rn(__int2float_rn(it.rx1 - it.rx0), __int2float_rn(S));
        fd.gy = __fdiv_rn(__int2float_rn(it.ry1 - it.ry0), __int2float_rn(S));
    }
    out[i] = fd;
}

template <int CAP>
static cudaError_t launch_adopt(const octo_stage* up, const octo_item_t* d_items, const int* d_n_items, int first,
                                int n, int S, FrameDesc* d_out, cudaStream_t stream) {
    FrameTable<CAP> tab;
    if (!up->tab_on_device)
        for (int i = 0; i < up->n_frames; ++i) tab.f[i] = up->frames[i];
    return launch_kernel(adopt_items_kernel<CAP>, dim3((n + 255) / 256), dim3(256), 0, stream, false, tab,
                         up->tab_on_device ? up->d_tab : (const FrameDesc*)nullptr, d_items, d_n_items, first, n, S,
                         d_out);
}

// Test support: a wait that nothing ends.  One thread arms an mbarrier for `bytes` bytes that no
// copy will ever deliver, polls it `polls` times, reports the timeout in the status word and
// returns.  No copy is in flight at any point and the shared memory dies with the CTA.
__global__ void wait_selftest_kernel(unsigned int* __restrict__ status, int polls) {
    __shared__ __align__(8) uint64_t bar;
    pdl_enter(0);
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        mbar_fence_init();
        mbar_expect_tx(&bar, 64u);
        if (!mbar_wait_bounded(&bar, 0, polls)) atomicOr(status, 0x4u);
    }
}
}  // namespace octo

extern "C" int octo_adopt_items_device(octo_stage_t* st, const octo_stage_t* upstream, int32_t branch, int32_t first,
                                       int32_t n, void* cuda_stream) {
    if (!st || !upstream || st == upstream || n < 1 || first < 0) return OCTO_E_INVALID_ARG;
    if (branch < 0 || branch >= upstream->cfg.num_branches) return OCTO_E_INVALID_ARG;
    if (upstream->cfg.device != st->cfg.device) return OCTO_E_INVALID_ARG;
    if (n > st->cfg.max_batch) return OCTO_E_CAPACITY;
    if ((long long)first + n > (long long)upstream->cfg.max_batch * upstream->cfg.max_det) return OCTO_E_CAPACITY;
    if (upstream->n_frames < 1) return OCTO_E_NO_PREPROCESS;
    if (!upstream->d_last_n_items[branch]) return OCTO_E_NO_POSTPROCESS;  // the branch was never cropped
    // the upstream crop (a plain stretch of the rectangle to S x S) is this stage's detector input
    if (upstream->cfg.branch[branch].out_w != st->cfg.net_size || upstream->cfg.branch[branch].out_h != st->cfg.net_size)
        return OCTO_E_INVALID_ARG;
    OCTO_CUDA(cudaSetDevice(st->cfg.device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st->n_frames = 0;
    st->have_dets = false;
    cudaError_t e;
    const int un = upstream->tab_on_device ? 1 : upstream->n_frames;
    if (un <= 8) e = launch_adopt<8>(upstream, upstream->d_items[branch], upstream->d_last_n_items[branch], first, n, st->cfg.net_size, st->d_tab, stream);
    else if (un <= 64) e = launch_adopt<64>(upstream, upstream->d_items[branch], upstream->d_last_n_items[branch], first, n, st->cfg.net_size, st->d_tab, stream);
    else e = launch_adopt<512>(upstream, upstream->d_items[branch], upstream->d_last_n_items[branch], first, n, st->cfg.net_size, st->d_tab, stream);
    if (e != cudaSuccess) return cuda_fail(e, "adopt_items_kernel");
    st->launches += 1;
    st->tab_on_device = true;
    st->max_w = 0;
    st->n_frames = n;
    return OCTO_OK;
}

extern "C" int octo_stage_selftest_wait(octo_stage_t* st, int32_t polls, void* cuda_stream) {
    if (!st || polls < 1 || polls > (1 << 20)) return OCTO_E_INVALID_ARG;
    OCTO_CUDA(cudaSetDevice(st->cfg.device));
    OCTO_CUDA(launch_kernel(wait_selftest_kernel, dim3(1), dim3(32), 0, static_cast<cudaStream_t>(cuda_stream), false,
                            &st->d_ctr->status, (int)polls));
    st->launches += 1;
    return OCTO_OK;
}

extern "C" int octo_postprocess_batch(octo_stage_t* st, const float* d_head, int32_t n, octo_det_t* d_dets,
                                      int32_t* d_counts, void* cuda_stream) {
    if (!st || !d_head || !d_dets || !d_counts) return OCTO_E_INVALID_ARG;
    if (st->n_frames < 1) return OCTO_E_NO_PREPROCESS;
    if (n != st->n_frames) return OCTO_E_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(d_head) & 3) || (reinterpret_cast<uintptr_t>(d_dets) & 3) ||
        (reinterpret_cast<uintptr_t>(d_counts) & 3))
        return OCTO_E_ALIGNMENT;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const octo_stage_config_t& c = st->cfg;
    st->have_dets = false;
    OCTO_CUDA(cudaSetDevice(c.device));
    {
        ScopedKernelTimer t(st, OCTO_K_DECODE, stream);
        DecodeArgs da;
        da.d_head = d_head;
        da.n = n; da.A = c.num_anchors; da.C = c.num_classes;
        da.layout = c.head_layout;
        da.logits = c.head_is_logits; da.class_agnostic = c.class_agnostic; da.multi_label = c.multi_label;
        da.conf = c.conf_thresh;
        da.key_stride = st->key_stride;
        da.d_keys = st->d_keys; da.d_cand_count = st->d_cand_count; da.d_status = &st->d_ctr->status;
        da.pdl = n <= kPdlMaxBatch;
        OCTO_CUDA(launch_decode(da, stream));
    }
    st->launches += 1;
    NmsArgs a;
    a.frames = st->frames;
    a.d_tab = st->tab_on_device ? st->d_tab : nullptr;
    a.pdl = n <= kPdlMaxBatch;
    a.n = n;
    a.d_head = d_head;
    a.A = c.num_anchors;
    a.C = c.num_classes;
    a.layout = c.head_layout;
    a.iou_thr = c.iou_thresh;
    a.max_det = c.max_det;
    a.key_stride = st->key_stride;
    a.d_keys = st->d_keys;
    a.d_boxes = st->d_boxes;
    a.d_cand_count = st->d_cand_count;
    a.d_dets = d_dets;
    a.d_counts = d_counts;
    a.num_branches = c.num_branches;
    a.class_agnostic = c.class_agnostic;
    memset(&a.masks, 0, sizeof(a.masks));
    for (int b = 0; b < c.num_branches; ++b) memcpy(a.masks.m[b], c.branch[b].class_mask, sizeof(uint32_t) * 4);
    a.d_bcount = st->d_bcount;
    a.d_bidx = st->d_bidx;
    a.max_batch = c.max_batch;
    a.d_ctr = st->d_ctr;
    // A cluster of CTAs per image while images with many candidates were seen in the kernel's latest
    // launches and the batch is too small to fill the GPU with one CTA per image.
    st->nms_seq += 1;
    a.cluster = 1;
    a.d_dense_seen = st->d_dense_seen;
    a.launch_seq = st->nms_seq;
    if (st->nms_cluster_mode > 0) {
        a.cluster = st->nms_cluster_mode < st->nms_max_cluster ? st->nms_cluster_mode : st->nms_max_cluster;
    } else if (st->h_dense_seen) {
        const int last_dense = *static_cast<const volatile int*>(st->h_dense_seen);
        if (st->nms_seq - last_dense <= kNmsClusterWindow) {
            const int want = n * 8 <= st->sm_count ? 8 : n * 4 <= st->sm_count ? 4 : n * 2 <= st->sm_count ? 2 : 1;
            a.cluster = want < st->nms_max_cluster ? want : st->nms_max_cluster;
        }
    }
    st->nms_cluster_last = a.cluster;
    // More images than SMs and no crowded image lately: two half-sized CTAs per SM, one wave.
    // (the half-sized kernel exists for the largest frame-table size only, i.e. for more than 64 images)
    a.half_ctas = a.cluster == 1 && n > st->sm_count && n > 64 && st->nms_cluster_mode == 0 && st->h_dense_seen &&
                  st->nms_seq - *static_cast<const volatile int*>(st->h_dense_seen) > kNmsClusterWindow;
    st->nms_half_last = a.half_ctas;
    cudaError_t e;
    {
        ScopedKernelTimer t(st, OCTO_K_NMS, stream);
        e = launch_nms(a, stream);
    }
    if (e != cudaSuccess) {
        // keep the "candidate counters are zero on entry" invariant after a failed launch
        cudaMemsetAsync(st->d_cand_count, 0, sizeof(int) * (size_t)c.max_batch, stream);
        return cuda_fail(e, "launch_nms");
    }
    st->launches += 1;
    st->have_dets = true;
    st->d_dets = d_dets;
    return OCTO_OK;
}

extern "C" int octo_crop_batch(octo_stage_t* st, int32_t branch, int32_t first_item, int32_t max_items,
                               void* d_out_f16, int32_t* d_offsets, int32_t* d_n_items, void* cuda_stream) {
    if (!st || !d_offsets || !d_n_items) return OCTO_E_INVALID_ARG;
    if (branch < 0 || branch >= st->cfg.num_branches) return OCTO_E_INVALID_ARG;
    if (first_item < 0 || max_items < 0) return OCTO_E_INVALID_ARG;
    if (max_items > 0 && !d_out_f16) return OCTO_E_INVALID_ARG;
    if (st->n_frames < 1) return OCTO_E_NO_PREPROCESS;
    if (!st->have_dets) return OCTO_E_NO_POSTPROCESS;
    if ((reinterpret_cast<uintptr_t>(d_out_f16) & 15) || (reinterpret_cast<uintptr_t>(d_offsets) & 3) ||
        (reinterpret_cast<uintptr_t>(d_n_items) & 3))
        return OCTO_E_ALIGNMENT;
    const octo_stage_config_t& c = st->cfg;
    const long long cap = (long long)c.max_batch * c.max_det;
    if (max_items > cap) max_items = (int32_t)cap;  // a branch can never hold more items
    CropArgs a;
    a.frames = st->frames;
    a.d_tab = st->tab_on_device ? st->d_tab : nullptr;
    a.pdl = st->n_frames <= kPdlMaxBatch;
    a.n = st->n_frames;
    a.max_det = c.max_det;
    a.first_item = first_item;
    a.max_items = max_items;
    a.d_bcount = st->d_bcount + (size_t)branch * c.max_batch;
    a.d_bidx = st->d_bidx + (size_t)branch * c.max_batch * c.max_det;
    a.d_dets = st->d_dets;
    a.d_offsets = d_offsets;
    a.d_n_items = d_n_items;
    a.d_items = st->d_items[branch];
    a.d_out = d_out_f16;
    a.out_w = c.branch[branch].out_w;
    a.out_h = c.branch[branch].out_h;
    a.swap_rb = c.swap_rb;
    a.sm_count = st->sm_count;
    a.d_ctr = st->d_ctr;
    a.general = c.branch[branch].keep_aspect != 0 || c.branch[branch].normalize != 0;
    fill_crop_opts(c.branch[branch], c.swap_rb, c.pad_value, &a.opts);
    OCTO_CUDA(cudaSetDevice(c.device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    {
        ScopedKernelTimer t(st, OCTO_K_CROP, stream);
        OCTO_CUDA(launch_crop(a, stream));
    }
    st->launches += 1;
    st->d_last_n_items[branch] = d_n_items;
    return OCTO_OK;
}

extern "C" int octo_stage_status(octo_stage_t* st, uint32_t* status_word, void* cuda_stream) {
    if (!st || !status_word) return OCTO_E_INVALID_ARG;
    OCTO_CUDA(cudaSetDevice(st->cfg.device));
    OCTO_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
    unsigned int w = 0;
    OCTO_CUDA(cudaMemcpy(&w, &st->d_ctr->status, sizeof(w), cudaMemcpyDeviceToHost));
    *status_word = w;
    return (w & OCTO_STATUS_COPY_TIMEOUT) ? OCTO_E_DEVICE_TIMEOUT : OCTO_OK;
}

extern "C" int octo_stage_clear_status(octo_stage_t* st, void* cuda_stream) {
    if (!st) return OCTO_E_INVALID_ARG;
    OCTO_CUDA(cudaSetDevice(st->cfg.device));
    OCTO_CUDA(cudaMemsetAsync(&st->d_ctr->status, 0, sizeof(unsigned int), static_cast<cudaStream_t>(cuda_stream)));
    return OCTO_OK;
}

extern "C" int octo_stage_get_stats(octo_stage_t* st, octo_stage_stats_t* stats, void* cuda_stream) {
    if (!st || !stats) return OCTO_E_INVALID_ARG;
    OCTO_CUDA(cudaSetDevice(st->cfg.device));
    OCTO_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
    StageCounters h;
    OCTO_CUDA(cudaMemcpy(&h, st->d_ctr, sizeof(h), cudaMemcpyDeviceToHost));
    stats->candidates = (int64_t)h.candidates;
    stats->kept = (int64_t)h.kept;
    stats->packed = h.packed;
    stats->total_items = h.total_items;
    stats->status_word = h.status;
    stats->max_candidates_per_image = h.max_cand;
    // candidates / kept accumulate over one postprocess call only: reset for the next one
    OCTO_CUDA(cudaMemset(st->d_ctr, 0, offsetof(StageCounters, status)));
    OCTO_CUDA(cudaMemset(&st->d_ctr->max_cand, 0, sizeof(int)));
    return OCTO_OK;
}

extern "C" int octo_stage_item_table(octo_stage_t* st, int32_t branch, const octo_item_t** d_items) {
    if (!st || !d_items || branch < 0 || branch >= st->cfg.num_branches) return OCTO_E_INVALID_ARG;
    *d_items = st->d_items[branch];
    return OCTO_OK;
}

extern "C" int octo_stage_copy_items(octo_stage_t* st, int32_t branch, octo_item_t* items_out, int32_t count,
                                     void* cuda_stream) {
    if (!st || branch < 0 || branch >= st->cfg.num_branches || count < 0) return OCTO_E_INVALID_ARG;
    if ((long long)count > (long long)st->cfg.max_batch * st->cfg.max_det) return OCTO_E_CAPACITY;
    if (count > 0 && !items_out) return OCTO_E_INVALID_ARG;
    OCTO_CUDA(cudaSetDevice(st->cfg.device));
    OCTO_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
    if (count > 0)
        OCTO_CUDA(cudaMemcpy(items_out, st->d_items[branch], sizeof(octo_item_t) * (size_t)count,
                             cudaMemcpyDeviceToHost));
    return OCTO_OK;
}

extern "C" int octo_stage_set_nms_cluster(octo_stage_t* st, int32_t cluster) {
    if (!st) return OCTO_E_INVALID_ARG;
    if (cluster != 0 && cluster != 1 && cluster != 2 && cluster != 4 && cluster != 8) return OCTO_E_INVALID_ARG;
    st->nms_cluster_mode = cluster;
    return OCTO_OK;
}

extern "C" int32_t octo_stage_last_nms_cluster(const octo_stage_t* st) { return st ? st->nms_cluster_last : 0; }
extern "C" int32_t octo_stage_last_nms_half_ctas(const octo_stage_t* st) { return st && st->nms_half_last ? 1 : 0; }

extern "C" int octo_stage_set_timing(octo_stage_t* st, int32_t enable) {
    if (!st) return OCTO_E_INVALID_ARG;
    OCTO_CUDA(cudaSetDevice(st->cfg.device));
    if (enable && !st->ev[0]) {
        for (int i = 0; i < 2 * kEventPairs; ++i) OCTO_CUDA(cudaEventCreate(&st->ev[i]));
    }
    st->timing = enable != 0;
    return OCTO_OK;
}

extern "C" int octo_stage_kernel_times(octo_stage_t* st, octo_kernel_times_t* times, void* cuda_stream) {
    if (!st || !times) return OCTO_E_INVALID_ARG;
    memset(times, 0, sizeof(*times));
    OCTO_CUDA(cudaSetDevice(st->cfg.device));
    OCTO_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
    for (int i = 0; i < st->ev_used; ++i) {
        float ms = 0.0f;
        OCTO_CUDA(cudaEventElapsedTime(&ms, st->ev[2 * i], st->ev[2 * i + 1]));
        times->ms[st->ev_kernel[i]] += (double)ms;
        times->launches[st->ev_kernel[i]] += 1;
    }
    times->dropped = st->ev_dropped;
    st->ev_used = 0;
    st->ev_dropped = 0;
    return OCTO_OK;
}

extern "C" int64_t octo_stage_workspace_bytes(const octo_stage_t* st) { return st ? st->workspace_bytes : 0; }
extern "C" int64_t octo_stage_launch_count(const octo_stage_t* st) { return st ? st->launches : 0; }

extern "C" const char* octo_strerror(int code) {
    switch (code) {
        case OCTO_OK: return "ok";
        case OCTO_E_INVALID_ARG: return "invalid argument";
        case OCTO_E_CAPACITY: return "capacity exceeded";
        case OCTO_E_ALIGNMENT: return "pointer or pitch not 16-byte aligned";
        case OCTO_E_NO_PREPROCESS: return "no batch has been preprocessed on this stage";
        case OCTO_E_CUDA: return "CUDA runtime error";
        case OCTO_E_DEVICE_TIMEOUT: return "a bounded device-side wait gave up";
        case OCTO_E_NO_POSTPROCESS: return "the current batch has not been postprocessed";
        case OCTO_E_NO_MEMORY: return "out of host or device memory";
        default: return "unknown status code";
    }
}

extern "C" const char* octo_last_cuda_error(void) { return g_cuda_err; }
extern "C" const char* octo_version(void) { return "0.1"; }
