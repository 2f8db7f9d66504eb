// Single-frame decode + NMS for callers that must not allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: a real-time inference loop
// whose memory was carved up at start-up and which may not touch the allocator again (an
// allocation can stall on other contexts and breaks latency guarantees), or a plug-in that
// lives inside another process's memory pool and was handed fixed buffers.  Creating a
// stage allocates its workspace, so such callers cannot use octo_postprocess_batch.  This
// file gives them one entry point that runs the same two kernels on a workspace that is
// part of the library image: a file-scope device array that every GPU loading the library
// holds from load to exit.
//
// Host code never passes the array's name to a kernel: on the host that name is only a
// stand-in.  The device address is looked up once per device with cudaGetSymbolAddress
// (with that device current) and kept.
#include <cstring>
#include <mutex>

#include "octo.h"
#include "octo_kernels.h"

using namespace octo;

namespace {

constexpr int kStaticMaxAnchors = OCTO_STATIC_MAX_ANCHORS;  // power of two: also the key stride
constexpr int kStaticMaxDet = OCTO_STATIC_MAX_DET;
constexpr int kMaxDevices = 64;

// Layout of the workspace (byte offsets, each a multiple of 256).
constexpr size_t kOffKeys = 0;                                                         // u64 [max anchors]
constexpr size_t kOffBoxes = kOffKeys + sizeof(unsigned long long) * kStaticMaxAnchors;  // float4 [max anchors]
constexpr size_t kOffBidx = kOffBoxes + sizeof(float4) * kStaticMaxAnchors;            // i32 [4][max_det]
constexpr size_t kOffBcount = kOffBidx + sizeof(int) * OCTO_MAX_BRANCHES * kStaticMaxDet;
constexpr size_t kOffCand = kOffBcount + 256;
constexpr size_t kOffCtr = kOffCand + 256;
constexpr size_t kScratchBytes = kOffCtr + 256;
static_assert(sizeof(StageCounters) <= 256, "counter block fits its slot");
static_assert((kStaticMaxAnchors & (kStaticMaxAnchors - 1)) == 0, "key stride must be a power of two");

// The workspace itself: about 0.8 MB of every GPU that loads this library, until exit.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

std::mutex g_mu;
unsigned char* g_dev_ptr[kMaxDevices];  // device address of g_static_scratch, per device
bool g_ready[kMaxDevices];

// First use on a device: resolve the device address of the array and opt the NMS kernel
// into its shared memory.  Neither call allocates.
cudaError_t setup_device(int device, unsigned char** out) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_ready[device]) {
        unsigned char* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch);
        if (e != cudaSuccess) return e;
        if (p == nullptr) return cudaErrorInvalidSymbol;
        e = prepare_nms(nullptr);
        if (e != cudaSuccess) return e;
        g_dev_ptr[device] = p;
        g_ready[device] = true;
    }
    *out = g_dev_ptr[device];
    return cudaSuccess;
}

// Same integer letterbox geometry as a stage computes for a frame (long side -> S, short
// side round-half-up, centred, odd remainder right/bottom); kept local so that the stage's
// own code is untouched.
void frame_geometry(int w, int h, int S, FrameDesc* fd) {
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
    fd->data = nullptr;
    fd->w = w;
    fd->h = h;
    fd->pitch = 0;
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

}  // namespace

extern "C" int octo_postprocess_frame_static(int32_t device, const float* d_head, int32_t num_anchors,
                                             int32_t num_classes, int32_t head_is_logits, float conf_thresh,
                                             float iou_thresh, int32_t max_det, int32_t net_size,
                                             int32_t frame_w, int32_t frame_h, octo_det_t* d_dets,
                                             int32_t* d_count, void* cuda_stream) {
    if (!d_head || !d_dets || !d_count) return OCTO_E_INVALID_ARG;
    if (device < 0 || device >= kMaxDevices) return OCTO_E_INVALID_ARG;
    if (num_anchors < 1 || num_classes < 1 || num_classes > OCTO_MAX_CLASSES) return OCTO_E_INVALID_ARG;
    if (head_is_logits != 0 && head_is_logits != 1) return OCTO_E_INVALID_ARG;
    if (!(conf_thresh >= 0.0f) || !(conf_thresh <= 1.0f)) return OCTO_E_INVALID_ARG;
    if (!(iou_thresh >= 0.0f) || !(iou_thresh <= 1.0f)) return OCTO_E_INVALID_ARG;
    if (max_det < 1) return OCTO_E_INVALID_ARG;
    if (net_size < 8 || net_size > 4096 || (net_size & 7)) return OCTO_E_INVALID_ARG;
    if (frame_w < 1 || frame_h < 1 || frame_w > 16384 || frame_h > 16384) return OCTO_E_INVALID_ARG;
    // the fixed workspace bounds the problem size
    if (num_anchors > kStaticMaxAnchors || max_det > kStaticMaxDet) return OCTO_E_CAPACITY;
    if ((reinterpret_cast<uintptr_t>(d_head) & 3) || (reinterpret_cast<uintptr_t>(d_dets) & 3) ||
        (reinterpret_cast<uintptr_t>(d_count) & 3))
        return OCTO_E_ALIGNMENT;

    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return report_cuda_error(e, "cudaSetDevice");
    unsigned char* base = nullptr;
    e = setup_device(device, &base);
    if (e != cudaSuccess) return report_cuda_error(e, "workspace set-up (cudaGetSymbolAddress)");
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);

    unsigned long long* d_keys = reinterpret_cast<unsigned long long*>(base + kOffKeys);
    float4* d_boxes = reinterpret_cast<float4*>(base + kOffBoxes);
    int* d_bidx = reinterpret_cast<int*>(base + kOffBidx);
    int* d_bcount = reinterpret_cast<int*>(base + kOffBcount);
    int* d_cand = reinterpret_cast<int*>(base + kOffCand);
    StageCounters* d_ctr = reinterpret_cast<StageCounters*>(base + kOffCtr);

    // The array keeps whatever the previous call left: the candidate counter and the counter
    // block must start at zero; keys and boxes are overwritten before they are read.
    e = cudaMemsetAsync(base + kOffBcount, 0, kScratchBytes - kOffBcount, stream);
    if (e != cudaSuccess) return report_cuda_error(e, "cudaMemsetAsync");

    int key_stride = 2;
    while (key_stride < num_anchors) key_stride <<= 1;  // <= kStaticMaxAnchors

    DecodeArgs da;
    da.d_head = d_head;
    da.n = 1; da.A = num_anchors; da.C = num_classes;
    da.layout = OCTO_HEAD_ROWS;
    da.logits = head_is_logits; da.class_agnostic = 0; da.multi_label = 0;
    da.conf = conf_thresh;
    da.key_stride = key_stride;
    da.d_keys = d_keys; da.d_cand_count = d_cand; da.d_status = &d_ctr->status;
    da.pdl = false;
    e = launch_decode(da, stream);
    if (e != cudaSuccess) return report_cuda_error(e, "decode_kernel");

    FrameDesc fd;
    frame_geometry(frame_w, frame_h, net_size, &fd);
    NmsArgs a;
    a.frames = &fd;
    a.d_tab = nullptr;
    a.pdl = false;
    a.n = 1;
    a.d_head = d_head;
    a.A = num_anchors;
    a.C = num_classes;
    a.layout = OCTO_HEAD_ROWS;
    a.iou_thr = iou_thresh;
    a.max_det = max_det;
    a.key_stride = key_stride;
    a.d_keys = d_keys;
    a.d_boxes = d_boxes;
    a.d_cand_count = d_cand;
    a.d_dets = d_dets;
    a.d_counts = d_count;
    a.num_branches = 0;  // no downstream branch lists here
    a.class_agnostic = 0;
    memset(&a.masks, 0, sizeof(a.masks));
    a.d_bcount = d_bcount;
    a.d_bidx = d_bidx;
    a.max_batch = 1;
    a.half_ctas = false;
    a.d_ctr = d_ctr;
    a.cluster = 1;
    a.d_dense_seen = nullptr;
    a.launch_seq = 0;
    e = launch_nms(a, stream);
    if (e != cudaSuccess) return report_cuda_error(e, "nms_kernel");
    return OCTO_OK;
}

extern "C" int octo_static_status(int32_t device, uint32_t* status_word, void* cuda_stream) {
    if (!status_word || device < 0 || device >= kMaxDevices) return OCTO_E_INVALID_ARG;
    cudaError_t e = cudaSetDevice(device);
    if (e != cudaSuccess) return report_cuda_error(e, "cudaSetDevice");
    unsigned char* base = nullptr;
    e = setup_device(device, &base);
    if (e != cudaSuccess) return report_cuda_error(e, "workspace set-up (cudaGetSymbolAddress)");
    e = cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return report_cuda_error(e, "cudaStreamSynchronize");
    unsigned int w = 0;
    e = cudaMemcpy(&w, &reinterpret_cast<StageCounters*>(base + kOffCtr)->status, sizeof(w), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return report_cuda_error(e, "cudaMemcpy");
    *status_word = w;
    return OCTO_OK;
}
