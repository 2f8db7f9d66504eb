// Internal launcher interface between the stage object (octo_stage.cu) and the kernels.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "octo.h"
#include "octo_common.cuh"

namespace octo {

typedef octo_det_t octo_det_rec;

struct BranchMasks {
    uint32_t m[OCTO_MAX_BRANCHES][4];
};

struct DecodeArgs {
    const float* d_head;
    int n, A, C;
    int layout;  // OCTO_HEAD_ROWS / OCTO_HEAD_PLANES
    int logits, class_agnostic, multi_label;
    float conf;
    int key_stride;
    unsigned long long* d_keys;
    int* d_cand_count;
    unsigned int* d_status;
    bool pdl;  // launch with programmatic stream serialisation (small batches)
};

struct NmsArgs {
    const FrameDesc* frames;  // host
    const FrameDesc* d_tab;   // device-resident frame table of a chained stage, or null
    bool pdl;                 // launch with programmatic stream serialisation (small batches)
    int n;
    const float* d_head;
    int A, C;
    int layout;  // OCTO_HEAD_ROWS / OCTO_HEAD_PLANES
    float iou_thr;
    int max_det, key_stride;
    unsigned long long* d_keys;
    float4* d_boxes;
    int* d_cand_count;
    octo_det_t* d_dets;
    int* d_counts;
    int num_branches;
    int class_agnostic;  // NMS across classes; the class of a survivor is recomputed for the output
    BranchMasks masks;
    int* d_bcount;
    int* d_bidx;
    int max_batch;
    StageCounters* d_ctr;
    // CTAs per image (a thread-block cluster; 1, 2, 4 or 8).  More than one pays off when few
    // images carry many candidates each.  d_dense_seen (device pointer to an integer the host can
    // read, or null): the kernel stores launch_seq there when an image had many candidates; the
    // caller picks the cluster size of later launches from it.
    int cluster;
    int* d_dense_seen;
    int launch_seq;
    // two half-sized CTAs per SM (half the threads and half the on-chip capacity each) instead of
    // one: for batches of more images than SMs whose images are sparse
    bool half_ctas;
};

// Branch options of the crop kernel, per INPUT channel c (output plane swap_rb ? 2 - c : c):
// value' = value * sc[c] + of[c]; fill[c] is the canvas value after the same mapping.
struct CropOpts {
    int keep_aspect;
    float sc[3], of[3], fill[3];
};

struct CropArgs {
    const FrameDesc* frames;  // host
    const FrameDesc* d_tab;   // device-resident frame table of a chained stage, or null
    bool pdl;                 // launch with programmatic stream serialisation (small batches)
    int n;
    int max_det, first_item, max_items;
    const int* d_bcount;  // this branch's [max_batch]
    const int* d_bidx;    // this branch's [max_batch][max_det]
    const octo_det_t* d_dets;
    int* d_offsets;
    int* d_n_items;
    octo_item_t* d_items;
    void* d_out;
    int out_w, out_h, swap_rb, sm_count;
    StageCounters* d_ctr;
    bool general;   // keep_aspect or normalize set for the branch
    CropOpts opts;
};

// Branch options -> kernel form (per input channel, see CropOpts).
void fill_crop_opts(const octo_branch_cfg_t& br, int swap_rb, int pad_value, CropOpts* out);
int validate_branch_options(const octo_branch_cfg_t& br);  // OCTO_OK or OCTO_E_INVALID_ARG

// Records the text that octo_last_cuda_error returns on this thread; returns OCTO_E_CUDA.
int report_cuda_error(cudaError_t e, const char* what);

// Opt the kernels of every table capacity into the shared memory they need (current device).
cudaError_t prepare_letterbox();
// max_cluster (optional): the largest cluster of the NMS kernel (8, 4, 2 or 1) that the current
// device can co-schedule.
cudaError_t prepare_nms(int* max_cluster = nullptr);
cudaError_t prepare_crop();

cudaError_t launch_letterbox(const FrameDesc* frames, int n, void* d_out, int S, int max_w, int pad_value,
                             int swap_rb, unsigned int* d_status, bool pdl, cudaStream_t stream);
cudaError_t launch_decode(const DecodeArgs& a, cudaStream_t stream);
cudaError_t launch_nms(const NmsArgs& a, cudaStream_t stream);
cudaError_t launch_crop(const CropArgs& a, cudaStream_t stream);  // batch assembler + crop-resize
cudaError_t launch_crop_queue(const QRecord* d_staged, const int* d_qpacked, int bz, void* d_out, int out_w,
                              int out_h, int swap_rb, int sm_count, unsigned int* d_status, int* d_sched,
                              const CropOpts* general, cudaStream_t stream);

constexpr int kLetterboxMaxWidth = 8192;  // widest frame the row staging supports

// Batches up to this size are launched with programmatic dependent launch (see pdl_enter).
constexpr int kPdlMaxBatch = 16;

// One kernel launch; with `pdl` the launch carries the programmatic stream serialisation
// attribute, so the kernel may be scheduled while its predecessor in the stream still runs (it
// waits for that predecessor in pdl_enter before it touches memory).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                 bool pdl, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1u : 0u;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// The same with a thread-block cluster of `cluster` CTAs along x (grid.x is a multiple of it).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_kernel_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                         cudaStream_t stream, bool pdl, int cluster, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    unsigned na = 0;
    if (cluster > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = (unsigned)cluster;
        attr[na].val.clusterDim.y = 1;
        attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

}  // namespace octo
