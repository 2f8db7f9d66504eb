// Internal definition of the stage object, shared by the files that implement the C ABI.
#pragma once

#include "octo.h"
#include "octo_kernels.h"

constexpr int kEventPairs = 2048;
constexpr int kNmsClusterWindow = 64;  // NMS launches that keep forming clusters after a crowded image was reported

struct octo_stage {
    octo_stage_config_t cfg;
    int sm_count;
    int key_stride;  // candidate slots per image: next power of two >= A
    // device workspace
    unsigned long long* d_keys;
    float4* d_boxes;
    int* d_cand_count;
    int* d_bcount;  // [branches][max_batch]
    int* d_bidx;    // [branches][max_batch][max_det]
    octo_item_t* d_items[OCTO_MAX_BRANCHES];
    octo::StageCounters* d_ctr;
    octo::FrameDesc* d_tab;  // [max_batch] frame table of a batch adopted on the device (chained stage)
    int64_t workspace_bytes;
    // host state of the current batch
    octo::FrameDesc frames[OCTO_MAX_BATCH];
    int n_frames;
    bool tab_on_device;  // the current batch's table is d_tab (octo_adopt_items_device), not `frames`
    int max_w;
    bool have_dets;
    const octo_det_t* d_dets;
    const int32_t* d_last_n_items[OCTO_MAX_BRANCHES];  // {packed, total} of the last crop call per branch (caller's buffer)
    int64_t launches;
    // Cluster size of the NMS launches.  The kernel reports through an integer in mapped host memory
    // (no copy, no synchronisation) the number of the latest launch that saw an image with many
    // candidates; for kNmsClusterWindow launches after it (the host may have enqueued many launches
    // that the GPU has not run yet), launches with few images give every image a cluster of CTAs.
    int nms_max_cluster;
    int nms_cluster_mode;  // 0 automatic, else the caller's size
    int nms_cluster_last;  // size of the latest launch
    bool nms_half_last;    // the latest launch ran two half-sized CTAs per SM
    int nms_seq;
    int* h_dense_seen;  // host view (volatile reads)
    int* d_dense_seen;  // device view of the same integer
    // optional per-kernel timing
    bool timing;
    cudaEvent_t ev[2 * kEventPairs];
    int ev_kernel[kEventPairs];
    int ev_used;
    int64_t ev_dropped;
};

