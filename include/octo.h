/*
 * octo.h -- C ABI of the cascade-stage tensor library (CUDA, sm_100a).
 *
 * A "stage" is one model instance of a DNN cascade as the paper states it: it receives a
 * batch of bz inputs, runs on an assigned execution stream and emits outputs that become
 * the inputs of its downstream models (Section II, Eq. 1 and Table II: In_m / Out_m =
 * "image - bounding box"; Section III-C "Inference Stream"; the traffic pipeline
 * [Object Detect -> Vehicle Classify, Plate Detect] of Section I).  This library is the
 * per-batch tensor work around the detector of such a stage:
 *
 *   octo_preprocess_batch   frames (BGR uint8)  -> letterboxed fp16 NCHW detector batch
 *   [the caller runs the detector]
 *   octo_postprocess_batch  detector head       -> per-frame detections (decode, confidence
 *                                                  filter, class-aware NMS, frame pixels)
 *   octo_crop_batch         detections + frames -> one downstream branch's fp16 batch
 *                                                  (batch assembler + ROI crop-resize)
 *
 * The paper gives no formula for this work; the numeric rules are fixed in the comments
 * below, and each has exactly one correct result.
 *
 * Conventions
 *   - Pointers named d_* are DEVICE pointers owned by the caller; everything else is host
 *     memory.  The library never frees or retains caller buffers, except that the frames
 *     passed to octo_preprocess_batch are read again by octo_crop_batch (see there).
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).  The three
 *     batch calls only enqueue work on it and return; they never synchronise.
 *   - A stage (or queue) object is not re-entrant: use it from one host thread and one stream
 *     at a time.  One exception: the kernel of octo_preprocess_batch shares no device data with
 *     the kernels of octo_postprocess_batch and octo_crop_batch of the same batch (it reads the
 *     frames and writes the detector input; they read the head and the frames; the status word
 *     is updated atomically), so the call may be given a second stream and its kernel runs beside
 *     theirs.  The host calls still come from one thread in the usual order, and the next
 *     batch's calls wait for both streams.  Different objects are independent: the library keeps no state outside them
 *     (apart from the fixed workspace of octo_postprocess_frame_static), so several host
 *     threads may each drive their own stage, on one GPU or on several.
 *   - Every function returns OCTO_OK (0) or a negative octo_status_t.  No exception
 *     crosses the boundary and nothing aborts the process.  Conditions detected on the
 *     device (non-finite head values, a wait that ran out) set bits in a status word read
 *     with octo_stage_status.
 */
#ifndef OCTO_H_
#define OCTO_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define OCTO_API __attribute__((visibility("default")))
#else
#define OCTO_API
#endif

#define OCTO_MAX_BRANCHES 4
#define OCTO_MAX_CLASSES 128
#define OCTO_MAX_BATCH 512

typedef enum {
    OCTO_OK = 0,
    OCTO_E_INVALID_ARG = -1,   /* null pointer, size out of range, bad configuration      */
    OCTO_E_CAPACITY = -2,      /* n > max_batch, frame wider than the stage supports      */
    OCTO_E_ALIGNMENT = -3,     /* pointer or pitch not a multiple of 16 bytes             */
    OCTO_E_NO_PREPROCESS = -4, /* post/crop called before any octo_preprocess_batch       */
    OCTO_E_CUDA = -5,          /* a CUDA runtime call failed (octo_last_cuda_error)       */
    OCTO_E_DEVICE_TIMEOUT = -6,/* a bounded device-side wait gave up (status word)        */
    OCTO_E_NO_POSTPROCESS = -7,/* crop called before octo_postprocess_batch of this batch */
    OCTO_E_NO_MEMORY = -8      /* host or device memory could not be allocated            */
} octo_status_t;

/* Bits of the device status word. */
#define OCTO_STATUS_NONFINITE 0x1u      /* an examined head row held NaN/Inf and was dropped */
#define OCTO_STATUS_TRUNCATED 0x2u      /* a crop window held fewer slots than items         */
#define OCTO_STATUS_COPY_TIMEOUT 0x4u   /* a bulk-copy wait ran out; that tile was skipped    */
#define OCTO_STATUS_BIG_NMS 0x8u        /* an image had more candidates than fit on chip and   */
                                        /* took the slower global-memory path (informational)  */
#define OCTO_STATUS_CAND_OVERFLOW 0x10u /* multi-label decode found more candidates in an image */
                                        /* than the workspace holds; the excess was dropped    */
#define OCTO_STATUS_BOUNDS 0x20u        /* checked build only (-DOCTO_BOUNDS_CHECK): an index    */
                                        /* left its range; the access was skipped               */

/* Head layouts (octo_stage_config_t.head_layout). */
#define OCTO_HEAD_ROWS 0   /* [n, A, 5 + C]: rows (cx, cy, w, h, obj, class_0 ..)              */
#define OCTO_HEAD_PLANES 1 /* [n, 4 + C, A]: planes cx, cy, w, h, class_0 ..; no objectness    */

typedef struct octo_stage octo_stage_t; /* opaque; owned by the library */

/* One downstream branch (e.g. vehicle classifier 224x224, plate detector 256x256).
 * class_mask: bit k (word k/32, bit k%32) set => detections of class k feed this branch.
 * The last four fields select what the downstream model expects of its input; all zero gives
 * the plain form (stretch, value / 255). */
typedef struct {
    int32_t out_w, out_h;   /* crop size; out_w must be a multiple of 8 */
    uint32_t class_mask[4];
    int32_t keep_aspect;    /* 1: fit the rectangle into out_w x out_h without distortion     */
                            /* (centred, rest of the slot = the stage's pad_value)            */
    int32_t normalize;      /* 1: output = (value / 255 - mean[p]) / std[p] for output plane p */
    float mean[3], std[3];  /* per OUTPUT plane (after swap_rb); std > 0; used if normalize   */
} octo_branch_cfg_t;

typedef struct {
    int32_t device;         /* CUDA device ordinal                                          */
    int32_t net_size;       /* S: side of the square detector input, multiple of 8 (640)    */
    int32_t max_batch;      /* upper bound on n; sizes the workspace (<= OCTO_MAX_BATCH)    */
    int32_t num_anchors;    /* A: rows of the head per image (25200 at S = 640)             */
    int32_t num_classes;    /* C <= OCTO_MAX_CLASSES; a head row is 5 + C floats            */
    int32_t head_is_logits; /* 1: obj / class values are logits; 0: probabilities           */
    float conf_thresh;      /* candidate iff score > conf_thresh (strict)                   */
    float iou_thresh;       /* suppress iff IoU > iou_thresh (strict)                       */
    int32_t max_det;        /* detections kept per frame                                    */
    int32_t pad_value;      /* canvas fill, 0..255 (114)                                    */
    int32_t swap_rb;        /* 1: output plane 0 = input channel 2 (BGR -> RGB)             */
    int32_t num_branches;   /* 1..OCTO_MAX_BRANCHES                                         */
    int32_t class_agnostic; /* 1: NMS suppresses across classes (one class for NMS only)    */
    int32_t head_layout;    /* OCTO_HEAD_ROWS (0) or OCTO_HEAD_PLANES; see octo_postprocess_batch */
    int32_t multi_label;    /* 1: every class above the threshold is a candidate of its own  */
    octo_branch_cfg_t branch[OCTO_MAX_BRANCHES];
} octo_stage_config_t;

/* One source frame: interleaved 3-channel uint8 rows, pixel (y, x) at
 * d_data + y * pitch_bytes + 3 * x.  d_data must be 16-byte aligned, pitch_bytes a multiple
 * of 16 and >= 3 * width (rows are fetched with 16-byte bulk copies). */
typedef struct {
    const uint8_t* d_data;
    int32_t width, height, pitch_bytes;
    int32_t _pad;
} octo_frame_t;

/* One detection, 32 bytes.  Box in source-frame pixels, clamped to the frame. */
typedef struct {
    float x1, y1, x2, y2, score;
    int32_t cls, anchor, _pad;
} octo_det_t;

/* One packed item of a branch batch: which detection it is and the integer source
 * rectangle [rx0, rx1) x [ry0, ry1) that was resized into the slot. */
typedef struct {
    int32_t frame, det, rx0, ry0, rx1, ry1, _pad[2];
} octo_item_t;

typedef struct {
    int64_t candidates;   /* rows that passed the confidence filter since the last get_stats */
    int64_t kept;         /* detections after NMS since the last get_stats                   */
    int64_t packed;       /* items written by the last crop call                            */
    int64_t total_items;  /* items the last crop call's branch holds in total               */
    uint32_t status_word; /* same as octo_stage_status                                      */
    int32_t max_candidates_per_image;
} octo_stage_stats_t;

/*
 * Create a stage on cfg->device and allocate its workspace (candidate keys
 * max_batch * A * 8 bytes, per-branch item tables, counters).  Arguments are validated
 * before any CUDA call, so OCTO_E_INVALID_ARG is reported even on a machine without a GPU.
 * On success *out owns the workspace until octo_stage_destroy.
 */
OCTO_API int octo_stage_create(const octo_stage_config_t* cfg, octo_stage_t** out);

/* Free the workspace.  The caller must have synchronised the streams that used it. */
OCTO_API int octo_stage_destroy(octo_stage_t* st);

/*
 * Letterbox n frames into the detector batch (stage input In_m of Table II).
 *   frames          host array of n descriptors; device pixels stay owned by the caller and
 *                   must remain valid and unchanged until the last octo_crop_batch of this
 *                   batch has run.
 *   d_out_f16_nchw  device, [n, 3, S, S] binary16, 16-byte aligned, fully overwritten.
 * Rule: the longer side maps to S, the other to round-half-up(h*S/w) in integer arithmetic
 * (at least 1); the image is centred, an odd remainder goes right/bottom; canvas =
 * pad_value/255.  Bilinear, half-pixel centres: source x = (dx + 0.5) * w/nw - 0.5 clamped
 * to [0, w-1], no antialiasing, raw 0..255 values; output = half(v / 255).  Plane order per
 * swap_rb.  Also records the frame table used by the next two calls.
 * Errors: OCTO_E_INVALID_ARG (null, n < 1, non-positive size, pitch < 3*width),
 * OCTO_E_CAPACITY (n > max_batch), OCTO_E_ALIGNMENT, OCTO_E_CUDA.
 */
OCTO_API int octo_preprocess_batch(octo_stage_t* st, const octo_frame_t* frames, int32_t n,
                          void* d_out_f16_nchw, void* cuda_stream);

/* One input of a chained (second-level) stage: the rectangle [rx0, rx1) x [ry0, ry1) of a source
 * frame, as reported in an upstream stage's item table. */
typedef struct {
    const uint8_t* d_data;                 /* the ORIGINAL frame (same rules as octo_frame_t) */
    int32_t width, height, pitch_bytes;
    int32_t rx0, ry0, rx1, ry1;
    int32_t _pad;
} octo_region_t;

/*
 * Chained stage (the paper's cascades continue below the first detector, e.g. vehicle crop ->
 * plate detector, person crop -> face detector; Section I and Section III-B, Observation 1).
 * Declares that this stage's current batch consists of n regions which an upstream stage has
 * already cropped and stretched to net_size x net_size: the upstream octo_crop_batch output
 * (a branch with out_w = out_h = net_size) IS this stage's detector input, so no kernel runs
 * here.  The call records the table that the next octo_postprocess_batch and octo_crop_batch
 * use: head boxes, given on the net_size x net_size grid, are mapped back into the rectangle of
 * the original frame, X = rx0 + x * fl((rx1 - rx0) / net_size), clamped to the rectangle, and
 * this stage's own crops are resampled from the original frame pixels.
 *   regions  host array of n entries, normally filled from octo_stage_copy_items of the
 *            upstream stage plus that stage's frame descriptors.
 * Errors: OCTO_E_INVALID_ARG (null, n < 1, rectangle empty or outside its frame, pitch < 3 *
 * width), OCTO_E_CAPACITY (n > max_batch), OCTO_E_ALIGNMENT.
 */
OCTO_API int octo_adopt_regions(octo_stage_t* st, const octo_region_t* regions, int32_t n, void* cuda_stream);

/*
 * The same hand-off without the host (Section I: the cascade continues below the first detector;
 * Section III-B, Observation 1: what a detector emits is what its downstream models receive).
 * This stage's batch becomes entries [first, first + n) of the item table that the LAST
 * octo_crop_batch of `branch` on `upstream` built (entry k = slot k of that call's window), read
 * on the device: one small kernel on `cuda_stream` writes this stage's frame table into its own
 * workspace, and the following octo_postprocess_batch / octo_crop_batch / octo_queue_push read it
 * there.  Nothing synchronises and no item travels through host memory, so a chained detector
 * can be enqueued right behind the upstream pass.  n is the batch size the downstream detector
 * runs with (the head has n images); if the upstream call packed fewer than first + n items,
 * the surplus entries are empty: they yield no detections whatever their head holds.
 * Requirements: both stages on one device; upstream.branch[branch] is net_size x net_size of
 * this stage; the upstream crop call was enqueued before this call, on the same stream or
 * ordered with it; the buffer that call wrote {packed, total} to (d_n_items) and the upstream
 * frames stay valid until this stage's batch is done.  Mapping rule and errors as
 * octo_adopt_regions, plus OCTO_E_NO_POSTPROCESS (the branch has not been cropped yet).
 */
OCTO_API int octo_adopt_items_device(octo_stage_t* st, const octo_stage_t* upstream, int32_t branch, int32_t first,
                                     int32_t n, void* cuda_stream);

/*
 * Decode the detector head of the batch last given to octo_preprocess_batch (n must match)
 * into detections (stage output Out_m of Table II; the per-frame count is what drives the
 * downstream request rate, Section III-B Observation 1).
 *   d_head    device, [n, A, 5 + C] float32 contiguous, rows (cx, cy, w, h, obj, class_0..)
 *             with the box in letterbox pixels; 4-byte aligned.
 *   d_dets    device, [n, max_det] records; entries [0, d_counts[i]) of frame i are written.
 *   d_counts  device, [n] int32.
 * Rules.  Candidate: every value of the row finite, w > 0, h > 0, k* = first maximal class
 * value, score = fl(sigma(obj) * sigma(c_k*)) (or fl(obj * c_k*) for probabilities),
 * score > conf_thresh.  sigma is a fixed sequence of binary32 operations (see the kernel
 * source), not the platform expf, so scores are reproducible bit for bit.  Order: score
 * descending, ties by lower anchor index.  NMS: walking that order, a candidate is kept iff
 * no earlier KEPT candidate of the same class has IoU > iou_thresh, IoU evaluated in
 * binary32 as inter / (area_a + area_b - inter) on letterbox-pixel corners
 * x1 = cx - w/2 ...; at most max_det are kept.  Kept boxes are mapped to frame pixels,
 * X = (x - pad_left) * fl(w / nw), clamped to [0, w] x [0, h].
 * Variants (stage configuration; the paper's pipelines mix detector families, Section V-A).
 *   head_layout = OCTO_HEAD_PLANES: d_head is [n, 4 + C, A] (anchor-free heads; value e of
 *     anchor a at e * A + a, 16-byte alignment lets the scan use vector loads).  There is no
 *     objectness: score = sigma(c_k*) for logits, c_k* for probabilities; everything else as
 *     above.
 *   multi_label = 1: every class k whose own score (sigma(obj) * sigma(c_k), or the planes
 *     form) exceeds conf_thresh is a candidate of class k; candidates of one anchor share its
 *     box.  Order: score descending, then anchor, then class.  The workspace holds 2 * P
 *     candidates per image (P = A rounded up to a power of two); an image that yields more
 *     sets OCTO_STATUS_CAND_OVERFLOW and loses the excess.  Not combinable with class_agnostic.
 * Errors: OCTO_E_INVALID_ARG, OCTO_E_NO_PREPROCESS, OCTO_E_CUDA.
 */
OCTO_API int octo_postprocess_batch(octo_stage_t* st, const float* d_head, int32_t n,
                           octo_det_t* d_dets, int32_t* d_counts, void* cuda_stream);

/*
 * Pack one branch's downstream batch (the model input that the scheduler's batch size bz of
 * Algorithm 1 cuts into batches): batch assembler, then ROI crop-resize.
 *   branch      index into cfg.branch.
 *   first_item, max_items  window [first_item, first_item + max_items) of the branch's item
 *               list; lets the caller cut the list into batches of bz.
 *   d_out_f16   device, [max_items, 3, out_h, out_w] binary16, 16-byte aligned.  Item i of
 *               the window is written to slot i - first_item; slots >= packed are untouched.
 *   d_offsets   device, [n + 1] int32: exclusive prefix sum of the per-frame number of kept
 *               detections whose class is in the branch's mask; d_offsets[n] = total.
 *   d_n_items   device, [2] int32: {packed, total}.  total > first_item + max_items is not
 *               an error (OCTO_STATUS_TRUNCATED is set).
 * Item offsets[f] + j is the j-th masked detection of frame f in NMS output order.  Its
 * rectangle is rx0 = clamp(floor(x1), 0, w-1), rx1 = clamp(ceil(x2), rx0 + 1, w), likewise
 * in y; the rectangle is stretched to out_w x out_h with the same bilinear rule as the
 * letterbox (taps clamped inside the rectangle), same plane order, /255, binary16.
 * Branch options.  keep_aspect: the cw x ch rectangle is resized to nw x nh, where the side
 * with the larger ratio fills the slot (nw = out_w if out_w * ch <= out_h * cw, else nh =
 * out_h) and the other is round-half-up of the exact quotient (at least 1), centred with the
 * odd pixel right / bottom as in the letterbox; the rest of the slot holds pad_value / 255.
 * normalize: every output value v (pixels and padding alike) becomes (v - mean[p]) / std[p].
 * Uses the detections written by the last octo_postprocess_batch (d_dets must still be
 * valid) and the frames of the last octo_preprocess_batch.
 * Errors: OCTO_E_INVALID_ARG, OCTO_E_NO_PREPROCESS, OCTO_E_NO_POSTPROCESS, OCTO_E_CUDA.
 */
OCTO_API int octo_crop_batch(octo_stage_t* st, int32_t branch, int32_t first_item, int32_t max_items,
                    void* d_out_f16, int32_t* d_offsets, int32_t* d_n_items, void* cuda_stream);

/* ---- device-side dynamic-batch queue -------------------------------------------------------
 * Downstream models take batches of the size bz the scheduler chose (Algorithm 1), while the
 * number of objects per frame varies and arrives in bursts; requests wait in a queue until a
 * batch fills, the first one waiting longest (Section II, Eq. 1 discussion; Section III-B,
 * Observation 1).  An octo_queue_t keeps such pending items of ONE downstream branch on the
 * device across successive detector batches: octo_queue_push appends the items of a stage's
 * current batch, octo_queue_pop crops the oldest bz of them into a downstream batch.  Order
 * is first in, first out: pushes in call order, inside a push the branch's item order.  Items
 * that do not fit are dropped (newest first) and counted.  Queued items refer to their source
 * frames by pointer: the caller keeps those frames alive and unchanged until the items are
 * popped.  Not re-entrant; use one stream at a time.
 */
typedef struct octo_queue octo_queue_t;

/* One queued item as reported by octo_queue_pop (48 bytes). */
typedef struct {
    const uint8_t* d_data;              /* source frame                                   */
    int32_t width, height, pitch_bytes;
    int32_t rx0, ry0, rx1, ry1;         /* crop rectangle                                 */
    int32_t seq;                        /* number of the push that queued it (from 0)     */
    int32_t frame, det;                 /* position in that push's batch                  */
} octo_qitem_t;

/* capacity: items the ring holds; out_w (multiple of 8) x out_h: crop size; max_bz: largest bz. */
OCTO_API int octo_queue_create(int32_t device, int32_t capacity, int32_t out_w, int32_t out_h, int32_t swap_rb,
                               int32_t max_bz, octo_queue_t** out);
OCTO_API int octo_queue_destroy(octo_queue_t* q);

/* Crop options of the queue's downstream model: keep_aspect, normalize, mean and std of *options
 * are used as in octo_branch_cfg_t (its other fields are ignored), pad_value (0..255) fills the
 * canvas of aspect-preserving crops.  Takes effect from the next pop.  Errors: OCTO_E_INVALID_ARG. */
OCTO_API int octo_queue_set_options(octo_queue_t* q, const octo_branch_cfg_t* options, int32_t pad_value);

/* Append the items of `branch` of the stage's current batch (after octo_postprocess_batch;
 * same item order and rectangles as octo_crop_batch would use).  Enqueues one kernel.
 * Errors: OCTO_E_INVALID_ARG, OCTO_E_NO_PREPROCESS, OCTO_E_NO_POSTPROCESS, OCTO_E_CUDA. */
OCTO_API int octo_queue_push(octo_queue_t* q, octo_stage_t* st, int32_t branch, void* cuda_stream);

/* Crop the oldest min(bz, pending) items into d_out_f16 [bz, 3, out_h, out_w] (slot i = i-th
 * oldest; slots >= popped untouched) and remove them.  d_items_out (may be NULL): [bz] records
 * of the popped items.  d_info: [4] int32 = {popped, pending after the pop, items dropped so far,
 * seq of the oldest item still pending or -1}.  Enqueues two kernels; nothing synchronises.
 * Errors: OCTO_E_INVALID_ARG (bz < 1 or > max_bz, null pointers), OCTO_E_ALIGNMENT, OCTO_E_CUDA. */
OCTO_API int octo_queue_pop(octo_queue_t* q, int32_t bz, void* d_out_f16, octo_qitem_t* d_items_out,
                            int32_t* d_info, void* cuda_stream);

/* octo_queue_pop with the release rule decided on the device, so that a serving loop can call it
 * after every detector batch without reading the queue state back: the oldest min(bz, pending)
 * items are released if a full batch is pending, or if the first pending item has waited for at
 * least max_wait pushes (a batch fills at the arrival rate and its first request waits longest,
 * Section II, discussion of Eq. 1); otherwise nothing is popped and d_info[0] = 0.  max_wait < 0
 * releases unconditionally (octo_queue_pop).  Same arguments and errors as octo_queue_pop. */
OCTO_API int octo_queue_pop_due(octo_queue_t* q, int32_t bz, int32_t max_wait, void* d_out_f16,
                                octo_qitem_t* d_items_out, int32_t* d_info, void* cuda_stream);

/* Synchronise `cuda_stream`, then read (and keep) the device status word. */
OCTO_API int octo_stage_status(octo_stage_t* st, uint32_t* status_word, void* cuda_stream);

/* Test support for the time-out path: enqueue a one-thread kernel that arms a barrier for bytes
 * that never arrive (no copy is issued), polls it `polls` times (1 .. 2^20) and then sets
 * OCTO_STATUS_COPY_TIMEOUT, exactly as the bulk-copy waits of the letterbox and crop kernels do
 * when they give up.  Afterwards octo_stage_status returns OCTO_E_DEVICE_TIMEOUT until the status
 * word is cleared; the context stays usable. */
OCTO_API int octo_stage_selftest_wait(octo_stage_t* st, int32_t polls, void* cuda_stream);

/* Clear the device status word (enqueued on the stream). */
OCTO_API int octo_stage_clear_status(octo_stage_t* st, void* cuda_stream);

/* Synchronise `cuda_stream`, then fill *stats from the stage's device counters; the
 * candidate / kept / max counters restart from zero afterwards. */
OCTO_API int octo_stage_get_stats(octo_stage_t* st, octo_stage_stats_t* stats, void* cuda_stream);

/* Device pointer to the item table the last octo_crop_batch of `branch` built (entries
 * [0, packed)); stage-owned, valid until the next crop call on that branch. */
OCTO_API int octo_stage_item_table(octo_stage_t* st, int32_t branch, const octo_item_t** d_items);

/* Synchronise `cuda_stream`, then copy the first `count` entries of that table to host
 * memory (count <= max_batch * max_det). */
OCTO_API int octo_stage_copy_items(octo_stage_t* st, int32_t branch, octo_item_t* items_out, int32_t count,
                                   void* cuda_stream);

/* Kernel order used by octo_kernel_times_t.  OCTO_K_ASSEMBLE stays zero: the batch assembler
 * runs inside the crop kernel. */
enum { OCTO_K_LETTERBOX = 0, OCTO_K_DECODE = 1, OCTO_K_NMS = 2, OCTO_K_ASSEMBLE = 3, OCTO_K_CROP = 4,
       OCTO_K_COUNT = 5 };

typedef struct {
    double ms[OCTO_K_COUNT];        /* summed device time of each kernel's launches            */
    int64_t launches[OCTO_K_COUNT]; /* launches measured                                       */
    int64_t dropped;                /* launches not measured because the event pool was full   */
} octo_kernel_times_t;

/* Per-kernel timing for profiling: while enabled, every kernel launch is bracketed by CUDA
 * events recorded on the launching stream (a small cost per launch).  Off by default. */
OCTO_API int octo_stage_set_timing(octo_stage_t* st, int32_t enable);

/* Synchronise `cuda_stream`, sum the event pairs recorded since the previous call into
 * *times and release them. */
OCTO_API int octo_stage_kernel_times(octo_stage_t* st, octo_kernel_times_t* times, void* cuda_stream);

/* CTAs per image of the NMS launches (paper Section III-C: a stage is scheduled by its latency,
 * and a crowded scene served at a small batch leaves most of the GPU idle with one CTA per image).
 * cluster = 0 (the default): automatic.  The stage gives every image a thread-block cluster of 2,
 * 4 or 8 CTAs while the batch has at most a half, a quarter or an eighth as many images as the GPU
 * has SMs and one of the stage's latest 64 NMS launches is known to have seen an image with more
 * than 1024 candidates (the kernel reports that through mapped host memory; nothing is copied or
 * synchronised, so the report of a launch may arrive a few calls late).  cluster =
 * 1, 2, 4, 8: that size for every launch (clamped to what the device can co-schedule).  Results do
 * not depend on the size.  OCTO_E_INVALID_ARG for any other value. */
OCTO_API int octo_stage_set_nms_cluster(octo_stage_t* st, int32_t cluster);

/* Cluster size of the stage's latest NMS launch (0 before the first one, or for a null stage). */
OCTO_API int32_t octo_stage_last_nms_cluster(const octo_stage_t* st);

/* 1 when the stage's latest NMS launch ran two half-sized CTAs per SM, else 0.  In automatic mode a
 * batch of more images than the GPU has SMs is launched that way (one wave of CTAs instead of
 * two) unless one of the stage's latest 64 NMS launches is known to have seen an image with more
 * than 1024 candidates; a half-sized CTA holds 4096 candidates on chip instead of 8192 and sends
 * a larger image through the global-memory path.  Results do not depend on the form. */
OCTO_API int32_t octo_stage_last_nms_half_ctas(const octo_stage_t* st);

/* Bytes of device memory the stage holds. */
OCTO_API int64_t octo_stage_workspace_bytes(const octo_stage_t* st);

/* Number of kernels the stage has launched since creation (for launch accounting). */
OCTO_API int64_t octo_stage_launch_count(const octo_stage_t* st);

/*
 * Decode + class-aware NMS of ONE frame's head without any device allocation.
 * (An addition for embedders; the paper has no counterpart to it.)
 *
 * Who needs it: callers that are not allowed to allocate GPU memory when they run, e.g. a
 * real-time loop that fixed its memory budget at start-up and may not enter the allocator
 * again, or a component hosted inside another application's memory pool with buffers handed
 * to it.  octo_stage_create allocates a workspace, so those callers cannot own a stage.
 * This call does the work of octo_postprocess_batch for n = 1 with the same kernels and the
 * same rules, on a fixed workspace that is part of the library itself: about 0.8 MB of
 * device memory that every GPU loading the library holds until the process exits.  It
 * calls no cudaMalloc / cudaFree and no allocating library routine.
 *
 * Limits: num_anchors <= OCTO_STATIC_MAX_ANCHORS and max_det <= OCTO_STATIC_MAX_DET, else
 * OCTO_E_CAPACITY.  The caller passes the input and both outputs:
 *   d_head   device, [num_anchors, 5 + num_classes] float32 (same layout as a stage's head)
 *   d_dets   device, [max_det] records; entries [0, *d_count) are written
 *   d_count  device, one int32
 * frame_w / frame_h / net_size give the letterbox geometry used to map boxes back to frame
 * pixels, exactly as a stage would after preprocessing a frame of that size.
 *
 * The first call on a device looks up the workspace's device address and configures the
 * kernels; make that first call before starting any stream capture.  All calls on a device
 * share the one workspace, which keeps the previous call's contents (the call clears what
 * has to start at zero): two calls whose GPU work overlaps, e.g. on different streams, race.
 * Issue them on one stream or order them with events.
 * Errors: OCTO_E_INVALID_ARG, OCTO_E_CAPACITY, OCTO_E_ALIGNMENT, OCTO_E_CUDA.
 */
#define OCTO_STATIC_MAX_ANCHORS 32768
#define OCTO_STATIC_MAX_DET 1024
OCTO_API int octo_postprocess_frame_static(int32_t device, const float* d_head, int32_t num_anchors,
                                           int32_t num_classes, int32_t head_is_logits, float conf_thresh,
                                           float iou_thresh, int32_t max_det, int32_t net_size,
                                           int32_t frame_w, int32_t frame_h, octo_det_t* d_dets,
                                           int32_t* d_count, void* cuda_stream);

/* Synchronise `cuda_stream`, then read the status word of the last octo_postprocess_frame_static
 * call on `device` (OCTO_STATUS_NONFINITE, OCTO_STATUS_BIG_NMS; every call starts from zero).
 * Allocates nothing.  (Part of the same addition; no counterpart in the paper.) */
OCTO_API int octo_static_status(int32_t device, uint32_t* status_word, void* cuda_stream);

/* ---- placement of model instances on GPU inference streams (host only) ---------------------
 * The paper's co-location scheduler (Section III-C "Inference Stream", Algorithm 2): a GPU runs
 * several streams side by side; an execution occupies a portion of one stream, as long as its
 * run time and as wide as the share of the GPU's compute it needs; a stream repeats with a duty
 * cycle (half the pipeline's SLO).  Instances are placed one replica number at a time over all
 * pipelines and their models in order.  Each goes to the stream whose free gap around the window
 * [start_us, end_us) is the tightest (the least spare room), among the streams where (1) that
 * window is free and inside the stream's cycle, (2) the GPU stays within memory (sum of weights +
 * per-stream largest intermediate memory <= mem_bytes) and utilisation (sum over streams of the
 * widest resident <= util_max_permille) and (3) the stream's duty cycle is not longer than the
 * instance's.  Ties go to the lower GPU, then the lower stream.  The first instance on a stream
 * fixes the stream's duty cycle; a stream without residents counts as an unbounded gap, so it is
 * only taken when no bounded gap fits.  All arrays are host memory; no CUDA call is made. */
typedef struct {
    int32_t pipeline, model, instance; /* pipeline index, position in its execution order, replica number */
    int32_t util_permille;             /* width: share of the GPU's compute, 0..1000            */
    int64_t start_us, end_us;          /* window inside the duty cycle, start < end <= duty cycle */
    int64_t duty_cycle_us;             /* duty cycle of the instance's pipeline                  */
    int64_t weight_bytes, inter_bytes; /* weight memory, intermediate (activation) memory        */
} octo_coral_instance_t;

typedef struct {
    int64_t mem_bytes;          /* memory available to models                         */
    int32_t util_max_permille;  /* utilisation limit                                  */
    int32_t num_streams;        /* streams the GPU is divided into, 1..1024           */
} octo_coral_gpu_t;

typedef struct {
    int32_t gpu, stream;        /* -1, -1: no portion found                            */
    int64_t start_us, end_us;   /* the portion given to the instance                   */
    int64_t duty_cycle_us;      /* duty cycle of the stream (<= the instance's own)    */
} octo_coral_placement_t;

/* out[i] receives the placement of inst[i].  Errors: OCTO_E_INVALID_ARG (null pointers, negative
 * sizes, a window outside its duty cycle, n_gpus < 1, num_streams out of range). */
OCTO_API int octo_coral_schedule(const octo_coral_instance_t* inst, int32_t n_inst, const octo_coral_gpu_t* gpus,
                                 int32_t n_gpus, octo_coral_placement_t* out);

/* Text of a status code; never NULL. */
OCTO_API const char* octo_strerror(int code);

/* Text of the last CUDA error a call on this thread reported as OCTO_E_CUDA. */
OCTO_API const char* octo_last_cuda_error(void);

/* Library version, "major.minor". */
OCTO_API const char* octo_version(void);

#ifdef __cplusplus
}
#endif
#endif /* OCTO_H_ */
