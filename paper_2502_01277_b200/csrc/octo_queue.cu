// Device-side dynamic-batch queue of one downstream branch (see include/octo.h).
//
// A ring of self-contained item records lives in device memory together with its head / tail
// counters, so pushes and pops are plain kernels on the caller's stream and never synchronise
// with the host.  push_kernel (one CTA) runs the batch assembler of a stage's branch (scan of
// the per-frame counts, item -> detection -> rectangle) and appends the records; pop_kernel
// (one CTA) moves the oldest records into a linear staging array, which the queue mode of the
// crop kernel then resamples into the downstream batch.
#include <new>

#include "octo.h"
#include "octo_kernels.h"
#include "octo_stage_internal.h"

using namespace octo;

namespace octo {

struct QueueState {
    long long head, tail;  // monotonic item counters; pending = tail - head
    long long dropped;
    int seq;               // pushes so far
    unsigned int status;
    int sched[2];          // tile scheduler words of the crop kernel (zero between launches)
};

constexpr int kQueueThreads = 1024;

template <int CAP>
__global__ void __launch_bounds__(kQueueThreads)
queue_push_kernel(const __grid_constant__ FrameTable<CAP> tab, const FrameDesc* __restrict__ gtab, int n, int max_det,
                  const int* __restrict__ bcount,
                  const int* __restrict__ bidx, const octo_det_t* __restrict__ dets, QRecord* __restrict__ ring,
                  int cap, QueueState* __restrict__ state) {
    __shared__ int s_off[CAP + 1];
    pdl_enter(0);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (warp == 0) {
        int run = 0;
        for (int base = 0; base < n; base += 32) {
            const int i = base + lane;
            const int v = i < n ? bcount[i] : 0;
            int inc = v;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const int t = __shfl_up_sync(0xffffffffu, inc, off);
                if (lane >= off) inc += t;
            }
            if (i < n) s_off[i] = run + inc - v;
            run += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (lane == 0) s_off[n] = run;
    }
    __syncthreads();
    const int total = s_off[n];
    const long long head = state->head, tail = state->tail;
    const int seq = state->seq;
    const long long room = (long long)cap - (tail - head);
    const int accepted = (int)(total < room ? total : (room < 0 ? 0 : room));
    for (int item = threadIdx.x; item < accepted; item += kQueueThreads) {
        int lo = 0, hi = n;  // largest f with s_off[f] <= item
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (s_off[mid] <= item) lo = mid; else hi = mid;
        }
        const int f = lo;
        const int det = bidx[(size_t)f * max_det + (item - s_off[f])];
        const octo_det_t d = dets[(size_t)f * max_det + det];
        const FrameDesc fd = gtab ? gtab[f] : tab.f[f];
        // outward-rounded rectangle, clamped so that it is never empty
        int rx0 = (int)floorf(d.x1), ry0 = (int)floorf(d.y1);
        int rx1 = (int)ceilf(d.x2), ry1 = (int)ceilf(d.y2);
        rx0 = min(max(rx0, 0), fd.w - 1);
        ry0 = min(max(ry0, 0), fd.h - 1);
        rx1 = min(max(rx1, rx0 + 1), fd.w);
        ry1 = min(max(ry1, ry0 + 1), fd.h);
        QRecord rec;
        rec.data = fd.data; rec.w = fd.w; rec.h = fd.h; rec.pitch = fd.pitch;
        rec.rx0 = rx0; rec.ry0 = ry0; rec.rx1 = rx1; rec.ry1 = ry1;
        rec.seq = seq; rec.frame = f; rec.det = det;
        ring[(tail + item) % cap] = rec;
    }
    __syncthreads();  // every thread has read head / tail / seq
    if (threadIdx.x == 0) {
        state->tail = tail + accepted;
        state->dropped += total - accepted;
        state->seq = seq + 1;
    }
}

__global__ void __launch_bounds__(256)
queue_pop_kernel(const QRecord* __restrict__ ring, int cap, QueueState* __restrict__ state, int bz, int max_wait,
                 QRecord* __restrict__ staged, QRecord* __restrict__ items_out, int* __restrict__ info,
                 int* __restrict__ qpacked) {
    pdl_enter(0);
    const long long head = state->head, tail = state->tail;
    const long long pending = tail - head;
    // max_wait < 0: release whatever is pending.  Otherwise a batch is released when it is full, or
    // when its first item has waited for max_wait pushes (the item queued by push s has waited
    // seq - 1 - s pushes once `seq` pushes have been made).
    bool due = true;
    if (max_wait >= 0 && pending < bz)
        due = pending > 0 && (state->seq - 1 - ring[head % cap].seq) >= max_wait;
    const int popped = due ? (int)(pending < bz ? pending : bz) : 0;
    for (int i = threadIdx.x; i < popped; i += blockDim.x) {
        const QRecord rec = ring[(head + i) % cap];
        staged[i] = rec;
        if (items_out) items_out[i] = rec;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const long long left = pending - popped;
        info[0] = popped;
        info[1] = (int)left;
        info[2] = (int)(state->dropped > 0x7fffffffLL ? 0x7fffffffLL : state->dropped);
        info[3] = left > 0 ? ring[(head + popped) % cap].seq : -1;
        *qpacked = popped;
        state->head = head + popped;
    }
}

template <int CAP>
static cudaError_t push_cap(const octo_stage* st, int branch, QRecord* ring, int cap, QueueState* state,
                            cudaStream_t stream) {
    FrameTable<CAP> tab;  // built per call (copied into kernel parameter space by the launch)
    if (!st->tab_on_device)
        for (int i = 0; i < st->n_frames; ++i) tab.f[i] = st->frames[i];
    const octo_stage_config_t& c = st->cfg;
    queue_push_kernel<CAP><<<1, kQueueThreads, 0, stream>>>(
        tab, st->tab_on_device ? st->d_tab : nullptr, st->n_frames, c.max_det, st->d_bcount + (size_t)branch * c.max_batch,
        st->d_bidx + (size_t)branch * c.max_batch * c.max_det, st->d_dets, ring, cap, state);
    return cudaGetLastError();
}

}  // namespace octo

struct octo_queue {
    int device, capacity, out_w, out_h, swap_rb, max_bz, sm_count;
    QRecord* d_ring;
    QRecord* d_staged;
    QueueState* d_state;
    int* d_qpacked;
    bool general;   // crop options set (octo_queue_set_options)
    CropOpts opts;
};

static void queue_free(octo_queue* q) {
    cudaFree(q->d_ring);
    cudaFree(q->d_staged);
    cudaFree(q->d_state);
    cudaFree(q->d_qpacked);
}

extern "C" int octo_queue_create(int32_t device, int32_t capacity, int32_t out_w, int32_t out_h, int32_t swap_rb,
                                 int32_t max_bz, octo_queue_t** out) {
    if (!out) return OCTO_E_INVALID_ARG;
    *out = nullptr;
    if (device < 0 || capacity < 1 || capacity > (1 << 24) || max_bz < 1 || max_bz > capacity)
        return OCTO_E_INVALID_ARG;
    if (out_w < 8 || out_w > 2048 || (out_w & 7) || out_h < 1 || out_h > 2048) return OCTO_E_INVALID_ARG;
    if (swap_rb != 0 && swap_rb != 1) return OCTO_E_INVALID_ARG;
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || device >= ndev) return ndev ? OCTO_E_INVALID_ARG : OCTO_E_CUDA;
    if (cudaSetDevice(device) != cudaSuccess) return OCTO_E_CUDA;
    octo_queue* q = new (std::nothrow) octo_queue();
    if (!q) return OCTO_E_INVALID_ARG;
    *q = octo_queue();
    q->device = device; q->capacity = capacity; q->out_w = out_w; q->out_h = out_h;
    q->swap_rb = swap_rb; q->max_bz = max_bz;
    cudaError_t e = cudaDeviceGetAttribute(&q->sm_count, cudaDevAttrMultiProcessorCount, device);
    if (e == cudaSuccess) e = cudaMalloc(&q->d_ring, sizeof(QRecord) * (size_t)capacity);
    if (e == cudaSuccess) e = cudaMalloc(&q->d_staged, sizeof(QRecord) * (size_t)max_bz);
    if (e == cudaSuccess) e = cudaMalloc(&q->d_state, sizeof(QueueState));
    if (e == cudaSuccess) e = cudaMalloc(&q->d_qpacked, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(q->d_state, 0, sizeof(QueueState));
    if (e == cudaSuccess) e = cudaMemset(q->d_qpacked, 0, sizeof(int));
    if (e == cudaSuccess) e = prepare_crop();
    if (e != cudaSuccess) {
        queue_free(q);
        delete q;
        return OCTO_E_CUDA;
    }
    *out = q;
    return OCTO_OK;
}

extern "C" int octo_queue_set_options(octo_queue_t* q, const octo_branch_cfg_t* options, int32_t pad_value) {
    if (!q || !options || pad_value < 0 || pad_value > 255) return OCTO_E_INVALID_ARG;
    if (validate_branch_options(*options) != OCTO_OK) return OCTO_E_INVALID_ARG;
    q->general = options->keep_aspect != 0 || options->normalize != 0;
    fill_crop_opts(*options, q->swap_rb, pad_value, &q->opts);
    return OCTO_OK;
}

extern "C" int octo_queue_destroy(octo_queue_t* q) {
    if (!q) return OCTO_E_INVALID_ARG;
    cudaSetDevice(q->device);
    queue_free(q);
    delete q;
    return OCTO_OK;
}

extern "C" int octo_queue_push(octo_queue_t* q, octo_stage_t* st, int32_t branch, void* cuda_stream) {
    if (!q || !st) return OCTO_E_INVALID_ARG;
    if (branch < 0 || branch >= st->cfg.num_branches || st->cfg.device != q->device) return OCTO_E_INVALID_ARG;
    if (st->n_frames < 1) return OCTO_E_NO_PREPROCESS;
    if (!st->have_dets) return OCTO_E_NO_POSTPROCESS;
    if (cudaSetDevice(q->device) != cudaSuccess) return OCTO_E_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e;
    if (st->n_frames <= 8) e = push_cap<8>(st, branch, q->d_ring, q->capacity, q->d_state, stream);
    else if (st->n_frames <= 64) e = push_cap<64>(st, branch, q->d_ring, q->capacity, q->d_state, stream);
    else e = push_cap<512>(st, branch, q->d_ring, q->capacity, q->d_state, stream);
    return e == cudaSuccess ? OCTO_OK : OCTO_E_CUDA;
}

extern "C" int octo_queue_pop(octo_queue_t* q, int32_t bz, void* d_out_f16, octo_qitem_t* d_items_out,
                              int32_t* d_info, void* cuda_stream) {
    return octo_queue_pop_due(q, bz, -1, d_out_f16, d_items_out, d_info, cuda_stream);
}

extern "C" int octo_queue_pop_due(octo_queue_t* q, int32_t bz, int32_t max_wait, void* d_out_f16,
                                  octo_qitem_t* d_items_out, int32_t* d_info, void* cuda_stream) {
    if (!q || !d_out_f16 || !d_info || bz < 1 || bz > q->max_bz) return OCTO_E_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(d_out_f16) & 15) || (reinterpret_cast<uintptr_t>(d_info) & 3) ||
        (reinterpret_cast<uintptr_t>(d_items_out) & 7))
        return OCTO_E_ALIGNMENT;
    if (cudaSetDevice(q->device) != cudaSuccess) return OCTO_E_CUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    static_assert(sizeof(octo_qitem_t) == sizeof(QRecord), "public and internal queue records match");
    queue_pop_kernel<<<1, 256, 0, stream>>>(q->d_ring, q->capacity, q->d_state, bz, max_wait, q->d_staged,
                                           reinterpret_cast<QRecord*>(d_items_out), d_info, q->d_qpacked);
    if (cudaGetLastError() != cudaSuccess) return OCTO_E_CUDA;
    cudaError_t e = launch_crop_queue(q->d_staged, q->d_qpacked, bz, d_out_f16, q->out_w, q->out_h, q->swap_rb,
                                      q->sm_count, &q->d_state->status, q->d_state->sched, q->general ? &q->opts : nullptr, stream);
    return e == cudaSuccess ? OCTO_OK : OCTO_E_CUDA;
}
