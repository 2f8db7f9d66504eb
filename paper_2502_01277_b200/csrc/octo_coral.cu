// Spatiotemporal placement of model instances on GPU inference streams (host code only).
//
// The paper's co-location scheduler (Section III-C, Algorithm 2) divides a GPU into concurrently
// running streams; an execution occupies a portion of a stream (its length is the execution time,
// its width the share of the GPU's compute it needs), and a stream repeats with a duty cycle.
// Instances are taken one replica number at a time over all pipelines and their models (so that
// every pipeline gets its first instance before any gets a second), and each goes to the
// best-fitting free portion that (1) contains the window the instance needs, (2) leaves the GPU
// within its memory and utilisation limits and (3) belongs to a stream whose duty cycle is not
// longer than the pipeline's.  The chosen portion is split and what is left goes back to the
// free list.
//
// Readings where the paper is silent: the free list is kept ordered by length (then GPU, stream,
// start), so the first feasible portion is the one with the least empty space; a stream without a
// duty cycle offers one unbounded portion, which is cut to the duty cycle once the first instance
// fixes it; all times are integer microseconds.
#include <algorithm>
#include <cstdint>
#include <vector>

#include "octo.h"

namespace {

constexpr int64_t kForever = INT64_MAX;

struct Portion {
    int32_t gpu, stream;
    int64_t start, end;
    int64_t length() const { return end == kForever ? kForever : end - start; }
};

bool portion_less(const Portion& a, const Portion& b) {
    if (a.length() != b.length()) return a.length() < b.length();
    if (a.gpu != b.gpu) return a.gpu < b.gpu;
    if (a.stream != b.stream) return a.stream < b.stream;
    return a.start < b.start;
}

struct StreamState {
    int64_t duty_cycle = 0;  // 0: not fixed yet
    int64_t inter = 0;       // I_s: largest intermediate memory of its residents
    int32_t util = 0;        // widest resident
};

struct GpuState {
    int64_t weights = 0;  // W_g
    int64_t inter = 0;    // I_g = sum of I_s
    std::vector<StreamState> streams;
};

}  // namespace

extern "C" int octo_coral_schedule(const octo_coral_instance_t* inst, int32_t n_inst, const octo_coral_gpu_t* gpus,
                                   int32_t n_gpus, octo_coral_placement_t* out) {
    if (!inst || !gpus || !out || n_inst < 0 || n_gpus < 1) return OCTO_E_INVALID_ARG;
    for (int32_t g = 0; g < n_gpus; ++g)
        if (gpus[g].num_streams < 1 || gpus[g].num_streams > 1024 || gpus[g].mem_bytes < 0 ||
            gpus[g].util_max_permille < 0)
            return OCTO_E_INVALID_ARG;
    for (int32_t i = 0; i < n_inst; ++i) {
        const octo_coral_instance_t& r = inst[i];
        if (r.start_us < 0 || r.end_us <= r.start_us || r.duty_cycle_us < r.end_us || r.weight_bytes < 0 ||
            r.inter_bytes < 0 || r.util_permille < 0 || r.pipeline < 0 || r.model < 0 || r.instance < 0)
            return OCTO_E_INVALID_ARG;
    }

    std::vector<GpuState> state((size_t)n_gpus);
    std::vector<Portion> free_list;
    for (int32_t g = 0; g < n_gpus; ++g) {
        state[(size_t)g].streams.resize((size_t)gpus[g].num_streams);
        for (int32_t s = 0; s < gpus[g].num_streams; ++s) free_list.push_back(Portion{g, s, 0, kForever});
    }
    std::sort(free_list.begin(), free_list.end(), portion_less);

    // one replica number at a time, pipelines in order, models in their pipeline's order
    std::vector<int32_t> order((size_t)n_inst);
    for (int32_t i = 0; i < n_inst; ++i) order[(size_t)i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
        if (inst[a].instance != inst[b].instance) return inst[a].instance < inst[b].instance;
        if (inst[a].pipeline != inst[b].pipeline) return inst[a].pipeline < inst[b].pipeline;
        return inst[a].model < inst[b].model;
    });

    for (int32_t idx : order) {
        const octo_coral_instance_t& r = inst[idx];
        octo_coral_placement_t& place = out[idx];
        place.gpu = -1; place.stream = -1; place.start_us = 0; place.end_us = 0; place.duty_cycle_us = 0;
        for (size_t k = 0; k < free_list.size(); ++k) {
            const Portion pt = free_list[k];
            GpuState& g = state[(size_t)pt.gpu];
            StreamState& s = g.streams[(size_t)pt.stream];
            // (1) the stream is free for the whole window
            if (!(pt.start <= r.start_us && pt.end >= r.end_us)) continue;
            // (2) memory and compute of the GPU with the instance on this stream
            const int64_t w_g = g.weights + r.weight_bytes;
            const int64_t i_g = g.inter - s.inter + std::max(s.inter, r.inter_bytes);
            int64_t u_g = 0;
            for (size_t q = 0; q < g.streams.size(); ++q)
                u_g += (&g.streams[q] == &s) ? std::max(s.util, r.util_permille) : g.streams[q].util;
            if (w_g + i_g > gpus[pt.gpu].mem_bytes || u_g > gpus[pt.gpu].util_max_permille) continue;
            // (3) the instance may not stretch the stream's duty cycle
            if (!(r.duty_cycle_us >= s.duty_cycle)) continue;

            free_list.erase(free_list.begin() + (long)k);
            if (s.duty_cycle == 0) {
                s.duty_cycle = r.duty_cycle_us;
                // the stream's unbounded portions now end with its duty cycle
                for (Portion& f : free_list)
                    if (f.gpu == pt.gpu && f.stream == pt.stream && f.end == kForever) f.end = s.duty_cycle;
            }
            const int64_t pt_end = pt.end == kForever ? s.duty_cycle : pt.end;
            place.gpu = pt.gpu; place.stream = pt.stream;
            place.start_us = r.start_us; place.end_us = r.end_us;
            place.duty_cycle_us = s.duty_cycle;
            g.weights = w_g;
            g.inter = i_g;
            s.inter = std::max(s.inter, r.inter_bytes);
            s.util = std::max(s.util, r.util_permille);
            // what the instance does not use goes back to the list
            if (pt.start < r.start_us) free_list.push_back(Portion{pt.gpu, pt.stream, pt.start, r.start_us});
            if (r.end_us < pt_end) free_list.push_back(Portion{pt.gpu, pt.stream, r.end_us, pt_end});
            std::sort(free_list.begin(), free_list.end(), portion_less);
            break;
        }
    }
    return OCTO_OK;
}
