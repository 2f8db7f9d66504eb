// Placement of model instances on GPU inference streams in space and time (host code only; the
// paper's co-location scheduler, Section III-C, Algorithm 2).
//
// What is computed.  A GPU is divided into concurrently running streams; an execution occupies a
// window of one stream's duty cycle and a share of the GPU's compute; a stream repeats with a duty
// cycle.  Instances are placed one replica number at a time over all pipelines and their models.
// Each goes to the stream whose free gap around the instance's window is the tightest, among the
// streams where (1) the window is free, (2) the GPU stays within its memory (weights + per stream
// the largest intermediate memory of its residents) and its utilisation limit (per stream the
// widest resident) and (3) the stream's duty cycle is not longer than the instance's.  Ties go
// to the lower GPU, then the lower stream.  The first resident of a stream fixes its duty cycle;
// a stream without one counts as an unbounded gap, so it is taken only when no bounded gap fits.
//
// How.  Every stream keeps its busy windows in an ordered map (start -> end), so the free gap
// around a window is found from the window's two neighbours in O(log residents); a window lies in
// at most one gap of a stream, hence comparing one candidate per stream finds the tightest gap
// overall.  A GPU's totals (weights, sum of the streams' intermediate maxima, sum of the streams'
// widths) are kept up to date, so the limits are tested in O(1) per candidate.
#include <algorithm>
#include <cstdint>
#include <iterator>
#include <map>
#include <numeric>
#include <vector>

#include "octo.h"

namespace {

constexpr int64_t kUnbounded = INT64_MAX;

class Stream {
  public:
    int64_t duty_cycle() const { return duty_; }
    int64_t inter() const { return inter_; }
    int32_t width() const { return width_; }

    // Free gap [lo, hi) around the window [a, b), or false if the window touches a busy one.
    bool gap_around(int64_t a, int64_t b, int64_t* lo, int64_t* hi) const {
        auto next = busy_.lower_bound(a);  // first busy window starting at or after a
        if (next != busy_.end() && next->first < b) return false;
        *hi = next != busy_.end() ? next->first : (duty_ ? duty_ : kUnbounded);
        *lo = 0;
        if (next != busy_.begin()) {
            auto prev = std::prev(next);
            if (prev->second > a) return false;
            *lo = prev->second;
        }
        return *hi == kUnbounded || b <= *hi;
    }

    void occupy(const octo_coral_instance_t& r) {
        if (!duty_) duty_ = r.duty_cycle_us;
        busy_.emplace(r.start_us, r.end_us);
        inter_ = std::max(inter_, r.inter_bytes);
        width_ = std::max(width_, r.util_permille);
    }

  private:
    std::map<int64_t, int64_t> busy_;
    int64_t duty_ = 0;  // 0: not fixed yet
    int64_t inter_ = 0;
    int32_t width_ = 0;
};

struct Gpu {
    std::vector<Stream> streams;
    int64_t weights = 0, inter_sum = 0;
    int32_t width_sum = 0;
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

    std::vector<Gpu> state((size_t)n_gpus);
    for (int32_t g = 0; g < n_gpus; ++g) state[(size_t)g].streams.resize((size_t)gpus[g].num_streams);

    // one replica number at a time, pipelines in order, models in their pipeline's order
    std::vector<int32_t> order((size_t)n_inst);
    std::iota(order.begin(), order.end(), 0);
    std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) {
        if (inst[a].instance != inst[b].instance) return inst[a].instance < inst[b].instance;
        if (inst[a].pipeline != inst[b].pipeline) return inst[a].pipeline < inst[b].pipeline;
        return inst[a].model < inst[b].model;
    });

    for (int32_t idx : order) {
        const octo_coral_instance_t& r = inst[idx];
        int32_t best_g = -1, best_s = -1;
        int64_t best_len = 0;
        for (int32_t g = 0; g < n_gpus; ++g) {
            const Gpu& gs = state[(size_t)g];
            for (int32_t s = 0; s < (int32_t)gs.streams.size(); ++s) {
                const Stream& st = gs.streams[(size_t)s];
                if (st.duty_cycle() > r.duty_cycle_us) continue;  // the instance may not stretch the cycle
                int64_t lo, hi;
                if (!st.gap_around(r.start_us, r.end_us, &lo, &hi)) continue;
                const int64_t mem = gs.weights + r.weight_bytes + gs.inter_sum - st.inter() + std::max(st.inter(), r.inter_bytes);
                const int64_t width = (int64_t)gs.width_sum - st.width() + std::max(st.width(), r.util_permille);
                if (mem > gpus[g].mem_bytes || width > gpus[g].util_max_permille) continue;
                const int64_t len = hi == kUnbounded ? kUnbounded : hi - lo;
                if (best_g < 0 || len < best_len) { best_g = g; best_s = s; best_len = len; }
            }
        }
        octo_coral_placement_t& place = out[idx];
        place.gpu = best_g; place.stream = best_s;
        place.start_us = 0; place.end_us = 0; place.duty_cycle_us = 0;
        if (best_g < 0) continue;
        Gpu& gs = state[(size_t)best_g];
        Stream& st = gs.streams[(size_t)best_s];
        gs.weights += r.weight_bytes;
        gs.inter_sum += std::max(st.inter(), r.inter_bytes) - st.inter();
        gs.width_sum += std::max(st.width(), r.util_permille) - st.width();
        st.occupy(r);
        place.start_us = r.start_us; place.end_us = r.end_us;
        place.duty_cycle_us = st.duty_cycle();
    }
    return OCTO_OK;
}
