// Shared device-side definitions of the cascade-stage kernels (sm_100a).
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace octo {

// One frame of the current batch plus its letterbox geometry (computed on the host in exact
// integer arithmetic).  Passed to kernels BY VALUE inside a FrameTable (kernel parameter
// space), so no host->device table copy sits on the critical path of a batch.
struct FrameDesc {
    const uint8_t* data;
    int32_t w, h, pitch;
    int32_t nw, nh, pad_l, pad_t;
    float gx, gy;  // fl(region width / nw), fl(region height / nh): scale-back gains
    // Region of the source frame that the detector input shows: the whole frame for a
    // first-level stage, the upstream crop rectangle for a chained stage.  Boxes are mapped
    // back into it and clamped to it.
    uint16_t ox, oy, rw, rh;
};
static_assert(sizeof(FrameDesc) == 56, "FrameDesc layout");

template <int CAP>
struct FrameTable {
    FrameDesc f[CAP];
};

// One queued item of a device-side dynamic-batch queue: everything needed to crop it later,
// independent of the stage batch it came from.
struct QRecord {
    const uint8_t* data;  // source frame
    int32_t w, h, pitch;
    int32_t rx0, ry0, rx1, ry1;
    int32_t seq;          // number of the push that queued it
    int32_t frame, det;   // position in that push's batch
};
static_assert(sizeof(QRecord) == 48, "QRecord layout");


// Device counters of a stage (one allocation, zeroed at creation).
struct StageCounters {
    unsigned long long candidates;
    unsigned long long kept;
    unsigned int status;
    int max_cand;
    int packed;
    int total_items;
    int sched[2];  // crop kernel: tiles handed out beyond each CTA's first, CTAs finished (both zero between launches)
};

// Range checks of the checked build (-DOCTO_BOUNDS_CHECK): an index outside its range sets the
// OCTO_STATUS_BOUNDS bit of the status word and the access is skipped; nothing traps.  In the
// normal build the condition is not evaluated.  Use as  if (OCTO_IN_RANGE(i < n, status)) a[i] = v;
#ifdef OCTO_BOUNDS_CHECK
#define OCTO_IN_RANGE(cond, status_ptr) ((cond) ? true : (atomicOr((status_ptr), 0x20u), false))
#else
#define OCTO_IN_RANGE(cond, status_ptr) (true)
#endif

// Programmatic dependent launch.  Every kernel of the library starts with pdl_enter: it waits
// until the kernel before it in the stream has completed and its writes are visible (a no-op
// for a launch without the programmatic attribute); with `early` set it then lets the next
// kernel of the stream be scheduled right away, where that kernel waits at its own pdl_enter.
// The hosts sets `early` (and the launch attribute) for small batches only: there the launch
// latency between the kernels of a pass is most of the pass, while a large grid loses more to
// the waiting CTAs of its successor than it gains.
__device__ __forceinline__ void pdl_enter(int early) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (early) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

constexpr int kKeyAnchorBits = 25;  // anchor index field of a candidate key
constexpr unsigned long long kKeySentinel = ~0ull;

// ---------------------------------------------------------------------------------------
// Exact source coordinate of destination index d when `src` samples are resized to `dst`
// (half-pixel centres): s = ((2d + 1) * src - dst) / (2 * dst), clamped to [0, src - 1].
// Returns i0 = floor(s) and the remainder r in [0, 2*dst) with frac = r / (2*dst); r == 0
// when clamped.  The quotient comes from a float estimate corrected in integers, which is
// exact for every value that fits 31 bits.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ void src_coord(int d, int src, int dst, float inv_den, int& i0, int& rem) {
    const int den = 2 * dst;
    int num = (2 * d + 1) * src - dst;
    if (num <= 0) { i0 = 0; rem = 0; return; }
    int q = __float2int_rz(__int2float_rn(num) * inv_den);
    int r = num - q * den;
    if (r < 0) { q -= 1; r += den; }
    else if (r >= den) { q += 1; r -= den; }
    if (q >= src - 1) { i0 = src - 1; rem = 0; return; }
    i0 = q; rem = r;
}

// ---------------------------------------------------------------------------------------
// Table-driven horizontal sampling.  For every destination column a kernel precomputes, once
// per tile, the byte offset of the left tap inside the staged source row and the two integer
// weights (den - rem, rem) with den = 2 * dst <= 65535, packed as two 16-bit halves.  The
// horizontal lerp of one colour channel is then a single two-way dot product of those
// weights with the two tap bytes (exact in integers); the result carries a factor `den`.
// ---------------------------------------------------------------------------------------
struct XEntry {
    uint32_t off;  // byte offset of pixel x0 in the staged row
    uint32_t wts;  // (den - rem) | rem << 16
};

__device__ __forceinline__ XEntry make_xentry(int d, int src, int dst, float inv_den, int byte_base) {
    int x0, rem;
    src_coord(d, src, dst, inv_den, x0, rem);
    XEntry e;
    e.off = (uint32_t)(byte_base + 3 * x0);
    e.wts = (uint32_t)(2 * dst - rem) | ((uint32_t)rem << 16);
    return e;
}

// Shared-memory loads through 32-bit shared-space addresses (no 64-bit generic pointer
// arithmetic in the inner loops).
__device__ __forceinline__ void lds32x3(uint32_t addr, uint32_t& a, uint32_t& b, uint32_t& c) {
    asm volatile("ld.shared.u32 %0, [%3];\n\tld.shared.u32 %1, [%3+4];\n\tld.shared.u32 %2, [%3+8];"
                 : "=r"(a), "=r"(b), "=r"(c)
                 : "r"(addr));
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
    return v;
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// Integer horizontal lerp of the three channels of one destination pixel.  `addr` is the
// shared-space address of the 4-byte aligned word that holds the left tap's first byte (the
// staged rows keep at least 12 readable bytes past any tap); only the low five bits of `sh`
// = 8 * byte offset matter (the funnel shift wraps).  The sums start from kF32Int, the bit
// pattern of 2^23: a sum v < 2^23 (255 * den with den <= 8192) then IS the binary32 number
// 2^23 + v, so no integer-to-float conversion is needed afterwards.
constexpr uint32_t kF32Int = 0x4B000000u;
constexpr float kF32IntValue = 8388608.0f;
__device__ __forceinline__ void hsample(uint32_t addr, uint32_t sh, uint32_t wts, float& c0, float& c1, float& c2) {
    uint32_t a, b, c;
    lds32x3(addr, a, b, c);
    const uint32_t lo = __funnelshift_r(a, b, sh);  // B0 G0 R0 B1
    const uint32_t hi = __funnelshift_r(b, c, sh);  // G1 R1 .. ..
    const uint32_t p01 = __byte_perm(lo, hi, 0x4130);  // B0 B1 G0 G1
    const uint32_t p2 = __byte_perm(lo, hi, 0x5252);   // R0 R1 R0 R1
    c0 = __uint_as_float(__dp2a_lo(wts, p01, kF32Int));
    c1 = __uint_as_float(__dp2a_hi(wts, p01, kF32Int));
    c2 = __uint_as_float(__dp2a_lo(wts, p2, kF32Int));
}

// One destination pixel: horizontal integer lerp on one or two staged rows (shared-space
// addresses row0, row0 + row_step), then the vertical lerp and all scaling in fp32 (wx / wy
// carry 1 / (255 * den_x * den_y); nwx = -2^23 * wx).  With h = 2^23 + v from hsample,
// fma(h, wx, nwx) rounds the exact product v * wx once, and h - 2^23 is exact, so the result
// is fl(fl(v0 * wx) + v1 * wy) bit for bit.
template <bool LERP_Y>
__device__ __forceinline__ void sample_px(uint32_t row0, uint32_t row_step, const uint32_t off, const uint32_t wts,
                                          float wx, float nwx, float wy, float& f0, float& f1, float& f2) {
    const uint32_t addr = row0 + (off & ~3u), sh = off << 3;
    float a0, a1, a2;
    hsample(addr, sh, wts, a0, a1, a2);
    f0 = __fmaf_rn(a0, wx, nwx);
    f1 = __fmaf_rn(a1, wx, nwx);
    f2 = __fmaf_rn(a2, wx, nwx);
    if (LERP_Y) {
        float b0, b1, b2;
        hsample(addr + row_step, sh, wts, b0, b1, b2);
        f0 = __fmaf_rn(__fsub_rn(b0, kF32IntValue), wy, f0);
        f1 = __fmaf_rn(__fsub_rn(b1, kF32IntValue), wy, f1);
        f2 = __fmaf_rn(__fsub_rn(b2, kF32IntValue), wy, f2);
    }
}

// Packed binary32 arithmetic (two independent IEEE operations per instruction, sm_100): the
// two pixels of a pair go through the vertical lerp together.
__device__ __forceinline__ unsigned long long f32x2(float lo, float hi) {
    unsigned long long v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
    unsigned long long d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
__device__ __forceinline__ unsigned long long mul_f32x2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ unsigned long long add_f32x2(unsigned long long a, unsigned long long b) {
    unsigned long long d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// binary16 pair from a packed binary32 pair (low element in the low half)
__device__ __forceinline__ uint32_t half2_of_f32x2(unsigned long long v) {
    float lo, hi;
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    __half2 h = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&h);
}

// Two neighbouring destination pixels (table entries ea, eb) of one output row: the integer
// horizontal lerps as in sample_px, then the vertical lerp and scaling of both pixels in packed
// arithmetic.  p0 / p1 / p2 receive (pixel a, pixel b) of the three input channels; every
// element goes through the same individually rounded operations as in sample_px.
template <bool LERP_Y>
__device__ __forceinline__ void sample_pair(uint32_t row0, uint32_t row_step, uint32_t offa, uint32_t wtsa,
                                            uint32_t offb, uint32_t wtsb, float wx, float nwx, float wy,
                                            unsigned long long& p0, unsigned long long& p1, unsigned long long& p2) {
    const uint32_t addra = row0 + (offa & ~3u), sha = offa << 3;
    const uint32_t addrb = row0 + (offb & ~3u), shb = offb << 3;
    float a0, a1, a2, b0, b1, b2;
    hsample(addra, sha, wtsa, a0, a1, a2);
    hsample(addrb, shb, wtsb, b0, b1, b2);
    const unsigned long long wx2 = f32x2(wx, wx), nwx2 = f32x2(nwx, nwx);
    p0 = fma_f32x2(f32x2(a0, b0), wx2, nwx2);
    p1 = fma_f32x2(f32x2(a1, b1), wx2, nwx2);
    p2 = fma_f32x2(f32x2(a2, b2), wx2, nwx2);
    if (LERP_Y) {
        hsample(addra + row_step, sha, wtsa, a0, a1, a2);
        hsample(addrb + row_step, shb, wtsb, b0, b1, b2);
        const unsigned long long wy2 = f32x2(wy, wy), m2 = f32x2(-kF32IntValue, -kF32IntValue);
        p0 = fma_f32x2(add_f32x2(f32x2(a0, b0), m2), wy2, p0);
        p1 = fma_f32x2(add_f32x2(f32x2(a1, b1), m2), wy2, p1);
        p2 = fma_f32x2(add_f32x2(f32x2(a2, b2), m2), wy2, p2);
    }
}

__device__ __forceinline__ uint32_t pack_half2(float a, float b) {
    __half2 h = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}

// One output row (or column tile of it) by one warp: lane l owns the pixel pairs l, l + 32, ...
// so neighbouring lanes read neighbouring table entries and row words (no bank conflicts)
// and the warp writes 128 contiguous bytes per plane and step.  row0 / xt are shared-space
// addresses of the first staged row and of the tile's first table entry; o0 / o1 / o2 point
// at the row's first pixel in the planes of input channels 0 / 1 / 2.  With FILL, columns
// whose table entry has zero weights (canvas outside the image) receive the binary16 fill value
// (fill_h2 holds it in both halves).
template <bool LERP_Y, bool FILL>
__device__ __forceinline__ void sample_row(uint32_t row0, uint32_t row_step, float wx, float wy, uint32_t xt,
                                           int pairs, int lane, __half* __restrict__ o0, __half* __restrict__ o1,
                                           __half* __restrict__ o2, uint32_t fill_h2) {
    const float nwx = -kF32IntValue * wx;
    for (int pair = lane; pair < pairs; pair += 32) {
        const uint4 ee = lds128(xt + 16u * (uint32_t)pair);  // two XEntry: {off, wts} x 2
        unsigned long long p0, p1, p2;
        sample_pair<LERP_Y>(row0, row_step, ee.x, ee.y, ee.z, ee.w, wx, nwx, wy, p0, p1, p2);
        uint32_t h0 = half2_of_f32x2(p0), h1 = half2_of_f32x2(p1), h2 = half2_of_f32x2(p2);
        if (FILL) {
            // canvas columns: replace the half of the pair that lies outside the image
            const uint32_t keep = (ee.y == 0u ? 0u : 0x0000ffffu) | (ee.w == 0u ? 0u : 0xffff0000u);
            const uint32_t fill = fill_h2 & ~keep;
            h0 = (h0 & keep) | fill;
            h1 = (h1 & keep) | fill;
            h2 = (h2 & keep) | fill;
        }
        const uint32_t o = 2u * (uint32_t)pair;
        *reinterpret_cast<uint32_t*>(o0 + o) = h0;
        *reinterpret_cast<uint32_t*>(o1 + o) = h1;
        *reinterpret_cast<uint32_t*>(o2 + o) = h2;
    }
}

// What a warp needs to know about one output row of a staged pass.
struct RowInfo {
    int32_t row0;  // byte offset of the first staged row relative to the row buffer
    int32_t step;  // distance to the second staged row (unused when wy == 0); < 0: canvas row
    float wx, wy;  // vertical weights with all scaling folded in
};


// ---------------------------------------------------------------------------------------
// mbarrier + bulk-copy (TMA engine, untiled) helpers.  Every wait is bounded.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One poll of the barrier's phase; the thread may be suspended by the hardware for up to about
// `hint_ns` nanoseconds while the phase is incomplete, so a waiting warp does not burn issue slots.
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity, uint32_t hint_ns = 2000u) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
        : "memory");
    return ok != 0;
}
// Returns false if the phase did not complete within the iteration limit.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, int limit = 1 << 20) {
    for (int i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// The same for a warp that expects to wait long (a producer waiting for its consumers): plain
// phase tests with a sleep in between, so that the waiting warp takes almost no issue slots
// from the working warps of its scheduler.
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_sleeping(uint64_t* bar, uint32_t parity, unsigned sleep_ns,
                                                   int limit = 1 << 20) {
    for (int i = 0; i < limit; ++i) {
        if (mbar_test_wait(bar, parity)) return true;
        __nanosleep(sleep_ns);
    }
    return false;
}
// Global -> shared bulk copy; both addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(dst_smem)),
        "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}

// ---------------------------------------------------------------------------------------
// Fixed binary32 arithmetic shared by decode and NMS.  Every operation is an explicitly
// rounded intrinsic so that compiler contraction cannot change a bit.
// ---------------------------------------------------------------------------------------
__device__ __forceinline__ bool finite_f(float v) { return (__float_as_uint(v) & 0x7f800000u) != 0x7f800000u; }

// Logistic function: clamp to [-30, 30]; n = rint(z*log2 e); r = z - n*ln2 (two fused steps
// with a hi/lo split of ln2); degree-7 Taylor polynomial of exp(r) by Horner; scale by 2^n
// through the exponent field; 1 / (1 + e) with IEEE add and divide.
__device__ __forceinline__ float sigmoid_fixed(float x) {
    const float t = fminf(fmaxf(x, -30.0f), 30.0f);
    const float z = -t;
    const float n = rintf(__fmul_rn(z, 0x1.715476p+0f));
    float r = __fmaf_rn(n, -0x1.62e4p-1f, z);
    r = __fmaf_rn(n, -0x1.7f7d1cp-20f, r);
    float p = 0x1.a01a02p-13f;
    p = __fmaf_rn(p, r, 0x1.6c16c2p-10f);
    p = __fmaf_rn(p, r, 0x1.111112p-7f);
    p = __fmaf_rn(p, r, 0x1.555556p-5f);
    p = __fmaf_rn(p, r, 0x1.555556p-3f);
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    const float two_n = __int_as_float((__float2int_rn(n) + 127) << 23);
    const float e = __fmul_rn(p, two_n);
    return __fdiv_rn(1.0f, __fadd_rn(1.0f, e));
}

// Corners of a head row's box: x1 = cx - 0.5*w, x2 = cx + 0.5*w (0.5*w is exact).
__device__ __forceinline__ float4 box_corners(float cx, float cy, float bw, float bh) {
    const float hw = __fmul_rn(0.5f, bw), hh = __fmul_rn(0.5f, bh);
    return make_float4(__fsub_rn(cx, hw), __fsub_rn(cy, hh), __fadd_rn(cx, hw), __fadd_rn(cy, hh));
}

// The two terms of IoU = inter / uni, operation by operation: uni = (area_a + area_b) - inter.
__device__ __forceinline__ void iou_terms(const float4 a, const float4 b, float& inter, float& uni) {
    float iw = __fsub_rn(fminf(a.z, b.z), fmaxf(a.x, b.x));
    float ih = __fsub_rn(fminf(a.w, b.w), fmaxf(a.y, b.y));
    iw = fmaxf(iw, 0.0f);
    ih = fmaxf(ih, 0.0f);
    inter = __fmul_rn(iw, ih);
    const float area_a = __fmul_rn(__fsub_rn(a.z, a.x), __fsub_rn(a.w, a.y));
    const float area_b = __fmul_rn(__fsub_rn(b.z, b.x), __fsub_rn(b.w, b.y));
    uni = __fsub_rn(__fadd_rn(area_a, area_b), inter);
}

// The test fl(inter / uni) > thr without the division.  The binary32 quotient rounds to a
// value above thr exactly when the real quotient lies above the midpoint `mid` of thr and the
// next float up (or on it, when that next float has an even mantissa and so wins the tie).
// inter, uni and mid have 24, 24 and 25 significant bits, so mid * uni is exact in binary64
// and the comparison is exact.  Non-finite operands compare false, like the quotient would.
struct IouTest {
    double mid;
    int tie_up;
};
__device__ __forceinline__ bool iou_above(const float4 a, const float4 b, const IouTest t) {
    float inter, uni;
    iou_terms(a, b, inter, uni);
    if (!(uni > 0.0f)) return false;
    const double lhs = (double)inter, rhs = __dmul_rn(t.mid, (double)uni);
    return t.tie_up ? lhs >= rhs : lhs > rhs;
}

}  // namespace octo
