/*
 * CPU oracle for the per-batch tensor work of a cascade pipeline stage.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition the CUDA library is
 * checked against.  It shares no code with the CUDA path and must never be linked into,
 * imported by or called from it; only the tests, the smoke check and the benchmark's CPU
 * baseline leg may use it.
 *
 * What the paper fixes and what it does not.  The paper (OctopInf) describes pipelines as
 * cascades of DNNs such as [Object Detect -> Vehicle Classify, Plate Detect] (Section I),
 * whose models map an image to bounding boxes (Table II, In_m / Out_m), run in batches of
 * size bz (Eq. 1, Algorithm 1) and hand their detections to downstream models
 * (Section III-B, Observation 1).  It gives no formula for the tensor work around the
 * model.  Every numeric rule below is therefore a stated reading (labelled R1..R8 in the
 * comments), chosen so that exactly one result is correct:
 *
 *   R1 letterbox geometry      integer, round-half-up of the scaled short side, centred
 *   R2 bilinear resize core    half-pixel centres, edge clamp, no antialias; double here
 *   R3 decode / score          best class by raw value, score = sigma(obj)*sigma(cls) in a
 *                              fixed sequence of binary32 operations
 *   R4 ordering                score descending, ties by lower anchor index
 *   R5 greedy class-aware NMS  IoU in a fixed binary32 formula, strict thresholds
 *   R6 scale-back              letterbox pixels -> frame pixels, binary32, clamped
 *   R7 crop rectangle + resize outward-rounded integer rectangle, stretched by R2
 *   R8 batch assembler         exclusive prefix sum of per-frame masked counts
 *
 * Floating point that decides an index (R3, R5, R6) is binary32 with every operation
 * rounded on its own (build with -ffp-contract=off); pixel values (R2) are double.
 * Parity pins live in tests/test_oracle_*.py; no function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------ */
/* R1: letterbox geometry.  The longer side maps to S; the other side is h*S/w rounded   */
/* half-up in exact integer arithmetic; the image is centred, an odd remainder puts the  */
/* extra canvas pixel on the right / bottom.                                             */
/* ------------------------------------------------------------------------------------ */
void orc_letterbox_geometry(int32_t w, int32_t h, int32_t S, int32_t* nw, int32_t* nh,
                            int32_t* pad_l, int32_t* pad_t) {
    int64_t W = w, H = h, s = S, a, b;
    if (W >= H) {
        a = s;
        b = (2 * H * s + W) / (2 * W);
        if (b < 1) b = 1;
    } else {
        b = s;
        a = (2 * W * s + H) / (2 * H);
        if (a < 1) a = 1;
    }
    *nw = (int32_t)a;
    *nh = (int32_t)b;
    *pad_l = (int32_t)((s - a) / 2);
    *pad_t = (int32_t)((s - b) / 2);
}

/* ------------------------------------------------------------------------------------ */
/* R2: bilinear resize of the rectangle [rx0, rx0+cw) x [ry0, ry0+ch) of an interleaved   */
/* 3-channel uint8 image to nw x nh.  Destination pixel centre (dx+0.5, dy+0.5) maps to   */
/* source coordinate (dx+0.5)*cw/nw - 0.5, clamped to [0, cw-1]; the four taps are        */
/* clamped inside the rectangle; raw 0..255 values, no intermediate rounding.             */
/* out: [3][nh][nw] doubles in the image's own channel order.                             */
/* ------------------------------------------------------------------------------------ */
static double resize_tap(const uint8_t* img, int32_t pitch, int32_t rx0, int32_t ry0,
                         int32_t x, int32_t y, int c) {
    return (double)img[(size_t)(ry0 + y) * (size_t)pitch + (size_t)(rx0 + x) * 3 + (size_t)c];
}

void orc_resize_f64(const uint8_t* img, int32_t pitch, int32_t rx0, int32_t ry0, int32_t cw,
                    int32_t ch, int32_t nw, int32_t nh, double* out) {
    for (int dy = 0; dy < nh; ++dy) {
        double sy = ((double)dy + 0.5) * ((double)ch / (double)nh) - 0.5;
        if (sy < 0.0) sy = 0.0;
        if (sy > (double)(ch - 1)) sy = (double)(ch - 1);
        int y0 = (int)floor(sy);
        int y1 = y0 + 1 < ch - 1 ? y0 + 1 : ch - 1;
        double fy = sy - (double)y0;
        for (int dx = 0; dx < nw; ++dx) {
            double sx = ((double)dx + 0.5) * ((double)cw / (double)nw) - 0.5;
            if (sx < 0.0) sx = 0.0;
            if (sx > (double)(cw - 1)) sx = (double)(cw - 1);
            int x0 = (int)floor(sx);
            int x1 = x0 + 1 < cw - 1 ? x0 + 1 : cw - 1;
            double fx = sx - (double)x0;
            for (int c = 0; c < 3; ++c) {
                double p00 = resize_tap(img, pitch, rx0, ry0, x0, y0, c);
                double p01 = resize_tap(img, pitch, rx0, ry0, x1, y0, c);
                double p10 = resize_tap(img, pitch, rx0, ry0, x0, y1, c);
                double p11 = resize_tap(img, pitch, rx0, ry0, x1, y1, c);
                double top = (1.0 - fx) * p00 + fx * p01;
                double bot = (1.0 - fx) * p10 + fx * p11;
                out[((size_t)c * (size_t)nh + (size_t)dy) * (size_t)nw + (size_t)dx] =
                    (1.0 - fy) * top + fy * bot;
            }
        }
    }
}

/* double -> IEEE binary16 bits, round to nearest even, one rounding (no float detour). */
uint16_t orc_f64_to_half(double v) {
    uint16_t sign = 0;
    if (v != v) return 0x7E00;
    if (v < 0.0) { sign = 0x8000; v = -v; }
    if (v == 0.0) return sign;
    if (v >= 65520.0) return (uint16_t)(sign | 0x7C00);
    int e;
    (void)frexp(v, &e); /* v = m * 2^e, m in [0.5, 1) */
    int E = e - 1;      /* v = 1.f * 2^E */
    if (E < -14) {
        double q = rint(ldexp(v, 24)); /* units of 2^-24 */
        return (uint16_t)(sign | (uint16_t)q);
    }
    double q = rint(ldexp(v, 10 - E)); /* in [1024, 2048] */
    if (q >= 2048.0) { q = 1024.0; E += 1; }
    if (E > 15) return (uint16_t)(sign | 0x7C00);
    return (uint16_t)(sign | (uint16_t)((E + 15) << 10) | (uint16_t)((int)q - 1024));
}

/* R1 + R2: one frame -> [3][S][S] half bits.  Plane p holds input channel (swap_rb ? 2-p : p);
 * value = half(v / 255); canvas outside the image = half(pad_value / 255). */
void orc_letterbox(const uint8_t* img, int32_t w, int32_t h, int32_t pitch, int32_t S,
                   int32_t pad_value, int32_t swap_rb, uint16_t* out) {
    int32_t nw, nh, pl, pt;
    orc_letterbox_geometry(w, h, S, &nw, &nh, &pl, &pt);
    double* tmp = (double*)malloc(sizeof(double) * 3 * (size_t)nw * (size_t)nh);
    orc_resize_f64(img, pitch, 0, 0, w, h, nw, nh, tmp);
    uint16_t fill = orc_f64_to_half((double)pad_value / 255.0);
    for (size_t i = 0; i < (size_t)3 * (size_t)S * (size_t)S; ++i) out[i] = fill;
    for (int p = 0; p < 3; ++p) {
        int c = swap_rb ? 2 - p : p;
        for (int y = 0; y < nh; ++y)
            for (int x = 0; x < nw; ++x)
                out[((size_t)p * (size_t)S + (size_t)(pt + y)) * (size_t)S + (size_t)(pl + x)] =
                    orc_f64_to_half(tmp[((size_t)c * (size_t)nh + (size_t)y) * (size_t)nw + (size_t)x] / 255.0);
    }
    free(tmp);
}

/* ------------------------------------------------------------------------------------ */
/* R3: logistic function as a fixed sequence of binary32 operations (each rounded to      */
/* nearest even; the only fused operations are the ones written as fmaf):                 */
/*   t = clamp(x, -30, 30); z = -t; n = rint(z * log2(e));                                */
/*   r = z - n*ln2 (two-constant split, two fmaf); p = sum_{k<=7} r^k/k! by Horner;       */
/*   e = p * 2^n (exact scaling); sigma = 1 / (1 + e).                                    */
/* The platform expf is deliberately not used: its last bits differ between machines and  */
/* would flip threshold tests and the score order.                                        */
/* ------------------------------------------------------------------------------------ */
float orc_sigmoid(float x) {
    float t = fminf(fmaxf(x, -30.0f), 30.0f);
    float z = -t;
    float n = rintf(z * 0x1.715476p+0f);
    float r = fmaf(n, -0x1.62e4p-1f, z);
    r = fmaf(n, -0x1.7f7d1cp-20f, r);
    float p = 0x1.a01a02p-13f;          /* 1/7! */
    p = fmaf(p, r, 0x1.6c16c2p-10f);    /* 1/6! */
    p = fmaf(p, r, 0x1.111112p-7f);     /* 1/5! */
    p = fmaf(p, r, 0x1.555556p-5f);     /* 1/4! */
    p = fmaf(p, r, 0x1.555556p-3f);     /* 1/3! */
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    union { uint32_t u; float f; } two_n;
    two_n.u = (uint32_t)((int32_t)n + 127) << 23;
    float e = p * two_n.f;
    return 1.0f / (1.0f + e);
}

typedef struct {
    float x1, y1, x2, y2, score;
    int32_t cls, anchor, _pad;
} orc_det_t; /* 32 bytes; same field order as the library's detection record */

static int finite_f(float v) { return v == v && v - v == 0.0f; }

/* R3: decode one image's head [A][5+C].  A row is a candidate iff every value in it is
 * finite, w > 0, h > 0 and score > conf (strict), with k* = first maximal class value and
 * score = fl(sigma(obj) * sigma(c_k*)) for logits, fl(obj * c_k*) for probabilities.
 * Corners: x1 = fl(cx - fl(0.5*w)), x2 = fl(cx + fl(0.5*w)), same in y (letterbox pixels).
 * Output in anchor order; returns the count.  out must hold A records. */
int32_t orc_decode(const float* head, int32_t A, int32_t C, int32_t logits, float conf,
                   orc_det_t* out) {
    int32_t n = 0;
    const int row = 5 + C;
    for (int32_t a = 0; a < A; ++a) {
        const float* p = head + (size_t)a * (size_t)row;
        int ok = 1;
        for (int k = 0; k < row; ++k) ok &= finite_f(p[k]);
        if (!ok) continue;
        if (!(p[2] > 0.0f) || !(p[3] > 0.0f)) continue;
        int best = 0;
        float bv = p[5];
        for (int k = 1; k < C; ++k)
            if (p[5 + k] > bv) { bv = p[5 + k]; best = k; }
        float score;
        if (logits) {
            float so = orc_sigmoid(p[4]);
            float sc = orc_sigmoid(bv);
            score = so * sc;
        } else {
            score = p[4] * bv;
        }
        if (!(score > conf)) continue;
        float hw = 0.5f * p[2], hh = 0.5f * p[3];
        orc_det_t d;
        d.x1 = p[0] - hw; d.y1 = p[1] - hh; d.x2 = p[0] + hw; d.y2 = p[1] + hh;
        d.score = score; d.cls = best; d.anchor = a; d._pad = 0;
        out[n++] = d;
    }
    return n;
}

/* R3 variants: other head layouts and multi-label candidates.
 *   layout 0  rows   [A][5 + C]: (cx, cy, w, h, obj, class_0 ..), the form above.
 *   layout 1  planes [4 + C][A]: element e of anchor a at head[e * A + a]; anchor-free heads
 *             carry no objectness, the score is the class value alone: sigma(c_k) for logits,
 *             c_k for probabilities.
 *   multi_label 0: one candidate per anchor, k* = first maximal class value.
 *   multi_label 1: every class k whose own score fl(sigma(obj) * sigma(c_k)) (rows) or
 *             sigma(c_k) (planes) exceeds conf is a candidate of that class; an anchor can
 *             yield several candidates that share its box.
 * The row filter is the same: every value of the anchor finite, w > 0, h > 0.  Output in
 * (anchor, class) order; returns the count (at most `cap` are written). */
int32_t orc_decode_ex(const float* head, int32_t A, int32_t C, int32_t logits, float conf,
                      int32_t layout, int32_t multi_label, orc_det_t* out, int32_t cap) {
    int32_t n = 0;
    const int nbox = layout == 0 ? 5 : 4; /* values before the class values */
    const int row = nbox + C;
    float* v = (float*)malloc(sizeof(float) * (size_t)row);
    for (int32_t a = 0; a < A; ++a) {
        for (int e = 0; e < row; ++e)
            v[e] = layout == 0 ? head[(size_t)a * (size_t)row + (size_t)e] : head[(size_t)e * (size_t)A + (size_t)a];
        int ok = 1;
        for (int e = 0; e < row; ++e) ok &= finite_f(v[e]);
        if (!ok) continue;
        if (!(v[2] > 0.0f) || !(v[3] > 0.0f)) continue;
        const float* cv = v + nbox;
        float so = 1.0f; /* objectness factor; absent in the planes layout */
        if (layout == 0) so = logits ? orc_sigmoid(v[4]) : v[4];
        float hw = 0.5f * v[2], hh = 0.5f * v[3];
        orc_det_t d;
        d.x1 = v[0] - hw; d.y1 = v[1] - hh; d.x2 = v[0] + hw; d.y2 = v[1] + hh;
        d.anchor = a; d._pad = 0;
        if (!multi_label) {
            int best = 0;
            float bv = cv[0];
            for (int k = 1; k < C; ++k)
                if (cv[k] > bv) { bv = cv[k]; best = k; }
            float sc = logits ? orc_sigmoid(bv) : bv;
            float score = layout == 0 ? so * sc : sc;
            if (!(score > conf)) continue;
            d.score = score; d.cls = best;
            if (n < cap) out[n] = d;
            n++;
        } else {
            for (int k = 0; k < C; ++k) {
                float sc = logits ? orc_sigmoid(cv[k]) : cv[k];
                float score = layout == 0 ? so * sc : sc;
                if (!(score > conf)) continue;
                d.score = score; d.cls = k;
                if (n < cap) out[n] = d;
                n++;
            }
        }
    }
    free(v);
    return n;
}

/* R4: total order -- score descending, then anchor ascending; candidates of one anchor
 * (multi-label decode) that tie in score go by ascending class. */
static int cand_cmp(const void* pa, const void* pb) {
    const orc_det_t* a = (const orc_det_t*)pa;
    const orc_det_t* b = (const orc_det_t*)pb;
    if (a->score > b->score) return -1;
    if (a->score < b->score) return 1;
    if (a->anchor != b->anchor) return (a->anchor > b->anchor) - (a->anchor < b->anchor);
    return (a->cls > b->cls) - (a->cls < b->cls);
}
void orc_sort(orc_det_t* c, int32_t n) { qsort(c, (size_t)n, sizeof(orc_det_t), cand_cmp); }

/* R5: IoU in binary32, operation by operation. */
float orc_iou(const orc_det_t* a, const orc_det_t* b) {
    float iw = fminf(a->x2, b->x2) - fmaxf(a->x1, b->x1);
    float ih = fminf(a->y2, b->y2) - fmaxf(a->y1, b->y1);
    iw = fmaxf(iw, 0.0f);
    ih = fmaxf(ih, 0.0f);
    float inter = iw * ih;
    float aw = a->x2 - a->x1, ah = a->y2 - a->y1;
    float bw = b->x2 - b->x1, bh = b->y2 - b->y1;
    float area_a = aw * ah, area_b = bw * bh;
    float sum = area_a + area_b;
    float uni = sum - inter;
    return uni > 0.0f ? inter / uni : 0.0f;
}

/* R5: greedy class-aware NMS over a list already in R4 order.  Element i is kept iff no
 * earlier KEPT element of the same class has IoU(j, i) > thr (strict); stops after max_det
 * kept.  keep[] receives the kept positions in order; returns their number. */
int32_t orc_nms_ex(const orc_det_t* c, int32_t n, float thr, int32_t max_det, int32_t agnostic, int32_t* keep) {
    int32_t k = 0;
    for (int32_t i = 0; i < n && k < max_det; ++i) {
        int alive = 1;
        for (int32_t t = 0; t < k; ++t) {
            const orc_det_t* j = &c[keep[t]];
            if ((agnostic || j->cls == c[i].cls) && orc_iou(j, &c[i]) > thr) { alive = 0; break; }
        }
        if (alive) keep[k++] = i;
    }
    return k;
}
/* Class-aware form (the default); with agnostic != 0 orc_nms_ex ignores the class test, i.e.
 * boxes of different classes suppress each other (decode variant, classes kept for output). */
int32_t orc_nms(const orc_det_t* c, int32_t n, float thr, int32_t max_det, int32_t* keep) {
    return orc_nms_ex(c, n, thr, max_det, 0, keep);
}

/* R6: detector-input pixels -> source-frame pixels in binary32.  The detector input shows a
 * region [ox, ox+rw) x [oy, oy+rh) of the source frame (the whole frame for a first-level
 * stage; the upstream crop rectangle for a chained stage), scaled to nw x nh and placed at
 * (pad_l, pad_t) on the canvas:  X = fl(fl(fl(x - pad_l) * g) + ox), g = fl(rw / nw), clamped
 * to [ox, ox + rw]; likewise in y.  With ox = 0 the last addition changes nothing. */
void orc_scale_back_region(orc_det_t* d, int32_t nw, int32_t nh, int32_t pad_l, int32_t pad_t,
                           int32_t ox, int32_t oy, int32_t rw, int32_t rh) {
    float gx = (float)rw / (float)nw, gy = (float)rh / (float)nh;
    float fpl = (float)pad_l, fpt = (float)pad_t;
    float xlo = (float)ox, ylo = (float)oy, xhi = (float)(ox + rw), yhi = (float)(oy + rh);
    float X1 = (d->x1 - fpl) * gx + xlo, X2 = (d->x2 - fpl) * gx + xlo;
    float Y1 = (d->y1 - fpt) * gy + ylo, Y2 = (d->y2 - fpt) * gy + ylo;
    d->x1 = fminf(fmaxf(X1, xlo), xhi);
    d->x2 = fminf(fmaxf(X2, xlo), xhi);
    d->y1 = fminf(fmaxf(Y1, ylo), yhi);
    d->y2 = fminf(fmaxf(Y2, ylo), yhi);
}

/* R6 for a first-level stage: the region is the whole w x h frame, letterboxed by R1. */
void orc_scale_back(orc_det_t* d, int32_t w, int32_t h, int32_t S) {
    int32_t nw, nh, pl, pt;
    orc_letterbox_geometry(w, h, S, &nw, &nh, &pl, &pt);
    orc_scale_back_region(d, nw, nh, pl, pt, 0, 0, w, h);
}

/* R3..R6 for one detector input: decode, order, NMS, cap, then every kept box mapped into the
 * source frame through the region map {nw, nh, pl, pt, ox, oy, rw, rh} of R6.  variants = 0 takes
 * the plain row decode (orc_decode), 1 the decode with head layout and multi-label candidates
 * (orc_decode_ex).  Returns the kept count; *n_cand receives the candidate count before NMS. */
static int32_t postprocess_core(const float* head, int32_t A, int32_t C, int32_t logits, float conf, float iou_thr,
                                int32_t max_det, int32_t agnostic, int32_t variants, int32_t layout,
                                int32_t multi_label, const int32_t map[8], orc_det_t* dets, int32_t* n_cand) {
    const size_t cap = (size_t)(A > 0 ? A : 1) * (size_t)(variants && multi_label ? (C > 0 ? C : 1) : 1);
    orc_det_t* cand = (orc_det_t*)malloc(sizeof(orc_det_t) * cap);
    int32_t* keep = (int32_t*)malloc(sizeof(int32_t) * (size_t)(max_det > 0 ? max_det : 1));
    int32_t n = variants ? orc_decode_ex(head, A, C, logits, conf, layout, multi_label, cand, (int32_t)cap)
                         : orc_decode(head, A, C, logits, conf, cand);
    orc_sort(cand, n);
    int32_t k = orc_nms_ex(cand, n, iou_thr, max_det, agnostic, keep);
    for (int32_t t = 0; t < k; ++t) {
        dets[t] = cand[keep[t]];
        orc_scale_back_region(&dets[t], map[0], map[1], map[2], map[3], map[4], map[5], map[6], map[7]);
    }
    if (n_cand) *n_cand = n;
    free(cand);
    free(keep);
    return k;
}

/* First-level stage: the region is the whole w x h frame, letterboxed by R1. */
static void frame_map(int32_t w, int32_t h, int32_t S, int32_t map[8]) {
    orc_letterbox_geometry(w, h, S, &map[0], &map[1], &map[2], &map[3]);
    map[4] = 0; map[5] = 0; map[6] = w; map[7] = h;
}

/* Chained (second-level) stage: the detector input is the upstream crop of the rectangle
 * [ox, ox+rw) x [oy, oy+rh), stretched to S x S (no padding), so the head's boxes live on that
 * S x S grid and map back into the rectangle of the ORIGINAL frame. */
static void region_map(int32_t S, int32_t ox, int32_t oy, int32_t rw, int32_t rh, int32_t map[8]) {
    map[0] = S; map[1] = S; map[2] = 0; map[3] = 0;
    map[4] = ox; map[5] = oy; map[6] = rw; map[7] = rh;
}

int32_t orc_postprocess_image_ex(const float* head, int32_t A, int32_t C, int32_t logits,
                                 float conf, float iou_thr, int32_t max_det, int32_t w, int32_t h,
                                 int32_t S, int32_t agnostic, orc_det_t* dets, int32_t* n_cand) {
    int32_t map[8];
    frame_map(w, h, S, map);
    return postprocess_core(head, A, C, logits, conf, iou_thr, max_det, agnostic, 0, 0, 0, map, dets, n_cand);
}

int32_t orc_postprocess_image(const float* head, int32_t A, int32_t C, int32_t logits,
                              float conf, float iou_thr, int32_t max_det, int32_t w, int32_t h,
                              int32_t S, orc_det_t* dets, int32_t* n_cand) {
    return orc_postprocess_image_ex(head, A, C, logits, conf, iou_thr, max_det, w, h, S, 0, dets, n_cand);
}

/* The same with the decode variants of orc_decode_ex. */
int32_t orc_postprocess_image_v2(const float* head, int32_t A, int32_t C, int32_t logits, float conf,
                                 float iou_thr, int32_t max_det, int32_t w, int32_t h, int32_t S,
                                 int32_t agnostic, int32_t layout, int32_t multi_label, orc_det_t* dets,
                                 int32_t* n_cand) {
    int32_t map[8];
    frame_map(w, h, S, map);
    return postprocess_core(head, A, C, logits, conf, iou_thr, max_det, agnostic, 1, layout, multi_label, map, dets,
                            n_cand);
}

/* R3..R6 for one item of a chained stage. */
int32_t orc_postprocess_region(const float* head, int32_t A, int32_t C, int32_t logits, float conf,
                               float iou_thr, int32_t max_det, int32_t S, int32_t ox, int32_t oy,
                               int32_t rw, int32_t rh, orc_det_t* dets, int32_t* n_cand) {
    int32_t map[8];
    region_map(S, ox, oy, rw, rh, map);
    return postprocess_core(head, A, C, logits, conf, iou_thr, max_det, 0, 0, 0, 0, map, dets, n_cand);
}

/* The same for the decode variants of orc_decode_ex (head layout, multi-label candidates). */
int32_t orc_postprocess_region_v2(const float* head, int32_t A, int32_t C, int32_t logits, float conf,
                                  float iou_thr, int32_t max_det, int32_t S, int32_t ox, int32_t oy,
                                  int32_t rw, int32_t rh, int32_t layout, int32_t multi_label,
                                  orc_det_t* dets, int32_t* n_cand) {
    int32_t map[8];
    region_map(S, ox, oy, rw, rh, map);
    return postprocess_core(head, A, C, logits, conf, iou_thr, max_det, 0, 1, layout, multi_label, map, dets, n_cand);
}

/* R7: integer crop rectangle of a frame-space box: rx0 = clamp(floor(X1), 0, w-1),
 * rx1 = clamp(ceil(X2), rx0+1, w), same in y.  rect = {rx0, ry0, rx1, ry1}. */
void orc_crop_rect(const orc_det_t* d, int32_t w, int32_t h, int32_t* rect) {
    int64_t x0 = (int64_t)floorf(d->x1), y0 = (int64_t)floorf(d->y1);
    int64_t x1 = (int64_t)ceilf(d->x2), y1 = (int64_t)ceilf(d->y2);
    if (x0 < 0) x0 = 0;
    if (x0 > w - 1) x0 = w - 1;
    if (y0 < 0) y0 = 0;
    if (y0 > h - 1) y0 = h - 1;
    if (x1 < x0 + 1) x1 = x0 + 1;
    if (x1 > w) x1 = w;
    if (y1 < y0 + 1) y1 = y0 + 1;
    if (y1 > h) y1 = h;
    rect[0] = (int32_t)x0; rect[1] = (int32_t)y0; rect[2] = (int32_t)x1; rect[3] = (int32_t)y1;
}

/* R7: cut the rectangle, stretch it to ow x oh by R2, same plane order and /255 as the
 * letterbox.  out: [3][oh][ow] half bits. */
void orc_crop(const uint8_t* img, int32_t w, int32_t h, int32_t pitch, const orc_det_t* d,
              int32_t ow, int32_t oh, int32_t swap_rb, uint16_t* out) {
    int32_t r[4];
    orc_crop_rect(d, w, h, r);
    double* tmp = (double*)malloc(sizeof(double) * 3 * (size_t)ow * (size_t)oh);
    orc_resize_f64(img, pitch, r[0], r[1], r[2] - r[0], r[3] - r[1], ow, oh, tmp);
    size_t plane = (size_t)ow * (size_t)oh;
    for (int p = 0; p < 3; ++p) {
        int c = swap_rb ? 2 - p : p;
        for (size_t i = 0; i < plane; ++i)
            out[(size_t)p * plane + i] = orc_f64_to_half(tmp[(size_t)c * plane + i] / 255.0);
    }
    free(tmp);
}

/* R7 variants (branch options).
 *   keep_aspect: the cw x ch rectangle keeps its shape inside the ow x oh slot.  The side with
 *     the larger ratio fills the slot: if ow*ch <= oh*cw then nw = ow and nh = ch*ow/cw rounded
 *     half-up in exact integer arithmetic (at least 1), else nh = oh and nw likewise; the image
 *     is centred, an odd remainder puts the extra canvas pixel right / bottom (the letterbox
 *     rule of R1 on a rectangular canvas); the canvas holds pad_value.
 *   normalize: every output value v (= raw / 255, pixels and canvas alike) becomes
 *     (v - mean[p]) / std[p] for output plane p, in double, before the single rounding to half.
 * geom receives {nw, nh, pad_l, pad_t}. */
void orc_fit_geometry(int32_t cw, int32_t ch, int32_t ow, int32_t oh, int32_t* geom) {
    int64_t CW = cw, CH = ch, OW = ow, OH = oh, nw, nh;
    if (OW * CH <= OH * CW) {
        nw = OW;
        nh = (2 * CH * OW + CW) / (2 * CW);
        if (nh < 1) nh = 1;
    } else {
        nh = OH;
        nw = (2 * CW * OH + CH) / (2 * CH);
        if (nw < 1) nw = 1;
    }
    geom[0] = (int32_t)nw;
    geom[1] = (int32_t)nh;
    geom[2] = (int32_t)((OW - nw) / 2);
    geom[3] = (int32_t)((OH - nh) / 2);
}

void orc_crop_ex(const uint8_t* img, int32_t w, int32_t h, int32_t pitch, const orc_det_t* d,
                 int32_t ow, int32_t oh, int32_t swap_rb, int32_t keep_aspect, int32_t pad_value,
                 int32_t normalize, const float* mean, const float* std, uint16_t* out) {
    int32_t r[4], g[4];
    orc_crop_rect(d, w, h, r);
    const int32_t cw = r[2] - r[0], ch = r[3] - r[1];
    g[0] = ow; g[1] = oh; g[2] = 0; g[3] = 0;
    if (keep_aspect) orc_fit_geometry(cw, ch, ow, oh, g);
    const int32_t nw = g[0], nh = g[1], pl = g[2], pt = g[3];
    double* tmp = (double*)malloc(sizeof(double) * 3 * (size_t)nw * (size_t)nh);
    orc_resize_f64(img, pitch, r[0], r[1], cw, ch, nw, nh, tmp);
    size_t plane = (size_t)ow * (size_t)oh;
    for (int p = 0; p < 3; ++p) {
        int c = swap_rb ? 2 - p : p;
        double m = normalize ? (double)mean[p] : 0.0, sd = normalize ? (double)std[p] : 1.0;
        uint16_t fill = orc_f64_to_half(((double)pad_value / 255.0 - m) / sd);
        for (size_t i = 0; i < plane; ++i) out[(size_t)p * plane + i] = fill;
        for (int y = 0; y < nh; ++y)
            for (int x = 0; x < nw; ++x) {
                double v = tmp[((size_t)c * (size_t)nh + (size_t)y) * (size_t)nw + (size_t)x] / 255.0;
                out[(size_t)p * plane + (size_t)(pt + y) * (size_t)ow + (size_t)(pl + x)] =
                    orc_f64_to_half((v - m) / sd);
            }
    }
    free(tmp);
}

/* R8: batch assembler for one branch.  m_n = number of frame n's kept detections whose
 * class bit is set in class_mask (128 bits, bit k of word k/32); offsets = exclusive prefix
 * sum, offsets[N] = total.  Item offsets[n]+j is the j-th such detection of frame n in NMS
 * output order.  items receives (frame, det) pairs for the window
 * [first_item, first_item + max_items); n_items = {packed, total}. */
void orc_assemble(const orc_det_t* dets, const int32_t* counts, int32_t N, int32_t max_det,
                  const uint32_t* class_mask, int32_t first_item, int32_t max_items,
                  int32_t* offsets, int32_t* items, int32_t* n_items) {
    int32_t run = 0, packed = 0;
    offsets[0] = 0;
    for (int32_t n = 0; n < N; ++n) {
        for (int32_t j = 0; j < counts[n]; ++j) {
            const orc_det_t* d = &dets[(size_t)n * (size_t)max_det + (size_t)j];
            uint32_t k = (uint32_t)d->cls;
            if (k < 128u && ((class_mask[k >> 5] >> (k & 31u)) & 1u)) {
                if (run >= first_item && run - first_item < max_items) {
                    items[2 * (size_t)(run - first_item)] = n;
                    items[2 * (size_t)(run - first_item) + 1] = j;
                    ++packed;
                }
                ++run;
            }
        }
        offsets[n + 1] = run;
    }
    n_items[0] = packed;
    n_items[1] = run;
}
