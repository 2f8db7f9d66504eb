/*
 * Seeded synthetic inputs for the cascade-stage hot path: camera-shaped BGR frames and
 * YOLOv5-style detector heads.  These stand in for the traffic / surveillance streams the
 * paper evaluates on (Section V-A "Data": 1280x720, 15 fps sources), which are not
 * redistributable.  Nothing here belongs to the method itself: no letterbox, decode, NMS
 * or crop arithmetic lives in this file.  Both the CPU oracle and the CUDA path read the
 * bytes produced here.
 *
 * Randomness: SplitMix64 used as a counter-based generator.  The i-th draw of stream `key`
 * is mix64(key + (i+1)*GOLDEN); keys are derived from (seed, kind, frame index).
 */
#define _GNU_SOURCE
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define GOLDEN 0x9E3779B97F4A7C15ull

static inline uint64_t mix64(uint64_t z) {
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

typedef struct { uint64_t key, ctr; } rng_t;

static rng_t rng_make(uint64_t seed, uint64_t kind, uint64_t index) {
    rng_t r;
    r.key = mix64(mix64(seed * GOLDEN + kind) + index * GOLDEN + 0x632BE59BD9B4E019ull);
    r.ctr = 0;
    return r;
}
static inline uint64_t rng_u64(rng_t* r) { r->ctr += 1; return mix64(r->key + r->ctr * GOLDEN); }
/* uniform in [0,1) with 53 bits */
static inline double rng_unit(rng_t* r) { return (double)(rng_u64(r) >> 11) * (1.0 / 9007199254740992.0); }
static inline double rng_range(rng_t* r, double lo, double hi) { return lo + (hi - lo) * rng_unit(r); }
static inline uint32_t rng_below(rng_t* r, uint32_t n) { return (uint32_t)(((rng_u64(r) >> 32) * (uint64_t)n) >> 32); }

/* Box-Muller, two standard normals per call. */
static inline void rng_normal2(rng_t* r, float* a, float* b) {
    uint64_t u = rng_u64(r);
    float u1 = ((float)(uint32_t)(u >> 40) + 0.5f) * (1.0f / 16777216.0f); /* (0,1) */
    float u2 = ((float)(uint32_t)((u >> 8) & 0xFFFFFFu)) * (1.0f / 16777216.0f);
    float m = sqrtf(-2.0f * logf(u1));
    float s, c;
    sincosf(6.28318530717958647692f * u2, &s, &c);
    *a = m * c;
    *b = m * s;
}

/* ---- frames ------------------------------------------------------------------------ */

/* Uniform random bytes (the "tiny" workload).  Bytes beyond 3*w in a row are zero. */
void wl_frame_uniform(uint64_t seed, int32_t frame, int32_t w, int32_t h, int32_t pitch, uint8_t* out) {
    rng_t r = rng_make(seed, 1, (uint64_t)frame);
    for (int y = 0; y < h; ++y) {
        uint8_t* row = out + (size_t)y * pitch;
        int nb = 3 * w, x = 0;
        for (; x + 8 <= nb; x += 8) { uint64_t v = rng_u64(&r); memcpy(row + x, &v, 8); }
        if (x < nb) { uint64_t v = rng_u64(&r); memcpy(row + x, &v, (size_t)(nb - x)); }
        if (pitch > nb) memset(row + nb, 0, (size_t)(pitch - nb));
    }
}

/* Smooth random gradients + one sinusoid + uniform noise per channel:
 * p(y,x,c) = clamp(round(a_c + b_c*x/w + d_c*y/h + 40*sin(2*pi*(fx*x/w + fy*y/h) + phi_c) + U(-8,8)), 0, 255) */
void wl_frame_smooth(uint64_t seed, int32_t frame, int32_t w, int32_t h, int32_t pitch, uint8_t* out) {
    rng_t r = rng_make(seed, 2, (uint64_t)frame);
    double a[3], b[3], d[3], phi[3];
    for (int c = 0; c < 3; ++c) {
        a[c] = rng_range(&r, 60.0, 180.0);
        b[c] = rng_range(&r, -60.0, 60.0);
        d[c] = rng_range(&r, -60.0, 60.0);
        phi[c] = rng_range(&r, 0.0, 6.283185307179586);
    }
    int fx = 1 + (int)rng_below(&r, 6), fy = 1 + (int)rng_below(&r, 6);
    float* sx = (float*)malloc(sizeof(float) * (size_t)w * 2);
    float* cx = sx + w;
    for (int x = 0; x < w; ++x) {
        double t = 6.283185307179586 * fx * (double)x / (double)w;
        sx[x] = (float)sin(t); cx[x] = (float)cos(t);
    }
    for (int y = 0; y < h; ++y) {
        rng_t rr = rng_make(seed, 3, ((uint64_t)frame << 20) + (uint64_t)y);
        uint8_t* row = out + (size_t)y * pitch;
        float sy[3], cy[3], base[3], bw[3];
        for (int c = 0; c < 3; ++c) {
            double t = 6.283185307179586 * fy * (double)y / (double)h + phi[c];
            sy[c] = (float)sin(t); cy[c] = (float)cos(t);
            base[c] = (float)(a[c] + d[c] * (double)y / (double)h);
            bw[c] = (float)(b[c] / (double)w);
        }
        uint64_t bits = 0; int nbits = 0;
        for (int x = 0; x < w; ++x) {
            for (int c = 0; c < 3; ++c) {
                if (nbits < 16) { bits = rng_u64(&rr); nbits = 64; }
                float noise = (float)(bits & 0xFFFF) * (16.0f / 65536.0f) - 8.0f;
                bits >>= 16; nbits -= 16;
                float v = base[c] + bw[c] * (float)x + 40.0f * (sx[x] * cy[c] + cx[x] * sy[c]) + noise;
                float rv = floorf(v + 0.5f);
                row[3 * x + c] = (uint8_t)(rv < 0.0f ? 0.0f : (rv > 255.0f ? 255.0f : rv));
            }
        }
        if (pitch > 3 * w) memset(row + 3 * w, 0, (size_t)(pitch - 3 * w));
    }
    free(sx);
}

/* ---- detector heads ---------------------------------------------------------------- */

/*
 * One image's head, [A, 5 + C] fp32, rows (cx, cy, w, h, obj, class_0 .. class_{C-1}).
 * Background rows: cx,cy ~ U(0,S); w,h ~ U(8,120); obj and class values ~ N(bg_mean, 1).
 * n_raised rows at distinct random anchor indices form n_groups clusters.  A cluster has a
 * centre box (w,h ~ U(size_lo,size_hi), placed inside x in [0,S], y in [y_lo,y_hi]) and one
 * class; each member jitters the centre by U(-jit,jit)*size and the size by U(s_lo,s_hi).
 * Raised rows get obj and their cluster's class value ~ N(fg_mean, fg_std).
 * With logits == 0 every obj/class value is passed through the logistic function so the
 * head holds probabilities instead.
 */
void wl_head(uint64_t seed, int32_t frame, int32_t S, int32_t A, int32_t C,
             int32_t n_raised, int32_t n_groups,
             float y_lo, float y_hi, float size_lo, float size_hi,
             float jit, float s_lo, float s_hi,
             float bg_mean, float fg_mean, float fg_std, int32_t logits, float* out) {
    const int row = 5 + C;
    /* background */
    rng_t r = rng_make(seed, 4, (uint64_t)frame);
    for (int a = 0; a < A; ++a) {
        float* p = out + (size_t)a * row;
        p[0] = (float)rng_range(&r, 0.0, (double)S);
        p[1] = (float)rng_range(&r, 0.0, (double)S);
        p[2] = (float)rng_range(&r, 8.0, 120.0);
        p[3] = (float)rng_range(&r, 8.0, 120.0);
        int k = 4;
        while (k < row) {
            float n0, n1;
            rng_normal2(&r, &n0, &n1);
            p[k++] = bg_mean + n0;
            if (k < row) p[k++] = bg_mean + n1;
        }
    }
    /* raised anchors: distinct indices by rejection against a byte map */
    if (n_raised > A) n_raised = A;
    if (n_groups < 1) n_groups = 1;
    if (n_groups > n_raised && n_raised > 0) n_groups = n_raised;
    rng_t q = rng_make(seed, 5, (uint64_t)frame);
    uint8_t* used = (uint8_t*)calloc((size_t)A, 1);
    int made = 0;
    for (int g = 0; g < n_groups && n_raised > 0; ++g) {
        int members = n_raised / n_groups + (g < n_raised % n_groups ? 1 : 0);
        float gw = (float)rng_range(&q, size_lo, size_hi);
        float gh = (float)rng_range(&q, size_lo, size_hi);
        float xlo = 0.5f * gw, xhi = (float)S - 0.5f * gw;
        float ylo = y_lo + 0.5f * gh, yhi = y_hi - 0.5f * gh;
        if (xhi < xlo) xlo = xhi = 0.5f * (float)S;
        if (yhi < ylo) ylo = yhi = 0.5f * (y_lo + y_hi);
        float gx = (float)rng_range(&q, xlo, xhi);
        float gy = (float)rng_range(&q, ylo, yhi);
        int cls = (int)rng_below(&q, (uint32_t)C);
        for (int m = 0; m < members; ++m, ++made) {
            uint32_t a;
            do { a = rng_below(&q, (uint32_t)A); } while (used[a]);
            used[a] = 1;
            float* p = out + (size_t)a * row;
            float bw = gw * (float)rng_range(&q, s_lo, s_hi);
            float bh = gh * (float)rng_range(&q, s_lo, s_hi);
            p[0] = gx + gw * (float)rng_range(&q, -jit, jit);
            p[1] = gy + gh * (float)rng_range(&q, -jit, jit);
            p[2] = bw;
            p[3] = bh;
            float n0, n1;
            rng_normal2(&q, &n0, &n1);
            p[4] = fg_mean + fg_std * n0;
            p[5 + cls] = fg_mean + fg_std * n1;
        }
    }
    free(used);
    if (!logits) {
        for (int a = 0; a < A; ++a) {
            float* p = out + (size_t)a * row;
            for (int k = 4; k < row; ++k) p[k] = 1.0f / (1.0f + expf(-p[k]));
        }
    }
}

/* Bernoulli(1/2) bit used to mix 720p and 1080p frames in the two-branch workload. */
int32_t wl_coin(uint64_t seed, int32_t frame) {
    rng_t r = rng_make(seed, 6, (uint64_t)frame);
    return (int32_t)(rng_u64(&r) >> 63);
}
