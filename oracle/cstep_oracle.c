/*
 * CPU oracle for the C-step of the learning-compression (L-C) scheme.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, plain definition that the
 * CUDA path is checked against. Nothing in the product path may include,
 * link or call it; it shares no code, header, table or helper with the
 * CUDA kernels.
 *
 * What it computes, with the passage each piece follows:
 *
 *  - compression mapping C(w) = argmin_Theta ||w - D(Theta)||^2 (Section 3.3,
 *    text under Eq. 1). For pruning, D is the identity and Theta is limited
 *    in its number of non-zeros, so the argmin keeps the entries (or whole
 *    structures) of largest magnitude (largest L2 norm) and zeroes the rest.
 *    Here that is written out literally: sort all units by magnitude and
 *    keep the first k.
 *  - target sparsity = proportion of zero-valued parameters (Introduction,
 *    definition of "target sparsity"): exactly Z = round(s * units) units are
 *    zeroed, one global ranking over all tensors ("global sparsity ...
 *    across all the layers", Section 3).
 *  - structured pruning aggregates filters (3-D blocks) or n-D blocks and
 *    prunes whole structures (Table 1, FilterPrune / BlockPrune); the
 *    criterion used here is the L2 norm, which is the argmin above.
 *  - low-precision approximation: each parameter gets the nearest value of
 *    the lower-precision format (Section 2, "quantization using a fixed
 *    codebook"); 32-bit to 16-bit floating point, done by explicit bit
 *    manipulation with round-to-nearest-even.
 *  - scheme order for P+Q is prune, then quantise (Evaluation, Objective 1).
 *  - augmented-Lagrangian quantities of the L-C algorithm (Section 3.3 cites
 *    the AL method; the paper prints no formulas): u = w - lambda/mu,
 *    lambda <- lambda - mu (w - theta), penalty gradient mu (w - theta) - lambda.
 *
 * All fp32 arithmetic is done one IEEE operation at a time (compile with
 * -ffp-contract=off and without -ffast-math); norms accumulate in fp64 in
 * index order.
 *
 * Pins: every function here is pinned by tests/test_oracle_pins.py (brute
 * force ranking, all-supports enumeration of the argmin, closed forms,
 * library routines, hand-computed binary16 values). The printed compression
 * ratios of Table 2 depend on trained weights and pin nothing here.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>

#define ORC_FUSE_FP16    1u
#define ORC_FUSE_LAMBDA  2u
#define ORC_FUSE_PENALTY 4u
#define ORC_FUSE_BF16    8u
#define ORC_FUSE_E4M3    16u
#define ORC_FUSE_E5M2    32u

typedef struct {
    const float *w;        /* weights, never written                          */
    const float *lambda;   /* multipliers, may be NULL (treated as zero)      */
    float *theta;          /* out: compressed weights                         */
    uint8_t *mask;         /* out: 1 = kept, may be NULL                      */
    float *lambda_out;     /* out: updated multipliers, may be NULL           */
    float *grad;           /* out: penalty gradient, may be NULL              */
    uint16_t *theta_h;     /* out: binary16 bits of theta, may be NULL        */
    int64_t numel;
    int32_t ndim;
    int64_t shape[4];
} orc_tensor;

typedef struct {
    int64_t n_units;   /* units that were ranked (elements or structures)     */
    int64_t n_zero;    /* Z                                                    */
    int64_t n_keep;    /* k = n_units - Z                                      */
    uint64_t tau_key;  /* key of the weakest kept unit                         */
    int64_t tau_id;    /* global id of the weakest kept unit, -1 if k == 0     */
    int64_t n_gt;      /* units with key  > tau                                */
    int64_t n_tie;     /* units with key == tau                                */
    int64_t n_tie_kept;/* of those, how many are kept (lowest ids first)       */
    float tau_norm;    /* structured: (float)sqrt(nu) of the weakest kept unit */
} orc_result;

/* ---- bit helpers ------------------------------------------------------- */
static uint32_t f32_bits(float x) { uint32_t b; memcpy(&b, &x, 4); return b; }
static float bits_f32(uint32_t b) { float x; memcpy(&x, &b, 4); return x; }
static uint64_t f64_bits(double x) { uint64_t b; memcpy(&b, &x, 8); return b; }

/* Z = round(s * n): half-up rounding of the product taken in double. */
int64_t orc_round_count(double s, int64_t n)
{
    double z = floor(s * (double)n + 0.5);
    if (z < 0.0) z = 0.0;
    if (z > (double)n) z = (double)n;
    return (int64_t)z;
}

/* ---- binary32 -> binary16, round to nearest even ------------------------ */
/* Returns the 16 bits. NaN maps to a quiet NaN that keeps the sign and drops
 * the payload; overflow goes to infinity; results below the smallest normal
 * are denormalised gradually. */
uint16_t orc_f32_to_f16(uint32_t b)
{
    uint32_t sign = (b >> 16) & 0x8000u;
    uint32_t e = (b >> 23) & 0xFFu;
    uint32_t m = b & 0x7FFFFFu;
    if (e == 0xFFu) {
        if (m != 0) return (uint16_t)(sign | 0x7E00u);
        return (uint16_t)(sign | 0x7C00u);
    }
    int32_t eh = (int32_t)e - 127 + 15;          /* exponent in binary16 bias */
    if (eh >= 31) return (uint16_t)(sign | 0x7C00u);
    if (eh <= 0) {
        /* subnormal half or zero: value = (1.m) * 2^(e-127); the half
         * subnormal unit is 2^-24. Shift the 24-bit significand right. */
        if (e == 0) return (uint16_t)sign;        /* fp32 subnormals are < 2^-126: round to 0 */
        int32_t shift = 14 - eh;                  /* >= 14 */
        if (shift > 25) return (uint16_t)sign;
        uint32_t sig = m | 0x800000u;
        uint32_t q = sig >> shift;
        uint32_t rem = sig & ((1u << shift) - 1u);
        uint32_t half = 1u << (shift - 1);
        if (rem > half || (rem == half && (q & 1u))) q += 1u;
        return (uint16_t)(sign | q);              /* q may carry into the normal range: still right */
    }
    uint32_t q = ((uint32_t)eh << 10) | (m >> 13);
    uint32_t rem = m & 0x1FFFu;
    if (rem > 0x1000u || (rem == 0x1000u && (q & 1u))) q += 1u;   /* may carry to the exponent / inf */
    return (uint16_t)(sign | q);
}

/* binary16 -> binary32, exact. */
uint32_t orc_f16_to_f32(uint16_t h)
{
    uint32_t sign = ((uint32_t)h & 0x8000u) << 16;
    uint32_t e = (h >> 10) & 0x1Fu;
    uint32_t m = h & 0x3FFu;
    if (e == 31) return sign | 0x7F800000u | (m << 13);
    if (e == 0) {
        if (m == 0) return sign;
        /* normalise the subnormal */
        int32_t ex = -14;
        while (!(m & 0x400u)) { m <<= 1; ex -= 1; }
        m &= 0x3FFu;
        return sign | ((uint32_t)(ex + 127) << 23) | (m << 13);
    }
    return sign | ((e - 15 + 127) << 23) | (m << 13);
}

/* binary32 -> bfloat16 (1 sign, 8 exponent, 7 fraction bits: the upper half of a
 * binary32), round to nearest even; NaN -> quiet NaN with the sign kept. A carry
 * out of the fraction moves to the exponent, up to infinity, as IEEE rounding wants. */
uint16_t orc_f32_to_bf16(uint32_t b)
{
    if ((b & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)(((b >> 16) & 0x8000u) | 0x7FC0u);
    uint32_t lower = b & 0xFFFFu, q = b >> 16;
    if (lower > 0x8000u || (lower == 0x8000u && (q & 1u))) q += 1u;
    return (uint16_t)q;
}

/* ---- binary32 -> 8-bit floating point (Table 1, Quantize(dtype); Conclusion: further
 * data types for quantization) -------------------------------------------------
 * Two formats (Micikevicius et al., "FP8 formats for deep learning", 2022):
 *   fmt 0  E4M3: 1 sign, 4 exponent (bias 7), 3 fraction bits; no infinities, the one
 *          NaN is S.1111.111; largest finite value 448 = S.1111.110.
 *   fmt 1  E5M2: 1 sign, 5 exponent (bias 15), 2 fraction bits, laid out like IEEE;
 *          largest finite value 57344 = S.11110.11.
 * Rounding is to nearest, ties to even, with gradual underflow. Reading taken for the
 * range: the conversion SATURATES - whatever rounds beyond the largest finite value,
 * infinities included, becomes that value with its sign (the formats' saturating mode,
 * and what the conversion instruction of the GPU does); an 8-bit weight format with
 * infinities in it would be of no use as a codebook. NaN maps to S.1111111. */
uint8_t orc_f32_to_fp8(uint32_t b, int fmt)
{
    const int M = fmt ? 2 : 3, bias = fmt ? 15 : 7;
    const uint32_t maxcode = fmt ? 0x7Bu : 0x7Eu;
    uint32_t sign = (b >> 24) & 0x80u;
    uint32_t e = (b >> 23) & 0xFFu;
    uint32_t m = b & 0x7FFFFFu;
    if (e == 0xFFu) return (uint8_t)(sign | (m ? 0x7Fu : maxcode));
    if (e == 0) return (uint8_t)sign;                      /* below 2^-126: far under the smallest code */
    int32_t eh = (int32_t)e - 127 + bias;                  /* exponent field if the value is normal there */
    uint32_t q;
    if (eh >= 1) {
        int drop = 23 - M;
        q = ((uint32_t)eh << M) | (m >> drop);
        uint32_t rem = m & ((1u << drop) - 1u), half = 1u << (drop - 1);
        if (rem > half || (rem == half && (q & 1u))) q += 1u;     /* may carry into the exponent */
        if (q > maxcode) q = maxcode;
    } else {
        int shift = (23 - M) + (1 - eh);                   /* the significand in units of the smallest subnormal */
        if (shift > 25) return (uint8_t)sign;
        uint32_t sig = m | 0x800000u;
        q = sig >> shift;
        uint32_t rem = sig & ((1u << shift) - 1u), half = 1u << (shift - 1);
        if (rem > half || (rem == half && (q & 1u))) q += 1u;     /* may reach the smallest normal: still right */
    }
    return (uint8_t)(sign | q);
}

/* 8-bit floating point -> binary32, exact. */
uint32_t orc_fp8_to_f32(uint8_t h, int fmt)
{
    const int M = fmt ? 2 : 3, E = fmt ? 5 : 4, bias = fmt ? 15 : 7;
    uint32_t sign = ((uint32_t)h & 0x80u) << 24;
    uint32_t e = ((uint32_t)h >> M) & ((1u << E) - 1u);
    uint32_t m = (uint32_t)h & ((1u << M) - 1u);
    if (fmt == 0 && e == 15u && m == 7u) return sign | 0x7FC00000u;
    if (fmt == 1 && e == 31u) return sign | 0x7F800000u | (m ? 0x400000u : 0u);
    if (e == 0) {
        if (m == 0) return sign;
        int32_t ex = 1 - bias;                             /* value = m * 2^(1 - bias - M): normalise */
        while (!(m & (1u << M))) { m <<= 1; ex -= 1; }
        m &= (1u << M) - 1u;
        return sign | ((uint32_t)(ex + 127) << 23) | (m << (23 - M));
    }
    return sign | ((e - (uint32_t)bias + 127u) << 23) | (m << (23 - M));
}

void orc_f32_to_fp8_array(const uint32_t *bits, int64_t n, int fmt, uint8_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_f32_to_fp8(bits[i], fmt);
}

void orc_f32_to_fp8_range(uint32_t first, int64_t n, int fmt, uint8_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_f32_to_fp8(first + (uint32_t)i, fmt);
}

void orc_f32_to_bf16_array(const uint32_t *bits, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_f32_to_bf16(bits[i]);
}

void orc_f32_to_bf16_range(uint32_t first, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_f32_to_bf16(first + (uint32_t)i);
}

void orc_f32_to_f16_array(const uint32_t *bits, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_f32_to_f16(bits[i]);
}

/* Convert the contiguous range of bit patterns [first, first + n). */
void orc_f32_to_f16_range(uint32_t first, int64_t n, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = orc_f32_to_f16(first + (uint32_t)i);
}

/* ---- elementwise pieces ------------------------------------------------ */
/* u = w - lambda / mu, two fp32 operations. */
void orc_form_u(const float *w, const float *lambda, float mu, int64_t n, float *u)
{
    for (int64_t i = 0; i < n; ++i) {
        if (lambda) {
            volatile float q = lambda[i] / mu;
            u[i] = w[i] - q;
        } else {
            u[i] = w[i];
        }
    }
}

/* Multiplier update and penalty gradient for one tensor, theta given.
 *   d = w - theta;  p = mu * d;  lambda' = lambda - p   (if FUSE_LAMBDA)
 *   g = p - lambda_used, lambda_used = lambda' when updated, else lambda. */
void orc_lagrange(const float *w, const float *theta, const float *lambda, float mu,
                  unsigned fuse, int64_t n, float *lambda_out, float *grad)
{
    for (int64_t i = 0; i < n; ++i) {
        float lam = lambda ? lambda[i] : 0.0f;
        volatile float d = w[i] - theta[i];
        volatile float p = mu * d;
        float lam_used = lam;
        if ((fuse & ORC_FUSE_LAMBDA) && lambda) {
            volatile float l2 = lam - p;
            lam_used = l2;
        }
        if (lambda_out) lambda_out[i] = lam_used;
        if ((fuse & ORC_FUSE_PENALTY) && grad) {
            volatile float g = p - lam_used;
            grad[i] = g;
        }
    }
}

/* theta (and mask, fp16 bits) for one tensor from u and a 0/1 keep decision
 * per element, then the multiplier / penalty arithmetic. */
static void finish_tensor(const orc_tensor *t, const float *u, const uint8_t *keep, float mu,
                          unsigned fuse)
{
    for (int64_t i = 0; i < t->numel; ++i) {
        uint32_t tb = 0u;
        uint16_t hb = 0u;
        if (keep[i]) {
            if (fuse & (ORC_FUSE_E4M3 | ORC_FUSE_E5M2)) {
                int fmt = (fuse & ORC_FUSE_E5M2) ? 1 : 0;
                hb = orc_f32_to_fp8(f32_bits(u[i]), fmt);   /* the 8-bit code, in the low byte */
                tb = orc_fp8_to_f32((uint8_t)hb, fmt);
            } else if (fuse & ORC_FUSE_BF16) {
                hb = orc_f32_to_bf16(f32_bits(u[i]));
                tb = (uint32_t)hb << 16;              /* exact widening */
            } else if (fuse & ORC_FUSE_FP16) {
                hb = orc_f32_to_f16(f32_bits(u[i]));
                tb = orc_f16_to_f32(hb);
            } else {
                tb = f32_bits(u[i]);
                hb = orc_f32_to_f16(tb);
            }
        }
        t->theta[i] = bits_f32(tb);
        if (t->mask) t->mask[i] = keep[i];
        if (t->theta_h) t->theta_h[i] = hb;
    }
    orc_lagrange(t->w, t->theta, t->lambda, mu, fuse, t->numel, t->lambda_out, t->grad);
}

/* ---- ranking ----------------------------------------------------------- */
typedef struct { uint64_t key; int64_t id; } unit_t;

/* Larger key first; among equal keys the lower id first. A total order, so
 * any comparison sort gives the same sequence as a stable descending sort. */
static int unit_cmp(const void *a, const void *b)
{
    const unit_t *x = (const unit_t *)a, *y = (const unit_t *)b;
    if (x->key != y->key) return (x->key > y->key) ? -1 : 1;
    if (x->id != y->id) return (x->id < y->id) ? -1 : 1;
    return 0;
}

/* Sort units, mark the first k as kept in keep_unit[id], fill the record. */
static void rank_units(unit_t *units, int64_t n, double s, uint8_t *keep_unit, orc_result *r,
                       uint64_t inf_key)
{
    int64_t z = orc_round_count(s, n);
    int64_t k = n - z;
    qsort(units, (size_t)n, sizeof(unit_t), unit_cmp);
    for (int64_t i = 0; i < n; ++i) keep_unit[units[i].id] = (uint8_t)(i < k);
    memset(r, 0, sizeof(*r));
    r->n_units = n; r->n_zero = z; r->n_keep = k;
    if (k == 0) {
        r->tau_key = inf_key; r->tau_id = -1;
        return;
    }
    uint64_t tau = units[k - 1].key;
    r->tau_key = tau;
    r->tau_id = units[k - 1].id;
    for (int64_t i = 0; i < n; ++i) {
        if (units[i].key > tau) r->n_gt++;
        else if (units[i].key == tau) { r->n_tie++; if (i < k) r->n_tie_kept++; }
    }
}

/* Unstructured magnitude pruning over the whole list (Table 1, Prune()). */
int orc_cstep_prune(const orc_tensor *ts, int32_t T, double s, float mu, unsigned fuse,
                    orc_result *res)
{
    int64_t N = 0;
    for (int32_t t = 0; t < T; ++t) N += ts[t].numel;
    float *u = (float *)malloc(sizeof(float) * (size_t)(N ? N : 1));
    unit_t *units = (unit_t *)malloc(sizeof(unit_t) * (size_t)(N ? N : 1));
    uint8_t *keep = (uint8_t *)malloc((size_t)(N ? N : 1));
    if (!u || !units || !keep) { free(u); free(units); free(keep); return -1; }
    int64_t off = 0;
    for (int32_t t = 0; t < T; ++t) {
        orc_form_u(ts[t].w, ts[t].lambda, mu, ts[t].numel, u + off);
        for (int64_t i = 0; i < ts[t].numel; ++i) {
            units[off + i].key = (uint64_t)(f32_bits(u[off + i]) & 0x7FFFFFFFu);
            units[off + i].id = off + i;
        }
        off += ts[t].numel;
    }
    rank_units(units, N, s, keep, res, 0x7F800000ull);
    off = 0;
    for (int32_t t = 0; t < T; ++t) {
        finish_tensor(&ts[t], u + off, keep + off, mu, fuse);
        off += ts[t].numel;
    }
    free(u); free(units); free(keep);
    return 0;
}

/* ---- structured pruning ---------------------------------------------------
 * A structure specification (Table 1: NeuronPrune / FilterPrune / StructurePrune
 * aggregate 1-D / 3-D blocks, BlockPrune(criteria, bs) aggregates n-D blocks of
 * size bs; each prunes "based on criteria"):
 *   kind 0  leading-index slices: filters [f, :, :, :] of 4-D tensors (kinds & 1)
 *           and/or neurons = rows [r, :] of 2-D tensors (kinds & 2);
 *   kind 1  n-D blocks: every tensor with ndim == nd is cut into blocks of
 *           bs[0] x ... x bs[nd-1] elements, numbered row-major over the grid of
 *           blocks; a block that sticks out over an edge holds only the elements
 *           that exist.
 * crit: the value a structure is ranked by, accumulated in fp64 over its elements
 * in row-major order: 0 = sum of u^2 (the squared L2 norm: the argmin of Section
 * 3.3), 1 = sum of |u| (L1 norm), 2 = max |u|. The paper names no criterion; L1 and
 * max are the usual alternatives and are NOT the argmin. Every other tensor
 * passes through unpruned. */
typedef struct {
    int32_t kind, kinds, nd, crit;
    int64_t bs[4];
} orc_spec;

static int spec_ranks(const orc_spec *sp, const orc_tensor *t)
{
    if (t->numel == 0) return 0;
    if (sp->kind == 0) return (t->ndim == 4 && (sp->kinds & 1)) || (t->ndim == 2 && (sp->kinds & 2));
    return t->ndim == sp->nd;
}

static int64_t structure_count(const orc_spec *sp, const orc_tensor *t)
{
    if (!spec_ranks(sp, t)) return 0;
    if (sp->kind == 0) return t->shape[0];
    int64_t n = 1;
    for (int d = 0; d < sp->nd; ++d) n *= (t->shape[d] + sp->bs[d] - 1) / sp->bs[d];
    return n;
}

/* Structure (numbered inside its tensor) that holds element i. */
static int64_t structure_of(const orc_spec *sp, const orc_tensor *t, int64_t i)
{
    if (sp->kind == 0) return i / (t->numel / t->shape[0]);
    int64_t coord[4], rest = i;
    for (int d = sp->nd - 1; d >= 0; --d) { coord[d] = rest % t->shape[d]; rest /= t->shape[d]; }
    int64_t id = 0;
    for (int d = 0; d < sp->nd; ++d)
        id = id * ((t->shape[d] + sp->bs[d] - 1) / sp->bs[d]) + coord[d] / sp->bs[d];
    return id;
}

static double crit_add(double acc, float u, int crit)
{
    double x = (double)u;
    if (crit == 0) return acc + x * x;
    if (crit == 1) return acc + fabs(x);
    double a = fabs(x);
    return (a > acc || a != a) ? a : acc;      /* a NaN element makes the value NaN (ranks first) */
}

static void structure_values(const orc_spec *sp, const orc_tensor *t, const float *u, double *nu)
{
    if (sp->kind == 0) {
        int64_t len = t->numel / t->shape[0];
        for (int64_t f = 0; f < t->shape[0]; ++f) {
            double acc = 0.0;
            for (int64_t j = 0; j < len; ++j) acc = crit_add(acc, u[f * len + j], sp->crit);
            nu[f] = acc;
        }
        return;
    }
    int64_t nb[4] = {1, 1, 1, 1}, sh[4] = {1, 1, 1, 1}, bs[4] = {1, 1, 1, 1};
    /* right-align to four dimensions so that one loop nest serves every nd */
    for (int d = 0; d < sp->nd; ++d) {
        sh[4 - sp->nd + d] = t->shape[d];
        bs[4 - sp->nd + d] = sp->bs[d];
    }
    for (int d = 0; d < 4; ++d) nb[d] = (sh[d] + bs[d] - 1) / bs[d];
    int64_t id = 0;
    for (int64_t b0 = 0; b0 < nb[0]; ++b0)
    for (int64_t b1 = 0; b1 < nb[1]; ++b1)
    for (int64_t b2 = 0; b2 < nb[2]; ++b2)
    for (int64_t b3 = 0; b3 < nb[3]; ++b3) {
        double acc = 0.0;
        for (int64_t i0 = b0 * bs[0]; i0 < (b0 + 1) * bs[0] && i0 < sh[0]; ++i0)
        for (int64_t i1 = b1 * bs[1]; i1 < (b1 + 1) * bs[1] && i1 < sh[1]; ++i1)
        for (int64_t i2 = b2 * bs[2]; i2 < (b2 + 1) * bs[2] && i2 < sh[2]; ++i2)
        for (int64_t i3 = b3 * bs[3]; i3 < (b3 + 1) * bs[3] && i3 < sh[3]; ++i3)
            acc = crit_add(acc, u[((i0 * sh[1] + i1) * sh[2] + i2) * sh[3] + i3], sp->crit);
        nu[id++] = acc;
    }
}

/* The ranked value of every structure in the list, in global structure order; returns
 * the count. nu may be NULL to only count. */
int64_t orc_structure_values(const orc_tensor *ts, int32_t T, float mu, const orc_spec *sp, double *nu)
{
    int64_t S = 0;
    for (int32_t t = 0; t < T; ++t) {
        int64_t c = structure_count(sp, &ts[t]);
        if (c && nu) {
            float *u = (float *)malloc(sizeof(float) * (size_t)ts[t].numel);
            orc_form_u(ts[t].w, ts[t].lambda, mu, ts[t].numel, u);
            structure_values(sp, &ts[t], u, nu + S);
            free(u);
        }
        S += c;
    }
    return S;
}

/* Older form of the same: kind 0 with the slice mask in `bh`, or kind 1 with 2-D
 * bh x bw blocks; squared L2 norm. */
int64_t orc_structure_norms(const orc_tensor *ts, int32_t T, float mu, int kind, int bh, int bw,
                            double *nu)
{
    orc_spec sp;
    memset(&sp, 0, sizeof(sp));
    sp.kind = kind;
    if (kind == 0) sp.kinds = bh; else { sp.nd = 2; sp.bs[0] = bh; sp.bs[1] = bw; }
    return orc_structure_values(ts, T, mu, &sp, nu);
}

int orc_cstep_structured(const orc_tensor *ts, int32_t T, double s, float mu, const orc_spec *sp,
                         unsigned fuse, orc_result *res)
{
    if (sp->kind == 0 && (sp->kinds < 1 || sp->kinds > 3)) return -2;
    if (sp->kind == 1) {
        if (sp->nd < 1 || sp->nd > 4) return -2;
        for (int d = 0; d < sp->nd; ++d) if (sp->bs[d] < 1) return -2;
    }
    if (sp->crit < 0 || sp->crit > 2) return -2;
    int64_t S = orc_structure_values(ts, T, mu, sp, NULL);
    double *nu = (double *)malloc(sizeof(double) * (size_t)(S ? S : 1));
    unit_t *units = (unit_t *)malloc(sizeof(unit_t) * (size_t)(S ? S : 1));
    uint8_t *keep_s = (uint8_t *)malloc((size_t)(S ? S : 1));
    if (!nu || !units || !keep_s) { free(nu); free(units); free(keep_s); return -1; }
    orc_structure_values(ts, T, mu, sp, nu);
    for (int64_t i = 0; i < S; ++i) { units[i].key = f64_bits(nu[i]); units[i].id = i; }
    rank_units(units, S, s, keep_s, res, 0x7FF0000000000000ull);
    /* reported value of the weakest kept structure: the norm for the L2 criterion, else the value itself */
    if (res->n_keep > 0) res->tau_norm = sp->crit == 0 ? (float)sqrt(nu[res->tau_id]) : (float)nu[res->tau_id];
    int64_t sbase = 0;
    for (int32_t t = 0; t < T; ++t) {
        int64_t n = ts[t].numel;
        int64_t c = structure_count(sp, &ts[t]);
        float *u = (float *)malloc(sizeof(float) * (size_t)(n ? n : 1));
        uint8_t *keep = (uint8_t *)malloc((size_t)(n ? n : 1));
        orc_form_u(ts[t].w, ts[t].lambda, mu, n, u);
        for (int64_t i = 0; i < n; ++i)
            keep[i] = c ? keep_s[sbase + structure_of(sp, &ts[t], i)] : 1;
        finish_tensor(&ts[t], u, keep, mu, fuse);
        free(u); free(keep);
        sbase += c;
    }
    free(nu); free(units); free(keep_s);
    return 0;
}

/* Filter pruning (Table 1, FilterPrune): 4-D tensors are ranked by filter,
 * every other tensor passes through unpruned (theta = u, mask = 1). */
int orc_cstep_filter(const orc_tensor *ts, int32_t T, double s, float mu, unsigned fuse,
                     orc_result *res)
{
    orc_spec sp;
    memset(&sp, 0, sizeof(sp));
    sp.kinds = 1;
    return orc_cstep_structured(ts, T, s, mu, &sp, fuse, res);
}

/* NeuronPrune / FilterPrune / StructurePrune in one call: `kinds` is the mask
 * 1 = filters of 4-D tensors, 2 = neurons (rows) of 2-D tensors. */
int orc_cstep_structure(const orc_tensor *ts, int32_t T, double s, float mu, int kinds, unsigned fuse,
                        orc_result *res)
{
    orc_spec sp;
    memset(&sp, 0, sizeof(sp));
    sp.kinds = kinds;
    return orc_cstep_structured(ts, T, s, mu, &sp, fuse, res);
}

/* Block pruning (Table 1, BlockPrune): 2-D tensors are ranked by bh x bw
 * block, every other tensor passes through unpruned. */
int orc_cstep_block(const orc_tensor *ts, int32_t T, double s, float mu, int bh, int bw,
                    unsigned fuse, orc_result *res)
{
    if (bh < 1 || bw < 1) return -2;
    orc_spec sp;
    memset(&sp, 0, sizeof(sp));
    sp.kind = 1; sp.nd = 2; sp.bs[0] = bh; sp.bs[1] = bw;
    return orc_cstep_structured(ts, T, s, mu, &sp, fuse, res);
}

unsigned orc_sizeof_spec(void) { return (unsigned)sizeof(orc_spec); }

/* Quantisation only (Table 1, Quantize(dtype)): theta = Q(u), mask = 1. The type is
 * binary16 unless `fuse` carries ORC_FUSE_BF16, ORC_FUSE_E4M3 or ORC_FUSE_E5M2. */
int orc_cstep_quantize(const orc_tensor *ts, int32_t T, float mu, unsigned fuse)
{
    for (int32_t t = 0; t < T; ++t) {
        int64_t n = ts[t].numel;
        float *u = (float *)malloc(sizeof(float) * (size_t)(n ? n : 1));
        uint8_t *keep = (uint8_t *)malloc((size_t)(n ? n : 1));
        orc_form_u(ts[t].w, ts[t].lambda, mu, n, u);
        memset(keep, 1, (size_t)n);
        finish_tensor(&ts[t], u, keep, mu, (fuse & (ORC_FUSE_BF16 | ORC_FUSE_E4M3 | ORC_FUSE_E5M2)) ? fuse : (fuse | ORC_FUSE_FP16));
        free(u); free(keep);
    }
    return 0;
}

/* Multiplier update / penalty gradient with theta supplied by the caller. */
int orc_lagrange_update(const orc_tensor *ts, int32_t T, float mu, unsigned fuse)
{
    for (int32_t t = 0; t < T; ++t)
        orc_lagrange(ts[t].w, ts[t].theta, ts[t].lambda, mu, fuse, ts[t].numel,
                     ts[t].lambda_out, ts[t].grad);
    return 0;
}

/* ---- L step: penalty gradient folded into the optimizer update ------------
 * The L step trains w on the loss plus the quadratic penalty (Section 3.3, "a
 * learning (L) step which trains the uncompressed model but with a quadratic
 * regularization term"), with SGD momentum 0.9 for the CNNs and Adam for the
 * LSTM (Evaluation, L-C optimizer settings). Every minibatch adds the penalty
 * gradient mu (w - theta) - lambda to the loss gradient and takes one
 * optimizer step; written here one fp32 operation at a time:
 *   d = w - theta; p = mu d; g1 = p - lambda; g = grad + g1; [g = g + wd w]
 *   SGD : b' = momentum b + g;  w' = w - lr b'
 *   Adam: m' = beta1 m + (1-beta1) g;  v' = beta2 v + (1-beta2) g g;
 *         w' = w - (lr / (1-beta1^t)) * m' / (sqrt(v') / sqrt(1-beta2^t) + eps)
 * (the usual SGD-with-momentum and Adam recurrences, bias correction included). */
typedef struct {
    float *w;              /* in/out */
    const float *theta;
    const float *lambda;   /* may be NULL */
    const float *grad;     /* loss gradient */
    float *buf1;           /* SGD momentum buffer / Adam first moment, in/out   */
    float *buf2;           /* Adam second moment, in/out                         */
    int64_t numel;
} orc_opt_tensor;

typedef struct {
    int32_t kind;          /* 0 = SGD with momentum, 1 = Adam */
    float lr, momentum, weight_decay, beta1, beta2, eps;
    int64_t step;          /* Adam: 1-based step number t */
} orc_opt;

int orc_lstep_update(const orc_opt_tensor *ts, int32_t T, float mu, const orc_opt *o)
{
    volatile float c1 = 1.0f - o->beta1, c2 = 1.0f - o->beta2;
    double bc1 = 1.0 - pow((double)o->beta1, (double)o->step);
    double bc2 = 1.0 - pow((double)o->beta2, (double)o->step);
    float step_size = (float)((double)o->lr / bc1);
    float sqrt_bc2 = (float)sqrt(bc2);
    for (int32_t t = 0; t < T; ++t) {
        const orc_opt_tensor *x = &ts[t];
        for (int64_t i = 0; i < x->numel; ++i) {
            volatile float d = x->w[i] - x->theta[i];
            volatile float p = mu * d;
            volatile float g1 = x->lambda ? p - x->lambda[i] : p;
            volatile float g = x->grad[i] + g1;
            if (o->weight_decay != 0.0f) {
                volatile float wd = o->weight_decay * x->w[i];
                g = g + wd;
            }
            if (o->kind == 0) {
                volatile float b = g;
                if (x->buf1) {
                    volatile float a = o->momentum * x->buf1[i];
                    b = a + g;
                    x->buf1[i] = b;
                }
                volatile float s = o->lr * b;
                x->w[i] = x->w[i] - s;
            } else {
                volatile float a = o->beta1 * x->buf1[i];
                volatile float b = c1 * g;
                volatile float m = a + b;
                volatile float a2 = o->beta2 * x->buf2[i];
                volatile float gg = g * g;
                volatile float b2 = c2 * gg;
                volatile float v = a2 + b2;
                x->buf1[i] = m;
                x->buf2[i] = v;
                volatile float sq = sqrtf(v);
                volatile float dn = sq / sqrt_bc2;
                dn = dn + o->eps;
                volatile float q = m / dn;
                volatile float s = step_size * q;
                x->w[i] = x->w[i] - s;
            }
        }
    }
    return 0;
}

unsigned orc_sizeof_opt_tensor(void) { return (unsigned)sizeof(orc_opt_tensor); }
unsigned orc_sizeof_opt(void) { return (unsigned)sizeof(orc_opt); }

/* 1 when subnormal fp32 arithmetic is intact in this process (no flush to
 * zero, no denormals-are-zero), which every function above relies on. */
int orc_denormals_ok(void)
{
    volatile float tiny = bits_f32(0x00000001u);
    volatile float two = 2.0f;
    volatile float r = tiny * two;
    volatile float mn = bits_f32(0x00800000u);
    volatile float half = 0.5f;
    volatile float r2 = mn * half;
    return f32_bits(r) == 0x00000002u && f32_bits(r2) == 0x00400000u;
}

unsigned orc_sizeof_tensor(void) { return (unsigned)sizeof(orc_tensor); }
unsigned orc_sizeof_result(void) { return (unsigned)sizeof(orc_result); }
