/*
 * Tri-Accel optimizer pass -- CPU ORACLE.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain restatement of the
 * paper's equations that the CUDA library is checked against.  It shares no
 * code, header, table or helper with the CUDA path and must never be linked,
 * imported or called by it.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may use it.
 *
 * Arithmetic: double for every sum and for the scalar recurrences, stored
 * per-layer state rounded to float where the method keeps float state.
 * No blocking, no SIMD, no threads: one loop per equation.
 *
 * What each function follows:
 *   orc_moments            Sec. 3.1, the Var[grad_l(t)] term of the v_l(t) recurrence
 *   EMA update             Sec. 3.1, v_l(t) = beta v_l(t-1) + (1-beta) Var[...]
 *   precision code         Sec. 3.1, the three-case rule for p_l(t)
 *   curvature signal       Abstract / Sec. 1 ("top-k Hessian or Fisher entries"),
 *                          read as a Hutchinson diagonal z*(Hz) with a per-layer
 *                          top-k magnitude mask; Sec. 3.2 max_{i<=k} lambda_i
 *   step size              Sec. 3.2, eta_l(t) = eta_0 / (1 + alpha * max lambda)
 *   promotion              Sec. 3.2, curvature above tau_curv raises precision
 *   control interval       Sec. 3.4, decisions every T_ctrl steps
 *   master update + cast   Sec. 2 (FP32 master copy, low-precision working copy),
 *                          Sec. 3.2 (per-layer step size), Sec. 4.1 (SGD)
 *   orc_power_iterate      Sec. 3.2, u <- H u / ||H u||, lambda ~ u^T H u / u^T u (with deflation for top-k)
 *   orc_batch_next         Sec. 3.3, the three-branch rule for B(t+1)
 *   orc_philox4x32_10      Salmon, Moraes, Dror, Shaw: "Parallel random numbers:
 *                          as easy as 1, 2, 3" (SC'11), Philox-4x32, 10 rounds.
 *                          The paper names no generator; this one is this
 *                          library's choice for the Rademacher probes.
 *
 * Pins (tests/, CPU only): Philox known-answer vectors; exact rational brute
 * force for the moments; EMA closed form; Hz = D*z  =>  estimate == D;
 * all 2^n sign vectors on a dense symmetric H; full-sort brute force for the
 * mask; power iteration against a dense symmetric eigensolver; exhaustive rounding-class enumeration of both casts against numpy /
 * torch conversions; boundary and monotonicity cases of the code rule.
 * Unpinned: the end-to-end trajectory over many steps (the paper prints no
 * worked example); it is pinned only through its parts.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct { uint64_t offset, length; } orc_segment;

typedef struct {
    float beta, tau_low, tau_high, tau_curv, alpha, eta0;
    uint32_t topk_ppm;    /* parts per million of each layer kept in the mask */
    uint32_t num_probes;  /* P */
    uint32_t t_ctrl;      /* control interval, >= 1 */
    uint32_t grad_dtype;  /* 0 = float, 1 = bfloat16 */
    float momentum;       /* SGD momentum (Sec. 4.1 names 0.9 for the baselines); 0 = none */
    float weight_decay;   /* L2 coefficient added to the gradient; 0 = none */
} orc_hparams;

typedef struct {
    double grad_mean, grad_var;      /* this step's moments (double) */
    double topk_mass;                /* sum masked |S| / sum all |S| */
    float ema_mean, ema_var;         /* m_l, v_l */
    float lambda_max;                /* max |S| / P */
    float topk_threshold;            /* k-th largest |S| */
    float eta_scale;                 /* s_l = 1 / (1 + alpha lambda) */
    uint32_t code;                   /* 0 FP16, 1 BF16, 2 FP32 */
    uint64_t k;                      /* mask population */
    uint32_t near_threshold;         /* a statistic within 1e-5 of a threshold */
    uint32_t pad;
} orc_layer;

typedef struct {
    uint64_t step;
    uint64_t nonfinite_count;
    uint32_t skipped;
    uint32_t near_threshold_count;
} orc_status;

typedef struct {
    uint32_t L;
    uint64_t n_total;
    orc_segment *seg;
    orc_hparams hp;
    orc_layer *layer;
    uint32_t *mask;       /* one bit per flat element, bit (i & 31) of word i >> 5 */
    uint64_t mask_words;
    float *mom;           /* momentum buffer, one float per flat element, starts at zero */
    orc_status status;
} orc_state;

/* ---------------------------------------------------------------- Philox */

void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * Rademacher bit of flat element i for probe p at step t.
 * The flat index space is cut into blocks of 4096 elements.  Inside a block,
 * element r = i mod 4096 sits in row r / 128 (32 rows), at slot (r / 4) mod 32
 * of its row, component r mod 4.  All 128 elements of one slot column (32 rows
 * x 4 components) take their bits from ONE Philox call:
 *   counter = (q_lo, q_hi, t, p),  q = 32 * (i / 4096) + slot,  key = seed
 *   bit number 4 * row + component of the 128-bit output (word = bit / 32).
 * z = +1 when the bit is 0, -1 when it is 1.  A pure function of (seed,t,p,i).
 */
uint32_t orc_rademacher_bit(uint64_t seed, uint64_t t, uint32_t p, uint64_t i)
{
    uint64_t block = i >> 12;
    uint32_t r = (uint32_t)(i & 4095u);
    uint32_t row = r >> 7, slot = (r >> 2) & 31u, comp = r & 3u;
    uint64_t q = block * 32u + slot;
    uint32_t ctr[4] = { (uint32_t)q, (uint32_t)(q >> 32), (uint32_t)t, p };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    uint32_t bit = 4u * row + comp;
    return (out[bit >> 5] >> (bit & 31u)) & 1u;
}

/* z for flat elements [first, first + n): +1.0f or -1.0f */
void orc_probe(uint64_t seed, uint64_t t, uint32_t p, uint64_t first, uint64_t n, float *z_out)
{
    for (uint64_t j = 0; j < n; ++j)
        z_out[j] = orc_rademacher_bit(seed, t, p, first + j) ? -1.0f : 1.0f;
}

/* ---------------------------------------------------------------- casts */

static uint32_t f32_bits(float x) { uint32_t u; memcpy(&u, &x, 4); return u; }
static float bits_f32(uint32_t u) { float x; memcpy(&x, &u, 4); return x; }

float orc_bf16_to_f32(uint16_t h) { return bits_f32((uint32_t)h << 16); }

/* float -> bfloat16, round to nearest, ties to even; NaN stays NaN (quiet) */
uint16_t orc_f32_to_bf16(float x)
{
    uint32_t u = f32_bits(x);
    if ((u & 0x7F800000u) == 0x7F800000u && (u & 0x007FFFFFu))
        return (uint16_t)((u >> 16) | 0x0040u);
    uint32_t keep = u >> 16;
    uint32_t rest = u & 0xFFFFu;
    if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u)))
        keep += 1u;                 /* carries into exponent, up to inf, correctly */
    return (uint16_t)keep;
}

/* float -> IEEE binary16, round to nearest even, subnormals kept, overflow -> inf */
uint16_t orc_f32_to_f16(float x)
{
    uint32_t u = f32_bits(x);
    uint16_t sign = (uint16_t)((u >> 16) & 0x8000u);
    uint32_t expo = (u >> 23) & 0xFFu;
    uint32_t man = u & 0x007FFFFFu;
    if (expo == 0xFFu)
        return (uint16_t)(sign | 0x7C00u | (man ? 0x0200u : 0u));
    int e = (int)expo - 127;                       /* unbiased */
    if (e > 15)
        return (uint16_t)(sign | 0x7C00u);
    if (e >= -14) {                                /* normal half, before rounding */
        uint32_t keep = ((uint32_t)(e + 15) << 10) | (man >> 13);
        uint32_t rest = man & 0x1FFFu;
        if (rest > 0x1000u || (rest == 0x1000u && (keep & 1u)))
            keep += 1u;                            /* may reach 0x7C00 = inf */
        return (uint16_t)(sign | keep);
    }
    if (expo == 0u || e < -25)                     /* below half of the smallest subnormal */
        return sign;
    /* subnormal half: value = full * 2^(e-23), unit = 2^-24 */
    uint32_t full = man | 0x00800000u;
    int shift = -e - 1;                            /* 14 .. 24 */
    uint32_t keep = full >> shift;
    uint32_t rest = full & ((1u << shift) - 1u);
    uint32_t half = 1u << (shift - 1);
    if (rest > half || (rest == half && (keep & 1u)))
        keep += 1u;
    return (uint16_t)(sign | keep);
}

void orc_cast_array(const float *x, uint64_t n, uint32_t to_bf16, uint16_t *out)
{
    for (uint64_t i = 0; i < n; ++i)
        out[i] = to_bf16 ? orc_f32_to_bf16(x[i]) : orc_f32_to_f16(x[i]);
}

/* ---------------------------------------------------------------- moments */

/* population mean and variance of x[0..n), two passes in double */
void orc_moments(const float *x, uint64_t n, double *mean, double *var)
{
    double s = 0.0;
    for (uint64_t i = 0; i < n; ++i) s += (double)x[i];
    double mu = s / (double)n;
    double q = 0.0;
    for (uint64_t i = 0; i < n; ++i) { double d = (double)x[i] - mu; q += d * d; }
    *mean = mu;
    *var = q / (double)n;
}

/* ---------------------------------------------------------------- state */

static int is_finite_f32(float x) { return (f32_bits(x) & 0x7F800000u) != 0x7F800000u; }

orc_state *orc_create(const orc_segment *table, uint32_t L, uint64_t n_total, const orc_hparams *hp)
{
    if (!table || !hp || L == 0) return NULL;
    uint64_t end = 0;
    for (uint32_t l = 0; l < L; ++l) {
        if (table[l].length == 0 || table[l].length >= 0xFFFFFFFFull || table[l].offset < end) return NULL;
        end = table[l].offset + table[l].length;
    }
    if (end > n_total) return NULL;
    if (hp->num_probes == 0 || hp->num_probes > 8 || hp->t_ctrl == 0) return NULL;
    if (hp->topk_ppm == 0 || hp->topk_ppm > 1000000u) return NULL;
    orc_state *st = (orc_state *)calloc(1, sizeof(orc_state));
    st->L = L;
    st->n_total = n_total;
    st->hp = *hp;
    st->seg = (orc_segment *)malloc(sizeof(orc_segment) * L);
    memcpy(st->seg, table, sizeof(orc_segment) * L);
    st->layer = (orc_layer *)calloc(L, sizeof(orc_layer));
    for (uint32_t l = 0; l < L; ++l) {
        st->layer[l].code = 1u;          /* BF16 is the default mode (Sec. 3.1) */
        st->layer[l].eta_scale = 1.0f;
    }
    st->mask_words = (n_total + 31u) / 32u;
    st->mask = (uint32_t *)calloc(st->mask_words ? st->mask_words : 1, sizeof(uint32_t));
    st->mom = hp->momentum != 0.0f ? (float *)calloc(n_total ? n_total : 1, sizeof(float)) : NULL;
    return st;
}

void orc_destroy(orc_state *st)
{
    if (!st) return;
    free(st->seg); free(st->layer); free(st->mask); free(st->mom); free(st);
}

void orc_set_lr(orc_state *st, float eta0) { st->hp.eta0 = eta0; }
void orc_get_layers(const orc_state *st, orc_layer *out) { memcpy(out, st->layer, sizeof(orc_layer) * st->L); }
void orc_get_status(const orc_state *st, orc_status *out) { *out = st->status; }
void orc_get_momentum(const orc_state *st, float *out) { if (st->mom) memcpy(out, st->mom, sizeof(float) * st->n_total); }
void orc_get_mask(const orc_state *st, uint32_t *out) { memcpy(out, st->mask, sizeof(uint32_t) * st->mask_words); }
uint64_t orc_mask_words(const orc_state *st) { return st->mask_words; }
uint64_t orc_sizeof_layer(void) { return sizeof(orc_layer); }

/* ---------------------------------------------------------------- top-k */

typedef struct { float a; uint32_t idx; } orc_cand;

static int cand_cmp(const void *pa, const void *pb)
{
    const orc_cand *x = (const orc_cand *)pa, *y = (const orc_cand *)pb;
    if (x->a > y->a) return -1;      /* larger magnitude first */
    if (x->a < y->a) return 1;
    if (x->idx < y->idx) return -1;  /* ties: lower index first */
    if (x->idx > y->idx) return 1;
    return 0;
}

/* balanced pairwise sum of v[0..n) in float: adjacent pairs, level by level,
 * an odd last term is carried up unchanged: ((0+1)+(2+3))+((4+5)+(6+7)) */
static float pairwise_sum_f32(float *v, uint32_t n)
{
    while (n > 1) {
        uint32_t m = 0;
        for (uint32_t j = 0; j + 1 < n; j += 2) {
            volatile float s = v[j] + v[j + 1];   /* one float rounding per add */
            v[m++] = s;
        }
        if (n & 1u) v[m++] = v[n - 1];
        n = m;
    }
    return v[0];
}

/*
 * Hutchinson magnitudes of one layer: a_j = | sum_p z_j^(p) * Hz_j^(p) |.
 * hz points at probe 0 of the flat buffer; probe p lives at hz + p * n_total.
 */
void orc_hutchinson_abs(const float *hz, uint64_t n_total, uint32_t P, uint64_t seed, uint64_t t,
                        uint64_t offset, uint64_t length, float *a_out)
{
    float term[8];
    for (uint64_t j = 0; j < length; ++j) {
        uint64_t i = offset + j;
        for (uint32_t p = 0; p < P; ++p) {
            float h = hz[(uint64_t)p * n_total + i];
            term[p] = orc_rademacher_bit(seed, t, p, i) ? -h : h;
        }
        a_out[j] = fabsf(pairwise_sum_f32(term, P));
    }
}

/* ---------------------------------------------------------------- the step */

/*
 * One optimizer pass.  w: float master weights (updated in place); g: gradients
 * (float or bfloat16 per hp.grad_dtype); hz: [P][n_total] float or NULL (then the
 * stored curvature signal is reused, Sec. 3.2: curvature only every T iterations);
 * c: 16-bit working copy (written for layers whose code is FP16 or BF16).
 * Returns 0, or 1 when the step was skipped because an input was not finite.
 */
int orc_step(orc_state *st, float *w, const void *g_any, const float *hz, uint16_t *c,
             uint64_t seed, uint64_t t)
{
    const orc_hparams *hp = &st->hp;
    const uint32_t P = hp->num_probes;
    const uint64_t N = st->n_total;

    /* widest layer, for scratch */
    uint64_t nmax = 0;
    for (uint32_t l = 0; l < st->L; ++l) if (st->seg[l].length > nmax) nmax = st->seg[l].length;
    float *gl = (float *)malloc(sizeof(float) * nmax);

    /* step 1: non-finite screen over everything the step would read */
    uint64_t bad = 0;
    for (uint32_t l = 0; l < st->L; ++l) {
        uint64_t off = st->seg[l].offset, n = st->seg[l].length;
        for (uint64_t j = 0; j < n; ++j) {
            float gv = hp->grad_dtype ? orc_bf16_to_f32(((const uint16_t *)g_any)[off + j])
                                      : ((const float *)g_any)[off + j];
            if (!is_finite_f32(gv)) ++bad;
            if (hz) for (uint32_t p = 0; p < P; ++p) if (!is_finite_f32(hz[(uint64_t)p * N + off + j])) ++bad;
        }
    }
    st->status.step = t;
    st->status.nonfinite_count = bad;
    st->status.skipped = bad ? 1u : 0u;
    if (bad) { free(gl); return 1; }

    const int control = (t % hp->t_ctrl) == 0;
    const double beta = (double)hp->beta;
    if (control) st->status.near_threshold_count = 0;

    float *a = hz ? (float *)malloc(sizeof(float) * nmax) : NULL;
    orc_cand *cand = (hz && hp->topk_ppm < 1000000u) ? (orc_cand *)malloc(sizeof(orc_cand) * nmax) : NULL;

    for (uint32_t l = 0; l < st->L; ++l) {
        orc_layer *ly = &st->layer[l];
        uint64_t off = st->seg[l].offset, n = st->seg[l].length;

        /* widen the gradient exactly */
        for (uint64_t j = 0; j < n; ++j)
            gl[j] = hp->grad_dtype ? orc_bf16_to_f32(((const uint16_t *)g_any)[off + j])
                                   : ((const float *)g_any)[off + j];

        /* step 2: moments (Sec. 3.1) */
        orc_moments(gl, n, &ly->grad_mean, &ly->grad_var);

        /* step 3: EMAs, from zero, no bias correction (Sec. 3.1) */
        ly->ema_mean = (float)(beta * (double)ly->ema_mean + (1.0 - beta) * ly->grad_mean);
        ly->ema_var  = (float)(beta * (double)ly->ema_var  + (1.0 - beta) * ly->grad_var);

        /* step 4: curvature signal */
        if (hz) {
            orc_hutchinson_abs(hz, N, P, seed, t, off, n, a);
            uint64_t k = (n * (uint64_t)hp->topk_ppm + 999999u) / 1000000u;
            if (k < 1) k = 1;
            float amax = a[0], amin = a[0];
            double sum_all = 0.0;
            for (uint64_t j = 0; j < n; ++j) {
                if (a[j] > amax) amax = a[j];
                if (a[j] < amin) amin = a[j];
                sum_all += (double)a[j];
            }
            /* clear this layer's mask bits */
            for (uint64_t j = 0; j < n; ++j) {
                uint64_t i = off + j;
                st->mask[i >> 5] &= ~(1u << (i & 31u));
            }
            double sum_masked = 0.0;
            float thr;
            if (hp->topk_ppm >= 1000000u) {
                for (uint64_t j = 0; j < n; ++j) { uint64_t i = off + j; st->mask[i >> 5] |= 1u << (i & 31u); }
                sum_masked = sum_all;
                thr = amin;
            } else {
                for (uint64_t j = 0; j < n; ++j) { cand[j].a = a[j]; cand[j].idx = (uint32_t)j; }
                qsort(cand, n, sizeof(orc_cand), cand_cmp);
                for (uint64_t r = 0; r < k; ++r) {
                    uint64_t i = off + cand[r].idx;
                    st->mask[i >> 5] |= 1u << (i & 31u);
                    sum_masked += (double)cand[r].a;
                }
                thr = cand[k - 1].a;
            }
            ly->k = k;
            ly->topk_threshold = thr;
            ly->lambda_max = amax / (float)P;
            ly->topk_mass = sum_all > 0.0 ? sum_masked / sum_all : 1.0;
        }

        /* step 5: decisions at control steps (Sec. 3.1 cases, Sec. 3.2, Sec. 3.4) */
        if (control) {
            float v = ly->ema_var;
            uint32_t code = v < hp->tau_low ? 0u : (v < hp->tau_high ? 1u : 2u);
            if (ly->lambda_max > hp->tau_curv && code < 2u) code += 1u;
            ly->code = code;
            volatile float prod = hp->alpha * ly->lambda_max;   /* three float roundings */
            volatile float den = 1.0f + prod;
            volatile float sc = 1.0f / den;
            ly->eta_scale = sc;
            uint32_t near = 0;
            if (fabs((double)v - (double)hp->tau_low) <= 1e-5 * fabs((double)hp->tau_low)) near = 1;
            if (fabs((double)v - (double)hp->tau_high) <= 1e-5 * fabs((double)hp->tau_high)) near = 1;
            if (fabs((double)ly->lambda_max - (double)hp->tau_curv) <= 1e-5 * fabs((double)hp->tau_curv)) near = 1;
            ly->near_threshold = near;
            st->status.near_threshold_count += near;
        }

        /* step 6: this layer's step size */
        volatile float eta_f = hp->eta0 * ly->eta_scale;
        double eta = (double)eta_f;

        /* step 7: master update and cast (Sec. 2 master copy; Sec. 3.2; Sec. 4.1 SGD) */
        for (uint64_t j = 0; j < n; ++j) {
            uint64_t i = off + j;
            /* SGD with weight decay and momentum (Sec. 4.1): d = g + wd w; b = mu b + d; w = w - eta b.
             * d and b are float, one rounding each (fused multiply-add); the buffer starts at zero. */
            float dir = gl[j];
            if (hp->weight_decay != 0.0f) dir = fmaf(hp->weight_decay, w[i], dir);
            if (st->mom) { dir = fmaf(hp->momentum, st->mom[i], dir); st->mom[i] = dir; }
            float wn = (float)((double)w[i] - eta * (double)dir);
            w[i] = wn;
            if (ly->code == 0u) c[i] = orc_f32_to_f16(wn);
            else if (ly->code == 1u) c[i] = orc_f32_to_bf16(wn);
        }
    }
    free(gl); free(a); free(cand);
    return 0;
}

/* ---------------------------------------------------------------- power iteration (Sec. 3.2) */

/*
 * One step of u <- H_l u / ||H_l u||, lambda ~ u^T H_l u / u^T u for every layer, with the products hu = H_l u
 * given.  m earlier eigenvectors v[j] (flat, [m][n_total]) with per-layer eigenvalues lam_v[j*L + l] are
 * deflated: t = hu - sum_j a_j v_j, a_j = float(lam_j * (v_j . u)), subtracted one after the other with one
 * float rounding each (fused multiply-add), in the order j = 0, 1, ...
 */
void orc_power_iterate(const orc_segment *table, uint32_t L, uint64_t n_total, const float *u, const float *hu,
                       const float *v, const float *lam_v, uint32_t m, float *u_next, float *lambda_out, float *norm_out)
{
    for (uint32_t l = 0; l < L; ++l) {
        const uint64_t off = table[l].offset, n = table[l].length;
        float a[8];
        for (uint32_t j = 0; j < m; ++j) {
            double dot = 0.0;
            for (uint64_t i = 0; i < n; ++i) dot += (double)v[(uint64_t)j * n_total + off + i] * (double)u[off + i];
            a[j] = (float)((double)lam_v[(uint64_t)j * L + l] * dot);
        }
        double uu = 0.0, ut = 0.0, tt = 0.0;
        for (uint64_t i = 0; i < n; ++i) {
            float t = hu[off + i];
            for (uint32_t j = 0; j < m; ++j) t = fmaf(-a[j], v[(uint64_t)j * n_total + off + i], t);
            uu += (double)u[off + i] * (double)u[off + i];
            ut += (double)u[off + i] * (double)t;
            tt += (double)t * (double)t;
        }
        const float nrm = (float)sqrt(tt);
        lambda_out[l] = uu > 0.0 ? (float)(ut / uu) : 0.0f;
        if (norm_out) norm_out[l] = nrm;
        for (uint64_t i = 0; i < n; ++i) {
            float t = hu[off + i];
            for (uint32_t j = 0; j < m; ++j) t = fmaf(-a[j], v[(uint64_t)j * n_total + off + i], t);
            volatile float q = nrm > 0.0f ? t / nrm : 0.0f;
            u_next[off + i] = q;
        }
    }
}

/* ---------------------------------------------------------------- batch rule */

/* Sec. 3.3: B+up if usage < rho_low*max; B-down if usage > rho_high*max; else B; clamped */
int64_t orc_batch_next(int64_t B, int64_t delta_up, int64_t delta_down, double rho_low, double rho_high,
                       double mem_usage, double mem_max, int64_t B_min, int64_t B_max)
{
    int64_t next = B;
    if (mem_usage < rho_low * mem_max) next = B + delta_up;
    else if (mem_usage > rho_high * mem_max) next = B - delta_down;
    if (next < B_min) next = B_min;
    if (next > B_max) next = B_max;
    return next;
}
