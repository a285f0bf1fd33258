/*
 * LASAD CPU oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, fp64 statement of what the LASAD operator (causal linear
 * attention with Spatial-Aware Decay) computes.  Only the tests, the smoke
 * check and the benchmark's CPU-baseline leg may call it; the CUDA library
 * shares no code with this file and never routes through it.
 *
 * Two forms, both written straight from the paper:
 *
 *   lasad_oracle_recurrent  -- Algorithm 1, the per-token loop body: choose the
 *       spatial decay (1 at a row-boundary step, the supplied decay otherwise),
 *       update the state  s_t = diag(lambda_t^spatial) s_{t-1} + k_t v_t^T,
 *       read out  o_t^T = q_t^T s_t   (the SAD recurrence and the SAD rule of
 *       Section 3.4).
 *
 *   lasad_oracle_quadratic  -- the same recurrence unrolled into its explicit
 *       sum over earlier tokens,
 *           o_t = sum_{s<=t} sum_c q_t[c] k_s[c] (prod_{u=s+1..t} L_u[c]) v_s ,
 *       where L_u[c] is the spatial decay of step u.  O(T^2 d).
 *
 * Decay is the paper's general form: a value per (batch, token, head, key
 * channel), addressed through four element strides so that a per-head constant
 * (data-independent decay, Section 3.3) is passed with zero strides.
 *
 * Row-boundary rule (Section 3.4, the SAD rule; Algorithm 1's if-statement):
 * with the paper's 1-based position t the decay is forced to 1 when
 * t mod w = 0.  Here positions are absolute 0-based indices i; the first
 * `prefix_len` positions are non-grid tokens (never boundaries) and the grid
 * position is i - prefix_len, so step i is a boundary iff
 *     grid_w > 0  and  i >= prefix_len  and  (i - prefix_len + 1) mod grid_w == 0.
 * prefix_len = 0 is the paper's rule verbatim.  grid_w = 0 switches the rule
 * off (plain 1-D decay, the recurrence of Section 3.3).
 *
 * Layout: q,k [B,T,H,dk], v [B,T,H,dv], o [B,T,H,dv], state [B,H,dk,dv], all
 * contiguous doubles.  state_in may be NULL (s_0 = 0); state_out may be NULL.
 *
 * A third function, lasad_oracle_layer_core, is Algorithm 1's loop body with the
 * operator's neighbours inside: q_t = SiLU(q~_t), lambda_t = Sigmoid(g~_t),
 * k_t = 1 - lambda_t (or a supplied key), the decay select, the state update and the
 * readout as above, and then Norm(o_t).  The paper does not say which norm; the
 * reading taken is a weight-free RMS norm over the d_v channels of a head,
 * o / sqrt(mean(o^2) + eps).
 *
 * Parity pins for all three functions live in tests/test_oracle_pins.py.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int32_t B, T, H, dk, dv;
    int32_t grid_w;      /* w; 0 = boundary rule off */
    int32_t prefix_len;  /* P */
    int64_t t0;          /* absolute index of the call's first token */
    double  scale;       /* multiplies o (the paper has none: 1.0) */
    int64_t decay_stride[4]; /* elements, for (b, t, h, c) */
} lasad_oracle_dims;

static int is_boundary(const lasad_oracle_dims* d, int64_t i)
{
    if (d->grid_w <= 0) return 0;
    if (i < d->prefix_len) return 0;
    return ((i - d->prefix_len + 1) % d->grid_w) == 0;
}

/* spatial decay of local step t, channel c (Algorithm 1: decay select) */
static double spatial_decay(const lasad_oracle_dims* d, const double* decay,
                            int b, int t, int h, int c)
{
    if (is_boundary(d, d->t0 + t)) return 1.0;
    return decay[b * d->decay_stride[0] + (int64_t)t * d->decay_stride[1] +
                 h * d->decay_stride[2] + c * d->decay_stride[3]];
}

int lasad_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Algorithm 1, state update and readout, one token at a time. */
int lasad_oracle_recurrent(const lasad_oracle_dims* d,
                           const double* q, const double* k, const double* v,
                           const double* decay, const double* state_in,
                           double* o, double* state_out)
{
    const int B = d->B, T = d->T, H = d->H, dk = d->dk, dv = d->dv;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H; ++h) {
            double* s = (double*)malloc(sizeof(double) * dk * dv);
            if (!s) { fail = 1; continue; }
            if (state_in)
                memcpy(s, state_in + ((size_t)b * H + h) * dk * dv, sizeof(double) * dk * dv);
            else
                memset(s, 0, sizeof(double) * dk * dv);
            for (int t = 0; t < T; ++t) {
                const double* qt = q + (((size_t)b * T + t) * H + h) * dk;
                const double* kt = k + (((size_t)b * T + t) * H + h) * dk;
                const double* vt = v + (((size_t)b * T + t) * H + h) * dv;
                double* ot = o + (((size_t)b * T + t) * H + h) * dv;
                /* s_t = diag(lambda_t^spatial) s_{t-1} + k_t v_t^T */
                for (int c = 0; c < dk; ++c) {
                    const double lam = spatial_decay(d, decay, b, t, h, c);
                    for (int e = 0; e < dv; ++e)
                        s[c * dv + e] = lam * s[c * dv + e] + kt[c] * vt[e];
                }
                /* o_t^T = q_t^T s_t */
                for (int e = 0; e < dv; ++e) {
                    double acc = 0.0;
                    for (int c = 0; c < dk; ++c) acc += qt[c] * s[c * dv + e];
                    ot[e] = d->scale * acc;
                }
            }
            if (state_out)
                memcpy(state_out + ((size_t)b * H + h) * dk * dv, s, sizeof(double) * dk * dv);
            free(s);
        }
    }
    return fail ? -1 : 0;
}

/* The recurrence unrolled: explicit masked-decay sum over earlier tokens. */
int lasad_oracle_quadratic(const lasad_oracle_dims* d,
                           const double* q, const double* k, const double* v,
                           const double* decay, const double* state_in,
                           double* o, double* state_out)
{
    const int B = d->B, T = d->T, H = d->H, dk = d->dk, dv = d->dv;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H; ++h) {
            double* w = (double*)malloc(sizeof(double) * dk); /* prod_{u=j+1..i} L_u[c] */
            if (!w) { fail = 1; continue; }
            const double* sin = state_in ? state_in + ((size_t)b * H + h) * dk * dv : NULL;
            for (int i = 0; i < T; ++i) {
                const double* qi = q + (((size_t)b * T + i) * H + h) * dk;
                double* oi = o + (((size_t)b * T + i) * H + h) * dv;
                for (int e = 0; e < dv; ++e) oi[e] = 0.0;
                for (int c = 0; c < dk; ++c) w[c] = 1.0; /* empty product at j = i */
                for (int j = i; j >= 0; --j) {
                    const double* kj = k + (((size_t)b * T + j) * H + h) * dk;
                    const double* vj = v + (((size_t)b * T + j) * H + h) * dv;
                    double a = 0.0; /* decayed score of the pair (i, j) */
                    for (int c = 0; c < dk; ++c) a += qi[c] * kj[c] * w[c];
                    for (int e = 0; e < dv; ++e) oi[e] += a * vj[e];
                    /* extend the product down to u = j for the next (earlier) token */
                    for (int c = 0; c < dk; ++c) w[c] *= spatial_decay(d, decay, b, j, h, c);
                }
                /* w[c] is now prod_{u=0..i} L_u[c]: the weight of the incoming state */
                if (sin)
                    for (int c = 0; c < dk; ++c)
                        for (int e = 0; e < dv; ++e) oi[e] += qi[c] * w[c] * sin[c * dv + e];
                for (int e = 0; e < dv; ++e) oi[e] *= d->scale;
            }
            if (state_out) {
                double* so = state_out + ((size_t)b * H + h) * dk * dv;
                for (int x = 0; x < dk * dv; ++x) so[x] = 0.0;
                for (int c = 0; c < dk; ++c) w[c] = 1.0; /* prod_{u=j+1..T-1} */
                for (int j = T - 1; j >= 0; --j) {
                    const double* kj = k + (((size_t)b * T + j) * H + h) * dk;
                    const double* vj = v + (((size_t)b * T + j) * H + h) * dv;
                    for (int c = 0; c < dk; ++c)
                        for (int e = 0; e < dv; ++e) so[c * dv + e] += w[c] * kj[c] * vj[e];
                    for (int c = 0; c < dk; ++c) w[c] *= spatial_decay(d, decay, b, j, h, c);
                }
                if (sin)
                    for (int c = 0; c < dk; ++c)
                        for (int e = 0; e < dv; ++e) so[c * dv + e] += w[c] * sin[c * dv + e];
            }
            free(w);
        }
    }
    return fail ? -1 : 0;
}

/*
 * Algorithm 1's loop body including the operator's neighbours: per token
 *     q_t = SiLU(q~_t),  lambda_t = Sigmoid(g~_t),  k_t = 1 - lambda_t (k == NULL) or the given key,
 *     lambda_t^spatial = 1 at a row-boundary step, lambda_t otherwise,
 *     s_t = diag(lambda_t^spatial) s_{t-1} + k_t v_t^T,   o_t^T = scale * q_t^T s_t,
 *     out_t = o_t / sqrt(mean_e(o_t[e]^2) + eps)          (the norm reading stated at the top).
 * q_pre, gate_pre [B,T,H,dk] are pre-activations; k may be NULL; layouts as above.
 */
int lasad_oracle_layer_core(const lasad_oracle_dims* d,
                            const double* q_pre, const double* k, const double* v,
                            const double* gate_pre, const double* state_in, double eps,
                            double* o, double* state_out)
{
    const int B = d->B, T = d->T, H = d->H, dk = d->dk, dv = d->dv;
    int fail = 0;
#pragma omp parallel for collapse(2) schedule(static)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H; ++h) {
            double* s = (double*)malloc(sizeof(double) * (dk * dv + 2 * dk));
            if (!s) { fail = 1; continue; }
            double* qt = s + dk * dv;   /* SiLU(q~_t) */
            double* kt = qt + dk;       /* key of this token */
            if (state_in)
                memcpy(s, state_in + ((size_t)b * H + h) * dk * dv, sizeof(double) * dk * dv);
            else
                memset(s, 0, sizeof(double) * dk * dv);
            for (int t = 0; t < T; ++t) {
                const size_t row = ((size_t)b * T + t) * H + h;
                const double* vt = v + row * dv;
                double* ot = o + row * dv;
                const int boundary = is_boundary(d, d->t0 + t);
                for (int c = 0; c < dk; ++c) {
                    const double x = q_pre[row * dk + c];
                    qt[c] = x / (1.0 + exp(-x));                               /* SiLU */
                    const double lam = 1.0 / (1.0 + exp(-gate_pre[row * dk + c])); /* Sigmoid */
                    kt[c] = k ? k[row * dk + c] : 1.0 - lam;
                    const double lam_spatial = boundary ? 1.0 : lam;
                    for (int e = 0; e < dv; ++e)
                        s[c * dv + e] = lam_spatial * s[c * dv + e] + kt[c] * vt[e];
                }
                double ss = 0.0;
                for (int e = 0; e < dv; ++e) {
                    double acc = 0.0;
                    for (int c = 0; c < dk; ++c) acc += qt[c] * s[c * dv + e];
                    ot[e] = d->scale * acc;
                    ss += ot[e] * ot[e];
                }
                const double r = 1.0 / sqrt(ss / dv + eps);
                for (int e = 0; e < dv; ++e) ot[e] *= r;
            }
            if (state_out)
                memcpy(state_out + ((size_t)b * H + h) * dk * dv, s, sizeof(double) * dk * dv);
            free(s);
        }
    }
    return fail ? -1 : 0;
}
