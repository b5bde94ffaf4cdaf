/*
 * FreqDepthKV CPU oracle -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, single-purpose restatement of what the method computes, written from the
 * paper's Method section: the depth transform (Eq. 1), the sparse high-frequency residual
 * (Eq. 3, in the entry-magnitude form, plus the paper's token-score form), the probe's
 * routing loss and mode rule (Eq. 2, Eq. 3 right half) and decode attention over the
 * reconstructed cache (the paragraph after Eq. 3).  No blocking, fusion or reordering:
 * every function walks the definition.  Only the tests, the smoke check and the benchmark's
 * CPU-baseline leg may call it; the CUDA library shares no code with this file.
 *
 * Storage values travel as float32 holding values that are exactly representable in the
 * storage type (float32 itself, or bf16).  Everything computed after the stored coefficients
 * (reconstruction, probe, attention) is float64.
 *
 * Pins (see tests/test_oracle_pins.py): round trip / Parseval of Eq. 1 and agreement with
 * scipy's orthonormal DCT-II; selection against numpy lexsort, brute force and invariants;
 * probe and attention against a dense numpy float64 evaluation of Eq. 1-3 and against
 * torch's scaled_dot_product_attention in the all-exact case; closed forms on the recipe.
 * Parity unpinned by the paper (fixed by this build's reading only): the scale of lambda
 * (mean over layers, group heads and probe queries in Eq. 2), the formula of Omega
 * (bytes / bytes(exact)), the probe-set composition, independent K and V entry sets.
 *
 * Build: gcc -O2 -ffp-contract=off -fopenmp -shared -fPIC (see oracle/build.py).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int fdkv_ref_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

static uint32_t f32_bits(float x) { uint32_t u; memcpy(&u, &x, 4); return u; }
static float bits_f32(uint32_t u) { float x; memcpy(&x, &u, 4); return x; }

/* round-to-nearest-even to bf16, result returned as float32 (finite inputs) */
static float round_bf16(float x) {
    uint32_t u = f32_bits(x);
    uint32_t lsb = (u >> 16) & 1u;
    u += 0x7FFFu + lsb;
    u &= 0xFFFF0000u;
    return bits_f32(u);
}

/* ---- Eq. 1, B = 2: Z = F_2 X with F_2 = [[c, c], [c, -c]], c = 1/sqrt(2) -------------------
 * Stored ("normative") arithmetic: one float32 add (or subtract), one float32 multiply by the
 * float32 nearest to 1/sqrt(2) (bit pattern 0x3F3504F3), then rounding to the storage type. */
void fdkv_ref_depth_split(const float* x0, const float* x1, int64_t n, int bf16, float* z0, float* z1) {
    const float c32 = bits_f32(0x3F3504F3u);
    for (int64_t i = 0; i < n; ++i) {
        volatile float s = x0[i] + x1[i];
        volatile float t = x0[i] - x1[i];
        float a = s * c32;
        float b = t * c32;
        z0[i] = bf16 ? round_bf16(a) : a;
        z1[i] = bf16 ? round_bf16(b) : b;
    }
}

/* Eq. 1 in exact-as-possible arithmetic (float64 coefficients), used by the invariant tests. */
void fdkv_ref_depth_split_f64(const double* x0, const double* x1, int64_t n, double* z0, double* z1) {
    const double c = sqrt(0.5);
    for (int64_t i = 0; i < n; ++i) {
        z0[i] = c * x0[i] + c * x1[i];
        z1[i] = c * x0[i] - c * x1[i];
    }
}

/* X = F_2^T Z: layer 0 = c (z0 + z1), layer 1 = c (z0 - z1).  Float64. */
void fdkv_ref_depth_merge_f64(const double* z0, const double* z1, int64_t n, double* x0, double* x1) {
    const double c = sqrt(0.5);
    for (int64_t i = 0; i < n; ++i) {
        x0[i] = c * z0[i] + c * z1[i];
        x1[i] = c * z0[i] - c * z1[i];
    }
}

/* ---- sparse residual, entry form: the k entries of z1 with the largest magnitude ------------
 * key = bit pattern of the stored coefficient with the sign cleared (so -0 == +0); order by
 * key descending, flat index ascending; keep the first k; emit ascending flat index. */
typedef struct { uint32_t key; int32_t idx; } key_idx;

static int cmp_key_desc_idx_asc(const void* a, const void* b) {
    const key_idx* x = (const key_idx*)a;
    const key_idx* y = (const key_idx*)b;
    if (x->key != y->key) return x->key > y->key ? -1 : 1;
    if (x->idx != y->idx) return x->idx < y->idx ? -1 : 1;
    return 0;
}
static int cmp_i32(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return (x > y) - (x < y);
}

int64_t fdkv_ref_select_entries(const float* z1, int64_t n, int64_t k, int32_t* idx_out) {
    if (k <= 0) return 0;
    if (k > n) k = n;
    key_idx* e = (key_idx*)malloc((size_t)n * sizeof(key_idx));
    if (!e) return -1;
    for (int64_t i = 0; i < n; ++i) {
        e[i].key = f32_bits(z1[i]) & 0x7FFFFFFFu;
        e[i].idx = (int32_t)i;
    }
    qsort(e, (size_t)n, sizeof(key_idx), cmp_key_desc_idx_asc);
    for (int64_t i = 0; i < k; ++i) idx_out[i] = e[i].idx;
    free(e);
    qsort(idx_out, (size_t)k, sizeof(int32_t), cmp_i32);
    return k;
}

/* ---- candidate caches (the three modes; Eq. 3 with S empty / the kept set / everything) ------
 * mode 0 shared:   c * z0
 * mode 1 residual: c * (z0 + s * z1m), z1m = z1 on the kept entries, 0 elsewhere; s = +1 for the
 *                  first layer of the pair, -1 for the second
 * mode 2 exact:    the original tensor of that layer, unchanged                                  */
void fdkv_ref_reconstruct(const float* z0, const float* z1, const int32_t* kept_idx, int64_t k, int64_t n,
                          int mode, int layer_in_pair, const float* x_exact, double* out) {
    const double c = sqrt(0.5);
    const double s = layer_in_pair == 0 ? 1.0 : -1.0;
    if (mode == 2) {
        for (int64_t i = 0; i < n; ++i) out[i] = (double)x_exact[i];
        return;
    }
    for (int64_t i = 0; i < n; ++i) out[i] = c * (double)z0[i];
    if (mode == 1)
        for (int64_t j = 0; j < k; ++j) {
            int64_t i = kept_idx[j];
            out[i] = c * ((double)z0[i] + s * (double)z1[i]);
        }
}

/* ---- Eq. 2, error term ---------------------------------------------------------------------
 * For a KV head h of a pair: K - Khat^(m) = s * c * R^(m) with R^(shared) = z1K and
 * R^(residual) = z1K with the kept entries removed (orthonormality of F_2).  For each layer of
 * the pair, each of the G query heads that read this KV head and each probe query q at position
 * pos[q], the logit difference against key j <= pos[q] is D[j] = Q . (c R[j,:]) / sqrt(d); the
 * error is the mean over (layer, group head, query) of sum_j D[j]^2.  E(exact) = 0.
 * q0, q1: [W][Hq][d] probe queries of the two layers.  e_out[0] = E(shared), e_out[1] = E(residual). */
void fdkv_ref_probe_error(const float* z1k, const int32_t* kept_idx, int64_t k, int64_t T, int64_t d,
                          const float* q0, const float* q1, int64_t Hq, int64_t G, int64_t h,
                          const int32_t* pos, int64_t W, double* e_out) {
    const double c = sqrt(0.5);
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    int64_t n = T * d;
    double* r_sh = (double*)malloc((size_t)n * sizeof(double));
    double* r_rs = (double*)malloc((size_t)n * sizeof(double));
    for (int64_t i = 0; i < n; ++i) { r_sh[i] = (double)z1k[i]; r_rs[i] = (double)z1k[i]; }
    for (int64_t j = 0; j < k; ++j) r_rs[kept_idx[j]] = 0.0;

    int64_t rows = 2 * G * W;
    double* row_sh = (double*)calloc((size_t)rows, sizeof(double));
    double* row_rs = (double*)calloc((size_t)rows, sizeof(double));
#pragma omp parallel for schedule(dynamic)
    for (int64_t r = 0; r < rows; ++r) {
        int64_t layer = r / (G * W), g = (r / W) % G, qi = r % W;
        const float* qv = (layer == 0 ? q0 : q1) + (qi * Hq + (h * G + g)) * d;
        double acc_sh = 0.0, acc_rs = 0.0;
        for (int64_t j = 0; j <= pos[qi] && j < T; ++j) {
            double d_sh = 0.0, d_rs = 0.0;
            for (int64_t ch = 0; ch < d; ++ch) {
                d_sh += (double)qv[ch] * (c * r_sh[j * d + ch]);
                d_rs += (double)qv[ch] * (c * r_rs[j * d + ch]);
            }
            d_sh *= inv_sqrt_d;
            d_rs *= inv_sqrt_d;
            acc_sh += d_sh * d_sh;
            acc_rs += d_rs * d_rs;
        }
        row_sh[r] = acc_sh;
        row_rs[r] = acc_rs;
    }
    double s_sh = 0.0, s_rs = 0.0;
    for (int64_t r = 0; r < rows; ++r) { s_sh += row_sh[r]; s_rs += row_rs[r]; }
    e_out[0] = s_sh / (double)rows;
    e_out[1] = s_rs / (double)rows;
    free(r_sh); free(r_rs); free(row_sh); free(row_rs);
}

/* ---- Eq. 2 penalty and Eq. 3 argmin ----------------------------------------------------------
 * Omega(m) = bytes(m) / bytes(exact), K and V together, index bytes counted:
 *   shared 2*T*d*e, residual 2*T*d*e + 2*k*(e+4), exact 4*T*d*e.
 * L(m) = E(m) + lambda * Omega(m); mode = argmin, ties to the lowest id (0 < 1 < 2).
 * margin = (L_second - L_best) / L_second (0 when L_second is 0).                               */
void fdkv_ref_omega(int64_t T, int64_t d, int64_t e_bytes, int64_t k, double* omega) {
    double b_sh = 2.0 * (double)T * (double)d * (double)e_bytes;
    double b_rs = b_sh + 2.0 * (double)k * (double)(e_bytes + 4);
    double b_ex = 4.0 * (double)T * (double)d * (double)e_bytes;
    omega[0] = b_sh / b_ex;
    omega[1] = b_rs / b_ex;
    omega[2] = b_ex / b_ex;
}

/* Same with the paper's token-granular residual (the paragraph before Eq. 3): the k_tok selected tokens keep all d
 * high-frequency coefficients of K and of V, one int32 token index each (the set is shared by K and V):
 *   residual 2*T*d*e + 2*k_tok*d*e + 4*k_tok.                                                                */
void fdkv_ref_omega_tokens(int64_t T, int64_t d, int64_t e_bytes, int64_t k_tok, double* omega) {
    double b_sh = 2.0 * (double)T * (double)d * (double)e_bytes;
    double b_rs = b_sh + 2.0 * (double)k_tok * (double)d * (double)e_bytes + 4.0 * (double)k_tok;
    double b_ex = 4.0 * (double)T * (double)d * (double)e_bytes;
    omega[0] = b_sh / b_ex;
    omega[1] = b_rs / b_ex;
    omega[2] = b_ex / b_ex;
}

int fdkv_ref_mode(double e_shared, double e_residual, const double* omega, double lambda, double* loss_out,
                  double* margin_out) {
    double L[3];
    L[0] = e_shared + lambda * omega[0];
    L[1] = e_residual + lambda * omega[1];
    L[2] = 0.0 + lambda * omega[2];
    int best = 0;
    for (int m = 1; m < 3; ++m)
        if (L[m] < L[best]) best = m;
    double second = INFINITY;
    for (int m = 0; m < 3; ++m)
        if (m != best && L[m] < second) second = L[m];
    if (loss_out) { loss_out[0] = L[0]; loss_out[1] = L[1]; loss_out[2] = L[2]; }
    if (margin_out) *margin_out = second > 0.0 ? (second - L[best]) / second : 0.0;
    return best;
}

/* ---- decode attention for one query head over reconstructed rows ----------------------------
 * khat, vhat: [n][d] float64 (prefill rows by mode, then the exact tail rows); q: [d].
 * logit = khat q / sqrt(d); p = exp(logit - max); out = p^T vhat / sum p.  No mask, no bias.    */
void fdkv_ref_attention(const double* khat, const double* vhat, int64_t n, int64_t d, const float* q,
                        double* out) {
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    double* logit = (double*)malloc((size_t)(n > 0 ? n : 1) * sizeof(double));
#pragma omp parallel for
    for (int64_t t = 0; t < n; ++t) {
        double s = 0.0;
        for (int64_t ch = 0; ch < d; ++ch) s += (double)q[ch] * khat[t * d + ch];
        logit[t] = s * inv_sqrt_d;
    }
    double mx = -INFINITY;
    for (int64_t t = 0; t < n; ++t)
        if (logit[t] > mx) mx = logit[t];
    double denom = 0.0;
    for (int64_t t = 0; t < n; ++t) { logit[t] = exp(logit[t] - mx); denom += logit[t]; }
#pragma omp parallel for
    for (int64_t ch = 0; ch < d; ++ch) {
        double acc = 0.0;
        for (int64_t t = 0; t < n; ++t) acc += logit[t] * vhat[t * d + ch];
        out[ch] = n > 0 ? acc / denom : 0.0;
    }
    free(logit);
}

/* ---- the paper's token rule for the residual set (the unnumbered score after Eq. 2) ---------
 * s_t = max over (layer of the pair, group head, probe query with pos >= t) of
 *       | Q . (K_t - Khat_t^shared) | = | Q . (c z1K[t,:]) |   (no 1/sqrt(d) in the paper's formula).
 * Tokens no probe query can see get score 0.                                                     */
void fdkv_ref_token_scores(const float* z1k, int64_t T, int64_t d, const float* q0, const float* q1,
                           int64_t Hq, int64_t G, int64_t h, const int32_t* pos, int64_t W, double* s_out) {
    const double c = sqrt(0.5);
#pragma omp parallel for
    for (int64_t t = 0; t < T; ++t) {
        double best = 0.0;
        for (int64_t layer = 0; layer < 2; ++layer)
            for (int64_t g = 0; g < G; ++g)
                for (int64_t qi = 0; qi < W; ++qi) {
                    if (pos[qi] < t) continue;
                    const float* qv = (layer == 0 ? q0 : q1) + (qi * Hq + (h * G + g)) * d;
                    double s = 0.0;
                    for (int64_t ch = 0; ch < d; ++ch) s += (double)qv[ch] * (c * (double)z1k[t * d + ch]);
                    if (fabs(s) > best) best = fabs(s);
                }
        s_out[t] = best;
    }
}

/* top-k tokens by score, ties to the lowest token; emitted ascending */
typedef struct { double s; int32_t t; } score_tok;
static int cmp_score_desc_tok_asc(const void* a, const void* b) {
    const score_tok* x = (const score_tok*)a;
    const score_tok* y = (const score_tok*)b;
    if (x->s != y->s) return x->s > y->s ? -1 : 1;
    return (x->t > y->t) - (x->t < y->t);
}
int64_t fdkv_ref_select_tokens(const double* s, int64_t T, int64_t k_tok, int32_t* tok_out) {
    if (k_tok <= 0) return 0;
    if (k_tok > T) k_tok = T;
    score_tok* e = (score_tok*)malloc((size_t)T * sizeof(score_tok));
    for (int64_t t = 0; t < T; ++t) { e[t].s = s[t]; e[t].t = (int32_t)t; }
    qsort(e, (size_t)T, sizeof(score_tok), cmp_score_desc_tok_asc);
    for (int64_t i = 0; i < k_tok; ++i) tok_out[i] = e[i].t;
    free(e);
    qsort(tok_out, (size_t)k_tok, sizeof(int32_t), cmp_i32);
    return k_tok;
}

/* ---- budgeted routing (Method: the memory budget is enforced by increasing lambda until the estimated peak KV
 * footprint satisfies the requested budget) ------------------------------------------------------------------------
 * Footprint(lambda) = sum over units of Omega(mode_u(lambda)) * bytes_exact_unit, with the mode rule above.  The plain
 * procedure: try lambda = 0, then lambda = lam_lo, lam_lo * ratio, lam_lo * ratio^2, ... (an ascending grid, ratio > 1)
 * and stop at the first value whose routing fits.  Returns 1 with that lambda, its modes and the grid value tried just
 * before it (which did not fit; -1 when lambda = 0 already fits).  The footprint cannot fall below the all-shared one,
 * so the scan gives up -- returns 0, lambda = +inf, every unit shared -- once a grid value routes every unit to shared
 * and still does not fit, or after max_steps values.                                                               */
int fdkv_ref_route_budget(const double* e_shared, const double* e_residual, int64_t n_units, const double* omega,
                          double bytes_exact_unit, double budget_bytes, double lam_lo, double ratio, int64_t max_steps,
                          double* lambda_out, double* lambda_prev_out, int32_t* modes_out) {
    double lam = 0.0, prev = -1.0;
    for (int64_t step = 0; step <= max_steps; ++step) {
        double total = 0.0;
        int all_shared = 1;
        for (int64_t u = 0; u < n_units; ++u) {
            int m = fdkv_ref_mode(e_shared[u], e_residual[u], omega, lam, NULL, NULL);
            modes_out[u] = m;
            total += omega[m] * bytes_exact_unit;
            if (m != 0) all_shared = 0;
        }
        if (total <= budget_bytes) {
            *lambda_out = lam;
            *lambda_prev_out = prev;
            return 1;
        }
        if (all_shared) break;
        prev = lam;
        lam = step == 0 ? lam_lo : lam * ratio;
    }
    *lambda_out = INFINITY;
    *lambda_prev_out = prev;
    for (int64_t u = 0; u < n_units; ++u) modes_out[u] = 0;
    return 0;
}
