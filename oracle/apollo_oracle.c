/*
 * CPU oracle for the APOLLO / APOLLO-Mini optimizer step.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, double-precision
 * restatement of the method (Algorithm 1 of the APOLLO paper, with Eq. 4 for the
 * norm-growth limiter and Eq. 5 for the scaling factors).  It shares no code, header,
 * table or constant with the CUDA library and must never be called from the product
 * path; only the tests, the smoke check and the CPU-baseline leg of the benchmark use it.
 *
 * Pinning status (see tests/test_oracle_*.py): every function below is pinned against
 * something other than itself -- published known-answer vectors for Philox, moment
 * statistics and chi-square laws for the projection (Appendix, "Norm Preservation"
 * theorem), numpy matmul for the contraction, textbook Adam written independently for the
 * moments, closed forms for the scales, and the inequalities Eq. 4 fixes for the limiter.
 * The paper prints no worked numeric example of a whole step, so the composition of the
 * steps has no external golden value: "parity unpinned" for the whole-step output beyond
 * those per-part pins.
 *
 * Notation follows the paper: the weight is viewed as m x n with m <= n (m = the shorter
 * stored side), P is r x m, R = P G is r x n, M and V are r x n, s has n entries.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG -1
#define ORACLE_ERR_MEM -2

/* ------------------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2,
 * 3", SC'11): ten rounds; each round multiplies counter words 0 and 2 by the two round
 * multipliers, keeps high and low halves, and mixes in the key; the key is bumped by the
 * two Weyl constants between rounds.
 * ---------------------------------------------------------------------------------- */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n1 = lo1;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        uint32_t n3 = lo0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/*
 * The stream that defines P (Algorithm 1: "P_t <- N_seed(0, 1/r)", resampled when
 * t mod T = 0).  The paper fixes only "Gaussian from a seed"; this library's reading:
 *   key     = (seed low word, seed high word)
 *   counter = (q, k, matrix_id, epoch)   with epoch = floor(t / T),
 * and the four output words of that call give the four entries P[k][4q .. 4q+3].
 * draws: r x ceil(m/4) x 4 words, row-major.
 */
void oracle_philox_draws(uint64_t seed, uint32_t matrix_id, uint32_t epoch,
                         int32_t r, int32_t m, uint32_t* draws)
{
    const int32_t quads = (m + 3) / 4;
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    for (int32_t k = 0; k < r; ++k)
        for (int32_t q = 0; q < quads; ++q) {
            uint32_t ctr[4] = { (uint32_t)q, (uint32_t)k, matrix_id, epoch };
            oracle_philox4x32_10(ctr, key, draws + ((size_t)k * quads + q) * 4);
        }
}

/* Round a double to the nearest bfloat16 (ties to even); result returned as a double. */
double oracle_round_bf16(double x)
{
    if (x != x || isinf(x) || x == 0.0) return x;
    float f = (float)x;
    uint32_t bits; memcpy(&bits, &f, 4);
    uint32_t down_bits = bits & 0xFFFF0000u;          /* toward zero */
    uint32_t up_bits = down_bits + 0x00010000u;       /* next bf16 away from zero */
    float down_f, up_f;
    memcpy(&down_f, &down_bits, 4); memcpy(&up_f, &up_bits, 4);
    double down = (double)down_f, up = (double)up_f;
    double d_down = fabs(x - down), d_up = fabs(up - x);
    if (fabs(x) < fabs(down)) return down;            /* (float)x rounded past x; down is nearest */
    if (d_down < d_up) return down;
    if (d_up < d_down) return up;
    return ((down_bits >> 16) & 1u) ? up : down;      /* tie: even mantissa */
}

/*
 * Box-Muller on the Philox words (x0,x1) and (x2,x3), using the top 23 bits of each word:
 *   u1 = 1 - (x >> 9) / 2^23 in (0,1],   angle = 2 pi ((x' >> 9) / 2^23 - 1/2) in [-pi, pi),
 *   z_a = sqrt(-2 ln u1) cos(angle),     z_b = sqrt(-2 ln u1) sin(angle).
 * z: r x m standard normals (entries past m of the last quad are dropped).
 */
void oracle_standard_normals(uint64_t seed, uint32_t matrix_id, uint32_t epoch,
                             int32_t r, int32_t m, double* z)
{
    const int32_t quads = (m + 3) / 4;
    const double two_pi = 6.283185307179586476925286766559;
    uint32_t key[2] = { (uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32) };
    for (int32_t k = 0; k < r; ++k)
        for (int32_t q = 0; q < quads; ++q) {
            uint32_t ctr[4] = { (uint32_t)q, (uint32_t)k, matrix_id, epoch };
            uint32_t x[4];
            oracle_philox4x32_10(ctr, key, x);
            double zz[4];
            for (int h = 0; h < 2; ++h) {
                double u1 = 1.0 - (double)(x[2 * h] >> 9) / 8388608.0;
                double angle = two_pi * ((double)(x[2 * h + 1] >> 9) / 8388608.0 - 0.5);
                double radius = sqrt(-2.0 * log(u1));
                zz[2 * h] = radius * cos(angle);
                zz[2 * h + 1] = radius * sin(angle);
            }
            for (int e = 0; e < 4; ++e) {
                int32_t i = 4 * q + e;
                if (i < m) z[(size_t)k * m + i] = zz[e];
            }
        }
}

/*
 * P = Z / sqrt(r), entries N(0, 1/r) (Algorithm 1; Appendix notation "P_ij ~ N(0,1/r)").
 * With round_bf16 != 0 the standard normal is first rounded to bfloat16, which is the
 * precision the library keeps P in; the 1/sqrt(r) factor is applied after the rounding (the default is no rounding).
 */
void oracle_projection(uint64_t seed, uint32_t matrix_id, uint32_t epoch,
                       int32_t r, int32_t m, int32_t round_bf16, double* P)
{
    oracle_standard_normals(seed, matrix_id, epoch, r, m, P);
    const double inv_sqrt_r = 1.0 / sqrt((double)r);
    for (size_t e = 0; e < (size_t)r * (size_t)m; ++e) {
        double z = round_bf16 ? oracle_round_bf16(P[e]) : P[e];
        P[e] = z * inv_sqrt_r;
    }
}

/* Plain contraction R = P Gv (Algorithm 1, "R_t <- P_t G_t"): r x m times m x n. */
void oracle_project(const double* P, const double* Gv, int32_t r, int32_t m, int32_t n, double* R)
{
    #pragma omp parallel for schedule(static)
    for (int32_t k = 0; k < r; ++k) {
        double* Rk = R + (size_t)k * n;
        for (int32_t j = 0; j < n; ++j) Rk[j] = 0.0;
        for (int32_t i = 0; i < m; ++i) {
            const double p = P[(size_t)k * m + i];
            const double* Gi = Gv + (size_t)i * n;
            for (int32_t j = 0; j < n; ++j) Rk[j] += p * Gi[j];
        }
    }
}

typedef struct {
    int32_t rank;             /* r */
    int32_t mode;             /* 0 = channel-wise scales (APOLLO), 1 = one tensor-wise scale (Mini) */
    int32_t dtype;            /* 0 = fp32 weights, 1 = bf16 weights (only the final store differs) */
    int32_t bias_correction;  /* 0 = moment equations exactly as printed; 1 = Adam's 1/(1-beta^t) terms */
    int32_t state_bf16;       /* 1 = M and V are kept in bfloat16: rounded after each update (R~ uses the unrounded values) */
    int32_t pad_;
    double alpha, gamma;      /* gradient scale factor; limiter threshold (<= 0 disables it) */
    double beta1, beta2, eps;
} oracle_config;

/*
 * One step for one matrix with the projection supplied by the caller.
 *
 *   W, G     rows x cols, row-major, float (bf16 values are exact in float); G is the
 *            gradient of the loss (the update subtracts).
 *   P        r x m with m = min(rows, cols)
 *   M, V     r x n moments, n = max(rows, cols) (on a tie the rows are projected), updated
 *   prev_norm  norm of the previous scaled gradient after limiting (0 before the first step)
 *   t        number of steps already taken (used only for bias correction)
 * Outputs: W_out (stored dtype, as float), dW (update before the final rounding),
 *   s (n scales), R_out (optional, r x n), norm_out (norm after limiting), c_out (limiter
 *   factor).  Any output pointer except W_out may be NULL.
 */
int oracle_apollo_step_with_P(const oracle_config* cfg, const double* P,
                              const float* W, const float* G, int64_t rows, int64_t cols,
                              int64_t t, double lr, double wd,
                              double* M, double* V, double* prev_norm,
                              float* W_out, double* dW, double* s_out, double* R_out,
                              double* norm_out, double* c_out)
{
    if (!cfg || !P || !W || !G || !M || !V || !prev_norm || !W_out) return ORACLE_ERR_ARG;
    if (rows < 1 || cols < 1 || cfg->rank < 1) return ORACLE_ERR_ARG;
    const int tall = rows > cols;                     /* step 0: orientation, m <= n */
    const int32_t m = (int32_t)(tall ? cols : rows);
    const int32_t n = (int32_t)(tall ? rows : cols);
    const int32_t r = cfg->rank;
    if (r > m) return ORACLE_ERR_ARG;

    double* Gv = (double*)malloc(sizeof(double) * (size_t)m * n);
    double* R = (double*)malloc(sizeof(double) * (size_t)r * n);
    double* Rt = (double*)malloc(sizeof(double) * (size_t)r * n);
    double* s = (double*)malloc(sizeof(double) * (size_t)n);
    if (!Gv || !R || !Rt || !s) { free(Gv); free(R); free(Rt); free(s); return ORACLE_ERR_MEM; }

    for (int32_t i = 0; i < m; ++i)
        for (int32_t j = 0; j < n; ++j)
            Gv[(size_t)i * n + j] = tall ? (double)G[(size_t)j * cols + i] : (double)G[(size_t)i * cols + j];

    /* step 2: R = P G */
    oracle_project(P, Gv, r, m, n, R);

    /* step 3: moments on R (the printed recursions), R~ = M / (sqrt(V) + eps) */
    double bc1 = 1.0, bc2 = 1.0;
    if (cfg->bias_correction) {
        bc1 = 1.0 - pow(cfg->beta1, (double)(t + 1));
        bc2 = 1.0 - pow(cfg->beta2, (double)(t + 1));
    }
    for (size_t e = 0; e < (size_t)r * n; ++e) {
        M[e] = cfg->beta1 * M[e] + (1.0 - cfg->beta1) * R[e];
        V[e] = cfg->beta2 * V[e] + (1.0 - cfg->beta2) * R[e] * R[e];
        Rt[e] = (M[e] / bc1) / (sqrt(V[e] / bc2) + cfg->eps);
        if (cfg->state_bf16) { M[e] = oracle_round_bf16(M[e]); V[e] = oracle_round_bf16(V[e]); }
    }

    /* step 4: scales (Eq. 5 per channel; one ratio of Frobenius norms for Mini) */
    if (cfg->mode == 0) {
        for (int32_t j = 0; j < n; ++j) {
            double num = 0.0, den = 0.0;
            for (int32_t k = 0; k < r; ++k) {
                num += Rt[(size_t)k * n + j] * Rt[(size_t)k * n + j];
                den += R[(size_t)k * n + j] * R[(size_t)k * n + j];
            }
            s[j] = den > 0.0 ? sqrt(num) / sqrt(den) : 0.0;
        }
    } else {
        double num = 0.0, den = 0.0;
        for (size_t e = 0; e < (size_t)r * n; ++e) { num += Rt[e] * Rt[e]; den += R[e] * R[e]; }
        const double st = den > 0.0 ? sqrt(num) / sqrt(den) : 0.0;
        for (int32_t j = 0; j < n; ++j) s[j] = st;
    }

    /* step 5: norm-growth limiter (Eq. 4) on the scaled gradient G diag(s) */
    double sq = 0.0;
    for (int32_t i = 0; i < m; ++i)
        for (int32_t j = 0; j < n; ++j) {
            const double v = s[j] * Gv[(size_t)i * n + j];
            sq += v * v;
        }
    double norm = sqrt(sq), c = 1.0;
    if (cfg->gamma > 0.0 && *prev_norm > 0.0 && norm / *prev_norm > cfg->gamma) {
        c = cfg->gamma * *prev_norm / norm;
        norm = c * norm;
    }
    *prev_norm = norm;

    /* step 6: W <- W - lr (alpha c s_j G_ij + wd W_ij), from the old W */
    for (int32_t i = 0; i < m; ++i)
        for (int32_t j = 0; j < n; ++j) {
            const size_t at = tall ? (size_t)j * cols + i : (size_t)i * cols + j;
            const double w = (double)W[at];
            const double delta = -lr * (cfg->alpha * c * s[j] * Gv[(size_t)i * n + j] + wd * w);
            const double w_new = w + delta;
            if (dW) dW[at] = delta;
            W_out[at] = (float)(cfg->dtype == 1 ? oracle_round_bf16(w_new) : w_new);
        }

    if (s_out) memcpy(s_out, s, sizeof(double) * (size_t)n);
    if (R_out) memcpy(R_out, R, sizeof(double) * (size_t)r * n);
    if (norm_out) *norm_out = norm;
    if (c_out) *c_out = c;
    free(Gv); free(R); free(Rt); free(s);
    return ORACLE_OK;
}

/*
 * One step for one matrix, generating P from (seed, matrix_id, epoch = floor(t / T)) as
 * Algorithm 1 does when t mod T = 0 and keeping it in between (regenerating the same
 * stream gives the same P, so nothing is stored).
 */
int oracle_apollo_step(const oracle_config* cfg, uint64_t seed, uint32_t matrix_id, int32_t T,
                       int32_t p_round_bf16,
                       const float* W, const float* G, int64_t rows, int64_t cols,
                       int64_t t, double lr, double wd,
                       double* M, double* V, double* prev_norm,
                       float* W_out, double* dW, double* s_out, double* R_out,
                       double* norm_out, double* c_out)
{
    if (!cfg || T < 1 || rows < 1 || cols < 1 || cfg->rank < 1) return ORACLE_ERR_ARG;
    const int32_t m = (int32_t)(rows > cols ? cols : rows);
    if (cfg->rank > m) return ORACLE_ERR_ARG;
    double* P = (double*)malloc(sizeof(double) * (size_t)cfg->rank * m);
    if (!P) return ORACLE_ERR_MEM;
    oracle_projection(seed, matrix_id, (uint32_t)(t / T), cfg->rank, m, p_round_bf16, P);
    int rc = oracle_apollo_step_with_P(cfg, P, W, G, rows, cols, t, lr, wd, M, V, prev_norm,
                                       W_out, dW, s_out, R_out, norm_out, c_out);
    free(P);
    return rc;
}

/*
 * AdamW for the parameters APOLLO does not project (embeddings, norms, output head): the
 * paper applies its method to 2-D weight matrices and leaves the rest to the base optimizer
 * (Eq. 1 with decoupled weight decay; bias-corrected moments as in Loshchilov & Hutter's
 * AdamW, which is what `bias_correction = 1` selects; 0 gives Eq. 1 exactly as printed).
 *   m <- b1 m + (1-b1) g;  v <- b2 v + (1-b2) g^2;
 *   p <- p - lr ( (m / c1) / (sqrt(v / c2) + eps) + wd p ),  c_i = 1 - b_i^(t+1) or 1.
 * p, g: float arrays holding values of the stored dtype; m, v: double state.
 */
int oracle_adamw_step(const float* p, const float* g, int64_t numel, int32_t dtype, int32_t bias_correction,
                      double lr, double beta1, double beta2, double eps, double wd, int64_t t,
                      double* m, double* v, float* p_out, double* dp)
{
    if (!p || !g || !m || !v || !p_out || numel < 0) return ORACLE_ERR_ARG;
    double c1 = 1.0, c2 = 1.0;
    if (bias_correction) {
        c1 = 1.0 - pow(beta1, (double)(t + 1));
        c2 = 1.0 - pow(beta2, (double)(t + 1));
    }
    for (int64_t i = 0; i < numel; ++i) {
        const double gi = (double)g[i], pi = (double)p[i];
        m[i] = beta1 * m[i] + (1.0 - beta1) * gi;
        v[i] = beta2 * v[i] + (1.0 - beta2) * gi * gi;
        const double delta = -lr * ((m[i] / c1) / (sqrt(v[i] / c2) + eps) + wd * pi);
        if (dp) dp[i] = delta;
        const double pn = pi + delta;
        p_out[i] = (float)(dtype == 1 ? oracle_round_bf16(pn) : pn);
    }
    return ORACLE_OK;
}
