/*
 * attn_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * Plain fp64 CPU statement of the attention operator of Section 2.2 of the paper:
 *
 *     Attention(Q, K, V) = Softmax(Mask(Q K^T / sqrt(d))) V
 *
 * written out as the definition: one score row at a time, a max, a sum of
 * exponentials, a weighted sum of V rows.  No tiling, no online softmax, no
 * exp2, no blocking.  FlashAttention-style kernels are an exact reformulation
 * of this (up to rounding order), so the definition is the oracle.
 *
 * Readings where the paper is silent:
 *   - scale is an explicit argument (the paper uses 1/sqrt(d));
 *   - the causal mask is lower-triangular including the diagonal and aligned
 *     to the top-left corner: key j is visible to query i iff j <= i, also
 *     when Sq != Sk;
 *   - the per-row logsumexp is the natural log of the sum of exponentials of
 *     the SCALED visible scores;
 *   - a row with no visible key gives O = 0 and LSE = -inf.
 *
 * Only tests, the smoke check and the benchmark's cpu_baseline leg may call
 * this file.  It shares nothing with the CUDA path.
 *
 * Build:  gcc -O2 -fopenmp -shared -fPIC -o liboracle.so attn_oracle.c -lm
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* ---- 16-bit storage formats -> double (exact widening) ------------------ */

/* IEEE binary16: 1 sign, 5 exponent (bias 15), 10 fraction bits. */
double oracle_f16_bits_to_f64(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 10) & 0x1f;
    int f = h & 0x3ff;
    double mag;
    if (e == 0)
        mag = ldexp((double)f, -24); /* subnormal: f * 2^-10 * 2^-14 */
    else if (e == 31)
        mag = f ? NAN : INFINITY;
    else
        mag = ldexp(1.0 + (double)f / 1024.0, e - 15);
    return sign ? -mag : mag;
}

/* bfloat16: 1 sign, 8 exponent (bias 127), 7 fraction bits. */
double oracle_bf16_bits_to_f64(uint16_t h)
{
    int sign = (h >> 15) & 1;
    int e = (h >> 7) & 0xff;
    int f = h & 0x7f;
    double mag;
    if (e == 0)
        mag = ldexp((double)f, -133); /* subnormal: f * 2^-7 * 2^-126 */
    else if (e == 255)
        mag = f ? NAN : INFINITY;
    else
        mag = ldexp(1.0 + (double)f / 128.0, e - 127);
    return sign ? -mag : mag;
}

/* dtype: 0 = binary16, 1 = bfloat16 (same numbering as the library's enum,
 * restated here because the two sides share no header). */
void oracle_widen(const uint16_t *src, double *dst, int64_t n, int dtype)
{
    int64_t i;
#pragma omp parallel for schedule(static)
    for (i = 0; i < n; ++i)
        dst[i] = dtype == 0 ? oracle_f16_bits_to_f64(src[i]) : oracle_bf16_bits_to_f64(src[i]);
}

/* ---- 8-bit storage format -> double (exact widening) -------------------- */

/* OCP 8-bit floating point, E4M3 flavour: 1 sign, 4 exponent (bias 7), 3 fraction bits; no
 * infinities; exponent 15 with fraction 7 is the only NaN, so the largest finite value is
 * 1.75 * 2^8 = 448.  (FP8 is the data type of the case study in Section 4.4, Table 6; the paper
 * does not say which 8-bit format or which scaling it uses: E4M3 with one dequantisation factor
 * per tensor is this build's reading.) */
double oracle_e4m3_bits_to_f64(uint8_t b)
{
    int sign = (b >> 7) & 1;
    int e = (b >> 3) & 0xf;
    int f = b & 7;
    double mag;
    if (e == 0)
        mag = ldexp((double)f, -9); /* subnormal: f * 2^-3 * 2^-6 */
    else if (e == 15 && f == 7)
        mag = NAN;
    else
        mag = ldexp(1.0 + (double)f / 8.0, e - 7);
    return sign ? -mag : mag;
}

/* dst[i] = factor * value(src[i]): the dequantised tensor (factor is the per-tensor scale). */
void oracle_widen_e4m3(const uint8_t *src, double *dst, int64_t n, double factor)
{
    int64_t i;
#pragma omp parallel for schedule(static)
    for (i = 0; i < n; ++i)
        dst[i] = factor * oracle_e4m3_bits_to_f64(src[i]);
}

/* ---- one query row ------------------------------------------------------ */

/* q: [D]; k, v: [Sk, D] of the row's (batch, head); s: scratch of Sk doubles.
 * n_vis = number of visible keys (keys 0 .. n_vis-1).  Writes o[D], *lse and,
 * when prowsum != NULL, the sum of the row's probabilities. */
static void attn_row_dv(const double *q, const double *k, const double *v, double *s, double *o,
                        double *lse, double *prowsum, int64_t n_vis, int D, int Dv, double scale);

static void attn_row(const double *q, const double *k, const double *v, double *s, double *o,
                     double *lse, double *prowsum, int64_t n_vis, int D, double scale)
{
    attn_row_dv(q, k, v, s, o, lse, prowsum, n_vis, D, D, scale);
}

/* q: [D]; k: [Sk, D]; v: [Sk, Dv] -- Q/K and V may have different head dims (the MLA head shape
 * of Section 4.1: 192 for Q/K, 128 for V); o: [Dv]. */
static void attn_row_dv(const double *q, const double *k, const double *v, double *s, double *o,
                        double *lse, double *prowsum, int64_t n_vis, int D, int Dv, double scale)
{
    int64_t j;
    int d;
    if (n_vis <= 0) {
        for (d = 0; d < Dv; ++d)
            o[d] = 0.0;
        *lse = -INFINITY;
        if (prowsum)
            *prowsum = 0.0;
        return;
    }
    /* s_j = scale * <q, k_j> */
    double m = -INFINITY;
    for (j = 0; j < n_vis; ++j) {
        double acc = 0.0;
        for (d = 0; d < D; ++d)
            acc += q[d] * k[j * D + d];
        s[j] = scale * acc;
        if (s[j] > m)
            m = s[j];
    }
    /* e_j = exp(s_j - m),  l = sum_j e_j */
    double l = 0.0;
    for (j = 0; j < n_vis; ++j) {
        s[j] = exp(s[j] - m);
        l += s[j];
    }
    /* p_j = e_j / l,  o = sum_j p_j v_j */
    for (d = 0; d < Dv; ++d)
        o[d] = 0.0;
    double psum = 0.0;
    for (j = 0; j < n_vis; ++j) {
        double p = s[j] / l;
        psum += p;
        for (d = 0; d < Dv; ++d)
            o[d] += p * v[j * Dv + d];
    }
    *lse = m + log(l);
    if (prowsum)
        *prowsum = psum;
}

static int64_t visible_keys(int64_t i, int64_t Sk, int causal)
{
    if (!causal)
        return Sk;
    return (i + 1 < Sk) ? i + 1 : Sk;
}

/* ---- whole problem ------------------------------------------------------ */

/* q: [B,H,Sq,D], k,v: [B,H,Sk,D], o: [B,H,Sq,D], lse: [B,H,Sq],
 * prowsum: [B,H,Sq] or NULL.  All row-major contiguous doubles on the host.
 * Returns 0, or -1 when scratch cannot be allocated. */
int attn_oracle_f64(const double *q, const double *k, const double *v, double *o, double *lse,
                    double *prowsum, int B, int H, int Sq, int Sk, int D, double scale, int causal)
{
    int64_t rows = (int64_t)B * H * Sq;
    int failed = 0;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(Sk > 0 ? Sk : 1));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        }
        int64_t r;
#pragma omp for schedule(dynamic, 16)
        for (r = 0; r < rows; ++r) {
            if (!s)
                continue;
            int64_t bh = r / Sq, i = r % Sq;
            attn_row(q + r * D, k + bh * Sk * D, v + bh * Sk * D, s, o + r * D, lse + r,
                     prowsum ? prowsum + r : NULL, visible_keys(i, Sk, causal), D, scale);
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/* Grouped-query attention (the GQA / MQA variants named in Section 2.2): K and V have Hkv heads,
 * [B,Hkv,Sk,D], and query head h reads key/value head h / (H / Hkv).  Same row function. */
int attn_oracle_gqa_f64(const double *q, const double *k, const double *v, double *o, double *lse,
                        int B, int H, int Hkv, int Sq, int Sk, int D, double scale, int causal)
{
    int64_t rows = (int64_t)B * H * Sq;
    int failed = 0;
    if (Hkv <= 0 || H % Hkv != 0)
        return -2;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(Sk > 0 ? Sk : 1));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        }
        int64_t r;
#pragma omp for schedule(dynamic, 16)
        for (r = 0; r < rows; ++r) {
            if (!s)
                continue;
            int64_t bh = r / Sq, i = r % Sq;
            int64_t b = bh / H, h = bh % H;
            int64_t kvh = b * Hkv + h / (H / Hkv);
            attn_row(q + r * D, k + kvh * Sk * D, v + kvh * Sk * D, s, o + r * D, lse + r, NULL,
                     visible_keys(i, Sk, causal), D, scale);
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/* One K/V shard (split-KV decoding / key-value sharding): k, v hold the keys with global indices
 * k_offset .. k_offset + Sk - 1; with the causal mask key k_offset + j is visible to query i iff
 * k_offset + j <= i.  Rows that see no key of the shard get O = 0, LSE = -inf. */
int attn_oracle_shard_f64(const double *q, const double *k, const double *v, double *o, double *lse,
                          int B, int H, int Hkv, int Sq, int Sk, int D, double scale, int causal,
                          int k_offset)
{
    int64_t rows = (int64_t)B * H * Sq;
    int failed = 0;
    if (Hkv <= 0 || H % Hkv != 0)
        return -2;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(Sk > 0 ? Sk : 1));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        }
        int64_t r;
#pragma omp for schedule(dynamic, 16)
        for (r = 0; r < rows; ++r) {
            if (!s)
                continue;
            int64_t bh = r / Sq, i = r % Sq;
            int64_t b = bh / H, h = bh % H;
            int64_t kvh = b * Hkv + h / (H / Hkv);
            int64_t n_vis = Sk;
            if (causal) {
                n_vis = i + 1 - k_offset;
                if (n_vis < 0)
                    n_vis = 0;
                if (n_vis > Sk)
                    n_vis = Sk;
            }
            attn_row(q + r * D, k + kvh * Sk * D, v + kvh * Sk * D, s, o + r * D, lse + r, NULL, n_vis,
                     D, scale);
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/* Merge of n_parts shard results (definition): LSE = ln sum_r exp(LSE_r), O = sum_r exp(LSE_r - LSE) O_r.
 * o_parts: [n_parts, rows, D], lse_parts: [n_parts, rows]. */
void attn_oracle_combine_f64(const double *o_parts, const double *lse_parts, int n_parts, double *o,
                             double *lse, int64_t rows, int D)
{
    int64_t row;
#pragma omp parallel for schedule(static)
    for (row = 0; row < rows; ++row) {
        int r, d;
        double mx = -INFINITY, sum = 0.0;
        for (r = 0; r < n_parts; ++r)
            if (lse_parts[r * rows + row] > mx)
                mx = lse_parts[r * rows + row];
        for (d = 0; d < D; ++d)
            o[row * D + d] = 0.0;
        if (mx == -INFINITY) {
            lse[row] = -INFINITY;
            continue;
        }
        for (r = 0; r < n_parts; ++r)
            sum += exp(lse_parts[r * rows + row] - mx);
        lse[row] = mx + log(sum);
        for (r = 0; r < n_parts; ++r) {
            double w = exp(lse_parts[r * rows + row] - lse[row]);
            for (d = 0; d < D; ++d)
                o[row * D + d] += w * o_parts[(r * rows + row) * D + d];
        }
    }
}

/* Grouped-query attention with separate head dims: q, k: D; v, o: Dv. */
int attn_oracle_gqa_dv_f64(const double *q, const double *k, const double *v, double *o, double *lse,
                           int B, int H, int Hkv, int Sq, int Sk, int D, int Dv, double scale, int causal)
{
    int64_t rows = (int64_t)B * H * Sq;
    int failed = 0;
    if (Hkv <= 0 || H % Hkv != 0)
        return -2;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(Sk > 0 ? Sk : 1));
        if (!s) {
#pragma omp atomic write
            failed = 1;
        }
        int64_t r;
#pragma omp for schedule(dynamic, 16)
        for (r = 0; r < rows; ++r) {
            if (!s)
                continue;
            int64_t bh = r / Sq, i = r % Sq;
            int64_t b = bh / H, h = bh % H;
            int64_t kvh = b * Hkv + h / (H / Hkv);
            attn_row_dv(q + r * D, k + kvh * Sk * D, v + kvh * Sk * Dv, s, o + r * Dv, lse + r, NULL,
                        visible_keys(i, Sk, causal), D, Dv, scale);
        }
        free(s);
    }
    return failed ? -1 : 0;
}

/* Same arithmetic for a chosen subset of rows, reading the 16-bit inputs directly
 * (widened exactly) so that full-size problems need no fp64 copy of Q, K, V.
 * rows[n_rows]: flat row indices r = (b*H + h)*Sq + i, in ascending order.
 * o: [n_rows, D], lse: [n_rows].
 * Rows of one (batch, head) share one widened copy of that head's K and V. */
int attn_oracle_rows_16(const uint16_t *q, const uint16_t *k, const uint16_t *v, int dtype,
                        const int64_t *rows, int64_t n_rows, double *o, double *lse, int B, int H,
                        int Sq, int Sk, int D, double scale, int causal)
{
    (void)B;
    (void)H;
    size_t nk = (size_t)(Sk > 0 ? Sk : 1);
    double *kd = (double *)malloc(sizeof(double) * nk * (size_t)D);
    double *vd = (double *)malloc(sizeof(double) * nk * (size_t)D);
    int failed = (!kd || !vd);
    int64_t t0 = 0;
    while (!failed && t0 < n_rows) {
        /* the run of requested rows that belong to one (batch, head) */
        int64_t bh = rows[t0] / Sq, t1 = t0;
        int64_t need = 0; /* keys that the run's longest row sees */
        while (t1 < n_rows && rows[t1] / Sq == bh) {
            int64_t nv = visible_keys(rows[t1] % Sq, Sk, causal);
            if (nv > need)
                need = nv;
            ++t1;
        }
        oracle_widen(k + bh * Sk * D, kd, need * D, dtype);
        oracle_widen(v + bh * Sk * D, vd, need * D, dtype);
#pragma omp parallel
        {
            double *s = (double *)malloc(sizeof(double) * nk);
            double *qd = (double *)malloc(sizeof(double) * (size_t)D);
            if (!s || !qd) {
#pragma omp atomic write
                failed = 1;
            }
            int64_t t;
#pragma omp for schedule(dynamic, 1)
            for (t = t0; t < t1; ++t) {
                if (!s || !qd)
                    continue;
                int64_t r = rows[t];
                int e;
                for (e = 0; e < D; ++e)
                    qd[e] = dtype == 0 ? oracle_f16_bits_to_f64(q[r * D + e])
                                       : oracle_bf16_bits_to_f64(q[r * D + e]);
                attn_row(qd, kd, vd, s, o + t * D, lse + t, NULL,
                         visible_keys(r % Sq, Sk, causal), D, scale);
            }
            free(s);
            free(qd);
        }
        t0 = t1;
    }
    free(kd);
    free(vd);
    return failed ? -1 : 0;
}

/* FP8 inputs: the same definition on the dequantised tensors q_f * Q, k_f * K, v_f * V (E4M3 bit
 * patterns, one factor per tensor), for a chosen subset of rows and with grouped K/V heads:
 * q: [B,H,Sq,D]; k, v: [B,Hkv,Sk,D]; rows ascending as in attn_oracle_rows_16. */
int attn_oracle_rows_e4m3(const uint8_t *q, const uint8_t *k, const uint8_t *v, double q_f, double k_f,
                          double v_f, const int64_t *rows, int64_t n_rows, double *o, double *lse,
                          int B, int H, int Hkv, int Sq, int Sk, int D, double scale, int causal)
{
    (void)B;
    if (Hkv <= 0 || H % Hkv != 0)
        return -2;
    size_t nk = (size_t)(Sk > 0 ? Sk : 1);
    double *kd = (double *)malloc(sizeof(double) * nk * (size_t)D);
    double *vd = (double *)malloc(sizeof(double) * nk * (size_t)D);
    int failed = (!kd || !vd);
    int64_t t0 = 0;
    while (!failed && t0 < n_rows) {
        int64_t bh = rows[t0] / Sq, t1 = t0;
        int64_t need = 0;
        while (t1 < n_rows && rows[t1] / Sq == bh) {
            int64_t nv = visible_keys(rows[t1] % Sq, Sk, causal);
            if (nv > need)
                need = nv;
            ++t1;
        }
        int64_t kvh = (bh / H) * Hkv + (bh % H) / (H / Hkv);
        oracle_widen_e4m3(k + kvh * Sk * D, kd, need * D, k_f);
        oracle_widen_e4m3(v + kvh * Sk * D, vd, need * D, v_f);
#pragma omp parallel
        {
            double *s = (double *)malloc(sizeof(double) * nk);
            double *qd = (double *)malloc(sizeof(double) * (size_t)D);
            if (!s || !qd) {
#pragma omp atomic write
                failed = 1;
            }
            int64_t t;
#pragma omp for schedule(dynamic, 1)
            for (t = t0; t < t1; ++t) {
                if (!s || !qd)
                    continue;
                int64_t r = rows[t];
                int e;
                for (e = 0; e < D; ++e)
                    qd[e] = q_f * oracle_e4m3_bits_to_f64(q[r * D + e]);
                attn_row(qd, kd, vd, s, o + t * D, lse + t, NULL,
                         visible_keys(r % Sq, Sk, causal), D, scale);
            }
            free(s);
            free(qd);
        }
        t0 = t1;
    }
    free(kd);
    free(vd);
    return failed ? -1 : 0;
}

/* ---- backward pass: gradients of the same operator ----------------------- */

/* Gradients of O = Softmax(Mask(scale Q K^T)) V (the operator of Section 2.2; the paper measures the forward
 * pass only, so this is the plain chain rule applied to that definition) with respect to Q, K and V,
 * given dO = dL/dO.  One query row at a time, nothing reused from a forward pass:
 *
 *     s_j  = scale <q_i, k_j>             p_j = exp(s_j - m) / sum_j' exp(s_j' - m)      (visible j)
 *     dp_j = <dO_i, v_j>                  (O_i = sum_j p_j v_j       =>  dL/dp_j)
 *     ds_j = p_j (dp_j - sum_j' p_j' dp_j')                          (softmax Jacobian)
 *     dq_i = scale sum_j ds_j k_j         dk_j += scale ds_j q_i     dv_j += p_j dO_i
 *
 * q, dout, dq: [B,H,Sq,D]; k, v, dk, dv: [B,Hkv,Sk,D] with H % Hkv == 0 (query head h reads K/V head
 * h / (H / Hkv), so dk and dv collect the contributions of all query heads of their group).
 * Top-left causal mask as in the forward pass.  Rows without a visible key contribute nothing.
 * Returns 0, -1 when scratch cannot be allocated, -2 for bad head counts.
 * Parallel over (batch, K/V head): each thread owns the dk, dv rows it accumulates into. */
int attn_oracle_bwd_f64(const double *q, const double *k, const double *v, const double *dout, double *dq,
                        double *dk, double *dv, int B, int H, int Hkv, int Sq, int Sk, int D, double scale,
                        int causal)
{
    if (Hkv <= 0 || H % Hkv != 0)
        return -2;
    int group = H / Hkv;
    int64_t n_kv_heads = (int64_t)B * Hkv;
    int failed = 0;
    int64_t g;
#pragma omp parallel for schedule(dynamic, 1)
    for (g = 0; g < n_kv_heads; ++g) {
        size_t nk = (size_t)(Sk > 0 ? Sk : 1);
        double *p = (double *)malloc(sizeof(double) * nk);
        double *dp = (double *)malloc(sizeof(double) * nk);
        if (!p || !dp) {
#pragma omp atomic write
            failed = 1;
            free(p);
            free(dp);
            continue;
        }
        int64_t b = g / Hkv, hk = g % Hkv;
        const double *kh = k + g * Sk * D, *vh = v + g * Sk * D;
        double *dkh = dk + g * Sk * D, *dvh = dv + g * Sk * D;
        int64_t j, i;
        int d, hq;
        for (j = 0; j < (int64_t)Sk * D; ++j) {
            dkh[j] = 0.0;
            dvh[j] = 0.0;
        }
        for (hq = 0; hq < group; ++hq) {
            int64_t bh = b * H + hk * group + hq;
            for (i = 0; i < Sq; ++i) {
                const double *qi = q + (bh * Sq + i) * D, *doi = dout + (bh * Sq + i) * D;
                double *dqi = dq + (bh * Sq + i) * D;
                int64_t n_vis = visible_keys(i, Sk, causal);
                for (d = 0; d < D; ++d)
                    dqi[d] = 0.0;
                if (n_vis <= 0)
                    continue;
                /* forward quantities of this row: p_j */
                double m = -INFINITY, l = 0.0;
                for (j = 0; j < n_vis; ++j) {
                    double acc = 0.0;
                    for (d = 0; d < D; ++d)
                        acc += qi[d] * kh[j * D + d];
                    p[j] = scale * acc;
                    if (p[j] > m)
                        m = p[j];
                }
                for (j = 0; j < n_vis; ++j) {
                    p[j] = exp(p[j] - m);
                    l += p[j];
                }
                for (j = 0; j < n_vis; ++j)
                    p[j] /= l;
                /* dp_j = <dO_i, v_j>, and the row's sum_j p_j dp_j */
                double pdp = 0.0;
                for (j = 0; j < n_vis; ++j) {
                    double acc = 0.0;
                    for (d = 0; d < D; ++d)
                        acc += doi[d] * vh[j * D + d];
                    dp[j] = acc;
                    pdp += p[j] * acc;
                }
                for (j = 0; j < n_vis; ++j) {
                    double ds = p[j] * (dp[j] - pdp);
                    for (d = 0; d < D; ++d) {
                        dqi[d] += scale * ds * kh[j * D + d];
                        dkh[j * D + d] += scale * ds * qi[d];
                        dvh[j * D + d] += p[j] * doi[d];
                    }
                }
            }
        }
        free(p);
        free(dp);
    }
    return failed ? -1 : 0;
}

int oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}
