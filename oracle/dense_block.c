/*
 * TEST INFRASTRUCTURE -- CPU oracle: one ordinary (ungated) adaLN-Zero transformer block.
 *
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may call this.
 * It shares no code with the CUDA library, and none with the regional oracle either: it is
 * a second, separately written statement of the block, working on whole matrices with no
 * mask and no index list.  It exists so that "no region skipped gives the baseline
 * trajectory" (paper Sec. 4.2, quality-bound theorem: the gap vanishes without gating) can
 * be checked by comparing two independent programs.
 *
 * Same numeric convention as the regional oracle: fp32 storage, fp64 accumulation in
 * ascending index order, one rounding per stored value.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* Y[r,o] = sum_k X[r,k] W[o,k] + bias[o] */
static void matmul_nt_bias(const float* X, const float* W, const float* bias, size_t rows, int K,
                           int O, float* Y) {
#pragma omp parallel for schedule(static)
    for (size_t r = 0; r < rows; ++r)
        for (int o = 0; o < O; ++o) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += (double)X[r * K + k] * (double)W[(size_t)o * K + k];
            Y[r * O + o] = (float)(acc + (double)bias[o]);
        }
}

/*
 * FP8 operands (not in the paper; this build's reading).  A projection with both operands in the 8-bit floating-point
 * format E4M3 (sign, 4 exponent bits biased by 7, 3 mantissa bits, gradual underflow below 2^-6, largest magnitude
 * 448, no infinity): the weight matrix arrives quantised, W[o,:] = s_w[o] * W8[o,:]; the activation matrix is divided
 * by its scale a (multiplied by the fp32 reciprocal) and rounded to the nearest E4M3 value, ties to the even mantissa,
 * magnitudes past 448 clamped; Y[r,o] = (sum_k X8[r,k] W8[o,k]) * (a * s_w[o]) + bias[o] with an exact sum.
 * The rounding is done on the bit pattern of the fp32 value.
 */
static float to_e4m3_value(float t) {
    uint32_t u;
    memcpy(&u, &t, 4);
    const uint32_t sign = u & 0x80000000u;
    uint32_t mag = u & 0x7fffffffu;
    if (mag > 0x7f800000u) return t;                      /* NaN stays NaN */
    if (mag >= 0x43e00000u) {
        mag = 0x43e00000u;                                /* 448 */
    } else if (mag < 0x3c800000u) {                       /* below 2^-6: multiples of 2^-9 */
        float a;
        memcpy(&a, &mag, 4);
        volatile float r = a + 16384.0f;                  /* fp32 spacing at 2^14 is 2^-9: the add rounds to the grid, ties to even */
        r = r - 16384.0f;
        a = r;
        memcpy(&mag, &a, 4);
    } else {                                              /* keep three mantissa bits, round the other twenty */
        mag += 0x7ffffu + ((mag >> 20) & 1u);
        mag &= 0xfff00000u;
    }
    u = sign | mag;
    memcpy(&t, &u, 4);
    return t;
}

static int matmul_nt_bias_fp8(const float* X, float a_scale, const float* W8, const float* w_scale, const float* bias,
                              size_t rows, int K, int O, float* Y) {
    float* X8 = (float*)malloc(sizeof(float) * rows * (size_t)K);
    if (!X8) return 1;
    const float inv = 1.0f / a_scale;
    for (size_t e = 0; e < rows * (size_t)K; ++e) X8[e] = to_e4m3_value(X[e] * inv);
#pragma omp parallel for schedule(static)
    for (size_t r = 0; r < rows; ++r)
        for (int o = 0; o < O; ++o) {
            double acc = 0.0;
            for (int k = 0; k < K; ++k) acc += (double)X8[r * K + k] * (double)W8[(size_t)o * K + k];
            Y[r * O + o] = (float)(acc * ((double)a_scale * (double)w_scale[o]) + (double)bias[o]);
        }
    free(X8);
    return 0;
}

void fdo_dense_e4m3(int n, const float* x, float* y) { for (int i = 0; i < n; ++i) y[i] = to_e4m3_value(x[i]); }

/* rows of one request: LayerNorm without affine, then * (1 + scale) + shift */
static void layernorm_modulate(const float* X, size_t rows, int H, const float* shift,
                               const float* scale, float eps, float* Y) {
#pragma omp parallel for schedule(static)
    for (size_t r = 0; r < rows; ++r) {
        const float* x = X + r * H;
        double m = 0.0;
        for (int c = 0; c < H; ++c) m += (double)x[c];
        m /= (double)H;
        double v = 0.0;
        for (int c = 0; c < H; ++c) { double d = (double)x[c] - m; v += d * d; }
        v /= (double)H;
        const double rs = 1.0 / sqrt(v + (double)eps);
        for (int c = 0; c < H; ++c)
            Y[r * H + c] = (float)((((double)x[c] - m) * rs) * (1.0 + (double)scale[c]) + (double)shift[c]);
    }
}

/* O[i, h*dh + c] = sum_t softmax_t(Q_i . K_t / sqrt(dh)) V[t, h*dh + c]: N queries against all T keys (T = N for the
 * block's self-attention) */
static void attention_nt(const float* Q, const float* K, const float* V, int N, int T, int heads, int dh, float* O);
static void full_attention(const float* Q, const float* K, const float* V, int N, int heads, int dh,
                           float* O) {
    attention_nt(Q, K, V, N, N, heads, dh, O);
}
static void attention_nt(const float* Q, const float* K, const float* V, int N, int T, int heads, int dh, float* O) {
    const int H = heads * dh;
    const double scale = 1.0 / sqrt((double)dh);
#pragma omp parallel
    {
        double* s = (double*)malloc(sizeof(double) * (size_t)T);
        double* acc = (double*)malloc(sizeof(double) * (size_t)dh);
#pragma omp for schedule(dynamic, 1) collapse(2)
        for (int i = 0; i < N; ++i)
            for (int h = 0; h < heads; ++h) {
                double mx = -INFINITY;
                for (int t = 0; t < T; ++t) {
                    double d = 0.0;
                    for (int c = 0; c < dh; ++c)
                        d += (double)Q[(size_t)i * H + h * dh + c] * (double)K[(size_t)t * H + h * dh + c];
                    s[t] = d * scale;
                    if (s[t] > mx) mx = s[t];
                }
                double z = 0.0;
                for (int c = 0; c < dh; ++c) acc[c] = 0.0;
                for (int t = 0; t < T; ++t) {
                    const double e = exp(s[t] - mx);
                    z += e;
                    for (int c = 0; c < dh; ++c) acc[c] += e * (double)V[(size_t)t * H + h * dh + c];
                }
                for (int c = 0; c < dh; ++c) O[(size_t)i * H + h * dh + c] = (float)(acc[c] / z);
            }
        free(s); free(acc);
    }
}

/*
 * Block variants (this build's readings of the architectures of the paper's evaluated models, Sec. 6.1), on whole
 * [N,H] matrices of one request.  rms_norm_heads: every head slice of every row is divided by its root mean square
 * (plus eps under the root) and multiplied channel-wise by gamma[dh].  rotate_pairs: the even/odd channel pairs of
 * every head are turned by the angle tabulated for the row's position t, i.e. multiplied as complex numbers
 * (even + i odd) by (cos + i sin).
 */
static void rms_norm_heads(float* X, int N, int heads, int dh, const float* gamma, float eps) {
#pragma omp parallel for schedule(static)
    for (int t = 0; t < N; ++t)
        for (int h = 0; h < heads; ++h) {
            float* v = X + ((size_t)t * heads + h) * dh;
            double sq = 0.0;
            for (int c = 0; c < dh; ++c) sq += (double)v[c] * (double)v[c];
            const double inv = 1.0 / sqrt(sq / (double)dh + (double)eps);
            for (int c = 0; c < dh; ++c) v[c] = (float)((double)v[c] * inv * (double)gamma[c]);
        }
}

static void rotate_pairs(float* X, int N, int heads, int dh, const float* cos_t, const float* sin_t) {
    const int half = dh / 2;
#pragma omp parallel for schedule(static)
    for (int t = 0; t < N; ++t)
        for (int h = 0; h < heads; ++h) {
            float* v = X + ((size_t)t * heads + h) * dh;
            for (int i = 0; i < half; ++i) {
                const double re = (double)v[2 * i], im = (double)v[2 * i + 1];
                const double cr = (double)cos_t[(size_t)t * half + i], ci = (double)sin_t[(size_t)t * half + i];
                v[2 * i] = (float)(re * cr - im * ci);          /* real part of (re + i im)(cr + i ci) */
                v[2 * i + 1] = (float)(re * ci + im * cr);      /* imaginary part */
            }
        }
}

/* test hook: the variants on given Q and K matrices [N,H] of one request (row t sits at position t) */
int fdo_dense_qk_variants(int N, int heads, int dh, float* Q, float* K, const float* qn_w, const float* kn_w,
                          float qk_eps, const float* rope_cos, const float* rope_sin) {
    if (qn_w) rms_norm_heads(Q, N, heads, dh, qn_w, qk_eps);
    if (kn_w) rms_norm_heads(K, N, heads, dh, kn_w, qk_eps);
    if (rope_cos) { rotate_pairs(Q, N, heads, dh, rope_cos, rope_sin); rotate_pairs(K, N, heads, dh, rope_cos, rope_sin); }
    return 0;
}

/*
 * x_in, x_out [B,N,H]; kv_out [B,2,N,H] receives K and V of every position.
 * cond [B,Hc]; adaLN chunk order shift_msa, scale_msa, gate_msa, shift_mlp, scale_mlp, gate_mlp.
 * fdo_dense_block_v adds the block variants (NULL = off): qn_w, kn_w [dh]; rope_cos, rope_sin [N, dh/2].
 * fdo_dense_block_d is the dual-stream block of joint text-image models: the last n_text tokens of every request
 * form a second stream with weights of its own for everything that acts per token (conditioning, QKV projection,
 * QK-norm, out-projection, MLP); the attention runs over all N tokens together.  Written on row ranges of whole
 * matrices: rows [0, N - n_text) with the first weight set, rows [N - n_text, N) with the second.
 */
typedef struct {
    const float *w_ada, *b_ada, *w_qkv, *b_qkv, *w_o, *b_o, *w_fc1, *b_fc1, *w_fc2, *b_fc2, *qn_w, *kn_w;
} fdo_dense_weights;

/*
 * fdo_dense_block_x adds cross-attention to a fixed context (reading of the text-conditioning path of Wan2.1 /
 * StableAudio-type blocks): after the self-attention update, res <- res + (Attn(LN(res) W_q^T + b_q, K_ctx, V_ctx)) W_o^T
 * + b_o, plain LayerNorm, no modulation, no gate; ctx_kv [B,2,T,H] is given.  On whole matrices: the LayerNorm is the
 * modulated one with zero shift and scale.
 */
typedef struct {
    const float *w_q, *b_q, *w_o, *b_o, *ctx_kv;
    int T;
} fdo_dense_cross;

/* fdo_dense_block_q: the QKV, fc1 and fc2 projections with FP8 operands (q8 = NULL: off; q8t: the second stream's
 * operands, given exactly when there is a second stream) */
typedef struct {
    const float *w_qkv, *s_qkv, *w_fc1, *s_fc1, *w_fc2, *s_fc2;   /* E4M3 weight values and per-row scales */
    float a_qkv, a_fc1, a_fc2;                                    /* activation scales */
} fdo_dense_fp8;

int fdo_dense_block_q(int B, int N, int H, int heads, int dh, int M, int Hc, const float* cond,
                      const fdo_dense_weights* wi, const fdo_dense_weights* wt, int n_text, float ln_eps,
                      const float* x_in, float* x_out, float* kv_out, float qk_eps, const float* rope_cos,
                      const float* rope_sin, const fdo_dense_cross* cross, const fdo_dense_fp8* q8, const fdo_dense_fp8* q8t);

int fdo_dense_block_x(int B, int N, int H, int heads, int dh, int M, int Hc, const float* cond,
                      const fdo_dense_weights* wi, const fdo_dense_weights* wt, int n_text, float ln_eps,
                      const float* x_in, float* x_out, float* kv_out, float qk_eps, const float* rope_cos,
                      const float* rope_sin, const fdo_dense_cross* cross) {
    return fdo_dense_block_q(B, N, H, heads, dh, M, Hc, cond, wi, wt, n_text, ln_eps, x_in, x_out, kv_out, qk_eps, rope_cos,
                             rope_sin, cross, NULL, NULL);
}

int fdo_dense_block_d(int B, int N, int H, int heads, int dh, int M, int Hc, const float* cond,
                      const fdo_dense_weights* wi, const fdo_dense_weights* wt, int n_text, float ln_eps,
                      const float* x_in, float* x_out, float* kv_out, float qk_eps, const float* rope_cos,
                      const float* rope_sin) {
    return fdo_dense_block_x(B, N, H, heads, dh, M, Hc, cond, wi, wt, n_text, ln_eps, x_in, x_out, kv_out, qk_eps, rope_cos,
                             rope_sin, NULL);
}

int fdo_dense_block_v(int B, int N, int H, int heads, int dh, int M, int Hc, const float* cond,
                      const float* w_ada, const float* b_ada, const float* w_qkv, const float* b_qkv,
                      const float* w_o, const float* b_o, const float* w_fc1, const float* b_fc1,
                      const float* w_fc2, const float* b_fc2, float ln_eps, const float* x_in,
                      float* x_out, float* kv_out, const float* qn_w, const float* kn_w, float qk_eps,
                      const float* rope_cos, const float* rope_sin) {
    const fdo_dense_weights w = {w_ada, b_ada, w_qkv, b_qkv, w_o, b_o, w_fc1, b_fc1, w_fc2, b_fc2, qn_w, kn_w};
    return fdo_dense_block_d(B, N, H, heads, dh, M, Hc, cond, &w, NULL, 0, ln_eps, x_in, x_out, kv_out, qk_eps, rope_cos,
                             rope_sin);
}

int fdo_dense_block(int B, int N, int H, int heads, int dh, int M, int Hc, const float* cond,
                    const float* w_ada, const float* b_ada, const float* w_qkv, const float* b_qkv,
                    const float* w_o, const float* b_o, const float* w_fc1, const float* b_fc1,
                    const float* w_fc2, const float* b_fc2, float ln_eps, const float* x_in,
                    float* x_out, float* kv_out) {
    return fdo_dense_block_v(B, N, H, heads, dh, M, Hc, cond, w_ada, b_ada, w_qkv, b_qkv, w_o, b_o, w_fc1, b_fc1, w_fc2,
                             b_fc2, ln_eps, x_in, x_out, kv_out, NULL, NULL, 0.f, NULL, NULL);
}

int fdo_dense_block_q(int B, int N, int H, int heads, int dh, int M, int Hc, const float* cond,
                      const fdo_dense_weights* wi, const fdo_dense_weights* wt, int n_text, float ln_eps,
                      const float* x_in, float* x_out, float* kv_out, float qk_eps, const float* rope_cos,
                      const float* rope_sin, const fdo_dense_cross* cross, const fdo_dense_fp8* q8, const fdo_dense_fp8* q8t) {
    if (heads * dh != H) return 2;
    if ((q8 != NULL && wt != NULL) != (q8t != NULL)) return 5;
    const fdo_dense_fp8* q8s[2] = {q8, q8t};
    if ((rope_cos == NULL) != (rope_sin == NULL) || (rope_cos && (dh & 1))) return 3;
    if (!wt) n_text = 0;
    if (n_text < 0 || n_text > N) return 4;
    const size_t NH = (size_t)N * H;
    float* act = (float*)malloc(sizeof(float) * (size_t)Hc);
    float* mod = (float*)malloc(sizeof(float) * (size_t)2 * 6 * H);
    float* xh = (float*)malloc(sizeof(float) * NH);
    float* qkv = (float*)malloc(sizeof(float) * NH * 3);
    float* Q = (float*)malloc(sizeof(float) * NH);
    float* att = (float*)malloc(sizeof(float) * NH);
    float* proj = (float*)malloc(sizeof(float) * NH);
    float* res = (float*)malloc(sizeof(float) * NH);
    float* hid = (float*)malloc(sizeof(float) * (size_t)N * M);
    int rc = 0;
    if (!act || !mod || !xh || !qkv || !Q || !att || !proj || !res || !hid) { rc = 1; goto done; }
    /* the two streams as row ranges [lo, hi) of a request's N rows; the second range is empty for a single stream */
    const int range_lo[2] = {0, N - n_text}, range_hi[2] = {N - n_text, N};
    const fdo_dense_weights* ws[2] = {wi, wt ? wt : wi};

    for (int b = 0; b < B; ++b) {
        const float* X = x_in + (size_t)b * NH;
        float* Kc = kv_out + ((size_t)b * 2 + 0) * NH;
        float* Vc = kv_out + ((size_t)b * 2 + 1) * NH;

        /* conditioning: six H-vectors per stream from SiLU(cond) */
        for (int c = 0; c < Hc; ++c) {
            const double v = (double)cond[(size_t)b * Hc + c];
            act[c] = (float)(v / (1.0 + exp(-v)));
        }
        for (int s = 0; s < 2; ++s) matmul_nt_bias(act, ws[s]->w_ada, ws[s]->b_ada, 1, Hc, 6 * H, mod + (size_t)s * 6 * H);

        /* attention branch: per-stream modulation and projection, then joint attention */
        for (int s = 0; s < 2; ++s) {
            const size_t lo = (size_t)range_lo[s], n = (size_t)(range_hi[s] - range_lo[s]);
            if (!n) continue;
            const float* md = mod + (size_t)s * 6 * H;
            layernorm_modulate(X + lo * H, n, H, md, md + H, ln_eps, xh + lo * H);
            if (q8) {
                if (matmul_nt_bias_fp8(xh + lo * H, q8s[s]->a_qkv, q8s[s]->w_qkv, q8s[s]->s_qkv, ws[s]->b_qkv, n, H, 3 * H, qkv + lo * 3 * H)) { rc = 1; goto done; }
            } else {
                matmul_nt_bias(xh + lo * H, ws[s]->w_qkv, ws[s]->b_qkv, n, H, 3 * H, qkv + lo * 3 * H);
            }
        }
        for (int t = 0; t < N; ++t) {
            memcpy(Q + (size_t)t * H, qkv + (size_t)t * 3 * H, sizeof(float) * (size_t)H);
            memcpy(Kc + (size_t)t * H, qkv + (size_t)t * 3 * H + H, sizeof(float) * (size_t)H);
            memcpy(Vc + (size_t)t * H, qkv + (size_t)t * 3 * H + 2 * H, sizeof(float) * (size_t)H);
        }
        for (int s = 0; s < 2; ++s) {
            const size_t lo = (size_t)range_lo[s];
            const int n = range_hi[s] - range_lo[s];
            if (!n) continue;
            if (ws[s]->qn_w) rms_norm_heads(Q + lo * H, n, heads, dh, ws[s]->qn_w, qk_eps);
            if (ws[s]->kn_w) rms_norm_heads(Kc + lo * H, n, heads, dh, ws[s]->kn_w, qk_eps);
        }
        if (rope_cos) {
            rotate_pairs(Q, N, heads, dh, rope_cos, rope_sin);
            rotate_pairs(Kc, N, heads, dh, rope_cos, rope_sin);
        }
        full_attention(Q, Kc, Vc, N, heads, dh, att);
        for (int s = 0; s < 2; ++s) {
            const size_t lo = (size_t)range_lo[s], n = (size_t)(range_hi[s] - range_lo[s]);
            if (!n) continue;
            const float* gate_a = mod + (size_t)s * 6 * H + 2 * H;
            matmul_nt_bias(att + lo * H, ws[s]->w_o, ws[s]->b_o, n, H, H, proj + lo * H);
            for (size_t e = lo * H; e < (lo + n) * H; ++e)
                res[e] = (float)((double)X[e] + (double)gate_a[e % H] * (double)proj[e]);
        }

        if (cross) {
            /* cross-attention of all N rows to the request's T context tokens; plain LayerNorm = zero shift and scale */
            float* zero = (float*)calloc((size_t)H, sizeof(float));
            if (!zero) { rc = 1; goto done; }
            layernorm_modulate(res, (size_t)N, H, zero, zero, ln_eps, xh);
            free(zero);
            matmul_nt_bias(xh, cross->w_q, cross->b_q, (size_t)N, H, H, Q);
            attention_nt(Q, cross->ctx_kv + ((size_t)b * 2 + 0) * cross->T * H, cross->ctx_kv + ((size_t)b * 2 + 1) * cross->T * H,
                         N, cross->T, heads, dh, att);
            matmul_nt_bias(att, cross->w_o, cross->b_o, (size_t)N, H, H, proj);
            for (size_t e = 0; e < NH; ++e) res[e] = (float)((double)res[e] + (double)proj[e]);
        }

        /* MLP branch, per stream */
        float* Y = x_out + (size_t)b * NH;
        for (int s = 0; s < 2; ++s) {
            const size_t lo = (size_t)range_lo[s], n = (size_t)(range_hi[s] - range_lo[s]);
            if (!n) continue;
            const float* md = mod + (size_t)s * 6 * H;
            layernorm_modulate(res + lo * H, n, H, md + 3 * H, md + 4 * H, ln_eps, xh + lo * H);
            if (q8) {
                if (matmul_nt_bias_fp8(xh + lo * H, q8s[s]->a_fc1, q8s[s]->w_fc1, q8s[s]->s_fc1, ws[s]->b_fc1, n, H, M, hid + lo * M)) { rc = 1; goto done; }
            } else {
                matmul_nt_bias(xh + lo * H, ws[s]->w_fc1, ws[s]->b_fc1, n, H, M, hid + lo * M);
            }
            for (size_t e = lo * M; e < (lo + n) * M; ++e) {
                const double a = (double)hid[e];
                hid[e] = (float)(0.5 * a * (1.0 + tanh(0.79788456080286535588 * (a + 0.044715 * a * a * a))));
            }
            if (q8) {
                if (matmul_nt_bias_fp8(hid + lo * M, q8s[s]->a_fc2, q8s[s]->w_fc2, q8s[s]->s_fc2, ws[s]->b_fc2, n, M, H, proj + lo * H)) { rc = 1; goto done; }
            } else {
                matmul_nt_bias(hid + lo * M, ws[s]->w_fc2, ws[s]->b_fc2, n, M, H, proj + lo * H);
            }
            const float* gate_m = md + 5 * H;
            for (size_t e = lo * H; e < (lo + n) * H; ++e)
                Y[e] = (float)((double)res[e] + (double)gate_m[e % H] * (double)proj[e]);
        }
    }
done:
    free(act); free(mod); free(xh); free(qkv); free(Q); free(att); free(proj); free(res); free(hid);
    return rc;
}
