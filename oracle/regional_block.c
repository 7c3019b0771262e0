/*
 * TEST INFRASTRUCTURE -- CPU oracle for one region-selective transformer block.
 *
 * Only tests, the smoke check and the CPU-baseline leg of the benchmark may call this.
 * It shares no code with the CUDA library.
 *
 * What it computes (paper Sec. 3 "Adaptive execution", Sec. 5 worker backend, Appendix A.6):
 * active patches are executed while skipped patches reuse cached state; active queries
 * attend to the K/V of every position, where skipped positions keep the K/V of the step at
 * which they last ran.  The block itself is the adaLN-Zero DiT block the paper builds on
 * (Sec. 2.1): LayerNorm without affine, (1+scale)/shift modulation, gated residuals,
 * tanh-GELU MLP.
 *
 * Numerics: every tensor is stored in fp32; every sum of more than a few terms is
 * accumulated in fp64 in ascending index order and rounded to fp32 once.  Rows are handled
 * one at a time with plain loops; OpenMP only spreads independent rows over cores.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double silu_d(double x) { return x / (1.0 + exp(-x)); }

static double gelu_tanh_d(double a) {
    const double c = 0.79788456080286535588; /* sqrt(2/pi) */
    return 0.5 * a * (1.0 + tanh(c * (a + 0.044715 * a * a * a)));
}

/* y[o] = sum_k x[k] * w[o*K + k] + bias[o], one output at a time */
static void row_linear(const float* x, const float* w, const float* bias, int K, int O, float* y) {
    for (int o = 0; o < O; ++o) {
        const float* wr = w + (size_t)o * K;
        double acc = 0.0;
        for (int k = 0; k < K; ++k) acc += (double)x[k] * (double)wr[k];
        y[o] = (float)(acc + (double)bias[o]);
    }
}

/*
 * FP8 operands (not in the paper: this build's reading of 8-bit floating-point inference as commonly deployed for
 * the paper's models).  The QKV, fc1 and fc2 projections take both operands in the OCP E4M3 format (1 sign, 4
 * exponent bits with bias 7, 3 mantissa bits; subnormals 2^-9 apart below 2^-6; largest finite value 448; no
 * infinities): the weights were quantised beforehand, row o of W standing for s_w[o] * w8[o,:], and the activation row
 * is quantised on the way in with one scale per tensor, x8[k] = E4M3(x[k] * (1 / a)), round to nearest even, values
 * beyond +-448 saturating.  The products of the 8-bit values are summed exactly (fp64 here) and scaled back:
 * y[o] = (sum_k x8[k] w8[o,k]) * (a * s_w[o]) + bias[o].  The out-projection and everything else stay as they are.
 */
static float e4m3_nearest(float t) {
    if (t != t) return t;
    const float a = fabsf(t);
    if (a >= 448.0f) return copysignf(448.0f, t);
    float step;
    if (a < 0.015625f) {
        step = 0.001953125f;                          /* below 2^-6: the subnormal grid */
    } else {
        int e;
        frexpf(a, &e);                                /* a in [2^(e-1), 2^e): eight steps per binade */
        step = ldexpf(1.0f, e - 4);
    }
    return copysignf(rintf(a / step) * step, t);     /* a / step is exact; rintf rounds ties to even */
}

/* the 8-bit form of row_linear; xq [K] is scratch for the quantised row */
static void row_linear_fp8(const float* x, float a_scale, const float* w8, const float* w_scale, const float* bias,
                           int K, int O, float* xq, float* y) {
    const float inv = 1.0f / a_scale;
    for (int k = 0; k < K; ++k) xq[k] = e4m3_nearest(x[k] * inv);
    for (int o = 0; o < O; ++o) {
        const float* wr = w8 + (size_t)o * K;
        double acc = 0.0;
        for (int k = 0; k < K; ++k) acc += (double)xq[k] * (double)wr[k];
        y[o] = (float)(acc * ((double)a_scale * (double)w_scale[o]) + (double)bias[o]);
    }
}

/* quantiser and projection on their own, for the pins */
void fdo_regional_e4m3(int n, const float* x, float* y) { for (int i = 0; i < n; ++i) y[i] = e4m3_nearest(x[i]); }
void fdo_regional_linear_fp8(const float* x, float a_scale, const float* w8, const float* w_scale, const float* bias,
                             int K, int O, float* y) {
    float* xq = (float*)malloc(sizeof(float) * (size_t)K);
    if (!xq) return;
    row_linear_fp8(x, a_scale, w8, w_scale, bias, K, O, xq, y);
    free(xq);
}

/* LayerNorm (biased variance, no affine) followed by (1+scale), shift */
static void row_ln_modulate(const float* u, const float* shift, const float* scale, int H,
                            float ln_eps, float* out) {
    double mean = 0.0;
    for (int c = 0; c < H; ++c) mean += (double)u[c];
    mean /= (double)H;
    double var = 0.0;
    for (int c = 0; c < H; ++c) { double d = (double)u[c] - mean; var += d * d; }
    var /= (double)H;
    const double rstd = 1.0 / sqrt(var + (double)ln_eps);
    for (int c = 0; c < H; ++c)
        out[c] = (float)((((double)u[c] - mean) * rstd) * (1.0 + (double)scale[c]) + (double)shift[c]);
}

/*
 * Block variants of the models the paper evaluates (Sec. 6.1: FLUX.1-dev, SD3-Medium, Wan2.1 use them; the
 * paper itself does not define them, so these are this build's readings of the published architectures):
 *   QK-RMSNorm: per head, x_c <- x_c / sqrt(mean_c x_c^2 + eps) * gamma_c, applied to queries (gamma_q) and keys
 *               (gamma_k) right after the projection; gamma has one entry per head channel, shared by all heads;
 *   RoPE:       after the norm, the channel pairs (2i, 2i+1) of every head are rotated by the angle whose cosine
 *               and sine the caller tabulated for the token's position: (a, b) <- (a cos - b sin, a sin + b cos).
 * The key is cached in this final form.  Either table may be NULL (variant off).
 */
static void head_rms_norm(float* x, int dh, const float* gamma, float eps) {
    double ss = 0.0;
    for (int c = 0; c < dh; ++c) ss += (double)x[c] * (double)x[c];
    const double r = 1.0 / sqrt(ss / (double)dh + (double)eps);
    for (int c = 0; c < dh; ++c) x[c] = (float)((double)x[c] * r * (double)gamma[c]);
}

static void head_rope(float* x, int dh, const float* cs, const float* sn) {
    for (int i = 0; i < dh / 2; ++i) {
        const double a = (double)x[2 * i], b = (double)x[2 * i + 1];
        const double c = (double)cs[i], s = (double)sn[i];
        x[2 * i] = (float)(a * c - b * s);
        x[2 * i + 1] = (float)(a * s + b * c);
    }
}

/* q and k rows [H] of the token at position j of its request, all heads, in place */
static void row_qk_variants(float* q, float* k, int heads, int dh, int j, const float* qn_w, const float* kn_w,
                            float qk_eps, const float* rope_cos, const float* rope_sin) {
    for (int h = 0; h < heads; ++h) {
        if (qn_w) head_rms_norm(q + h * dh, dh, qn_w, qk_eps);
        if (kn_w) head_rms_norm(k + h * dh, dh, kn_w, qk_eps);
        if (rope_cos) {
            head_rope(q + h * dh, dh, rope_cos + (size_t)j * (dh / 2), rope_sin + (size_t)j * (dh / 2));
            head_rope(k + h * dh, dh, rope_cos + (size_t)j * (dh / 2), rope_sin + (size_t)j * (dh / 2));
        }
    }
}

/* test hook: the variants applied to given q / k rows [n, H] of tokens at positions pos[n] */
int fdo_regional_qk_variants(int n, int heads, int dh, const int32_t* pos, float* q, float* k, const float* qn_w,
                             const float* kn_w, float qk_eps, const float* rope_cos, const float* rope_sin) {
    for (int r = 0; r < n; ++r)
        row_qk_variants(q + (size_t)r * heads * dh, k + (size_t)r * heads * dh, heads, dh, pos[r], qn_w, kn_w, qk_eps,
                        rope_cos, rope_sin);
    return 0;
}

/* mod[b, 6H] = W_ada * SiLU(cond[b]) + b_ada ; chunk order shift_msa, scale_msa, gate_msa,
 * shift_mlp, scale_mlp, gate_mlp */
int fdo_adaln(int B, int H, int Hc, const float* cond, const float* w_ada, const float* b_ada,
              float* mod) {
    float* s = (float*)malloc(sizeof(float) * (size_t)Hc);
    if (!s) return 1;
    for (int b = 0; b < B; ++b) {
        for (int c = 0; c < Hc; ++c) s[c] = (float)silu_d((double)cond[(size_t)b * Hc + c]);
        row_linear(s, w_ada, b_ada, Hc, 6 * H, mod + (size_t)b * 6 * H);
    }
    free(s);
    return 0;
}

/*
 * One block over the active rows only.
 *   active_idx[A]   global token ids b*N + j, ascending
 *   u_in/u_out[A,H] compact residual stream entering / leaving the block
 *   kv[B,2,N,H]     this block's K (index 0) and V (index 1) cache, updated in place for
 *                   active rows; every other row is left as it is
 *   finish[n_finish] compact rows whose attention + MLP are evaluated (NULL = all A rows);
 *                   K/V are always refreshed for all A rows because every query needs them.
 * Rows outside `finish` get no u_out.
 * fdo_regional_block_v adds the block variants: qn_w, kn_w [dh] (QK-RMSNorm, NULL = off), rope_cos, rope_sin
 * [N, dh/2] (NULL = off).
 * fdo_regional_block_s adds the dual-stream form of joint text-image blocks (the architecture of the paper's
 * FLUX / SD3 models; this build's reading): a token belongs to one of two streams, and its stream selects the
 * weights of every per-token operation -- the adaLN vectors, the QKV projection, the QK-norm weights, the
 * out-projection and the MLP -- while the attention stays joint over all tokens of the request.  tok_text[B*N] marks
 * the tokens of the second ("text") stream; txt = NULL means a single stream.
 */
typedef struct {
    const float *mod;                       /* [B,6H] adaLN vectors of this block for this stream */
    const float *w_qkv, *b_qkv, *w_o, *b_o, *w_fc1, *b_fc1, *w_fc2, *b_fc2;
    const float *qn_w, *kn_w;               /* [dh] or NULL */
} fdo_stream;

/*
 * Cross-attention to a fixed context (the text-conditioning path of the paper's Wan2.1 / StableAudio-type models;
 * not defined in the paper, this build's reading): between the self-attention update and the MLP,
 *     r1 <- r1 + W_o . Attn(LN(r1) W_q^T + b_q, K_ctx, V_ctx) + b_o
 * with a plain LayerNorm (no affine, no modulation), softmax(q k^T / sqrt(dh)) per head over the T context tokens
 * of the row's request, and no gate.  K_ctx and V_ctx do not change over the denoising steps and are given:
 * ctx_kv [B,2,T,H].  cross = NULL: no cross-attention.
 */
typedef struct {
    const float *w_q, *b_q, *w_o, *b_o;     /* [H,H], [H] */
    const float *ctx_kv;                    /* [B,2,T,H] */
    int T;
} fdo_cross;

/* FP8 operands of the QKV, fc1 and fc2 projections; fp8 = NULL: off.  With two streams each has its own quantised
 * weights and activation scales: fp8_txt for the second one (both or neither). */
typedef struct {
    const float *w_qkv, *s_qkv;             /* [3H,H] E4M3 values of the quantised weights, [3H] scales per output row */
    const float *w_fc1, *s_fc1;             /* [M,H], [M] */
    const float *w_fc2, *s_fc2;             /* [H,M], [H] */
    float a_qkv, a_fc1, a_fc2;              /* activation scales: the inputs of QKV, fc1 and fc2 */
} fdo_fp8;

int fdo_regional_block_q(int B, int N, int H, int heads, int dh, int M, int A, const int32_t* active_idx,
                         const fdo_stream* img, const fdo_stream* txt, const uint8_t* tok_text,
                         float ln_eps, const float* u_in, float* u_out, float* kv, int n_finish, const int32_t* finish,
                         float qk_eps, const float* rope_cos, const float* rope_sin, const fdo_cross* cross,
                         const fdo_fp8* fp8, const fdo_fp8* fp8_txt);

int fdo_regional_block_x(int B, int N, int H, int heads, int dh, int M, int A, const int32_t* active_idx,
                         const fdo_stream* img, const fdo_stream* txt, const uint8_t* tok_text,
                         float ln_eps, const float* u_in, float* u_out, float* kv, int n_finish, const int32_t* finish,
                         float qk_eps, const float* rope_cos, const float* rope_sin, const fdo_cross* cross) {
    return fdo_regional_block_q(B, N, H, heads, dh, M, A, active_idx, img, txt, tok_text, ln_eps, u_in, u_out, kv, n_finish,
                                finish, qk_eps, rope_cos, rope_sin, cross, NULL, NULL);
}

int fdo_regional_block_s(int B, int N, int H, int heads, int dh, int M, int A, const int32_t* active_idx,
                         const fdo_stream* img, const fdo_stream* txt, const uint8_t* tok_text,
                         float ln_eps, const float* u_in, float* u_out, float* kv, int n_finish, const int32_t* finish,
                         float qk_eps, const float* rope_cos, const float* rope_sin) {
    return fdo_regional_block_x(B, N, H, heads, dh, M, A, active_idx, img, txt, tok_text, ln_eps, u_in, u_out, kv, n_finish,
                                finish, qk_eps, rope_cos, rope_sin, NULL);
}

int fdo_regional_block_v(int B, int N, int H, int heads, int dh, int M, int A,
                         const int32_t* active_idx, const float* mod,
                         const float* w_qkv, const float* b_qkv, const float* w_o, const float* b_o,
                         const float* w_fc1, const float* b_fc1, const float* w_fc2, const float* b_fc2,
                         float ln_eps, const float* u_in, float* u_out, float* kv,
                         int n_finish, const int32_t* finish,
                         const float* qn_w, const float* kn_w, float qk_eps, const float* rope_cos, const float* rope_sin) {
    const fdo_stream one = {mod, w_qkv, b_qkv, w_o, b_o, w_fc1, b_fc1, w_fc2, b_fc2, qn_w, kn_w};
    return fdo_regional_block_s(B, N, H, heads, dh, M, A, active_idx, &one, NULL, NULL, ln_eps, u_in, u_out, kv, n_finish,
                                finish, qk_eps, rope_cos, rope_sin);
}

int fdo_regional_block(int B, int N, int H, int heads, int dh, int M, int A,
                       const int32_t* active_idx, const float* mod,
                       const float* w_qkv, const float* b_qkv, const float* w_o, const float* b_o,
                       const float* w_fc1, const float* b_fc1, const float* w_fc2, const float* b_fc2,
                       float ln_eps, const float* u_in, float* u_out, float* kv,
                       int n_finish, const int32_t* finish) {
    return fdo_regional_block_v(B, N, H, heads, dh, M, A, active_idx, mod, w_qkv, b_qkv, w_o, b_o, w_fc1, b_fc1, w_fc2,
                                b_fc2, ln_eps, u_in, u_out, kv, n_finish, finish, NULL, NULL, 0.f, NULL, NULL);
}

int fdo_regional_block_q(int B, int N, int H, int heads, int dh, int M, int A, const int32_t* active_idx,
                         const fdo_stream* img, const fdo_stream* txt, const uint8_t* tok_text,
                         float ln_eps, const float* u_in, float* u_out, float* kv, int n_finish, const int32_t* finish,
                         float qk_eps, const float* rope_cos, const float* rope_sin, const fdo_cross* cross,
                         const fdo_fp8* fp8, const fdo_fp8* fp8_txt) {
    if (heads * dh != H) return 2;
    if ((rope_cos == NULL) != (rope_sin == NULL) || (rope_cos && (dh & 1))) return 3;
    if ((fp8 != NULL && txt != NULL) != (fp8_txt != NULL)) return 5;
    (void)B;
    float* q_all = (float*)malloc(sizeof(float) * (size_t)(A > 0 ? A : 1) * H);
    if (!q_all) return 1;
    int err = 0;

    /* pass 1: normalise, modulate, project; scatter K and V of every active row */
#pragma omp parallel
    {
        float* uh = (float*)malloc(sizeof(float) * (size_t)H);
        float* qkv = (float*)malloc(sizeof(float) * (size_t)3 * H);
        float* xq = (float*)malloc(sizeof(float) * (size_t)H);
        if (!uh || !qkv || !xq) {
#pragma omp atomic write
            err = 1;
        } else {
#pragma omp for schedule(dynamic, 4)
            for (int a = 0; a < A; ++a) {
                const int b = active_idx[a] / N, j = active_idx[a] % N;
                const fdo_stream* st = (txt && tok_text[active_idx[a]]) ? txt : img;      /* the token's stream */
                const float* md = st->mod + (size_t)b * 6 * H;
                row_ln_modulate(u_in + (size_t)a * H, md + 0 * H, md + 1 * H, H, ln_eps, uh);
                const fdo_fp8* f8 = (st == txt) ? fp8_txt : fp8;               /* the stream's 8-bit operands */
                if (f8) row_linear_fp8(uh, f8->a_qkv, f8->w_qkv, f8->s_qkv, st->b_qkv, H, 3 * H, xq, qkv);
                else row_linear(uh, st->w_qkv, st->b_qkv, H, 3 * H, qkv);
                row_qk_variants(qkv, qkv + H, heads, dh, j, st->qn_w, st->kn_w, qk_eps, rope_cos, rope_sin);
                memcpy(q_all + (size_t)a * H, qkv, sizeof(float) * (size_t)H);
                memcpy(kv + (((size_t)b * 2 + 0) * N + j) * H, qkv + H, sizeof(float) * (size_t)H);
                memcpy(kv + (((size_t)b * 2 + 1) * N + j) * H, qkv + 2 * H, sizeof(float) * (size_t)H);
            }
        }
        free(uh); free(qkv); free(xq);
    }
    if (err) { free(q_all); return err; }

    /* pass 2: attention against all N cached keys of the row's request, then the MLP */
    const int n_rows = finish ? n_finish : A;
    const double sm_scale = 1.0 / sqrt((double)dh);
#pragma omp parallel
    {
        double* s = (double*)malloc(sizeof(double) * (size_t)(cross && cross->T > N ? cross->T : N));
        double* oacc = (double*)malloc(sizeof(double) * (size_t)dh);
        float* o = (float*)malloc(sizeof(float) * (size_t)H);
        float* proj = (float*)malloc(sizeof(float) * (size_t)H);
        float* r1 = (float*)malloc(sizeof(float) * (size_t)H);
        float* mh = (float*)malloc(sizeof(float) * (size_t)H);
        float* g = (float*)malloc(sizeof(float) * (size_t)M);
        float* xq = (float*)malloc(sizeof(float) * (size_t)(M > H ? M : H));
        if (!s || !oacc || !o || !proj || !r1 || !mh || !g || !xq) {
#pragma omp atomic write
            err = 1;
        } else {
#pragma omp for schedule(dynamic, 1)
            for (int i = 0; i < n_rows; ++i) {
                const int a = finish ? finish[i] : i;
                const int b = active_idx[a] / N;
                const fdo_stream* st = (txt && tok_text[active_idx[a]]) ? txt : img;
                const float* md = st->mod + (size_t)b * 6 * H;
                const float* Kb = kv + ((size_t)b * 2 + 0) * N * H;
                const float* Vb = kv + ((size_t)b * 2 + 1) * N * H;
                const float* q = q_all + (size_t)a * H;
                for (int h = 0; h < heads; ++h) {
                    const float* qh = q + h * dh;
                    double smax = -INFINITY;
                    for (int t = 0; t < N; ++t) {
                        const float* kt = Kb + (size_t)t * H + h * dh;
                        double acc = 0.0;
                        for (int c = 0; c < dh; ++c) acc += (double)qh[c] * (double)kt[c];
                        s[t] = acc * sm_scale;
                        if (s[t] > smax) smax = s[t];
                    }
                    double denom = 0.0;
                    for (int c = 0; c < dh; ++c) oacc[c] = 0.0;
                    for (int t = 0; t < N; ++t) {
                        const double p = exp(s[t] - smax);
                        const float* vt = Vb + (size_t)t * H + h * dh;
                        denom += p;
                        for (int c = 0; c < dh; ++c) oacc[c] += p * (double)vt[c];
                    }
                    for (int c = 0; c < dh; ++c) o[h * dh + c] = (float)(oacc[c] / denom);
                }
                const float* u = u_in + (size_t)a * H;
                row_linear(o, st->w_o, st->b_o, H, H, proj);
                for (int c = 0; c < H; ++c)
                    r1[c] = (float)((double)u[c] + (double)md[2 * H + c] * (double)proj[c]);
                if (cross) {
                    /* cross-attention of this row to the T context tokens of its request */
                    const int T = cross->T;
                    const float* Kc = cross->ctx_kv + ((size_t)b * 2 + 0) * T * H;
                    const float* Vc = cross->ctx_kv + ((size_t)b * 2 + 1) * T * H;
                    double mean = 0.0, var = 0.0;
                    for (int c = 0; c < H; ++c) mean += (double)r1[c];
                    mean /= (double)H;
                    for (int c = 0; c < H; ++c) { const double d = (double)r1[c] - mean; var += d * d; }
                    const double rstd = 1.0 / sqrt(var / (double)H + (double)ln_eps);
                    for (int c = 0; c < H; ++c) mh[c] = (float)(((double)r1[c] - mean) * rstd);
                    row_linear(mh, cross->w_q, cross->b_q, H, H, proj);              /* proj holds the cross queries */
                    for (int h = 0; h < heads; ++h) {
                        double smax = -INFINITY;
                        for (int t = 0; t < T; ++t) {
                            double acc = 0.0;
                            for (int c = 0; c < dh; ++c) acc += (double)proj[h * dh + c] * (double)Kc[(size_t)t * H + h * dh + c];
                            s[t] = acc * sm_scale;
                            if (s[t] > smax) smax = s[t];
                        }
                        double denom = 0.0;
                        for (int c = 0; c < dh; ++c) oacc[c] = 0.0;
                        for (int t = 0; t < T; ++t) {
                            const double p = exp(s[t] - smax);
                            denom += p;
                            for (int c = 0; c < dh; ++c) oacc[c] += p * (double)Vc[(size_t)t * H + h * dh + c];
                        }
                        for (int c = 0; c < dh; ++c) o[h * dh + c] = (float)(oacc[c] / denom);
                    }
                    row_linear(o, cross->w_o, cross->b_o, H, H, proj);
                    for (int c = 0; c < H; ++c) r1[c] = (float)((double)r1[c] + (double)proj[c]);
                }
                row_ln_modulate(r1, md + 3 * H, md + 4 * H, H, ln_eps, mh);
                const fdo_fp8* f8 = (st == txt) ? fp8_txt : fp8;
                if (f8) row_linear_fp8(mh, f8->a_fc1, f8->w_fc1, f8->s_fc1, st->b_fc1, H, M, xq, g);
                else row_linear(mh, st->w_fc1, st->b_fc1, H, M, g);
                for (int c = 0; c < M; ++c) g[c] = (float)gelu_tanh_d((double)g[c]);
                if (f8) row_linear_fp8(g, f8->a_fc2, f8->w_fc2, f8->s_fc2, st->b_fc2, M, H, xq, proj);
                else row_linear(g, st->w_fc2, st->b_fc2, M, H, proj);
                float* out = u_out + (size_t)a * H;
                for (int c = 0; c < H; ++c)
                    out[c] = (float)((double)r1[c] + (double)md[5 * H + c] * (double)proj[c]);
            }
        }
        free(s); free(oacc); free(o); free(proj); free(r1); free(mh); free(g); free(xq);
    }
    free(q_all);
    return err;
}
