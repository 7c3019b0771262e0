// C-ABI of libflashdiff: argument checks, workspace layout, and the host-side planner that
// queues one region-selective step (compaction, adaLN vectors, then per block: gather + LN +
// modulation, QKV with K/V scatter, attention over all keys, out-projection, MLP, residual
// scatter) on the caller's stream without ever reading the active count back to the host.
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "tc.cuh"

namespace fd {
int simt_attention_tile_rows();
}

using namespace fd;

namespace {

thread_local std::string g_create_error;

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
    size_t control, acc_ss, acc_cnt, block_counts, tiles, text_tiles, consts, ada_act, mod, resid, act, q, o, g, part, attn_ws, total;
    int Mcap, q_ld, tile_cap;
};

bool config_ok(const fd_config* c, std::string* why) {
    auto bad = [&](const char* m) { if (why) *why = m; return false; };
    if (!c) return bad("config is null");
    if (c->n_blocks < 1 || c->hidden < 1 || c->n_heads < 1 || c->head_dim < 1 || c->mlp_dim < 1 || c->cond_dim < 1)
        return bad("non-positive model dimension");
    if (c->hidden != c->n_heads * c->head_dim) return bad("hidden != n_heads * head_dim");
    if (c->max_batch < 1 || c->max_tokens < 1 || c->max_regions < 1) return bad("non-positive limit");
    if ((long long)c->max_batch * c->max_tokens > (1LL << 30)) return bad("max_batch * max_tokens too large");
    if (c->dtype != FD_F32 && c->dtype != FD_BF16) return bad("unknown dtype");
    if (c->engine < FD_ENGINE_AUTO || c->engine > FD_ENGINE_TC) return bad("unknown engine");
    if (c->hidden % 16 || c->mlp_dim % 16 || c->cond_dim % 8) return bad("hidden, mlp_dim must be multiples of 16 and cond_dim of 8");
    if (c->head_dim % 4 || c->head_dim > 128) return bad("head_dim must be a multiple of 4, at most 128");
    if (c->max_skip_k < 0 || !(c->ln_eps > 0.f) || c->gate_eta < 0.f) return bad("bad ln_eps / gate_eta / max_skip_k");
    return true;
}

int esize(const fd_config& c) { return c.dtype == FD_BF16 ? 2 : 4; }

Layout make_layout(const fd_config& c) {
    Layout l{};
    const size_t es = esize(c);
    const size_t BR = (size_t)c.max_batch * c.max_regions;
    l.Mcap = (int)align_up((size_t)c.max_batch * c.max_tokens, 128) + 128;
    // room for Q with padded heads (tensor-core attention stores head dim 72 as 80)
    l.q_ld = c.dtype == FD_BF16 ? c.n_heads * tc_attention_head_pad(c.head_dim) : c.hidden;
    const int min_tile = 16;
    l.tile_cap = c.max_batch * ((c.max_tokens + min_tile - 1) / min_tile + 1);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    l.control = take(sizeof(Control));
    l.acc_ss = take(BR * sizeof(double));
    l.acc_cnt = take(BR * sizeof(int32_t));
    l.block_counts = take((size_t)c.max_batch * ((c.max_tokens + 2047) / 2048 + 1) * sizeof(int32_t));
    l.tiles = take((size_t)2 * l.tile_cap * sizeof(QTile));      // work list, then the list of double-height tiles
    // dual stream: the 128-row and the 256-row tiles that hold rows of the second stream
    l.text_tiles = take(((size_t)l.Mcap / 128 + (size_t)l.Mcap / 256 + 2) * sizeof(int32_t));
    l.consts = take((size_t)2 * c.hidden * sizeof(float));       // [H] zeros, then [H] ones
    l.ada_act = take((size_t)2 * ((c.max_batch + 7) / 8 * 8) * c.cond_dim * 2);   // SiLU(cond): bf16 head + remainder
    l.mod = take((size_t)2 * c.n_blocks * c.max_batch * 6 * c.hidden * sizeof(float));   // adaLN vectors, then the second stream's
    l.resid = take((size_t)l.Mcap * c.hidden * sizeof(float));
    l.act = take((size_t)l.Mcap * c.hidden * es);
    l.q = take((size_t)l.Mcap * l.q_ld * es);
    l.o = take((size_t)l.Mcap * c.hidden * es);
    l.g = take((size_t)l.Mcap * c.mlp_dim * es);
    l.part = take(partition_scratch_bytes(c.max_batch, c.max_tokens, c.max_regions));
    l.attn_ws = take(c.dtype == FD_BF16 && tc_attention_supported(c) ? tc_attention_scratch_bytes(c.head_dim) : 0);
    l.total = off;
    return l;
}

}  // namespace

struct fd_ctx {
    fd_config cfg;
    fd_weights w;
    Layout lay;
    char* ws;
    bool use_tc;         // tensor-core GEMMs
    bool use_tc_attn;    // tensor-core attention
    int tile_rows;
    int64_t launches;
    std::string err;
    TcPlan* tc;
    fd_block_variants var{};   // block variants (all pointers null: off)
    fd_weights text_w{};       // second stream's weights (dual stream; w_qkv null: single stream)
    bool dual = false;
    fd_cross_attention cross{};   // cross-attention to a fixed context (w_q null: off)
    fd_fp8_operands fp8{};        // FP8 operands of QKV, fc1, fc2 (w8_qkv null: off)
    std::vector<float> fp8_a;     // [L, 3] activation scales (host copy)
    fd_fp8_operands fp8_text{};   // the second stream's FP8 operands (dual stream with FP8 operands)
    std::vector<float> fp8_text_a;
    // optional per-kernel timing
    bool profiling = false;
    struct Span { cudaEvent_t a, b; int group, kernels; };
    std::vector<Span> spans;
    std::vector<cudaEvent_t> pool;

    cudaEvent_t get_event() {
        if (!pool.empty()) { cudaEvent_t e = pool.back(); pool.pop_back(); return e; }
        cudaEvent_t e = nullptr;
        cudaEventCreate(&e);
        return e;
    }
    void span_begin(int group, cudaStream_t st) {
        if (!profiling) return;
        Span s{get_event(), get_event(), group, 0};
        cudaEventRecord(s.a, st);
        spans.push_back(s);
    }
    void span_end(int kernels, cudaStream_t st) {
        if (!profiling) return;
        spans.back().kernels = kernels;
        cudaEventRecord(spans.back().b, st);
    }

    fd_status fail(fd_status s, const char* fmt, ...) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof buf, fmt, ap);
        va_end(ap);
        err = buf;
        return s;
    }
    template <typename P> P* at(size_t off) const { return reinterpret_cast<P*>(ws + off); }
    Control* ctl() const { return at<Control>(lay.control); }
};

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }
bool aligned4(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 3) == 0; }

template <typename T>
fd_status run_step(fd_ctx* c, const void* x_, const void* cond_, const int32_t* labels, const uint8_t* mask, int B,
                   int N, int R, void* kv_, void* y_, int32_t* active_idx, int32_t* cu_active, cudaStream_t st,
                   double* region_mass = nullptr) {
    const fd_config& cf = c->cfg;
    const Layout& l = c->lay;
    const int H = cf.hidden, M = cf.mlp_dim, L = cf.n_blocks, Hc = cf.cond_dim;
    const T* x = static_cast<const T*>(x_);
    const T* cond = static_cast<const T*>(cond_);
    T* kv = static_cast<T*>(kv_);
    Control* ctl = c->ctl();
    float* mod = c->at<float>(l.mod);
    float* resid = c->at<float>(l.resid);
    T* act = c->at<T>(l.act);
    T* q = c->at<T>(l.q);
    T* o = c->at<T>(l.o);
    T* g = c->at<T>(l.g);
    QTile* tiles = c->at<QTile>(l.tiles);
    QTile* tiles2 = c->use_tc_attn ? tiles + l.tile_cap : nullptr;
    const int rows_cap = B * N;
    // what the switches set on the context ask of this step, checked before anything is launched
    const bool dual = c->dual;
    const fd_cross_attention& xa = c->cross;
    if (xa.w_q && B != xa.ctx_batch)
        return c->fail(FD_ERR_SHAPE, "B=%d differs from the cross-attention context's batch %d", B, xa.ctx_batch);
    const bool f8 = c->fp8.w8_qkv != nullptr;
    if (f8 && dual && !c->fp8_text.w8_qkv)
        return c->fail(FD_ERR_UNSUPPORTED, "FP8 operands with a second stream need that stream's operands too (fd_set_fp8_text_stream)");
    int nl = 0;
    cudaError_t e;
#define FD_TRY(group, call)                                                                              \
    do {                                                                                                 \
        const int nl_before = nl;                                                                        \
        c->span_begin(group, st);                                                                        \
        e = (call);                                                                                      \
        c->span_end(nl - nl_before, st);                                                                 \
        if (e != cudaSuccess) {                                                                          \
            c->launches += nl;                                                                           \
            return c->fail(FD_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e));                  \
        }                                                                                                \
    } while (0)

    FD_TRY(FD_PROF_COMPACT, launch_compact(mask, labels, B, N, R, active_idx, cu_active, c->at<int32_t>(l.block_counts), tiles,
                          c->tile_rows, ctl, st, &nl, tiles2));
    FD_TRY(FD_PROF_ADALN, launch_adaln<T>(cond, static_cast<const T*>(c->w.w_ada), static_cast<const T*>(c->w.b_ada), mod, L, B, H,
                           Hc, c->ws + l.ada_act, st, &nl));
    // dual stream: tokens with label R use a second weight set for everything that acts per token
    const long long text_mod_off = (long long)L * B * 6 * H;         // second stream's adaLN vectors follow the first's
    int32_t* text128 = c->at<int32_t>(l.text_tiles);
    int32_t* text256 = text128 + l.Mcap / 128 + 1;
    TextSel ts{nullptr, 0, 0};
    if (dual) {
        FD_TRY(FD_PROF_ADALN, launch_adaln<T>(cond, static_cast<const T*>(c->text_w.w_ada), static_cast<const T*>(c->text_w.b_ada),
                                               mod + text_mod_off, L, B, H, Hc, c->ws + l.ada_act, st, &nl));
        FD_TRY(FD_PROF_COMPACT, launch_text_tiles(active_idx, labels, R, rows_cap, text128, text256, ctl, st, &nl));
        ts = TextSel{labels, R, text_mod_off, 0.f};
    }
    // One launch per stream where the weights differ: the first finishes the first stream's rows (all rows when there
    // is a single stream), the second walks the row tiles that hold rows of the second stream and finishes those.
    auto stream_ptr = [&](const void* base0, const void* base1, size_t off, int pass) -> const T* {
        return static_cast<const T*>(pass ? base1 : base0) + off;
    };
    const int n_pass = dual ? 2 : 1;
    const int max_tiles = B * ((N + c->tile_rows - 1) / c->tile_rows);
    const float* zeros = c->at<float>(l.consts);
    const float* ones = zeros + H;
    const fd_fp8_operands* f8ops[2] = {&c->fp8, &c->fp8_text};
    const std::vector<float>* f8a[2] = {&c->fp8_a, &c->fp8_text_a};
    const bool pdl = c->use_tc && c->tc && tc_plan_pdl(c->tc);
    for (int blk = 0; blk < L; ++blk) {
        const float* mod_b = mod + (size_t)blk * B * 6 * H;
        T* kv_b = kv + (size_t)blk * B * 2 * N * H;

        EpiParams ep{};
        ep.active_idx = active_idx;
        ep.N = N;
        ep.H = H;
        ep.labels = labels;
        ep.R = R;
        ep.group = -1;
        ep.text_mod_off = (int32_t)text_mod_off;

        // FP8 operands: this block's activation scales (inputs of QKV, fc1, fc2)
        // [stream][QKV, fc1, fc2]
        float a8[2][3] = {{0.f, 0.f, 0.f}, {0.f, 0.f, 0.f}};
        for (int sx = 0; f8 && sx < n_pass; ++sx)
            for (int g8 = 0; g8 < 3; ++g8) a8[sx][g8] = (*f8a[sx])[(size_t)blk * 3 + g8];
        TextSel ts1 = ts, ts2 = ts;                          // per-row scale of the second stream's rows
        if (f8 && dual) { ts1.fp8_inv_text = 1.0f / a8[1][0]; ts2.fp8_inv_text = 1.0f / a8[1][1]; }
        // gather (first block) or read the residual stream; LayerNorm; attention-branch modulation
        FD_TRY(FD_PROF_LN, launch_ln_modulate<T>(blk == 0 ? x : nullptr, resid, resid, act, active_idx, mod_b + 0 * H,
                                     mod_b + 1 * H, 6 * H, N, H, rows_cap, cf.ln_eps, ctl, st, &nl, pdl, ts1,
                                     f8 ? 1.0f / a8[0][0] : 0.f));
        // QKV projection; K and V rows go straight into the cache
        ep.q = q;
        ep.q_ld = l.q_ld;
        if (c->use_tc_attn && tc_attention_head_pad(cf.head_dim) != cf.head_dim) {
            ep.q_head_dim = cf.head_dim;
            ep.q_head_pad = tc_attention_head_pad(cf.head_dim);
        }
        ep.kv = kv_b;
        // block variants inside the projection's epilogue where the tile shapes allow it, else in a kernel behind it
        const bool have_var = c->var.q_norm_w || c->var.rope_cos;
        const bool qk_fused = have_var && c->use_tc && tc_plan_qk_fusable(c->tc);
        auto norm_w = [&](const void* base) -> const T* {
            return base ? static_cast<const T*>(base) + (size_t)blk * cf.head_dim : nullptr;
        };
        const bool text_norm = dual && c->var.q_norm_w_text != nullptr;
        if (qk_fused) {
            ep.qk_head_dim = cf.head_dim;
            ep.qk_eps = c->var.qk_norm_eps;
            ep.qn_w = norm_w(c->var.q_norm_w);
            ep.kn_w = norm_w(c->var.k_norm_w);
            ep.qn_w2 = text_norm ? norm_w(c->var.q_norm_w_text) : ep.qn_w;
            ep.kn_w2 = text_norm ? norm_w(c->var.k_norm_w_text) : ep.kn_w;
            ep.rope_cos = c->var.rope_cos;
            ep.rope_sin = c->var.rope_sin;
        }
        // (dual stream: one grouped launch where the CTA-pair kernel runs the projection, else one launch per stream)
        const bool grp_qkv = dual && c->use_tc && tc_plan_grouped(c->tc, TC_GEMM_QKV);
        if (grp_qkv) {
            ep.bias = stream_ptr(c->w.b_qkv, c->text_w.b_qkv, (size_t)blk * 3 * H, 0);
            ep.bias2 = stream_ptr(c->w.b_qkv, c->text_w.b_qkv, (size_t)blk * 3 * H, 1);
            if (f8) {
                ep.col_scale = f8ops[0]->s_qkv + (size_t)blk * 3 * H; ep.act_scale = a8[0][0];
                ep.col_scale2 = f8ops[1]->s_qkv + (size_t)blk * 3 * H; ep.act_scale2 = a8[1][0];
            }
            FD_TRY(FD_PROF_GEMM_QKV, tc_gemm_both(c->tc, TC_GEMM_QKV, blk, ep, ctl, st, &nl, f8));
        }
        for (int pass = 0; pass < n_pass && !grp_qkv; ++pass) {
            ep.group = dual ? pass : -1;
            ep.bias = stream_ptr(c->w.b_qkv, c->text_w.b_qkv, (size_t)blk * 3 * H, pass);
            if (qk_fused && pass == 1) { ep.qn_w = ep.qn_w2; ep.kn_w = ep.kn_w2; }
            if (f8) {
                ep.col_scale = f8ops[pass]->s_qkv + (size_t)blk * 3 * H;
                ep.act_scale = a8[pass][0];
                FD_TRY(FD_PROF_GEMM_QKV, tc_gemm_fp8(c->tc, TC_GEMM_QKV, blk, ep, ctl, st, &nl, pass == 1));
            } else if (c->use_tc)
                FD_TRY(FD_PROF_GEMM_QKV, tc_gemm(c->tc, TC_GEMM_QKV, blk, ep, ctl, st, &nl, pass == 1));
            else
                FD_TRY(FD_PROF_GEMM_QKV, launch_simt_gemm<T>(EPI_QKV, act, H, stream_ptr(c->w.w_qkv, c->text_w.w_qkv, (size_t)blk * 3 * H * H, pass),
                                                             3 * H, H, rows_cap, ep, ctl, st, &nl));
        }
        ep.qk_head_dim = 0;                          // (the cross-attention's query projection shares this epilogue)
        // block variants: QK-RMSNorm and rotary embedding on the fresh Q rows and the K rows just written
        if (have_var && !qk_fused) {
            const int q_stride = c->use_tc_attn ? tc_attention_head_pad(cf.head_dim) : cf.head_dim;
            FD_TRY(FD_PROF_QK_VARIANTS, launch_qk_variants<T>(q, l.q_ld, q_stride, kv_b, active_idx, N, H, cf.n_heads, cf.head_dim,
                                                               norm_w(c->var.q_norm_w), norm_w(c->var.k_norm_w), c->var.qk_norm_eps,
                                                               c->var.rope_cos, c->var.rope_sin, rows_cap, ctl, st, &nl,
                                                               text_norm ? norm_w(c->var.q_norm_w_text) : nullptr,
                                                               text_norm ? norm_w(c->var.k_norm_w_text) : nullptr,
                                                               text_norm ? labels : nullptr, R, pdl));
        }
        // active queries against all N keys of their request (joint over both streams); the first block can also
        // report, per region, the softmax mass its queries put on keys of their own region (paper Sec. 4.2)
        double* mass = blk == 0 ? region_mass : nullptr;
        if (mass) {
            e = cudaMemsetAsync(mass, 0, (size_t)B * R * sizeof(double), st);
            if (e != cudaSuccess) { c->launches += nl; return c->fail(FD_ERR_CUDA, "memset failed: %s", cudaGetErrorString(e)); }
        }
        if (c->use_tc_attn) {
            FD_TRY(FD_PROF_ATTENTION, tc_attention(c->tc, blk, kv_b, B, N, tiles, max_tiles, ctl, st, &nl, labels, active_idx,
                                                   mass, R, tiles2));
        } else {
            FD_TRY(FD_PROF_ATTENTION, launch_simt_attention<T>(q, l.q_ld, kv_b, o, H, tiles, max_tiles, N, H, cf.n_heads, cf.head_dim,
                                            ctl, st, &nl, 0, labels, active_idx, mass, R));
        }
        // out-projection, gated residual (a row's gate vector is its stream's: the epilogue adds the offset)
        ep.resid = resid;
        ep.gate = mod_b + 2 * H;
        ep.y = nullptr;
        const bool grp_out = dual && c->use_tc && tc_plan_grouped(c->tc, TC_GEMM_OUT);
        if (grp_out) {
            ep.bias = stream_ptr(c->w.b_o, c->text_w.b_o, (size_t)blk * H, 0);
            ep.bias2 = stream_ptr(c->w.b_o, c->text_w.b_o, (size_t)blk * H, 1);
            FD_TRY(FD_PROF_GEMM_OUT, tc_gemm_both(c->tc, TC_GEMM_OUT, blk, ep, ctl, st, &nl, false));
        }
        for (int pass = 0; pass < n_pass && !grp_out; ++pass) {
            ep.group = dual ? pass : -1;
            ep.bias = stream_ptr(c->w.b_o, c->text_w.b_o, (size_t)blk * H, pass);
            if (c->use_tc)
                FD_TRY(FD_PROF_GEMM_OUT, tc_gemm(c->tc, TC_GEMM_OUT, blk, ep, ctl, st, &nl, pass == 1));
            else
                FD_TRY(FD_PROF_GEMM_OUT, launch_simt_gemm<T>(EPI_RESID, o, H, stream_ptr(c->w.w_o, c->text_w.w_o, (size_t)blk * H * H, pass), H, H,
                                                             rows_cap, ep, ctl, st, &nl));
        }
        // cross-attention to the fixed context: plain LayerNorm, query projection, the attention kernel over the
        // context's keys and values in place of the cache, out-projection added without a gate
        if (xa.w_q) {
            const T* ctx_b = static_cast<const T*>(xa.ctx_kv) + (size_t)blk * B * 2 * xa.n_ctx * H;
            FD_TRY(FD_PROF_CROSS, launch_ln_modulate<T>(nullptr, resid, nullptr, act, active_idx, zeros, zeros, 0, N, H, rows_cap,
                                                        cf.ln_eps, ctl, st, &nl, pdl, TextSel{nullptr, 0, 0}));
            ep.group = -1;
            ep.bias = static_cast<const T*>(xa.b_q) + (size_t)blk * H;
            if (c->use_tc)
                FD_TRY(FD_PROF_CROSS, tc_gemm(c->tc, TC_GEMM_XQ, blk, ep, ctl, st, &nl));
            else
                FD_TRY(FD_PROF_CROSS, launch_simt_gemm<T>(EPI_QKV, act, H, static_cast<const T*>(xa.w_q) + (size_t)blk * H * H, H, H,
                                                          rows_cap, ep, ctl, st, &nl));
            if (c->use_tc_attn)
                FD_TRY(FD_PROF_CROSS, tc_attention(c->tc, blk, const_cast<T*>(ctx_b), B, xa.n_ctx, tiles, max_tiles, ctl, st, &nl));
            else
                FD_TRY(FD_PROF_CROSS, launch_simt_attention<T>(q, l.q_ld, ctx_b, o, H, tiles, max_tiles, xa.n_ctx, H, cf.n_heads,
                                                               cf.head_dim, ctl, st, &nl, 0, nullptr, nullptr, nullptr, 0));
            ep.gate = ones;
            ep.ungated = 1;
            ep.bias = static_cast<const T*>(xa.b_o) + (size_t)blk * H;
            if (c->use_tc)
                FD_TRY(FD_PROF_CROSS, tc_gemm(c->tc, TC_GEMM_XO, blk, ep, ctl, st, &nl));
            else
                FD_TRY(FD_PROF_CROSS, launch_simt_gemm<T>(EPI_RESID, o, H, static_cast<const T*>(xa.w_o) + (size_t)blk * H * H, H, H,
                                                          rows_cap, ep, ctl, st, &nl));
            ep.ungated = 0;
        }
        // MLP branch
        FD_TRY(FD_PROF_LN, launch_ln_modulate<T>(nullptr, resid, nullptr, act, active_idx, mod_b + 3 * H, mod_b + 4 * H, 6 * H, N,
                                     H, rows_cap, cf.ln_eps, ctl, st, &nl, pdl, ts2, f8 ? 1.0f / a8[0][1] : 0.f));
        ep.out = g;
        ep.out_ld = M;
        const bool grp_fc1 = dual && c->use_tc && tc_plan_grouped(c->tc, TC_GEMM_FC1);
        if (grp_fc1) {
            ep.bias = stream_ptr(c->w.b_fc1, c->text_w.b_fc1, (size_t)blk * M, 0);
            ep.bias2 = stream_ptr(c->w.b_fc1, c->text_w.b_fc1, (size_t)blk * M, 1);
            if (f8) {
                ep.col_scale = f8ops[0]->s_fc1 + (size_t)blk * M; ep.act_scale = a8[0][1]; ep.out_inv_scale = 1.0f / a8[0][2];
                ep.col_scale2 = f8ops[1]->s_fc1 + (size_t)blk * M; ep.act_scale2 = a8[1][1]; ep.out_inv_scale2 = 1.0f / a8[1][2];
            }
            FD_TRY(FD_PROF_GEMM_FC1, tc_gemm_both(c->tc, TC_GEMM_FC1, blk, ep, ctl, st, &nl, f8));
        }
        for (int pass = 0; pass < n_pass && !grp_fc1; ++pass) {
            ep.group = dual ? pass : -1;
            ep.bias = stream_ptr(c->w.b_fc1, c->text_w.b_fc1, (size_t)blk * M, pass);
            if (f8) {
                ep.col_scale = f8ops[pass]->s_fc1 + (size_t)blk * M;
                ep.act_scale = a8[pass][1];
                ep.out_inv_scale = 1.0f / a8[pass][2];      // the hidden activations leave as E4M3 bytes, row stride M
                FD_TRY(FD_PROF_GEMM_FC1, tc_gemm_fp8(c->tc, TC_GEMM_FC1, blk, ep, ctl, st, &nl, pass == 1));
            } else if (c->use_tc)
                FD_TRY(FD_PROF_GEMM_FC1, tc_gemm(c->tc, TC_GEMM_FC1, blk, ep, ctl, st, &nl, pass == 1));
            else
                FD_TRY(FD_PROF_GEMM_FC1, launch_simt_gemm<T>(EPI_GELU, act, H, stream_ptr(c->w.w_fc1, c->text_w.w_fc1, (size_t)blk * M * H, pass), M,
                                                             H, rows_cap, ep, ctl, st, &nl));
        }
        ep.gate = mod_b + 5 * H;
        ep.y = (blk == L - 1) ? y_ : nullptr;       // the last block scatters the rows back
        const bool grp_fc2 = dual && c->use_tc && tc_plan_grouped(c->tc, TC_GEMM_FC2);
        if (grp_fc2) {
            ep.bias = stream_ptr(c->w.b_fc2, c->text_w.b_fc2, (size_t)blk * H, 0);
            ep.bias2 = stream_ptr(c->w.b_fc2, c->text_w.b_fc2, (size_t)blk * H, 1);
            if (f8) {
                ep.col_scale = f8ops[0]->s_fc2 + (size_t)blk * H; ep.act_scale = a8[0][2];
                ep.col_scale2 = f8ops[1]->s_fc2 + (size_t)blk * H; ep.act_scale2 = a8[1][2];
            }
            FD_TRY(FD_PROF_GEMM_FC2, tc_gemm_both(c->tc, TC_GEMM_FC2, blk, ep, ctl, st, &nl, f8));
        }
        for (int pass = 0; pass < n_pass && !grp_fc2; ++pass) {
            ep.group = dual ? pass : -1;
            ep.bias = stream_ptr(c->w.b_fc2, c->text_w.b_fc2, (size_t)blk * H, pass);
            if (f8) {
                ep.col_scale = f8ops[pass]->s_fc2 + (size_t)blk * H;
                ep.act_scale = a8[pass][2];
                FD_TRY(FD_PROF_GEMM_FC2, tc_gemm_fp8(c->tc, TC_GEMM_FC2, blk, ep, ctl, st, &nl, pass == 1));
            } else if (c->use_tc)
                FD_TRY(FD_PROF_GEMM_FC2, tc_gemm(c->tc, TC_GEMM_FC2, blk, ep, ctl, st, &nl, pass == 1));
            else
                FD_TRY(FD_PROF_GEMM_FC2, launch_simt_gemm<T>(EPI_RESID, g, M, stream_ptr(c->w.w_fc2, c->text_w.w_fc2, (size_t)blk * H * M, pass), H,
                                                             M, rows_cap, ep, ctl, st, &nl));
        }
    }
#undef FD_TRY
    c->launches += nl;
    return FD_OK;
}

}  // namespace

extern "C" {

size_t fd_workspace_bytes(const fd_config* cfg) {
    if (!config_ok(cfg, nullptr)) return 0;
    return make_layout(*cfg).total;
}

fd_status fd_create(const fd_config* cfg, const fd_weights* weights, void* workspace, size_t workspace_bytes,
                    fd_ctx** out) {
    if (!out) { g_create_error = "out is null"; return FD_ERR_INVALID_ARG; }
    *out = nullptr;
    std::string why;
    if (!config_ok(cfg, &why)) { g_create_error = why; return FD_ERR_SHAPE; }
    if (!weights) { g_create_error = "weights is null"; return FD_ERR_INVALID_ARG; }
    const void* wp[10] = {weights->w_qkv, weights->b_qkv, weights->w_o, weights->b_o, weights->w_fc1,
                          weights->b_fc1, weights->w_fc2, weights->b_fc2, weights->w_ada, weights->b_ada};
    for (const void* p : wp)
        if (!p || !aligned16(p)) { g_create_error = "weight pointer null or not 16-byte aligned"; return FD_ERR_INVALID_ARG; }
    const Layout lay = make_layout(*cfg);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < lay.total) {
        g_create_error = "workspace null, not 256-byte aligned, or smaller than fd_workspace_bytes";
        return FD_ERR_WORKSPACE;
    }
    bool use_tc = false;
    if (cfg->engine == FD_ENGINE_TC || (cfg->engine == FD_ENGINE_AUTO && cfg->dtype == FD_BF16)) {
        std::string tc_why;
        if (cfg->dtype == FD_BF16 && tc_supported(*cfg, &tc_why)) {
            use_tc = true;
        } else if (cfg->engine == FD_ENGINE_TC) {
            g_create_error = "tensor-core engine unavailable for this configuration: " + tc_why;
            return FD_ERR_UNSUPPORTED;
        }
    }
    int dev_count = 0;
    cudaError_t e = cudaGetDeviceCount(&dev_count);
    if (e != cudaSuccess || dev_count == 0) {
        g_create_error = std::string("no CUDA device: ") + cudaGetErrorString(e);
        return FD_ERR_CUDA;
    }
    fd_ctx* c = new (std::nothrow) fd_ctx();
    if (!c) { g_create_error = "out of host memory"; return FD_ERR_INVALID_ARG; }
    c->cfg = *cfg;
    c->w = *weights;
    c->lay = lay;
    c->ws = static_cast<char*>(workspace);
    c->use_tc = use_tc;
    c->use_tc_attn = use_tc && tc_attention_supported(*cfg);
    c->tile_rows = c->use_tc_attn ? tc_attention_tile_rows() : simt_attention_tile_rows();
    c->launches = 0;
    c->tc = nullptr;
    // control block and gate accumulators start at zero; the compact buffers start finite
    e = cudaMemset(workspace, 0, lay.ada_act);
    if (e == cudaSuccess) e = cudaMemset(c->ws + lay.resid, 0, lay.part - lay.resid);
    if (e == cudaSuccess) {
        const std::vector<float> one(cfg->hidden, 1.0f);
        e = cudaMemcpy(c->ws + lay.consts + (size_t)cfg->hidden * sizeof(float), one.data(), one.size() * sizeof(float),
                       cudaMemcpyHostToDevice);
    }
    if (e == cudaSuccess && use_tc) {
        TcBuffers tb{};
        tb.act = c->ws + lay.act; tb.q = c->ws + lay.q; tb.o = c->ws + lay.o; tb.g = c->ws + lay.g;
        tb.Mcap = lay.Mcap; tb.q_ld = lay.q_ld;
        tb.resid = c->ws + lay.resid;
        tb.attn_ws = c->ws + lay.attn_ws;
        tb.attn_slots = TC_ATTENTION_SLOTS;
        std::string tc_err;
        c->tc = tc_plan_create(*cfg, *weights, tb, &tc_err);
        if (!c->tc) {
            g_create_error = "tensor-core plan: " + tc_err;
            delete c;
            return FD_ERR_CUDA;
        }
    }
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        g_create_error = std::string("workspace initialisation failed: ") + cudaGetErrorString(e);
        tc_plan_destroy(c->tc);
        delete c;
        return FD_ERR_CUDA;
    }
    *out = c;
    return FD_OK;
}

fd_status fd_partition_regions(fd_ctx* c, const float* attn_map, int B, int N, int T, const int32_t* salient_cols,
                               int T_s, int R, int min_region_tokens, int max_region_tokens, int32_t* labels_out,
                               int32_t* region_sizes_out, void* cuda_stream) {
    if (!c) return FD_ERR_INVALID_ARG;
    if (!attn_map || !labels_out) return c->fail(FD_ERR_INVALID_ARG, "attn_map / labels_out is null");
    if (B < 1 || N < 1 || T < 1 || R < 1) return c->fail(FD_ERR_SHAPE, "B, N, T, R must be positive");
    if (B > c->cfg.max_batch || N > c->cfg.max_tokens || R > c->cfg.max_regions)
        return c->fail(FD_ERR_SHAPE, "B=%d N=%d R=%d exceed the limits %d/%d/%d", B, N, R, c->cfg.max_batch,
                       c->cfg.max_tokens, c->cfg.max_regions);
    if (R > N) return c->fail(FD_ERR_SHAPE, "R=%d exceeds N=%d", R, N);
    if (N >= 65536) return c->fail(FD_ERR_UNSUPPORTED, "partitioner handles N < 65536");
    if (salient_cols && T_s < 1) return c->fail(FD_ERR_SHAPE, "T_s must be positive when salient_cols is given");
    if (min_region_tokens < 1) min_region_tokens = 1;
    if (max_region_tokens <= 0 || max_region_tokens > N) max_region_tokens = N;
    int nl = 0;
    c->span_begin(FD_PROF_PARTITION, static_cast<cudaStream_t>(cuda_stream));
    cudaError_t e = launch_partition(attn_map, B, N, T, salient_cols, salient_cols ? T_s : T, R, min_region_tokens,
                                     max_region_tokens, labels_out, region_sizes_out, c->ws + c->lay.part, c->ctl(),
                                     static_cast<cudaStream_t>(cuda_stream), &nl);
    c->span_end(nl, static_cast<cudaStream_t>(cuda_stream));
    c->launches += nl;
    if (e != cudaSuccess) return c->fail(FD_ERR_CUDA, "partition launch failed: %s", cudaGetErrorString(e));
    return FD_OK;
}

fd_status fd_region_activity(fd_ctx* c, const float* z_cur, const float* z_prev, const int32_t* labels, int B, int N,
                             int D, int R, const float* eps, float* delta_state, int32_t* skip_count,
                             uint8_t* prev_active, float* score_out, float* weight_out, uint8_t* mask_out,
                             void* cuda_stream) {
    if (!c) return FD_ERR_INVALID_ARG;
    if (!z_cur || !z_prev || !labels || !eps || !delta_state || !skip_count || !prev_active || !score_out ||
        !weight_out || !mask_out)
        return c->fail(FD_ERR_INVALID_ARG, "null pointer argument");
    if (B < 1 || N < 1 || D < 1 || R < 1) return c->fail(FD_ERR_SHAPE, "B, N, D, R must be positive");
    if (B > c->cfg.max_batch || N > c->cfg.max_tokens || R > c->cfg.max_regions)
        return c->fail(FD_ERR_SHAPE, "B=%d N=%d R=%d exceed the limits %d/%d/%d", B, N, R, c->cfg.max_batch,
                       c->cfg.max_tokens, c->cfg.max_regions);
    int nl = 0;
    c->span_begin(FD_PROF_ACTIVITY, static_cast<cudaStream_t>(cuda_stream));
    cudaError_t e = launch_activity(z_cur, z_prev, labels, B, N, D, R, eps, delta_state, skip_count, prev_active,
                                    score_out, weight_out, mask_out, c->cfg.gate_eta, c->cfg.max_skip_k,
                                    c->at<double>(c->lay.acc_ss), c->at<int32_t>(c->lay.acc_cnt), c->ctl(),
                                    static_cast<cudaStream_t>(cuda_stream), &nl);
    c->span_end(nl, static_cast<cudaStream_t>(cuda_stream));
    c->launches += nl;
    if (e != cudaSuccess) return c->fail(FD_ERR_CUDA, "activity launch failed: %s", cudaGetErrorString(e));
    return FD_OK;
}

namespace {
fd_status sampler_args_ok(fd_ctx* c, const fd_sampler_weights* sw, int B, int N) {
    if (!sw) return c->fail(FD_ERR_INVALID_ARG, "null sampler weights");
    if (!sw->w_in || !sw->b_in || !sw->pos || !sw->w_out || !sw->b_out) return c->fail(FD_ERR_INVALID_ARG, "null sampler weight pointer");
    if (!aligned16(sw->w_in) || !aligned16(sw->b_in) || !aligned16(sw->pos) || !aligned16(sw->w_out) || !aligned16(sw->b_out))
        return c->fail(FD_ERR_INVALID_ARG, "sampler weights must be 16-byte aligned");
    if (sw->latent_dim < 4 || sw->latent_dim % 4 || sw->latent_dim > 256)
        return c->fail(FD_ERR_SHAPE, "latent_dim must be a multiple of 4 in [4, 256]");
    if (B < 1 || N < 1) return c->fail(FD_ERR_SHAPE, "B and N must be positive");
    if (B > c->cfg.max_batch || N > c->cfg.max_tokens)
        return c->fail(FD_ERR_SHAPE, "B=%d N=%d exceed the limits %d/%d", B, N, c->cfg.max_batch, c->cfg.max_tokens);
    return FD_OK;
}
}  // namespace

fd_status fd_embed_latent(fd_ctx* c, const fd_sampler_weights* sw, const float* z, int B, int N, void* x_out,
                          void* cuda_stream) {
    if (!c) return FD_ERR_INVALID_ARG;
    if (!z || !x_out) return c->fail(FD_ERR_INVALID_ARG, "null pointer argument");
    if (!aligned16(z) || !aligned16(x_out)) return c->fail(FD_ERR_INVALID_ARG, "z and x_out must be 16-byte aligned");
    fd_status s = sampler_args_ok(c, sw, B, N);
    if (s != FD_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int nl = 0;
    c->span_begin(FD_PROF_SAMPLER, st);
    cudaError_t e;
    if (c->cfg.dtype == FD_BF16)
        e = launch_embed<__nv_bfloat16>(z, static_cast<const __nv_bfloat16*>(sw->w_in), static_cast<const __nv_bfloat16*>(sw->b_in),
                                        static_cast<const __nv_bfloat16*>(sw->pos), static_cast<__nv_bfloat16*>(x_out), B, N,
                                        sw->latent_dim, c->cfg.hidden, st, &nl);
    else
        e = launch_embed<float>(z, static_cast<const float*>(sw->w_in), static_cast<const float*>(sw->b_in),
                                static_cast<const float*>(sw->pos), static_cast<float*>(x_out), B, N, sw->latent_dim,
                                c->cfg.hidden, st, &nl);
    c->span_end(nl, st);
    c->launches += nl;
    if (e != cudaSuccess) return c->fail(FD_ERR_CUDA, "embed launch failed: %s", cudaGetErrorString(e));
    return FD_OK;
}

fd_status fd_update_latent(fd_ctx* c, const fd_sampler_weights* sw, const float* z, const void* y,
                           const int32_t* active_idx, const int32_t* cu_active, const float* h, int B, int N,
                           float* drift_cache, float* z_next, void* cuda_stream) {
    if (!c) return FD_ERR_INVALID_ARG;
    if (!z || !y || !active_idx || !cu_active || !h || !drift_cache || !z_next)
        return c->fail(FD_ERR_INVALID_ARG, "null pointer argument");
    if (!aligned16(z) || !aligned16(y) || !aligned16(drift_cache) || !aligned16(z_next))
        return c->fail(FD_ERR_INVALID_ARG, "z, y, drift_cache and z_next must be 16-byte aligned");
    fd_status s = sampler_args_ok(c, sw, B, N);
    if (s != FD_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int nl = 0;
    c->span_begin(FD_PROF_SAMPLER, st);
    cudaError_t e;
    if (c->cfg.dtype == FD_BF16)
        e = launch_update<__nv_bfloat16>(z, static_cast<const __nv_bfloat16*>(y), active_idx, cu_active, h,
                                         static_cast<const __nv_bfloat16*>(sw->w_out), static_cast<const __nv_bfloat16*>(sw->b_out),
                                         drift_cache, z_next, B, N, sw->latent_dim, c->cfg.hidden, c->cfg.ln_eps, st, &nl);
    else
        e = launch_update<float>(z, static_cast<const float*>(y), active_idx, cu_active, h, static_cast<const float*>(sw->w_out),
                                 static_cast<const float*>(sw->b_out), drift_cache, z_next, B, N, sw->latent_dim, c->cfg.hidden,
                                 c->cfg.ln_eps, st, &nl);
    c->span_end(nl, st);
    c->launches += nl;
    if (e != cudaSuccess) return c->fail(FD_ERR_CUDA, "latent update launch failed: %s", cudaGetErrorString(e));
    return FD_OK;
}

fd_status fd_region_activity_noalloc(const float* z_cur, const float* z_prev, const int32_t* labels, int B, int N,
                                     int D, int R, const float* eps, float eta, int max_skip_k, float* delta_state,
                                     int32_t* skip_count, uint8_t* prev_active, float* score_out, float* weight_out,
                                     uint8_t* mask_out, int32_t* status_out, void* cuda_stream) {
    auto fail = [](fd_status s, const char* m) { g_create_error = m; return s; };
    if (!z_cur || !z_prev || !labels || !eps || !delta_state || !skip_count || !prev_active || !score_out ||
        !weight_out || !mask_out)
        return fail(FD_ERR_INVALID_ARG, "fd_region_activity_noalloc: null pointer argument");
    if (B < 1 || N < 1 || D < 1 || R < 1) return fail(FD_ERR_SHAPE, "fd_region_activity_noalloc: B, N, D, R must be positive");
    if ((long long)B * R > FD_NOALLOC_MAX_REGION_SLOTS)
        return fail(FD_ERR_SHAPE, "fd_region_activity_noalloc: B * R exceeds FD_NOALLOC_MAX_REGION_SLOTS");
    if (!(eta >= 0.f) || max_skip_k < 0) return fail(FD_ERR_INVALID_ARG, "fd_region_activity_noalloc: bad eta / max_skip_k");
    cudaError_t e = noalloc_gate(z_cur, z_prev, labels, B, N, D, R, eps, eta, max_skip_k, delta_state, skip_count,
                                 prev_active, score_out, weight_out, mask_out, status_out,
                                 static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) {
        g_create_error = std::string("fd_region_activity_noalloc: ") + cudaGetErrorString(e);
        return FD_ERR_CUDA;
    }
    return FD_OK;
}

static fd_status fd_regional_step_check(fd_ctx* c, const void* x, const void* cond, const int32_t* labels, const uint8_t* mask,
                                        int B, int N, int R, void* kv_cache, void* y, int32_t* active_idx_out,
                                        int32_t* cu_active_out) {
    if (!x || !cond || !labels || !mask || !kv_cache || !y || !active_idx_out || !cu_active_out)
        return c->fail(FD_ERR_INVALID_ARG, "null pointer argument");
    if (!aligned16(x) || !aligned16(cond) || !aligned16(kv_cache) || !aligned16(y))
        return c->fail(FD_ERR_INVALID_ARG, "x, cond, kv_cache, y must be 16-byte aligned");
    if (B < 1 || N < 1 || R < 1) return c->fail(FD_ERR_SHAPE, "B, N, R must be positive");
    if (B > c->cfg.max_batch || N > c->cfg.max_tokens || R > c->cfg.max_regions)
        return c->fail(FD_ERR_SHAPE, "B=%d N=%d R=%d exceed the limits %d/%d/%d", B, N, R, c->cfg.max_batch,
                       c->cfg.max_tokens, c->cfg.max_regions);
    if (R > N) return c->fail(FD_ERR_SHAPE, "R=%d exceeds N=%d", R, N);
    if (!aligned4(labels) || !aligned4(active_idx_out) || !aligned4(cu_active_out))
        return c->fail(FD_ERR_INVALID_ARG, "labels, active_idx_out, cu_active_out must be 4-byte aligned");
    return FD_OK;
}

fd_status fd_regional_step(fd_ctx* c, const void* x, const void* cond, const int32_t* labels, const uint8_t* mask,
                           int B, int N, int R, void* kv_cache, void* y, int32_t* active_idx_out,
                           int32_t* cu_active_out, void* cuda_stream) {
    if (!c) return FD_ERR_INVALID_ARG;
    fd_status s = fd_regional_step_check(c, x, cond, labels, mask, B, N, R, kv_cache, y, active_idx_out, cu_active_out);
    if (s != FD_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (c->cfg.dtype == FD_BF16)
        return run_step<__nv_bfloat16>(c, x, cond, labels, mask, B, N, R, kv_cache, y, active_idx_out, cu_active_out, st);
    return run_step<float>(c, x, cond, labels, mask, B, N, R, kv_cache, y, active_idx_out, cu_active_out, st);
}

fd_status fd_regional_step_mass(fd_ctx* c, const void* x, const void* cond, const int32_t* labels, const uint8_t* mask, int B,
                                int N, int R, void* kv_cache, void* y, int32_t* active_idx_out, int32_t* cu_active_out,
                                double* region_mass_out, void* cuda_stream) {
    if (!c) return FD_ERR_INVALID_ARG;
    if (!region_mass_out) return c->fail(FD_ERR_INVALID_ARG, "region_mass_out is null");
    fd_status s = fd_regional_step_check(c, x, cond, labels, mask, B, N, R, kv_cache, y, active_idx_out, cu_active_out);
    if (s != FD_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (c->cfg.dtype == FD_BF16)
        return run_step<__nv_bfloat16>(c, x, cond, labels, mask, B, N, R, kv_cache, y, active_idx_out, cu_active_out, st,
                                       region_mass_out);
    return run_step<float>(c, x, cond, labels, mask, B, N, R, kv_cache, y, active_idx_out, cu_active_out, st, region_mass_out);
}

fd_status fd_region_activity_attn(fd_ctx* c, const double* region_mass, const int32_t* region_sizes, int B, int R,
                                  const float* eps, float* rbar_state, float* delta_state, int32_t* skip_count,
                                  uint8_t* prev_active, float* importance_out, float* weight_out, uint8_t* mask_out,
                                  void* cuda_stream) {
    if (!c) return FD_ERR_INVALID_ARG;
    if (!region_mass || !region_sizes || !eps || !rbar_state || !delta_state || !skip_count || !prev_active ||
        !importance_out || !weight_out || !mask_out)
        return c->fail(FD_ERR_INVALID_ARG, "null pointer argument");
    if (B < 1 || R < 1) return c->fail(FD_ERR_SHAPE, "B and R must be positive");
    if (B > c->cfg.max_batch || R > c->cfg.max_regions)
        return c->fail(FD_ERR_SHAPE, "B=%d R=%d exceed the limits %d/%d", B, R, c->cfg.max_batch, c->cfg.max_regions);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int nl = 0;
    c->span_begin(FD_PROF_ACTIVITY, st);
    cudaError_t e = launch_attn_gate(region_mass, region_sizes, B, R, eps, c->cfg.gate_eta, c->cfg.max_skip_k, rbar_state,
                                     delta_state, skip_count, prev_active, importance_out, weight_out, mask_out, st, &nl);
    c->span_end(nl, st);
    c->launches += nl;
    if (e != cudaSuccess) return c->fail(FD_ERR_CUDA, "attention gate launch failed: %s", cudaGetErrorString(e));
    return FD_OK;
}

fd_status fd_set_block_variants(fd_ctx* c, const fd_block_variants* v) {
    if (!c) return FD_ERR_INVALID_ARG;
    if (!v) { c->var = fd_block_variants{}; return FD_OK; }
    if ((v->q_norm_w == nullptr) != (v->k_norm_w == nullptr))
        return c->fail(FD_ERR_INVALID_ARG, "q_norm_w and k_norm_w must be given together");
    if ((v->rope_cos == nullptr) != (v->rope_sin == nullptr))
        return c->fail(FD_ERR_INVALID_ARG, "rope_cos and rope_sin must be given together");
    if (v->rope_cos && (c->cfg.head_dim & 1)) return c->fail(FD_ERR_SHAPE, "rotary embedding needs an even head_dim");
    if (v->q_norm_w && !(v->qk_norm_eps >= 0.f)) return c->fail(FD_ERR_INVALID_ARG, "qk_norm_eps must be non-negative");
    const uintptr_t wmask = c->cfg.dtype == FD_BF16 ? 3 : 7;
    if ((reinterpret_cast<uintptr_t>(v->q_norm_w) | reinterpret_cast<uintptr_t>(v->k_norm_w) |
         reinterpret_cast<uintptr_t>(v->q_norm_w_text) | reinterpret_cast<uintptr_t>(v->k_norm_w_text)) & wmask)
        return c->fail(FD_ERR_INVALID_ARG, "QK-norm weights are misaligned");
    if ((v->q_norm_w_text == nullptr) != (v->k_norm_w_text == nullptr) || (v->q_norm_w_text && !v->q_norm_w))
        return c->fail(FD_ERR_INVALID_ARG, "the second stream's QK-norm weights come in pairs and need the first stream's");
    if ((reinterpret_cast<uintptr_t>(v->rope_cos) | reinterpret_cast<uintptr_t>(v->rope_sin)) & 3)
        return c->fail(FD_ERR_INVALID_ARG, "rotary tables are misaligned");
    c->var = *v;
    return FD_OK;
}

fd_status fd_set_text_stream(fd_ctx* c, const fd_weights* text_weights) {
    if (!c) return FD_ERR_INVALID_ARG;
    int32_t* text128 = c->at<int32_t>(c->lay.text_tiles);
    int32_t* text256 = text128 + c->lay.Mcap / 128 + 1;
    if (!text_weights) {
        c->dual = false;
        c->text_w = fd_weights{};
        if (c->tc) tc_plan_set_text(c->tc, nullptr, text128, text256, nullptr);
        return FD_OK;
    }
    const void* wp[10] = {text_weights->w_qkv, text_weights->b_qkv, text_weights->w_o, text_weights->b_o, text_weights->w_fc1,
                          text_weights->b_fc1, text_weights->w_fc2, text_weights->b_fc2, text_weights->w_ada, text_weights->b_ada};
    for (const void* p : wp)
        if (!p || !aligned16(p)) return c->fail(FD_ERR_INVALID_ARG, "weight pointer null or not 16-byte aligned");
    if (c->tc) {
        std::string err;
        if (!tc_plan_set_text(c->tc, text_weights, text128, text256, &err))
            return c->fail(FD_ERR_CUDA, "tensor maps of the second stream's weights: %s", err.c_str());
    }
    c->text_w = *text_weights;
    c->dual = true;
    return FD_OK;
}

fd_status fd_set_cross_attention(fd_ctx* c, const fd_cross_attention* x) {
    if (!c) return FD_ERR_INVALID_ARG;
    if (!x) {
        c->cross = fd_cross_attention{};
        if (c->tc) tc_plan_set_cross(c->tc, nullptr, nullptr, nullptr);
        return FD_OK;
    }
    const void* wp[5] = {x->w_q, x->b_q, x->w_o, x->b_o, x->ctx_kv};
    for (const void* p : wp)
        if (!p || !aligned16(p)) return c->fail(FD_ERR_INVALID_ARG, "cross-attention pointer null or not 16-byte aligned");
    if (x->n_ctx < 1 || x->ctx_batch < 1 || x->ctx_batch > c->cfg.max_batch)
        return c->fail(FD_ERR_SHAPE, "n_ctx must be positive and ctx_batch in [1, max_batch]");
    if (c->tc) {
        std::string err;
        if (!tc_plan_set_cross(c->tc, x->w_q, x->w_o, &err))
            return c->fail(FD_ERR_CUDA, "tensor maps of the cross-attention weights: %s", err.c_str());
    }
    c->cross = *x;
    return FD_OK;
}

namespace {
// shared by the two FP8 entry points: checks, tensor maps, host copy of the activation scales
fd_status set_fp8(fd_ctx* c, const fd_fp8_operands* f, bool text) {
    fd_fp8_operands& dst = text ? c->fp8_text : c->fp8;
    std::vector<float>& dst_a = text ? c->fp8_text_a : c->fp8_a;
    if (!f) {
        dst = fd_fp8_operands{};
        dst_a.clear();
        if (c->tc) tc_plan_set_fp8(c->tc, nullptr, nullptr, nullptr, nullptr, text);
        return FD_OK;
    }
    if (!c->use_tc || !c->tc) return c->fail(FD_ERR_UNSUPPORTED, "FP8 operands need the tensor-core engine (bf16 storage)");
    const void* wp[6] = {f->w8_qkv, f->s_qkv, f->w8_fc1, f->s_fc1, f->w8_fc2, f->s_fc2};
    for (const void* p : wp)
        if (!p || !aligned16(p)) return c->fail(FD_ERR_INVALID_ARG, "FP8 operand pointer null or not 16-byte aligned");
    if (!f->a_scale) return c->fail(FD_ERR_INVALID_ARG, "a_scale is null");
    const size_t n = (size_t)c->cfg.n_blocks * 3;
    for (size_t i = 0; i < n; ++i)
        if (!(f->a_scale[i] > 0.f) || !(1.0f / f->a_scale[i] < 3.0e38f))
            return c->fail(FD_ERR_INVALID_ARG, "activation scales must be positive and finite");
    std::string err;
    if (!tc_plan_set_fp8(c->tc, f->w8_qkv, f->w8_fc1, f->w8_fc2, &err, text))
        return c->fail(FD_ERR_UNSUPPORTED, "FP8 operands: %s", err.c_str());
    dst = *f;
    dst_a.assign(f->a_scale, f->a_scale + n);
    dst.a_scale = nullptr;                    // the host array was copied
    return FD_OK;
}
}  // namespace

fd_status fd_set_fp8_operands(fd_ctx* c, const fd_fp8_operands* f) {
    if (!c) return FD_ERR_INVALID_ARG;
    return set_fp8(c, f, false);
}

fd_status fd_set_fp8_text_stream(fd_ctx* c, const fd_fp8_operands* f) {
    if (!c) return FD_ERR_INVALID_ARG;
    return set_fp8(c, f, true);
}

fd_status fd_poll_status(fd_ctx* c, void* cuda_stream) {
    if (!c) return FD_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    Control h{};
    cudaError_t e = cudaMemcpyAsync(&h, c->ctl(), sizeof(Control), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return c->fail(FD_ERR_CUDA, "status read failed: %s", cudaGetErrorString(e));
    if (h.status != 0) {
        cudaMemsetAsync(c->ctl(), 0, 2 * sizeof(int32_t), st);
        return c->fail(static_cast<fd_status>(h.status), "device-side check failed: code %d, detail %d", h.status,
                       h.detail);
    }
    return FD_OK;
}

fd_status fd_debug_buffer(fd_ctx* c, int which, void** device_ptr_out, size_t* bytes_out) {
    if (!c) return FD_ERR_INVALID_ARG;
    if (!device_ptr_out || !bytes_out) return c->fail(FD_ERR_INVALID_ARG, "null output pointer");
    const Layout& l = c->lay;
    const size_t es = c->cfg.dtype == FD_BF16 ? 2 : 4;
    switch (which) {
        case FD_BUF_ACT: *device_ptr_out = c->ws + l.act; *bytes_out = (size_t)l.Mcap * c->cfg.hidden * es; break;
        case FD_BUF_HIDDEN: *device_ptr_out = c->ws + l.g; *bytes_out = (size_t)l.Mcap * c->cfg.mlp_dim * es; break;
        case FD_BUF_RESID: *device_ptr_out = c->ws + l.resid; *bytes_out = (size_t)l.Mcap * c->cfg.hidden * sizeof(float); break;
        case FD_BUF_Q: *device_ptr_out = c->ws + l.q; *bytes_out = (size_t)l.Mcap * l.q_ld * es; break;
        case FD_BUF_ATTN: *device_ptr_out = c->ws + l.o; *bytes_out = (size_t)l.Mcap * c->cfg.hidden * es; break;
        default: return c->fail(FD_ERR_INVALID_ARG, "unknown buffer %d", which);
    }
    return FD_OK;
}

fd_status fd_profile_enable(fd_ctx* c, int enable) {
    if (!c) return FD_ERR_INVALID_ARG;
    c->profiling = enable != 0;
    return FD_OK;
}

fd_status fd_profile_read(fd_ctx* c, void* cuda_stream, float* ms_out, int32_t* kernels_out) {
    if (!c) return FD_ERR_INVALID_ARG;
    if (!ms_out || !kernels_out) return c->fail(FD_ERR_INVALID_ARG, "null output array");
    cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return c->fail(FD_ERR_CUDA, "stream synchronise failed: %s", cudaGetErrorString(e));
    for (auto& s : c->spans) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, s.a, s.b) == cudaSuccess && s.group >= 0 && s.group < FD_PROF_GROUPS) {
            ms_out[s.group] += ms;
            kernels_out[s.group] += s.kernels;
        }
        c->pool.push_back(s.a);
        c->pool.push_back(s.b);
    }
    c->spans.clear();
    return FD_OK;
}

fd_status fd_selftest_bounded_wait(fd_ctx* c, void* cuda_stream) {
    if (!c) return FD_ERR_INVALID_ARG;
    int nl = 0;
    cudaError_t e = launch_bounded_wait_selftest(c->ctl(), static_cast<cudaStream_t>(cuda_stream), &nl);
    c->launches += nl;
    if (e != cudaSuccess) return c->fail(FD_ERR_CUDA, "self-test launch failed: %s", cudaGetErrorString(e));
    return FD_OK;
}

int64_t fd_launch_count(const fd_ctx* c) { return c ? c->launches : 0; }

fd_status fd_destroy(fd_ctx* c) {
    if (!c) return FD_ERR_INVALID_ARG;
    // Wait for whatever the context still has in flight (the workspace goes back to the caller), then report a
    // device-side problem nobody has polled for yet.
    fd_status pending = FD_OK;
    Control h{};
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess) e = cudaMemcpy(&h, c->ctl(), sizeof(Control), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) {
        pending = FD_ERR_CUDA;
        g_create_error = std::string("fd_destroy: ") + cudaGetErrorString(e);
    } else if (h.status != 0) {
        pending = static_cast<fd_status>(h.status);
        char buf[128];
        snprintf(buf, sizeof buf, "fd_destroy: unpolled device-side status %d, detail %d", h.status, h.detail);
        g_create_error = buf;
    }
    tc_plan_destroy(c->tc);
    for (auto& s : c->spans) { c->pool.push_back(s.a); c->pool.push_back(s.b); }
    for (cudaEvent_t ev : c->pool) cudaEventDestroy(ev);
    delete c;
    return pending;
}

const char* fd_last_error(const fd_ctx* c) { return c ? c->err.c_str() : g_create_error.c_str(); }

}  // extern "C"
