// GEMM epilogues shared by the CUDA-core and tensor-core kernels.  Each call finishes four
// consecutive output columns of one compact row:
//   EPI_QKV   bias, then Q stays compact while K and V rows are scattered into the request's cache
//             (skipped tokens' rows are never written: they keep the previous step's K/V),
//   EPI_RESID bias, adaLN gate, residual add into the fp32 stream; the last block also scatters
//             the row into y,
//   EPI_GELU  bias and tanh-GELU.
#pragma once
#include <cuda.h>
#include "common.cuh"
#include "ptx.cuh"

namespace fd {

template <typename T> __device__ __forceinline__ void store4(T* p, float a, float b, float c, float d);
template <> __device__ __forceinline__ void store4<float>(float* p, float a, float b, float c, float d) {
    *reinterpret_cast<float4*>(p) = make_float4(a, b, c, d);
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float a, float b, float c, float d) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&lo);
    u.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = u;
}
template <typename T> __device__ __forceinline__ void load4(const T* p, float* f);
template <> __device__ __forceinline__ void load4<float>(const float* p, float* f) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}
template <> __device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float* f) {
    const uint2 u = *reinterpret_cast<const uint2*>(p);
    f[0] = __uint_as_float(u.x << 16); f[1] = __uint_as_float(u.x & 0xffff0000u);
    f[2] = __uint_as_float(u.y << 16); f[3] = __uint_as_float(u.y & 0xffff0000u);
}

// row: compact row (< a_total), col: first of four columns, tok: active_idx[row]
template <typename T, int KIND>
__device__ __forceinline__ void epilogue4(const EpiParams& ep, int row, int col, int tok, const float* acc) {
    float bias[4];
    load4<T>(reinterpret_cast<const T*>(ep.bias) + col, bias);
    float v[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) v[i] = acc[i] + bias[i];
    if constexpr (KIND == EPI_QKV) {
        const int sec = col / ep.H, c = col - sec * ep.H;
        if (sec == 0) {
            store4<T>(reinterpret_cast<T*>(ep.q) + (size_t)row * ep.q_ld + c, v[0], v[1], v[2], v[3]);
        } else {
            const int b = tok / ep.N, j = tok - b * ep.N;
            T* dst = reinterpret_cast<T*>(ep.kv) + (((size_t)b * 2 + (sec - 1)) * ep.N + j) * ep.H + c;
            store4<T>(dst, v[0], v[1], v[2], v[3]);
        }
    } else if constexpr (KIND == EPI_RESID) {
        const int b = tok / ep.N;
        const float4 g = *reinterpret_cast<const float4*>(ep.gate + (ep.ungated ? (size_t)0 : (size_t)b * 6 * ep.H) + col);
        float* rp = ep.resid + (size_t)row * ep.H + col;
        float4 r = *reinterpret_cast<const float4*>(rp);
        r.x = fmaf(g.x, v[0], r.x); r.y = fmaf(g.y, v[1], r.y);
        r.z = fmaf(g.z, v[2], r.z); r.w = fmaf(g.w, v[3], r.w);
        *reinterpret_cast<float4*>(rp) = r;
        if (ep.y) store4<T>(reinterpret_cast<T*>(ep.y) + (size_t)tok * ep.H + col, r.x, r.y, r.z, r.w);
    } else {
        store4<T>(reinterpret_cast<T*>(ep.out) + (size_t)row * ep.out_ld + col, gelu_tanh(v[0]), gelu_tanh(v[1]),
                  gelu_tanh(v[2]), gelu_tanh(v[3]));
    }
}

}  // namespace fd

// ---- tensor-core epilogues: 16-byte units transposed through shared memory ----------------------
// After tcgen05.ld every thread holds consecutive columns of ONE row, so storing straight from those
// registers makes each warp instruction touch 32 different rows (16 bytes out of 32 different
// 128-byte lines).  That pattern saturates the L1/LSU pipe and slows the MMAs running next to it.
// Instead the warp's chunk (32 rows x 128 bytes of output) goes through a 4 KB shared-memory tile in
// 16-byte units: row t writes its 8 units, then lane t reads unit (t % 8) of rows 4 i + t / 8.  Each
// global instruction then covers 4 complete 128-byte row segments.  The unit index is XORed with the
// row's low bits so that both the writes and the reads are bank-conflict free.
namespace fd {

constexpr int EPI_STAGE_BYTES_PER_WARP = 32 * 128;

__device__ __forceinline__ float tanh_fast(float x) {
    float y;
    asm("tanh.approx.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float gelu_tanh_fast(float a) {
    const float u = 0.7978845608028654f * fmaf(0.044715f * a * a, a, a);
    return 0.5f * a * (1.0f + tanh_fast(u));
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&h);
}
__device__ __forceinline__ uint4* unit_ptr(uint8_t* stage, int row, int u) {
    return reinterpret_cast<uint4*>(stage + row * 128 + ((u ^ (row & 7)) << 4));
}

// What lane t knows about "its" row (row_base + t) of the warp's 32 rows, computed once per tile so that the
// chunk loops contain no divisions and no 64-bit multiplies; other lanes fetch it with shuffles.
struct RowInfo {
    uint32_t valid;    // bit t: row t of the warp's 32 exists and belongs to the stream this launch finishes (same in all lanes)
    int gate_off;      // b * 6H: offset of the request's adaLN vectors (of the row's stream)
    uint32_t y_lo, y_hi;   // tok * H: element offset of the row in y (EPI_RESID) or of the token in the K plane (EPI_QKV)
    int pos;           // EPI_QKV: the token's index inside its request (row of the rotary tables)
};

// EPI_RESID: 32 fp32 accumulator columns per row; resid += gate * (acc + bias); the last block also
// scatters the row into y.
// F8: the accumulator holds products of 8-bit operands and is scaled by col_scale[col] * act_scale before the bias.
template <bool F8>
__device__ __forceinline__ void epilogue_resid_chunk(const EpiParams& ep, uint8_t* stage, int lane, int row_base,
                                                     int col0, const uint32_t* acc, const RowInfo& ri) {
    using T = __nv_bfloat16;
#pragma unroll
    for (int u = 0; u < 8; ++u) *unit_ptr(stage, lane, u) = make_uint4(acc[4 * u], acc[4 * u + 1], acc[4 * u + 2], acc[4 * u + 3]);
    __syncwarp();
    const int u = lane & 7, rsub = lane >> 3;
    const int col = col0 + u * 4;
    float bias[4];
    load4<T>(reinterpret_cast<const T*>(ep.bias) + col, bias);
    float4 cs = make_float4(1.f, 1.f, 1.f, 1.f);
    if constexpr (F8) {
        cs = __ldg(reinterpret_cast<const float4*>(ep.col_scale + col));
        cs.x *= ep.act_scale; cs.y *= ep.act_scale; cs.z *= ep.act_scale; cs.w *= ep.act_scale;
    }
    // acc (+ scaling) + bias of one staged unit
    auto lin = [&](const uint4& a, float& x, float& y, float& z, float& w) {
        if constexpr (F8) {
            x = fmaf(__uint_as_float(a.x), cs.x, bias[0]); y = fmaf(__uint_as_float(a.y), cs.y, bias[1]);
            z = fmaf(__uint_as_float(a.z), cs.z, bias[2]); w = fmaf(__uint_as_float(a.w), cs.w, bias[3]);
        } else {
            x = __uint_as_float(a.x) + bias[0]; y = __uint_as_float(a.y) + bias[1];
            z = __uint_as_float(a.z) + bias[2]; w = __uint_as_float(a.w) + bias[3];
        }
    };
    float* rp = ep.resid + (size_t)(row_base + rsub) * ep.H + col;      // rows rsub, rsub + 4, ...
    const size_t rstride = (size_t)4 * ep.H;
    const float* gp = ep.gate + col;
    T* yb = reinterpret_cast<T*>(ep.y);
    if (!yb) {
        // Every element of the residual stream receives exactly one contribution from this kernel, so the
        // update is a plain "add to memory": a vector reduction instruction does it without reading the row
        // back into the SM (no load latency in the epilogue, half the memory instructions); the result is the
        // same single fp32 addition as load / add / store.
        float4 gv[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int go = __shfl_sync(0xffffffffu, ri.gate_off, 4 * i + rsub);
            if ((ri.valid >> (4 * i + rsub)) & 1u) gv[i] = __ldg(reinterpret_cast<const float4*>(gp + go));
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = 4 * i + rsub;
            if ((ri.valid >> r) & 1u) {
                const uint4 a = *unit_ptr(stage, r, u);
                float x, y, z, w;
                lin(a, x, y, z, w);
                x *= gv[i].x; y *= gv[i].y; z *= gv[i].z; w *= gv[i].w;
                asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(rp + i * rstride), "f"(x), "f"(y), "f"(z), "f"(w)
                             : "memory");
            }
        }
        __syncwarp();
        return;
    }
    // last block: the final value is needed for the scatter into y, so read, add, write
    float4 rv[8], gv[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = 4 * i + rsub;
        const int go = __shfl_sync(0xffffffffu, ri.gate_off, r);
        if ((ri.valid >> r) & 1u) {
            rv[i] = *reinterpret_cast<const float4*>(rp + i * rstride);
            gv[i] = __ldg(reinterpret_cast<const float4*>(gp + go));
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = 4 * i + rsub;
        const uint32_t ylo = __shfl_sync(0xffffffffu, ri.y_lo, r), yhi = __shfl_sync(0xffffffffu, ri.y_hi, r);
        if ((ri.valid >> r) & 1u) {
            const uint4 a = *unit_ptr(stage, r, u);
            float4 v = rv[i];
            float x, y, z, w;
            lin(a, x, y, z, w);
            v.x = fmaf(gv[i].x, x, v.x); v.y = fmaf(gv[i].y, y, v.y);
            v.z = fmaf(gv[i].z, z, v.z); v.w = fmaf(gv[i].w, w, v.w);
            *reinterpret_cast<float4*>(rp + i * rstride) = v;
            store4<T>(yb + (((size_t)yhi << 32) | ylo) + col, v.x, v.y, v.z, v.w);
        }
    }
    __syncwarp();
}

// EPI_RESID through the TMA: the warp's 32 x 32 products gate * (acc + bias) go back into its staging tile as
// plain fp32 rows and one bulk tensor reduction adds the tile onto the residual stream.  The SM's load/store path
// issues per-thread reductions at about 9 bytes per clock, which made this epilogue as long as the main loop of a
// K = 1536 tile; the bulk form hands whole 128-byte rows to the L2.
template <bool F8>
__device__ __forceinline__ void epilogue_resid_chunk_tma(const EpiParams& ep, uint8_t* stage, int lane, int row_base,
                                                         int col0, const uint32_t* acc, const RowInfo& ri,
                                                         const CUtensorMap* tm_r) {
    using T = __nv_bfloat16;
    if (lane == 0) ptx::bulk_wait_read_all();                      // the previous chunk's reduction has read the tile
    __syncwarp();
#pragma unroll
    for (int k = 0; k < 8; ++k) *unit_ptr(stage, lane, k) = make_uint4(acc[4 * k], acc[4 * k + 1], acc[4 * k + 2], acc[4 * k + 3]);
    __syncwarp();
    const int u = lane & 7, rsub = lane >> 3;
    const int col = col0 + u * 4;
    float bias[4];
    load4<T>(reinterpret_cast<const T*>(ep.bias) + col, bias);
    const float* gp = ep.gate + col;
    float4 cs = make_float4(1.f, 1.f, 1.f, 1.f);
    if constexpr (F8) {
        cs = __ldg(reinterpret_cast<const float4*>(ep.col_scale + col));
        cs.x *= ep.act_scale; cs.y *= ep.act_scale; cs.z *= ep.act_scale; cs.w *= ep.act_scale;
    }
    float4 gv[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int go = __shfl_sync(0xffffffffu, ri.gate_off, 4 * i + rsub);
        gv[i] = ((ri.valid >> (4 * i + rsub)) & 1u) ? __ldg(reinterpret_cast<const float4*>(gp + go)) : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // The tile is rewritten in place, row by row: the eight lanes of a row read their (swizzled) units, then write the
    // row's 128 bytes in plain order; rows past the last active row (or of the other stream) add zeros.
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int r = 4 * i + rsub;
        const uint4 a = *unit_ptr(stage, r, u);
        __syncwarp();
        float4 v;
        if constexpr (F8) {
            v.x = gv[i].x * fmaf(__uint_as_float(a.x), cs.x, bias[0]); v.y = gv[i].y * fmaf(__uint_as_float(a.y), cs.y, bias[1]);
            v.z = gv[i].z * fmaf(__uint_as_float(a.z), cs.z, bias[2]); v.w = gv[i].w * fmaf(__uint_as_float(a.w), cs.w, bias[3]);
        } else {
            v.x = gv[i].x * (__uint_as_float(a.x) + bias[0]); v.y = gv[i].y * (__uint_as_float(a.y) + bias[1]);
            v.z = gv[i].z * (__uint_as_float(a.z) + bias[2]); v.w = gv[i].w * (__uint_as_float(a.w) + bias[3]);
        }
        *reinterpret_cast<float4*>(stage + r * 128 + u * 16) = v;
    }
    ptx::fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) ptx::tma_reduce_add_2d(tm_r, col0, row_base, stage);
}

// EPI_QKV / EPI_GELU: 64 fp32 accumulator columns per row, bf16 outputs (8 columns per 16-byte unit).
// F8: the accumulator holds products of 8-bit operands and is scaled by col_scale[col] * act_scale before the bias;
// EPI_GELU then writes its 64 values per row as 64 E4M3 bytes of value * out_inv_scale (the fc2 operand).
// QkVar: block variants fused into EPI_QKV for this chunk (all lanes alike): the lane's row is scaled by `rs` (its
// head's 1 / rms) and the channel weights gamma[64] (this chunk's part of the head; nullptr: no normalisation), then
// its channel pairs are rotated by the row's angles cs / sn [32] (this chunk's part; nullptr: no rotation).
struct QkVar {
    float rs;
    const __nv_bfloat16* gamma;
    const float* cs;
    const float* sn;
};

template <int KIND, bool F8>
__device__ __forceinline__ void epilogue_bf16_chunk(const EpiParams& ep, uint8_t* stage, int lane, int row_base,
                                                    int col0, const uint32_t* acc, const RowInfo& ri,
                                                    const QkVar* var = nullptr) {
    using T = __nv_bfloat16;
    const uint4* bp = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(ep.bias) + col0);
    const float4* sp = reinterpret_cast<const float4*>(ep.col_scale + col0);
    uint32_t q8[4];                                            // F8 GELU: four values per word, a 16-byte unit per two u
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const uint4 b = __ldg(bp + u);
        const uint32_t w[4] = {b.x, b.y, b.z, b.w};
        float v[8];
        if constexpr (F8) {
            const float4 s0 = __ldg(sp + 2 * u), s1 = __ldg(sp + 2 * u + 1);
            const float sc[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                v[2 * k] = fmaf(__uint_as_float(acc[8 * u + 2 * k]), sc[2 * k] * ep.act_scale, __uint_as_float(w[k] << 16));
                v[2 * k + 1] = fmaf(__uint_as_float(acc[8 * u + 2 * k + 1]), sc[2 * k + 1] * ep.act_scale,
                                    __uint_as_float(w[k] & 0xffff0000u));
            }
        } else {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                v[2 * k] = __uint_as_float(acc[8 * u + 2 * k]) + __uint_as_float(w[k] << 16);
                v[2 * k + 1] = __uint_as_float(acc[8 * u + 2 * k + 1]) + __uint_as_float(w[k] & 0xffff0000u);
            }
        }
        if constexpr (KIND == EPI_GELU) {
#pragma unroll
            for (int k = 0; k < 8; ++k) v[k] = gelu_tanh_fast(v[k]);
        }
        if constexpr (KIND == EPI_QKV) {
            if (var) {
                if (var->gamma) {
                    const uint4 g = __ldg(reinterpret_cast<const uint4*>(var->gamma) + u);
                    const uint32_t gw[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        v[2 * k] *= var->rs * __uint_as_float(gw[k] << 16);
                        v[2 * k + 1] *= var->rs * __uint_as_float(gw[k] & 0xffff0000u);
                    }
                }
                if (var->cs) {
                    const float4 c4 = __ldg(reinterpret_cast<const float4*>(var->cs) + u);
                    const float4 s4 = __ldg(reinterpret_cast<const float4*>(var->sn) + u);
                    const float cc[4] = {c4.x, c4.y, c4.z, c4.w}, ss[4] = {s4.x, s4.y, s4.z, s4.w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const float a = v[2 * k], b = v[2 * k + 1];
                        v[2 * k] = a * cc[k] - b * ss[k];
                        v[2 * k + 1] = a * ss[k] + b * cc[k];
                    }
                }
            }
        }
        if constexpr (KIND == EPI_GELU && F8) {
            const float qs = ep.out_inv_scale;
            q8[2 * (u & 1)] = pack4_e4m3(v[0] * qs, v[1] * qs, v[2] * qs, v[3] * qs);
            q8[2 * (u & 1) + 1] = pack4_e4m3(v[4] * qs, v[5] * qs, v[6] * qs, v[7] * qs);
            if (u & 1) *unit_ptr(stage, lane, u >> 1) = make_uint4(q8[0], q8[1], q8[2], q8[3]);
        } else {
            *unit_ptr(stage, lane, u) = make_uint4(pack2_bf16(v[0], v[1]), pack2_bf16(v[2], v[3]), pack2_bf16(v[4], v[5]),
                                                   pack2_bf16(v[6], v[7]));
        }
    }
    __syncwarp();
    if constexpr (KIND == EPI_GELU && F8) {
        // lane t: unit t % 4 (16 columns) of rows 8 i + t / 4: every store instruction covers eight 64-byte row segments
        const int u4 = lane & 3, rs8 = lane >> 2;
        uint8_t* ob = reinterpret_cast<uint8_t*>(ep.out) + (size_t)(row_base + rs8) * ep.out_ld + col0 + u4 * 16;
        const size_t ostride = (size_t)8 * ep.out_ld;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int r = 8 * i + rs8;
            if ((ri.valid >> r) & 1u) *reinterpret_cast<uint4*>(ob + i * ostride) = *unit_ptr(stage, r, u4);
        }
        __syncwarp();
        return;
    }
    const int u = lane & 7, rsub = lane >> 3;
    const int col = col0 + u * 8;
    if constexpr (KIND == EPI_GELU) {
        T* ob = reinterpret_cast<T*>(ep.out) + (size_t)(row_base + rsub) * ep.out_ld + col;
        const size_t ostride = (size_t)4 * ep.out_ld;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int r = 4 * i + rsub;
            if ((ri.valid >> r) & 1u) *reinterpret_cast<uint4*>(ob + i * ostride) = *unit_ptr(stage, r, u);
        }
    } else {
        const int sec = col0 / ep.H;                              // the 64 columns of a chunk share their section
        const int c = col - sec * ep.H;
        if (sec == 0) {
            int qc = c;
            if (ep.q_head_dim) { const int hd = c / ep.q_head_dim; qc = hd * ep.q_head_pad + (c - hd * ep.q_head_dim); }
            T* qb = reinterpret_cast<T*>(ep.q) + (size_t)(row_base + rsub) * ep.q_ld + qc;
            const size_t qstride = (size_t)4 * ep.q_ld;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = 4 * i + rsub;
                if ((ri.valid >> r) & 1u) *reinterpret_cast<uint4*>(qb + i * qstride) = *unit_ptr(stage, r, u);
            }
        } else {
            T* kvb = reinterpret_cast<T*>(ep.kv) + (size_t)(sec - 1) * ep.N * ep.H + c;     // K plane, or V plane N*H further
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = 4 * i + rsub;
                const uint32_t lo = __shfl_sync(0xffffffffu, ri.y_lo, r), hi = __shfl_sync(0xffffffffu, ri.y_hi, r);
                if ((ri.valid >> r) & 1u) *reinterpret_cast<uint4*>(kvb + (((size_t)hi << 32) | lo)) = *unit_ptr(stage, r, u);
            }
        }
    }
    __syncwarp();
}

// The residual rows an EPI_RESID tile will read usually sit in DRAM by the time the GEMM runs (32 MB of
// fp32 rows, several kernels since they were written).  The epilogue warps are idle while the tile's MMAs
// run, so they pull their rows' segments into L2 first; the loads in the epilogue then cost an L2 hit.
__device__ __forceinline__ void epilogue_prefetch_resid(const EpiParams& ep, int lane, int row_base, int a_total,
                                                        int col_begin, int n_cols) {
    const int row = row_base + lane;
    if (row < a_total) {
        const char* p = reinterpret_cast<const char*>(ep.resid + (size_t)row * ep.H + col_begin);
        for (int off = 0; off < n_cols * 4; off += 128)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(p + off));
    }
}

// Per-lane row data of a warp's 32 rows (request, cache / output row): depends only on the tile, so the caller can
// fetch it while the tile's products are still running.
template <int KIND>
__device__ __forceinline__ RowInfo epilogue_row_info(const EpiParams& ep, int lane, int row_base, int a_total) {
    RowInfo ri{0u, 0, 0u, 0u, 0};
    bool ok = row_base + lane < a_total;
    if ((KIND != EPI_GELU || ep.group >= 0) && ok) {
        const int tok = ep.active_idx[row_base + lane];
        const int b = tok / ep.N;
        ri.gate_off = ep.ungated ? 0 : b * 6 * ep.H;
        if (ep.group >= 0) {                                     // dual stream: this launch owns one stream's rows
            const int text = ep.labels[tok] == ep.R ? 1 : 0;
            ok = text == ep.group;
            if (text && !ep.ungated) ri.gate_off += ep.text_mod_off;
        }
        const size_t off = KIND == EPI_RESID ? (size_t)tok * ep.H : ((size_t)b * 2 * ep.N + (tok - b * ep.N)) * ep.H;
        ri.y_lo = (uint32_t)off;
        ri.y_hi = (uint32_t)(off >> 32);
        ri.pos = tok - b * ep.N;
    }
    ri.valid = __ballot_sync(0xffffffffu, ok);
    return ri;
}

// one warp's share of a tile: rows [row_base, row_base + 32), columns [c_begin, c_end) of the accumulator at t_row
template <int KIND, bool F8 = false>
__device__ __forceinline__ void epilogue_warp(const EpiParams& ep, uint8_t* stage, int lane, int row_base, int a_total,
                                              uint32_t t_row, int tile_col0, int c_begin, int c_end, const RowInfo& ri,
                                              const CUtensorMap* tm_r = nullptr) {
    const bool live = ri.valid != 0u;                            // warp-uniform
    (void)a_total;
    if constexpr (KIND == EPI_RESID) {
#pragma unroll 1
        for (int c0 = c_begin; c0 < c_end; c0 += 32) {
            uint32_t r[32];
            ptx::tmem_ld32(t_row + c0, r);
            ptx::tmem_wait_ld();
            if (live) {
                if (tm_r && !ep.y) epilogue_resid_chunk_tma<F8>(ep, stage, lane, row_base, tile_col0 + c0, r, ri, tm_r);
                else epilogue_resid_chunk<F8>(ep, stage, lane, row_base, tile_col0 + c0, r, ri);
            }
        }
    } else {
        if constexpr (KIND == EPI_QKV) {
            if (ep.qk_head_dim) {
                // Block variants fused: one head (of Q, K or V) at a time.  The head's sum of squares needs all of its
                // columns, which are one or two chunks of the accumulator: a first pass over them only sums, the
                // second one normalises, rotates and stores (the accumulator is read twice; it sits in TMEM).
                using T = __nv_bfloat16;
                const int dh = ep.qk_head_dim;
#pragma unroll 1
                for (int h0 = c_begin; h0 < c_end; h0 += dh) {
                    const int col_h = tile_col0 + h0;
                    const int sec = col_h / ep.H;                        // 0: queries, 1: keys, 2: values
                    const T* gamma = sec == 0 ? static_cast<const T*>(ep.qn_w) : sec == 1 ? static_cast<const T*>(ep.kn_w) : nullptr;
                    const bool rot = sec < 2 && ep.rope_cos != nullptr;
                    QkVar var{1.f, nullptr, nullptr, nullptr};
                    if (gamma) {
                        float ssq = 0.f;
#pragma unroll 1
                        for (int c0 = h0; c0 < h0 + dh; c0 += 64) {
                            uint32_t r[64];
                            ptx::tmem_ld32(t_row + c0, r);
                            ptx::tmem_ld32(t_row + c0 + 32, r + 32);
                            ptx::tmem_wait_ld();
                            const uint4* bp = reinterpret_cast<const uint4*>(reinterpret_cast<const T*>(ep.bias) + tile_col0 + c0);
                            const float4* sp = reinterpret_cast<const float4*>(ep.col_scale + tile_col0 + c0);
#pragma unroll
                            for (int u = 0; u < 8; ++u) {
                                const uint4 b = __ldg(bp + u);
                                const uint32_t w[4] = {b.x, b.y, b.z, b.w};
                                float sc[8] = {1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f, 1.f};
                                if constexpr (F8) {
                                    const float4 s0 = __ldg(sp + 2 * u), s1 = __ldg(sp + 2 * u + 1);
                                    sc[0] = s0.x * ep.act_scale; sc[1] = s0.y * ep.act_scale; sc[2] = s0.z * ep.act_scale; sc[3] = s0.w * ep.act_scale;
                                    sc[4] = s1.x * ep.act_scale; sc[5] = s1.y * ep.act_scale; sc[6] = s1.z * ep.act_scale; sc[7] = s1.w * ep.act_scale;
                                }
#pragma unroll
                                for (int k = 0; k < 4; ++k) {
                                    const float a = fmaf(__uint_as_float(r[8 * u + 2 * k]), sc[2 * k], __uint_as_float(w[k] << 16));
                                    const float bb = fmaf(__uint_as_float(r[8 * u + 2 * k + 1]), sc[2 * k + 1], __uint_as_float(w[k] & 0xffff0000u));
                                    ssq = fmaf(a, a, ssq);
                                    ssq = fmaf(bb, bb, ssq);
                                }
                            }
                        }
                        var.rs = rsqrtf(ssq / (float)dh + ep.qk_eps);
                    }
#pragma unroll 1
                    for (int c0 = h0; c0 < h0 + dh; c0 += 64) {
                        uint32_t r[64];
                        ptx::tmem_ld32(t_row + c0, r);
                        ptx::tmem_ld32(t_row + c0 + 32, r + 32);
                        ptx::tmem_wait_ld();
                        var.gamma = gamma ? gamma + (c0 - h0) : nullptr;
                        var.cs = rot ? ep.rope_cos + (size_t)ri.pos * (dh >> 1) + ((c0 - h0) >> 1) : nullptr;
                        var.sn = rot ? ep.rope_sin + (size_t)ri.pos * (dh >> 1) + ((c0 - h0) >> 1) : nullptr;
                        if (live) epilogue_bf16_chunk<KIND, F8>(ep, stage, lane, row_base, tile_col0 + c0, r, ri, (gamma || rot) ? &var : nullptr);
                    }
                }
                return;
            }
        }
#pragma unroll 1
        for (int c0 = c_begin; c0 < c_end; c0 += 64) {
            uint32_t r[64];
            ptx::tmem_ld32(t_row + c0, r);
            ptx::tmem_ld32(t_row + c0 + 32, r + 32);
            ptx::tmem_wait_ld();
            if (live) epilogue_bf16_chunk<KIND, F8>(ep, stage, lane, row_base, tile_col0 + c0, r, ri);
        }
    }
}

}  // namespace fd
