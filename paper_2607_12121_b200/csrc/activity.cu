// Patch Gate on the latent change (paper Sec. 4.2; Appendix A.1 Eq. delta-i, Eq. gate-weight,
// Eq. forced-reactivation).
//
// Kernel 1 streams z_cur / z_prev once and accumulates, per region, the sum of squared differences
// (fp32 within a run of tokens of one region, fp64 across runs and CTAs) and the token count.  Tokens of
// regions whose change magnitude is frozen (skipped at the previous step) are not read at all.  Its main
// form stages both operands through shared memory with bulk copies (below); rows wider than a ring
// stage take the plain vector-load form (per-CTA shared accumulators, up to ACT_SMEM_LIMIT / 12 regions);
// unaligned rows, channel counts that are no multiple of 4 and larger region counts take the scalar form,
// which adds straight into the global accumulators.
// Kernel 2 (one CTA per request) turns the sums into delta, weights, mask and the next state, and
// clears the accumulators for the next call.
#include "common.cuh"
#include "ptx.cuh"

#include <mutex>

namespace fd {

namespace {

constexpr int ACT_THREADS = 256;
constexpr int ACT_SMEM_LIMIT = 200 * 1024;   // dynamic shared memory the reduction kernels may ask for

// V = float4 vectors per token (D / 4).  GROUP = lanes that share one token.
template <int UNROLL>
__global__ void __launch_bounds__(ACT_THREADS, 8)
activity_reduce_kernel(const float4* __restrict__ z_cur, const float4* __restrict__ z_prev,
                       const int32_t* __restrict__ labels, const uint8_t* __restrict__ prev_active,
                       int N, int V, int R, int tokens_per_cta, double* __restrict__ acc_ss,
                       int32_t* __restrict__ acc_cnt, Control* ctl) {
    extern __shared__ double s_ss[];            // [R]
    int32_t* s_cnt = reinterpret_cast<int32_t*>(s_ss + R);
    const int b = blockIdx.y;
    const int t0 = blockIdx.x * tokens_per_cta;
    const int t1 = min(N, t0 + tokens_per_cta);
    for (int i = threadIdx.x; i < R; i += ACT_THREADS) { s_ss[i] = 0.0; s_cnt[i] = 0; }
    __syncthreads();
    if (t0 < N) {
        const size_t base = (size_t)b * N * V;
        const int32_t* lab_b = labels + (size_t)b * N;
        const uint8_t* pa_b = prev_active + (size_t)b * R;
        const long long n_vec = (long long)(t1 - t0) * V;
        // lanes sharing one token: the largest power of two dividing gcd(V, 32)
        int group = 1;
        while (group < 32 && (V % (group * 2)) == 0) group *= 2;
        const long long span = (long long)ACT_THREADS * UNROLL;
        // Each group leader keeps a running sum for the region it is currently in and only touches the
        // shared accumulators when the region changes: consecutive tokens mostly share their region, and
        // fp64 shared-memory atomics on one hot address would otherwise serialise the whole CTA.
        const bool leader = (threadIdx.x & (group - 1)) == 0;
        int cur_lab = -1, cur_cnt = 0;
        float cur_sum = 0.f;
        for (long long i0 = 0; i0 < n_vec; i0 += span) {
            float part[UNROLL];
            int lab[UNROLL];
            bool lead[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const long long i = i0 + (long long)u * ACT_THREADS + threadIdx.x;
                part[u] = 0.f;
                lab[u] = -1;
                lead[u] = false;
                if (i < n_vec) {
                    const int tok = t0 + (int)(i / V);
                    const int l = __ldg(lab_b + tok);
                    if (l < 0 || l > R) {
                        report(ctl, FD_ERR_STATE, tok);
                    } else if (l < R && __ldg(pa_b + l)) {
                        const size_t e = base + (size_t)t0 * V + (size_t)i;
                        const float4 a = __ldg(z_cur + e);
                        const float4 p = __ldg(z_prev + e);
                        const float dx = a.x - p.x, dy = a.y - p.y, dz = a.z - p.z, dw = a.w - p.w;
                        part[u] = dx * dx + dy * dy + dz * dz + dw * dw;
                        lab[u] = l;
                        lead[u] = (i % V) == 0;   // first vector of the token: counts the token once
                    }
                }
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                float v = part[u];
                // lanes [g*group, (g+1)*group) hold vectors of the same token
                for (int o = group >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lab[u] >= 0 && leader) {
                    if (lab[u] != cur_lab) {
                        if (cur_lab >= 0) {
                            atomicAdd(&s_ss[cur_lab], (double)cur_sum);
                            if (cur_cnt) atomicAdd(&s_cnt[cur_lab], cur_cnt);
                        }
                        cur_lab = lab[u];
                        cur_sum = 0.f;
                        cur_cnt = 0;
                    }
                    cur_sum += v;
                    cur_cnt += lead[u] ? 1 : 0;      // the first vector of a token sits on a group leader
                }
            }
        }
        if (cur_lab >= 0) {
            atomicAdd(&s_ss[cur_lab], (double)cur_sum);
            if (cur_cnt) atomicAdd(&s_cnt[cur_lab], cur_cnt);
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < R; i += ACT_THREADS) {
        if (s_cnt[i] != 0 || s_ss[i] != 0.0) {
            atomicAdd(&acc_ss[(size_t)b * R + i], s_ss[i]);
            atomicAdd(&acc_cnt[(size_t)b * R + i], s_cnt[i]);
        }
    }
}

// ---------------------------------------------------------------------------------------------
// The streaming form of kernel 1.  z is [B, N, D] contiguous, so a CTA's share of the B*N tokens is
// one byte range of z_cur and one of z_prev.  A producer warp brings both in with bulk copies,
// 8 KB per operand and ring stage, several stages ahead; eight consumer warps reduce a stage from
// shared memory.  The bytes in flight no longer depend on registers or occupancy, which is what a
// read-only stream needs to approach the HBM rate.  A chunk whose tokens all belong to frozen
// regions is not copied at all.
// ---------------------------------------------------------------------------------------------
constexpr int BULK_STAGES = 4;
constexpr int BULK_CHUNK_BYTES = 8192;                   // per operand and stage
constexpr int BULK_MAX_TOK = BULK_CHUNK_BYTES / 16;      // tokens of a chunk at the narrowest row (D = 4)
constexpr int BULK_CONSUMERS = 256;
constexpr int BULK_THREADS = BULK_CONSUMERS + 32;
constexpr int BULK_FIXED_SMEM = BULK_STAGES * 2 * BULK_CHUNK_BYTES + BULK_STAGES * BULK_MAX_TOK * 4 + 128;

__global__ void __launch_bounds__(BULK_THREADS)
activity_reduce_bulk_kernel(const char* __restrict__ z_cur, const char* __restrict__ z_prev,
                            const int32_t* __restrict__ labels, const uint8_t* __restrict__ prev_active,
                            int B, int N, int V, int R, int c_tok, long long tokens_per_cta,
                            double* __restrict__ acc_ss, int32_t* __restrict__ acc_cnt, Control* ctl) {
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char* ring = smem;                                          // [stage][operand][BULK_CHUNK_BYTES]
    int* s_lab = reinterpret_cast<int*>(smem + BULK_STAGES * 2 * BULK_CHUNK_BYTES);   // [stage][token]: region, or -1 = not read
    uint64_t* full = reinterpret_cast<uint64_t*>(s_lab + BULK_STAGES * BULK_MAX_TOK);
    uint64_t* empty = full + BULK_STAGES;
    int* s_skip = reinterpret_cast<int*>(empty + BULK_STAGES);           // [stage]: nothing was copied
    volatile int* abort_flag = s_skip + BULK_STAGES;
    double* s_ss = reinterpret_cast<double*>(smem + BULK_FIXED_SMEM);
    int32_t* s_cnt = reinterpret_cast<int32_t*>(s_ss + R);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row_bytes = V * 16;
    if (threadIdx.x == 0) {
        for (int s = 0; s < BULK_STAGES; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], BULK_CONSUMERS / 32); }
        *abort_flag = 0;
        ptx::fence_barrier_init();
    }
    for (int i = threadIdx.x; i < R; i += BULK_THREADS) { s_ss[i] = 0.0; s_cnt[i] = 0; }
    __syncthreads();
    const long long total = (long long)B * N;
    const long long lo = (long long)blockIdx.x * tokens_per_cta;
    const long long hi = lo + tokens_per_cta < total ? lo + tokens_per_cta : total;
    uint32_t it = 0;                                     // ring position, continues across requests
    bool ok = true;
    // lanes sharing one token: the largest power of two dividing gcd(V, 32)
    int group = 1;
    while (group < 32 && (V % (group * 2)) == 0) group *= 2;
    const bool leader = (lane & (group - 1)) == 0;
    const int q_step = 32 / V, r_step = 32 % V;          // how token index and vector index move when i grows by 32
    if (lo < hi) {
        for (int b = (int)(lo / N); b <= (int)((hi - 1) / N); ++b) {
            const long long s0 = lo > (long long)b * N ? lo : (long long)b * N;
            const long long s1 = hi < (long long)(b + 1) * N ? hi : (long long)(b + 1) * N;
            const int n_chunks = (int)((s1 - s0 + c_tok - 1) / c_tok);
            if (warp == BULK_CONSUMERS / 32) {
                // ------------------------------------------------------------ producer warp
                const uint8_t* pa_b = prev_active + (size_t)b * R;
                for (int k = 0; k < n_chunks && ok; ++k, ++it) {
                    const int st = it % BULK_STAGES;
                    const long long g0 = s0 + (long long)k * c_tok;
                    const int n_tok = (int)(s1 - g0 < c_tok ? s1 - g0 : c_tok);
                    if (!ptx::mbar_wait(&empty[st], ((it / BULK_STAGES) & 1) ^ 1, abort_flag)) { ok = false; break; }
                    // what the consumers need to know about the chunk's tokens: the region whose sum a token
                    // feeds, or -1 (background token, or a region whose change magnitude is frozen)
                    bool live = false;
                    for (int t = lane; t < n_tok; t += 32) {
                        int l = __ldg(labels + g0 + t);
                        if (l < 0 || l > R) {
                            report(ctl, FD_ERR_STATE, (int)((g0 + t) % N));
                            l = -1;
                        } else if (l == R || !__ldg(pa_b + l)) {
                            l = -1;
                        }
                        s_lab[st * BULK_MAX_TOK + t] = l;
                        live |= l >= 0;
                    }
                    live = __any_sync(0xffffffffu, live);
                    __syncwarp();                                        // every lane's labels are written before lane 0 signals
                    if (lane == 0) {
                        s_skip[st] = live ? 0 : 1;
                        if (live) {
                            const uint32_t bytes = (uint32_t)n_tok * row_bytes;
                            ptx::mbar_expect_tx(&full[st], 2 * bytes);
                            ptx::bulk_load(ring + (st * 2 + 0) * BULK_CHUNK_BYTES, z_cur + (size_t)g0 * row_bytes, bytes, &full[st]);
                            ptx::bulk_load(ring + (st * 2 + 1) * BULK_CHUNK_BYTES, z_prev + (size_t)g0 * row_bytes, bytes, &full[st]);
                        } else {
                            ptx::mbar_arrive(&full[st]);
                        }
                    }
                    __syncwarp();
                }
                if (!ok && lane == 0) report(ctl, FD_ERR_TIMEOUT, 1000 + (int)blockIdx.x);
            } else {
                // ------------------------------------------------------------ consumer warps
                // Every lane sums "its" vector column over consecutive tokens of one region; the lanes of a
                // token are only added up (and the shared accumulators touched) when the region changes.
                int cur_lab = -1, cur_cnt = 0;
                float cur_sum = 0.f;
                auto flush = [&](bool chg, int next_lab) {
                    float v = chg ? cur_sum : 0.f;
                    for (int o = group >> 1; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                    if (chg) {
                        if (leader && cur_lab >= 0) {
                            atomicAdd(&s_ss[cur_lab], (double)v);
                            if (cur_cnt) atomicAdd(&s_cnt[cur_lab], cur_cnt);
                        }
                        cur_lab = next_lab;
                        cur_sum = 0.f;
                        cur_cnt = 0;
                    }
                };
                for (int k = 0; k < n_chunks && ok; ++k, ++it) {
                    const int st = it % BULK_STAGES;
                    if (!ptx::mbar_wait(&full[st], (it / BULK_STAGES) & 1, abort_flag)) { ok = false; break; }
                    if (!s_skip[st]) {
                        const long long g0 = s0 + (long long)k * c_tok;
                        const int n_tok = (int)(s1 - g0 < c_tok ? s1 - g0 : c_tok);
                        // every warp takes a contiguous run of the chunk's tokens
                        const int tok_per_warp = (n_tok + BULK_CONSUMERS / 32 - 1) / (BULK_CONSUMERS / 32);
                        const int w0 = min(warp * tok_per_warp, n_tok);
                        const int w1 = min(w0 + tok_per_warp, n_tok);
                        const int n_vec = (w1 - w0) * V;
                        const float4* cur = reinterpret_cast<const float4*>(ring + (st * 2 + 0) * BULK_CHUNK_BYTES) + w0 * V;
                        const float4* prv = reinterpret_cast<const float4*>(ring + (st * 2 + 1) * BULK_CHUNK_BYTES) + w0 * V;
                        const int* lab = s_lab + st * BULK_MAX_TOK + w0;
                        int tok = lane / V, vi = lane - tok * V;         // token and vector index of element i = i0 + lane
                        for (int i0 = 0; i0 < n_vec; i0 += 32) {
                            const int i = i0 + lane;
                            const bool in = i < n_vec;
                            const int l = in ? lab[tok] : cur_lab;       // lanes past the end keep their state
                            if (__any_sync(0xffffffffu, l != cur_lab)) flush(l != cur_lab, l);
                            if (in && l >= 0) {
                                const float4 a = cur[i], p = prv[i];
                                const float dx = a.x - p.x, dy = a.y - p.y, dz = a.z - p.z, dw = a.w - p.w;
                                cur_sum += dx * dx + dy * dy + dz * dz + dw * dw;
                                cur_cnt += vi == 0 ? 1 : 0;              // first vector of the token: counts the token once
                            }
                            tok += q_step;
                            vi += r_step;
                            if (vi >= V) { vi -= V; ++tok; }
                        }
                    }
                    __syncwarp();
                    if (lane == 0) ptx::mbar_arrive(&empty[st]);
                }
                flush(true, -1);                                         // the request ends: nothing stays in registers
                if (!ok && lane == 0) report(ctl, FD_ERR_TIMEOUT, 1100 + (int)blockIdx.x);
            }
            // the request's sums leave the CTA before the next request's tokens are added
            __syncthreads();
            for (int i = threadIdx.x; i < R; i += BULK_THREADS) {
                if (s_cnt[i] != 0 || s_ss[i] != 0.0) {
                    atomicAdd(&acc_ss[(size_t)b * R + i], s_ss[i]);
                    atomicAdd(&acc_cnt[(size_t)b * R + i], s_cnt[i]);
                    s_ss[i] = 0.0;
                    s_cnt[i] = 0;
                }
            }
            __syncthreads();
        }
    }
}

// Scalar fallback when D is not a multiple of 4 or the rows are not 16-byte aligned.
__global__ void __launch_bounds__(ACT_THREADS)
activity_reduce_scalar_kernel(const float* __restrict__ z_cur, const float* __restrict__ z_prev,
                              const int32_t* __restrict__ labels, const uint8_t* __restrict__ prev_active,
                              int N, int D, int R, double* __restrict__ acc_ss,
                              int32_t* __restrict__ acc_cnt, Control* ctl) {
    const int b = blockIdx.y;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int tok = blockIdx.x * (ACT_THREADS / 32) + warp; tok < N; tok += gridDim.x * (ACT_THREADS / 32)) {
        const int l = labels[(size_t)b * N + tok];
        if (l < 0 || l > R) { if (lane == 0) report(ctl, FD_ERR_STATE, tok); continue; }
        if (l == R || !prev_active[(size_t)b * R + l]) continue;
        const size_t e = ((size_t)b * N + tok) * D;
        float v = 0.f;
        for (int c = lane; c < D; c += 32) { const float d = z_cur[e + c] - z_prev[e + c]; v += d * d; }
        v = warp_sum(v);
        if (lane == 0) {
            atomicAdd(&acc_ss[(size_t)b * R + l], (double)v);
            atomicAdd(&acc_cnt[(size_t)b * R + l], 1);
        }
    }
}

__global__ void __launch_bounds__(256)
gate_kernel(int R, int D, const float* __restrict__ eps, float eta, int K, double* __restrict__ acc_ss,
            int32_t* __restrict__ acc_cnt, float* __restrict__ delta_state, int32_t* __restrict__ skip_count,
            uint8_t* __restrict__ prev_active, float* __restrict__ score, float* __restrict__ weight,
            uint8_t* __restrict__ mask) {
    __shared__ double s_red[256];
    const int b = blockIdx.x;
    const size_t o = (size_t)b * R;
    double local = 0.0;
    for (int i = threadIdx.x; i < R; i += blockDim.x) {
        float d;
        if (prev_active[o + i]) {                       // ran last step: fresh change magnitude
            const int cnt = acc_cnt[o + i];
            d = cnt > 0 ? (float)sqrt(acc_ss[o + i] / ((double)cnt * (double)D)) : 0.f;
            delta_state[o + i] = d;
        } else {
            d = delta_state[o + i];                     // skipped: frozen at its last-active value
        }
        acc_ss[o + i] = 0.0;
        acc_cnt[o + i] = 0;
        score[o + i] = d;
        local += (double)d + (double)eta;
    }
    s_red[threadIdx.x] = local;
    __syncthreads();
    for (int s = blockDim.x >> 1; s > 0; s >>= 1) {
        if (threadIdx.x < s) s_red[threadIdx.x] += s_red[threadIdx.x + s];
        __syncthreads();
    }
    const double dn = s_red[0];
    const double e = (double)eps[b];
    for (int i = threadIdx.x; i < R; i += blockDim.x) {
        const double num = (double)score[o + i] + (double)eta;
        const bool gate_on = dn > 0.0 ? (num >= e * dn) : true;      // w_i >= eps
        weight[o + i] = dn > 0.0 ? (float)(num / dn) : 1.0f / (float)R;
        const int sk = skip_count[o + i];
        const bool on = gate_on || (sk >= K);                        // forced reactivation
        mask[o + i] = on ? 1 : 0;
        prev_active[o + i] = on ? 1 : 0;
        skip_count[o + i] = on ? 0 : sk + 1;
    }
}

// The same gate on the paper's own signal (Sec. 4.2): R_i = mass_i / |A_i|^2 for the patches executed at the step that
// produced `mass`; Delta_i = |R_i - Rbar_i| and Rbar_i <- R_i for those, frozen Delta_i for the skipped ones.
__global__ void __launch_bounds__(256)
attn_gate_kernel(int R, const double* __restrict__ mass, const int32_t* __restrict__ region_sizes, const float* __restrict__ eps,
                 float eta, int K, float* __restrict__ rbar, float* __restrict__ delta_state, int32_t* __restrict__ skip_count,
                 uint8_t* __restrict__ prev_active, float* __restrict__ importance, float* __restrict__ weight,
                 uint8_t* __restrict__ mask) {
    __shared__ double s_red[256];
    const int b = blockIdx.x;
    const size_t o = (size_t)b * R;
    double local = 0.0;
    for (int i = threadIdx.x; i < R; i += blockDim.x) {
        float d;
        if (prev_active[o + i]) {
            const double n = (double)region_sizes[o + i];
            const float r = n > 0.0 ? (float)(mass[o + i] / (n * n)) : 0.f;
            d = (float)fabs((double)r - (double)rbar[o + i]);
            delta_state[o + i] = d;
            rbar[o + i] = r;
        } else {
            d = delta_state[o + i];
        }
        importance[o + i] = rbar[o + i];
        local += (double)d + (double)eta;
    }
    s_red[threadIdx.x] = local;
    __syncthreads();
    for (int s = blockDim.x >> 1; s > 0; s >>= 1) {
        if (threadIdx.x < s) s_red[threadIdx.x] += s_red[threadIdx.x + s];
        __syncthreads();
    }
    const double dn = s_red[0];
    const double e = (double)eps[b];
    for (int i = threadIdx.x; i < R; i += blockDim.x) {
        const double num = (double)delta_state[o + i] + (double)eta;
        const bool gate_on = dn > 0.0 ? (num >= e * dn) : true;      // w_i >= eps
        weight[o + i] = dn > 0.0 ? (float)(num / dn) : 1.0f / (float)R;
        const int sk = skip_count[o + i];
        const bool on = gate_on || (sk >= K);                        // forced reactivation
        mask[o + i] = on ? 1 : 0;
        prev_active[o + i] = on ? 1 : 0;
        skip_count[o + i] = on ? 0 : sk + 1;
    }
}

}  // namespace

cudaError_t launch_attn_gate(const double* region_mass, const int32_t* region_sizes, int B, int R, const float* eps,
                             float eta, int K, float* rbar, float* delta, int32_t* skip_count, uint8_t* prev_active,
                             float* importance, float* weight, uint8_t* mask, cudaStream_t st, int* n_launch) {
    attn_gate_kernel<<<B, 256, 0, st>>>(R, region_mass, region_sizes, eps, eta, K, rbar, delta, skip_count, prev_active,
                                        importance, weight, mask);
    ++*n_launch;
    return cudaGetLastError();
}

namespace {

// Per-device set-up of the reduction kernels, done once: the dynamic shared-memory ceiling is a property
// of the function (not of a launch), so it is raised to the fixed upper bound here instead of to a
// call-dependent value on every call, and the SM count is looked up once.
constexpr int MAX_DEVICES = 64;
std::mutex g_setup_mu;
int g_sm_count[MAX_DEVICES];                // 0 = not set up yet

cudaError_t activity_setup(int* sms) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mu);
    if (!g_sm_count[dev]) {
        int n = 0;
        e = cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(activity_reduce_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ACT_SMEM_LIMIT);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(activity_reduce_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, ACT_SMEM_LIMIT);
        if (e != cudaSuccess) return e;
        g_sm_count[dev] = n > 0 ? n : 148;
    }
    *sms = g_sm_count[dev];
    return cudaSuccess;
}

}  // namespace

cudaError_t launch_activity(const float* z_cur, const float* z_prev, const int32_t* labels, int B, int N,
                            int D, int R, const float* eps, float* delta, int32_t* skip_count,
                            uint8_t* prev_active, float* score, float* weight, uint8_t* mask, float eta,
                            int K, double* acc_ss, int32_t* acc_cnt, Control* ctl, cudaStream_t st,
                            int* n_launch) {
    int sms = 148;
    cudaError_t es = activity_setup(&sms);
    if (es != cudaSuccess) return es;
    const bool vec = (D % 4 == 0) && ((reinterpret_cast<uintptr_t>(z_cur) | reinterpret_cast<uintptr_t>(z_prev)) % 16 == 0);
    const size_t acc_smem = (size_t)R * (sizeof(double) + sizeof(int32_t));
    const size_t bulk_smem = (size_t)BULK_FIXED_SMEM + acc_smem;
    if (vec && D * 4 <= BULK_CHUNK_BYTES && bulk_smem <= (size_t)ACT_SMEM_LIMIT) {
        const int V = D / 4;
        const int c_tok = BULK_CHUNK_BYTES / (D * 4);
        // three CTAs per SM fit (64 KB of ring each); every CTA gets one contiguous share of the B*N tokens, at
        // least four chunks so that the ring fills, in whole chunks
        const long long total = (long long)B * N;
        const long long max_ctas = (long long)sms * 3;
        long long per = (total + max_ctas - 1) / max_ctas;
        if (per < 4LL * c_tok) per = 4LL * c_tok;
        per = (per + c_tok - 1) / c_tok * c_tok;
        const int grid = (int)((total + per - 1) / per);
        activity_reduce_bulk_kernel<<<grid, BULK_THREADS, bulk_smem, st>>>(
            reinterpret_cast<const char*>(z_cur), reinterpret_cast<const char*>(z_prev), labels, prev_active, B, N, V,
            R, c_tok, per, acc_ss, acc_cnt, ctl);
    } else if (vec && acc_smem <= (size_t)ACT_SMEM_LIMIT) {
        const int V = D / 4;
        // At least 32 KB of each operand per CTA (enough work to amortise set-up and the flush); for large
        // batches fewer, longer chunks: about 16 CTAs per SM in total keep every SM streaming without a long tail.
        const int by_size = (int)(((long long)N * V + 2047) / 2048);
        const int by_sms = (sms * 16 + B - 1) / B;
        const int want = max(1, min(by_size, by_sms));
        const int tokens_per_cta = (N + want - 1) / want;
        const int chunks = (N + tokens_per_cta - 1) / tokens_per_cta;
        dim3 grid(chunks, B);
        activity_reduce_kernel<4><<<grid, ACT_THREADS, acc_smem, st>>>(
            reinterpret_cast<const float4*>(z_cur), reinterpret_cast<const float4*>(z_prev), labels,
            prev_active, N, V, R, tokens_per_cta, acc_ss, acc_cnt, ctl);
    } else {
        // any alignment, any channel count, any region count: one warp per token, sums added straight into the
        // global accumulators
        dim3 grid(min(1024, (N + 7) / 8), B);
        activity_reduce_scalar_kernel<<<grid, ACT_THREADS, 0, st>>>(z_cur, z_prev, labels, prev_active, N,
                                                                    D, R, acc_ss, acc_cnt, ctl);
    }
    ++*n_launch;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    gate_kernel<<<B, 256, 0, st>>>(R, D, eps, eta, K, acc_ss, acc_cnt, delta, skip_count, prev_active, score,
                                   weight, mask);
    ++*n_launch;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Gate without a context or a workspace: the accumulators live in a fixed device array.
// ---------------------------------------------------------------------------------------------
namespace {

// per-(request, region) accumulators (sum of squares fp64, token count i32) and one status block
constexpr size_t NOALLOC_BYTES = sizeof(Control) + 192 /*keeps the arrays 256-byte aligned*/ +
                                 (size_t)FD_NOALLOC_MAX_REGION_SLOTS * (sizeof(double) + sizeof(int32_t));
static __device__ __align__(256) unsigned char g_gate_scratch[NOALLOC_BYTES];

void* g_scratch_addr[MAX_DEVICES];          // device address of g_gate_scratch, per device
std::mutex g_scratch_mu;

}  // namespace

cudaError_t noalloc_gate(const float* z_cur, const float* z_prev, const int32_t* labels, int B, int N, int D,
                         int R, const float* eps, float eta, int K, float* delta, int32_t* skip_count,
                         uint8_t* prev_active, float* score, float* weight, uint8_t* mask, int32_t* status_out,
                         cudaStream_t st) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    unsigned char* base = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_scratch_mu);
        if (!g_scratch_addr[dev]) {
            // In host code the array's name is only a handle; the address the kernels need comes from
            // the runtime, looked up once per device while that device is current.
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_gate_scratch);
            if (e != cudaSuccess) return e;
            g_scratch_addr[dev] = p;
        }
        base = static_cast<unsigned char*>(g_scratch_addr[dev]);
    }
    Control* ctl = reinterpret_cast<Control*>(base);
    double* acc_ss = reinterpret_cast<double*>(base + 256);
    int32_t* acc_cnt = reinterpret_cast<int32_t*>(base + 256 + (size_t)FD_NOALLOC_MAX_REGION_SLOTS * sizeof(double));
    // the array keeps whatever the previous call left: everything read before written starts at zero
    e = cudaMemsetAsync(base, 0, 256 + (size_t)B * R * sizeof(double), st);
    if (e == cudaSuccess) e = cudaMemsetAsync(acc_cnt, 0, (size_t)B * R * sizeof(int32_t), st);
    if (e != cudaSuccess) return e;
    int nl = 0;
    e = launch_activity(z_cur, z_prev, labels, B, N, D, R, eps, delta, skip_count, prev_active, score, weight, mask,
                        eta, K, acc_ss, acc_cnt, ctl, st, &nl);
    if (e != cudaSuccess) return e;
    if (status_out) e = cudaMemcpyAsync(status_out, &ctl->status, sizeof(int32_t), cudaMemcpyDeviceToDevice, st);
    return e;
}

}  // namespace fd
