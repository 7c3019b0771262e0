// Patch Gate on the latent change (paper Sec. 4.2; Appendix A.1 Eq. delta-i, Eq. gate-weight,
// Eq. forced-reactivation).
//
// Kernel 1 streams z_cur / z_prev once with 128-bit loads and accumulates, per region, the sum of
// squared differences (fp32 inside a token, fp64 across tokens) and the token count.  Tokens of
// regions whose change magnitude is frozen (skipped at the previous step) are not read at all.
// Kernel 2 (one CTA per request) turns the sums into delta, weights, mask and the next state, and
// clears the accumulators for the next call.
#include "common.cuh"

namespace fd {

namespace {

constexpr int ACT_THREADS = 256;

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

}  // namespace

cudaError_t launch_activity(const float* z_cur, const float* z_prev, const int32_t* labels, int B, int N,
                            int D, int R, const float* eps, float* delta, int32_t* skip_count,
                            uint8_t* prev_active, float* score, float* weight, uint8_t* mask, float eta,
                            int K, double* acc_ss, int32_t* acc_cnt, Control* ctl, cudaStream_t st,
                            int* n_launch) {
    const bool vec = (D % 4 == 0) && ((reinterpret_cast<uintptr_t>(z_cur) | reinterpret_cast<uintptr_t>(z_prev)) % 16 == 0);
    if (vec) {
        const int V = D / 4;
        // At least 32 KB of each operand per CTA (enough work to amortise set-up and the flush); for large
        // batches fewer, longer chunks: about 16 CTAs per SM in total keep every SM streaming without a long tail.
        const int by_size = (int)(((long long)N * V + 2047) / 2048);
        const int by_sms = (148 * 16 + B - 1) / B;
        const int want = max(1, min(by_size, by_sms));
        const int tokens_per_cta = (N + want - 1) / want;
        const int chunks = (N + tokens_per_cta - 1) / tokens_per_cta;
        dim3 grid(chunks, B);
        const size_t smem = (size_t)R * (sizeof(double) + sizeof(int32_t));
        activity_reduce_kernel<4><<<grid, ACT_THREADS, smem, st>>>(
            reinterpret_cast<const float4*>(z_cur), reinterpret_cast<const float4*>(z_prev), labels,
            prev_active, N, V, R, tokens_per_cta, acc_ss, acc_cnt, ctl);
    } else {
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

constexpr int MAX_DEVICES = 64;
void* g_scratch_addr[MAX_DEVICES];          // device address of g_gate_scratch, per device

}  // namespace

cudaError_t noalloc_gate(const float* z_cur, const float* z_prev, const int32_t* labels, int B, int N, int D,
                         int R, const float* eps, float eta, int K, float* delta, int32_t* skip_count,
                         uint8_t* prev_active, float* score, float* weight, uint8_t* mask, int32_t* status_out,
                         cudaStream_t st) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= MAX_DEVICES) return cudaErrorInvalidDevice;
    if (!g_scratch_addr[dev]) {
        // In host code the array's name is only a handle; the address the kernels need comes from
        // the runtime, looked up once per device while that device is current.
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_gate_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = p;
    }
    unsigned char* base = static_cast<unsigned char*>(g_scratch_addr[dev]);
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
