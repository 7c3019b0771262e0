// Patch Partitioner (paper Sec. 4.1; Appendix A.3 Eq. otsu and the hierarchical-extension remark).
//
// One CTA per request (runs once per request, off the per-step path; plain ALU / latency bound):
//   1. saliency S_j = mean over the salient columns of the attention map (fp64 accumulation in
//      column order), min-max normalised and quantised to 16 bits with individually rounded fp32
//      operations, so every later decision is exact integer arithmetic;
//   2. the tokens are sorted by (code, token index) with a bitonic sort of the packed 32-bit key
//      (code << 16 | index); every node of the recursion is then a contiguous range of that order
//      and prefix sums of the codes give class sums in O(1);
//   3. nodes are taken from an explicit stack: all threads scan the node's candidate cuts, the
//      between-class variance (n_c S_f - n_f S_c)^2 / (n_f n_c) is compared by 128-bit
//      cross-multiplication (ties: lowest threshold), the region budget is split by
//      r_f = argmin_r |r n - R n_f| (ties: smaller r), and a cut is admissible only if both sides
//      can hold their regions within the size bounds;
//   4. a node without an admissible cut is chopped in token order into equal chunks;
//   5. regions are renumbered by their smallest token index.
#include "common.cuh"

namespace fd {

namespace {

constexpr int PT_THREADS = 1024;
constexpr int PT_MAX_R = 1024;

struct Node { int s, e, r; };

struct Best {
    unsigned long long num_hi, num_lo;   // 128-bit numerator
    unsigned int den;
    int p, r_f;
};

__device__ __forceinline__ unsigned __int128 num128(const Best& b) {
    return ((unsigned __int128)b.num_hi << 64) | b.num_lo;
}
// true if a is a strictly better cut than b (larger variance; ties -> lower position)
__device__ __forceinline__ bool better(const Best& a, const Best& b) {
    if (a.p < 0) return false;
    if (b.p < 0) return true;
    const unsigned __int128 l = num128(a) * b.den, r = num128(b) * a.den;
    if (l != r) return l > r;
    return a.p < b.p;
}

__device__ __forceinline__ int allocate(long long n_f, long long n_c, int R) {
    const long long n = n_f + n_c;
    const long long lo = ((long long)R * n_f) / n;
    int best_r = 0;
    long long best_d = -1;
    for (int t = 0; t < 2; ++t) {
        long long r = lo + t;
        r = r < 1 ? 1 : (r > R - 1 ? R - 1 : r);
        long long d = r * n - (long long)R * n_f;
        d = d < 0 ? -d : d;
        if (best_d < 0 || d < best_d) { best_d = d; best_r = (int)r; }
    }
    return best_r;
}

// exclusive scan of vals[0..n) in place, all threads of the CTA; returns nothing, total in *total
__device__ void cta_exclusive_scan(unsigned int* vals, int n, unsigned int* s_part, unsigned int* total) {
    const int per = (n + PT_THREADS - 1) / PT_THREADS;
    const int lo = min(n, (int)threadIdx.x * per), hi = min(n, lo + per);
    unsigned int sum = 0;
    for (int i = lo; i < hi; ++i) sum += vals[i];
    s_part[threadIdx.x] = sum;
    __syncthreads();
    // Hillis-Steele inclusive scan over the 1024 partial sums
    for (int off = 1; off < PT_THREADS; off <<= 1) {
        unsigned int v = threadIdx.x >= off ? s_part[threadIdx.x - off] : 0u;
        __syncthreads();
        s_part[threadIdx.x] += v;
        __syncthreads();
    }
    unsigned int run = threadIdx.x == 0 ? 0u : s_part[threadIdx.x - 1];
    if (total && threadIdx.x == PT_THREADS - 1) *total = s_part[PT_THREADS - 1];
    for (int i = lo; i < hi; ++i) { const unsigned int v = vals[i]; vals[i] = run; run += v; }
    __syncthreads();
}

__global__ void __launch_bounds__(PT_THREADS, 1)
partition_kernel(const float* __restrict__ attn_map, int N, int T, const int32_t* __restrict__ salient_cols,
                 int T_s, int R, int m_min, int m_max, int32_t* __restrict__ labels_out,
                 int32_t* __restrict__ sizes_out, unsigned int* __restrict__ scratch, int n_pad,
                 size_t scratch_stride, Control* ctl) {
    __shared__ float s_f[PT_THREADS];
    __shared__ unsigned int s_u[PT_THREADS];
    __shared__ Best s_best[PT_THREADS / 32];
    __shared__ Node s_stack[PT_MAX_R];
    __shared__ int s_leaf_min[PT_MAX_R];
    __shared__ int s_leaf_rank[PT_MAX_R];
    __shared__ int s_sp, s_leaves;
    __shared__ Node s_cur;
    __shared__ unsigned int s_total;

    const int b = blockIdx.x, tid = threadIdx.x;
    const float* amap = attn_map + (size_t)b * N * T;
    int32_t* labels = labels_out + (size_t)b * N;
    unsigned int* keys = scratch + (size_t)b * scratch_stride;     // [n_pad]
    unsigned int* pre = keys + n_pad;                               // [N + 1]
    unsigned int* aux = pre + (N + 1);                              // [N]

    // 1. saliency, min / max
    float lo = INFINITY, hi = -INFINITY;
    for (int j = tid; j < N; j += PT_THREADS) {
        double acc = 0.0;
        if (salient_cols) {
            for (int t = 0; t < T_s; ++t) {
                const int c = salient_cols[t];
                if (c < 0 || c >= T) { report(ctl, FD_ERR_STATE, c); continue; }
                acc += (double)amap[(size_t)j * T + c];
            }
        } else {
            for (int t = 0; t < T; ++t) acc += (double)amap[(size_t)j * T + t];
        }
        const float s = (float)(acc / (double)T_s);
        aux[j] = __float_as_uint(s);
        lo = fminf(lo, s);
        hi = fmaxf(hi, s);
    }
    s_f[tid] = lo;
    __syncthreads();
    for (int o = PT_THREADS / 2; o > 0; o >>= 1) { if (tid < o) s_f[tid] = fminf(s_f[tid], s_f[tid + o]); __syncthreads(); }
    lo = s_f[0];
    __syncthreads();
    s_f[tid] = hi;
    __syncthreads();
    for (int o = PT_THREADS / 2; o > 0; o >>= 1) { if (tid < o) s_f[tid] = fmaxf(s_f[tid], s_f[tid + o]); __syncthreads(); }
    hi = s_f[0];
    __syncthreads();

    // 2. 16-bit codes, packed keys, bitonic sort
    const float span = __fsub_rn(hi, lo);
    for (int j = tid; j < n_pad; j += PT_THREADS) {
        unsigned int key = 0xFFFFFFFFu;
        if (j < N) {
            unsigned int q = 0;
            if (hi != lo) {
                float t = __fsub_rn(__uint_as_float(aux[j]), lo);
                t = __fdiv_rn(t, span);
                t = __fmul_rn(t, 65535.0f);
                t = __fadd_rn(t, 0.5f);
                q = (unsigned int)floorf(t);
                q = q > 65535u ? 65535u : q;
            }
            key = (q << 16) | (unsigned int)j;
        }
        keys[j] = key;
    }
    __syncthreads();
    for (int k = 2; k <= n_pad; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            for (int i = tid; i < n_pad; i += PT_THREADS) {
                const int x = i ^ j;
                if (x > i) {
                    const unsigned int a = keys[i], c = keys[x];
                    const bool up = (i & k) == 0;
                    if ((a > c) == up) { keys[i] = c; keys[x] = a; }
                }
            }
            __syncthreads();
        }
    }
    // 3. exclusive prefix sums of the codes in sorted order: pre[i] = sum of codes before position i
    for (int i = tid; i < N; i += PT_THREADS) pre[i] = keys[i] >> 16;
    __syncthreads();
    cta_exclusive_scan(pre, N, s_u, &s_total);
    if (tid == 0) {
        pre[N] = s_total;
        s_stack[0] = Node{0, N, R};
        s_sp = 1;
        s_leaves = 0;
    }
    __syncthreads();

    // 4. recursion with an explicit stack
    while (true) {
        if (tid == 0) {
            if (s_sp > 0) s_cur = s_stack[--s_sp]; else s_cur = Node{0, 0, 0};
        }
        __syncthreads();
        const Node nd = s_cur;
        if (nd.r == 0) break;
        const int n = nd.e - nd.s;
        if (nd.r == 1) {
            const int leaf = s_leaves;
            for (int i = nd.s + tid; i < nd.e; i += PT_THREADS) labels[keys[i] & 0xFFFFu] = leaf;
            __syncthreads();
            if (tid == 0) s_leaves = leaf + 1;
            __syncthreads();
            continue;
        }
        // best admissible cut of this node
        Best mine;
        mine.p = -1; mine.num_hi = mine.num_lo = 0; mine.den = 1; mine.r_f = 0;
        const unsigned long long base = pre[nd.s], tot = (unsigned long long)pre[nd.e] - base;
        for (int p = nd.s + 1 + tid; p < nd.e; p += PT_THREADS) {
            if ((keys[p - 1] >> 16) == (keys[p] >> 16)) continue;      // a threshold cannot separate equal codes
            const long long n_c = p - nd.s, n_f = nd.e - p;
            const int r_f = allocate(n_f, n_c, nd.r), r_c = nd.r - r_f;
            if (!((long long)m_min * r_f <= n_f && n_f <= (long long)m_max * r_f &&
                  (long long)m_min * r_c <= n_c && n_c <= (long long)m_max * r_c))
                continue;
            const unsigned long long s_c = (unsigned long long)pre[p] - base, s_ff = tot - s_c;
            const long long diff = (long long)(n_c * (long long)s_ff) - (long long)(n_f * (long long)s_c);
            const unsigned long long ad = (unsigned long long)(diff < 0 ? -diff : diff);
            const unsigned __int128 num = (unsigned __int128)ad * ad;
            Best cand;
            cand.num_hi = (unsigned long long)(num >> 64);
            cand.num_lo = (unsigned long long)num;
            cand.den = (unsigned int)(n_f * n_c);
            cand.p = p;
            cand.r_f = r_f;
            if (better(cand, mine)) mine = cand;
        }
        // warp-level reduction with shuffles, then the 32 warp winners in shared memory
        for (int o = 16; o > 0; o >>= 1) {
            Best other;
            other.num_hi = __shfl_down_sync(0xffffffffu, mine.num_hi, o);
            other.num_lo = __shfl_down_sync(0xffffffffu, mine.num_lo, o);
            other.den = __shfl_down_sync(0xffffffffu, mine.den, o);
            other.p = __shfl_down_sync(0xffffffffu, mine.p, o);
            other.r_f = __shfl_down_sync(0xffffffffu, mine.r_f, o);
            if (better(other, mine)) mine = other;
        }
        if ((tid & 31) == 0) s_best[tid >> 5] = mine;
        __syncthreads();
        if (tid < 32) {
            Best m2 = s_best[tid];
            for (int o = 16; o > 0; o >>= 1) {
                Best other;
                other.num_hi = __shfl_down_sync(0xffffffffu, m2.num_hi, o);
                other.num_lo = __shfl_down_sync(0xffffffffu, m2.num_lo, o);
                other.den = __shfl_down_sync(0xffffffffu, m2.den, o);
                other.p = __shfl_down_sync(0xffffffffu, m2.p, o);
                other.r_f = __shfl_down_sync(0xffffffffu, m2.r_f, o);
                if (better(other, m2)) m2 = other;
            }
            if (tid == 0) s_best[0] = m2;
        }
        __syncthreads();
        const Best win = s_best[0];
        __syncthreads();
        if (win.p >= 0) {
            if (tid == 0) {
                s_stack[s_sp++] = Node{nd.s, win.p, nd.r - win.r_f};       // context: codes below the threshold
                s_stack[s_sp++] = Node{win.p, nd.e, win.r_f};              // focus
            }
            __syncthreads();
            continue;
        }
        // fallback: the node's tokens in ascending token order, nd.r chunks whose sizes differ by at most one
        for (int j = tid; j < N; j += PT_THREADS) aux[j] = 0u;
        __syncthreads();
        for (int i = nd.s + tid; i < nd.e; i += PT_THREADS) aux[keys[i] & 0xFFFFu] = 1u;
        __syncthreads();
        // rank of every member among the members (exclusive scan of the flags); flags are recovered
        // from the scan afterwards (rank[j+1] - rank[j])
        cta_exclusive_scan(aux, N, s_u, &s_total);
        const int leaf0 = s_leaves;
        const int q_sz = n / nd.r, extra = n % nd.r;
        for (int j = tid; j < N; j += PT_THREADS) {
            const unsigned int rk = aux[j];
            const unsigned int nxt = (j + 1 < N) ? aux[j + 1] : s_total;
            if (nxt != rk) {                                               // token j belongs to the node
                const int big = extra * (q_sz + 1);
                const int chunk = (int)rk < big ? (int)rk / (q_sz + 1) : extra + ((int)rk - big) / max(q_sz, 1);
                labels[j] = leaf0 + chunk;
            }
        }
        __syncthreads();
        if (tid == 0) s_leaves = leaf0 + nd.r;
        __syncthreads();
    }

    // 5. canonical numbering by smallest token index, region sizes
    const int n_leaves = s_leaves;                     // equals R
    for (int i = tid; i < PT_MAX_R; i += PT_THREADS) { s_leaf_min[i] = N; s_leaf_rank[i] = 0; }
    __syncthreads();
    for (int j = tid; j < N; j += PT_THREADS) atomicMin(&s_leaf_min[labels[j]], j);
    __syncthreads();
    for (int i = tid; i < n_leaves; i += PT_THREADS) {
        int rk = 0;
        const int mi = s_leaf_min[i];
        for (int k = 0; k < n_leaves; ++k) {
            const int mk = s_leaf_min[k];
            rk += (mk < mi || (mk == mi && k < i)) ? 1 : 0;
        }
        s_leaf_rank[i] = rk;
    }
    if (sizes_out) for (int i = tid; i < R; i += PT_THREADS) sizes_out[(size_t)b * R + i] = 0;
    __syncthreads();
    for (int j = tid; j < N; j += PT_THREADS) {
        const int lab = s_leaf_rank[labels[j]];
        labels[j] = lab;
        if (sizes_out) atomicAdd(&sizes_out[(size_t)b * R + lab], 1);
    }
}

int pad_pow2(int n) { int p = 2; while (p < n) p <<= 1; return p; }
size_t stride_words(int N) { return (size_t)pad_pow2(N) + (size_t)(N + 1) + (size_t)N + 64; }

}  // namespace

size_t partition_scratch_bytes(int max_batch, int max_tokens, int /*max_regions*/) {
    const int n = max_tokens < 65536 ? max_tokens : 65535;
    return (size_t)max_batch * stride_words(n) * sizeof(unsigned int);
}

cudaError_t launch_partition(const float* attn_map, int B, int N, int T, const int32_t* salient_cols, int T_s,
                             int R, int m_min, int m_max, int32_t* labels, int32_t* sizes, void* scratch,
                             Control* ctl, cudaStream_t st, int* n_launch) {
    if (R > PT_MAX_R) return cudaErrorInvalidValue;
    partition_kernel<<<B, PT_THREADS, 0, st>>>(attn_map, N, T, salient_cols, T_s, R, m_min, m_max, labels, sizes,
                                              static_cast<unsigned int*>(scratch), pad_pow2(N), stride_words(N), ctl);
    ++*n_launch;
    return cudaGetLastError();
}

}  // namespace fd
