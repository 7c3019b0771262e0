// Compaction of the active regions' tokens into a ragged, ascending index list across requests
// (Algorithm 1: the PatchGate's active set selects what runs; Sec. 5: workers execute only their
// active patches).  Two small kernels: per-chunk counts, then an order-preserving write that uses
// warp ballots and a prefix over the chunk counts.  The second kernel also emits the per-request
// offsets, the active-row total and the attention work list, all on the device: the host never
// learns the count.
#include "common.cuh"

namespace fd {

namespace {

constexpr int CP_THREADS = 256;
constexpr int CP_WARPS = CP_THREADS / 32;
constexpr int CP_CHUNK = 2048;                 // tokens per CTA
constexpr int CP_PER_WARP = CP_CHUNK / CP_WARPS;

__device__ __forceinline__ bool token_flag(const uint8_t* mask_b, const int32_t* lab_b, int tok, int N,
                                           int R, Control* ctl) {
    if (tok >= N) return false;
    const int l = lab_b[tok];
    if (l < 0 || l > R) { if (ctl) report(ctl, FD_ERR_STATE, tok); return false; }
    return l == R || mask_b[l] != 0;
}

__global__ void __launch_bounds__(CP_THREADS)
compact_count_kernel(const uint8_t* __restrict__ mask, const int32_t* __restrict__ labels, int N, int R,
                     int32_t* __restrict__ block_counts, Control* ctl) {
    __shared__ int s_warp[CP_WARPS];
    const int b = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint8_t* mask_b = mask + (size_t)b * R;
    const int32_t* lab_b = labels + (size_t)b * N;
    const int w0 = blockIdx.x * CP_CHUNK + warp * CP_PER_WARP;
    int cnt = 0;
    for (int t = 0; t < CP_PER_WARP; t += 32)
        cnt += __popc(__ballot_sync(0xffffffffu, token_flag(mask_b, lab_b, w0 + t + lane, N, R, ctl)));
    if (lane == 0) s_warp[warp] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) {
        int s = 0;
        for (int w = 0; w < CP_WARPS; ++w) s += s_warp[w];
        block_counts[b * gridDim.x + blockIdx.x] = s;
    }
}

__global__ void __launch_bounds__(CP_THREADS)
compact_write_kernel(const uint8_t* __restrict__ mask, const int32_t* __restrict__ labels, int B, int N, int R,
                     const int32_t* __restrict__ block_counts, int32_t* __restrict__ active_idx,
                     int32_t* __restrict__ cu_active, QTile* __restrict__ tiles, int tile_rows, Control* ctl,
                     QTile* __restrict__ tiles2) {
    __shared__ int s_warp[CP_WARPS];
    __shared__ int s_red[CP_WARPS];
    __shared__ int s_red2[CP_WARPS];
    __shared__ int s_base;
    const int b = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int chunks = gridDim.x;
    const int me = b * chunks + blockIdx.x;
    // rows written by all chunks before this one
    int part = 0;
    for (int i = threadIdx.x; i < me; i += CP_THREADS) part += block_counts[i];
    part = (int)__reduce_add_sync(0xffffffffu, part);
    if (lane == 0) s_red[warp] = part;
    const uint8_t* mask_b = mask + (size_t)b * R;
    const int32_t* lab_b = labels + (size_t)b * N;
    const int w0 = blockIdx.x * CP_CHUNK + warp * CP_PER_WARP;
    unsigned bal[CP_PER_WARP / 32];
    int cnt = 0;
#pragma unroll
    for (int t = 0; t < CP_PER_WARP / 32; ++t) {
        bal[t] = __ballot_sync(0xffffffffu, token_flag(mask_b, lab_b, w0 + t * 32 + lane, N, R, nullptr));
        cnt += __popc(bal[t]);
    }
    if (lane == 0) s_warp[warp] = cnt;
    __syncthreads();
    if (threadIdx.x == 0) {
        int s = 0;
        for (int w = 0; w < CP_WARPS; ++w) s += s_red[w];
        s_base = s;
        if (blockIdx.x == 0) cu_active[b] = s;
        if (me == B * chunks - 1) {
            int mine = 0;
            for (int w = 0; w < CP_WARPS; ++w) mine += s_warp[w];
            cu_active[B] = s + mine;
            ctl->a_total = s + mine;
        }
    }
    __syncthreads();
    int pos = s_base;
    for (int w = 0; w < warp; ++w) pos += s_warp[w];
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int t = 0; t < CP_PER_WARP / 32; ++t) {
        if (bal[t] & (1u << lane)) active_idx[pos + __popc(bal[t] & lt)] = b * N + w0 + t * 32 + lane;
        pos += __popc(bal[t]);
    }
    // attention work list: chunk 0 of each request lists that request's query tiles
    if (blockIdx.x == 0) {
        // rows of this request and tiles of the requests before it
        int rows_b = 0;
        for (int i = threadIdx.x; i < chunks; i += CP_THREADS) rows_b += block_counts[b * chunks + i];
        int tiles_before = 0, tiles2_before = 0;
        for (int bb = warp; bb < b; bb += CP_WARPS) {          // one warp per earlier request
            int r = 0;
            for (int i = lane; i < chunks; i += 32) r += block_counts[bb * chunks + i];
            r = (int)__reduce_add_sync(0xffffffffu, r);
            tiles_before += (r + tile_rows - 1) / tile_rows;
            tiles2_before += (r + 2 * tile_rows - 1) / (2 * tile_rows);
        }
        __syncthreads();
        rows_b = (int)__reduce_add_sync(0xffffffffu, rows_b);
        if (lane == 0) { s_warp[warp] = rows_b; s_red[warp] = tiles_before; s_red2[warp] = tiles2_before; }
        __syncthreads();
        int rows = 0, tb = 0, tb2 = 0;
        for (int w = 0; w < CP_WARPS; ++w) { rows += s_warp[w]; tb += s_red[w]; tb2 += s_red2[w]; }
        const int nt = (rows + tile_rows - 1) / tile_rows;
        for (int t = threadIdx.x; t < nt; t += CP_THREADS) {
            QTile q;
            q.b = b;
            q.row0 = s_base + t * tile_rows;
            q.rows = min(tile_rows, rows - t * tile_rows);
            q.pad = 0;
            tiles[tb + t] = q;
        }
        if (b == B - 1 && threadIdx.x == 0) ctl->n_qtiles = tb + nt;
        if (tiles2) {
            // the same rows as double-height tiles: one per CTA pair, each CTA of the pair takes tile_rows of them
            const int nt2 = (rows + 2 * tile_rows - 1) / (2 * tile_rows);
            for (int t = threadIdx.x; t < nt2; t += CP_THREADS) {
                QTile q;
                q.b = b;
                q.row0 = s_base + t * 2 * tile_rows;
                q.rows = min(2 * tile_rows, rows - t * 2 * tile_rows);
                q.pad = 0;
                tiles2[tb2 + t] = q;
            }
            if (b == B - 1 && threadIdx.x == 0) ctl->n_qtiles2 = tb2 + nt2;
        }
    }
}

// Dual stream: which 128-row and which 256-row tiles of the compact rows hold at least one row of the second stream
// (label R).  One CTA: a thread per 128-row tile flags it, a ballot-based prefix keeps the lists ascending.
__global__ void __launch_bounds__(CP_THREADS)
text_tiles_kernel(const int32_t* __restrict__ active_idx, const int32_t* __restrict__ labels, int R,
                  int32_t* __restrict__ list128, int32_t* __restrict__ list256, Control* ctl) {
    __shared__ int s_cnt[CP_WARPS];
    __shared__ int s_base[2];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int a_total = ctl->a_total;
    const int n128 = (a_total + 127) / 128;
    if (threadIdx.x == 0) { s_base[0] = 0; s_base[1] = 0; }
    __syncthreads();
    for (int gran = 0; gran < 2; ++gran) {
        const int rows = gran ? 256 : 128;
        const int n_tiles = gran ? (a_total + 255) / 256 : n128;
        int32_t* list = gran ? list256 : list128;
        for (int t0 = 0; t0 < n_tiles; t0 += CP_THREADS) {
            const int t = t0 + threadIdx.x;
            bool has = false;
            if (t < n_tiles) {
                const int r1 = min(a_total, (t + 1) * rows);
                for (int r = t * rows; r < r1 && !has; ++r) has = labels[active_idx[r]] == R;
            }
            const unsigned bal = __ballot_sync(0xffffffffu, has);
            if (lane == 0) s_cnt[warp] = __popc(bal);
            __syncthreads();
            int pos = s_base[gran];
            for (int w = 0; w < warp; ++w) pos += s_cnt[w];
            if (has) list[pos + __popc(bal & ((1u << lane) - 1u))] = t;
            __syncthreads();
            if (threadIdx.x == 0) {
                int tot = 0;
                for (int w = 0; w < CP_WARPS; ++w) tot += s_cnt[w];
                s_base[gran] += tot;
            }
            __syncthreads();
        }
    }
    if (threadIdx.x == 0) { ctl->n_text_tiles[0] = s_base[0]; ctl->n_text_tiles[1] = s_base[1]; }
}

}  // namespace

cudaError_t launch_text_tiles(const int32_t* active_idx, const int32_t* labels, int R, int rows_cap, int32_t* list128,
                              int32_t* list256, Control* ctl, cudaStream_t st, int* n_launch) {
    (void)rows_cap;
    text_tiles_kernel<<<1, CP_THREADS, 0, st>>>(active_idx, labels, R, list128, list256, ctl);
    ++*n_launch;
    return cudaGetLastError();
}

cudaError_t launch_compact(const uint8_t* mask, const int32_t* labels, int B, int N, int R,
                           int32_t* active_idx, int32_t* cu_active, int32_t* block_counts, QTile* tiles,
                           int tile_rows, Control* ctl, cudaStream_t st, int* n_launch, QTile* tiles2) {
    const int chunks = (N + CP_CHUNK - 1) / CP_CHUNK;
    dim3 grid(chunks, B);
    compact_count_kernel<<<grid, CP_THREADS, 0, st>>>(mask, labels, N, R, block_counts, ctl);
    ++*n_launch;
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    compact_write_kernel<<<grid, CP_THREADS, 0, st>>>(mask, labels, B, N, R, block_counts, active_idx,
                                                      cu_active, tiles, tile_rows, ctl, tiles2);
    ++*n_launch;
    return cudaGetLastError();
}

}  // namespace fd
