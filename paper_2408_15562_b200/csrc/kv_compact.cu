// Accepted-path KV compaction, the cache append of the accepted path, and the tree-row scatter used by the host entry.
//
// After verification the rejected tokens leave the sequence (paper, Section
// "Preliminaries": differing tokens and their descendants are discarded), so
// for every layer, K and V, sequence and kv head the rows of the accepted path
// move up to directly follow the prefix: row L + path[j] -> row L + j.
//
// path[] is strictly increasing with path[j] >= j, so a destination row j is
// never the source of a later move and moves can be applied in index order
// with no staging copy: one warp owns one (layer, K/V, sequence, head) slice,
// loads up to eight rows (16-byte chunks, two rows per warp instruction) before
// storing them, then goes on to the next eight.  Rows already in place are
// skipped.  Pure data movement: HBM-bound, no arithmetic.
#include "common.cuh"

namespace {

constexpr int kWarpsPerCta = 8;
constexpr int kRowBytes = FSPAD_HEAD_DIM * 2;        // 256
constexpr int kChunks = kRowBytes / 16;              // 16 uint4 per row
constexpr int kBatchIters = 4;                       // 4 iterations x 2 rows in flight per warp

__global__ void __launch_bounds__(kWarpsPerCta * 32)
kv_compact_kernel(uint4 *__restrict__ cache, const int *__restrict__ path, const int *__restrict__ n_acc,
                  const int *__restrict__ prefix_len, int n_layers, int B, int Hkv, int max_len,
                  int path_stride, int n_tree_max, int *__restrict__ new_len, int *__restrict__ status)
{
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long slice = (long long)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    const long long n_slices = (long long)n_layers * 2 * B * Hkv;
    if (slice >= n_slices) return;
    const int b = (int)((slice / Hkv) % B);
    int L = prefix_len[b], n = n_acc[b];
    const int *pth = path + (size_t)b * path_stride;
    bool bad = false;
    if (n < 0 || n > path_stride || n > n_tree_max) { bad = true; n = 0; }
    if (L < 0 || L + n > max_len) { bad = true; n = 0; }
    // the slices of layer 0 / K / head 0 (one per sequence) publish the new length
    if (new_len && lane == 0 && slice < (long long)B * Hkv && slice % Hkv == 0) new_len[b] = L + n;
    uint4 *base = cache + (size_t)slice * max_len * kChunks;
    const int chunk = lane & 15, half = lane >> 4;
    for (int j0 = 0; j0 < n; j0 += 2 * kBatchIters) {
        uint4 v[kBatchIters];
        int dst[kBatchIters];
#pragma unroll
        for (int u = 0; u < kBatchIters; ++u) {
            const int j = j0 + 2 * u + half;
            dst[u] = -1;
            if (j < n) {
                const int src = pth[j];
                if (src < j || src >= n_tree_max || L + src >= max_len || (j > 0 && src <= pth[j - 1])) {
                    bad = true;
                    continue;
                }
                if (src != j) {
                    v[u] = base[(size_t)(L + src) * kChunks + chunk];
                    dst[u] = j;
                }
            }
        }
        // the two half-warps own different rows and a destination of one may be a source of the
        // other: every load of the batch is ordered before any of its stores
        __syncwarp();
#pragma unroll
        for (int u = 0; u < kBatchIters; ++u)
            if (dst[u] >= 0) base[(size_t)(L + dst[u]) * kChunks + chunk] = v[u];
    }
    if (bad) fspad_report(status, FSPAD_ERR_RANGE);
}

// The same moves on a cache kept as a pool of 128-row blocks, [layers][2][n_blocks][Hkv][128][d]: cache row r
// of sequence b lives in block table[b * stride + r / 128] at offset r % 128.  One warp per (layer, K/V,
// sequence, head); blocks are looked up per row (a handful of rows per slice).
__global__ void __launch_bounds__(kWarpsPerCta * 32)
kv_compact_paged_kernel(uint4 *__restrict__ pool, const int *__restrict__ table, int table_stride, int n_blocks,
                        const int *__restrict__ path, const int *__restrict__ n_acc, const int *__restrict__ prefix_len,
                        int n_layers, int B, int Hkv, int path_stride, int n_tree_max, int *__restrict__ new_len,
                        int *__restrict__ status)
{
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long slice = (long long)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    const long long n_slices = (long long)n_layers * 2 * B * Hkv;
    if (slice >= n_slices) return;
    const int h = (int)(slice % Hkv);
    const int b = (int)((slice / Hkv) % B);
    const long long lk = slice / ((long long)Hkv * B);              // layer * 2 + (K or V)
    const int max_len = table_stride * 128;
    int L = prefix_len[b], n = n_acc[b];
    const int *pth = path + (size_t)b * path_stride;
    bool bad = false;
    if (n < 0 || n > path_stride || n > n_tree_max) { bad = true; n = 0; }
    if (L < 0 || L + n > max_len) { bad = true; n = 0; }
    if (new_len && lane == 0 && lk == 0 && h == 0) new_len[b] = L + n;
    // first 16-byte chunk of cache row r of this slice
    auto row_ptr = [&](int r) -> uint4 * {
        int blk = table[(size_t)b * table_stride + (r >> 7)];
        if (blk < 0 || blk >= n_blocks) { bad = true; blk = 0; }
        return pool + ((((size_t)lk * n_blocks + blk) * Hkv + h) * 128 + (r & 127)) * kChunks;
    };
    const int chunk = lane & 15, half = lane >> 4;
    for (int j0 = 0; j0 < n; j0 += 2 * kBatchIters) {
        uint4 v[kBatchIters];
        int dst[kBatchIters];
#pragma unroll
        for (int u = 0; u < kBatchIters; ++u) {
            const int j = j0 + 2 * u + half;
            dst[u] = -1;
            if (j < n) {
                const int src = pth[j];
                if (src < j || src >= n_tree_max || L + src >= max_len || (j > 0 && src <= pth[j - 1])) {
                    bad = true;
                    continue;
                }
                if (src != j) {
                    v[u] = row_ptr(L + src)[chunk];
                    dst[u] = j;
                }
            }
        }
        __syncwarp();      // every load of the batch before any of its stores (the half-warps own different rows)
#pragma unroll
        for (int u = 0; u < kBatchIters; ++u)
            if (dst[u] >= 0) row_ptr(L + dst[u])[chunk] = v[u];
    }
    if (bad) fspad_report(status, FSPAD_ERR_RANGE);
}

// Cache append of the accepted path: the tree's K/V rows of every layer are held outside the cache,
// [layers][2][B][Hkv][N][d], and only the accepted ones are written, directly behind the prefix:
// cache[..][L + j][:] = tree_kv[..][path[j]][:].  The N - n rejected rows never reach the cache, so neither
// the write of all N rows nor the later move of the accepted ones happens.  One warp per (layer, K/V,
// sequence, head) slice, eight rows in flight; source and destination are different arrays, so there
// is no ordering to keep.
__global__ void __launch_bounds__(kWarpsPerCta * 32)
kv_append_kernel(uint4 *__restrict__ cache, const uint4 *__restrict__ tree_kv, const int *__restrict__ path,
                 const int *__restrict__ n_acc, const int *__restrict__ prefix_len, int n_layers, int B, int Hkv,
                 int max_len, int N, int path_stride, int *__restrict__ new_len, int *__restrict__ status)
{
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long slice = (long long)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    const long long n_slices = (long long)n_layers * 2 * B * Hkv;
    if (slice >= n_slices) return;
    const int b = (int)((slice / Hkv) % B);
    int L = prefix_len[b], n = n_acc[b];
    const int *pth = path + (size_t)b * path_stride;
    bool bad = false;
    if (n < 0 || n > path_stride || n > N) { bad = true; n = 0; }
    if (L < 0 || L + n > max_len) { bad = true; n = 0; }
    if (new_len && lane == 0 && slice < (long long)B * Hkv && slice % Hkv == 0) new_len[b] = L + n;
    uint4 *dst_base = cache + ((size_t)slice * max_len + L) * kChunks;
    const uint4 *src_base = tree_kv + (size_t)slice * N * kChunks;
    const int chunk = lane & 15, half = lane >> 4;
    for (int j0 = 0; j0 < n; j0 += 2 * kBatchIters) {
        uint4 v[kBatchIters];
        int dst[kBatchIters];
#pragma unroll
        for (int u = 0; u < kBatchIters; ++u) {
            const int j = j0 + 2 * u + half;
            dst[u] = -1;
            if (j < n) {
                const int src = pth[j];
                if (src < 0 || src >= N) { bad = true; continue; }
                v[u] = __ldg(src_base + (size_t)src * kChunks + chunk);
                dst[u] = j;
            }
        }
#pragma unroll
        for (int u = 0; u < kBatchIters; ++u)
            if (dst[u] >= 0) dst_base[(size_t)dst[u] * kChunks + chunk] = v[u];
    }
    if (bad) fspad_report(status, FSPAD_ERR_RANGE);
}

// cache[layer 0][K|V][b][h][L_b + j][:] = tree_{k|v}[b][h][j][:]
__global__ void __launch_bounds__(256)
tree_scatter_kernel(uint4 *__restrict__ cache, const uint4 *__restrict__ tk, const uint4 *__restrict__ tv,
                    const int *__restrict__ prefix_len, int N, int B, int Hkv, int max_len,
                    int *__restrict__ status)
{
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const long long total = (long long)2 * B * Hkv * N * kChunks;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const int chunk = (int)(i % kChunks);
        long long r = i / kChunks;
        const int j = (int)(r % N); r /= N;
        const int h = (int)(r % Hkv); r /= Hkv;
        const int b = (int)(r % B);
        const int kv = (int)(r / B);
        const int L = prefix_len[b];
        if (L < 0 || L + N > max_len) { fspad_report(status, FSPAD_ERR_RANGE); continue; }
        const uint4 *src = (kv ? tv : tk) + (((size_t)b * Hkv + h) * N + j) * kChunks + chunk;
        cache[((((size_t)kv * B + b) * Hkv + h) * max_len + (L + j)) * kChunks + chunk] = *src;
    }
}

}  // namespace

cudaError_t fspad_launch_kv_compact(fspad_ctx *ctx, fspad_bf16 *cache, const int *path,
                                    const int *n_acc, const int *prefix_len, int B, int *new_len,
                                    cudaStream_t st, bool pdl)
{
    if (B == 0) return cudaSuccess;
    const fspad_config &c = ctx->cfg;
    const long long slices = (long long)c.n_layers * 2 * B * c.n_kv_heads;
    const unsigned grid = (unsigned)((slices + kWarpsPerCta - 1) / kWarpsPerCta);
    ctx->launches++;
    return fspad_launch_opt(pdl, kv_compact_kernel, dim3(grid), dim3(kWarpsPerCta * 32), 0, st, 0,
                        reinterpret_cast<uint4 *>(cache), path, n_acc, prefix_len, c.n_layers, B, c.n_kv_heads,
                        c.max_len, c.max_nodes, c.max_nodes, new_len, ctx->d_status);
}

cudaError_t fspad_launch_kv_append(fspad_ctx *ctx, fspad_bf16 *cache, const fspad_bf16 *tree_kv, const int *path,
                                   const int *n_acc, const int *prefix_len, int N, int B, int *new_len, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    const fspad_config &c = ctx->cfg;
    const long long slices = (long long)c.n_layers * 2 * B * c.n_kv_heads;
    const unsigned grid = (unsigned)((slices + kWarpsPerCta - 1) / kWarpsPerCta);
    ctx->launches++;
    return fspad_launch(kv_append_kernel, dim3(grid), dim3(kWarpsPerCta * 32), 0, st, 0, reinterpret_cast<uint4 *>(cache),
                        reinterpret_cast<const uint4 *>(tree_kv), path, n_acc, prefix_len, c.n_layers, B, c.n_kv_heads,
                        c.max_len, N, c.max_nodes, new_len, ctx->d_status);
}

cudaError_t fspad_launch_tree_scatter(fspad_ctx *ctx, fspad_bf16 *cache, const fspad_bf16 *tk,
                                      const fspad_bf16 *tv, const int *prefix_len, int N, int B,
                                      cudaStream_t st)
{
    if (B == 0 || N == 0) return cudaSuccess;
    const fspad_config &c = ctx->cfg;
    const long long total = (long long)2 * B * c.n_kv_heads * N * kChunks;
    unsigned grid = (unsigned)((total + 255) / 256);
    if (grid > (unsigned)ctx->sm_count * 8) grid = (unsigned)ctx->sm_count * 8;
    ctx->launches++;
    return fspad_launch(tree_scatter_kernel, dim3(grid), dim3(256), 0, st, 0, reinterpret_cast<uint4 *>(cache),
                        reinterpret_cast<const uint4 *>(tk), reinterpret_cast<const uint4 *>(tv), prefix_len, N, B,
                        c.n_kv_heads, c.max_len, ctx->d_status);
}

cudaError_t fspad_launch_kv_compact_paged(fspad_ctx *ctx, fspad_bf16 *pool, FspadPaged paged, const int *path,
                                          const int *n_acc, const int *prefix_len, int B, int *new_len, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    const fspad_config &c = ctx->cfg;
    const long long slices = (long long)c.n_layers * 2 * B * c.n_kv_heads;
    const unsigned grid = (unsigned)((slices + kWarpsPerCta - 1) / kWarpsPerCta);
    ctx->launches++;
    return fspad_launch(kv_compact_paged_kernel, dim3(grid), dim3(kWarpsPerCta * 32), 0, st, 0,
                        reinterpret_cast<uint4 *>(pool), paged.table, paged.stride, paged.n_blocks, path, n_acc, prefix_len,
                        c.n_layers, B, c.n_kv_heads, c.max_nodes, c.max_nodes, new_len, ctx->d_status);
}
