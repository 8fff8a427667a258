// Dynamic token tree, one draft step (paper, Section "Preliminaries", last
// paragraph: the output of each draft step is truncated to its top-k and every
// token carries the joint probability of its path).
//
// Three small kernels per call:
//   1. draft_topk_partial_kernel - grid (pieces of 4096 tokens, rows): the top-k of the
//      piece from one pass: a lower bound of the k-th largest value from the half-warp
//      maxima, the few tokens that reach it listed in shared memory and ranked by
//      counting; the one HBM pass over the rows.
//   2. draft_topk_row_kernel - one CTA per row: the pieces' lists (at most 1024
//      entries) through the sorting network; the first k become candidates
//      base + f k + r with the frontier node as parent and the joint
//      log-probability frontier_logp + value, one single-precision addition.
//   3. draft_frontier_kernel - one CTA per sequence: the F k new joint values
//      through the network; the first `width` are the next frontier.
// Comparisons and one addition only, so every decision is the oracle's bit for bit.
#include "common.cuh"
#include "sort_network.cuh"

namespace {

constexpr int kThreads = kSortThreads;                 // 256
constexpr int kPerThread = 16;                         // tokens per thread in the partial kernel
constexpr int kPiece = kThreads * kPerThread;          // 4096 tokens per CTA

// The top-k of one piece of one row.  The k-th largest of the 16 half-warp maxima is a lower bound of
// the piece's k-th largest value, because k tokens at least that large exist; every token whose value
// reaches the bound goes to a shared list (a few dozen entries on ordinary data, the whole piece at
// worst) as a 64-bit key (order-preserving image of the value, complemented token index: larger key
// = larger value, or equal value and lower token), and the list's members are ranked by counting.
// One pass over the data: per token one maximum and one comparison.
__global__ void __launch_bounds__(kThreads)
draft_topk_partial_kernel(const float *__restrict__ logprobs, int V, int k, int pieces, uint2 *__restrict__ part)
{
    __shared__ unsigned long long s_list[kPiece];               // tokens whose value reaches the bound
    __shared__ float s_hmax[kThreads / 16];
    __shared__ float s_bound;
    __shared__ int s_cnt;
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const int tid = threadIdx.x, lane = tid & 31;
    const int piece = blockIdx.x, row = blockIdx.y;
    const float *x = logprobs + (size_t)row * V;
    const int e0 = piece * kPiece;
    const bool vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(logprobs) & 15) == 0);
    if (tid == 0) s_cnt = 0;
    float val[kPerThread];                                       // positions past the row's end hold -inf
    float bv = -INFINITY;
#pragma unroll
    for (int i = 0; i < kPerThread / 4; ++i) {
        const int e = e0 + 4 * (i * kThreads + tid);
        if (vec && e + 3 < V) {
            const float4 t4 = __ldg(reinterpret_cast<const float4 *>(x + e));
            val[4 * i] = t4.x; val[4 * i + 1] = t4.y; val[4 * i + 2] = t4.z; val[4 * i + 3] = t4.w;
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) val[4 * i + c] = (e + c < V) ? x[e + c] : -INFINITY;
        }
#pragma unroll
        for (int c = 0; c < 4; ++c) bv = fmaxf(bv, val[4 * i + c]);
    }
    // maxima of the 16 half-warps (a half-warp without any token reports -inf, which can only lower
    // the bound and so lengthen the list, never lose a token)
#pragma unroll
    for (int off = 8; off > 0; off >>= 1) bv = fmaxf(bv, __shfl_xor_sync(0xffffffffu, bv, off));
    if ((lane & 15) == 0) s_hmax[tid >> 4] = bv;
    __syncthreads();
    if (tid < kThreads / 16) {
        const float me = s_hmax[tid];
        int rank = 0;
#pragma unroll
        for (int o = 0; o < kThreads / 16; ++o) {
            const float ot = s_hmax[o];
            rank += (ot > me || (ot == me && o < tid)) ? 1 : 0;
        }
        if (rank == k - 1) s_bound = me;                         // k <= 16: exactly one thread
    }
    __syncthreads();
    const float bound = s_bound;
#pragma unroll
    for (int u = 0; u < kPerThread; ++u) {
        if (val[u] >= bound) {
            const int tok = e0 + 4 * ((u >> 2) * kThreads + tid) + (u & 3);
            if (tok < V) s_list[atomicAdd(&s_cnt, 1)] = fspad_sort_key(val[u], (uint32_t)tok);
        }
    }
    __syncthreads();
    const int n = s_cnt;
    uint2 *out = part + ((size_t)row * pieces + piece) * k;
    for (int i = tid; i < n; i += kThreads) {
        const unsigned long long me = s_list[i];
        int rank = 0;
        for (int o = 0; o < n; ++o) rank += (s_list[o] > me) ? 1 : 0;
        if (rank < k) out[rank] = make_uint2(__float_as_uint(fspad_key_value(me)), fspad_key_index(me));
    }
    for (int r = n + tid; r < k; r += kThreads) out[r] = make_uint2(__float_as_uint(-INFINITY), 0x7fffffffu);   // empty slots
}

// one row: partial lists -> top-k -> candidates
__global__ void __launch_bounds__(kThreads)
draft_topk_row_kernel(const uint2 *__restrict__ part, const float *__restrict__ frontier_logp,
                      const int *__restrict__ frontier_cand, int F, int k, int pieces, int base, int cap,
                      int *__restrict__ cand_parent, int *__restrict__ cand_token, float *__restrict__ cand_logp)
{
    __shared__ unsigned long long s_key[kSortEntries];
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const int tid = threadIdx.x, row = blockIdx.x;
    const int b = row / F, f = row % F;
    const int n = pieces * k;                                    // <= 1024 (checked on the host)
    const uint2 *in = part + (size_t)row * n;
    unsigned long long v[kSortPerThread];
#pragma unroll
    for (int r = 0; r < kSortPerThread; ++r) {
        const int i = kSortPerThread * tid + r;
        unsigned long long key = 0ull;
        if (i < n) {
            const uint2 e = in[i];
            if (e.y != 0x7fffffffu) key = fspad_sort_key(__uint_as_float(e.x), e.y);   // empty slots stay padding
        }
        v[r] = key;
    }
    fspad_bitonic_sort_desc(v, s_key, tid);
#pragma unroll
    for (int r = 0; r < kSortPerThread; ++r) {
        const int i = kSortPerThread * tid + r;
        if (i < k && v[r] != 0ull) {
            const size_t c = (size_t)b * cap + base + f * k + i;
            cand_parent[c] = frontier_cand[row];
            cand_token[c] = (int)fspad_key_index(v[r]);
            cand_logp[c] = __fadd_rn(frontier_logp[row], fspad_key_value(v[r]));   // one fp32 addition
        }
    }
}

// one sequence: F k new joint values -> next frontier
__global__ void __launch_bounds__(kThreads)
draft_frontier_kernel(const float *__restrict__ cand_logp, int n_new, int width, int base, int cap,
                      int *__restrict__ next_cand, float *__restrict__ next_logp)
{
    __shared__ unsigned long long s_key[kSortEntries];
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const int tid = threadIdx.x, b = blockIdx.x;
    const float *cl = cand_logp + (size_t)b * cap + base;
    unsigned long long v[kSortPerThread];
#pragma unroll
    for (int r = 0; r < kSortPerThread; ++r) {
        const int i = kSortPerThread * tid + r;
        v[r] = (i < n_new) ? fspad_sort_key(cl[i], (uint32_t)i) : 0ull;
    }
    fspad_bitonic_sort_desc(v, s_key, tid);
#pragma unroll
    for (int r = 0; r < kSortPerThread; ++r) {
        const int i = kSortPerThread * tid + r;
        if (i < width) {
            const int c = (int)fspad_key_index(v[r]);
            next_cand[(size_t)b * width + i] = base + c;
            next_logp[(size_t)b * width + i] = cl[c];
        }
    }
}

}  // namespace

int fspad_draft_expand_pieces(int V) { return (V + kPiece - 1) / kPiece; }

cudaError_t fspad_launch_draft_expand(fspad_ctx *ctx, const float *logprobs, const float *frontier_logp,
                                      const int *frontier_cand, int F, int k, int width, int base, int cap, int B,
                                      int *cand_parent, int *cand_token, float *cand_logp, int *next_cand,
                                      float *next_logp, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    const int V = ctx->cfg.vocab, pieces = fspad_draft_expand_pieces(V), rows = B * F;
    uint2 *part = reinterpret_cast<uint2 *>(ctx->dx_part);
    ctx->launches += 3;
    cudaError_t e = fspad_launch(draft_topk_partial_kernel, dim3(pieces, rows), dim3(kThreads), 0, st, 0, logprobs, V,
                                 k, pieces, part);
    if (e != cudaSuccess) return e;
    e = fspad_launch(draft_topk_row_kernel, dim3(rows), dim3(kThreads), 0, st, 0, (const uint2 *)part, frontier_logp,
                     frontier_cand, F, k, pieces, base, cap, cand_parent, cand_token, cand_logp);
    if (e != cudaSuccess) return e;
    return fspad_launch(draft_frontier_kernel, dim3(B), dim3(kThreads), 0, st, 0, (const float *)cand_logp, F * k,
                        width, base, cap, next_cand, next_logp);
}
