// Tree-masked verify attention: host-side launch and the split-KV merge.
// (paper, Section "Preliminaries": the target takes the flattened token tree as
// input and the attention mask built from the tree introduces the dependencies
// between its tokens).  The split kernel itself (tcgen05 tensor cores, tensor
// memory) lives in tree_attn_umma.cu; it leaves one partial (unnormalised O row,
// running maximum, sum) per key range, which the kernel below merges by
// log-sum-exp and writes as bf16.
#include "common.cuh"

namespace {

constexpr int D = FSPAD_HEAD_DIM;      // 128
constexpr float kLog2e = 1.4426950408889634f;

struct AttnArgs {
    const fspad_bf16 *q, *kc, *vc, *tk, *tv;
    const int *parent, *prefix_len;
    int N, Hq, Hkv, G, M, max_len, n_splits, mtiles;
    float scale_log2;
    float *part_o, *part_ml;
    fspad_bf16 *out;
    int *status;
};

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// Merge the split partials of one output row by log-sum-exp; one warp per row.  kBatch = how many
// ranges' rows a lane requests at once (few ranges: a small batch keeps the kernel light; many:
// a large one saves dependent round trips through L2).
template <int kBatch>
__global__ void __launch_bounds__(128)
tree_attn_combine_kernel(const AttnArgs a, int B)
{
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);   // over [B][Hkv][M]
    const long long total = (long long)B * a.Hkv * a.M;
    if (row >= total) return;
    const int gr = (int)(row % a.M);
    const int g = (int)((row / a.M) % a.Hkv);
    const int b = (int)(row / ((long long)a.M * a.Hkv));
    const size_t pbase = ((size_t)b * a.Hkv + g) * a.n_splits;
    // all (max, sum) pairs of the row are fetched at once, two splits per lane (n_splits <= 64)
    const int ns = a.n_splits;
    float m0 = -INFINITY, l0 = 0.f, m1 = -INFINITY, l1 = 0.f;
    if (lane < ns) {
        const float2 t = __ldcg(reinterpret_cast<const float2 *>(a.part_ml + ((pbase + lane) * a.M + gr) * 2));
        m0 = t.x; l0 = t.y;
    }
    if (lane + 32 < ns) {
        const float2 t = __ldcg(reinterpret_cast<const float2 *>(a.part_ml + ((pbase + lane + 32) * a.M + gr) * 2));
        m1 = t.x; l1 = t.y;
    }
    float mmax = fmaxf(m0, m1);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) mmax = fmaxf(mmax, __shfl_xor_sync(0xffffffffu, mmax, off));
    const float w0 = (m0 == -INFINITY) ? 0.f : exp2f(m0 - mmax);
    const float w1 = (m1 == -INFINITY) ? 0.f : exp2f(m1 - mmax);
    float denom = w0 * l0 + w1 * l1;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) denom += __shfl_xor_sync(0xffffffffu, denom, off);
    // The partial rows are requested before the weights are known (one round trip through L2 for up
    // to kBatch ranges instead of one per dependent step); a range that saw no key left its row
    // unwritten, so what was loaded for a zero weight is discarded, not multiplied.
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < ns; s0 += kBatch) {
        float4 v[kBatch];
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int sidx = s0 + u;
            v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (sidx < ns)
                v[u] = __ldcg(reinterpret_cast<const float4 *>(a.part_o + ((pbase + sidx) * a.M + gr) * D + lane * 4));
        }
#pragma unroll
        for (int u = 0; u < kBatch; ++u) {
            const int sidx = s0 + u;
            const float wa = __shfl_sync(0xffffffffu, w0, sidx & 31), wb = __shfl_sync(0xffffffffu, w1, sidx & 31);
            const float w = (sidx < ns) ? ((sidx < 32) ? wa : wb) : 0.f;
            if (w != 0.f) { acc.x += w * v[u].x; acc.y += w * v[u].y; acc.z += w * v[u].z; acc.w += w * v[u].w; }
        }
    }
    const float inv = denom > 0.f ? 1.f / denom : 0.f;
    const int node = gr / a.G, hh = gr % a.G;
    fspad_bf16 *dst = a.out + (((size_t)b * a.N + node) * a.Hq + g * a.G + hh) * D + lane * 4;
    uint2 pk;
    pk.x = pack_bf16(acc.x * inv, acc.y * inv);
    pk.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2 *>(dst) = pk;
}

}  // namespace

cudaError_t fspad_launch_tree_attn(fspad_ctx *ctx, const fspad_bf16 *q, const fspad_bf16 *kc,
                                   const fspad_bf16 *vc, const fspad_bf16 *tk, const fspad_bf16 *tv,
                                   const int *parent, const int *prefix_len, int N, int B,
                                   fspad_bf16 *out, cudaStream_t st, int sms, FspadPaged paged, bool merge_pdl)
{
    if (B == 0 || N == 0) return cudaSuccess;
    const fspad_config &c = ctx->cfg;
    AttnArgs a;
    a.q = q; a.kc = kc; a.vc = vc; a.tk = tk; a.tv = tv; a.parent = parent; a.prefix_len = prefix_len;
    a.N = N; a.Hq = c.n_q_heads; a.Hkv = c.n_kv_heads; a.G = c.n_q_heads / c.n_kv_heads;
    a.M = N * a.G; a.max_len = paged.table ? paged.stride * 128 : c.max_len;
    a.n_splits = fspad_attn_umma_splits(ctx, N, B, sms);
    a.mtiles = (a.M + 127) / 128;
    a.scale_log2 = ctx->scale * kLog2e;
    a.part_o = ctx->part_o; a.part_ml = ctx->part_ml; a.out = out; a.status = ctx->d_status;
    cudaError_t e = fspad_launch_attn_umma_split(ctx, q, kc, vc, tk, tv, parent, prefix_len, N, B, a.n_splits,
                                                 a.scale_log2, st, paged);
    if (e != cudaSuccess) return e;
    const long long rows = (long long)B * c.n_kv_heads * a.M;
    ctx->launches++;
    const dim3 grid((unsigned)((rows + 3) / 4));
    if (a.n_splits <= 4) return fspad_launch_opt(merge_pdl, tree_attn_combine_kernel<4>, grid, dim3(128), 0, st, 0, a, B);
    return fspad_launch_opt(merge_pdl, tree_attn_combine_kernel<12>, grid, dim3(128), 0, st, 0, a, B);
}
