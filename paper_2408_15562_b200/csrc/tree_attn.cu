// Tree-masked verify attention (paper, Section "Preliminaries": the target
// takes the flattened token tree as input and the attention mask built from
// the tree introduces the dependencies between its tokens).
//
// Split-KV flash-decode.  All query rows that share a kv head (tree node x
// GQA group member) form one M x 128 operand, so every K/V tile fetched from
// HBM is used by all of them.  A CTA owns (sequence, kv head, 16*NWARPS query
// rows, one contiguous range of 64-key tiles): K/V tiles are staged through a
// double-buffered, XOR-swizzled shared-memory ring with 16-byte asynchronous
// copies, S = Q K^T and O += P V run on the tensor cores (bf16 inputs, fp32
// accumulate), softmax is the online form kept in registers with quad
// shuffles.  The ancestor mask is a 64-bit word per node held in shared
// memory and is applied only on tiles that reach past the cached prefix.
// Partial (O, max, sum) per split go to scratch and a second kernel merges
// them by log-sum-exp and writes bf16.
#include "common.cuh"

namespace {

constexpr int D = FSPAD_HEAD_DIM;      // 128
constexpr int BN = 64;                 // keys per tile
constexpr int ROWB = D * 2;            // bytes per row
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

__device__ __forceinline__ uint32_t smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
// byte offset of 16-byte chunk `chunk` of row `row` in a swizzled [rows][128] bf16 tile
__device__ __forceinline__ uint32_t swz(int row, int chunk)
{
    return (uint32_t)(row * ROWB + ((chunk ^ (row & 7)) << 4));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid)
{
    const int sz = valid ? 16 : 0;   // 0: the 16 destination bytes are zero-filled, src is not read
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;\n" ::"n"(N));
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];\n"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};\n"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

template <int NWARPS>
__global__ void __launch_bounds__(NWARPS * 32)
tree_attn_splitkv_kernel(const AttnArgs a)
{
    constexpr int BM = NWARPS * 16;
    constexpr int NT = NWARPS * 32;
    extern __shared__ __align__(128) unsigned char smem[];
    unsigned char *sQ = smem;                        // BM rows
    unsigned char *sK = sQ + BM * ROWB;              // 2 x BN rows
    unsigned char *sV = sK + 2 * BN * ROWB;          // 2 x BN rows
    unsigned long long *s_anc = reinterpret_cast<unsigned long long *>(sV + 2 * BN * ROWB);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.x;
    const int g = blockIdx.y / a.mtiles, mt = blockIdx.y % a.mtiles;
    const int b = blockIdx.z;
    const int N = a.N, G = a.G, M = a.M;

    int L = a.prefix_len[b];
    if (L < 0 || L + N > a.max_len) {
        if (tid == 0) fspad_report(a.status, FSPAD_ERR_RANGE);
        L = max(0, min(L, a.max_len - N));
    }
    const int Ltot = L + N;
    const int n_tiles = (Ltot + BN - 1) / BN;
    const int per = (n_tiles + a.n_splits - 1) / a.n_splits;
    const int t0 = split * per, t1 = min(n_tiles, t0 + per);

    // ancestor-or-self bit masks of the tree
    if (tid < N) {
        const int *par = a.parent + (size_t)b * N;
        unsigned long long mask = 0ull;
        int cur = tid;
        bool bad = false;
        for (int step = 0; step <= N && cur >= 0; ++step) {
            mask |= 1ull << cur;
            const int p = par[cur];
            if (cur == 0) { bad |= (p != -1); break; }
            if (p < 0 || p >= cur) { bad = true; break; }
            cur = p;
        }
        if (bad) fspad_report(a.status, FSPAD_ERR_BAD_TREE);
        s_anc[tid] = mask;
    }

    const fspad_bf16 *kcb = a.kc + ((size_t)b * a.Hkv + g) * (size_t)a.max_len * D;
    const fspad_bf16 *vcb = a.vc + ((size_t)b * a.Hkv + g) * (size_t)a.max_len * D;
    const fspad_bf16 *tkb = a.tk ? a.tk + ((size_t)b * a.Hkv + g) * (size_t)N * D : kcb + (size_t)L * D;
    const fspad_bf16 *tvb = a.tv ? a.tv + ((size_t)b * a.Hkv + g) * (size_t)N * D : vcb + (size_t)L * D;

    const size_t prow = ((size_t)b * a.Hkv + g) * a.n_splits + split;   // partial block index
    const int r_lo = warp * 16 + (lane >> 2);        // this thread's two rows inside the CTA tile
    const int gr0 = mt * BM + r_lo, gr1 = gr0 + 8;   // rows inside the kv head's M rows

    if (t0 >= t1) {
        // nothing to do for this split: publish an empty partial
        if ((lane & 3) == 0) {
            if (gr0 < M) { float *ml = a.part_ml + (prow * M + gr0) * 2; ml[0] = -INFINITY; ml[1] = 0.f; }
            if (gr1 < M) { float *ml = a.part_ml + (prow * M + gr1) * 2; ml[0] = -INFINITY; ml[1] = 0.f; }
        }
        return;
    }

    // ---- stage Q (once) and the first K/V tile ----
    for (int i = tid; i < BM * 16; i += NT) {
        const int r = i >> 4, c = i & 15;
        const int gr = mt * BM + r;
        const bool ok = gr < M;
        const int node = ok ? gr / G : 0, hh = ok ? gr % G : 0;
        const fspad_bf16 *src = a.q + (((size_t)b * N + node) * a.Hq + g * G + hh) * D + c * 8;
        cp_async16(smem_u32(sQ + swz(r, c)), src, ok);
    }
    auto load_tile = [&](int t, int buf) {
        unsigned char *dK = sK + buf * BN * ROWB, *dV = sV + buf * BN * ROWB;
        for (int i = tid; i < BN * 16; i += NT) {
            const int r = i >> 4, c = i & 15;
            const int key = t * BN + r;
            const bool ok = key < Ltot;
            const fspad_bf16 *ks = kcb, *vs = vcb;
            if (ok) {
                if (key < L) { ks = kcb + (size_t)key * D + c * 8; vs = vcb + (size_t)key * D + c * 8; }
                else { ks = tkb + (size_t)(key - L) * D + c * 8; vs = tvb + (size_t)(key - L) * D + c * 8; }
            }
            cp_async16(smem_u32(dK + swz(r, c)), ks, ok);
            cp_async16(smem_u32(dV + swz(r, c)), vs, ok);
        }
    };
    load_tile(t0, 0);
    cp_async_commit();

    uint32_t qf[8][4];
    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    const int node0 = (gr0 < M) ? gr0 / G : 0, node1 = (gr1 < M) ? gr1 / G : 0;

    for (int t = t0; t < t1; ++t) {
        const int buf = (t - t0) & 1;
        if (t + 1 < t1) {
            load_tile(t + 1, buf ^ 1);
            cp_async_commit();
            cp_async_wait<1>();
        } else {
            cp_async_wait<0>();
        }
        __syncthreads();
        if (t == t0) {
#pragma unroll
            for (int kk = 0; kk < 8; ++kk)
                ldsm_x4(smem_u32(sQ + swz(warp * 16 + (lane & 15), kk * 2 + (lane >> 4))), qf[kk][0], qf[kk][1],
                        qf[kk][2], qf[kk][3]);
        }
        const unsigned char *bK = sK + buf * BN * ROWB, *bV = sV + buf * BN * ROWB;

        // ---- S = Q K^T (16 x 64 per warp) ----
        float s[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
#pragma unroll
        for (int kk = 0; kk < 8; ++kk) {
#pragma unroll
            for (int np = 0; np < 4; ++np) {
                uint32_t r0, r1, r2, r3;
                const int key = np * 16 + (lane & 7) + ((lane >> 4) << 3);
                const int chunk = kk * 2 + ((lane >> 3) & 1);
                ldsm_x4(smem_u32(bK + swz(key, chunk)), r0, r1, r2, r3);
                mma_bf16(s[2 * np], qf[kk], r0, r1);
                mma_bf16(s[2 * np + 1], qf[kk], r2, r3);
            }
        }

        // ---- mask (only tiles that reach past the cached prefix) ----
        if ((t + 1) * BN > L) {
            const unsigned long long a0 = s_anc[node0], a1 = s_anc[node1];
#pragma unroll
            for (int nt = 0; nt < 8; ++nt) {
#pragma unroll
                for (int e = 0; e < 2; ++e) {
                    const int key = t * BN + nt * 8 + 2 * (lane & 3) + e;
                    bool ok0 = true, ok1 = true;
                    if (key >= L) {
                        const int j = key - L;
                        ok0 = (key < Ltot) && ((a0 >> j) & 1ull);
                        ok1 = (key < Ltot) && ((a1 >> j) & 1ull);
                    }
                    if (!ok0) s[nt][e] = -INFINITY;
                    if (!ok1) s[nt][2 + e] = -INFINITY;
                }
            }
        }

        // ---- online softmax (base-2 domain) ----
        float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            mx0 = fmaxf(mx0, fmaxf(s[nt][0], s[nt][1]));
            mx1 = fmaxf(mx1, fmaxf(s[nt][2], s[nt][3]));
        }
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
        const float mn0 = fmaxf(m0, mx0 * a.scale_log2), mn1 = fmaxf(m1, mx1 * a.scale_log2);
        const float ms0 = (mn0 == -INFINITY) ? 0.f : mn0, ms1 = (mn1 == -INFINITY) ? 0.f : mn1;
        const float al0 = exp2f(m0 - ms0), al1 = exp2f(m1 - ms1);
        m0 = mn0; m1 = mn1;
        // P is rounded to bf16 for the tensor-core product; the row sums are taken over the
        // rounded values so that the weights actually applied to V sum to the normaliser
        float rs0 = 0.f, rs1 = 0.f;
        uint32_t pk[8][2];
#pragma unroll
        for (int nt = 0; nt < 8; ++nt) {
            pk[nt][0] = pack_bf16(exp2f(fmaf(s[nt][0], a.scale_log2, -ms0)), exp2f(fmaf(s[nt][1], a.scale_log2, -ms0)));
            pk[nt][1] = pack_bf16(exp2f(fmaf(s[nt][2], a.scale_log2, -ms1)), exp2f(fmaf(s[nt][3], a.scale_log2, -ms1)));
            const float2 f0 = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162 *>(&pk[nt][0]));
            const float2 f1 = __bfloat1622float2(*reinterpret_cast<__nv_bfloat162 *>(&pk[nt][1]));
            rs0 += f0.x + f0.y;
            rs1 += f1.x + f1.y;
        }
        l0 = l0 * al0 + rs0;
        l1 = l1 * al1 + rs1;
#pragma unroll
        for (int i = 0; i < 16; ++i) { o[i][0] *= al0; o[i][1] *= al0; o[i][2] *= al1; o[i][3] *= al1; }

        // ---- O += P V ----
#pragma unroll
        for (int kt = 0; kt < 4; ++kt) {
            uint32_t pa[4];
            pa[0] = pk[2 * kt][0];
            pa[1] = pk[2 * kt][1];
            pa[2] = pk[2 * kt + 1][0];
            pa[3] = pk[2 * kt + 1][1];
#pragma unroll
            for (int dp = 0; dp < 8; ++dp) {
                uint32_t r0, r1, r2, r3;
                const int key = kt * 16 + (lane & 7) + (((lane >> 3) & 1) << 3);
                const int chunk = dp * 2 + (lane >> 4);
                ldsm_x4_t(smem_u32(bV + swz(key, chunk)), r0, r1, r2, r3);
                mma_bf16(o[2 * dp], pa, r0, r1);
                mma_bf16(o[2 * dp + 1], pa, r2, r3);
            }
        }
        __syncthreads();   // the next iteration's prefetch overwrites this buffer's sibling
    }

    // ---- publish the partial ----
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
    l1 += __shfl_xor_sync(0xffffffffu, l1, 2);
    const int col = 2 * (lane & 3);
    if (gr0 < M) {
        float *po = a.part_o + (prow * M + gr0) * D;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) *reinterpret_cast<float2 *>(po + nt * 8 + col) = make_float2(o[nt][0], o[nt][1]);
        if ((lane & 3) == 0) { float *ml = a.part_ml + (prow * M + gr0) * 2; ml[0] = m0; ml[1] = l0; }
    }
    if (gr1 < M) {
        float *po = a.part_o + (prow * M + gr1) * D;
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) *reinterpret_cast<float2 *>(po + nt * 8 + col) = make_float2(o[nt][2], o[nt][3]);
        if ((lane & 3) == 0) { float *ml = a.part_ml + (prow * M + gr1) * 2; ml[0] = m1; ml[1] = l1; }
    }
}

// Merge the split partials of one output row by log-sum-exp; one warp per row.
__global__ void __launch_bounds__(128)
tree_attn_combine_kernel(const AttnArgs a, int B)
{
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
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int s0 = 0; s0 < ns; s0 += 4) {
        float4 v[4];
        float w[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int sidx = s0 + u;
            const float wa = __shfl_sync(0xffffffffu, w0, sidx & 31), wb = __shfl_sync(0xffffffffu, w1, sidx & 31);
            w[u] = (sidx < ns) ? ((sidx < 32) ? wa : wb) : 0.f;
            v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (w[u] != 0.f)
                v[u] = __ldcg(reinterpret_cast<const float4 *>(a.part_o + ((pbase + sidx) * a.M + gr) * D + lane * 4));
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            acc.x += w[u] * v[u].x; acc.y += w[u] * v[u].y; acc.z += w[u] * v[u].z; acc.w += w[u] * v[u].w;
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

template <int NWARPS>
constexpr int attn_smem_bytes()
{
    return NWARPS * 16 * ROWB + 4 * BN * ROWB + FSPAD_MAX_NODES * 8;
}

inline int attn_bm(int M) { return M > 64 ? 128 : 64; }

}  // namespace

int fspad_attn_splits(const fspad_ctx *ctx, int N, int B)
{
    const int G = ctx->cfg.n_q_heads / ctx->cfg.n_kv_heads;
    const int M = N * G, BM = attn_bm(M);
    const int mtiles = (M + BM - 1) / BM;
    const long long base = (long long)B * ctx->cfg.n_kv_heads * mtiles;
    long long s = ctx->sm_count / base;           // one CTA per SM, never a partial second wave
    const int max_tiles = (ctx->cfg.max_len + BN - 1) / BN;
    if (s > max_tiles) s = max_tiles;
    if (s > 64) s = 64;
    if (s < 1) s = 1;
    return (int)s;
}

cudaError_t fspad_launch_tree_attn(fspad_ctx *ctx, const fspad_bf16 *q, const fspad_bf16 *kc,
                                   const fspad_bf16 *vc, const fspad_bf16 *tk, const fspad_bf16 *tv,
                                   const int *parent, const int *prefix_len, int N, int B,
                                   fspad_bf16 *out, cudaStream_t st)
{
    if (B == 0 || N == 0) return cudaSuccess;
    const fspad_config &c = ctx->cfg;
    AttnArgs a;
    a.q = q; a.kc = kc; a.vc = vc; a.tk = tk; a.tv = tv; a.parent = parent; a.prefix_len = prefix_len;
    a.N = N; a.Hq = c.n_q_heads; a.Hkv = c.n_kv_heads; a.G = c.n_q_heads / c.n_kv_heads;
    a.M = N * a.G; a.max_len = c.max_len;
    a.n_splits = fspad_attn_umma_splits(ctx, N, B);
    a.mtiles = (a.M + 127) / 128;
    a.scale_log2 = ctx->scale * kLog2e;
    a.part_o = ctx->part_o; a.part_ml = ctx->part_ml; a.out = out; a.status = ctx->d_status;
    cudaError_t e = fspad_launch_attn_umma_split(ctx, q, kc, vc, tk, tv, parent, prefix_len, N, B, a.n_splits,
                                                 a.scale_log2, st);
    if (e != cudaSuccess) return e;
    const long long rows = (long long)B * c.n_kv_heads * a.M;
    tree_attn_combine_kernel<<<(unsigned)((rows + 3) / 4), 128, 0, st>>>(a, B);
    ctx->launches++;
    return cudaGetLastError();
}
