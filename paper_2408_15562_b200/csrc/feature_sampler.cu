// Feature Sampler forward (paper, Section "Feature Sampling"): the Up projector maps the feature f
// and the Gate projector the token embedding e to intermediate size, the embedding's image is
// activated by SiLU and multiplied element by element with the feature's image, the Down projector
// maps the product back to hidden size, and the residual connection adds f:
//     eta = Wdown (silu(Wgate e) * (Wup f)) + f
// The draft model runs this on a handful of rows per step (the frontier of the draft tree), so the
// three products are bound by streaming their matrices once (3 * 2 * H * I bytes).  One tcgen05
// kernel serves all of them: a persistent CTA per SM takes work items (problem, tile of 256 output
// columns, range of the inner dimension), streams the matrix slab and the rows through a TMA ring
// of 128-byte-swizzled [128][64] / [256][64] bf16 stages into 128 x 256 x 16 tensor-core instructions with two
// accumulators in tensor memory, and writes fp32 partial sums; the inner dimension is split so that
// the items fill the SMs evenly.  Two small kernels add the partial sums: one applies SiLU and the
// product (bf16 out, the Down projector's operand), one adds the residual (bf16 out).
#include <cuda.h>

#include "common.cuh"
#include "umma_common.cuh"

namespace fsm {

using namespace umma;

constexpr int BM = 128, BN = 256, BKE = 64;
constexpr int STAGE_A = BM * 128;       // bytes of one [128][64] bf16 stage of the rows
constexpr int STAGE_B = BN * 128;       // bytes of one [256][64] bf16 stage of the matrix
constexpr int NSTG = 4;
constexpr int NT = 192;                 // warp 0: copies; warp 1: tensor cores; warps 2-5: epilogue
constexpr int SMEM_BYTES = NSTG * (STAGE_A + STAGE_B) + 1024;
constexpr uint32_t TMEM_COLS = 512;     // two fp32 accumulators of 256 columns

struct Args {
    int R, K, N;                        // rows (<= 128), inner dimension, output columns
    int n_tiles, splits, kps;           // tiles of 256 output columns; ranges of the inner dimension; stages per range
    int n_problems;                     // 1 or 2 products that share the shape (different operands)
    float *out[2];                      // [splits][R][N] fp32 partial sums of each problem
    int *status;
};

__global__ void __launch_bounds__(NT, 1)
skinny_gemm_kernel(const Args a, const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
                   const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1)
{
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long s_bar[2 * NSTG + 4];
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;

    fspad_pdl_wait();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = base, sB = base + NSTG * STAGE_A;
    const uint32_t bar0 = smem_u32(&s_bar[0]);
    auto full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty = [&](int s) { return bar0 + 8u * (uint32_t)(NSTG + s); };
    auto accf = [&](int b) { return bar0 + 8u * (uint32_t)(2 * NSTG + b); };
    auto acce = [&](int b) { return bar0 + 8u * (uint32_t)(2 * NSTG + 2 + b); };
    const int n_k = (a.K + BKE - 1) / BKE;
    const int per_problem = a.n_tiles * a.splits;
    const int n_items = per_problem * a.n_problems;
    const int my_items = ((int)blockIdx.x < n_items) ? (n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x : 0;
    // item -> (problem, tile, first stage, stages)
    auto decode = [&](int j, int &prob, int &tile, int &k0, int &nk) {
        const int item = (int)blockIdx.x + j * (int)gridDim.x;
        prob = item / per_problem;
        const int r = item % per_problem;
        tile = r / a.splits;
        const int sp = r % a.splits;
        k0 = sp * a.kps;
        nk = min(n_k, k0 + a.kps) - k0;
        return sp;
    };

    if (tid == 0) {
        for (int i = 0; i < 2 * NSTG + 4; ++i) mbar_init(bar0 + 8u * i, i >= 2 * NSTG + 2 ? 4 : 1);
        s_fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    if (warp == 1) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n"
                     :: "r"(smem_u32(&s_tmem)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    bool failed = false;
    int total_stages = 0;

    if (warp == 0) {
        // ================= copy warp =================
        // one thread's loop (its waits are plain polls; nothing is shuffled to the other lanes)
        int it = 0;
        if (lane == 0) {
            for (int j = 0; j < my_items; ++j) {
                int prob, tile, k0, nk;
                decode(j, prob, tile, k0, nk);
                const CUtensorMap *mA = prob ? &tmA1 : &tmA0, *mB = prob ? &tmB1 : &tmB0;
                for (int k = 0; k < nk; ++k, ++it) {
                    const int s = it % NSTG;
                    const uint32_t ph = (uint32_t)(it / NSTG) & 1u;
                    if (it >= NSTG && !failed && !mbar_wait_thread(empty(s), ph ^ 1u)) failed = true;
                    if (!failed) {
                        mbar_expect_tx(full(s), STAGE_A + STAGE_B);
                        tma_load_2d(sA + s * STAGE_A, mA, (k0 + k) * BKE, 0, full(s));
                        tma_load_2d(sB + s * STAGE_B, mB, (k0 + k) * BKE, tile * BN, full(s));
                    }
                }
            }
            if (failed) s_fail = 1;
        }
        it = __shfl_sync(0xffffffffu, it, 0);
        total_stages = it;
    } else if (warp == 1) {
        // ================= tensor-core warp =================
        if (lane == 0) {                              // one thread's loop, as the copy warp's
        const uint32_t elect = 1;
        const uint32_t hi = (uint32_t)(make_desc(0, 16) >> 32);
        const uint32_t a_lo = (uint32_t)make_desc(sA, 16), b_lo = (uint32_t)make_desc(sB, 16);
        const uint32_t idesc = make_idesc(false, BN);
        int it = 0;
        for (int j = 0; j < my_items; ++j) {
            int prob, tile, k0, nk;
            decode(j, prob, tile, k0, nk);
            const int buf = j & 1;
            if (j >= 2 && !failed && !mbar_wait_thread(acce(buf), (uint32_t)((j - 2) >> 1) & 1u)) failed = true;
            tc_fence_after();
            for (int k = 0; k < nk; ++k, ++it) {
                const int s = it % NSTG;
                const uint32_t ph = (uint32_t)(it / NSTG) & 1u;
                if (!failed && !mbar_wait_thread(full(s), ph)) failed = true;
                if (!failed) {
                    tc_fence_after();
                    const uint32_t soa = (uint32_t)s * (STAGE_A >> 4), sob = (uint32_t)s * (STAGE_B >> 4);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        mma_f16_lo(tmem + (uint32_t)buf * BN, a_lo + soa + ks * 2, hi, b_lo + sob + ks * 2, hi, idesc,
                                   (k > 0) || (ks > 0), elect);
                    mma_commit_if(empty(s), elect);
                    if (k == nk - 1) mma_commit_if(accf(buf), elect);
                }
            }
        }
        if (failed) s_fail = 1;
        }
        __syncwarp();
    } else {
        // ================= epilogue warps: one row per thread, fp32 partial sums out =================
        const int q = warp & 3;
        const int row = q * 32 + lane;
        const bool row_ok = row < a.R;
        for (int j = 0; j < my_items; ++j) {
            int prob, tile, k0, nk;
            const int sp = decode(j, prob, tile, k0, nk);
            const int buf = j & 1;
            if (!failed && !mbar_wait(accf(buf), (uint32_t)(j >> 1) & 1u)) failed = true;
            tc_fence_after();
            float *dst = a.out[prob] + ((size_t)sp * a.R + (row_ok ? row : 0)) * a.N + (size_t)tile * BN;
#pragma unroll 1
            for (int blk = 0; blk < BN / 32; ++blk) {
                float v[32];
                tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * BN + (uint32_t)blk * 32u, v);
                const int c = tile * BN + blk * 32;
                if (row_ok && !failed) {
                    if (c + 32 <= a.N && (a.N & 3) == 0) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            *reinterpret_cast<float4 *>(dst + blk * 32 + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (c + i < a.N) dst[blk * 32 + i] = v[i];
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(acce(buf));
        }
        if (failed) s_fail = 1;
    }
    fspad_pdl_trigger();
    tc_fence_before();
    __syncthreads();
    if (s_fail != 0) {
        // a wait ran out: what was started asynchronously gets a bounded time to land before the shared
        // and tensor memory go back to the SM
        if (tid == 0) fspad_report(a.status, FSPAD_ERR_TIMEOUT);
        if (warp == 0) {
            for (int s = 0; s < NSTG; ++s) {
                const int fills = (total_stages - s + NSTG - 1) / NSTG;
                if (fills > 0) (void)mbar_wait(full(s), (uint32_t)(fills - 1) & 1u, 20000);
            }
        } else if (warp == 1) {
            mma_commit_if(accf(0), lane == 0);
            __syncwarp();
        }
    }
    __syncthreads();
    if (warp != 1) return;
    tc_fence_after();
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" :: "r"(tmem), "r"(TMEM_COLS) : "memory");
}

__device__ __forceinline__ uint32_t pack2(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}

// s[r][i] = silu(sum of the Gate partials) * (sum of the Up partials), rounded to bf16; four columns per thread
__global__ void __launch_bounds__(256)
gate_product_kernel(const float *__restrict__ up, const float *__restrict__ gate, int splits, long long n4,
                    long long stride4, uint2 *__restrict__ out)
{
    fspad_pdl_trigger();
    fspad_pdl_wait();
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
        float4 u = make_float4(0.f, 0.f, 0.f, 0.f), g = u;
        for (int s = 0; s < splits; ++s) {
            const float4 a = __ldcg(reinterpret_cast<const float4 *>(up) + s * stride4 + i);
            const float4 b = __ldcg(reinterpret_cast<const float4 *>(gate) + s * stride4 + i);
            u.x += a.x; u.y += a.y; u.z += a.z; u.w += a.w;
            g.x += b.x; g.y += b.y; g.z += b.z; g.w += b.w;
        }
        auto silu = [](float x) { return x / (1.0f + __expf(-x)); };
        out[i] = make_uint2(pack2(silu(g.x) * u.x, silu(g.y) * u.y), pack2(silu(g.z) * u.z, silu(g.w) * u.w));
    }
}

// eta[r][h] = (sum of the Down partials) + f[r][h], rounded to bf16
__global__ void __launch_bounds__(256)
residual_out_kernel(const float *__restrict__ part, int splits, long long n4, long long stride4,
                    const uint2 *__restrict__ f, uint2 *__restrict__ out)
{
    fspad_pdl_trigger();
    fspad_pdl_wait();
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (long long)gridDim.x * blockDim.x) {
        float4 d = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int s = 0; s < splits; ++s) {
            const float4 a = __ldcg(reinterpret_cast<const float4 *>(part) + s * stride4 + i);
            d.x += a.x; d.y += a.y; d.z += a.z; d.w += a.w;
        }
        const uint2 fv = f[i];
        const float2 f0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&fv.x));
        const float2 f1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&fv.y));
        out[i] = make_uint2(pack2(d.x + f0.x, d.y + f0.y), pack2(d.z + f1.x, d.w + f1.y));
    }
}

// Ranges of the inner dimension per tile so that tiles * problems * ranges fills the SMs evenly: the
// smallest count (<= 8, every range at least four stages) whose last round is at least 85 % full,
// else the one with the fullest last round.
static void pick_splits(int sms, int items_per_split, int n_k, int *splits, int *kps)
{
    int best = 1;
    double best_eff = 0.0;
    for (int s = 1; s <= 8 && (n_k + s - 1) / s >= 4; ++s) {
        const int k = (n_k + s - 1) / s;
        if ((n_k + k - 1) / k != s) continue;                 // no empty range
        const long long items = (long long)items_per_split * s;
        const double eff = (double)items / (double)(((items + sms - 1) / sms) * sms);
        if (eff > best_eff + 1e-9) { best_eff = eff; best = s; }
        if (eff >= 0.85) { best = s; break; }
    }
    *splits = best;
    *kps = (n_k + best - 1) / best;
}

}  // namespace fsm

size_t fspad_feature_sampler_scratch_floats(int rows, int H, int I)
{
    // Up and Gate partials [2][<= 8][rows][I] and Down partials [<= 8][rows][H]
    return (size_t)8 * rows * ((size_t)2 * I + H);
}

cudaError_t fspad_launch_feature_sampler(fspad_ctx *ctx, const fspad_bf16 *f, const fspad_bf16 *e, const fspad_bf16 *wup,
                                         const fspad_bf16 *wgate, const fspad_bf16 *wdown, int R, int H, int I,
                                         fspad_bf16 *inter, fspad_bf16 *eta, float *scratch, cudaStream_t st)
{
    using namespace fsm;
    if (!ctx->fs_attr_done) {
        cudaError_t e0 = cudaFuncSetAttribute(skinny_gemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
        if (e0 != cudaSuccess) return e0;
        ctx->fs_attr_done = 1;
    }
    const int sms = ctx->sm_count;
    // ---- Up and Gate: two products [R][H] x [I][H]^T in one launch ----
    CUtensorMap mAf, mAe, mUp, mGate, mS, mDown;
    if (!fspad_make_tmap_bf16_2d(&mAf, f, (size_t)H, (size_t)R, BM) || !fspad_make_tmap_bf16_2d(&mAe, e, (size_t)H, (size_t)R, BM) ||
        !fspad_make_tmap_bf16_2d(&mUp, wup, (size_t)H, (size_t)I, BN, true) || !fspad_make_tmap_bf16_2d(&mGate, wgate, (size_t)H, (size_t)I, BN, true) ||
        !fspad_make_tmap_bf16_2d(&mS, inter, (size_t)I, (size_t)R, BM) || !fspad_make_tmap_bf16_2d(&mDown, wdown, (size_t)I, (size_t)H, BN, true))
        return cudaErrorInvalidValue;
    float *p_up = scratch, *p_gate = scratch + (size_t)8 * R * I, *p_down = scratch + (size_t)16 * R * I;
    Args a;
    a.R = R; a.K = H; a.N = I; a.n_tiles = (I + BN - 1) / BN; a.n_problems = 2;
    pick_splits(sms, a.n_tiles * 2, (H + BKE - 1) / BKE, &a.splits, &a.kps);
    a.out[0] = p_up; a.out[1] = p_gate; a.status = ctx->d_status;
    int items = a.n_tiles * a.splits * 2;
    ctx->launches++;
    cudaError_t err = fspad_launch(skinny_gemm_kernel, dim3(items < sms ? items : sms), dim3(NT), SMEM_BYTES, st, 0, a, mAf, mUp,
                                   mAe, mGate);
    if (err != cudaSuccess) return err;
    {
        const long long n4 = (long long)R * I / 4;
        const unsigned grid = (unsigned)((n4 + 255) / 256 < (long long)sms * 8 ? (n4 + 255) / 256 : (long long)sms * 8);
        ctx->launches++;
        err = fspad_launch(gate_product_kernel, dim3(grid), dim3(256), 0, st, 0, (const float *)p_up, (const float *)p_gate,
                           a.splits, n4, n4, reinterpret_cast<uint2 *>(inter));
        if (err != cudaSuccess) return err;
    }
    // ---- Down: [R][I] x [H][I]^T, then the residual ----
    Args d;
    d.R = R; d.K = I; d.N = H; d.n_tiles = (H + BN - 1) / BN; d.n_problems = 1;
    pick_splits(sms, d.n_tiles, (I + BKE - 1) / BKE, &d.splits, &d.kps);
    d.out[0] = p_down; d.out[1] = p_down; d.status = ctx->d_status;
    items = d.n_tiles * d.splits;
    ctx->launches++;
    err = fspad_launch(skinny_gemm_kernel, dim3(items < sms ? items : sms), dim3(NT), SMEM_BYTES, st, 0, d, mS, mDown, mS, mDown);
    if (err != cudaSuccess) return err;
    const long long n4 = (long long)R * H / 4;
    const unsigned grid = (unsigned)((n4 + 255) / 256 < (long long)sms * 8 ? (n4 + 255) / 256 : (long long)sms * 8);
    ctx->launches++;
    return fspad_launch(residual_out_kernel, dim3(grid), dim3(256), 0, st, 0, (const float *)p_down, d.splits, n4, n4,
                        reinterpret_cast<const uint2 *>(f), reinterpret_cast<uint2 *>(eta));
}
