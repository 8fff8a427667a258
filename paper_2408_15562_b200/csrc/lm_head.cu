// Target LM head with the per-node vocabulary scan as its epilogue.
//
// The acceptance stage compares the tree with the target's distribution at every
// tree node (paper, Section "Preliminaries": one target forward over the
// flattened tree, then strict comparison).  The last step of that forward is the
// product of the nodes' final hidden states with the vocabulary matrix; here its
// tiles are reduced to the scan's partial results (maximum, lowest index of the
// maximum, sum of exponentials) as they leave the tensor cores, so the logits
// need not make a round trip through HBM before they are scanned, and need not be
// written at all when every sequence is greedy.
//
//   logits[r][v] = sum_h hidden[r][h] * weight[v][h]      bf16 x bf16 -> fp32
//
// With a handful of rows the product is bound by streaming the vocabulary matrix
// once (2 * H * V bytes).  One persistent CTA per SM walks over work items of 256
// vocabulary entries (and, for what does not fill a whole round of the grid, of
// 128, so that the last round is short instead of idle); per item it streams the
// [256][H] slab of the matrix and the hidden states (up to 128 rows, re-read from
// L2) through a ring of 128-byte-swizzled [256][64] / [128][64] bf16 stages filled
// by TMA, accumulates 128 x 256 x 16 tcgen05.mma into one of two tensor-memory
// accumulators, and four epilogue warps (one row per thread) reduce the finished
// accumulator, 128 columns (one tile of partial results) at a time, while the next
// item is being multiplied.  Measured on 60 x 4096 x 128256: 128-wide items with six
// 16 KB matrix stages 214 us, 256-wide items with four 32 KB stages 207 us, and with
// the matrix's tensor map asking L2 for 256 bytes per request (the next stage of the
// same rows comes along: fewer, longer DRAM bursts per open page) 196 us.  Roles meet
// only on mbarriers; every wait is bounded.
#include <cuda.h>

#include "common.cuh"
#include "umma_common.cuh"

namespace lmh {

using namespace umma;

constexpr int BM = 128;                 // rows of hidden states per CTA (one accumulator lane each)
constexpr int BN = 128;                 // vocabulary entries per tile (one partial result per row and tile)
constexpr int BKE = 64;                 // hidden elements per stage (128 bytes: the swizzle span)
constexpr int STAGE = 128 * 128;        // bytes of one [128][64] bf16 box
constexpr int STAGE_B = 2 * STAGE;      // matrix stage: two boxes = 256 vocabulary entries
constexpr int NSTG = 4;                 // stages in flight
constexpr int NT = 192;                 // warp 0: copies; warp 1: tensor cores; warps 2-5: epilogue
constexpr int SMEM_BYTES = NSTG * (STAGE + STAGE_B) + 1024;
constexpr uint32_t TMEM_COLS = 512;     // two fp32 accumulators of 256 columns
constexpr float kLog2e = 1.4426950408889634f;

struct Args {
    int R, H, V, n_tiles, rows_per_seq, ld_logits, row0;   // row0: number of the slab's first row in the caller's arrays
    const float *temperature;
    float *logits;                      // [R][ld_logits] or NULL
    FspadStatsPart *parts;              // [R][n_tiles]
    int *status;
};

__global__ void __launch_bounds__(NT, 1)
lm_head_stats_kernel(const Args a, const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB)
{
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long s_bar[2 * NSTG + 4];
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;

    fspad_pdl_wait();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sA = base, sB = base + NSTG * STAGE;     // rows: NSTG x 16 KB, matrix: NSTG x 32 KB
    const uint32_t bar0 = smem_u32(&s_bar[0]);
    auto full = [&](int s) { return bar0 + 8u * (uint32_t)s; };
    auto empty = [&](int s) { return bar0 + 8u * (uint32_t)(NSTG + s); };
    auto accf = [&](int b) { return bar0 + 8u * (uint32_t)(2 * NSTG + b); };
    auto acce = [&](int b) { return bar0 + 8u * (uint32_t)(2 * NSTG + 2 + b); };
    const int n_k = (a.H + BKE - 1) / BKE;
    // Work items: pairs of tiles for as many whole rounds of the grid as there are, single tiles after that.
    const int G = (int)gridDim.x;
    const int wide_rounds = (a.n_tiles / 2) / G;
    const int first_single = 2 * wide_rounds * G;                   // tiles from here on go out one by one
    const int n_single = a.n_tiles - first_single;
    const int my_single = ((int)blockIdx.x < n_single) ? (n_single - (int)blockIdx.x + G - 1) / G : 0;
    const int my_items = wide_rounds + my_single;
    // item j of this CTA -> first tile and number of tiles (2 or 1)
    auto item = [&](int j, int &tile, int &width) {
        if (j < wide_rounds) { tile = 2 * ((int)blockIdx.x + j * G); width = 2; }
        else { tile = first_single + (int)blockIdx.x + (j - wide_rounds) * G; width = 1; }
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

    if (warp == 0) {
        // ================= copy warp: one thread runs the whole loop (its waits are plain polls) =================
        if (lane == 0) {
            int it = 0;
            for (int j = 0; j < my_items; ++j) {
                int tile, width;
                item(j, tile, width);
                for (int k = 0; k < n_k; ++k, ++it) {
                    const int s = it % NSTG;
                    const uint32_t ph = (uint32_t)(it / NSTG) & 1u;
                    if (it >= NSTG && !failed && !mbar_wait_thread(empty(s), ph ^ 1u)) failed = true;
                    if (!failed) {
                        mbar_expect_tx(full(s), (1 + width) * STAGE);
                        tma_load_2d(sA + s * STAGE, &tmA, k * BKE, 0, full(s));
                        tma_load_2d(sB + s * STAGE_B, &tmB, k * BKE, tile * BN, full(s));
                        if (width == 2) tma_load_2d(sB + s * STAGE_B + STAGE, &tmB, k * BKE, (tile + 1) * BN, full(s));
                    }
                }
            }
            if (failed) s_fail = 1;
        }
        __syncwarp();
    } else if (warp == 1) {
        // ================= tensor-core warp: one thread runs the whole loop =================
        if (lane == 0) {
        const uint32_t elect = 1;
        const uint32_t hi = (uint32_t)(make_desc(0, 16) >> 32);
        const uint32_t a_lo = (uint32_t)make_desc(sA, 16), b_lo = (uint32_t)make_desc(sB, 16);
        const uint32_t idesc2 = make_idesc(false, 2 * BN), idesc1 = make_idesc(false, BN);
        int it = 0;
        for (int j = 0; j < my_items; ++j) {
            int tile, width;
            item(j, tile, width);
            const uint32_t idesc = width == 2 ? idesc2 : idesc1;
            const int buf = j & 1;
            // the accumulator is free once the epilogue has read the tile that used it two tiles ago
            if (j >= 2 && !failed && !mbar_wait_thread(acce(buf), (uint32_t)((j - 2) >> 1) & 1u)) failed = true;
            tc_fence_after();
            for (int k = 0; k < n_k; ++k, ++it) {
                const int s = it % NSTG;
                const uint32_t ph = (uint32_t)(it / NSTG) & 1u;
                if (!failed && !mbar_wait_thread(full(s), ph)) failed = true;
                if (!failed) {
                    tc_fence_after();
                    const uint32_t soa = (uint32_t)s * (STAGE >> 4), sob = (uint32_t)s * (STAGE_B >> 4);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)      // 16 hidden elements = 32 bytes per instruction
                        mma_f16_lo(tmem + (uint32_t)buf * (2 * BN), a_lo + soa + ks * 2, hi, b_lo + sob + ks * 2, hi, idesc,
                                   (k > 0) || (ks > 0), elect);
                    mma_commit_if(empty(s), elect);
                    if (k == n_k - 1) mma_commit_if(accf(buf), elect);
                }
            }
        }
        if (failed) s_fail = 1;
        }
        __syncwarp();
    } else {
        // ================= epilogue warps: one row per thread =================
        const int q = warp & 3;                          // tensor-memory lane quarter this warp may read
        const int row = q * 32 + lane;
        const bool row_ok = row < a.R;
        float T = 1.0f;
        if (row_ok && a.temperature) T = a.temperature[(a.row0 + row) / a.rows_per_seq];
        if (!(T > 0.0f)) T = 1.0f;
        const float kk = kLog2e / T;
        for (int j = 0; j < my_items; ++j) {
            int tile0, width;
            item(j, tile0, width);
            const int buf = j & 1;
            if (!failed && !mbar_wait(accf(buf), (uint32_t)(j >> 1) & 1u)) failed = true;
            tc_fence_after();
#pragma unroll 1
          for (int half = 0; half < width; ++half) {
            const int tile = tile0 + half;
            float m = -INFINITY, s = 0.f;
            int arg = 0x7fffffff;
            const int col0 = tile * BN;
#pragma unroll 1
            for (int blk = 0; blk < BN / 32; ++blk) {
                float v[32];
                tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * (2 * BN) + (uint32_t)(half * BN + blk * 32), v);
                const int c = col0 + blk * 32;
                if (c + 32 > a.V) {
#pragma unroll
                    for (int i = 0; i < 32; ++i)
                        if (c + i >= a.V) v[i] = -INFINITY;
                }
                if (a.logits != nullptr && row_ok && !failed) {
                    float *dst = a.logits + (size_t)row * a.ld_logits + c;
                    if (c + 32 <= a.V && (a.ld_logits & 3) == 0) {
#pragma unroll
                        for (int i = 0; i < 32; i += 4)
                            *reinterpret_cast<float4 *>(dst + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
                    } else {
#pragma unroll
                        for (int i = 0; i < 32; ++i)
                            if (c + i < a.V) dst[i] = v[i];
                    }
                }
                float bm = v[0];
#pragma unroll
                for (int i = 1; i < 32; ++i) bm = fmaxf(bm, v[i]);
                if (bm > m) {
                    s = (m == -INFINITY) ? 0.f : s * ex2f((m - bm) * kk);
                    m = bm;
                    int first = 0;
#pragma unroll
                    for (int i = 31; i >= 0; --i)
                        if (v[i] == bm) first = i;
                    arg = c + first;
                }
                if (m != -INFINITY) {
                    float acc = 0.f;
#pragma unroll
                    for (int i = 0; i < 32; ++i) acc += ex2f((v[i] - m) * kk);
                    s += acc;
                }
            }
            if (row_ok && !failed) {
                FspadStatsPart out;
                out.m = m; out.s = s; out.a = (arg == 0x7fffffff) ? col0 : arg; out.pad = 0;
                a.parts[(size_t)row * a.n_tiles + tile] = out;
            }
          }
            // the accumulator may be overwritten: every lane's loads have completed (tmem_ld32 waits)
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
        // a wait ran out: whatever was started asynchronously gets a bounded time to land before the
        // shared and tensor memory go back to the SM
        if (tid == 0) fspad_report(a.status, FSPAD_ERR_TIMEOUT);
        if (warp == 0) {
            const int total = my_items * n_k;
            for (int s = 0; s < NSTG; ++s) {
                const int fills = (total - s + NSTG - 1) / NSTG;     // upper bound of the fills started in stage s
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

// merge of two partial results (maximum, lowest index, sum rescaled to the common maximum)
__device__ __forceinline__ void merge_part(float &m, float &s, int &arg, float om, float os, int oa, float kk)
{
    if (om == -INFINITY) return;
    if (m == -INFINITY) { m = om; s = os; arg = oa; return; }
    const float mn = fmaxf(m, om);
    s = s * exp2f((m - mn) * kk) + os * exp2f((om - mn) * kk);
    if (om > m || (om == m && oa < arg)) arg = oa;
    m = mn;
}

// Tile partials -> one partial per output slot.  Slot (row, p) covers the tiles [t0, t1) that the
// caller's geometry gives it; one warp per slot.  With `rows_out` the result goes out as row
// statistics (one slot per row), otherwise as FspadStatsPart into out_parts[row * slots + p].
__global__ void __launch_bounds__(128)
lm_head_merge_kernel(const FspadStatsPart *__restrict__ tile_parts, int R, int n_tiles, int rows_per_seq,
                     const float *__restrict__ temperature, int row0, FspadStatsGeom g, int tile_units,
                     FspadStatsPart *__restrict__ out_parts, float *__restrict__ row_max, double *__restrict__ row_sum,
                     int *__restrict__ row_arg)
{
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const int lane = threadIdx.x & 31;
    const long long wi = (long long)blockIdx.x * 4 + (threadIdx.x >> 5);
    const bool as_rows = out_parts == nullptr;
    const int per_row = as_rows ? 1 : g.slots;
    if (wi >= (long long)R * per_row) return;
    const int r = (int)(wi / per_row), p = (int)(wi % per_row);     // r: row inside this slab
    const int grow = row0 + r;                                       // row in the caller's numbering
    int t0 = 0, t1 = n_tiles;
    if (!as_rows) {
        // piece p of the row in the flat geometry: units [max(row_lo, (first+p) chunk), min(row_hi, (first+p+1) chunk))
        const long long row_lo = (long long)grow * g.upr, row_hi = row_lo + g.upr;
        const long long first = row_lo / g.chunk;
        const long long u_lo = max(row_lo, (first + p) * g.chunk), u_hi = min(row_hi, (first + p + 1) * g.chunk);
        if (u_lo >= u_hi) return;                                    // the row has fewer pieces
        t0 = (int)((u_lo - row_lo) / tile_units);
        t1 = (int)((u_hi - row_lo + tile_units - 1) / tile_units);
    }
    float T = temperature ? temperature[grow / rows_per_seq] : 1.0f;
    if (!(T > 0.0f)) T = 1.0f;
    const float kk = lmh::kLog2e / T;
    float m = -INFINITY, s = 0.f;
    int arg = 0x7fffffff;
    // A lane's partials are requested eight at a time, before any of them is merged: the merge carries a
    // dependency from one partial to the next, and with one request per step a row of a thousand tiles was
    // thirty-two trips to L2 one after the other (about 19 us of a 190 us call).
    constexpr int kAhead = 8;
    for (int tb = t0 + lane; tb < t1; tb += 32 * kAhead) {
        int4 v[kAhead];
#pragma unroll
        for (int u = 0; u < kAhead; ++u) {
            const int t = tb + 32 * u;
            v[u] = make_int4(__float_as_int(-INFINITY), 0, 0x7fffffff, 0);
            if (t < t1) v[u] = __ldcg(reinterpret_cast<const int4 *>(tile_parts + (size_t)r * n_tiles + t));
        }
#pragma unroll
        for (int u = 0; u < kAhead; ++u)
            if (tb + 32 * u < t1) merge_part(m, s, arg, __int_as_float(v[u].x), __int_as_float(v[u].y), v[u].z, kk);
    }
    double sd = 0.0;
    {
        float mm = m;
        int aa = arg;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, mm, off);
            const int oa = __shfl_xor_sync(0xffffffffu, aa, off);
            if (om > mm || (om == mm && oa < aa)) { mm = om; aa = oa; }
        }
        sd = (m == -INFINITY) ? 0.0 : (double)s * (double)exp2f((m - mm) * kk);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) sd += __shfl_xor_sync(0xffffffffu, sd, off);
        m = mm;
        arg = aa;
    }
    if (lane == 0) {
        if (as_rows) {
            row_max[grow] = m;
            row_sum[grow] = sd;
            row_arg[grow] = (arg == 0x7fffffff) ? 0 : arg;
        } else {
            FspadStatsPart out;
            out.m = m; out.s = (float)sd; out.a = arg; out.pad = 0;
            out_parts[(size_t)grow * g.slots + p] = out;
        }
    }
}

}  // namespace lmh

int fspad_lm_head_tiles(int V) { return (V + lmh::BN - 1) / lmh::BN; }

// Geometry under which the walk reads the merged partials: pieces of whole tiles, at most 16 per row,
// when the rows are whole numbers of tiles; one piece per row otherwise.
FspadStatsGeom fspad_lm_head_geom(int rows, int V, bool vec, int slots)
{
    FspadStatsGeom g;
    g.unit = vec ? 4 : 1;
    g.upr = V / g.unit;
    g.slots = slots;
    g.total = (long long)rows * g.upr;
    g.threads = FSPAD_STATS_THREADS;            // no scan kernel runs on this geometry; the walk reads the pieces only
    const int tile_units = lmh::BN / g.unit;
    if (V % lmh::BN == 0) {
        const int n_tiles = V / lmh::BN;
        const int tp = (n_tiles + 13) / 14;               // tiles per piece: a row then spans at most 16 pieces
        g.chunk = (long long)tp * tile_units;
    } else {
        g.chunk = g.upr;
    }
    g.n_cta = (int)((g.total + g.chunk - 1) / g.chunk);
    return g;
}

// rows 0 .. R-1 of hidden ([R][H]) against weight ([V][H]); slabs of 128 rows, one launch each
cudaError_t fspad_launch_lm_head(fspad_ctx *ctx, const fspad_bf16 *hidden, const fspad_bf16 *weight, int H, int R,
                                 int rows_per_seq, const float *temperature, float *logits, const FspadStatsGeom *walk_geom,
                                 float *row_max, double *row_sum, int *row_arg, cudaStream_t st)
{
    const int V = ctx->cfg.vocab;
    const int n_tiles = fspad_lm_head_tiles(V);
    if (!ctx->lm_attr_done) {
        cudaError_t e = cudaFuncSetAttribute(lmh::lm_head_stats_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             lmh::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        ctx->lm_attr_done = 1;
    }
    CUtensorMap mB;
    if (!fspad_make_tmap_bf16_2d(&mB, weight, (size_t)H, (size_t)V, lmh::BN, true)) return cudaErrorInvalidValue;
    for (int r0 = 0; r0 < R; r0 += lmh::BM) {
        const int rs = (R - r0 < lmh::BM) ? R - r0 : lmh::BM;
        CUtensorMap mA;
        if (!fspad_make_tmap_bf16_2d(&mA, hidden + (size_t)r0 * H, (size_t)H, (size_t)rs, lmh::BM)) return cudaErrorInvalidValue;
        lmh::Args a;
        a.R = rs; a.H = H; a.V = V; a.n_tiles = n_tiles; a.rows_per_seq = rows_per_seq; a.ld_logits = V; a.row0 = r0;
        a.temperature = temperature;
        a.logits = logits ? logits + (size_t)r0 * V : nullptr;
        a.parts = ctx->lm_parts;
        a.status = ctx->d_status;
        const int grid = ctx->sm_count < n_tiles ? ctx->sm_count : n_tiles;
        ctx->launches++;
        cudaError_t e = fspad_launch_opt(r0 == 0, lmh::lm_head_stats_kernel, dim3(grid), dim3(lmh::NT), lmh::SMEM_BYTES, st, 0,
                                         a, mA, mB);
        if (e != cudaSuccess) return e;
        ctx->launches++;
        const bool as_rows = walk_geom == nullptr;
        FspadStatsGeom g = as_rows ? FspadStatsGeom() : *walk_geom;
        const long long warps = (long long)rs * (as_rows ? 1 : g.slots);
        e = fspad_launch(lmh::lm_head_merge_kernel, dim3((unsigned)((warps + 3) / 4)), dim3(128), 0, st, 0,
                         (const FspadStatsPart *)ctx->lm_parts, rs, n_tiles, rows_per_seq, temperature, r0, g,
                         as_rows ? 1 : lmh::BN / g.unit, as_rows ? (FspadStatsPart *)nullptr : ctx->st_part, row_max, row_sum,
                         row_arg);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}
