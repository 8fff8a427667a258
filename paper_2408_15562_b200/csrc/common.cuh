// Internal declarations shared by the translation units of libfspad.so.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include <utility>

#include "fspad.h"

#define FSPAD_MAX_NODES 64           /* nodes of a tree on the one-mask-word paths */
#define FSPAD_MAX_NODES_WIDE 256     /* nodes of a tree, any call of the verify step */
#define FSPAD_MAX_CANDIDATES 1024
#define FSPAD_MAX_FRONTIER 16      /* frontier nodes per sequence, and top-k per row, of a draft step */
#define FSPAD_HEAD_DIM 128
#define FSPAD_STATS_THREADS 256

// Scratch and bookkeeping owned by a context (all device pointers unless noted).
struct fspad_ctx {
    fspad_config cfg;
    int device;
    int sm_count;
    float scale;              // softmax scale actually used
    long long launches;       // host counter of kernels launched

    int *d_status;            // first device-detected error (0 = none)

    // split-KV attention partials
    int attn_max_splits;
    int attn_attr_done;       // dynamic shared-memory limit raised for the attention kernels
    // TMA descriptors of the K and V cache planes last seen (re-encoded when they change)
    alignas(64) unsigned char attn_tmap_k[128];
    alignas(64) unsigned char attn_tmap_v[128];
    const void *attn_tmap_kptr, *attn_tmap_vptr;
    size_t attn_tmap_rows;
    int attn_tmap_ok;
    float *part_o;            // [batch][Hkv][splits][M][d]
    float *part_ml;           // [batch][Hkv][splits][M][2]  (running max in log2 units, sum)

    // per-node vocabulary scan
    int stats_slots;          // partial slots per row in st_part
    struct FspadStatsPart *st_part;   // [rows][stats_slots]
    float *row_max;           // [rows]
    double *row_sum;
    int *row_arg;
    int walk_cluster;         // cluster size used by the sampling walk (0 = not probed yet)

    // whole-step entry point: attention runs on `side`, forked from and joined into the caller's stream
    cudaStream_t side;
    cudaEvent_t ev_fork, ev_join;

    // LM head: per-(row, vocabulary tile) partials of one slab of 128 rows, [128][tiles]
    struct FspadStatsPart *lm_parts;
    int lm_attr_done;
    int fs_attr_done;         // dynamic shared-memory limit raised for the Feature Sampler's product kernel

    void *dx_part;            // draft step: per-piece top-k lists [max_batch * 16 rows][pieces][16] (value, token)

    // device staging for the host entry point (h_ready: every buffer below is allocated)
    int h_ready;
    fspad_bf16 *h_q, *h_tk, *h_tv, *h_out;
    int *h_parent, *h_prefix, *h_tokens, *h_path, *h_nacc, *h_bonus, *h_newlen;
    float *h_logits, *h_draft, *h_temp, *h_unif;
};

// One CTA's contribution to a row of the vocabulary scan.
struct FspadStatsPart {
    float m;   // maximum over the CTA's part of the row
    float s;   // sum of exp2((x - m) * log2(e) / T) over that part
    int a;     // lowest index attaining m
    int pad;
};

// How the flat [rows x V] logits array is cut into equal per-CTA ranges.
struct FspadStatsGeom {
    int unit;          // floats per load unit: 4 (128-bit loads) or 1
    int upr;           // units per row
    int n_cta;         // CTAs in the grid
    int slots;         // partial slots per row (capacity)
    long long chunk;   // units per CTA
    long long total;   // rows * upr
    int threads;       // threads per CTA of the scan: FSPAD_STATS_THREADS, or half of it for a small array
};

// small_ctas: the scan may use CTAs of half the size when the array is small (the pieces, one of which the
// acceptance walk's bonus draw sweeps, halve with them; on a large array the smaller CTAs cost bandwidth:
// 5.93 against 6.20 TB/s on 960 rows of 128256)
static inline FspadStatsGeom fspad_stats_geom(int sm_count, int rows, int V, bool vec, int slots, bool small_ctas = false)
{
    FspadStatsGeom g;
    g.unit = vec ? 4 : 1;
    g.upr = V / g.unit;
    g.slots = slots;
    g.total = (long long)rows * g.upr;
    g.threads = FSPAD_STATS_THREADS;
    // up to 32 units per thread of one wave at 1024 threads per SM
    if (small_ctas && g.total <= (long long)sm_count * 1024 * 32) g.threads = FSPAD_STATS_THREADS / 2;
    long long n = (long long)sm_count * (1024 / g.threads);   // 1024 threads per SM, one wave
    const long long by_size = (g.total + g.threads - 1) / g.threads;   // at least one unit per thread
    if (n > by_size) n = by_size;
    if (n < 1) n = 1;
    g.chunk = (g.total + n - 1) / n;
    // A CTA whose range crosses a row boundary runs its reduction sequence twice and finishes about a
    // microsecond behind the others.  Where a row divides evenly into a whole number k of pieces such that
    // rows * k CTAs still fill three quarters of the wave, ranges are cut at the rows instead.
    if (rows >= 1 && n >= rows) {
        bool cut = false;
        // The acceptance walk keeps the masses of at most 16 pieces per row for its bonus draw (with more it
        // sweeps the whole row): with few rows, 16 pieces per row are preferred to a full wave as long as
        // every SM still gets a CTA.
        if (n / rows > 16 && (long long)rows * 16 >= sm_count) {
            for (long long k = 16; k >= 8 && !cut; --k)
                if (g.upr % k == 0) { g.chunk = g.upr / k; cut = true; }
        }
        for (long long k = n / rows; !cut && k >= 1 && (long long)rows * k * 4 >= n * 3; --k)
            if (g.upr % k == 0) { g.chunk = g.upr / k; cut = true; }
    }
    // a row may be shared by at most `slots` CTAs
    const long long min_chunk = (g.upr + (slots - 2) - 1) / (slots - 2);
    if (g.chunk < min_chunk) g.chunk = min_chunk;
    g.n_cta = (int)((g.total + g.chunk - 1) / g.chunk);
    return g;
}

#ifdef __CUDACC__
// Merge the per-CTA partials of one row (warp-collective: all 32 lanes call it and all get
// the result): maximum, its lowest index, and the sum of exponentials rescaled to that
// maximum (k = log2(e)/T).  Every lane fetches up to two partial slots, so the loads of a
// row are in flight together instead of one after another.
__device__ __forceinline__ void fspad_stats_merge_warp(const FspadStatsPart *__restrict__ parts,
                                                       const FspadStatsGeom &g, int row, float k, int lane,
                                                       float &M, double &S, int &A)
{
    const long long r0 = (long long)row * g.upr;
    const int first = (int)(r0 / g.chunk), last = (int)((r0 + g.upr - 1) / g.chunk);
    const int cnt = last - first + 1;                       // <= g.slots <= 64
    const FspadStatsPart *p = parts + (size_t)row * g.slots;
    float m0 = -INFINITY, m1 = -INFINITY, s0 = 0.f, s1 = 0.f;
    int a0 = 0x7fffffff, a1 = 0x7fffffff;
    if (lane < cnt) {
        const int4 v = __ldcg(reinterpret_cast<const int4 *>(p + lane));
        m0 = __int_as_float(v.x); s0 = __int_as_float(v.y); a0 = v.z;
    }
    if (lane + 32 < cnt) {
        const int4 v = __ldcg(reinterpret_cast<const int4 *>(p + lane + 32));
        m1 = __int_as_float(v.x); s1 = __int_as_float(v.y); a1 = v.z;
    }
    float m = m0;
    int a = a0;
    if (m1 > m || (m1 == m && a1 < a)) { m = m1; a = a1; }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, off);
        const int oa = __shfl_xor_sync(0xffffffffu, a, off);
        if (om > m || (om == m && oa < a)) { m = om; a = oa; }
    }
    double s = 0.0;
    if (m0 != -INFINITY) s += (double)s0 * (double)exp2f((m0 - m) * k);
    if (m1 != -INFINITY) s += (double)s1 * (double)exp2f((m1 - m) * k);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off);
    M = m;
    S = s;
    A = (a == 0x7fffffff) ? 0 : a;
}

// The same merge by a half-warp (16 lanes, up to four slots per lane), so that one warp
// serves two rows at once.  Both halves of the warp must call it together; `valid` is false
// for a half that has no row (it only takes part in the shuffles).  With `piece_w` given, the
// mass of each of the row's pieces relative to the row maximum (what it adds to S) is stored
// there, slot by slot, when the row has at most 16 pieces; *piece_cnt is the number of pieces,
// or 0 when there are more than 16.
__device__ __forceinline__ void fspad_stats_merge_half(const FspadStatsPart *__restrict__ parts,
                                                       const FspadStatsGeom &g, int row, bool valid, float k,
                                                       int lane16, float &M, double &S, int &A,
                                                       double *piece_w = nullptr, int *piece_cnt = nullptr)
{
    int cnt = 0;
    const FspadStatsPart *p = parts;
    if (valid) {
        const long long r0 = (long long)row * g.upr;
        const int first = (int)(r0 / g.chunk), last = (int)((r0 + g.upr - 1) / g.chunk);
        cnt = last - first + 1;
        p = parts + (size_t)row * g.slots;
    }
    float mi[4], si[4];
    int ai[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        mi[u] = -INFINITY; si[u] = 0.f; ai[u] = 0x7fffffff;
        const int sl = lane16 + 16 * u;
        if (sl < cnt) {
            const int4 v = __ldcg(reinterpret_cast<const int4 *>(p + sl));
            mi[u] = __int_as_float(v.x); si[u] = __int_as_float(v.y); ai[u] = v.z;
        }
    }
    float m = mi[0];
    int a = ai[0];
#pragma unroll
    for (int u = 1; u < 4; ++u)
        if (mi[u] > m || (mi[u] == m && ai[u] < a)) { m = mi[u]; a = ai[u]; }
#pragma unroll
    for (int off = 8; off > 0; off >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, m, off, 16);
        const int oa = __shfl_xor_sync(0xffffffffu, a, off, 16);
        if (om > m || (om == m && oa < a)) { m = om; a = oa; }
    }
    double s = 0.0;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const double w = (mi[u] != -INFINITY) ? (double)si[u] * (double)exp2f((mi[u] - m) * k) : 0.0;
        s += w;
        if (u == 0 && piece_w != nullptr && valid && lane16 < cnt && cnt <= 16) piece_w[lane16] = w;
    }
    if (piece_cnt != nullptr && valid && lane16 == 0) *piece_cnt = (cnt <= 16) ? cnt : 0;
#pragma unroll
    for (int off = 8; off > 0; off >>= 1) s += __shfl_xor_sync(0xffffffffu, s, off, 16);
    M = m;
    S = s;
    A = (a == 0x7fffffff) ? 0 : a;
}
#endif

// ---- programmatic dependent launch -----------------------------------------------------
// Every kernel of the library is launched with the programmatic-serialization attribute and
// follows one rule: it lets its successor start launching at once (fspad_pdl_trigger) and it
// touches global memory only after the whole preceding kernel of the stream has completed and
// flushed (fspad_pdl_wait).  Launch latency and the memory-free part of a prologue (barrier
// set-up, tensor-memory allocation, table fills) then overlap the tail of the previous kernel,
// while results stay exactly those of plain stream order.
#ifdef __CUDACC__
__device__ __forceinline__ void fspad_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void fspad_pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t fspad_launch_opt(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                           cudaStream_t st, unsigned cluster_x, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    int n = 0;
    if (pdl) {
        attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n].val.programmaticStreamSerializationAllowed = 1;
        ++n;
    }
    if (cluster_x > 0) {
        attr[n].id = cudaLaunchAttributeClusterDimension;
        attr[n].val.clusterDim.x = cluster_x; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
        ++n;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n;
    return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
template <typename... KArgs, typename... Args>
static inline cudaError_t fspad_launch(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                       cudaStream_t st, unsigned cluster_x, Args &&...args)
{
    return fspad_launch_opt(true, kernel, grid, block, smem, st, cluster_x, std::forward<Args>(args)...);
}
#endif

static inline cudaStream_t fspad_stream(void *s) { return reinterpret_cast<cudaStream_t>(s); }

// Record the first device-side error; later ones are dropped.
__device__ __forceinline__ void fspad_report(int *status, int err)
{
    atomicCAS(status, 0, err);
}

// launchers implemented in the kernel translation units (return cudaError_t)
cudaError_t fspad_launch_accept_stats(fspad_ctx *ctx, const float *logits, const float *temperature,
                                      int rows, int rows_per_seq, int V, float *row_max,
                                      double *row_sum, int *row_arg, cudaStream_t st);
// cache != NULL: the walk also compacts the accepted path's rows of `cache` (all layers of the context) and
// writes new_len; the caller then launches no compaction
struct FspadWalkCompact {
    fspad_bf16 *cache = nullptr;
    const int *prefix_len = nullptr;
    int *new_len = nullptr;
};
cudaError_t fspad_launch_accept_walk(fspad_ctx *ctx, const float *logits, const float *draft,
                                     const int *tokens, const int *parent, const float *temperature,
                                     const float *uniforms, const FspadStatsGeom &geom, int N, int B, int V,
                                     int *path, int *n_acc, int *bonus, cudaStream_t st, FspadWalkCompact kv = {});
// pdl = false: launched as a plain dependent of what precedes it in the stream (griddepcontrol.wait is
// then a no-op; the guarantee its successor relies on holds either way)
cudaError_t fspad_launch_stats_partials(fspad_ctx *ctx, const float *logits, const float *temperature,
                                        int rows, int rows_per_seq, int V, FspadStatsGeom *geom,
                                        cudaStream_t st, bool pdl = true, int sms = 0);   // sms > 0: one wave on that many SMs
cudaError_t fspad_launch_tree_build(fspad_ctx *ctx, const int *cand_parent, const int *cand_token,
                                    const float *cand_logp, const int *root_token, int n_cand, int n_nodes,
                                    int B, int *parent_out, int *token_out, int *cand_out,
                                    unsigned long long *anc_out, int *n_out, cudaStream_t st);
int fspad_draft_expand_pieces(int V);
cudaError_t fspad_launch_draft_expand(fspad_ctx *ctx, const float *logprobs, const float *frontier_logp,
                                      const int *frontier_cand, int F, int k, int width, int base, int cap, int B,
                                      int *cand_parent, int *cand_token, float *cand_logp, int *next_cand,
                                      float *next_logp, cudaStream_t st);
cudaError_t fspad_launch_kv_compact(fspad_ctx *ctx, fspad_bf16 *cache, const int *path,
                                    const int *n_acc, const int *prefix_len, int B, int *new_len,
                                    cudaStream_t st, bool pdl = true);
// A cache kept as a pool of 128-row blocks: table[b * stride + i] is the block with rows 128 i .. 128 i + 127
// of sequence b (table == NULL: contiguous cache).
struct FspadPaged {
    const int *table;
    int stride, n_blocks;
};
// sms: how many SMs the call may fill with CTAs (0 = all of them).  merge_pdl: the merge kernel is a programmatic
// dependent of the attention kernel (its CTAs become resident, waiting, as the attention's last CTAs finish).
cudaError_t fspad_launch_tree_attn(fspad_ctx *ctx, const fspad_bf16 *q, const fspad_bf16 *kc,
                                   const fspad_bf16 *vc, const fspad_bf16 *tk, const fspad_bf16 *tv,
                                   const int *parent, const int *prefix_len, int N, int B,
                                   fspad_bf16 *out, cudaStream_t st, int sms = 0, FspadPaged paged = FspadPaged{nullptr, 0, 0},
                                   bool merge_pdl = true);
cudaError_t fspad_launch_tree_scatter(fspad_ctx *ctx, fspad_bf16 *cache, const fspad_bf16 *tk,
                                      const fspad_bf16 *tv, const int *prefix_len, int N, int B,
                                      cudaStream_t st);
int fspad_attn_umma_splits(const fspad_ctx *ctx, int N, int B, int sms = 0);
int fspad_lm_head_tiles(int V);
size_t fspad_feature_sampler_scratch_floats(int rows, int H, int I);
cudaError_t fspad_launch_feature_sampler(fspad_ctx *ctx, const fspad_bf16 *f, const fspad_bf16 *e, const fspad_bf16 *wup,
                                         const fspad_bf16 *wgate, const fspad_bf16 *wdown, int R, int H, int I,
                                         fspad_bf16 *inter, fspad_bf16 *eta, float *scratch, cudaStream_t st);
FspadStatsGeom fspad_lm_head_geom(int rows, int V, bool vec, int slots);
// LM head over R rows; with walk_geom the merged partials go to the context's scan scratch in that
// geometry (for the acceptance walk), otherwise to row_max / row_sum / row_arg
cudaError_t fspad_launch_lm_head(fspad_ctx *ctx, const fspad_bf16 *hidden, const fspad_bf16 *weight, int H, int R,
                                 int rows_per_seq, const float *temperature, float *logits, const FspadStatsGeom *walk_geom,
                                 float *row_max, double *row_sum, int *row_arg, cudaStream_t st);
int fspad_walk_ctas(fspad_ctx *ctx, int B, int V);   // CTAs of the sampling walk for B sequences
cudaError_t fspad_launch_wait_selftest(fspad_ctx *ctx, int polls, cudaStream_t st);
cudaError_t fspad_launch_attn_umma_split(fspad_ctx *ctx, const fspad_bf16 *q, const fspad_bf16 *kc,
                                         const fspad_bf16 *vc, const fspad_bf16 *tk, const fspad_bf16 *tv,
                                         const int *parent, const int *prefix_len, int N, int B, int n_splits,
                                         float scale_log2, cudaStream_t st, FspadPaged paged);
cudaError_t fspad_launch_kv_append(fspad_ctx *ctx, fspad_bf16 *cache, const fspad_bf16 *tree_kv, const int *path,
                                   const int *n_acc, const int *prefix_len, int N, int B, int *new_len, cudaStream_t st);
cudaError_t fspad_launch_kv_compact_paged(fspad_ctx *ctx, fspad_bf16 *pool, FspadPaged paged, const int *path,
                                          const int *n_acc, const int *prefix_len, int B, int *new_len, cudaStream_t st);
