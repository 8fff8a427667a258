// C ABI of libfspad.so: context management, argument validation and the
// host-buffer entry point.  All arithmetic of the verify step lives in the
// kernel translation units; nothing here computes on the host.
#include <cmath>
#include <cstdlib>
#include <cstring>
#include <new>

#include "common.cuh"

namespace {

inline bool misaligned(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; }

template <typename T>
bool dev_alloc(T **p, size_t count)
{
    *p = nullptr;
    if (count == 0) count = 1;
    return cudaMalloc(reinterpret_cast<void **>(p), count * sizeof(T)) == cudaSuccess;
}

int check_common(const fspad_ctx *ctx, int n_nodes, int batch)
{
    if (!ctx) return FSPAD_ERR_NULL;
    if (n_nodes > FSPAD_MAX_NODES_WIDE || n_nodes > ctx->cfg.max_nodes) return FSPAD_ERR_TREE_TOO_LARGE;
    if (n_nodes < 1 || batch < 0 || batch > ctx->cfg.max_batch) return FSPAD_ERR_SHAPE;
    return FSPAD_OK;
}

}  // namespace

extern "C" {

const char *fspad_strerror(int err)
{
    switch (err) {
    case FSPAD_OK: return "ok";
    case FSPAD_ERR_NULL: return "required pointer is NULL";
    case FSPAD_ERR_ALIGN: return "pointer is not 16-byte aligned";
    case FSPAD_ERR_SHAPE: return "sizes inconsistent with the context";
    case FSPAD_ERR_TREE_TOO_LARGE: return "tree has more nodes than supported";
    case FSPAD_ERR_RANGE: return "value out of range (prefix length, token id, temperature or path)";
    case FSPAD_ERR_CUDA: return "CUDA runtime call failed";
    case FSPAD_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case FSPAD_ERR_BAD_TREE: return "parent[] is not a topologically ordered tree rooted at node 0";
    case FSPAD_ERR_NOMEM: return "allocation failed";
    case FSPAD_ERR_TOO_LARGE: return "size exceeds the fixed capacity of the no-allocation entry point";
    default: return "unknown error";
    }
}

int fspad_create(const fspad_config *cfg, fspad_ctx **out)
{
    if (!out) return FSPAD_ERR_NULL;
    *out = nullptr;
    if (!cfg) return FSPAD_ERR_NULL;
    if (cfg->head_dim != FSPAD_HEAD_DIM || cfg->n_kv_heads < 1 || cfg->n_q_heads < 1 ||
        cfg->n_q_heads % cfg->n_kv_heads != 0 || cfg->vocab < 1 || cfg->n_layers < 1 ||
        cfg->max_len < 1 || cfg->max_batch < 1 || cfg->max_nodes < 1)
        return FSPAD_ERR_SHAPE;
    if (cfg->max_nodes > FSPAD_MAX_NODES_WIDE) return FSPAD_ERR_TREE_TOO_LARGE;
    if (cfg->max_nodes > cfg->max_len) return FSPAD_ERR_RANGE;
    if (!(cfg->softmax_scale >= 0.0f)) return FSPAD_ERR_RANGE;

    fspad_ctx *ctx = new (std::nothrow) fspad_ctx();
    if (!ctx) return FSPAD_ERR_NOMEM;
    std::memset(ctx, 0, sizeof(*ctx));
    ctx->cfg = *cfg;
    ctx->scale = cfg->softmax_scale > 0.0f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
    if (cudaGetDevice(&ctx->device) != cudaSuccess ||
        cudaDeviceGetAttribute(&ctx->sm_count, cudaDevAttrMultiProcessorCount, ctx->device) != cudaSuccess) {
        delete ctx;
        return FSPAD_ERR_CUDA;
    }

    const int G = cfg->n_q_heads / cfg->n_kv_heads;
    const size_t B = (size_t)cfg->max_batch, Nmax = (size_t)cfg->max_nodes;
    // split-KV partials: worst case over every (n_nodes, batch) a call may pass
    size_t part_rows = 0;
    int max_splits = 1;
    for (int n = 1; n <= cfg->max_nodes; ++n)
        for (int b = 1; b <= cfg->max_batch; ++b) {
            const int s = fspad_attn_umma_splits(ctx, n, b);
            const size_t rows = (size_t)b * cfg->n_kv_heads * s * n * G;
            if (rows > part_rows) part_rows = rows;
            if (s > max_splits) max_splits = s;
        }
    ctx->attn_max_splits = max_splits;
    const size_t rows = B * Nmax;
    ctx->stats_slots = 64;

    bool ok = dev_alloc(&ctx->d_status, 1);
    ok = ok && dev_alloc(&ctx->part_o, part_rows * FSPAD_HEAD_DIM);
    ok = ok && dev_alloc(&ctx->part_ml, part_rows * 2);
    ok = ok && dev_alloc(&ctx->st_part, rows * ctx->stats_slots);
    ok = ok && dev_alloc(&ctx->row_max, rows);
    ok = ok && dev_alloc(&ctx->row_sum, rows);
    ok = ok && dev_alloc(&ctx->row_arg, rows);
    {
        uint2 *dx = nullptr;
        ok = ok && dev_alloc(&dx, B * FSPAD_MAX_FRONTIER * (size_t)fspad_draft_expand_pieces(cfg->vocab) * FSPAD_MAX_FRONTIER);
        ctx->dx_part = dx;
    }
    ok = ok && dev_alloc(&ctx->lm_parts, (size_t)128 * fspad_lm_head_tiles(cfg->vocab));
    ok = ok && cudaStreamCreateWithFlags(&ctx->side, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) == cudaSuccess;
    if (ok) {
        ok = cudaMemset(ctx->d_status, 0, sizeof(int)) == cudaSuccess && cudaDeviceSynchronize() == cudaSuccess;
    }
    if (!ok) {
        fspad_destroy(ctx);
        return FSPAD_ERR_NOMEM;
    }
    *out = ctx;
    return FSPAD_OK;
}

void fspad_destroy(fspad_ctx *ctx)
{
    if (!ctx) return;
    cudaDeviceSynchronize();
    void *ptrs[] = {ctx->lm_parts, ctx->dx_part, ctx->d_status, ctx->part_o, ctx->part_ml, ctx->st_part, ctx->row_max, ctx->row_sum, ctx->row_arg, ctx->h_q, ctx->h_tk,
                    ctx->h_tv, ctx->h_out, ctx->h_parent, ctx->h_prefix, ctx->h_tokens, ctx->h_path,
                    ctx->h_nacc, ctx->h_bonus, ctx->h_newlen, ctx->h_logits, ctx->h_draft, ctx->h_temp,
                    ctx->h_unif};
    for (void *p : ptrs)
        if (p) cudaFree(p);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->side) cudaStreamDestroy(ctx->side);
    delete ctx;
}

int fspad_status(fspad_ctx *ctx, void *stream)
{
    if (!ctx) return FSPAD_ERR_NULL;
    cudaStream_t st = fspad_stream(stream);
    int h = 0;
    if (cudaMemcpyAsync(&h, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess)
        return FSPAD_ERR_CUDA;
    if (h != 0) {
        if (cudaMemsetAsync(ctx->d_status, 0, sizeof(int), st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess)
            return FSPAD_ERR_CUDA;
    }
    return h;
}

long long fspad_launch_count(const fspad_ctx *ctx) { return ctx ? ctx->launches : 0; }

int fspad_selftest_wait_timeout(fspad_ctx *ctx, int polls, void *stream)
{
    if (!ctx) return FSPAD_ERR_NULL;
    if (polls < 1 || polls > 4096) return FSPAD_ERR_RANGE;
    return fspad_launch_wait_selftest(ctx, polls, fspad_stream(stream)) == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_tree_attn(fspad_ctx *ctx, const fspad_bf16 *q, const fspad_bf16 *k_cache,
                    const fspad_bf16 *v_cache, const fspad_bf16 *tree_k, const fspad_bf16 *tree_v,
                    const int32_t *parent, const int32_t *prefix_len, int n_nodes, int batch,
                    fspad_bf16 *out, void *stream)
{
    int rc = check_common(ctx, n_nodes, batch);
    if (rc) return rc;
    if (!q || !k_cache || !v_cache || !parent || !prefix_len || !out) return FSPAD_ERR_NULL;
    if ((tree_k == nullptr) != (tree_v == nullptr)) return FSPAD_ERR_NULL;
    if (misaligned(q) || misaligned(k_cache) || misaligned(v_cache) || misaligned(tree_k) ||
        misaligned(tree_v) || misaligned(out))
        return FSPAD_ERR_ALIGN;
    if (n_nodes > ctx->cfg.max_len) return FSPAD_ERR_RANGE;
    if (batch == 0) return FSPAD_OK;
    cudaError_t e = fspad_launch_tree_attn(ctx, q, k_cache, v_cache, tree_k, tree_v, parent, prefix_len,
                                           n_nodes, batch, out, fspad_stream(stream));
    return e == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_accept_stats(fspad_ctx *ctx, const float *logits, const float *temperature, int rows,
                       int rows_per_seq, float *row_max, double *row_sum, int32_t *row_arg,
                       void *stream)
{
    if (!ctx) return FSPAD_ERR_NULL;
    const bool scan_only = !row_max && !row_sum && !row_arg;
    if (!logits || (!scan_only && (!row_max || !row_sum || !row_arg))) return FSPAD_ERR_NULL;
    if (rows < 0 || rows_per_seq < 1 || rows > ctx->cfg.max_batch * ctx->cfg.max_nodes)
        return FSPAD_ERR_SHAPE;
    if (rows == 0) return FSPAD_OK;
    if (scan_only) {
        FspadStatsGeom geom;
        return fspad_launch_stats_partials(ctx, logits, temperature, rows, rows_per_seq, ctx->cfg.vocab, &geom,
                                           fspad_stream(stream)) == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
    }
    cudaError_t e = fspad_launch_accept_stats(ctx, logits, temperature, rows, rows_per_seq, ctx->cfg.vocab,
                                              row_max, row_sum, row_arg, fspad_stream(stream));
    return e == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_tree_accept(fspad_ctx *ctx, const float *target_logits, const float *draft_probs,
                      const int32_t *draft_tokens, const int32_t *parent, const float *temperature,
                      const float *uniforms, int n_nodes, int batch, int32_t *accepted_path,
                      int32_t *n_accepted, int32_t *bonus_token, void *stream)
{
    int rc = check_common(ctx, n_nodes, batch);
    if (rc) return rc;
    if (!target_logits || !draft_tokens || !parent || !temperature || !accepted_path || !n_accepted ||
        !bonus_token)
        return FSPAD_ERR_NULL;
    if ((draft_probs == nullptr) != (uniforms == nullptr)) return FSPAD_ERR_NULL;
    if (misaligned(target_logits) || misaligned(draft_probs)) return FSPAD_ERR_ALIGN;
    if (batch == 0) return FSPAD_OK;
    cudaStream_t st = fspad_stream(stream);
    FspadStatsGeom geom;
    cudaError_t e = fspad_launch_stats_partials(ctx, target_logits, temperature, batch * n_nodes, n_nodes,
                                                ctx->cfg.vocab, &geom, st);
    if (e != cudaSuccess) return FSPAD_ERR_CUDA;
    e = fspad_launch_accept_walk(ctx, target_logits, draft_probs, draft_tokens, parent, temperature,
                                 uniforms, geom, n_nodes, batch, ctx->cfg.vocab, accepted_path, n_accepted,
                                 bonus_token, st);
    return e == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_lm_head_stats(fspad_ctx *ctx, const fspad_bf16 *hidden, const fspad_bf16 *lm_head, int hidden_dim, int rows,
                        int rows_per_seq, const float *temperature, float *logits_out, float *row_max, double *row_sum,
                        int32_t *row_arg, void *stream)
{
    if (!ctx) return FSPAD_ERR_NULL;
    if (!hidden || !lm_head || !row_max || !row_sum || !row_arg) return FSPAD_ERR_NULL;
    if (misaligned(hidden) || misaligned(lm_head) || misaligned(logits_out)) return FSPAD_ERR_ALIGN;
    if (hidden_dim < 8 || hidden_dim % 8 != 0 || rows < 0 || rows_per_seq < 1 ||
        rows > ctx->cfg.max_batch * ctx->cfg.max_nodes)
        return FSPAD_ERR_SHAPE;
    if (rows == 0) return FSPAD_OK;
    return fspad_launch_lm_head(ctx, hidden, lm_head, hidden_dim, rows, rows_per_seq, temperature, logits_out, nullptr,
                                row_max, row_sum, row_arg, fspad_stream(stream)) == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_lm_head_accept(fspad_ctx *ctx, const fspad_bf16 *hidden, const fspad_bf16 *lm_head, int hidden_dim,
                         const float *draft_probs, const int32_t *draft_tokens, const int32_t *parent,
                         const float *temperature, const float *uniforms, int n_nodes, int batch, float *logits,
                         int32_t *accepted_path, int32_t *n_accepted, int32_t *bonus_token, void *stream)
{
    int rc = check_common(ctx, n_nodes, batch);
    if (rc) return rc;
    if (!hidden || !lm_head || !draft_tokens || !parent || !temperature || !accepted_path || !n_accepted || !bonus_token)
        return FSPAD_ERR_NULL;
    if ((draft_probs == nullptr) != (uniforms == nullptr)) return FSPAD_ERR_NULL;
    if (draft_probs != nullptr && logits == nullptr) return FSPAD_ERR_NULL;     // the sampling walk reads logits rows
    if (misaligned(hidden) || misaligned(lm_head) || misaligned(logits) || misaligned(draft_probs)) return FSPAD_ERR_ALIGN;
    if (hidden_dim < 8 || hidden_dim % 8 != 0) return FSPAD_ERR_SHAPE;
    if (batch == 0) return FSPAD_OK;
    cudaStream_t st = fspad_stream(stream);
    const int V = ctx->cfg.vocab, rows = batch * n_nodes;
    const bool vec = (V % 4 == 0);          // logits and draft rows are 16-byte aligned (checked above)
    const FspadStatsGeom geom = fspad_lm_head_geom(rows, V, vec, ctx->stats_slots);
    if (fspad_launch_lm_head(ctx, hidden, lm_head, hidden_dim, rows, n_nodes, temperature, logits, &geom, nullptr, nullptr,
                             nullptr, st) != cudaSuccess)
        return FSPAD_ERR_CUDA;
    // a greedy walk needs only the partials; logits may be NULL then, and the walk never reads them
    return fspad_launch_accept_walk(ctx, logits, draft_probs, draft_tokens, parent, temperature, uniforms, geom, n_nodes,
                                    batch, V, accepted_path, n_accepted, bonus_token, st) == cudaSuccess
               ? FSPAD_OK : FSPAD_ERR_CUDA;
}

size_t fspad_feature_sampler_workspace_bytes(int rows, int hidden_dim, int inter_dim)
{
    if (rows < 1 || hidden_dim < 1 || inter_dim < 1) return 0;
    return fspad_feature_sampler_scratch_floats(rows, hidden_dim, inter_dim) * sizeof(float);
}

int fspad_feature_sampler(fspad_ctx *ctx, const fspad_bf16 *f, const fspad_bf16 *e, const fspad_bf16 *w_up,
                          const fspad_bf16 *w_gate, const fspad_bf16 *w_down, int rows, int hidden_dim, int inter_dim,
                          fspad_bf16 *inter, fspad_bf16 *eta, void *workspace, size_t workspace_bytes, void *stream)
{
    if (!ctx) return FSPAD_ERR_NULL;
    if (!f || !e || !w_up || !w_gate || !w_down || !inter || !eta || !workspace) return FSPAD_ERR_NULL;
    if (misaligned(f) || misaligned(e) || misaligned(w_up) || misaligned(w_gate) || misaligned(w_down) || misaligned(inter) ||
        misaligned(eta) || misaligned(workspace))
        return FSPAD_ERR_ALIGN;
    if (rows < 0 || rows > 128 || hidden_dim < 8 || hidden_dim % 8 != 0 || inter_dim < 8 || inter_dim % 8 != 0)
        return FSPAD_ERR_SHAPE;
    if (rows == 0) return FSPAD_OK;
    if (workspace_bytes < fspad_feature_sampler_workspace_bytes(rows, hidden_dim, inter_dim)) return FSPAD_ERR_RANGE;
    return fspad_launch_feature_sampler(ctx, f, e, w_up, w_gate, w_down, rows, hidden_dim, inter_dim, inter, eta,
                                        static_cast<float *>(workspace), fspad_stream(stream)) == cudaSuccess
               ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_tree_attn_paged(fspad_ctx *ctx, const fspad_bf16 *q, const fspad_bf16 *k_pool, const fspad_bf16 *v_pool,
                          const int32_t *block_table, int blocks_per_seq, int n_blocks, const fspad_bf16 *tree_k,
                          const fspad_bf16 *tree_v, const int32_t *parent, const int32_t *prefix_len, int n_nodes,
                          int batch, fspad_bf16 *out, void *stream)
{
    int rc = check_common(ctx, n_nodes, batch);
    if (rc) return rc;
    if (!q || !k_pool || !v_pool || !block_table || !parent || !prefix_len || !out) return FSPAD_ERR_NULL;
    if ((tree_k == nullptr) != (tree_v == nullptr)) return FSPAD_ERR_NULL;
    if (misaligned(q) || misaligned(k_pool) || misaligned(v_pool) || misaligned(tree_k) || misaligned(tree_v) || misaligned(out))
        return FSPAD_ERR_ALIGN;
    if (blocks_per_seq < 1 || n_blocks < 1 || (long long)blocks_per_seq * 128 < n_nodes) return FSPAD_ERR_SHAPE;
    if (batch == 0) return FSPAD_OK;
    // a CTA keeps the blocks of its chunks in shared memory: at most 128 of them
    const int splits = fspad_attn_umma_splits(ctx, n_nodes, batch);
    if ((blocks_per_seq + splits - 1) / splits > 128) return FSPAD_ERR_TOO_LARGE;
    const FspadPaged pg{block_table, blocks_per_seq, n_blocks};
    return fspad_launch_tree_attn(ctx, q, k_pool, v_pool, tree_k, tree_v, parent, prefix_len, n_nodes, batch, out,
                                  fspad_stream(stream), 0, pg) == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_kv_compact_paged(fspad_ctx *ctx, fspad_bf16 *pool, const int32_t *block_table, int blocks_per_seq, int n_blocks,
                           const int32_t *accepted_path, const int32_t *n_accepted, const int32_t *prefix_len, int batch,
                           int32_t *new_len, void *stream)
{
    if (!ctx) return FSPAD_ERR_NULL;
    if (!pool || !block_table || !accepted_path || !n_accepted || !prefix_len) return FSPAD_ERR_NULL;
    if (misaligned(pool)) return FSPAD_ERR_ALIGN;
    if (batch < 0 || batch > ctx->cfg.max_batch || blocks_per_seq < 1 || n_blocks < 1) return FSPAD_ERR_SHAPE;
    if (batch == 0) return FSPAD_OK;
    const FspadPaged pg{block_table, blocks_per_seq, n_blocks};
    return fspad_launch_kv_compact_paged(ctx, pool, pg, accepted_path, n_accepted, prefix_len, batch, new_len,
                                         fspad_stream(stream)) == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_kv_compact(fspad_ctx *ctx, fspad_bf16 *cache, const int32_t *accepted_path,
                     const int32_t *n_accepted, const int32_t *prefix_len, int batch,
                     int32_t *new_len, void *stream)
{
    if (!ctx) return FSPAD_ERR_NULL;
    if (!cache || !accepted_path || !n_accepted || !prefix_len) return FSPAD_ERR_NULL;
    if (misaligned(cache)) return FSPAD_ERR_ALIGN;
    if (batch < 0 || batch > ctx->cfg.max_batch) return FSPAD_ERR_SHAPE;
    if (batch == 0) return FSPAD_OK;
    cudaError_t e = fspad_launch_kv_compact(ctx, cache, accepted_path, n_accepted, prefix_len, batch,
                                            new_len, fspad_stream(stream));
    return e == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_kv_append(fspad_ctx *ctx, fspad_bf16 *cache, const fspad_bf16 *tree_kv, const int32_t *accepted_path,
                    const int32_t *n_accepted, const int32_t *prefix_len, int n_nodes, int batch, int32_t *new_len,
                    void *stream)
{
    int rc = check_common(ctx, n_nodes, batch);
    if (rc) return rc;
    if (!cache || !tree_kv || !accepted_path || !n_accepted || !prefix_len) return FSPAD_ERR_NULL;
    if (misaligned(cache) || misaligned(tree_kv)) return FSPAD_ERR_ALIGN;
    if (batch == 0) return FSPAD_OK;
    cudaError_t e = fspad_launch_kv_append(ctx, cache, tree_kv, accepted_path, n_accepted, prefix_len, n_nodes, batch,
                                           new_len, fspad_stream(stream));
    return e == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_tree_build(fspad_ctx *ctx, const int32_t *cand_parent, const int32_t *cand_token,
                     const float *cand_logp, const int32_t *root_token, int n_cand, int n_nodes, int batch,
                     int32_t *parent_out, int32_t *token_out, int32_t *cand_out, uint64_t *anc_out,
                     int32_t *n_out, void *stream)
{
    int rc = check_common(ctx, n_nodes, batch);
    if (rc) return rc;
    if (!cand_parent || !cand_token || !cand_logp || !root_token || !parent_out || !token_out || !cand_out || !n_out)
        return FSPAD_ERR_NULL;
    if (n_nodes > FSPAD_MAX_NODES) return FSPAD_ERR_TREE_TOO_LARGE;      // the builder's masks are one word per node
    if (n_cand < 1 || n_cand > FSPAD_MAX_CANDIDATES) return FSPAD_ERR_SHAPE;
    if (batch == 0) return FSPAD_OK;
    cudaError_t e = fspad_launch_tree_build(ctx, cand_parent, cand_token, cand_logp, root_token, n_cand, n_nodes,
                                            batch, parent_out, token_out, cand_out,
                                            reinterpret_cast<unsigned long long *>(anc_out), n_out, fspad_stream(stream));
    return e == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_draft_expand(fspad_ctx *ctx, const float *logprobs, const float *frontier_logp,
                       const int32_t *frontier_cand, int n_frontier, int top_k, int width, int base, int n_cand_cap,
                       int batch, int32_t *cand_parent, int32_t *cand_token, float *cand_logp, int32_t *next_cand,
                       float *next_logp, void *stream)
{
    if (!ctx) return FSPAD_ERR_NULL;
    if (!logprobs || !frontier_logp || !frontier_cand || !cand_parent || !cand_token || !cand_logp || !next_cand ||
        !next_logp)
        return FSPAD_ERR_NULL;
    if (batch < 0 || batch > ctx->cfg.max_batch) return FSPAD_ERR_SHAPE;
    if (n_frontier < 1 || n_frontier > FSPAD_MAX_FRONTIER || top_k < 1 || top_k > FSPAD_MAX_FRONTIER ||
        top_k > ctx->cfg.vocab)
        return FSPAD_ERR_SHAPE;
    if (width < 1 || width > n_frontier * top_k || base < 0 || base + n_frontier * top_k > n_cand_cap)
        return FSPAD_ERR_SHAPE;
    if ((long long)fspad_draft_expand_pieces(ctx->cfg.vocab) * top_k > FSPAD_MAX_CANDIDATES) return FSPAD_ERR_TOO_LARGE;
    if (batch == 0) return FSPAD_OK;
    cudaError_t e = fspad_launch_draft_expand(ctx, logprobs, frontier_logp, frontier_cand, n_frontier, top_k, width,
                                              base, n_cand_cap, batch, cand_parent, cand_token, cand_logp, next_cand,
                                              next_logp, fspad_stream(stream));
    return e == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_verify_step(fspad_ctx *ctx, fspad_bf16 *cache, int attn_layer, const fspad_bf16 *q,
                      const fspad_bf16 *tree_k, const fspad_bf16 *tree_v, const int32_t *parent,
                      const int32_t *prefix_len, const float *target_logits, const float *draft_probs,
                      const int32_t *draft_tokens, const float *temperature, const float *uniforms,
                      int n_nodes, int batch, fspad_bf16 *attn_out, int32_t *accepted_path,
                      int32_t *n_accepted, int32_t *bonus_token, int32_t *new_len, void *stream)
{
    int rc = check_common(ctx, n_nodes, batch);
    if (rc) return rc;
    if (!cache || !q || !parent || !prefix_len || !target_logits || !draft_tokens || !temperature || !attn_out ||
        !accepted_path || !n_accepted || !bonus_token)
        return FSPAD_ERR_NULL;
    if ((tree_k == nullptr) != (tree_v == nullptr)) return FSPAD_ERR_NULL;
    if ((draft_probs == nullptr) != (uniforms == nullptr)) return FSPAD_ERR_NULL;
    if (misaligned(cache) || misaligned(q) || misaligned(tree_k) || misaligned(tree_v) || misaligned(attn_out) ||
        misaligned(target_logits) || misaligned(draft_probs))
        return FSPAD_ERR_ALIGN;
    if (attn_layer < 0 || attn_layer >= ctx->cfg.n_layers) return FSPAD_ERR_SHAPE;
    if (n_nodes > ctx->cfg.max_len) return FSPAD_ERR_RANGE;
    if (batch == 0) return FSPAD_OK;
    const fspad_config &c = ctx->cfg;
    cudaStream_t st = fspad_stream(stream);
    const size_t plane = (size_t)batch * c.n_kv_heads * (size_t)c.max_len * FSPAD_HEAD_DIM;
    const fspad_bf16 *kc = cache + (size_t)attn_layer * 2 * plane, *vc = kc + plane;

    // Which of the two goes first.  The acceptance is a streaming scan over every SM followed by a walk
    // that one cluster per sampling sequence carries out; the attention is one CTA per SM.  When the
    // attention's CTAs leave a good part of the SMs free, both start at once and the acceptance lives on
    // the free SMs.  Otherwise the scan goes first on all SMs and the attention is forked behind it, sized
    // to leave the walk's SMs alone, so that the walk (the longer chain) and the attention run side by side.
    const int sms = ctx->sm_count;
    const int G = c.n_q_heads / c.n_kv_heads;
    const long long attn_ctas = (long long)batch * c.n_kv_heads * ((n_nodes * G + 127) / 128) *
                                fspad_attn_umma_splits(ctx, n_nodes, batch);
    const bool may_sample = draft_probs != nullptr;
    const bool scan_first = may_sample && sms - attn_ctas < sms / 4;
    int attn_sms = 0;
    if (scan_first) {
        const int walk = fspad_walk_ctas(ctx, batch, c.vocab);
        attn_sms = sms - (walk < sms / 2 ? walk : sms / 2);
    }
    cudaError_t ce = cudaSuccess;
    FspadStatsGeom geom;
    const int rows = batch * n_nodes;
    if (scan_first)
        ce = fspad_launch_stats_partials(ctx, target_logits, temperature, rows, n_nodes, c.vocab, &geom, st);
    // fork: the attention of this step on the context's second stream
    if (ce != cudaSuccess || cudaEventRecord(ctx->ev_fork, st) != cudaSuccess ||
        cudaStreamWaitEvent(ctx->side, ctx->ev_fork, 0) != cudaSuccess)
        return FSPAD_ERR_CUDA;
    int rc_attn = FSPAD_OK;
    if (!scan_first) {
        // An all-greedy acceptance is a scan and a one-CTA walk: beside an attention that holds most SMs the
        // scan's CTAs only get going when the attention's leave.  Where the context is short enough for the
        // attention to stay short on half the SMs (at most 8 chunks per CTA by the context's max_len), it
        // gets half and the two really run side by side (17.2 against 20.5 us on the 26-node greedy workload).
        int both_sms = 0;
        if (!may_sample && attn_ctas > sms / 2) {
            const int s_half = fspad_attn_umma_splits(ctx, n_nodes, batch, sms / 2);
            const int max_chunks = (c.max_len + 127) / 128;
            if ((max_chunks + s_half - 1) / s_half <= 8) both_sms = sms / 2;
        }
        rc_attn = fspad_launch_tree_attn(ctx, q, kc, vc, tree_k, tree_v, parent, prefix_len, n_nodes, batch, attn_out,
                                         ctx->side, both_sms) == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
        // Here the scan is launched as a plain dependent: as a programmatic dependent of the previous
        // step's last kernel it was seen to hold the forked attention back behind the whole acceptance
        // (steps replayed from one CUDA graph: 72.5 us per step against 48.8 on the 52-head shape).
        // Where the acceptance is the longer chain (a sampling walk follows, or the attention is the short
        // one above), the scan is cut for the SMs the attention leaves free - one wave of two CTAs per SM
        // there: cut for the whole chip its CTAs queue for those few SMs in several waves, each with a
        // launch's fixed cost (45.5 -> 41.2 us on the 52-head sampling workload, 17.1 -> 14.7 us on the
        // 26-node greedy one).  Under a long attention with a greedy walk the short-lived CTAs of the
        // full-size scan are the better neighbours (37.6 against 39.0 us): an attention CTA that finds
        // its SM taken waits for a scan CTA's whole life.
        int scan_sms = 0;
        if (may_sample || both_sms > 0) {
            const long long attn_now = (long long)batch * c.n_kv_heads * ((n_nodes * G + 127) / 128) *
                                       fspad_attn_umma_splits(ctx, n_nodes, batch, both_sms);
            scan_sms = sms - (int)(attn_now < sms ? attn_now : sms);
            if (scan_sms < sms / 8) scan_sms = sms / 8;
        }
        ce = fspad_launch_stats_partials(ctx, target_logits, temperature, rows, n_nodes, c.vocab, &geom, st, false, scan_sms);
    }
    // With the tree rows given apart from the cache the compaction depends on the walk alone, and when the
    // sequence's slices are few (one warp each among the 16 x 32 warps of a sampling walk's cluster; an
    // all-greedy walk is a single small CTA and keeps the kernel) the walk makes the moves itself at its
    // end: one dependent launch less on the step's longest chain.
    const bool aliased = tree_k == nullptr;      // attention reads the cache rows that compaction rewrites
    const bool walk_compacts = !aliased && may_sample && c.n_layers * 2 * c.n_kv_heads <= 64;
    FspadWalkCompact kv;
    if (walk_compacts) { kv.cache = cache; kv.prefix_len = prefix_len; kv.new_len = new_len; }
    if (ce == cudaSuccess)
        ce = fspad_launch_accept_walk(ctx, target_logits, draft_probs, draft_tokens, parent, temperature, uniforms, geom,
                                      n_nodes, batch, c.vocab, accepted_path, n_accepted, bonus_token, st, kv);
    rc = ce == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
    if (scan_first) {
        // When the walk's clusters need more than one wave, merge CTAs that sit resident waiting for the
        // attention would keep the later clusters off their SMs (244 against 224 us on the ragged batch):
        // the merge kernel is then a plain dependent.
        const bool walk_one_wave = fspad_walk_ctas(ctx, batch, c.vocab) <= sms / 2;   // the attention was sized to leave that many free
        rc_attn = fspad_launch_tree_attn(ctx, q, kc, vc, tree_k, tree_v, parent, prefix_len, n_nodes, batch, attn_out,
                                         ctx->side, attn_sms, FspadPaged{nullptr, 0, 0}, walk_one_wave) == cudaSuccess
                      ? FSPAD_OK : FSPAD_ERR_CUDA;
    }
    // the join is queued whatever happened in between, so that a capture of `stream` never ends
    // with the second stream left unjoined
    const bool ev_ok = cudaEventRecord(ctx->ev_join, ctx->side) == cudaSuccess;
    bool joined = false;
    if (aliased) joined = cudaStreamWaitEvent(st, ctx->ev_join, 0) == cudaSuccess;
    if (rc == FSPAD_OK && rc_attn == FSPAD_OK && !walk_compacts) {
        // behind a join the compaction has two predecessors, so it is launched as a plain dependent
        cudaError_t e = fspad_launch_kv_compact(ctx, cache, accepted_path, n_accepted, prefix_len, batch, new_len, st,
                                                !aliased);
        if (e != cudaSuccess) rc = FSPAD_ERR_CUDA;
    }
    if (!aliased) joined = cudaStreamWaitEvent(st, ctx->ev_join, 0) == cudaSuccess;
    if (rc_attn) return rc_attn;
    if (rc) return rc;
    return (ev_ok && joined) ? FSPAD_OK : FSPAD_ERR_CUDA;
}

int fspad_verify_step_host(fspad_ctx *ctx, fspad_bf16 *cache, const fspad_bf16 *q,
                           const fspad_bf16 *tree_k, const fspad_bf16 *tree_v, const int32_t *parent,
                           const int32_t *prefix_len, const float *target_logits,
                           const float *draft_probs, const int32_t *draft_tokens,
                           const float *temperature, const float *uniforms, int n_nodes, int batch,
                           fspad_bf16 *attn_out, int32_t *accepted_path, int32_t *n_accepted,
                           int32_t *bonus_token, int32_t *new_len, void *stream)
{
    int rc = check_common(ctx, n_nodes, batch);
    if (rc) return rc;
    if (!cache || !q || !tree_k || !tree_v || !parent || !prefix_len || !target_logits || !draft_tokens ||
        !temperature || !attn_out || !accepted_path || !n_accepted || !bonus_token || !new_len)
        return FSPAD_ERR_NULL;
    if ((draft_probs == nullptr) != (uniforms == nullptr)) return FSPAD_ERR_NULL;
    if (misaligned(cache)) return FSPAD_ERR_ALIGN;
    if (batch == 0) return FSPAD_OK;
    const fspad_config &c = ctx->cfg;
    cudaStream_t st = fspad_stream(stream);

    // staging buffers are created by the first call, sized for the context's maxima; a failed
    // attempt frees what it got, so that a later call starts over instead of using half a set
    if (!ctx->h_ready) {
        const size_t B = (size_t)c.max_batch, N = (size_t)c.max_nodes;
        bool ok = dev_alloc(&ctx->h_q, B * N * c.n_q_heads * FSPAD_HEAD_DIM);
        ok = ok && dev_alloc(&ctx->h_out, B * N * c.n_q_heads * FSPAD_HEAD_DIM);
        ok = ok && dev_alloc(&ctx->h_tk, B * c.n_kv_heads * N * FSPAD_HEAD_DIM);
        ok = ok && dev_alloc(&ctx->h_tv, B * c.n_kv_heads * N * FSPAD_HEAD_DIM);
        ok = ok && dev_alloc(&ctx->h_parent, B * N) && dev_alloc(&ctx->h_tokens, B * N);
        ok = ok && dev_alloc(&ctx->h_prefix, B) && dev_alloc(&ctx->h_nacc, B);
        ok = ok && dev_alloc(&ctx->h_bonus, B) && dev_alloc(&ctx->h_newlen, B);
        ok = ok && dev_alloc(&ctx->h_path, B * N) && dev_alloc(&ctx->h_temp, B);
        ok = ok && dev_alloc(&ctx->h_unif, B * (N + 1));
        ok = ok && dev_alloc(&ctx->h_logits, B * N * c.vocab);
        ok = ok && dev_alloc(&ctx->h_draft, B * N * c.vocab);
        if (!ok) {
            void **slots[] = {(void **)&ctx->h_q, (void **)&ctx->h_out, (void **)&ctx->h_tk, (void **)&ctx->h_tv,
                              (void **)&ctx->h_parent, (void **)&ctx->h_tokens, (void **)&ctx->h_prefix,
                              (void **)&ctx->h_nacc, (void **)&ctx->h_bonus, (void **)&ctx->h_newlen,
                              (void **)&ctx->h_path, (void **)&ctx->h_temp, (void **)&ctx->h_unif,
                              (void **)&ctx->h_logits, (void **)&ctx->h_draft};
            for (void **sl : slots) {
                if (*sl) cudaFree(*sl);
                *sl = nullptr;
            }
            (void)cudaGetLastError();
            return FSPAD_ERR_NOMEM;
        }
        ctx->h_ready = 1;
    }
    const size_t B = (size_t)batch, N = (size_t)n_nodes;
    const size_t q_bytes = B * N * c.n_q_heads * FSPAD_HEAD_DIM * sizeof(fspad_bf16);
    const size_t t_bytes = B * c.n_kv_heads * N * FSPAD_HEAD_DIM * sizeof(fspad_bf16);
    const size_t lg_bytes = B * N * c.vocab * sizeof(float);
    bool ok = true;
    auto h2d = [&](void *dst, const void *src, size_t bytes) {
        ok = ok && cudaMemcpyAsync(dst, src, bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
    };
    auto d2h = [&](void *dst, const void *src, size_t bytes) {
        ok = ok && cudaMemcpyAsync(dst, src, bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
    };
    h2d(ctx->h_q, q, q_bytes);
    h2d(ctx->h_tk, tree_k, t_bytes);
    h2d(ctx->h_tv, tree_v, t_bytes);
    h2d(ctx->h_parent, parent, B * N * sizeof(int));
    h2d(ctx->h_prefix, prefix_len, B * sizeof(int));
    h2d(ctx->h_tokens, draft_tokens, B * N * sizeof(int));
    h2d(ctx->h_temp, temperature, B * sizeof(float));
    h2d(ctx->h_logits, target_logits, lg_bytes);
    if (draft_probs) {
        h2d(ctx->h_draft, draft_probs, lg_bytes);
        h2d(ctx->h_unif, uniforms, B * (N + 1) * sizeof(float));
    }
    if (!ok) return FSPAD_ERR_CUDA;

    // the tree rows go into cache rows L_b .. of layer 0 (K at [0][0], V at [0][1]); the step then
    // takes them from there
    if (fspad_launch_tree_scatter(ctx, cache, ctx->h_tk, ctx->h_tv, ctx->h_prefix, n_nodes, batch, st) !=
        cudaSuccess)
        return FSPAD_ERR_CUDA;
    rc = fspad_verify_step(ctx, cache, 0, ctx->h_q, nullptr, nullptr, ctx->h_parent, ctx->h_prefix, ctx->h_logits,
                           draft_probs ? ctx->h_draft : nullptr, ctx->h_tokens, ctx->h_temp,
                           draft_probs ? ctx->h_unif : nullptr, n_nodes, batch, ctx->h_out, ctx->h_path, ctx->h_nacc,
                           ctx->h_bonus, ctx->h_newlen, stream);
    if (rc) return rc;

    d2h(attn_out, ctx->h_out, q_bytes);
    // the device path array has max_nodes entries per sequence, and so has the host one
    d2h(accepted_path, ctx->h_path, B * (size_t)c.max_nodes * sizeof(int));
    d2h(n_accepted, ctx->h_nacc, B * sizeof(int));
    d2h(bonus_token, ctx->h_bonus, B * sizeof(int));
    d2h(new_len, ctx->h_newlen, B * sizeof(int));
    if (!ok) return FSPAD_ERR_CUDA;
    return fspad_status(ctx, stream);
}

}  // extern "C"
