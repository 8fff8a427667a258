/*
 * fp64 CPU oracle for the tree-verification step of lossless speculative
 * decoding (paper Section "Preliminaries": flattened token tree + attention
 * mask -> one target forward -> strict comparison, mismatching tokens and
 * their descendants discarded; Section "Experiments": temperature 0 and 1,
 * acceptance conditions never relaxed).
 *
 * TEST INFRASTRUCTURE ONLY. This file defines what the CUDA library must
 * compute and is deliberately slow and plain: scalar loops in double
 * precision, no blocking, no fusion. It shares no code with the CUDA path.
 * Only the tests, the smoke check and the benchmark's CPU-baseline leg may
 * call it; the product never does.
 *
 * Parity pins (tests/test_oracle_*.py): chain tree == dense causal
 * attention, per-path brute force, greedy == naive per-path comparison,
 * exact emitted-token distribution of the rejection sampler at vocab 8,
 * hand-worked decision traces, brute-force compaction; tree builder
 * (tests/test_oracle_tree_build.py): hand-worked cases, stable library sort,
 * brute force over ancestor-closed subsets, flattened-tree invariants; draft
 * step: hand-worked cases, library sorts plus numpy's own fp32 addition,
 * levels chained into the builder.
 *
 * The only parallelism is an OpenMP loop over independent units (heads,
 * node rows, cache slices); each unit runs the plain definition.
 *
 * Conventions (the paper is silent on them; they are the library's stated
 * reading): node 0 is the root (last emitted token, always accepted,
 * parent[0] = -1); nodes are in topological order (parent[i] < i); children
 * are visited in increasing node index; kv head of query head h is
 * h / (Hq / Hkv); softmax scale is passed in; bf16 inputs are converted to
 * double exactly.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_f64(uint16_t h)
{
    uint32_t u = (uint32_t)h << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------------
 * Tree-masked verify attention ("Preliminaries": the mask built from the
 * token tree makes every token see only what it depends on).
 * Query node i sees the L cached prefix keys and tree key j iff j == i or j
 * is an ancestor of i.  out = softmax(q.k * scale) . v over that set.
 *
 *   q        [B][N][Hq][d]        bf16 bits
 *   k_cache  [B][Hkv][max_len][d] bf16 bits (v_cache alike)
 *   tree_k   [B][Hkv][N][d]       bf16 bits, or NULL: tree rows are cache
 *                                 rows prefix_len[b] .. prefix_len[b]+N-1
 *   out      [B][N][Hq][d]        double
 * ---------------------------------------------------------------------- */
int oracle_tree_attn(const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                     const uint16_t *tree_k, const uint16_t *tree_v, const int32_t *parent,
                     const int32_t *prefix_len, int B, int N, int Hq, int Hkv, int d, int max_len,
                     double scale, double *out)
{
    if (Hkv <= 0 || Hq % Hkv != 0) return -1;
    const int G = Hq / Hkv;
    int bad = 0;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < Hq; ++h) {
            const int g = h / G;
            const int L = prefix_len[b];
            const int32_t *par = parent + (size_t)b * N;
            double *s = (double *)malloc(sizeof(double) * (size_t)(L + N));
            char *vis = (char *)malloc((size_t)N);
            if (!s || !vis) { bad = 1; free(s); free(vis); continue; }
            const uint16_t *kc = k_cache + ((size_t)b * Hkv + g) * (size_t)max_len * d;
            const uint16_t *vc = v_cache + ((size_t)b * Hkv + g) * (size_t)max_len * d;
            const uint16_t *tk = tree_k ? tree_k + ((size_t)b * Hkv + g) * (size_t)N * d
                                        : kc + (size_t)L * d;
            const uint16_t *tv = tree_v ? tree_v + ((size_t)b * Hkv + g) * (size_t)N * d
                                        : vc + (size_t)L * d;
            for (int i = 0; i < N; ++i) {
                const uint16_t *qi = q + (((size_t)b * N + i) * Hq + h) * d;
                memset(vis, 0, (size_t)N);
                for (int a = i; a >= 0; a = par[a]) vis[a] = 1;
                double m = -INFINITY;
                for (int t = 0; t < L + N; ++t) {
                    if (t >= L && !vis[t - L]) { s[t] = -INFINITY; continue; }
                    const uint16_t *kr = t < L ? kc + (size_t)t * d : tk + (size_t)(t - L) * d;
                    double acc = 0.0;
                    for (int c = 0; c < d; ++c) acc += bf16_to_f64(qi[c]) * bf16_to_f64(kr[c]);
                    s[t] = acc * scale;
                    if (s[t] > m) m = s[t];
                }
                double denom = 0.0;
                for (int t = 0; t < L + N; ++t) {
                    s[t] = (s[t] == -INFINITY) ? 0.0 : exp(s[t] - m);
                    denom += s[t];
                }
                double *o = out + (((size_t)b * N + i) * Hq + h) * d;
                for (int c = 0; c < d; ++c) o[c] = 0.0;
                for (int t = 0; t < L + N; ++t) {
                    if (s[t] == 0.0) continue;
                    const uint16_t *vr = t < L ? vc + (size_t)t * d : tv + (size_t)(t - L) * d;
                    for (int c = 0; c < d; ++c) o[c] += s[t] * bf16_to_f64(vr[c]);
                }
                for (int c = 0; c < d; ++c) o[c] /= denom;
            }
            free(s);
            free(vis);
        }
    }
    return bad ? -2 : 0;
}

/* ------------------------------------------------------------------------
 * Per-node vocabulary scan: m = max logit, a = its lowest index,
 * S = sum_j exp((x_j - m) / T)   (T <= 0 is treated as 1 for S).
 *   logits [R][V] fp32 ; row_max, row_sum double [R] ; row_arg int32 [R]
 * ---------------------------------------------------------------------- */
int oracle_row_stats(const float *logits, int R, int V, double T, double *row_max, double *row_sum,
                     int32_t *row_arg)
{
    const double Td = T > 0.0 ? T : 1.0;
#pragma omp parallel for schedule(static)
    for (int r = 0; r < R; ++r) {
        const float *x = logits + (size_t)r * V;
        double m = -INFINITY;
        int a = 0;
        for (int j = 0; j < V; ++j)
            if ((double)x[j] > m) { m = (double)x[j]; a = j; }
        double S = 0.0;
        for (int j = 0; j < V; ++j) S += exp(((double)x[j] - m) / Td);
        row_max[r] = m;
        row_sum[r] = S;
        row_arg[r] = a;
    }
    return 0;
}

/* ------------------------------------------------------------------------
 * Target LM head followed by the per-node vocabulary scan ("Preliminaries":
 * the target's single forward over the flattened tree yields, for every tree
 * node, the distribution the acceptance stage compares the tree with).  The
 * last step of that forward is the product of the final hidden states with the
 * vocabulary matrix; its rows are the logits the scan above is defined on:
 *   z[r][v] = sum_h hidden[r][h] * weight[v][h]          (fp64, index order)
 *   m = max_v z, a = its lowest index, S = sum_v exp((z - m) / T)
 *   hidden [R][H], weight [V][H]: bf16 bit patterns
 *   logits (may be NULL) [R][V] double ; row_max, row_sum double [R] ; row_arg int32 [R]
 *   row_gap (may be NULL) double [R]: m minus the second largest value (ties: 0)
 * ---------------------------------------------------------------------- */
int oracle_lm_head_stats(const uint16_t *hidden, const uint16_t *weight, int R, int H, int V, double T,
                         double *logits, double *row_max, double *row_sum, int32_t *row_arg, double *row_gap)
{
    const double Td = T > 0.0 ? T : 1.0;
    int bad = 0;
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < R; ++r) {
        double *z = (double *)malloc((size_t)V * sizeof(double));
        double *hr = (double *)malloc((size_t)H * sizeof(double));
        if (!z || !hr) {
            bad = 1;
            free(z);
            free(hr);
            continue;
        }
        for (int h = 0; h < H; ++h) hr[h] = bf16_to_f64(hidden[(size_t)r * H + h]);
        for (int v = 0; v < V; ++v) {
            const uint16_t *wv = weight + (size_t)v * H;
            double acc = 0.0;
            for (int h = 0; h < H; ++h) acc += hr[h] * bf16_to_f64(wv[h]);
            z[v] = acc;
        }
        double m = -INFINITY, second = -INFINITY;
        int a = 0;
        for (int v = 0; v < V; ++v) {
            if (z[v] > m) { second = m; m = z[v]; a = v; }
            else if (z[v] > second) second = z[v];
        }
        double S = 0.0;
        for (int v = 0; v < V; ++v) S += exp((z[v] - m) / Td);
        row_max[r] = m;
        row_sum[r] = S;
        row_arg[r] = a;
        if (row_gap) row_gap[r] = m - second;
        if (logits) memcpy(logits + (size_t)r * V, z, (size_t)V * sizeof(double));
        free(z);
        free(hr);
    }
    return bad ? -1 : 0;
}

/* ------------------------------------------------------------------------
 * Feature Sampler forward ("Feature Sampling": three projectors and a sampling
 * operation in the intermediate space).  The Up projector maps the feature f and
 * the Gate projector the token embedding e to intermediate size; the embedding's
 * image is activated by SiLU and multiplied element by element with the
 * feature's image; the Down projector maps the result back to hidden size, where
 * the residual connection the section mentions adds the input feature:
 *   u = Wup f,  g = Wgate e,  s = silu(g) * u,  eta = Wdown s + f      (fp64)
 *   f, e [R][H]; Wup, Wgate [I][H]; Wdown [H][I]: bf16 bit patterns; eta [R][H] double
 *   inter (may be NULL) [R][I] double receives s.
 * ---------------------------------------------------------------------- */
int oracle_feature_sampler(const uint16_t *f, const uint16_t *e, const uint16_t *wup, const uint16_t *wgate,
                           const uint16_t *wdown, int R, int H, int I, double *eta, double *inter)
{
    int bad = 0;
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < R; ++r) {
        double *fr = (double *)malloc((size_t)H * sizeof(double));
        double *er = (double *)malloc((size_t)H * sizeof(double));
        double *s = (double *)malloc((size_t)I * sizeof(double));
        if (!fr || !er || !s) {
            bad = 1;
            free(fr); free(er); free(s);
            continue;
        }
        for (int h = 0; h < H; ++h) {
            fr[h] = bf16_to_f64(f[(size_t)r * H + h]);
            er[h] = bf16_to_f64(e[(size_t)r * H + h]);
        }
        for (int i = 0; i < I; ++i) {
            double u = 0.0, g = 0.0;
            for (int h = 0; h < H; ++h) {
                u += bf16_to_f64(wup[(size_t)i * H + h]) * fr[h];
                g += bf16_to_f64(wgate[(size_t)i * H + h]) * er[h];
            }
            s[i] = g / (1.0 + exp(-g)) * u;
        }
        for (int h = 0; h < H; ++h) {
            double acc = 0.0;
            for (int i = 0; i < I; ++i) acc += bf16_to_f64(wdown[(size_t)h * I + i]) * s[i];
            eta[(size_t)r * H + h] = acc + fr[h];
        }
        if (inter) memcpy(inter + (size_t)r * I, s, (size_t)I * sizeof(double));
        free(fr); free(er); free(s);
    }
    return bad ? -1 : 0;
}

/* Inverse-CDF draw: weights w_j >= 0 summed in index order to Z; the token is
 * the smallest j whose running sum exceeds u*Z; if rounding leaves none, the
 * largest j with w_j > 0.  info (may be NULL) receives
 * {u*Z, lower edge, upper edge, Z, previous positive token, next positive token}. */
static int inverse_cdf(const double *w, int V, double u, double *info)
{
    double Z = 0.0;
    for (int j = 0; j < V; ++j) Z += w[j];
    const double target = u * Z;
    double run = 0.0, lo = 0.0;
    int tok = -1;
    for (int j = 0; j < V; ++j) {
        lo = run;
        run += w[j];
        if (run > target) { tok = j; break; }
    }
    if (tok < 0) {
        for (int j = V - 1; j >= 0; --j)
            if (w[j] > 0.0) { tok = j; break; }
        if (tok < 0) tok = 0;
        lo = run - w[tok];
    }
    if (info) {
        int prev = -1, next = -1;
        for (int j = tok - 1; j >= 0; --j) if (w[j] > 0.0) { prev = j; break; }
        for (int j = tok + 1; j < V; ++j) if (w[j] > 0.0) { next = j; break; }
        info[0] = target; info[1] = lo; info[2] = lo + w[tok]; info[3] = Z;
        info[4] = (double)prev; info[5] = (double)next;
    }
    return tok;
}

/* ------------------------------------------------------------------------
 * Lossless tree acceptance ("Preliminaries": strict comparison, differing
 * tokens and their descendants discarded; "Experiments": T = 0 greedy,
 * T = 1 sampling with unrelaxed acceptance).
 *
 * Per sequence b:
 *   T == 0: from cur = root, accept the first child (index order) whose
 *           token equals argmax of cur's target row (lowest index on ties);
 *           stop when none matches; bonus = argmax of the last node's row.
 *   T  > 0: recursive speculative rejection sampling.  At node cur,
 *           p = softmax(logits[cur] / T), q = draft_probs[cur].  For each
 *           child c in index order with token x and uniform r = uniforms[c]:
 *           accept iff r * q[x] < p[x]; on reject, p <- normalise(max(p - q, 0))
 *           (p kept if that sum is 0), q[x] <- 0, q <- q / sum(q) (kept if 0).
 *           When no child is accepted (or cur is a leaf) the bonus token is
 *           the inverse-CDF draw from the current p with uniforms[N].
 *
 *   target_logits [B][N][V] fp32 ; draft_probs [B][N][V] fp32 (NULL if every T is 0)
 *   draft_tokens, parent [B][N] int32 ; temperature [B] fp32 ; uniforms [B][N+1] fp32
 *   force [B][N] int32 or NULL: 0 reject / 1 accept overrides the test at that child, -1 natural
 *   accepted_path [B][N] int32 (-1 padded) ; n_accepted [B] ; bonus_token [B]
 *   trace_rq, trace_p [B][N] double or NULL: r*q[x] and p[x] at each tested child (NaN if untested)
 *   bonus_info [B][6] double or NULL: see inverse_cdf (greedy: all zero)
 * ---------------------------------------------------------------------- */
int oracle_tree_accept(const float *target_logits, const float *draft_probs,
                       const int32_t *draft_tokens, const int32_t *parent, const float *temperature,
                       const float *uniforms, const int32_t *force, int B, int N, int V,
                       int32_t *accepted_path, int32_t *n_accepted, int32_t *bonus_token,
                       double *trace_rq, double *trace_p, double *bonus_info)
{
    int bad = 0;
    for (int b = 0; b < B; ++b) {
        const float *lg = target_logits + (size_t)b * N * V;
        const int32_t *par = parent + (size_t)b * N;
        const int32_t *tok = draft_tokens + (size_t)b * N;
        const int32_t *frc = force ? force + (size_t)b * N : NULL;
        int32_t *path = accepted_path + (size_t)b * N;
        const double T = (double)temperature[b];
        for (int i = 0; i < N; ++i) path[i] = -1;
        if (trace_rq) for (int i = 0; i < N; ++i) trace_rq[(size_t)b * N + i] = NAN;
        if (trace_p) for (int i = 0; i < N; ++i) trace_p[(size_t)b * N + i] = NAN;
        if (bonus_info) for (int i = 0; i < 6; ++i) bonus_info[(size_t)b * 6 + i] = 0.0;

        /* step: per-node vocabulary scan over all N rows */
        double *rmax = (double *)malloc(sizeof(double) * N);
        double *rsum = (double *)malloc(sizeof(double) * N);
        int32_t *rarg = (int32_t *)malloc(sizeof(int32_t) * N);
        if (!rmax || !rsum || !rarg) { free(rmax); free(rsum); free(rarg); return -2; }
        oracle_row_stats(lg, N, V, T, rmax, rsum, rarg);

        int cur = 0, len = 1;
        path[0] = 0;
        if (!(T > 0.0)) {
            for (;;) {
                int next = -1;
                for (int c = cur + 1; c < N; ++c) {
                    if (par[c] != cur) continue;
                    int take = tok[c] == rarg[cur];
                    if (frc && frc[c] >= 0) take = frc[c];
                    if (take) { next = c; break; }
                }
                if (next < 0) break;
                path[len++] = next;
                cur = next;
            }
            bonus_token[b] = rarg[cur];
        } else {
            if (!draft_probs || !uniforms) { free(rmax); free(rsum); free(rarg); return -3; }
            const float *dp = draft_probs + (size_t)b * N * V;
            const float *un = uniforms + (size_t)b * (N + 1);
            double *p = (double *)malloc(sizeof(double) * V);
            double *qd = (double *)malloc(sizeof(double) * V);
            if (!p || !qd) { bad = 1; free(p); free(qd); free(rmax); free(rsum); free(rarg); break; }
            for (;;) {
                const float *x = lg + (size_t)cur * V;
                for (int j = 0; j < V; ++j) p[j] = exp(((double)x[j] - rmax[cur]) / T) / rsum[cur];
                for (int j = 0; j < V; ++j) qd[j] = (double)dp[(size_t)cur * V + j];
                int next = -1;
                for (int c = cur + 1; c < N; ++c) {
                    if (par[c] != cur) continue;
                    const int xt = tok[c];
                    const double rq = (double)un[c] * qd[xt];
                    if (trace_rq) trace_rq[(size_t)b * N + c] = rq;
                    if (trace_p) trace_p[(size_t)b * N + c] = p[xt];
                    int take = rq < p[xt];
                    if (frc && frc[c] >= 0) take = frc[c];
                    if (take) { next = c; break; }
                    /* residual target distribution */
                    double Z = 0.0;
                    for (int j = 0; j < V; ++j) {
                        double wj = p[j] - qd[j];
                        Z += wj > 0.0 ? wj : 0.0;
                    }
                    if (Z > 0.0)
                        for (int j = 0; j < V; ++j) {
                            double wj = p[j] - qd[j];
                            p[j] = (wj > 0.0 ? wj : 0.0) / Z;
                        }
                    /* draft distribution without the rejected token */
                    qd[xt] = 0.0;
                    double s = 0.0;
                    for (int j = 0; j < V; ++j) s += qd[j];
                    if (s > 0.0)
                        for (int j = 0; j < V; ++j) qd[j] /= s;
                }
                if (next < 0) break;
                path[len++] = next;
                cur = next;
            }
            bonus_token[b] = inverse_cdf(p, V, (double)un[N], bonus_info ? bonus_info + (size_t)b * 6 : NULL);
            free(p);
            free(qd);
        }
        n_accepted[b] = len;
        free(rmax); free(rsum); free(rarg);
    }
    return bad ? -2 : 0;
}

/* ------------------------------------------------------------------------
 * Accepted-path KV compaction ("Preliminaries": rejected tokens are
 * discarded, so only the accepted path's rows stay in the cache).
 * For every layer, K and V, sequence, kv head: row L + path[j] moves to row
 * L + j for j = 0 .. n-1, as if all moves happened at once.  Rows at or after
 * L + n are left untouched.  new_len[b] = L + n.
 *   cache [layers][2][B][Hkv][max_len][d] bf16 bits, in place
 * ---------------------------------------------------------------------- */
int oracle_kv_compact(uint16_t *cache, const int32_t *accepted_path, const int32_t *n_accepted,
                      const int32_t *prefix_len, int n_layers, int B, int Hkv, int max_len, int d,
                      int path_stride, int32_t *new_len)
{
    int bad = 0;
#pragma omp parallel for collapse(2) schedule(static)
    for (int l = 0; l < n_layers; ++l) {
        for (int kv = 0; kv < 2; ++kv) {
            for (int b = 0; b < B; ++b) {
                const int L = prefix_len[b], n = n_accepted[b];
                const int32_t *path = accepted_path + (size_t)b * path_stride;
                uint16_t *tmp = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)(n > 0 ? n : 1) * d);
                if (!tmp) { bad = 1; continue; }
                for (int h = 0; h < Hkv; ++h) {
                    uint16_t *base = cache + ((((size_t)l * 2 + kv) * B + b) * Hkv + h) * (size_t)max_len * d;
                    for (int j = 0; j < n; ++j)
                        memcpy(tmp + (size_t)j * d, base + (size_t)(L + path[j]) * d, sizeof(uint16_t) * d);
                    for (int j = 0; j < n; ++j)
                        memcpy(base + (size_t)(L + j) * d, tmp + (size_t)j * d, sizeof(uint16_t) * d);
                }
                free(tmp);
            }
        }
    }
    if (new_len)
        for (int b = 0; b < B; ++b) new_len[b] = prefix_len[b] + n_accepted[b];
    return bad ? -2 : 0;
}

/* ------------------------------------------------------------------------
 * Cache append of the accepted path ("Preliminaries": of the tree the target
 * ran over, the accepted tokens continue the sequence and the rest is
 * discarded).  The tree's K/V rows of every layer are held outside the cache;
 * only the accepted ones are written, directly behind the prefix:
 *   cache[l][kv][b][h][L_b + j][:] = tree_kv[l][kv][b][h][path[b][j]][:],  j < n_b
 * Nothing else in the cache changes.  new_len[b] = L_b + n_b.
 *   cache   [layers][2][B][Hkv][max_len][d] bf16 bits, in place
 *   tree_kv [layers][2][B][Hkv][N][d] bf16 bits
 * ---------------------------------------------------------------------- */
int oracle_kv_append(uint16_t *cache, const uint16_t *tree_kv, const int32_t *accepted_path,
                     const int32_t *n_accepted, const int32_t *prefix_len, int n_layers, int B, int Hkv,
                     int max_len, int N, int d, int path_stride, int32_t *new_len)
{
    for (int b = 0; b < B; ++b) {
        const int L = prefix_len[b], n = n_accepted[b];
        if (n < 0 || n > N || L < 0 || L + n > max_len) return -1;
        for (int j = 0; j < n; ++j) {
            const int src = accepted_path[(size_t)b * path_stride + j];
            if (src < 0 || src >= N) return -1;
        }
    }
    for (int l = 0; l < n_layers; ++l)
        for (int kv = 0; kv < 2; ++kv)
            for (int b = 0; b < B; ++b)
                for (int h = 0; h < Hkv; ++h) {
                    const size_t slice = (((size_t)l * 2 + kv) * B + b) * Hkv + h;
                    const int L = prefix_len[b], n = n_accepted[b];
                    for (int j = 0; j < n; ++j) {
                        const int src = accepted_path[(size_t)b * path_stride + j];
                        memcpy(cache + (slice * max_len + (size_t)(L + j)) * d, tree_kv + (slice * N + (size_t)src) * d,
                               sizeof(uint16_t) * d);
                    }
                }
    if (new_len)
        for (int b = 0; b < B; ++b) new_len[b] = prefix_len[b] + n_accepted[b];
    return 0;
}

/* -------------------------------------------------------------------------
 * O5  Dynamic token tree, final stage (paper, Section "Preliminaries", last
 * paragraph: every draft step is truncated to its top-k, each token carries
 * the joint probability of its path, and one top-k over all tokens after the
 * draft phase yields a valid tree of bounded size; Section "Performance on
 * Fewer Candidate Tokens" halves both budgets).
 *
 * Input: C candidates per sequence, listed level by level, so that the parent
 * of a candidate has a lower index; cand_parent = -1 for the children of the
 * root; cand_logp = joint log-probability of the path, never larger than the
 * parent's.  The N - 1 candidates with the largest joint probability are kept
 * (equal values: the lower index first, which keeps parents before children).
 * Because the joint probability cannot grow along a path the kept set is
 * closed under "parent of"; an input that violates this is reported (-3).
 * Output: the flattened tree the verification step takes.  Node 0 is the root
 * (root_token); the kept candidates follow ordered by depth and, inside a
 * depth, by candidate index (breadth-first numbering, so parent[i] < i).
 *   parent_out, token_out, cand_out [B][N] (cand_out[0] = -1; entries at and
 *   beyond n_out[b] are -1), n_out[b] = 1 + min(N - 1, C); anc_out [B][N]
 *   (optional): bit j of anc_out[i] set iff node j is node i or one of its
 *   ancestors - the mask under which the target verifies the tree
 *   ("Preliminaries": the mask is updated from the token tree); 0 beyond n_out.
 * Plain selection: one pass per kept node over all candidates.
 * ---------------------------------------------------------------------- */
int oracle_tree_build(const int32_t *cand_parent, const int32_t *cand_token, const float *cand_logp,
                      const int32_t *root_token, int B, int C, int N, int32_t *parent_out,
                      int32_t *token_out, int32_t *cand_out, uint64_t *anc_out, int32_t *n_out)
{
    int rc = 0;
    for (int b = 0; b < B; ++b) {
        const int32_t *cp = cand_parent + (size_t)b * C, *ct = cand_token + (size_t)b * C;
        const float *lp = cand_logp + (size_t)b * C;
        int32_t *po = parent_out + (size_t)b * N, *to = token_out + (size_t)b * N, *co = cand_out + (size_t)b * N;
        char *kept = (char *)calloc((size_t)(C > 0 ? C : 1), 1);
        int *depth = (int *)calloc((size_t)(C > 0 ? C : 1), sizeof(int));
        int *node_of = (int *)malloc(sizeof(int) * (size_t)(C > 0 ? C : 1));
        if (!kept || !depth || !node_of) { free(kept); free(depth); free(node_of); return -2; }
        for (int i = 0; i < N; ++i) { po[i] = -1; to[i] = -1; co[i] = -1; }
        const int want = (N - 1 < C) ? N - 1 : C;
        /* selection: repeatedly take the best candidate not yet kept */
        for (int s = 0; s < want; ++s) {
            int best = -1;
            for (int c = 0; c < C; ++c) {
                if (kept[c]) continue;
                if (best < 0 || lp[c] > lp[best]) best = c;   /* strict: equal values keep the lower index */
            }
            kept[best] = 1;
        }
        /* closure and depths (parents precede children) */
        for (int c = 0; c < C; ++c) {
            node_of[c] = -1;
            if (cp[c] < -1 || cp[c] >= c) { rc = -3; continue; }
            depth[c] = (cp[c] < 0) ? 1 : depth[cp[c]] + 1;
            if (kept[c] && cp[c] >= 0 && !kept[cp[c]]) rc = -3;
        }
        /* breadth-first numbering: by depth, then by candidate index */
        po[0] = -1; to[0] = root_token[b]; co[0] = -1;
        int n = 1;
        for (int d = 1; n < want + 1 && d <= C; ++d)
            for (int c = 0; c < C; ++c)
                if (kept[c] && depth[c] == d) {
                    node_of[c] = n;
                    co[n] = c;
                    to[n] = ct[c];
                    po[n] = (cp[c] < 0) ? 0 : node_of[cp[c]];
                    ++n;
                }
        n_out[b] = n;
        /* attention mask of the flattened tree: node i sees itself and its ancestors */
        if (anc_out) {
            uint64_t *ao = anc_out + (size_t)b * N;
            for (int i = 0; i < N; ++i) ao[i] = 0;
            for (int i = 0; i < n; ++i) ao[i] = ((i > 0) ? ao[po[i]] : 0) | ((uint64_t)1 << i);
        }
        free(kept); free(depth); free(node_of);
    }
    return rc;
}

/* -------------------------------------------------------------------------
 * O6  Dynamic token tree, one draft step (paper, Section "Preliminaries", last
 * paragraph: "the output of each step can be truncated by selecting the
 * top-k" and "the computation of joint probabilities for each token").
 *
 * For every frontier node f of sequence b the row logprobs[b][f][.] holds the
 * draft model's log-probabilities of the next token.  Its top_k entries
 * (largest value; equal values: the lower token first) become new candidates,
 * numbered base + f * top_k + r with r = 0 for the most probable, with parent
 * frontier_cand[b][f] and joint log-probability frontier_logp[b][f] + value,
 * formed by ONE single-precision addition (so that the order of the joint
 * values is the same on every implementation).  The `width` new candidates
 * with the largest joint value (equal values: the lower candidate index first)
 * form the next frontier, returned in that order.
 *   logprobs [B][F][V] float; frontier_logp [B][F] float; frontier_cand [B][F]
 *   cand_parent, cand_token, cand_logp [B][cap]: entries base .. base + F*top_k - 1 written
 *   next_cand [B][width] int32, next_logp [B][width] float
 * Plain selection loops.
 * ---------------------------------------------------------------------- */
int oracle_draft_expand(const float *logprobs, const float *frontier_logp, const int32_t *frontier_cand,
                        int B, int F, int V, int top_k, int width, int base, int cap,
                        int32_t *cand_parent, int32_t *cand_token, float *cand_logp, int32_t *next_cand,
                        float *next_logp)
{
    if (top_k < 1 || top_k > V || width < 1 || width > F * top_k || base < 0 || base + F * top_k > cap) return -1;
    for (int b = 0; b < B; ++b) {
        int32_t *cp = cand_parent + (size_t)b * cap, *ct = cand_token + (size_t)b * cap;
        float *cl = cand_logp + (size_t)b * cap;
        for (int f = 0; f < F; ++f) {
            const float *row = logprobs + ((size_t)b * F + f) * V;
            char *taken = (char *)calloc((size_t)V, 1);
            if (!taken) return -2;
            for (int r = 0; r < top_k; ++r) {
                int best = -1;
                for (int j = 0; j < V; ++j) {
                    if (taken[j]) continue;
                    if (best < 0 || row[j] > row[best]) best = j;      /* strict: the lower token wins a tie */
                }
                taken[best] = 1;
                const int c = base + f * top_k + r;
                cp[c] = frontier_cand[(size_t)b * F + f];
                ct[c] = best;
                const volatile float joint = frontier_logp[(size_t)b * F + f] + row[best];   /* one fp32 addition */
                cl[c] = joint;
            }
            free(taken);
        }
        const int n_new = F * top_k;
        char *used = (char *)calloc((size_t)n_new, 1);
        if (!used) return -2;
        for (int w = 0; w < width; ++w) {
            int best = -1;
            for (int i = 0; i < n_new; ++i) {
                if (used[i]) continue;
                if (best < 0 || cl[base + i] > cl[base + best]) best = i;
            }
            used[best] = 1;
            next_cand[(size_t)b * width + w] = base + best;
            next_logp[(size_t)b * width + w] = cl[base + best];
        }
        free(used);
    }
    return 0;
}
