// Lossless tree acceptance, second stage: the walk from the root.
//
// Greedy (T = 0): strict comparison of each child's draft token with the
// target's argmax at its parent (paper, Section "Preliminaries": differing
// tokens and their descendants are discarded).  Sampling (T > 0, Section
// "Experiments": T = 1 with unrelaxed acceptance): recursive rejection
// sampling over the children of the current node with residual-distribution
// resampling over the whole vocabulary.
//
// One thread-block cluster serves one sequence.  The walk itself is a short
// serial chain of scalar decisions taken in fp64; whenever a decision needs a
// whole-vocabulary quantity (an exact softmax denominator, the mass of a
// residual distribution, the inverse CDF of the bonus draw) the cluster sweeps
// the node's rows, every CTA reducing its contiguous slice of the vocabulary
// and the CTAs exchanging partial sums through distributed shared memory.
// Only rows on the realised path are ever read.  The first sweep at a node
// evaluates exp((x - max)/T) in fp64 once per token and parks the values (and
// the draft row) in shared memory, so later sweeps at that node are cheap.
//
// The residual after k rejections at a node is kept in closed form instead of
// as a vector: for a token j that has not been rejected,
//     u_j = max(p_j - c * q_j, 0),   p_j = softmax(logits/T)_j,  q_j = draft_j
// with one scalar c that grows with every rejection; a rejected token keeps the
// value it had when it was rejected.  The current target distribution is u / U
// (U = sum of u) and the current draft distribution is q restricted to the
// tokens not yet rejected, divided by its sum D.  A rejection of token x turns
// c into c + U / D, which is exactly p <- norm(max(p - q, 0)), q <- norm(q
// without x) written without materialising either vector.
//
// The per-row maximum and argmax come exact from the vocabulary scan; its sum
// of exponentials is fp32-accurate and is trusted only when a decision clears
// a 1e-4 relative margin, otherwise (and before any residual) the exact sum is
// swept here.
#include <cooperative_groups.h>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace {

constexpr int kMaxCluster = 16;
constexpr int kWalkThreads = 1024;
constexpr int kWarps = kWalkThreads / 32;
constexpr int kSmemBudget = 200 * 1024;   // dynamic shared memory for the per-node cache
constexpr int kSmemBudgetWide = 188 * 1024;   // the same for the instance with room for 256 nodes (its static part is larger)
constexpr double kAmbiguous = 1e-4;
constexpr double kScanRel = 1e-6;          // bound taken for the relative error of the scan's sum of exponentials
constexpr double kFusedTol = 1e-9;         // relative error the fused first-rejection sweep may leave in the residual mass
constexpr float kLog2eF = 1.4426950408889634f;
constexpr int kPieceSlots = 16;            // pieces of a row whose scan sums are kept for the bonus draw
enum { REQ_DONE = 0, REQ_EXP = 1, REQ_EXP_Q = 2, REQ_FUSED = 3, REQ_RESID = 4 };

// 2^(i/64), i = 0..63, correctly rounded
__constant__ double kExp2Tbl[64] = {
    1.0, 1.0108892860517005, 1.0218971486541166, 1.0330248790212284,
    1.0442737824274138, 1.0556451783605572, 1.0671404006768237, 1.0787607977571199,
    1.0905077326652577, 1.102382583307841, 1.1143867425958924, 1.1265216186082418,
    1.1387886347566916, 1.1511892299529827, 1.1637248587775775, 1.1763969916502812,
    1.189207115002721, 1.202156731452703, 1.215247359980469, 1.22848053610687,
    1.241857812073484, 1.255380757024691, 1.2690509571917332, 1.2828700160787783,
    1.2968395546510096, 1.3109612115247644, 1.3252366431597413, 1.339667524053303,
    1.3542555469368927, 1.3690024229745905, 1.383909881963832, 1.3989796725383112,
    1.4142135623730951, 1.42961333839197, 1.4451808069770467, 1.460917794180647,
    1.4768261459394993, 1.4929077282912648, 1.5091644275934228, 1.5255981507445384,
    1.5422108254079407, 1.559004400237837, 1.5759808451078865, 1.593142151342267,
    1.6104903319492543, 1.6280274218573478, 1.645755478153965, 1.6636765803267364,
    1.681792830507429, 1.7001063537185235, 1.718619298122478, 1.7373338352737062,
    1.7562521603732995, 1.7753764925265212, 1.7947090750031072, 1.8142521755003989,
    1.8340080864093424, 1.8539791250833855, 1.8741676341103, 1.8945759815869656,
    1.9152065613971474, 1.9360617934922943, 1.9571441241754002, 1.978456026387951,
};

struct WalkArgs {
    const float *logits, *draft, *temperature, *uniforms;
    const int *tokens, *parent;
    const FspadStatsPart *parts;
    FspadStatsGeom geom;
    int N, V, path_stride, cache_ok;
    int *path, *n_acc, *bonus, *status;
    // optional: the cluster that has walked a sequence also moves its accepted K/V rows up (NULL: not asked for)
    uint4 *kv_cache;                    // [layers][2][B][Hkv][max_len][d] bf16 as 16-byte chunks
    const int *kv_prefix;
    int *kv_new_len;
    int kv_layers, kv_B, kv_H, kv_max_len;
};

// A set of tree nodes as a bit mask of W 64-bit words (W = 1: trees of up to 64 nodes, the common case;
// W = 4: up to 256).
template <int W> struct NodeSet {
    unsigned long long w[W];
    __device__ __forceinline__ bool any() const
    {
        unsigned long long o = 0ull;
#pragma unroll
        for (int i = 0; i < W; ++i) o |= w[i];
        return o != 0ull;
    }
    __device__ __forceinline__ int first() const          // lowest member (the set is not empty)
    {
#pragma unroll
        for (int i = 0; i < W; ++i)
            if (w[i]) return i * 64 + __ffsll((long long)w[i]) - 1;
        return -1;
    }
    __device__ __forceinline__ void drop_first()
    {
#pragma unroll
        for (int i = 0; i < W; ++i)
            if (w[i]) { w[i] &= w[i] - 1; return; }
    }
    __device__ __forceinline__ bool single() const        // exactly one member
    {
        NodeSet t = *this;
        t.drop_first();
        return any() && !t.any();
    }
};

// MAXN: capacity in tree nodes of this instance of the kernel (64 or FSPAD_MAX_NODES_WIDE)
template <int MAXN> struct SharedT {
    static constexpr int W = MAXN / 64;
    static constexpr int kPieceRows = (MAXN == 64) ? 64 : 1;   // the per-piece masses are kept only by the 64-node instance
    double exp_tbl[64];             // 2^(i/64)
    int parent[MAXN];
    int tok[MAXN];
    int path[MAXN];
    // state of the current node (written by thread 0, read by all after a barrier)
    double S, invS, c, U, D, m, invT;
    NodeSet<W> child_mask[MAXN];    // c in child_mask[i] iff parent[c] == i
    int exact, nrem, decision, xnew, ridx, next, len, cur, have_e, have_q, sel;
    double cprime, ex, qx;
    int rem_tok[MAXN];
    double rem_frozen[MAXN];
    // gathered once, in parallel, before the walk: the scan result of every row and, for
    // every node, its parent's logit and draft probability at the node's token and its uniform
    float rowM[MAXN];
    double rowS[MAXN];
    double rowInvS[MAXN];   // 1 / rowS, so that no division sits on the serial path
    int rowA[MAXN];
    float cx[MAXN], cq[MAXN], cu[MAXN];
    double cex[MAXN];    // exp((logit - row max)/T) of each node's token in its parent's row
    float ubonus;
    int want_q;
    int bonus_ok;                   // the last residual sweep already holds the bonus draw's per-thread sums
    // reductions
    double warp_a[kWarps], warp_b[kWarps], warp_off[kWarps];
    double slot[2][kMaxCluster][2]; // partial sums received from every CTA of the cluster, by pass parity
    double tot[2];                  // cluster totals
    double warp5[kWarps][5], slot5[2][kMaxCluster][5], tot5[5];   // the same exchange for five values
    int fused_fallback;
    double cta_total[2][kMaxCluster];  // bonus draw: every CTA's total, received from the peers (by attempt)
    int verdict[2];                    // bonus draw from one piece of the row: 1 = settled, 2 = the whole row must be swept
    // serial walk -> sweeps: what thread 0 asks the CTA to do next
    int req, req_child, req_last;
    NodeSet<W> rem;                    // children of the current node not tested yet
    // approximate mass of every (row, CTA) piece of the vocabulary scan, relative to the row maximum;
    // piece_cnt[row] = 0 when the row has more than kPieceSlots pieces (the draw then sweeps the whole row)
    double piece_w[kPieceRows][kPieceSlots];
    int piece_cnt[kPieceRows];
};

// exp(a) for a <= 0 in double precision: a = (64 n + i) ln2/64 + r, |r| <= ln2/128,
// exp(a) = 2^n * 2^(i/64) * (1 + r + r^2/2 + r^3/6 + r^4/24); relative error below 5e-14
// (truncation r^5/120 < 4e-14, one-step argument reduction < 3e-14 at the far end of the range).
// Every operation is an fp64 multiply-add: the rounding to the nearest integer is done by adding
// and subtracting 1.5 * 2^52 (the integer then sits in the low word of the sum), because the
// conversions between integers and doubles cost as much as an fp64 operation each.
__device__ __forceinline__ double exp_neg(double a, const double *tbl)
{
    if (!(a > -700.0)) return 0.0;                        // also -inf and NaN
    const double magic = 6755399441055744.0;              // 1.5 * 2^52
    const double tm = fma(a, 92.33248261689366, magic);   // a * 64 / ln 2, rounded to an integer
    const int k = __double2loint(tm);
    const double kd = tm - magic;
    const double r = fma(-kd, 0.010830424696249145, a);   // ln2/64
    double p = fma(r, 1.0 / 24.0, 1.0 / 6.0);
    p = fma(p, r, 0.5);
    p = fma(p, r, 1.0);
    p = fma(p, r, 1.0);
    const double y = tbl[k & 63] * p;
    const int n = k >> 6;                                  // floor(k / 64), n in [-1010, 0]
    return __hiloint2double(__double2hiint(y) + (n << 20), __double2loint(y));
}

__device__ __forceinline__ double warp_sum(double v)
{
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

__device__ __forceinline__ double weight(double e, double q, double invS, double c)
{
    const double w = e * invS - c * q;
    return w > 0.0 ? w : 0.0;
}

enum { MODE_EXP = 0, MODE_RESID = 1, MODE_CDF = 2 };

struct Sweep {
    double a, b;
};

// One sweep of this thread's contiguous chunk [lo, hi) of the vocabulary.
//   MODE_EXP  : a = sum of e_j = exp((x_j - m)/T); e_j parked in shared memory
//   MODE_RESID: a = sum of residual weights at coefficient c (tokens already
//               rejected contribute their frozen value), b = sum of q over
//               tokens neither rejected before nor equal to xnew
//   MODE_CDF  : a = sum of the weights the bonus token is drawn from
//               (nothing rejected at this node: the e_j themselves)
// With `locate` the running sum starts at run0 and *found receives the first
// token where base + run exceeds target (else the last positive-weight token).
template <int MODE, class Shared>
__device__ Sweep sweep_chunk(const Shared &sh, const float *__restrict__ x, const float *__restrict__ q,
                             double *__restrict__ se, float *__restrict__ sq, int tid, int nthr, int lo, int hi,
                             bool vec, bool cache_ok, bool have_e, bool have_q, double c, int xnew,
                             bool locate, double base, double run0, double target, int *found)
{
    const double m = sh.m, invT = sh.invT;
    const int nrem = sh.nrem;
    // bonus draw with nothing rejected at this node: the weights are the e_j themselves
    const double invS = (MODE == MODE_CDF && c == 0.0 && nrem == 0) ? 1.0 : sh.invS;
    // the exact-sum sweep that precedes a rejection also parks the draft row for the sweeps to come
    const bool need_q = (MODE == MODE_RESID) || (MODE == MODE_CDF && c != 0.0) || (MODE == MODE_EXP && xnew == -2);
    bool special = false;
    if (MODE != MODE_EXP) {
        for (int r = 0; r < nrem; ++r) special |= (sh.rem_tok[r] >= lo && sh.rem_tok[r] < hi);
        if (MODE == MODE_RESID) special |= (xnew >= lo && xnew < hi);
    }
    double a = 0.0, b = 0.0, run = run0;
    int last_pos = -1, hit = -1;
    for (int j = lo; j < hi; j += 4) {
        const int n = min(4, hi - j);
        double ev[4];
        float qv[4] = {0.f, 0.f, 0.f, 0.f};
        if (have_e) {
#pragma unroll
            for (int t = 0; t < 4; ++t) ev[t] = (t < n) ? se[(j - lo + t) * nthr + tid] : 0.0;
        } else {
            float xv[4];
            if (vec && n == 4) {
                const float4 t4 = __ldg(reinterpret_cast<const float4 *>(x + j));
                xv[0] = t4.x; xv[1] = t4.y; xv[2] = t4.z; xv[3] = t4.w;
            } else {
#pragma unroll
                for (int t = 0; t < 4; ++t) xv[t] = (t < n) ? x[j + t] : -INFINITY;
            }
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                ev[t] = exp_neg(((double)xv[t] - m) * invT, sh.exp_tbl);
                if (cache_ok && t < n) se[(j - lo + t) * nthr + tid] = ev[t];
            }
        }
        if (need_q) {
            if (have_q) {
#pragma unroll
                for (int t = 0; t < 4; ++t) qv[t] = (t < n) ? sq[(j - lo + t) * nthr + tid] : 0.f;
            } else {
                if (vec && n == 4) {
                    const float4 u4 = __ldg(reinterpret_cast<const float4 *>(q + j));
                    qv[0] = u4.x; qv[1] = u4.y; qv[2] = u4.z; qv[3] = u4.w;
                } else {
#pragma unroll
                    for (int t = 0; t < 4; ++t) qv[t] = (t < n) ? q[j + t] : 0.f;
                }
                if (cache_ok) {
#pragma unroll
                    for (int t = 0; t < 4; ++t) if (t < n) sq[(j - lo + t) * nthr + tid] = qv[t];
                }
            }
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            if (t >= n) break;
            if (MODE == MODE_EXP) {
                a += ev[t];
                continue;
            }
            double w = weight(ev[t], (double)qv[t], invS, c);
            bool q_counts = true;
            if (special) {
                const int id = j + t;
                for (int r = 0; r < nrem; ++r)
                    if (sh.rem_tok[r] == id) { w = sh.rem_frozen[r]; q_counts = false; }
                if (id == xnew) q_counts = false;
            }
            a += w;
            if (MODE == MODE_RESID) {
                if (q_counts) b += (double)qv[t];
            } else if (locate) {
                run += w;
                if (w > 0.0) last_pos = j + t;
                if (hit < 0 && base + run > target) hit = j + t;
            }
        }
    }
    if (locate) *found = (hit >= 0) ? hit : last_pos;
    return Sweep{a, b};
}

// The first rejection at a node, in one sweep instead of two.  The exact denominator S is not known
// yet, but the residual sum_j max(e_j / S - c q_j, 0) is linear in 1 / S over a fixed set of positive
// terms: with P = { j : e_j / S' - c q_j > 0 } taken at the scan's S' it equals (sum_P e_j) / S -
// c sum_P q_j for every S that leaves P unchanged.  The sweep returns
//   v[0] = sum e_j (= S)      v[1] = sum_P e_j      v[2] = sum_P q_j
//   v[3] = sum of q_j over j != xnew (the next draft mass)
//   v[4] = sum of e_j / S' over the tokens whose sign a relative error kScanRel of S' could flip;
// a flipped token changes the result by at most kScanRel times its probability, so kScanRel * v[4]
// bounds the error and the caller falls back to the two-sweep path when that is not negligible.
// e_j and q_j are parked in shared memory as in the exact-sum sweep.
struct Sweep5 {
    double v[5];
};
template <class Shared>
__device__ Sweep5 fused_reject_sweep(const Shared &sh, const float *__restrict__ x, const float *__restrict__ q,
                                     double *__restrict__ se, float *__restrict__ sq, int tid, int nthr, int lo, int hi,
                                     bool vec, bool cache_ok, double inv_s_scan, double c, int xnew)
{
    const double m = sh.m, invT = sh.invT;
    Sweep5 r{{0.0, 0.0, 0.0, 0.0, 0.0}};
    for (int j = lo; j < hi; j += 4) {
        const int n = min(4, hi - j);
        float xv[4], qv[4];
        if (vec && n == 4) {
            const float4 t4 = __ldg(reinterpret_cast<const float4 *>(x + j));
            const float4 u4 = __ldg(reinterpret_cast<const float4 *>(q + j));
            xv[0] = t4.x; xv[1] = t4.y; xv[2] = t4.z; xv[3] = t4.w;
            qv[0] = u4.x; qv[1] = u4.y; qv[2] = u4.z; qv[3] = u4.w;
        } else {
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                xv[t] = (t < n) ? x[j + t] : -INFINITY;
                qv[t] = (t < n) ? q[j + t] : 0.f;
            }
        }
#pragma unroll
        for (int t = 0; t < 4; ++t) {
            if (t >= n) break;
            const double e = exp_neg(((double)xv[t] - m) * invT, sh.exp_tbl);
            const double qd = (double)qv[t];
            if (cache_ok) {
                se[(j - lo + t) * nthr + tid] = e;
                sq[(j - lo + t) * nthr + tid] = qv[t];
            }
            const double pe = e * inv_s_scan;
            const double w = pe - c * qd;
            r.v[0] += e;
            if (w > 0.0) { r.v[1] += e; r.v[2] += qd; }
            if (j + t != xnew) r.v[3] += qd;
            // |w| <= kScanRel * pe needs the binary exponent of w at least 19 below that of pe: an
            // integer comparison sorts out all but a handful of tokens
            if ((__double2hiint(w) & 0x7ff00000) <= (__double2hiint(pe) & 0x7ff00000) - (19 << 20))
                if (pe > 0.0 && fabs(w) <= kScanRel * pe) r.v[4] += pe;
        }
    }
    return r;
}

// Compaction of the accepted path by the CTAs that walked it (every CTA of the cluster holds the same path in
// its shared memory): row L + path[j] -> row L + j of every (layer, K/V, head) slice of the sequence, one warp
// per slice, eight rows in flight, every load of a batch before any of its stores (path[j] >= j and the path
// is increasing, so moves in index order never overwrite a row that is still to be read).  The same moves as
// the stand-alone compaction kernel makes; doing them here saves the step one dependent launch.
template <typename Shared>
__device__ __forceinline__ void compact_accepted(const WalkArgs &args, const Shared &sh, int b, int rank, int C, int tid, int nthr)
{
    if (args.kv_cache == nullptr) return;
    const int lane = tid & 31, n_warps = nthr >> 5;
    int n = sh.len;
    const int L = args.kv_prefix[b];
    if (L < 0 || n < 1 || L + sh.path[n - 1] >= args.kv_max_len) {
        if (rank == 0 && tid == 0) fspad_report(args.status, FSPAD_ERR_RANGE);
        n = 0;
    }
    if (rank == 0 && tid == 0 && args.kv_new_len) args.kv_new_len[b] = max(L, 0) + n;
    const int per_seq = args.kv_layers * 2 * args.kv_H;
    const int chunk = lane & 15, half = lane >> 4;
    for (int s = rank * n_warps + (tid >> 5); s < per_seq; s += C * n_warps) {
        const int lk = s / args.kv_H, h = s % args.kv_H;
        uint4 *base = args.kv_cache + ((((size_t)lk * args.kv_B + b) * args.kv_H + h) * args.kv_max_len + L) * 16;
        for (int j0 = 0; j0 < n; j0 += 8) {
            uint4 v[4];
            int dst[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int j = j0 + 2 * u + half;
                dst[u] = -1;
                if (j < n) {
                    const int src = sh.path[j];
                    if (src != j) {
                        v[u] = base[(size_t)src * 16 + chunk];
                        dst[u] = j;
                    }
                }
            }
            __syncwarp();
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (dst[u] >= 0) base[(size_t)dst[u] * 16 + chunk] = v[u];
        }
    }
}

template <int MAXN>
__global__ void __launch_bounds__(kWalkThreads, 1)
accept_walk_kernel(const WalkArgs args)
{
    typedef SharedT<MAXN> Shared;
    constexpr int W = Shared::W;
    cg::cluster_group cluster = cg::this_cluster();
    const int C = (int)cluster.num_blocks();
    const int rank = (int)cluster.block_rank();
    const int b = blockIdx.x / C;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int N = args.N, V = args.V;

    __shared__ Shared sh;
    extern __shared__ __align__(16) unsigned char dyn_smem[];

    fspad_pdl_trigger();
    if (tid < 64) sh.exp_tbl[tid] = kExp2Tbl[tid];
    if (tid < MAXN) {
#pragma unroll
        for (int i = 0; i < W; ++i) sh.child_mask[tid].w[i] = 0ull;
    }
    // The vocabulary scan that precedes this kernel in the stream lets it start only after the scan's
    // own predecessor has completed, and the scan writes nothing but its partial results.  So the
    // caller's arrays may be read before the scan has finished: the prologue's two round trips of
    // dependent loads run under the scan's tail.
    // Round trip 1: everything that depends on nothing - temperature, tree arrays, uniforms.
    float Tf = args.temperature[b];
    int p = -1, t = 0;
    float uval = 0.f;
    if (tid < N) {
        p = args.parent[(size_t)b * N + tid];
        t = args.tokens[(size_t)b * N + tid];
    }
    if (args.uniforms != nullptr && tid <= N)      // thread c: node c's uniform; thread 0: the bonus uniform
        uval = args.uniforms[(size_t)b * (N + 1) + (tid == 0 ? N : tid)];
    if (!(Tf >= 0.0f)) {
        if (tid == 0 && rank == 0) fspad_report(args.status, FSPAD_ERR_RANGE);
        Tf = 0.0f;
    }
    const bool sampling = Tf > 0.0f && args.draft != nullptr && args.uniforms != nullptr;
    if (Tf > 0.0f && !sampling && tid == 0 && rank == 0) fspad_report(args.status, FSPAD_ERR_NULL);
    __syncthreads();                             // child masks are zeroed

    const float *lg = args.logits + (size_t)b * N * V;
    const float *dp = args.draft ? args.draft + (size_t)b * N * V : nullptr;
    int *out_path = args.path + (size_t)b * args.path_stride;
    const float kT = kLog2eF / (Tf > 0.0f ? Tf : 1.0f);

    // Round trip 2: thread c owns node c (tree arrays, the child bit of its parent and the scalars
    // its accept test needs: target logit and draft probability of its token in its parent's row).
    float xv = 0.f, qv = 0.f;
    if (tid < N) {
        if (tid == 0) {
            if (p != -1) fspad_report(args.status, FSPAD_ERR_BAD_TREE);
            p = -1;
        } else if (p < 0 || p >= tid) {
            fspad_report(args.status, FSPAD_ERR_BAD_TREE);
            p = 0;
        }
        if (t < 0 || t >= V) {
            fspad_report(args.status, FSPAD_ERR_RANGE);
            t = 0;
        }
        sh.parent[tid] = p;
        sh.tok[tid] = t;
        if (tid >= 1) {
            atomicOr(&sh.child_mask[p].w[tid >> 6], 1ull << (tid & 63));
            if (sampling) {
                const size_t at = (size_t)p * V + t;
                xv = lg[at];
                qv = dp[at];
            }
        }
    }
    // The root's draft row is the one most likely to be swept: ask for it now (a hint, no register
    // is tied up and nothing waits for it).
    const bool vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(args.logits) & 15) == 0) &&
                     ((reinterpret_cast<uintptr_t>(args.draft) & 15) == 0);
    // contiguous slice per CTA, contiguous chunk per thread (multiples of 4 tokens)
    const int per_cta = (((V + C - 1) / C) + 3) & ~3;
    const int per_thr = (((per_cta + nthr - 1) / nthr) + 3) & ~3;
    const int cta_lo = rank * per_cta, cta_hi = min(V, cta_lo + per_cta);
    const int lo = min(cta_hi, cta_lo + tid * per_thr), hi = min(cta_hi, lo + per_thr);
    if (sampling && lo < hi)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(dp + lo));
    if (sampling && tid < N) {
        if (tid >= 1) { sh.cx[tid] = xv; sh.cq[tid] = qv; sh.cu[tid] = uval; }
        else sh.ubonus = uval;
    }

    fspad_pdl_wait();                            // from here on the scan's partial results may be read
    {
        // half-warps merge the scan partials of the rows
        const int lane16 = tid & 15, n_half = nthr >> 4;
        for (int r0 = 0; r0 < N; r0 += n_half) {                 // whole warps iterate together
            const int row = r0 + (tid >> 4);
            float M; double S; int A;
            if (MAXN == 64)
                fspad_stats_merge_half(args.parts, args.geom, b * N + row, row < N, kT, lane16, M, S, A,
                                       sh.piece_w[row < N ? row : 0], &sh.piece_cnt[row < N ? row : 0]);
            else
                fspad_stats_merge_half(args.parts, args.geom, b * N + row, row < N, kT, lane16, M, S, A);
            if (lane16 == 0 && row < N) { sh.rowM[row] = M; sh.rowS[row] = S; sh.rowInvS[row] = 1.0 / S; sh.rowA[row] = A; }
        }
    }
    __syncthreads();
    if (sampling && tid >= 1 && tid < N)
        sh.cex[tid] = exp_neg(((double)sh.cx[tid] - (double)sh.rowM[sh.parent[tid]]) * (1.0 / (double)Tf), sh.exp_tbl);
    __syncthreads();

    if (!sampling) {
        // ---- greedy: strict token comparison against the target argmax ----
        if (tid == 0) {                               // every CTA of the cluster: same data, same path
            int cur = 0, len = 1;
            sh.path[0] = 0;
            for (;;) {
                const int want = sh.rowA[cur];
                int next = -1;
                for (NodeSet<W> rem = sh.child_mask[cur]; rem.any(); rem.drop_first()) {
                    const int c = rem.first();
                    if (sh.tok[c] == want) { next = c; break; }
                }
                if (next < 0) { if (rank == 0) args.bonus[b] = want; break; }
                sh.path[len++] = next;
                cur = next;
            }
            if (rank == 0) args.n_acc[b] = len;
            sh.len = len;
        }
        __syncthreads();
        if (rank == 0)
            for (int i = tid; i < args.path_stride; i += nthr) out_path[i] = (i < sh.len) ? sh.path[i] : -1;
        compact_accepted(args, sh, b, rank, C, tid, nthr);
        return;   // the whole cluster takes this branch together; no peer memory is touched
    }

    // ---- sampling ----
    const bool cache_ok = args.cache_ok != 0;
    double *se = reinterpret_cast<double *>(dyn_smem);
    // the cache is laid out [k][thread] (k-th token of each thread's chunk): conflict-free
    float *sq = reinterpret_cast<float *>(dyn_smem + (size_t)per_thr * nthr * sizeof(double));
    int parity = 0;

    // cluster-wide reduction of (a, b); result in sh.tot[] (read by thread 0 only).  Every level
    // is a warp butterfly; the CTAs exchange by remote stores (each writes its pair into every
    // peer's slot before the barrier), so after the barrier all reads are local, and every CTA
    // performs the same operations on the same values.
    auto reduce_exchange = [&](double a, double bb) {
        const int lane = tid & 31, wid = tid >> 5, nwarps = nthr >> 5;
        a = warp_sum(a);
        bb = warp_sum(bb);
        if (lane == 0) { sh.warp_a[wid] = a; sh.warp_b[wid] = bb; }
        __syncthreads();
        if (wid == 0) {
            double sa = (lane < nwarps) ? sh.warp_a[lane] : 0.0;
            double sb = (lane < nwarps) ? sh.warp_b[lane] : 0.0;
            sa = warp_sum(sa);
            sb = warp_sum(sb);
            if (lane < C) {
                double *peer = cluster.map_shared_rank(&sh.slot[parity][rank][0], lane);
                peer[0] = sa;
                peer[1] = sb;
            }
        }
        cluster.sync();
        if (wid == 0) {
            double ta = (lane < C) ? sh.slot[parity][lane][0] : 0.0;
            double tb = (lane < C) ? sh.slot[parity][lane][1] : 0.0;
            ta = warp_sum(ta);
            tb = warp_sum(tb);
            if (lane == 0) { sh.tot[0] = ta; sh.tot[1] = tb; }
        }
        __syncthreads();
        parity ^= 1;
    };

    const double invT = 1.0 / (double)Tf;        // every thread: off the serial path of thread 0
    // the same exchange for the five sums of the fused sweep; result in sh.tot5[]
    auto reduce_exchange5 = [&](const Sweep5 &in) {
        const int lane = tid & 31, wid = tid >> 5, nwarps = nthr >> 5;
        double v[5];
#pragma unroll
        for (int k = 0; k < 5; ++k) v[k] = warp_sum(in.v[k]);
        if (lane == 0) {
#pragma unroll
            for (int k = 0; k < 5; ++k) sh.warp5[wid][k] = v[k];
        }
        __syncthreads();
        if (wid == 0) {
#pragma unroll
            for (int k = 0; k < 5; ++k) v[k] = warp_sum((lane < nwarps) ? sh.warp5[lane][k] : 0.0);
            if (lane < C) {
                double *peer = cluster.map_shared_rank(&sh.slot5[parity][rank][0], lane);
#pragma unroll
                for (int k = 0; k < 5; ++k) peer[k] = v[k];
            }
        }
        cluster.sync();
        if (wid == 0) {
#pragma unroll
            for (int k = 0; k < 5; ++k) {
                const double t5 = warp_sum((lane < C) ? sh.slot5[parity][lane][k] : 0.0);
                if (lane == 0) sh.tot5[k] = t5;
            }
        }
        __syncthreads();
        parity ^= 1;
    };

    // Thread 0 of every CTA (all on identical data, so all take identical steps) walks ahead through
    // every decision that needs nothing but scalars, and stops only to ask the CTA for a sweep of the
    // current node's rows.  enter() makes a node the current one.
    auto enter = [&](int node) {
        sh.cur = node;
        sh.m = (double)sh.rowM[node];
        sh.S = sh.rowS[node];
        sh.invS = sh.rowInvS[node];
        sh.exact = 0; sh.have_e = 0; sh.have_q = 0;
        sh.c = 0.0; sh.U = 1.0; sh.D = 1.0;
        sh.nrem = 0;
        sh.bonus_ok = 0;
        sh.rem = sh.child_mask[node];
    };
    if (tid == 0) { sh.len = 1; sh.path[0] = 0; sh.invT = invT; enter(0); }
    double last_a = 0.0;                         // this thread's sum of weights in the latest residual sweep

    for (;;) {
        if (tid == 0) {
            int req = REQ_DONE;
            while (sh.rem.any()) {
                const int ch = sh.rem.first();
                const int xt = sh.tok[ch];
                const double r = (double)sh.cu[ch];
                const double qx = (double)sh.cq[ch];
                const double ex = sh.cex[ch];
                int ridx = -1;
                for (int k = 0; k < sh.nrem; ++k) if (sh.rem_tok[k] == xt) ridx = k;
                // accept iff r * q_k(x) < p_k(x) with q_k = qx / D and p_k = u / U: compared as
                // r * qx * U < u * D (both normalisers are positive), so no division is needed
                const double u = (ridx >= 0) ? sh.rem_frozen[ridx] : weight(ex, qx, sh.invS, sh.c);
                const double lhs = (ridx >= 0) ? 0.0 : r * qx * sh.U;
                const double rhs = u * sh.D;
                const bool acc = lhs < rhs;
                if (!sh.exact) {
                    // the scan's sum of exponentials is trusted only outside a margin around the boundary
                    const double big = fmax(lhs, rhs);
                    if (big > 0.0 && fabs(lhs - rhs) <= kAmbiguous * big) {
                        req = acc ? REQ_EXP : REQ_EXP_Q;      // exact denominator first (and park the draft row if a rejection is likely)
                        break;
                    }
                }
                if (acc) {
                    sh.path[sh.len++] = ch;
                    enter(ch);
                    continue;
                }
                // rejected: one sweep gives the new residual mass and the new draft mass
                sh.ex = ex; sh.qx = qx; sh.ridx = ridx; sh.xnew = xt;
                sh.cprime = sh.c + sh.U / sh.D;
                req = sh.exact ? REQ_RESID : REQ_FUSED;       // first rejection at a node: exact denominator and residual in one sweep
                break;
            }
            sh.req = req;
            if (req != REQ_DONE) {
                sh.req_child = sh.rem.first();
                sh.req_last = sh.rem.single() ? 1 : 0;
            }
        }
        __syncthreads();
        const int req = sh.req;
        if (req == REQ_DONE) break;                           // uniform
        const int cur = sh.cur;
        const float *x = lg + (size_t)cur * V;
        const float *q = dp + (size_t)cur * V;
        if (req == REQ_EXP || req == REQ_EXP_Q) {
            // exact softmax denominator of this node (parks e_j in shared memory)
            const bool with_q = req == REQ_EXP_Q;
            Sweep sw = sweep_chunk<MODE_EXP>(sh, x, q, se, sq, tid, nthr, lo, hi, vec, cache_ok, false, false, 0.0,
                                             with_q ? -2 : -1, false, 0, 0, 0, nullptr);
            reduce_exchange(sw.a, 0.0);
            if (tid == 0) {
                sh.S = sh.tot[0]; sh.invS = 1.0 / sh.S; sh.exact = 1; sh.have_e = cache_ok;
                if (with_q) sh.have_q = cache_ok;
            }
            continue;                                         // thread 0 repeats the test with the exact sum
        }
        const int xt = sh.xnew;
        bool fused_done = false;
        if (req == REQ_FUSED) {
            // first rejection at this node, nothing exact yet (c = 0, U = D = 1, nothing removed)
            const double cp = sh.cprime;
            const Sweep5 f = fused_reject_sweep(sh, x, q, se, sq, tid, nthr, lo, hi, vec, cache_ok, sh.invS, cp, xt);
            reduce_exchange5(f);
            if (tid == 0) {
                const double S = sh.tot5[0], invS = 1.0 / S;
                const double W = sh.tot5[1] * invS - cp * sh.tot5[2];
                sh.S = S; sh.invS = invS; sh.exact = 1; sh.have_e = cache_ok; sh.have_q = cache_ok;
                sh.fused_fallback = !(W > 0.0 && kScanRel * sh.tot5[4] <= kFusedTol * W);
                if (!sh.fused_fallback) {
                    sh.tot[0] = W;
                    sh.tot[1] = sh.tot5[3];
                }
            }
            __syncthreads();
            fused_done = !sh.fused_fallback;
            // (the exact sum is taken from the exchange's result, which nothing rewrites before the next
            // exchange; thread 0 may already be changing the walk's state)
            if (fused_done) last_a = f.v[1] * (1.0 / sh.tot5[0]) - cp * f.v[2];
        }
        if (!fused_done) {
            Sweep sw = sweep_chunk<MODE_RESID>(sh, x, q, se, sq, tid, nthr, lo, hi, vec, cache_ok, sh.have_e != 0,
                                               sh.have_q != 0, sh.cprime, xt, false, 0, 0, 0, nullptr);
            last_a = sw.a;
            reduce_exchange(sw.a, sw.b);
        }
        // When this was the node's last child, the weights just summed (residual at the new
        // coefficient, the rejected tokens at their frozen values) are the ones the bonus token is
        // drawn from, thread by thread in the same order: the draw reuses the sums (last_a).
        if (tid == 0) {
            const double W = sh.tot[0], Dn = sh.tot[1];
            double frozen;
            if (W > 0.0) {
                frozen = weight(sh.ex, sh.qx, sh.invS, sh.cprime);
                sh.c = sh.cprime;
                sh.U = W;
                sh.bonus_ok = sh.req_last;
            } else {
                frozen = weight(sh.ex, sh.qx, sh.invS, sh.c);   // residual vanished: p is kept
            }
            if (sh.ridx < 0 && sh.nrem < MAXN) {
                sh.rem_tok[sh.nrem] = xt;
                sh.rem_frozen[sh.nrem] = frozen;
                sh.nrem++;
            }
            if (Dn > 0.0) sh.D = Dn;
            sh.have_q = cache_ok;
            sh.rem.drop_first();                                // this child is done
        }
        // no barrier here: only thread 0 touches the walk's state until the next request is published
    }

    // ---- bonus token: inverse CDF of the current residual at the last node ----
    {
        const int cur = sh.cur;
        const float *x = lg + (size_t)cur * V;
        const float *q = dp + (size_t)cur * V;
        const double c = sh.c;
        const bool have_e = sh.have_e != 0, have_q = sh.have_q != 0;
        const int lane = tid & 31, wid = tid >> 5;

        // block-wide scan of one value per thread (index order): this thread's exclusive and inclusive
        // prefix, the CTA total in sh.warp_a[kWarps - 1] ... returned through `total` (valid in every thread)
        auto block_scan = [&](double v, double &excl_out, double &incl_out, double &total) {
            double incl = v;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const double t2 = __shfl_up_sync(0xffffffffu, incl, off);
                if (lane >= off) incl += t2;
            }
            const double prev_incl = __shfl_up_sync(0xffffffffu, incl, 1);
            if (lane == 31) sh.warp_a[wid] = incl;
            __syncthreads();
            if (wid == 0) {
                // exclusive scan of the warp totals; the last inclusive value is the CTA total
                const int nwarps = nthr >> 5;
                const double wv = (lane < nwarps) ? sh.warp_a[lane] : 0.0;
                double sc = wv;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const double t2 = __shfl_up_sync(0xffffffffu, sc, off);
                    if (lane >= off) sc += t2;
                }
                const double excl = __shfl_up_sync(0xffffffffu, sc, 1);
                if (lane < nwarps) sh.warp_off[lane] = (lane == 0) ? 0.0 : excl;
                if (lane == nwarps - 1) sh.warp_b[0] = sc;
            }
            __syncthreads();
            const double woff = sh.warp_off[wid];
            incl_out = woff + incl;
            excl_out = (lane == 0) ? woff : woff + prev_incl;
            total = sh.warp_b[0];
        };

        // A draw at a node where nothing was rejected (a leaf, typically) is taken from the softmax
        // of the row itself.  The scan left the mass of every piece of the row, accurate to kScanRel:
        // enough to name the piece the target falls into and the mass in front of it.  That piece is
        // then swept with single-precision exponentials - by every CTA on its own, all on the same
        // data with the same arithmetic, so all reach the same verdict and nothing is exchanged - and
        // the token is taken when the target clears both ends of its interval by more than the
        // uncertainty of all the approximations together.  Otherwise, and for every other kind of
        // draw, the cluster sweeps the whole row exactly.
        bool settled = false;
        const int n_piece = (MAXN == 64) ? sh.piece_cnt[MAXN == 64 ? cur : 0] : 0;
        if (!sh.bonus_ok && c == 0.0 && sh.nrem == 0 && n_piece > 0) {
            double Zs = 0.0;
            for (int i = 0; i < n_piece; ++i) Zs += sh.piece_w[MAXN == 64 ? cur : 0][i];
            const double target = (double)sh.ubonus * Zs;
            int pick = -1;
            double pre = 0.0;
            for (int i = 0; i < n_piece; ++i) {
                const double nxt = pre + sh.piece_w[MAXN == 64 ? cur : 0][i];
                if (nxt > target) { pick = i; break; }
                pre = nxt;
            }
            // error budget: the masses in front of the piece and the total (scan, kScanRel each, doubled
            // for slack) and the single-precision sums inside the piece (argument rounding of the
            // exponential 1.3e-7 per unit of |log2 e_j|, the approximation itself 2.4e-7, the partial sums)
            const double tol = 4.0 * kScanRel * Zs + (pick >= 0 ? 4e-6 * sh.piece_w[MAXN == 64 ? cur : 0][pick] : 0.0);
            if (pick >= 0 && target - pre > tol && pre + sh.piece_w[MAXN == 64 ? cur : 0][pick] - target > tol) {
                // token range of that piece: CTA `first + pick` of the scan, clipped to the row
                const FspadStatsGeom &g = args.geom;
                const long long row_lo = (long long)(b * N + cur) * g.upr;
                const long long first = row_lo / g.chunk;
                const long long u_lo = max(row_lo, (first + pick) * g.chunk), u_hi = min(row_lo + g.upr, (first + pick + 1) * g.chunk);
                const int p_lo = (int)(u_lo - row_lo) * g.unit, p_hi = (int)(u_hi - row_lo) * g.unit;
                const int pt = ((((p_hi - p_lo) + nthr - 1) / nthr) + 3) & ~3;
                const int t_lo = min(p_hi, p_lo + tid * pt), t_hi = min(p_hi, t_lo + pt);
                const float Mf = sh.rowM[cur];
                // weights relative to the row maximum, as the table's: e_j = exp2((x_j - max) * log2(e) / T)
                auto e32 = [&](float xv2) {
                    float y;
                    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"((xv2 - Mf) * kT));
                    return xv2 == -INFINITY ? 0.f : y;
                };
                double mine = 0.0;
                for (int j = t_lo; j < t_hi; j += 4) {
                    float xs[4];
                    if (vec && j + 4 <= t_hi) {
                        const float4 t4 = __ldg(reinterpret_cast<const float4 *>(x + j));
                        xs[0] = t4.x; xs[1] = t4.y; xs[2] = t4.z; xs[3] = t4.w;
                    } else {
#pragma unroll
                        for (int t2 = 0; t2 < 4; ++t2) xs[t2] = (j + t2 < t_hi) ? x[j + t2] : -INFINITY;
                    }
                    mine += (double)((e32(xs[0]) + e32(xs[1])) + (e32(xs[2]) + e32(xs[3])));
                }
                double E, P, total;
                block_scan(mine, E, P, total);
                const double tgt = target - pre;                  // within the piece
                if (tid == 0) { sh.sel = 0x7fffffff; sh.verdict[0] = 2; }
                __syncthreads();
                if (P > tgt) atomicMin(&sh.sel, tid);
                __syncthreads();
                if (tid == sh.sel) {
                    double run = E;
                    for (int j = t_lo; j < t_hi; ++j) {
                        const double before = run;
                        run += (double)e32(x[j]);
                        if (run > tgt) {
                            if (tgt - before > tol && run - tgt > tol) {
                                sh.verdict[0] = 1;
                                if (rank == 0) args.bonus[b] = j;
                            }
                            break;
                        }
                    }
                }
                __syncthreads();
                settled = sh.verdict[0] == 1;
            }
        }
        if (rank == 0) {
            if (tid == 0) args.n_acc[b] = sh.len;
            for (int i = tid; i < args.path_stride; i += nthr) out_path[i] = (i < sh.len) ? sh.path[i] : -1;
        }
        compact_accepted(args, sh, b, rank, C, tid, nthr);   // the path is final; only the bonus token may still be open
        if (settled) return;                                // uniform over the cluster; no peer memory is touched after the walk's last exchange

        // ---- exact draw over the whole row: every CTA a contiguous slice, every thread a contiguous chunk ----
        {
            // with nothing rejected at this node (c == 0) the weights are the e_j themselves and the
            // denominator cancels, so no separate exact-sum sweep is needed
            Sweep sw{last_a, 0.0};
            if (!sh.bonus_ok)
                sw = sweep_chunk<MODE_CDF>(sh, x, q, se, sq, tid, nthr, lo, hi, vec, cache_ok, have_e, have_q, c, -1, false, 0, 0,
                                           0, nullptr);
            double E, P, total;
            block_scan(sw.a, E, P, total);
            // the CTA total goes to every CTA of the cluster (remote stores; read locally after the barrier)
            if (tid < C) *cluster.map_shared_rank(&sh.cta_total[0][rank], tid) = total;
            cluster.sync();
            double Z = 0.0, base = 0.0;
            for (int r = 0; r < C; ++r) {
                if (r == rank) base = Z;
                Z = Z + sh.cta_total[0][r];
            }
            const double target = (double)sh.ubonus * Z;
            int owner = -1;
            {
                double cum = 0.0;
                for (int r = 0; r < C; ++r) {
                    cum = cum + sh.cta_total[0][r];
                    if (cum > target) { owner = r; break; }
                }
            }
            if (owner == rank) {
                // the first thread (index order) whose inclusive prefix passes the target owns the draw
                if (tid == 0) sh.sel = 0x7fffffff;
                __syncthreads();
                if (base + P > target) atomicMin(&sh.sel, tid);
                __syncthreads();
                // rounding of the two-level prefix can leave no thread above the target although the
                // CTA total is: the last non-empty chunk then takes the draw
                if (tid == 0 && sh.sel == 0x7fffffff) sh.sel = max(0, (cta_hi - cta_lo - 1) / per_thr);
                __syncthreads();
                if (tid == sh.sel) {
                    int found = -1;
                    sweep_chunk<MODE_CDF>(sh, x, q, se, sq, tid, nthr, lo, hi, vec, false, cache_ok, cache_ok && (c != 0.0),
                                          c, -1, true, base, E, target, &found);
                    if (found < 0) found = min(lo, V - 1);
                    args.bonus[b] = found;
                }
            }
            if (owner < 0 && rank == 0 && tid == 0) args.bonus[b] = 0;   // no positive weight anywhere
        }
        // no CTA touches a peer's shared memory after the cluster barrier above, so each may leave on its own
    }
}

}  // namespace

// Cluster size of the sampling walk.  Once per context: raise the dynamic shared-memory limit and find
// the largest cluster the device can co-schedule for this kernel: 16 (opt-in), else 8.  Small
// vocabularies do not need the whole cluster.  (Halving the clusters of a batch whose CTAs outnumber the
// SMs was measured and not kept: on 16 sequences, half of them greedy and gone at once, the acceptance
// took 186 us with clusters of 8 against 143 us with clusters of 16 in two waves.)
static int walk_cluster_size(fspad_ctx *ctx, int B, int V)
{
    if (ctx->walk_cluster == 0) {
        ctx->walk_cluster = 8;
        cudaFuncSetAttribute(accept_walk_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
        cudaFuncSetAttribute(accept_walk_kernel<FSPAD_MAX_NODES_WIDE>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudgetWide);
        if (cudaFuncSetAttribute(accept_walk_kernel<64>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) == cudaSuccess &&
            cudaFuncSetAttribute(accept_walk_kernel<FSPAD_MAX_NODES_WIDE>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1) ==
                cudaSuccess) {
            cudaLaunchConfig_t probe = {};
            probe.gridDim = dim3(kMaxCluster);
            probe.blockDim = dim3(kWalkThreads);
            probe.dynamicSmemBytes = kSmemBudget;
            cudaLaunchAttribute at[1];
            at[0].id = cudaLaunchAttributeClusterDimension;
            at[0].val.clusterDim.x = kMaxCluster; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
            probe.attrs = at; probe.numAttrs = 1;
            int n = 0;
            int n2 = 0;
            cudaLaunchConfig_t probe2 = probe;
            probe2.dynamicSmemBytes = kSmemBudgetWide;
            if (cudaOccupancyMaxActiveClusters(&n, accept_walk_kernel<64>, &probe) == cudaSuccess && n >= 1 &&
                cudaOccupancyMaxActiveClusters(&n2, accept_walk_kernel<FSPAD_MAX_NODES_WIDE>, &probe2) == cudaSuccess && n2 >= 1)
                ctx->walk_cluster = kMaxCluster;
        }
        (void)cudaGetLastError();
    }
    int cluster = ctx->walk_cluster;
    while (cluster > 1 && (V + cluster - 1) / cluster < 2048) cluster >>= 1;
    return cluster;
}

int fspad_walk_ctas(fspad_ctx *ctx, int B, int V) { return B * walk_cluster_size(ctx, B, V); }

cudaError_t fspad_launch_accept_walk(fspad_ctx *ctx, const float *logits, const float *draft,
                                     const int *tokens, const int *parent, const float *temperature,
                                     const float *uniforms, const FspadStatsGeom &geom, int N, int B, int V,
                                     int *path, int *n_acc, int *bonus, cudaStream_t st, FspadWalkCompact kv)
{
    if (B == 0) return cudaSuccess;
    WalkArgs a;
    a.kv_cache = reinterpret_cast<uint4 *>(kv.cache); a.kv_prefix = kv.prefix_len; a.kv_new_len = kv.new_len;
    a.kv_layers = ctx->cfg.n_layers; a.kv_B = B; a.kv_H = ctx->cfg.n_kv_heads; a.kv_max_len = ctx->cfg.max_len;
    a.logits = logits; a.draft = draft; a.temperature = temperature; a.uniforms = uniforms;
    a.tokens = tokens; a.parent = parent;
    a.parts = ctx->st_part; a.geom = geom;
    a.N = N; a.V = V; a.path_stride = ctx->cfg.max_nodes; a.cache_ok = 0;
    a.path = path; a.n_acc = n_acc; a.bonus = bonus; a.status = ctx->d_status;

    const bool sampling = draft != nullptr && uniforms != nullptr;
    int cluster = 1, threads = 256;
    size_t smem = 0;
    if (sampling) {
        threads = kWalkThreads;
        cluster = walk_cluster_size(ctx, B, V);
        const size_t per_cta = (size_t)((((V + cluster - 1) / cluster) + 3) & ~3);
        const size_t per_thr = ((per_cta + kWalkThreads - 1) / kWalkThreads + 3) & ~(size_t)3;
        const size_t need = per_thr * kWalkThreads * (sizeof(double) + sizeof(float));
        if (need <= (size_t)(N <= 64 ? kSmemBudget : kSmemBudgetWide)) { smem = need; a.cache_ok = 1; }
    }
    ctx->launches++;
    // trees of up to 64 nodes (one mask word per node, per-piece masses kept for the bonus draw) and up to
    // FSPAD_MAX_NODES_WIDE nodes are two instances of the kernel
    if (N <= 64)
        return fspad_launch(accept_walk_kernel<64>, dim3((unsigned)(B * cluster)), dim3(threads), smem, st, (unsigned)cluster, a);
    return fspad_launch(accept_walk_kernel<FSPAD_MAX_NODES_WIDE>, dim3((unsigned)(B * cluster)), dim3(threads), smem, st,
                        (unsigned)cluster, a);
}
