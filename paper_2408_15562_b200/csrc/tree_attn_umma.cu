// Tree-masked verify attention on the 5th-generation tensor cores (paper,
// Section "Preliminaries": the target processes the flattened token tree under
// the attention mask built from the tree).
//
// Split-KV flash-decode with tcgen05: all query rows that share a kv head (tree
// node x GQA group member) form the M = 128 operand of one CTA; keys are
// consumed in chunks of 128.  Per chunk: S = Q K^T is one chain of eight
// tcgen05.mma (128 x 128 x 16, bf16 -> fp32) into tensor memory; a softmax
// thread per query row reads its scores back with tcgen05.ld, applies the
// ancestor mask (only on chunks that reach past the cached prefix) and the
// softmax in registers, and writes P as packed bf16 pairs back into tensor
// memory, over the scores; O += P V is a second chain of eight tcgen05.mma whose
// A operand is read from tensor memory and whose B operand is V in its
// [key][d] layout (MN-major).  O stays in tensor memory across chunks.  The
// work is split over three kinds of warps that meet only on mbarriers (see the
// kernel's comment); K/V chunks go through a three-deep ring of 128-byte-swizzled
// tiles, filled by TMA for chunks inside the cached prefix and by 16-byte
// asynchronous copies for Q and the one chunk that mixes prefix, tree rows and
// zero padding.  Per-split partials are merged by the combine kernel.
//
// Every wait on an mbarrier is bounded; on expiry the CTA records
// FSPAD_ERR_TIMEOUT, skips the remaining tensor-core work, frees its tensor
// memory and returns.
#include <cuda.h>

#include "common.cuh"
#include "umma_common.cuh"

namespace umma {

constexpr int D = FSPAD_HEAD_DIM;      // 128
constexpr int BM = 128;                // query rows per CTA
constexpr int BK = 128;                // keys per chunk
constexpr int NT = 320;                // threads per CTA: two per query row + a copy warp + a tensor-core warp
constexpr int HALF = 128 * 128;        // bytes of one [128 rows][64 bf16] half tile
constexpr int TILE = 2 * HALF;         // bytes of one [128][128] bf16 tile
constexpr int NS = 3;                  // K / V chunks in flight per CTA
constexpr int SMEM_BYTES = (1 + 2 * NS) * TILE + 1024;   // Q, K[NS], V[NS] + alignment slack
constexpr uint32_t TMEM_COLS = 512;    // S/P of group 0, of group 1: columns 0..255; O of group 0, of group 1: 256..511
constexpr int kMaxBlocksPerCta = 128;  // paged cache: chunks (= blocks) one CTA may be given
constexpr float kLazyLog2 = 8.f;        // a row's reference maximum may lag its true maximum by this much (log2)
struct Args {
    const fspad_bf16 *q, *kc, *vc, *tk, *tv;
    const int *parent, *prefix_len;
    int N, Hq, Hkv, G, M, max_len, n_splits, mtiles, use_tma;
    int longest_first;                  // the launch needs several waves of CTAs: blockIdx.z counts the sequences from the longest down
    // paged cache: the planes are pools of 128-row blocks [n_blocks][Hkv][128][d] and block_table[b][i] names
    // the block that holds rows 128 i .. 128 i + 127 of sequence b (NULL: contiguous planes)
    const int *block_table;
    int table_stride, n_blocks;
    float scale_log2;
    float *part_o, *part_ml;
    int *status;
};

// byte offset of 16-byte chunk c (0..15) of row r inside a [128][128] bf16 tile stored as two
// 128-byte-swizzled halves (columns 0..63 | 64..127), each [128 rows][128 bytes]
__device__ __forceinline__ uint32_t tile_off(int r, int c)
{
    return (uint32_t)((c >> 3) * HALF + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}


// Roles.  Warps 0-7 are the softmax warps, in two groups of four (128 threads, one query row per
// thread, a warp reaching the tensor-memory lane quarter given by its index modulo 4).  Group g
// owns keys 64 g .. 64 g + 63 of every chunk: its half of each score buffer, its own running
// reference maximum, sum and O accumulator, merged with the other group's by log-sum-exp when the
// loop ends.  Warp 8 is the copy warp: it issues every TMA copy of the loop and gathers
// the one chunk TMA cannot describe.  Warp 9 is the tensor-core warp: one of its threads issues
// every tcgen05.mma; the warp owns the tensor memory.
// Tensor memory: columns [128 p, 128 p + 128) hold the fp32 scores S of the chunks of parity p, the
// 64 columns at 128 p + 64 g being group g's, and then, written over the first 32 of those, P_g as
// packed bf16 pairs, which the second product reads directly as its A operand; columns
// [256 + 128 g, 384 + 128 g) hold O_g.
// With two score buffers the scores of chunk c + 1 are complete long before the groups have
// finished chunk c, and O_g += P V runs under the group's next softmax: a group never waits for
// the tensor cores unless it has to rescale O.
// The sides meet only on mbarriers, never on a CTA-wide barrier inside the loop:
//   kfull/vfull(b)  K / V ring slot b filled (TMA bytes, or one arrival)     tensor-core warp waits
//   kfree/vfree(b)  both S (both P V) of the chunk in slot b complete        copy warp waits
//   sfull(p)        S of a chunk of parity p complete (tcgen05.commit)       both groups wait
//   pfull(p)        P written and O rescaled by the 8 warps of both groups    tensor-core warp waits (one wait and
//                                                                            one fence for both groups' products)
//   odone(g, p)     O_g += P_g V of a chunk of parity p complete             group g waits (rescale, end)
// A new phase of a barrier can only begin after every side that waits on it has seen the previous
// one (a parity wait must never fall two phases behind).
// Tensor-core order: S(0) S(1) | PV_0(0) PV_1(0) S(2) | PV_0(1) PV_1(1) S(3) | ...
// NW: 64-bit words of a node's ancestor mask.  NW = 1 (trees of up to 64 nodes): the masks are built once per
// CTA in shared memory.  NW = 4 (up to 256 nodes): there is no shared memory left for them, so every softmax
// thread follows its own node's parent chain in global memory (a few cached loads) and keeps the mask in registers.
template <int NW>
__global__ void __launch_bounds__(NT, 1)
tree_attn_umma_kernel(const Args a, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV)
{
    extern __shared__ unsigned char smem_raw[];
    __shared__ __align__(8) unsigned long long s_bar[4 * NS + 13];
    __shared__ uint32_t s_tmem;
    __shared__ int s_fail;
    __shared__ int s_seq;
    __shared__ int s_par[NW == 1 ? FSPAD_MAX_NODES : 1];
    __shared__ int s_blk[kMaxBlocksPerCta];       // paged cache: blocks of this CTA's chunks
    __shared__ unsigned long long s_anc[NW == 1 ? FSPAD_MAX_NODES : 1];

    fspad_pdl_wait();
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool producer = warp >= 8;         // warp 8 copies, warp 9 drives the tensor cores
    const int row = tid & (BM - 1), grp = (tid >> 7) & 1;
    const int split = blockIdx.x;
    const int g = blockIdx.y / a.mtiles, mt = blockIdx.y % a.mtiles;
    int b = blockIdx.z;
    if (a.longest_first) {
        // CTAs are dispatched in index order as SMs come free, so with more CTAs than SMs the sequences
        // handled last decide the tail: they should be the short ones.  Every CTA ranks the sequences by
        // length (ties by index, so the ranks are a permutation) and takes the one whose rank is blockIdx.z.
        const int nb = (int)gridDim.z;
        for (int t = tid; t < nb; t += NT) {
            const int Lt = a.prefix_len[t];
            int rank = 0;
            for (int u = 0; u < nb; ++u) {
                const int Lu = a.prefix_len[u];
                rank += (Lu > Lt || (Lu == Lt && u < t)) ? 1 : 0;
            }
            if (rank == (int)blockIdx.z) s_seq = t;
        }
        __syncthreads();
        b = s_seq;
    }
    const int N = a.N, G = a.G, M = a.M;

    int L = a.prefix_len[b];
    if (L < 0 || L + N > a.max_len) {
        if (tid == 0) fspad_report(a.status, FSPAD_ERR_RANGE);
        L = max(0, min(L, a.max_len - N));
    }
    const int Ltot = L + N;
    const int n_chunks = (Ltot + BK - 1) / BK;
    const int per = (n_chunks + a.n_splits - 1) / a.n_splits;
    const int c0 = split * per, c1 = min(n_chunks, c0 + per);
    const int n_ch = c1 - c0;

    const int gr = mt * BM + row;                 // this thread's row among the kv head's M rows
    const bool row_ok = gr < M && !producer;
    const int node = row_ok ? gr / G : 0;
    const size_t prow = ((size_t)b * a.Hkv + g) * a.n_splits + split;

    if (c0 >= c1) {                               // nothing to do for this split: empty partial
        if (row_ok && grp == 0) { float *ml = a.part_ml + (prow * M + gr) * 2; ml[0] = -INFINITY; ml[1] = 0.f; }
        return;
    }

    // 1024-byte aligned tiles: Q | K[NS] | V[NS]
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t sQ = base, sK = base + TILE, sV = base + (1 + NS) * TILE;
    const uint32_t bar0 = smem_u32(&s_bar[0]);
    auto kfull = [&](int buf) { return bar0 + 8u * (uint32_t)buf; };
    auto vfull = [&](int buf) { return bar0 + 8u * (uint32_t)(NS + buf); };
    auto kfree = [&](int buf) { return bar0 + 8u * (uint32_t)(2 * NS + buf); };
    auto vfree = [&](int buf) { return bar0 + 8u * (uint32_t)(3 * NS + buf); };
    auto sfull = [&](int par) { return bar0 + 8u * (uint32_t)(4 * NS + par); };
    auto pfull = [&](int par) { return bar0 + 8u * (uint32_t)(4 * NS + 4 + par); };
    auto odone = [&](int grp2, int par) { return bar0 + 8u * (uint32_t)(4 * NS + 8 + 2 * grp2 + par); };
    const uint32_t drain = bar0 + 8u * (uint32_t)(4 * NS + 12);   // used only when a wait has run out
    const bool tma_ok = a.use_tma != 0;
    // The thread that issues the first TMA copies also initialises the barriers, so those copies
    // leave as soon as the prefix length is known, ahead of the CTA's first barrier.
    if (tid == 256) {
#pragma unroll
        for (int i = 0; i < 4 * NS + 13; ++i) mbar_init(bar0 + 8u * i, (i >= 4 * NS + 4 && i < 4 * NS + 6) ? 8 : 1);
        s_fail = 0;
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }

    const bool paged = a.block_table != nullptr;
    if (paged) {
        // the blocks of this CTA's chunks (a chunk is one block); an entry out of range is reported and replaced
        if (n_ch > kMaxBlocksPerCta && tid == 0) fspad_report(a.status, FSPAD_ERR_SHAPE);
        for (int i = tid; i < n_ch && i < kMaxBlocksPerCta; i += NT) {
            int blk = a.block_table[(size_t)b * a.table_stride + c0 + i];
            if (blk < 0 || blk >= a.n_blocks) { fspad_report(a.status, FSPAD_ERR_RANGE); blk = 0; }
            s_blk[i] = blk;
        }
        __syncthreads();
    }
    const int plane_row0 = (b * a.Hkv + g) * a.max_len;   // contiguous planes: first row of this kv head
    // row of the plane matrix [rows][128] that holds cache row `key` of this sequence and kv head
    // (key inside this CTA's chunks)
    auto phys_row = [&](int key) -> size_t {
        if (!paged) return (size_t)plane_row0 + (size_t)key;
        const int i = min((key >> 7) - c0, kMaxBlocksPerCta - 1);
        return ((size_t)s_blk[i] * a.Hkv + g) * 128 + (size_t)(key & 127);
    };
    const fspad_bf16 *tkb = a.tk ? a.tk + ((size_t)b * a.Hkv + g) * (size_t)N * D : nullptr;
    const fspad_bf16 *tvb = a.tv ? a.tv + ((size_t)b * a.Hkv + g) * (size_t)N * D : nullptr;
    auto is_tma = [&](int ch) { return tma_ok && (ch + 1) * BK <= L; };

    // Start the fill of an operand buffer with chunk `ch`.  A chunk inside the cached prefix comes
    // by TMA (two 64 x 128 boxes, issued by one lane of the producer warp, completion counted on
    // the buffer's mbarrier); the chunk that mixes prefix, tree rows and zero padding is gathered
    // with 16-byte asynchronous copies by the threads t0, t0 + nt, ... that the caller names (the
    // whole CTA in the prologue, the producer warp alone inside the loop).
    auto gather = [&](int ch, int buf, bool is_v, int t0, int nt) {
        const uint32_t dst = (is_v ? sV : sK) + buf * TILE;
        const fspad_bf16 *cb = is_v ? a.vc : a.kc, *tb = is_v ? tvb : tkb;
        for (int i = t0; i < BK * 16; i += nt) {
            const int r = i >> 4, c = i & 15;
            const int key = ch * BK + r;
            const bool ok = key < Ltot;
            const fspad_bf16 *src = cb;
            // prefix rows, and tree rows that live in the cache, come from the planes; explicit tree rows from their array
            if (ok) src = (key < L || tb == nullptr) ? cb + phys_row(key) * D + c * 8 : tb + (size_t)(key - L) * D + c * 8;
            cp_async16(dst + tile_off(r, c), src, ok);
        }
    };
    auto tma_fill = [&](int ch, int buf, bool is_v) {       // one lane
        const uint32_t dst = (is_v ? sV : sK) + buf * TILE;
        const uint32_t bar = is_v ? vfull(buf) : kfull(buf);
        const CUtensorMap *map = is_v ? &tmV : &tmK;
        mbar_expect_tx(bar, TILE);
        const int y = (int)phys_row(ch * BK);
        tma_load_2d(dst, map, 0, y, bar);
        tma_load_2d(dst + HALF, map, 64, y, bar);
    };

    // ---- prologue: the first NS chunks and Q go out first, the rest hides under their latency ----
#pragma unroll
    for (int u = 0; u < NS; ++u) {
        if (u >= n_ch) break;
        if (is_tma(c0 + u)) {
            if (tid == 256) { tma_fill(c0 + u, u, false); tma_fill(c0 + u, u, true); }
        } else {
            gather(c0 + u, u, false, tid, NT);
            gather(c0 + u, u, true, tid, NT);
        }
    }
    for (int i = tid; i < BM * 16; i += NT) {
        const int r = i >> 4, c = i & 15;
        const int grr = mt * BM + r;
        const bool ok = grr < M;
        const int nd = ok ? grr / G : 0, hh = ok ? grr % G : 0;
        const fspad_bf16 *src = a.q + (((size_t)b * N + nd) * a.Hq + g * G + hh) * D + c * 8;
        cp_async16(sQ + tile_off(r, c), src, ok);
    }
    cp_async_commit();
    if (NW == 1 && tid < N) s_par[tid] = a.parent[(size_t)b * N + tid];
    __syncthreads();                              // barriers initialised, parents staged
    if (warp == 9) {
        __syncwarp();
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;\n"
                     :: "r"(smem_u32(&s_tmem)), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;\n" ::: "memory");
    } else if (NW == 1 && tid < N) {
        // tree -> ancestor-or-self masks (parents were staged in shared memory above)
        unsigned long long mask = 0ull;
        int cur = tid;
        bool bad = false;
        for (int step = 0; step <= N && cur >= 0; ++step) {
            mask |= 1ull << cur;
            const int p = s_par[cur];
            if (cur == 0) { bad |= (p != -1); break; }
            if (p < 0 || p >= cur) { bad = true; break; }
            cur = p;
        }
        if (bad) fspad_report(a.status, FSPAD_ERR_BAD_TREE);
        s_anc[tid] = mask;
    }
    cp_async_wait<0>();                           // Q and any gathered chunk
    fence_async_smem();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = s_tmem;
    const uint32_t idesc_s = make_idesc(false, 128), idesc_o = make_idesc(true, 128);
    const uint32_t tO = tmem + ((uint32_t)((warp & 3) * 32) << 16) + 256u + (uint32_t)grp * 128u;   // this group's O row
    bool failed = false;
    int filled_k = min(n_ch, NS), filled_v = filled_k;   // copy warp: chunks whose K (V) fill has been started

    if (warp == 8) {
        // ================= copy warp: refills the K / V buffers =================
        // chunks gathered by the whole CTA in the prologue are announced here
        if (lane == 0) {
            for (int u = 0; u < NS && u < n_ch; ++u)
                if (!is_tma(c0 + u)) { mbar_arrive(kfull(u)); mbar_arrive(vfull(u)); }
        }
        auto fill = [&](int ch, int buf, bool is_v) {
            if (is_tma(ch)) {
                if (lane == 0) tma_fill(ch, buf, is_v);
            } else {
                gather(ch, buf, is_v, lane, 32);
                cp_async_commit();
                cp_async_wait<0>();
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(is_v ? vfull(buf) : kfull(buf));
            }
            __syncwarp();
        };
        int buf = 0;                             // i modulo NS
        uint32_t ph = 0;                         // flips each time the ring wraps
        for (int i = 0; i + NS < n_ch; ++i) {
            // the K buffer of chunk i is free once S(i) has completed, its V buffer once O += P(i) V(i) has
            if (!failed && !mbar_wait(kfree(buf), ph)) failed = true;
            if (!failed) { fill(c0 + i + NS, buf, false); ++filled_k; }
            if (!failed && !mbar_wait(vfree(buf), ph)) failed = true;
            if (!failed) { fill(c0 + i + NS, buf, true); ++filled_v; }
            if (++buf == NS) { buf = 0; ph ^= 1u; }
        }
        if (failed) s_fail = 1;
    } else if (warp == 9) {
        // ================= tensor-core warp: one thread issues every tcgen05.mma =================
        if (lane == 0) {
            const uint32_t elect = 1;             // the whole loop is this one thread's
            // low words of the shared-memory descriptors (start address and leading byte offset);
            // the high word (8-row group stride, version, swizzle mode) is the same for all
            const uint32_t hi = (uint32_t)(make_desc(0, 16) >> 32);
            const uint32_t q_lo = (uint32_t)make_desc(sQ, 16), k_lo = (uint32_t)make_desc(sK, 16);
            const uint32_t v_lo = (uint32_t)make_desc(sV, HALF);
            int kbuf = 0, vbuf = 0;              // ring slots of the next chunk to score / to multiply by V
            uint32_t kph = 0, vph = 0;           // and their phases (flip each time the ring wraps)
            // S(c) = Q K(c)^T into score buffer c & 1 (columns 0..63 of it belong to group 0, 64..127 to
            // group 1); K(c) sits in ring slot kbuf, which the second commit releases
            auto issue_s = [&](int c) {
                if (!failed && !mbar_wait_thread(kfull(kbuf), kph)) failed = true;
                if (!failed) {
                    // no tcgen05 fence here: the K chunk comes through the barrier's own acquire, and the
                    // score buffer's last readers and writers (softmax of chunk c - 2) were ordered before this
                    // thread's instructions by the fence behind its pfull wait of that chunk
                    const uint32_t kb = k_lo + (uint32_t)kbuf * (TILE >> 4);
                    const uint32_t d = tmem + (uint32_t)(c & 1) * 128u;
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) { // K = 16 per instruction over d = 128
                        const uint32_t koff = ((ks >> 2) * HALF + (ks & 3) * 32) >> 4;
                        mma_f16_lo(d, q_lo + koff, hi, kb + koff, hi, idesc_s, ks > 0, elect);
                    }
                    mma_commit_if(sfull(c & 1), elect);
                    mma_commit_if(kfree(kbuf), elect);
                }
                if (++kbuf == NS) { kbuf = 0; kph ^= 1u; }
            };
            issue_s(0);
            if (n_ch > 1) issue_s(1);
            for (int c = 0; c < n_ch; ++c) {
                const int p = c & 1;
                const uint32_t ph = (uint32_t)(c >> 1) & 1u;
                const uint32_t vb = v_lo + (uint32_t)vbuf * (TILE >> 4);
#pragma unroll
                for (int g2 = 0; g2 < 2; ++g2) {
                    // O[g2] += P_g2(c) V(c)[64 g2 .. 64 g2 + 63]: P from the four warps of group g2 (in tensor
                    // memory, over the scores it was computed from) and the V chunk
                    if (g2 == 0 && !failed && !mbar_wait_thread(pfull(p), ph)) failed = true;
                    if (g2 == 0 && !failed && !mbar_wait_thread(vfull(vbuf), vph)) failed = true;
                    if (!failed) {
                        if (g2 == 0) tc_fence_after();
                        const uint32_t a_t = tmem + (uint32_t)p * 128u + (uint32_t)g2 * 64u;
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) { // K = 16 keys per instruction = 8 columns of packed bf16 pairs
                            // V as an MN-major operand: d is contiguous, the two 64-wide halves are HALF bytes apart
                            mma_f16_ts(tmem + 256u + (uint32_t)g2 * 128u, a_t + (uint32_t)ks * 8u,
                                       vb + (uint32_t)((g2 * 64 + ks * 16) * 128 >> 4), hi, idesc_o, (c > 0) || (ks > 0), elect);
                        }
                        mma_commit_if(odone(g2, p), elect);
                        if (g2 == 1) mma_commit_if(vfree(vbuf), elect);
                    }
                }
                // tensor-core work completes in issue order, so the scores of chunk c + 2 may replace P(c)
                if (c + 2 < n_ch) issue_s(c + 2);
                if (++vbuf == NS) { vbuf = 0; vph ^= 1u; }
            }
            if (failed) s_fail = 1;
        }
        __syncwarp();
    } else {
        // ================= softmax warps =================
        const uint32_t lanes = (uint32_t)((warp & 3) * 32) << 16;
        unsigned long long anc[NW];
        if (NW == 1) {
            anc[0] = s_anc[node];
        } else {
#pragma unroll
            for (int w = 0; w < NW; ++w) anc[w] = 0ull;
            if (row_ok) {
                const int *par = a.parent + (size_t)b * N;
                int cur = node;
                bool bad = false;
                for (int step = 0; step <= N && cur >= 0; ++step) {
#pragma unroll
                    for (int w = 0; w < NW; ++w) anc[w] |= ((cur >> 6) == w) ? (1ull << (cur & 63)) : 0ull;
                    const int p = __ldg(par + cur);
                    if (cur == 0) { bad |= (p != -1); break; }
                    if (p < 0 || p >= cur) { bad = true; break; }
                    cur = p;
                }
                if (bad) fspad_report(a.status, FSPAD_ERR_BAD_TREE);
            }
        }
        // 32 bits of the mask from tree index `off` on (prefix keys, off < 0, count as set; bits beyond the mask are clear)
        auto mask_word = [&](int off) -> uint32_t {
            if (off >= 64 * NW) return 0u;
            if (off <= -32) return ~0u;
            if (off < 0) return ((1u << (-off)) - 1u) | (uint32_t)(anc[0] << (-off));
            const int w = off >> 6, sft = off & 63;
            unsigned long long lo = 0ull, hi = 0ull;
#pragma unroll
            for (int i = 0; i < NW; ++i) {
                if (i == w) lo = anc[i];
                if (i == w + 1) hi = anc[i];
            }
            unsigned long long v = lo >> sft;
            if (sft > 32) v |= hi << (64 - sft);
            return (uint32_t)v;
        };
        const float scale = a.scale_log2;
        float m_run = -INFINITY, l_run = 0.f;

        for (int c = 0; c < n_ch; ++c) {
            const int ch = c0 + c, p = c & 1;
            const uint32_t tS = tmem + lanes + (uint32_t)p * 128u + (uint32_t)grp * 64u;   // scores, then P
            if (!failed && !mbar_wait(sfull(p), (uint32_t)(c >> 1) & 1u)) failed = true;
            tc_fence_after();
            const bool masked = (ch + 1) * BK > L;   // only chunks that reach past the cached prefix
            // Validity of this group's 64 keys for this row as two 32-bit words: prefix keys are
            // valid, tree key L + t is valid iff bit t of the row's ancestor mask is set (bits at and
            // beyond the tree size are clear, which also rules out the zero padding).
            uint32_t valid[2] = {~0u, ~0u};
            if (masked) {
#pragma unroll
                for (int blk = 0; blk < 2; ++blk) {
                    const int off = ch * BK + grp * 64 + blk * 32 - L;      // tree index of the word's first key
                    valid[blk] = mask_word(off);
                }
            }
            // ---- this row's 64 scores of the group, in registers after one trip to tensor memory, with the
            // tree mask applied where it matters; the row maximum as four independent chains ----
            float v[64];
            {
                uint32_t r0[32], r1[32];
                __syncwarp();
                tmem_ld32_issue(tS, r0);
                tmem_ld32_issue(tS + 32u, r1);
                tmem_ld_wait(r0);
                tmem_ld_pin(r1);
#pragma unroll
                for (int j = 0; j < 32; ++j) { v[j] = __uint_as_float(r0[j]); v[32 + j] = __uint_as_float(r1[j]); }
            }
            if (masked) {
#pragma unroll
                for (int j = 0; j < 64; ++j)
                    if (!((valid[j >> 5] >> (j & 31)) & 1u)) v[j] = -INFINITY;
            }
            float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
            for (int j = 0; j < 64; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], v[j]);
            const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
            // The reference value m of a row (P = exp2(s * scale - m), O and the sum are relative to it)
            // only has to bound the scores loosely: it follows the row maximum when some row of the warp
            // would otherwise see a P above 2^kLazyLog2, and stays put - no pass over O - when not.
            // (The decision is taken per warp because the tensor-memory accesses are warp-collective;
            // a comparison with -inf - -inf = NaN is false and so counts as a move.)
            const float m_cand = fmaxf(m_run, mx * scale);
            const bool move = !__all_sync(0xffffffffu, m_cand - m_run <= kLazyLog2);
            const float m_new = move ? m_cand : m_run;
            const float m_safe = (m_new == -INFINITY) ? 0.f : m_new;
            const float alpha = move ? ex2f(m_run - m_safe) : 1.f;
            // ---- rescale this row of O[grp], once the group's product of the previous chunk is complete ----
            if (c >= 1 && move) {
                if (!failed && !mbar_wait(odone(grp, (c - 1) & 1), (uint32_t)((c - 1) >> 1) & 1u)) failed = true;
                tc_fence_after();
#pragma unroll
                for (int blk = 0; blk < 4; ++blk) {
                    float o[32];
                    tmem_ld32(tO + (uint32_t)blk * 32u, o);
#pragma unroll
                    for (int j = 0; j < 32; ++j) o[j] *= alpha;
                    tmem_st32(tO + (uint32_t)blk * 32u, o);
                }
            }
            // ---- P = exp2(s * scale - m) as bf16 pairs, written over the group's score columns (every score
            // is in registers by now); the row sum as four independent chains ----
            float rs4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int blk = 0; blk < 2; ++blk) {
                uint32_t w[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const float p0 = ex2f(fmaf(v[blk * 32 + 2 * e], scale, -m_safe));
                    const float p1 = ex2f(fmaf(v[blk * 32 + 2 * e + 1], scale, -m_safe));
                    rs4[e & 3] += p0 + p1;
                    w[e] = pack_bf16(p0, p1);
                }
                tmem_st16(tS + (uint32_t)blk * 16u, w);
            }
            const float rs = (rs4[0] + rs4[1]) + (rs4[2] + rs4[3]);
            l_run = l_run * alpha + rs;
            m_run = m_new;
            asm volatile("tcgen05.wait::st.sync.aligned;\n" ::: "memory");
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(pfull(p));
        }
        // ---- each group waits for its own last product (tensor-core work completes in order, so the
        // one before it is complete too); the CTA-wide barrier below then orders both accumulators
        // before the merge ----
        if (!failed && !mbar_wait(odone(grp, (n_ch - 1) & 1), (uint32_t)((n_ch - 1) >> 1) & 1u)) failed = true;
        tc_fence_after();
        if (failed) s_fail = 1;
        // the Q tile is dead (every S was issued before that product and completes before it): it
        // carries the groups' (max, sum) exchange
        float2 *s_ml = reinterpret_cast<float2 *>(smem_raw + (base - smem_u32(smem_raw)));
        s_ml[grp * BM + row] = make_float2(m_run, l_run);
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
        // ---- publish the partial: the two groups' (max, sum, O row) merged by log-sum-exp ----
        // Thread (row, grp) owns output columns grp*64 .. grp*64+63.  Every lane of every softmax warp
        // takes part in the tensor-memory loads (they are warp-collective); only the stores to global
        // memory depend on whether the lane's row exists.
        const bool any_fail = s_fail != 0;
        if (any_fail && tid == 0) fspad_report(a.status, FSPAD_ERR_TIMEOUT);
        const bool store = row_ok && !any_fail;
        const float2 ml0 = s_ml[row], ml1 = s_ml[BM + row];
        const float m_all = fmaxf(ml0.x, ml1.x);
        const float m_fin = (m_all == -INFINITY) ? 0.f : m_all;
        const float f0 = ex2f(ml0.x - m_fin), f1 = ex2f(ml1.x - m_fin);     // exp2(-inf) = 0 for a fully masked half
        // The merged rows go through shared memory (the K ring is idle by now), so that the global
        // stores are whole 512-byte rows per warp instead of 32 row-strided pieces per instruction
        // (every such piece is a transaction of its own: the direct stores cost 3 us per CTA).
        constexpr int SROW = D + 4;                   // floats per staged row; the pad keeps 16-byte stores conflict-free
        float *stg = reinterpret_cast<float *>(smem_raw + (base - smem_u32(smem_raw)) + TILE);
        float *ps = stg + row * SROW + grp * 64;
        const uint32_t tO0 = tmem + lanes + 256u + (uint32_t)grp * 64u, tO1 = tO0 + 128u;
#pragma unroll
        for (int q2 = 0; q2 < 2; ++q2) {
            float o[32], o1[32];
            tmem_ld32(tO0 + q2 * 32, o);
            tmem_ld32(tO1 + q2 * 32, o1);
#pragma unroll
            for (int j = 0; j < 32; ++j) o[j] = fmaf(o1[j], f1, o[j] * f0);
#pragma unroll
            for (int j = 0; j < 32; j += 4)
                *reinterpret_cast<float4 *>(ps + q2 * 32 + j) = make_float4(o[j], o[j + 1], o[j + 2], o[j + 3]);
        }
        if (store && grp == 0) {
            float *ml = a.part_ml + (prow * M + gr) * 2;
            ml[0] = m_all;
            ml[1] = ml0.y * f0 + ml1.y * f1;
        }
        asm volatile("bar.sync 1, 256;\n" ::: "memory");   // the eight softmax warps
        if (!any_fail) {
            for (int r = warp; r < BM; r += 8) {
                const int grr = mt * BM + r;
                if (grr < M)
                    *reinterpret_cast<float4 *>(a.part_o + (prow * M + grr) * D + lane * 4) =
                        *reinterpret_cast<const float4 *>(stg + r * SROW + lane * 4);
            }
        }
        fspad_pdl_trigger();                      // partial written: the merge kernel may start launching
        tc_fence_before();
        __syncthreads();
        return;
    }
    // copy and tensor-core warps: meet the softmax warps at their two CTA-wide barriers; the warp
    // that allocated the tensor memory then frees it
    tc_fence_before();
    __syncthreads();
    if (s_fail != 0) {
        // A wait ran out somewhere in this CTA.  Before the shared and tensor memory go back to
        // the SM, whatever was started asynchronously is given a bounded time to land: the copy warp
        // waits for the last fill it started in every ring slot, the tensor-core warp for everything
        // its thread has issued (one more commit on a barrier of its own).
        if (warp == 8) {
            for (int sl = 0; sl < NS; ++sl) {
                const int nk = (filled_k - sl + NS - 1) / NS, nv = (filled_v - sl + NS - 1) / NS;   // fills of slot sl
                if (nk > 0) (void)mbar_wait(kfull(sl), (uint32_t)(nk - 1) & 1u);
                if (nv > 0) (void)mbar_wait(vfull(sl), (uint32_t)(nv - 1) & 1u);
            }
        } else {
            mma_commit_if(drain, lane == 0);
            (void)mbar_wait(drain, 0u);
        }
    }
    __syncthreads();
    if (warp != 9) return;
    tc_fence_after();
    __syncwarp();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;\n" :: "r"(tmem), "r"(TMEM_COLS) : "memory");
}

// Self-test of the bounded wait: one warp waits, with a small cap, on a barrier that nothing ever
// arrives on; the wait must run out, the kernel records FSPAD_ERR_TIMEOUT and returns normally.
__global__ void __launch_bounds__(32)
wait_timeout_selftest_kernel(int *status, uint32_t cap)
{
    __shared__ __align__(8) unsigned long long bar;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;\n" ::: "memory");
    }
    __syncwarp();
    const bool ok = mbar_wait(smem_u32(&bar), 0u, cap);
    if (!ok && threadIdx.x == 0) fspad_report(status, FSPAD_ERR_TIMEOUT);
}

}  // namespace umma

cudaError_t fspad_launch_wait_selftest(fspad_ctx *ctx, int polls, cudaStream_t st)
{
    ctx->launches++;
    return fspad_launch_opt(false, umma::wait_timeout_selftest_kernel, dim3(1), dim3(32), 0, st, 0, ctx->d_status,
                            (uint32_t)polls);
}

int fspad_attn_umma_splits(const fspad_ctx *ctx, int N, int B, int sms)
{
    if (sms <= 0 || sms > ctx->sm_count) sms = ctx->sm_count;
    const int G = ctx->cfg.n_q_heads / ctx->cfg.n_kv_heads;
    const int mtiles = (N * G + umma::BM - 1) / umma::BM;
    const long long base = (long long)B * ctx->cfg.n_kv_heads * mtiles;
    long long s = sms / base;                     // one CTA per SM, never a partial second wave
    const int max_chunks = (ctx->cfg.max_len + umma::BK - 1) / umma::BK;
    if (s > max_chunks) s = max_chunks;
    if (s > 64) s = 64;
    if (s < 1) s = 1;
    return (int)s;
}

// ---- TMA descriptors of the K and V cache planes ----------------------------------------
// Each plane is viewed as one row-major matrix [batch * Hkv * max_len][128] bf16; a box is
// 64 columns (128 bytes, the swizzle span) by 128 rows and lands as one half tile.
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        (void)cudaGetLastError();
    }
    return fn;
}

bool fspad_make_tmap_bf16_2d(CUtensorMap *map, const fspad_bf16 *base, size_t cols, size_t rows, unsigned box_rows,
                             bool wide_l2_fetch)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn || rows == 0 || rows > 0x7fffffffull || cols == 0 || (cols * sizeof(fspad_bf16)) % 16 != 0) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)cols * sizeof(fspad_bf16)};
    const cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1u, 1u};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<fspad_bf16 *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
              wide_l2_fetch ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static bool make_plane_map(CUtensorMap *map, const fspad_bf16 *plane, size_t rows)
{
    return fspad_make_tmap_bf16_2d(map, plane, (size_t)umma::D, rows, (unsigned)umma::BK);
}

cudaError_t fspad_launch_attn_umma_split(fspad_ctx *ctx, const fspad_bf16 *q, const fspad_bf16 *kc,
                                         const fspad_bf16 *vc, const fspad_bf16 *tk, const fspad_bf16 *tv,
                                         const int *parent, const int *prefix_len, int N, int B, int n_splits,
                                         float scale_log2, cudaStream_t st, FspadPaged paged)
{
    const fspad_config &c = ctx->cfg;
    umma::Args a;
    a.q = q; a.kc = kc; a.vc = vc; a.tk = tk; a.tv = tv; a.parent = parent; a.prefix_len = prefix_len;
    a.N = N; a.Hq = c.n_q_heads; a.Hkv = c.n_kv_heads; a.G = c.n_q_heads / c.n_kv_heads;
    a.M = N * a.G; a.max_len = paged.table ? paged.stride * umma::BK : c.max_len; a.n_splits = n_splits;
    a.block_table = paged.table; a.table_stride = paged.stride; a.n_blocks = paged.n_blocks;
    a.mtiles = (a.M + umma::BM - 1) / umma::BM;
    // (every CTA ranks all sequences itself, B loads each for B / 320 of its threads: kept to batches where that is small change)
    a.longest_first = (B > 1 && B <= 128 && (long long)B * c.n_kv_heads * a.mtiles * n_splits > ctx->sm_count) ? 1 : 0;
    a.scale_log2 = scale_log2;
    a.part_o = ctx->part_o; a.part_ml = ctx->part_ml; a.status = ctx->d_status;
    if (!ctx->attn_attr_done) {
        cudaError_t e = cudaFuncSetAttribute(umma::tree_attn_umma_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             umma::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(umma::tree_attn_umma_kernel<4>, cudaFuncAttributeMaxDynamicSharedMemorySize, umma::SMEM_BYTES);
        if (e != cudaSuccess) return e;
        ctx->attn_attr_done = 1;
    }
    // descriptors are re-encoded only when a plane pointer or the batch changes
    static_assert(sizeof(CUtensorMap) <= sizeof(ctx->attn_tmap_k), "tensor map storage");
    CUtensorMap *mk = reinterpret_cast<CUtensorMap *>(ctx->attn_tmap_k);
    CUtensorMap *mv = reinterpret_cast<CUtensorMap *>(ctx->attn_tmap_v);
    // rows of the plane matrix: every sequence's cache, or the whole pool of blocks
    const size_t rows = paged.table ? (size_t)paged.n_blocks * c.n_kv_heads * umma::BK : (size_t)B * c.n_kv_heads * c.max_len;
    if (ctx->attn_tmap_kptr != kc || ctx->attn_tmap_vptr != vc || ctx->attn_tmap_rows != rows) {
        ctx->attn_tmap_ok = make_plane_map(mk, kc, rows) && make_plane_map(mv, vc, rows);
        ctx->attn_tmap_kptr = kc; ctx->attn_tmap_vptr = vc; ctx->attn_tmap_rows = rows;
    }
    a.use_tma = ctx->attn_tmap_ok ? 1 : 0;
    dim3 grid(n_splits, c.n_kv_heads * a.mtiles, B);
    ctx->launches++;
    if (N <= FSPAD_MAX_NODES)
        return fspad_launch_opt(false, umma::tree_attn_umma_kernel<1>, grid, dim3(umma::NT), umma::SMEM_BYTES, st, 0, a, *mk, *mv);
    return fspad_launch_opt(false, umma::tree_attn_umma_kernel<4>, grid, dim3(umma::NT), umma::SMEM_BYTES, st, 0, a, *mk, *mv);
}
