// Dynamic token tree, final stage (paper, Section "Preliminaries", last
// paragraph: every draft step is cut to its top-k, each token carries the joint
// probability of its path, and one top-k over all tokens after the draft phase
// gives a valid tree of bounded size; Section "Performance on Fewer Candidate
// Tokens" halves both budgets).
//
// One CTA per sequence.  The candidates (at most 1024, level by level, joint
// log-probabilities that never grow along a path) are sorted in shared memory by
// a 1024-entry bitonic network over 64-bit composites (order-preserving image of
// the float in the high word, complemented candidate index in the low word; four
// entries per thread in registers, exchanges by shuffle inside a warp and through
// shared memory only for the three widest distances), so equal probabilities
// keep the lower index and parents stay ahead of their children.
// The first N - 1 entries are the kept set; one thread per kept candidate walks
// its parent chain (depth, and that every ancestor was kept), takes its
// breadth-first position by counting the kept candidates that come before it in
// (depth, index) order, and writes the flattened tree the verification step
// consumes, with (optionally) each node's ancestor-or-self mask.  Integer work throughout; no arithmetic on the probabilities.
#include "common.cuh"
#include "sort_network.cuh"

namespace {

constexpr int kThreads = kSortThreads;
constexpr int kPerThread = kSortPerThread;   // 4 entries of the sorting network per thread
static_assert(FSPAD_MAX_CANDIDATES == kSortEntries, "the network is sized for the candidate limit");

__global__ void __launch_bounds__(kThreads)
tree_build_kernel(const int *__restrict__ cand_parent, const int *__restrict__ cand_token,
                  const float *__restrict__ cand_logp, const int *__restrict__ root_token, int C, int N,
                  int *__restrict__ parent_out, int *__restrict__ token_out, int *__restrict__ cand_out,
                  unsigned long long *__restrict__ anc_out, int *__restrict__ n_out, int *__restrict__ status)
{
    __shared__ unsigned long long s_key[FSPAD_MAX_CANDIDATES];   // exchange buffer, then the sorted composites
    __shared__ short s_par[FSPAD_MAX_CANDIDATES];                // parent candidate (-1: child of the root)
    __shared__ short s_node[FSPAD_MAX_CANDIDATES];               // node number of a kept candidate, else -1
    __shared__ short s_kc[FSPAD_MAX_NODES], s_kd[FSPAD_MAX_NODES];   // kept candidates and their depths
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const int b = blockIdx.x, tid = threadIdx.x;
    const int *cp = cand_parent + (size_t)b * C;
    const float *lp = cand_logp + (size_t)b * C;
    bool bad = false;
    // thread t holds entries 4 t .. 4 t + 3 of the 1024-entry network in registers
    unsigned long long v[kPerThread];
#pragma unroll
    for (int r = 0; r < kPerThread; ++r) {
        const int c = kPerThread * tid + r;
        unsigned long long key = 0ull;                           // padding sorts behind every candidate
        int p = -1;
        if (c < C) {
            key = fspad_sort_key(lp[c], (uint32_t)c);
            p = cp[c];
            if (p < -1 || p >= c) { bad = true; p = -1; }
        }
        v[r] = key;
        s_par[c] = (short)p;
        s_node[c] = -1;
    }
    fspad_bitonic_sort_desc(v, s_key, tid);
#pragma unroll
    for (int r = 0; r < kPerThread; ++r) s_key[kPerThread * tid + r] = v[r];
    __syncthreads();
    const int want = min(N - 1, C);
    if (tid < want) s_node[fspad_key_index(s_key[tid])] = 0;   // kept (number follows)
    __syncthreads();
    int my_c = -1, my_d = 0;
    if (tid < want) {
        my_c = (int)fspad_key_index(s_key[tid]);
        for (int a = my_c; a >= 0; a = s_par[a]) {               // indices strictly decrease: the walk ends
            if (s_node[a] < 0) bad = true;                       // an ancestor was not kept
            ++my_d;
        }
        s_kc[tid] = (short)my_c;
        s_kd[tid] = (short)my_d;
    }
    __syncthreads();
    int pos = 0;
    if (tid < want) {
        pos = 1;
        for (int o = 0; o < want; ++o) {
            const int od = s_kd[o], oc = s_kc[o];
            pos += (od < my_d || (od == my_d && oc < my_c)) ? 1 : 0;
        }
        s_node[my_c] = (short)pos;
    }
    __syncthreads();
    int *po = parent_out + (size_t)b * N, *to = token_out + (size_t)b * N, *co = cand_out + (size_t)b * N;
    if (tid < want) {
        const int p = s_par[my_c];
        po[pos] = (p < 0) ? 0 : (int)s_node[p];
        to[pos] = cand_token[(size_t)b * C + my_c];
        co[pos] = my_c;
        if (anc_out) {                                           // the node, its ancestors and the root
            unsigned long long mask = 1ull;
            for (int a = my_c; a >= 0; a = s_par[a]) mask |= 1ull << s_node[a];
            anc_out[(size_t)b * N + pos] = mask;
        }
    }
    if (tid == 0) {
        po[0] = -1; to[0] = root_token[b]; co[0] = -1; n_out[b] = want + 1;
        if (anc_out) anc_out[(size_t)b * N] = 1ull;
    }
    for (int i = want + 1 + tid; i < N; i += kThreads) {
        po[i] = -1; to[i] = -1; co[i] = -1;
        if (anc_out) anc_out[(size_t)b * N + i] = 0ull;
    }
    if (bad) fspad_report(status, FSPAD_ERR_BAD_TREE);
}

}  // namespace

cudaError_t fspad_launch_tree_build(fspad_ctx *ctx, const int *cand_parent, const int *cand_token,
                                    const float *cand_logp, const int *root_token, int n_cand, int n_nodes,
                                    int B, int *parent_out, int *token_out, int *cand_out,
                                    unsigned long long *anc_out, int *n_out, cudaStream_t st)
{
    if (B == 0) return cudaSuccess;
    ctx->launches++;
    return fspad_launch(tree_build_kernel, dim3(B), dim3(kThreads), 0, st, 0, cand_parent, cand_token, cand_logp,
                        root_token, n_cand, n_nodes, parent_out, token_out, cand_out, anc_out, n_out, ctx->d_status);
}
