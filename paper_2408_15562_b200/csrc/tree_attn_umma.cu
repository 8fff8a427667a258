// Tree-masked verify attention on the 5th-generation tensor cores (paper,
// Section "Preliminaries": the target processes the flattened token tree under
// the attention mask built from the tree).
//
// Split-KV flash-decode with tcgen05: all query rows that share a kv head (tree
// node x GQA group member) form the M = 128 operand of one CTA; keys are
// consumed in chunks of 128.  Per chunk: S = Q K^T is one chain of eight
// tcgen05.mma (128 x 128 x 16, bf16 -> fp32) into tensor memory; every thread
// owns one query row, reads its 128 scores back with tcgen05.ld, applies the
// ancestor mask (only on chunks that reach past the cached prefix) and the
// softmax in registers with no cross-thread traffic, and writes P as bf16 into
// a 128-byte-swizzled shared-memory tile; O += P V is a second chain of eight
// tcgen05.mma with V read directly in its [key][d] layout (MN-major operand).
// O stays in tensor memory across chunks and is rescaled there when the running
// maximum moves.  K/V chunks are double buffered with 16-byte asynchronous
// copies into the swizzled layout the matrix descriptors expect.  Per-split
// partials are merged by the combine kernel.
//
// Every wait on an mbarrier is bounded; on expiry the CTA records
// FSPAD_ERR_TIMEOUT, skips the remaining tensor-core work, frees its tensor
// memory and returns.
#include "common.cuh"

namespace umma {

constexpr int D = FSPAD_HEAD_DIM;      // 128
constexpr int BM = 128;                // query rows per CTA
constexpr int BK = 128;                // keys per chunk
constexpr int NT = 128;                // threads per CTA: one per query row
constexpr int HALF = 128 * 128;        // bytes of one [128 rows][64 bf16] half tile
constexpr int TILE = 2 * HALF;         // bytes of one [128][128] bf16 tile
constexpr int SMEM_BYTES = 6 * TILE + 1024;   // Q, K[2], V[2], P + alignment slack
constexpr uint32_t TMEM_COLS = 256;    // S: columns 0..127, O: columns 128..255
constexpr uint32_t WAIT_CAP = 4u << 20;
constexpr float kLog2e = 1.4426950408889634f;

struct Args {
    const fspad_bf16 *q, *kc, *vc, *tk, *tv;
    const int *parent, *prefix_len;
    int N, Hq, Hkv, G, M, max_len, n_splits, mtiles;
    float scale_log2;
    float *part_o, *part_ml;
    int *status;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// byte offset of 16-byte chunk c (0..15) of row r inside a [128][128] bf16 tile stored as two
// 128-byte-swizzled halves (columns 0..63 | 64..127), each [128 rows][128 bytes]
__device__ __forceinline__ uint32_t tile_off(int r, int c)
{
    return (uint32_t)((c >> 3) * HALF + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid)
{
    const int sz = valid ? 16 : 0;   // 0: destination zero-filled, source not read
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;\n" ::"r"(dst), "l"(src), "r"(sz));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N)); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;\n" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;\n" ::: "memory"); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;\n" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded wait; false if the cap ran out
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t i = 0; i < WAIT_CAP; ++i)
        if (mbar_try(bar, parity)) return true;
    return false;
}

// shared-memory matrix descriptor, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;
    d |= (uint64_t)((1024u >> 4) & 0x3FFF) << 32;
    d |= (uint64_t)1 << 46;                 // descriptor version
    d |= (uint64_t)2 << 61;                 // SWIZZLE_128B
    return d;
}
// instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = 128
__device__ __forceinline__ uint32_t make_idesc(bool b_mn_major)
{
    uint32_t d = 0;
    d |= 1u << 4;                           // accumulator fp32
    d |= 1u << 7;                           // A bf16
    d |= 1u << 10;                          // B bf16
    d |= (b_mn_major ? 1u : 0u) << 16;      // B major: 0 = K, 1 = MN
    d |= (128u >> 3) << 17;                 // N
    d |= (128u >> 4) << 24;                 // M
    return d;
}
__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                        uint32_t accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}\n"
                 :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t addr, float (&v)[32])
{
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];\n"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                   "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                   "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
                 : "r"(addr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;\n" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_st32(uint32_t addr, const float (&v)[32])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                 "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};\n"
                 :: "r"(addr),
                    "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
                    "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
                    "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
                    "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
                    "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
                    "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
                    "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
                    "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
                 : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi)
{
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t *>(&v);
}
