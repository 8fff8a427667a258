// Per-node vocabulary scan: the first stage of lossless tree acceptance.
// One streaming pass over every row of the target logits gives the row
// maximum, its lowest index and the sum of exponentials at the row's
// temperature.  The strict comparison of the paper's verification stage
// (Section "Preliminaries") needs the target's result for every tree node;
// this kernel produces all of them in one HBM-bound sweep.
//
// Layout: logits [rows][V] fp32, viewed as one flat array that is cut into
// equal contiguous ranges, one per CTA (1024 threads per SM in a single wave:
// CTAs of 128 threads for a small array, of 256 otherwise), so the load is
// balanced whatever rows and V are.  Where the sizes allow, the ranges are cut at
// the rows; otherwise a range may cross row boundaries and runs the reductions
// once per row it touches.  Each (row, CTA) piece yields one partial (max, argmax, sum).
// A thread works in batches of four 128-bit loads, with the next batch already
// in flight: it takes the maximum of the 16 values in registers, rescales its
// running sum once and adds the 16 exponentials: no per-element branch.  Partials are merged per
// row by whoever needs them (the acceptance walk for the rows it visits, or
// the small merge kernel behind fspad_accept_stats).
#include <atomic>

#include "common.cuh"

namespace {

constexpr int kThreads = FSPAD_STATS_THREADS;   // 256; small arrays are scanned by CTAs of half that
constexpr int kDeep = 4;                  // load units per batch per thread (two batches in flight)
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct Acc {
    float m, s;
    int a;
};

__device__ __forceinline__ void acc_merge(Acc &p, float om, float os, float k)
{
    const float mn = fmaxf(p.m, om);
    const float sp = (p.m == -INFINITY) ? 0.f : p.s * ex2((p.m - mn) * k);
    const float so = (om == -INFINITY) ? 0.f : os * ex2((om - mn) * k);
    p.m = mn;
    p.s = sp + so;
}

// one load unit: a float4 (UNIT == 4) or a float (UNIT == 1)
template <int UNIT> struct Unit;
template <> struct Unit<4> {
    typedef float4 T;
    static __device__ __forceinline__ T pad() { return make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY); }
    static __device__ __forceinline__ float vmax(const T &v) { return fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w)); }
    static __device__ __forceinline__ float vsum(const T &v, float m, float k)
    {
        return (ex2((v.x - m) * k) + ex2((v.y - m) * k)) + (ex2((v.z - m) * k) + ex2((v.w - m) * k));
    }
    // lowest position inside the unit equal to bm, or keep `a`
    static __device__ __forceinline__ int first_eq(const T &v, float bm, int j, int a)
    {
        if (v.w == bm) a = j + 3;
        if (v.z == bm) a = j + 2;
        if (v.y == bm) a = j + 1;
        if (v.x == bm) a = j;
        return a;
    }
};
template <> struct Unit<1> {
    typedef float T;
    static __device__ __forceinline__ T pad() { return -INFINITY; }
    static __device__ __forceinline__ float vmax(const T &v) { return v; }
    static __device__ __forceinline__ float vsum(const T &v, float m, float k) { return ex2((v - m) * k); }
    static __device__ __forceinline__ int first_eq(const T &v, float bm, int j, int a) { return v == bm ? j : a; }
};

template <int UNIT, int kThreads>
__global__ void __launch_bounds__(kThreads, 1024 / kThreads)
accept_stats_kernel(const float *__restrict__ logits, const float *__restrict__ temperature,
                    int rows_per_seq, const FspadStatsGeom g, FspadStatsPart *__restrict__ parts)
{
    typedef typename Unit<UNIT>::T U;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const long long lo = (long long)blockIdx.x * g.chunk;
    const long long hi = min(g.total, lo + g.chunk);
    __shared__ Acc wacc[kThreads / 32];
    __shared__ float s_bmax;
    __shared__ int s_barg;
    // Wait first, then let the successor start: a kernel that follows this one in the stream (the
    // acceptance walk) can then rely on everything queued before the scan having completed, and may
    // read the caller's arrays, which the scan never writes, while the scan is still running.
    fspad_pdl_wait();
    fspad_pdl_trigger();

    long long seg_lo = lo;
    while (seg_lo < hi) {
        const int row = (int)(seg_lo / g.upr);
        const long long row_lo = (long long)row * g.upr;
        const long long seg_hi = min(hi, row_lo + g.upr);
        const int n = (int)(seg_hi - seg_lo);                 // units in this piece of the row
        const int off = (int)(seg_lo - row_lo);               // position of the piece inside the row
        const U *px = reinterpret_cast<const U *>(logits) + seg_lo;
        float T = temperature ? temperature[row / rows_per_seq] : 1.0f;
        if (!(T > 0.0f)) T = 1.0f;
        const float k = kLog2e / T;

        // software pipeline: the next batch of loads is in flight while this one is reduced
        Acc p{-INFINITY, 0.f, 0x7fffffff};
        U cur[kDeep], nxt[kDeep];
#pragma unroll
        for (int u = 0; u < kDeep; ++u) {
            const int i = u * kThreads + tid;
            cur[u] = (i < n) ? __ldg(px + i) : Unit<UNIT>::pad();
        }
        for (int base = 0; base < n; base += kThreads * kDeep) {
            const int nb = base + kThreads * kDeep;
            if (nb < n) {
#pragma unroll
                for (int u = 0; u < kDeep; ++u) {
                    const int i = nb + u * kThreads + tid;
                    nxt[u] = (i < n) ? __ldg(px + i) : Unit<UNIT>::pad();
                }
            }
            float bm = Unit<UNIT>::vmax(cur[0]);
#pragma unroll
            for (int u = 1; u < kDeep; ++u) bm = fmaxf(bm, Unit<UNIT>::vmax(cur[u]));
            if (bm > p.m) {
                // only the batch is remembered; the position inside it is looked up once, at the
                // end, by the threads that hold the block's maximum
                p.s = (p.m == -INFINITY) ? 0.f : p.s * ex2((p.m - bm) * k);
                p.m = bm;
                p.a = base;
            }
            if (p.m != -INFINITY) {
                float s0 = 0.f;
#pragma unroll
                for (int u = 0; u < kDeep; ++u) s0 += Unit<UNIT>::vsum(cur[u], p.m, k);
                p.s += s0;
            }
            if (nb < n) {
#pragma unroll
                for (int u = 0; u < kDeep; ++u) cur[u] = nxt[u];
            }
        }
        // block reduction of (m, s); then the lowest index of the block's maximum
        const float my_m = p.m;
        const int my_base = p.a;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, p.m, o);
            const float os = __shfl_xor_sync(0xffffffffu, p.s, o);
            acc_merge(p, om, os, k);
        }
        if (lane == 0) wacc[wid] = p;
        if (tid == 0) s_barg = 0x7fffffff;
        __syncthreads();
        if (wid == 0) {
            Acc q = (lane < kThreads / 32) ? wacc[lane] : Acc{-INFINITY, 0.f, 0};
#pragma unroll
            for (int o = kThreads / 64; o > 0; o >>= 1) {
                const float om = __shfl_xor_sync(0xffffffffu, q.m, o);
                const float os = __shfl_xor_sync(0xffffffffu, q.s, o);
                acc_merge(q, om, os, k);
            }
            if (lane == 0) { wacc[0] = q; s_bmax = q.m; }
        }
        __syncthreads();
        const float bmax = s_bmax;
        if (my_m == bmax && bmax != -INFINITY) {
            // this thread's batch `my_base` holds the maximum: fetch it again (cache hit) and scan it
            int a = 0x7fffffff;
#pragma unroll
            for (int u = kDeep - 1; u >= 0; --u) {
                const int i = my_base + u * kThreads + tid;
                if (i < n) a = Unit<UNIT>::first_eq(__ldg(px + i), bmax, (off + i) * UNIT, a);
            }
            atomicMin(&s_barg, a);
        }
        __syncthreads();
        if (tid == 0) {
            const int first = (int)(row_lo / g.chunk);
            FspadStatsPart out;
            out.m = wacc[0].m; out.s = wacc[0].s; out.a = s_barg; out.pad = 0;
            parts[(size_t)row * g.slots + (blockIdx.x - first)] = out;
        }
        __syncthreads();
        seg_lo = seg_hi;
    }
}

// rows -> (max, sum, argmax) from the partials; one warp per row
__global__ void __launch_bounds__(128)
accept_stats_merge_kernel(const FspadStatsPart *__restrict__ parts, const FspadStatsGeom g,
                          const float *__restrict__ temperature, int rows, int rows_per_seq,
                          float *__restrict__ row_max, double *__restrict__ row_sum, int *__restrict__ row_arg)
{
    fspad_pdl_trigger();
    fspad_pdl_wait();
    const int lane = threadIdx.x & 31;
    const int row = blockIdx.x * 4 + (threadIdx.x >> 5);
    if (row >= rows) return;
    float T = temperature ? temperature[row / rows_per_seq] : 1.0f;
    if (!(T > 0.0f)) T = 1.0f;
    float M;
    double S;
    int A;
    fspad_stats_merge_warp(parts, g, row, kLog2e / T, lane, M, S, A);
    if (lane == 0) {
        row_max[row] = M;
        row_sum[row] = S;
        row_arg[row] = A;
    }
}

cudaError_t launch_partials(const float *logits, const float *temperature, int rows_per_seq,
                            const FspadStatsGeom &g, FspadStatsPart *parts, cudaStream_t st, bool pdl = true)
{
    if (g.threads == kThreads / 2) {
        if (g.unit == 4)
            return fspad_launch_opt(pdl, accept_stats_kernel<4, kThreads / 2>, dim3(g.n_cta), dim3(kThreads / 2), 0, st, 0, logits,
                                    temperature, rows_per_seq, g, parts);
        return fspad_launch_opt(pdl, accept_stats_kernel<1, kThreads / 2>, dim3(g.n_cta), dim3(kThreads / 2), 0, st, 0, logits,
                                temperature, rows_per_seq, g, parts);
    }
    if (g.unit == 4)
        return fspad_launch_opt(pdl, accept_stats_kernel<4, kThreads>, dim3(g.n_cta), dim3(kThreads), 0, st, 0, logits, temperature,
                            rows_per_seq, g, parts);
    return fspad_launch_opt(pdl, accept_stats_kernel<1, kThreads>, dim3(g.n_cta), dim3(kThreads), 0, st, 0, logits, temperature,
                            rows_per_seq, g, parts);
}

}  // namespace

cudaError_t fspad_launch_stats_partials(fspad_ctx *ctx, const float *logits, const float *temperature,
                                        int rows, int rows_per_seq, int V, FspadStatsGeom *geom,
                                        cudaStream_t st, bool pdl, int sms)
{
    const bool vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15) == 0);
    if (sms <= 0 || sms > ctx->sm_count) sms = ctx->sm_count;
    *geom = fspad_stats_geom(sms, rows, V, vec, ctx->stats_slots, true);
    ctx->launches++;
    return launch_partials(logits, temperature, rows_per_seq, *geom, ctx->st_part, st, pdl);
}

cudaError_t fspad_launch_accept_stats(fspad_ctx *ctx, const float *logits, const float *temperature,
                                      int rows, int rows_per_seq, int V, float *row_max,
                                      double *row_sum, int *row_arg, cudaStream_t st)
{
    if (rows == 0) return cudaSuccess;
    FspadStatsGeom g;
    cudaError_t e = fspad_launch_stats_partials(ctx, logits, temperature, rows, rows_per_seq, V, &g, st);
    if (e != cudaSuccess) return e;
    ctx->launches++;
    return fspad_launch(accept_stats_merge_kernel, dim3((rows + 3) / 4), dim3(128), 0, st, 0,
                        (const FspadStatsPart *)ctx->st_part, g, temperature, rows, rows_per_seq, row_max, row_sum,
                        row_arg);
}

// ---------------------------------------------------------------------------
// The same scan for callers that must not allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a
// serving process whose memory pool owns the whole device and forbids outside
// allocations, or in a start-up path where an allocation (which synchronises
// the device) is not acceptable.  They cannot create an fspad_ctx, so this entry
// point needs none: the per-CTA partials live in the fixed device array below,
// which every GPU that loads the library holds until the process exits (0.5 MB).
// ---------------------------------------------------------------------------
namespace {

constexpr int kNoAllocMaxRows = 1024;     // e.g. 16 sequences x 64 nodes
constexpr int kNoAllocSlots = 32;         // partial slots per row
constexpr size_t kNaBytes = (size_t)kNoAllocMaxRows * kNoAllocSlots * sizeof(FspadStatsPart);

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNaBytes];

constexpr int kMaxDevices = 64;
struct NoAllocDevice {
    std::atomic<unsigned char *> scratch;   // device address of g_noalloc_scratch on this device (NULL = not set up)
    int sm_count;                            // written before `scratch` is published
};
NoAllocDevice g_na_dev[kMaxDevices];

}  // namespace

extern "C" int fspad_accept_stats_noalloc(const float *logits, const float *temperature, int rows,
                                          int rows_per_seq, int vocab, float *row_max, double *row_sum,
                                          int32_t *row_arg, void *stream)
{
    if (!logits || !row_max || !row_sum || !row_arg) return FSPAD_ERR_NULL;
    if (rows < 0 || rows_per_seq < 1 || vocab < 1) return FSPAD_ERR_SHAPE;
    if (rows > kNoAllocMaxRows) return FSPAD_ERR_TOO_LARGE;
    if (rows == 0) return FSPAD_OK;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return FSPAD_ERR_CUDA;
    NoAllocDevice &nd = g_na_dev[dev];
    unsigned char *scratch = nd.scratch.load(std::memory_order_acquire);
    if (!scratch) {
        // First call on this device: g_noalloc_scratch is only a host-side handle here, the
        // kernels need the array's address in this device's memory.  Host threads that race on
        // this first call all compute the same two values; the address is published last, so a
        // thread that sees it also sees the SM count.
        void *p = nullptr;
        int sms = 0;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return FSPAD_ERR_CUDA;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1)
            return FSPAD_ERR_CUDA;
        nd.sm_count = sms;
        scratch = static_cast<unsigned char *>(p);
        nd.scratch.store(scratch, std::memory_order_release);
    }
    cudaStream_t st = fspad_stream(stream);
    const bool vec = (vocab % 4 == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15) == 0);
    const FspadStatsGeom g = fspad_stats_geom(nd.sm_count, rows, vocab, vec, kNoAllocSlots);
    FspadStatsPart *parts = reinterpret_cast<FspadStatsPart *>(scratch);
    // every slot the merge reads is rewritten by this call's first kernel, so the contents an
    // earlier call left in the shared array never need clearing
    if (launch_partials(logits, temperature, rows_per_seq, g, parts, st) != cudaSuccess) return FSPAD_ERR_CUDA;
    return fspad_launch(accept_stats_merge_kernel, dim3((rows + 3) / 4), dim3(128), 0, st, 0,
                        (const FspadStatsPart *)parts, g, temperature, rows, rows_per_seq, row_max, row_sum,
                        (int *)row_arg) == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}
