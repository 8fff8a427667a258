// Per-node vocabulary scan: the first stage of lossless tree acceptance.
// One streaming pass over every row of the target logits gives the row
// maximum, its lowest index and the sum of exponentials at the row's
// temperature.  The strict comparison of the paper's verification stage
// (Section "Preliminaries") needs the target's result for every tree node;
// this kernel produces all of them in one HBM-bound sweep.
//
// Layout: logits [rows][V] fp32.  Grid rows*slices: a CTA owns one
// contiguous slice of one row, issues all of its 128-bit loads up front,
// reduces with warp shuffles, and the last CTA of a row to finish merges the
// row's slice partials (a self-resetting arrival counter, no second launch).
#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kBatch = 4;                 // float4 loads in flight per thread per round
constexpr float kLog2e = 1.4426950408889634f;

struct Part {
    float m;     // running maximum
    float s;     // sum of exp2((x - m) * k)
    int a;       // lowest index of the maximum
};

__device__ __forceinline__ float safe_sub(float m_old, float m_new)
{
    // (m_old - m_new) with -inf - -inf := -inf, so that an all -inf prefix scales to zero
    return (m_old == -INFINITY) ? -INFINITY : m_old - m_new;
}

__device__ __forceinline__ void merge(Part &p, const Part &o, float k)
{
    const float mn = fmaxf(p.m, o.m);
    const float sp = p.s * exp2f(safe_sub(p.m, mn) * k);
    const float so = o.s * exp2f(safe_sub(o.m, mn) * k);
    const bool take_o = (o.m > p.m) || (o.m == p.m && o.a < p.a);
    p.a = take_o ? o.a : p.a;
    p.m = mn;
    p.s = sp + so;
}

__device__ __forceinline__ void absorb4(Part &p, const float4 v, int j, float k)
{
    float bm = fmaxf(fmaxf(v.x, v.y), fmaxf(v.z, v.w));
    if (bm > p.m) {
        p.s *= exp2f(safe_sub(p.m, bm) * k);
        p.m = bm;
        p.a = (v.x == bm) ? j : (v.y == bm) ? j + 1 : (v.z == bm) ? j + 2 : j + 3;
    }
    if (p.m != -INFINITY) {
        const float m = p.m;
        p.s += exp2f((v.x - m) * k) + exp2f((v.y - m) * k) + exp2f((v.z - m) * k) +
               exp2f((v.w - m) * k);
    }
}

__device__ __forceinline__ void absorb1(Part &p, float x, int j, float k)
{
    if (x > p.m) {
        p.s *= exp2f(safe_sub(p.m, x) * k);
        p.m = x;
        p.a = j;
    }
    if (p.m != -INFINITY) p.s += exp2f((x - p.m) * k);
}

template <bool VEC4>
__global__ void __launch_bounds__(kThreads)
accept_stats_kernel(const float *__restrict__ logits, const float *__restrict__ temperature, int V,
                    int rows_per_seq, int slices, float *__restrict__ pmax, double *__restrict__ psum,
                    int *__restrict__ parg, unsigned *__restrict__ counter, float *__restrict__ row_max,
                    double *__restrict__ row_sum, int *__restrict__ row_arg)
{
    const int row = blockIdx.x / slices, slice = blockIdx.x % slices, tid = threadIdx.x;
    float T = temperature ? temperature[row / rows_per_seq] : 1.0f;
    if (!(T > 0.0f)) T = 1.0f;
    const float k = kLog2e / T;
    const float *x = logits + (size_t)row * V;

    Part p{-INFINITY, 0.0f, 0x7fffffff};
    if (VEC4) {
        const int n4 = V >> 2;
        const int per = (n4 + slices - 1) / slices;
        const int lo = slice * per, hi = min(n4, lo + per);
        const float4 *x4 = reinterpret_cast<const float4 *>(x);
        int i = lo + tid;
        for (; i + (kBatch - 1) * kThreads < hi; i += kBatch * kThreads) {
            float4 v[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u) v[u] = __ldg(x4 + i + u * kThreads);
#pragma unroll
            for (int u = 0; u < kBatch; ++u) absorb4(p, v[u], (i + u * kThreads) << 2, k);
        }
        for (; i < hi; i += kThreads) absorb4(p, __ldg(x4 + i), i << 2, k);
    } else {
        const int per = (V + slices - 1) / slices;
        const int lo = slice * per, hi = min(V, lo + per);
        for (int i = lo + tid; i < hi; i += kThreads) absorb1(p, x[i], i, k);
    }

    // warp reduction
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Part o;
        o.m = __shfl_xor_sync(0xffffffffu, p.m, off);
        o.s = __shfl_xor_sync(0xffffffffu, p.s, off);
        o.a = __shfl_xor_sync(0xffffffffu, p.a, off);
        merge(p, o, k);
    }
    __shared__ Part wp[kThreads / 32];
    __shared__ bool is_last;
    if ((tid & 31) == 0) wp[tid >> 5] = p;
    __syncthreads();
    if (tid == 0) {
        // block merge in double for the sum
        float m = wp[0].m;
        int a = wp[0].a;
        for (int w = 1; w < kThreads / 32; ++w) {
            if (wp[w].m > m || (wp[w].m == m && wp[w].a < a)) { m = wp[w].m; a = wp[w].a; }
        }
        double s = 0.0;
        for (int w = 0; w < kThreads / 32; ++w)
            s += (double)wp[w].s * (double)exp2f(safe_sub(wp[w].m, m) * k);
        const size_t slot = (size_t)row * slices + slice;
        pmax[slot] = m;
        psum[slot] = s;
        parg[slot] = a;
        __threadfence();
        const unsigned prev = atomicAdd(counter + row, 1u);
        is_last = (prev == (unsigned)slices - 1u);
        if (is_last) {
            __threadfence();
            const size_t base = (size_t)row * slices;
            float M = -INFINITY;
            int A = 0x7fffffff;
            for (int sl = 0; sl < slices; ++sl) {
                const float ms = __ldcg(pmax + base + sl);
                const int as = __ldcg(parg + base + sl);
                if (ms > M || (ms == M && as < A)) { M = ms; A = as; }
            }
            double S = 0.0;
            for (int sl = 0; sl < slices; ++sl) {
                const float ms = __ldcg(pmax + base + sl);
                S += __ldcg(psum + base + sl) * exp2((double)safe_sub(ms, M) * (double)k);
            }
            row_max[row] = M;
            row_sum[row] = S;
            row_arg[row] = (A == 0x7fffffff) ? 0 : A;
            counter[row] = 0u;       // ready for the next call
        }
    }
}

}  // namespace

int fspad_stats_slices(const fspad_ctx *ctx, int rows, int V)
{
    // about four CTAs per SM in one wave, each with at least a few KB to read
    const int target_ctas = ctx->sm_count * 4;
    int s = (target_ctas + rows - 1) / rows;
    const int max_by_size = (V + 4 * kThreads - 1) / (4 * kThreads);   // >= one float4 per thread
    if (s > max_by_size) s = max_by_size;
    if (s > ctx->stats_max_slices) s = ctx->stats_max_slices;
    if (s < 1) s = 1;
    return s;
}

cudaError_t fspad_launch_accept_stats(fspad_ctx *ctx, const float *logits, const float *temperature,
                                      int rows, int rows_per_seq, int V, float *row_max,
                                      double *row_sum, int *row_arg, cudaStream_t st)
{
    if (rows == 0) return cudaSuccess;
    const int slices = fspad_stats_slices(ctx, rows, V);
    dim3 grid((unsigned)slices * (unsigned)rows);
    const bool vec = (V % 4 == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15) == 0);
    if (vec)
        accept_stats_kernel<true><<<grid, kThreads, 0, st>>>(logits, temperature, V, rows_per_seq, slices,
                                                             ctx->st_pmax, ctx->st_psum, ctx->st_parg,
                                                             ctx->st_counter, row_max, row_sum, row_arg);
    else
        accept_stats_kernel<false><<<grid, kThreads, 0, st>>>(logits, temperature, V, rows_per_seq, slices,
                                                              ctx->st_pmax, ctx->st_psum, ctx->st_parg,
                                                              ctx->st_counter, row_max, row_sum, row_arg);
    ctx->launches++;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------
// The same scan for callers that must not allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a
// serving process whose memory pool owns the whole device and forbids outside
// allocations, or in a start-up path where an allocation (which synchronises
// the device) is not acceptable.  They cannot create an fspad_ctx, so this entry
// point needs none: the slice partials and arrival counters live in the fixed
// device array below, which every GPU that loads the library holds until the
// process exits (about 0.5 MB).
// ---------------------------------------------------------------------------
namespace {

constexpr int kNoAllocMaxRows = 1024;     // e.g. 16 sequences x 64 nodes
constexpr int kNoAllocMaxSlices = 32;
constexpr size_t kNaSlots = (size_t)kNoAllocMaxRows * kNoAllocMaxSlices;
constexpr size_t kNaOffSum = 0;                                        // double[kNaSlots]
constexpr size_t kNaOffMax = kNaOffSum + kNaSlots * sizeof(double);    // float [kNaSlots]
constexpr size_t kNaOffArg = kNaOffMax + kNaSlots * sizeof(float);     // int   [kNaSlots]
constexpr size_t kNaOffCnt = kNaOffArg + kNaSlots * sizeof(int);       // unsigned[kNoAllocMaxRows]
constexpr size_t kNaBytes = kNaOffCnt + kNoAllocMaxRows * sizeof(unsigned);

static __device__ __align__(256) unsigned char g_noalloc_scratch[kNaBytes];

constexpr int kMaxDevices = 64;
struct NoAllocDevice {
    unsigned char *scratch;   // device address of g_noalloc_scratch on this device (NULL = not set up)
    int sm_count;
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
    if (!nd.scratch) {
        // First call on this device: g_noalloc_scratch is only a host-side handle here, the
        // kernel needs the array's address in this device's memory.
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) return FSPAD_ERR_CUDA;
        if (cudaDeviceGetAttribute(&nd.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
            return FSPAD_ERR_CUDA;
        nd.scratch = static_cast<unsigned char *>(p);
    }
    int slices = (nd.sm_count * 4 + rows - 1) / rows;
    const int max_by_size = (vocab + 4 * kThreads - 1) / (4 * kThreads);
    if (slices > max_by_size) slices = max_by_size;
    if (slices > kNoAllocMaxSlices) slices = kNoAllocMaxSlices;
    if (slices < 1) slices = 1;

    cudaStream_t st = fspad_stream(stream);
    double *psum = reinterpret_cast<double *>(nd.scratch + kNaOffSum);
    float *pmax = reinterpret_cast<float *>(nd.scratch + kNaOffMax);
    int *parg = reinterpret_cast<int *>(nd.scratch + kNaOffArg);
    unsigned *counter = reinterpret_cast<unsigned *>(nd.scratch + kNaOffCnt);
    // the arrival counters must start at zero whatever an earlier call left behind
    if (cudaMemsetAsync(counter, 0, (size_t)rows * sizeof(unsigned), st) != cudaSuccess) return FSPAD_ERR_CUDA;
    dim3 grid((unsigned)slices * (unsigned)rows);
    const bool vec = (vocab % 4 == 0) && ((reinterpret_cast<uintptr_t>(logits) & 15) == 0);
    if (vec)
        accept_stats_kernel<true><<<grid, kThreads, 0, st>>>(logits, temperature, vocab, rows_per_seq, slices, pmax,
                                                             psum, parg, counter, row_max, row_sum, row_arg);
    else
        accept_stats_kernel<false><<<grid, kThreads, 0, st>>>(logits, temperature, vocab, rows_per_seq, slices, pmax,
                                                              psum, parg, counter, row_max, row_sum, row_arg);
    return cudaGetLastError() == cudaSuccess ? FSPAD_OK : FSPAD_ERR_CUDA;
}
