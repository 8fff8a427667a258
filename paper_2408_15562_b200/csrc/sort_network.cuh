// A 1024-entry bitonic sorting network for one CTA of 256 threads, descending, over 64-bit keys.
// Thread t holds entries 4 t .. 4 t + 3 in registers.  Partners 1 or 2 apart sit in the same
// thread, partners up to 64 apart in the same warp (shuffles); only the three widest distances
// (128, 256, 512) go through the 8 KB shared-memory buffer `buf`, with a CTA barrier on each side.
// Used by the tree builder (joint probabilities of candidates) and by the draft step (per-row and
// per-sequence top-k).  Keys are composites: an order-preserving image of a float in the high word,
// the complemented index in the low word, so equal values keep the lower index; 0 is the padding
// key and sorts behind everything else.
#pragma once
#include <stdint.h>

constexpr int kSortEntries = 1024;
constexpr int kSortThreads = 256;
constexpr int kSortPerThread = kSortEntries / kSortThreads;

// order-preserving map float -> uint32 (larger float, larger integer)
__device__ __forceinline__ uint32_t fspad_orderable(float f)
{
    const uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float fspad_from_orderable(uint32_t o)
{
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7fffffffu) : ~o);
}
__device__ __forceinline__ unsigned long long fspad_sort_key(float value, uint32_t index)
{
    // value + 0.0f turns -0.0 into +0.0, so the two zeros compare equal as they do for the float itself
    return ((unsigned long long)fspad_orderable(value + 0.0f) << 32) | (unsigned long long)(0xffffffffu - index);
}
__device__ __forceinline__ uint32_t fspad_key_index(unsigned long long key)
{
    return 0xffffffffu - (uint32_t)(key & 0xffffffffull);
}
__device__ __forceinline__ float fspad_key_value(unsigned long long key)
{
    return fspad_from_orderable((uint32_t)(key >> 32));
}

// Every thread of the CTA calls it; on return v[] holds the thread's slice of the sorted sequence.
__device__ __forceinline__ void fspad_bitonic_sort_desc(unsigned long long (&v)[kSortPerThread],
                                                        unsigned long long *buf, int tid)
{
    for (int k = 2; k <= kSortEntries; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            if (j < kSortPerThread) {
#pragma unroll
                for (int r = 0; r < kSortPerThread; ++r) {
                    const int l = r ^ j;
                    if (l > r) {
                        const bool desc = ((kSortPerThread * tid + r) & k) == 0;
                        const unsigned long long x = v[r], y = v[l];
                        if (desc ? (x < y) : (x > y)) { v[r] = y; v[l] = x; }
                    }
                }
            } else {
                unsigned long long o[kSortPerThread];
                if (j < kSortPerThread * 32) {
#pragma unroll
                    for (int r = 0; r < kSortPerThread; ++r) o[r] = __shfl_xor_sync(0xffffffffu, v[r], j / kSortPerThread);
                } else {
                    __syncthreads();                             // the buffer's previous readers are done
#pragma unroll
                    for (int r = 0; r < kSortPerThread; ++r) buf[kSortPerThread * tid + r] = v[r];
                    __syncthreads();
                    const int pt = tid ^ (j / kSortPerThread);
#pragma unroll
                    for (int r = 0; r < kSortPerThread; ++r) o[r] = buf[kSortPerThread * pt + r];
                }
                const int i0 = kSortPerThread * tid;
                const bool lower = (i0 & j) == 0, desc = (i0 & k) == 0;   // same for the thread's four entries
                const bool take_max = lower == desc;
#pragma unroll
                for (int r = 0; r < kSortPerThread; ++r)
                    v[r] = take_max ? (v[r] > o[r] ? v[r] : o[r]) : (v[r] < o[r] ? v[r] : o[r]);
            }
        }
    }
    __syncthreads();
}
