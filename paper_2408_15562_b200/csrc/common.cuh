// Internal declarations shared by the translation units of libfspad.so.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

#include "fspad.h"

#define FSPAD_MAX_NODES 64
#define FSPAD_HEAD_DIM 128

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
    float *part_o;            // [batch][Hkv][splits][M][d]
    float *part_ml;           // [batch][Hkv][splits][M][2]  (running max in log2 units, sum)

    // per-node vocabulary scan
    int stats_max_slices;
    float *st_pmax;           // [rows][slices]
    double *st_psum;
    int *st_parg;
    unsigned *st_counter;     // [rows], zero between calls
    float *row_max;           // [rows]
    double *row_sum;
    int *row_arg;
    int walk_cluster;         // cluster size used by the sampling walk (0 = not probed yet)

    // device staging for the host entry point
    fspad_bf16 *h_q, *h_tk, *h_tv, *h_out;
    int *h_parent, *h_prefix, *h_tokens, *h_path, *h_nacc, *h_bonus, *h_newlen;
    float *h_logits, *h_draft, *h_temp, *h_unif;
};

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
cudaError_t fspad_launch_accept_walk(fspad_ctx *ctx, const float *logits, const float *draft,
                                     const int *tokens, const int *parent, const float *temperature,
                                     const float *uniforms, int N, int B, int V, int *path,
                                     int *n_acc, int *bonus, cudaStream_t st);
cudaError_t fspad_launch_kv_compact(fspad_ctx *ctx, fspad_bf16 *cache, const int *path,
                                    const int *n_acc, const int *prefix_len, int B, int *new_len,
                                    cudaStream_t st);
cudaError_t fspad_launch_tree_attn(fspad_ctx *ctx, const fspad_bf16 *q, const fspad_bf16 *kc,
                                   const fspad_bf16 *vc, const fspad_bf16 *tk, const fspad_bf16 *tv,
                                   const int *parent, const int *prefix_len, int N, int B,
                                   fspad_bf16 *out, cudaStream_t st);
cudaError_t fspad_launch_tree_scatter(fspad_ctx *ctx, fspad_bf16 *cache, const fspad_bf16 *tk,
                                      const fspad_bf16 *tv, const int *prefix_len, int N, int B,
                                      cudaStream_t st);
int fspad_attn_splits(const fspad_ctx *ctx, int N, int B);
int fspad_stats_slices(const fspad_ctx *ctx, int rows, int V);
