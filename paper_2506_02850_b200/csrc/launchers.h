// Host-side launch helpers shared between translation units of the METok library.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace metok {

// Class-wise top-k + ascending keep list, one cluster per problem p in [0, problems):
// scores + p*score_stride, keep_idx + p*keep_stride, counts written to count_a[p]
// and count_b[p] (either may be null).  token_group may be null (single class).
// budgets_host is a HOST array of G ints.  With replicas > 1 (problems == 1) the one
// list and its length are written `replicas` times, keep_stride apart.
int launch_class_topk(const float* scores, size_t score_stride, const int32_t* token_group, int n_vis, int G,
                      const int32_t* budgets_host, int S, int vis_start, int32_t* keep_idx, size_t keep_stride,
                      int replicas, int32_t* count_a, int32_t* count_b, int problems, cudaStream_t st);

// dst[i] = src[idx[i]] for i < *n_rows (device scalar), by bulk copies through shared memory; rows of
// any multiple of 16 bytes; src has src_rows rows.  timer_name labels the launch in the per-kernel
// timing report.  `status` receives METOK_ERR_TIMEOUT if a device-side wait gave up.
int launch_gather_rows_bulk(const void* src, void* dst, const int32_t* idx, const int32_t* n_rows, size_t row_bytes,
                            int src_rows, int32_t* status, const char* timer_name, cudaStream_t st);

// Text->visual attention scores on the tensor cores (bf16, dh 64 or 128): leaves
// n_planes partial column sums of n_vis floats each in part_col; their sum divided by
// Hq*Lt is the score.  attn_mma_workspace gives the element counts of part_m / part_l
// (each) and of part_col.  `status` receives METOK_ERR_TIMEOUT if a device-side wait gave up.
void attn_mma_workspace(int Hq, int Hkv, int Lt, int S, int n_vis, size_t* n_part_ml, size_t* n_part_col,
                        int* n_planes);
int launch_attn_scores_mma(const void* q_text, const void* k_all, int Hq, int Hkv, int Lt, int S, int dh,
                           int vis_start, int n_vis, float scale, float* part_m, float* part_l, float* part_col,
                           int32_t* status, cudaStream_t st);

}  // namespace metok
