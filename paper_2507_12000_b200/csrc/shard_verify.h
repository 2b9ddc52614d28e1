// Host-side interface of the kernels of the vocabulary-sharded round that have no dense
// counterpart: the combination of the shards' partial sums and the emission of one shard's slice
// of row P_n (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace dssd {

constexpr int kShardMax = 1024;  // most shards a combination takes

struct CombineParams {
    // gathered from the G shards, shard-major
    const float *part_ref;    // [G, B, gamma+1]
    const double *part_sum;   // [G, B, gamma+1]
    const float *tok_logit;   // [G, B, gamma]
    int G;
    const int32_t *draft_tokens;
    const float *draft_q_tok;
    const float *uniforms;
    float c1;  // log2(e) / T rounded to float32, as the partial sums were formed
    int B, gamma, V;  // V: the whole vocabulary
    int32_t *accept_len;
    float *row_scale;  // [B, 2]: row n's reference exponent and 1 / sum
    float *p_tok;
    float *lse;
    uint32_t *flags;
};

cudaError_t shard_combine_launch(const CombineParams &P, cudaStream_t stream);

struct EmitShardParams {
    const void *logits;  // this shard's slice of the rows
    int64_t row_stride;
    const int32_t *accept_len;
    const float *row_scale;
    float c1;
    int B, gamma, V;  // V: entries of the slice
    float *p_row;     // [B, V] with p_stride elements between rows
    int64_t p_stride;
};

cudaError_t shard_emit_launch(const EmitShardParams &P, int dtype, cudaStream_t stream);

}  // namespace dssd
