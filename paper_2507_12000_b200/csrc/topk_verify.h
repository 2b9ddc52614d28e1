// Host-side interface of the truncated-support (top-k) kernels (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace dssd {

constexpr int kTopkBlock = 2048;     // vocabulary entries per scheduling block
constexpr int kTopkMergeKeys = 128;  // most keys that one row's pieces hold together
constexpr int kTopkMaxPieces = 16;   // most CTAs that share one row

struct TopkParams {
    // caller's arrays
    const void *logits;
    int64_t row_stride;
    const int32_t *draft_tokens;
    const float *draft_q_tok;
    const float *uniforms;
    float temperature;
    int B, gamma, V, k;
    int32_t *accept_len;
    int32_t *p_idx;
    float *p_val;
    float *p_tok;
    uint32_t *flags;
    // geometry: rows are cut into blocks of kTopkBlock entries, the blocks of all rows are numbered
    // row by row, and CTA c owns blocks [c * total_blocks / grid, (c + 1) * total_blocks / grid)
    int nb;                           // blocks per row
    int max_pieces;                   // list slots per row (a row is shared by at most this many CTAs)
    unsigned long long total_blocks;  // rows * nb
    int grid;
    // workspace
    unsigned *error;                  // nonzero once a bounded wait has run out (zeroed by the kernel before use)
    unsigned *seq_done;               // [B] rows of the sequence that have been judged (zeroed by the kernel before use)
    unsigned *row_done;               // [rows] pieces of the row whose lists have been published (zeroed likewise)
    unsigned *verdict;                // [rows] accepted / rejected and the row's flag bits, written when the row is judged
    unsigned long long *lists;        // [rows, max_pieces, k] candidate keys of each piece of a row; once the row has
                                      // been judged its first slot holds the row's k (index, probability) pairs
    size_t zero_bytes;
};

// slots per row for a given k (depends on k only)
int topk_max_pieces(int k);

// Carves the workspace; returns the bytes needed.  With P == nullptr only computes the size.
size_t topk_workspace_layout(int B, int gamma, int k, TopkParams *P, char *base);

// Fills the geometry, clears the counters and launches the kernel on `stream`.
cudaError_t topk_verify_launch(TopkParams &P, int dtype, void *workspace, cudaStream_t stream);

struct TopkResampleParams {
    const int32_t *p_idx;
    const float *p_val;
    const int32_t *q_idx;
    const float *q_val;
    const int32_t *accept_len;
    const float *uniforms;
    int B, gamma, k;
    int32_t *token;
    uint32_t *flags;
};

cudaError_t topk_resample_launch(const TopkResampleParams &P, cudaStream_t stream);

}  // namespace dssd
