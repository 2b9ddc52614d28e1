// Host-side interface of the resample kernel (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace dssd {

constexpr int kResampleSub = 4096;  // vocabulary entries per chunk sum; a ticket covers one or two of them

struct ResampleParams {
    const void *p_row;   // float32 entries, or IEEE binary16 bit patterns when p_half is set
    int p_half;
    // instead of p_row (fused verification): the target logits, from which row n's probabilities are
    // formed on the fly with the (ref2, 1/S) that the edge kernel left in its workspace
    const void *logits;  // nullptr: read p_row
    int64_t row_stride;
    int logits_dtype;
    float c1;            // log2(e) / T, as the edge kernel used it
    const void *ready;   // [B] ReadySlot
    const float *draft_q;
    const int32_t *accept_len;
    const float *uniforms;
    int B, gamma, V;
    // which sequences are drawn for: 0 all; 1 only fully accepted ones (n == gamma: the bonus token
    // drawn at the edge; the others get token -1 and flags 0); 2 only rejected ones (n < gamma; the
    // entries of fully accepted sequences are left as they are)
    int select;
    int32_t *token;
    uint32_t *flags;
    int subs;       // chunk sums per ticket: 2, or 1 when there are few tickets per resident CTA
    int n_chunks;   // tickets per sequence (subs * kResampleSub entries each)
    int n_sub;      // chunk sums per sequence
    unsigned long long total_tickets;
    // scratch
    unsigned long long *ticket;       // next chunk ticket
    unsigned long long *draw_ticket;  // next sequence to draw
    double *chunk_sum;   // [B, n_sub]
    size_t fill_bytes;
    unsigned spin_limit;
    // test hook (0: off): the chunk sums of sequence test_drop_seq_plus1 - 1 are never stored, and its
    // draw polls at most test_poll_limit times for a chunk sum
    int test_drop_seq_plus1;
    unsigned test_poll_limit;
};

// Carves the scratch (its size does not depend on P->subs, which the caller sets before: 1 or 2).
size_t resample_workspace_layout(int B, int V, ResampleParams *P, char *base);

cudaError_t resample_launch(ResampleParams &P, void *workspace, cudaStream_t stream);

// ---- one shard of the vocabulary (entries v_begin .. v_begin + V - 1 of every row) ----
struct ShardResampleParams {
    const float *p_row;     // [B, V] this shard's slice of row P_n, p_stride elements between rows
    int64_t p_stride;
    const float *draft_q;   // [B, gamma, V] this shard's slice of the device's rows, q_stride elements between rows
    int64_t q_stride;
    const int32_t *accept_len;
    int B, gamma, V;
    int n_sub;              // chunk sums per sequence
    double *chunk_sum;      // scratch [B, n_sub, 2]: residual mass and plain mass of every chunk
    // mass
    double *mass;           // [B, 2] out: the slice's residual mass and plain mass
    // draw
    const double *masses;   // [G, B, 2] gathered from all shards
    int G, g, v_begin;
    const float *uniforms;
    int32_t *token;
    uint32_t *flags;
};

size_t shard_resample_workspace_bytes(int B, int V);
cudaError_t shard_mass_launch(ShardResampleParams &P, void *workspace, cudaStream_t stream);
cudaError_t shard_draw_launch(ShardResampleParams &P, const void *workspace, cudaStream_t stream);

void set_last_cuda_error(int e);  // defined with the C ABI

}  // namespace dssd
