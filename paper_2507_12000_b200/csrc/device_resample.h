// Host-side interface of the resample kernel (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace dssd {

constexpr int kResampleChunk = 8192;  // vocabulary entries per ticket

struct ResampleParams {
    const void *p_row;   // float32 entries, or IEEE binary16 bit patterns when p_half is set
    int p_half;
    const float *draft_q;
    const int32_t *accept_len;
    const float *uniforms;
    int B, gamma, V;
    int32_t *token;
    uint32_t *flags;
    int n_chunks;   // tickets per sequence (kResampleChunk entries each)
    int n_sub;      // chunk sums per sequence (two per ticket)
    unsigned long long total_tickets;
    // scratch
    unsigned long long *ticket;       // next chunk ticket
    unsigned long long *draw_ticket;  // next sequence to draw
    double *chunk_sum;   // [B, n_sub]
    size_t fill_bytes;
    unsigned spin_limit;
};

size_t resample_workspace_layout(int B, int V, ResampleParams *P, char *base);

cudaError_t resample_launch(ResampleParams &P, void *workspace, cudaStream_t stream);

void set_last_cuda_error(int e);  // defined with the C ABI

}  // namespace dssd
