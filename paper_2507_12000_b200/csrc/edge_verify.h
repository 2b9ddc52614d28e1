// Host-side interface of the edge verification kernel (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace dssd {

constexpr int kEdgeLseSliceBytes = 32768;  // logits bytes per LSE ticket
constexpr int kEdgeEmitSlice = 8192;       // vocabulary entries per EMIT ticket

struct EdgeParams {
    // caller's arrays
    const void *logits;
    int64_t row_stride;
    const int32_t *draft_tokens;
    const float *draft_q_tok;
    const float *uniforms;
    float temperature;
    float c1;  // log2(e) / T
    int B, gamma, V;
    int32_t *accept_len;
    float *p_row;
    float *p_tok;
    float *lse;
    uint32_t *flags;
    // ticket geometry
    int lse_slice, emit_slice;        // elements per slice
    int n_lse_slices, n_emit_slices;  // slices per row
    int lse_tickets;                  // (gamma + 1) * n_lse_slices
    int lag;                          // EMIT(b) sits in ticket group b + lag
    unsigned long long tickets_per_group, total_tickets;
    unsigned spin_limit;
    // workspace
    unsigned long long *ticket;
    unsigned *error;
    unsigned *row_cnt, *seq_cnt, *seq_ready;
    float *row_M, *row_invS;
    unsigned *row_bits;  // bit0 accepted, bit1 bad token id, bit2 non-finite row
    float2 *part;        // [rows, n_lse_slices] (max, sum of 2^((z - max) * c1))
    size_t zero_bytes;
};

// Carves the workspace; returns the bytes needed.  With P == nullptr only computes the size.
size_t edge_workspace_layout(int B, int gamma, int V, int n_lse_slices, EdgeParams *P, char *base);

// Fills the geometry fields of P, clears the counters and launches the kernel on `stream`.
cudaError_t edge_verify_launch(EdgeParams &P, int dtype, void *workspace, cudaStream_t stream);

}  // namespace dssd
