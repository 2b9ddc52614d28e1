// Host-side interface of the edge verification kernel (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace dssd {

constexpr int kEdgeVecPerLane = 8;                              // 16-byte vectors per lane per half slice
constexpr int kEdgeLseSliceBytes = 2 * 32 * 16 * kEdgeVecPerLane;  // logits bytes per LSE ticket (one warp)
constexpr int kEdgeEmitSlice = 2048;                        // vocabulary entries per EMIT ticket (one warp)
constexpr int kEdgeCtasPerSm = 2;                           // resident CTAs per SM the kernel is built for
constexpr int kEdgeEmitLagSweeps = 2;                       // EMIT trails LSE by this many tickets per resident warp

struct RowInfo {   // written by the warp that folds a row, polled by the EMIT warps
    float M;       // row maximum of the raw logits      } one 8-byte store; M is never NaN, so the
    float invS;    // 1 / sum_v exp((l_v - M) / T)       } cleared pattern (all ones) means "not yet"
    unsigned bits; // bit0 accepted, bit1 bad token id, bit2 non-finite row; all ones = "not yet"
    unsigned pad;
};

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
    // ticket geometry: group g of the list = [LSE tickets of sequence g][EMIT tickets of sequence g - lag]
    int lse_slice, emit_slice;        // elements per slice
    int n_lse_slices, n_emit_slices;  // slices per row
    int lse_tickets;                  // (gamma + 1) * n_lse_slices
    int lag;
    unsigned tickets_per_group, total_tickets;
    unsigned spin_limit;
    // workspace; everything below is filled with 0xFF before the launch, so counters start at
    // "logical 0" (raw + 1) and 8-byte slots read "not yet" until their one store has landed
    unsigned *ticket;                 // next ticket to draw
    unsigned *error;                  // all ones = no error
    unsigned *row_cnt;                // [rows] LSE tickets arrived
    RowInfo *row_info;                // [rows]
    float2 *part;                     // [rows, n_lse_slices] (max, sum of 2^((z - max) * c1))
    size_t fill_bytes;
};

// Carves the workspace; returns the bytes needed.  With P == nullptr only computes the size.
size_t edge_workspace_layout(int B, int gamma, int V, int n_lse_slices, EdgeParams *P, char *base);

// Fills the geometry fields of P, clears the workspace and launches the kernel on `stream`.
cudaError_t edge_verify_launch(EdgeParams &P, int dtype, void *workspace, cudaStream_t stream);

}  // namespace dssd
