// Host-side interface of the edge verification kernel (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace dssd {

#ifndef DSSD_EDGE_WARPS
#define DSSD_EDGE_WARPS 8
#endif
#ifndef DSSD_EDGE_SLICE_BYTES
#define DSSD_EDGE_SLICE_BYTES 8192
#endif
#ifndef DSSD_EDGE_STAGES
#define DSSD_EDGE_STAGES 3
#endif
#ifndef DSSD_EDGE_MAX_RUN
#define DSSD_EDGE_MAX_RUN 4
#endif
#ifndef DSSD_EDGE_TICKETS_PER_WARP
#define DSSD_EDGE_TICKETS_PER_WARP 16
#endif

constexpr int kEdgeWarps = DSSD_EDGE_WARPS;            // warps per CTA; each owns a private ring
constexpr int kEdgeThreads = 32 * kEdgeWarps;
constexpr int kEdgeSliceBytes = DSSD_EDGE_SLICE_BYTES;  // logits bytes per ring stage (one bulk copy)
constexpr int kEdgeStages = DSSD_EDGE_STAGES;           // ring stages per warp
constexpr int kEdgeMaxRun = DSSD_EDGE_MAX_RUN;          // most consecutive slices of a row in one ticket
constexpr int kEdgeTicketsPerWarp = DSSD_EDGE_TICKETS_PER_WARP;  // tickets aimed at per resident warp

// Result of folding one target row; two 8-byte slots, each valid once it differs from the
// all-ones pattern the workspace is filled with before the launch.
struct RowInfo {
    float ref2;     // integer-valued reference exponent: terms are 2^(l * c1 - ref2); never NaN
    float invS;     // 1 / sum_v 2^(l_v * c1 - ref2)   (NaN for a row without finite log-sum-exp)
    unsigned bits;  // bit0 accepted, bit1 bad token id, bit2 non-finite row, bit3 wait ran out
    unsigned pad;
};

// One entry of the queue of sequences whose row P_n can be emitted; two self-validating 8-byte slots.
struct ReadySlot {
    int b;  // sequence (>= 0)
    int n;  // accepted length, or -1 if a wait ran out
    float ref2;
    float invS;
};

struct EdgeParams {
    // caller's arrays
    const void *logits;
    int64_t row_stride;
    const int32_t *draft_tokens;
    const float *draft_q_tok;
    const float *uniforms;
    float temperature;
    float c1;  // log2(e) / T, rounded to float32; the kernel's temperature scaling throughout
    int B, gamma, V;
    int32_t *accept_len;
    float *p_row;
    float *p_tok;
    float *lse;
    uint32_t *flags;
    // ticket geometry
    int n_slices;                  // slices per row
    int lse_run, emit_run;         // slices per LSE / EMIT ticket
    int n_lse_runs, n_emit_runs;   // tickets per row
    unsigned long long total_lse;  // rows * n_lse_runs
    unsigned long long total_emit; // B * n_emit_runs
    unsigned spin_limit;
    // workspace, filled with 0xFF before the launch: counters then read "logical 0" (raw + 1)
    // and 8-byte slots read "not yet" until their one store has landed
    unsigned long long *lse_ticket;  // next LSE ticket
    unsigned long long *emit_head;   // next EMIT ticket
    unsigned *ready_tail;            // sequences pushed to `ready`
    unsigned *error;                 // all ones = no error
    unsigned *row_cnt;               // [rows] LSE tickets of the row that have arrived
    unsigned *seq_cnt;               // [B] rows of the sequence that have been folded
    RowInfo *row_info;               // [rows]
    unsigned long long *part;        // [rows, n_lse_runs] (ref2, sum) of one ticket
    ReadySlot *ready;                // [B]
    size_t fill_bytes;
};

// Most LSE tickets a row can have for a vocabulary of V entries (any dtype, any run length).
int edge_max_runs_per_row(int V);

// Carves the workspace for `runs_per_row` partial slots per row; returns the bytes needed.
// With P == nullptr only computes the size.
size_t edge_workspace_layout(int B, int gamma, int runs_per_row, EdgeParams *P, char *base);

// Fills the geometry fields of P, clears the workspace and launches the kernel on `stream`.
cudaError_t edge_verify_launch(EdgeParams &P, int dtype, void *workspace, cudaStream_t stream);

}  // namespace dssd
