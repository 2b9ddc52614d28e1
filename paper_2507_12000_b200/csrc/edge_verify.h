// Host-side interface of the edge verification kernel (internal to the library).
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace dssd {

constexpr int kEdgeEndgameWaves = 3;  // EMIT claims are held back during the last so many waves of LSE tickets
constexpr int kEdgeEndgameLongRows = 8;                                  // ... with at least so many positions per sequence ...
constexpr int kEdgeEndgameLongWaves = 32;      // launches of at least so many waves ...
constexpr int kEdgeEndgameLongEighths = 7;  // ... hold them back during the last so many eighths of the waves
constexpr int kEdgeKeepLastRowGamma = 4;  // up to so many drafted positions the last row's first read carries no evict_first hint
constexpr int kEdgeConsumers = 16;      // consumer warps per CTA
constexpr int kEdgeThreads = 32 * (kEdgeConsumers + 3);  // + the producer warp, the fold warp and the scout warp
constexpr int kEdgeStageBytes = 32768;   // logits bytes per ring stage (one bulk copy)
constexpr int kEdgeStages = 6;            // ring stages per CTA
constexpr int kEdgeMaxRun = 32;           // most consecutive stages of a row in one ticket
constexpr int kEdgeEmitRun = 2;        // most stages of row n in one EMIT ticket
constexpr int kEdgeTicketsPerCta = 2;  // tickets aimed at per resident CTA

// What the emission of row P_n needs to know about a folded sequence: two 8-byte slots, each
// valid once it differs from the all-ones pattern the kernel clears the workspace to.
struct ReadySlot {
    int b;       // sequence (>= 0)
    int n;       // accepted length, or -1 if a wait ran out
    float ref2;  // row n's integer-valued reference exponent: terms are 2^(l * c1 - ref2); never NaN
    float invS;  // 1 / sum_v 2^(l_v * c1 - ref2)   (NaN for a row without finite log-sum-exp)
};

struct EdgeParams {
    // caller's arrays
    const void *logits;
    int64_t row_stride;
    const int32_t *draft_tokens;
    const float *draft_q_tok;
    const float *draft_q_rows;  // instead of draft_q_tok: the full rows [B, gamma, V]; q_i(x_i) is read out of them
    const float *uniforms;
    float temperature;
    float c1;  // log2(e) / T, rounded to float32; the kernel's temperature scaling throughout
    int B, gamma, V;
    int32_t *accept_len;
    float *p_row;          // float32 payload, or
    uint16_t *p_row16;     // IEEE binary16 payload (exactly one of the two is set)
    float *p_tok;
    float *lse;
    uint32_t *flags;
    int skip_bonus_row;    // 1: no row is emitted for fully accepted sequences (n == gamma)
    // one shard of the vocabulary (entries v_begin .. v_begin + V - 1 of every row): when shard_sum is
    // set the kernel only forms each row's partial sum, sum_v 2^(l_v c1) = shard_sum * 2^shard_ref, and
    // looks up the logits of the drafted tokens it holds; nothing is tested or emitted
    float *shard_ref;         // [B, gamma+1]
    double *shard_sum;        // [B, gamma+1]
    float *shard_tok_logit;   // [B, gamma]; NaN where the token lies outside the shard
    int v_begin;
    // ticket geometry
    int n_slices;                  // stages per row
    int lse_run, emit_run;         // stages per LSE / EMIT ticket
    int n_lse_runs, n_emit_runs;   // tickets per row
    unsigned long long total_lse;  // rows * n_lse_runs
    unsigned long long total_emit; // B * n_emit_runs
    int first_read_hint;  // 1: the first reads of the rows carry the L2 evict_first hint
    unsigned long long endgame_tickets;  // EMIT claims are held back once so few LSE tickets are left
    unsigned long long lse_magic, emit_magic;  // ceil(2^64 / n_*_runs) when multiply-high division is exact, else 0
    unsigned spin_limit;
    // test hook (0: off): the partial sums of row test_drop_row_plus1 - 1 are counted but never stored,
    // and the fold polls at most test_poll_limit times for that row's partial sums
    long long test_drop_row_plus1;
    unsigned test_poll_limit;
    // workspace, set to 0xFF by the kernel before use: counters then read "logical 0" (raw + 1)
    // and 8-byte slots read "not yet" until their one store has landed
    unsigned long long *lse_ticket;  // next LSE ticket
    unsigned long long *emit_head;   // next EMIT ticket
    unsigned *ready_count;           // sequences whose `ready` entry has been written
    unsigned *error;                 // all ones = no error
    unsigned *seq_cnt;               // [B] LSE tickets of the sequence that have arrived
    unsigned long long *part;        // [rows, n_lse_runs] (ref2, sum) of one ticket
    unsigned long long *tokz;        // [rows] (logit of the row's drafted token, 1 if the token lies in the row else 0)
    unsigned long long *tokq;        // [rows] (q_i(x_i), u_i) of the row's position, NaNs canonical
    ReadySlot *ready;                // [B] indexed by sequence
    size_t fill_bytes;
};

// Most LSE tickets a row can have for a vocabulary of V entries (any dtype, any run length).
int edge_max_runs_per_row(int V);

// Carves the workspace for `runs_per_row` partial slots per row; returns the bytes needed.
// With P == nullptr only computes the size.
size_t edge_workspace_layout(int B, int gamma, int runs_per_row, EdgeParams *P, char *base);

// Fills the geometry fields of P and launches the kernel (which clears the workspace itself) on `stream`.
cudaError_t edge_verify_launch(EdgeParams &P, int dtype, void *workspace, cudaStream_t stream);

}  // namespace dssd
