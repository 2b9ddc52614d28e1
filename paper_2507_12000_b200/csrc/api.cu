// C ABI of the library: argument checks, workspace carving, launches.  See include/dssd.h.
#include <cuda_runtime.h>
#include <math.h>

#include "device_resample.h"
#include "dssd.h"
#include "dssd_test_hooks.h"
#include "edge_verify.h"
#include "shard_verify.h"
#include "topk_verify.h"

namespace {

thread_local int t_last_cuda_error = 0;

dssd_status cuda_fail(cudaError_t e)
{
    t_last_cuda_error = (int)e;
    return DSSD_ERR_CUDA;
}

// 0 = fine, else the status to return
dssd_status check_sizes(int B, int gamma, int V)
{
    if (B < 1 || gamma < 0 || V < 1) return DSSD_ERR_INVALID_ARG;
    if (V > DSSD_MAX_V) return DSSD_ERR_UNSUPPORTED;
    if ((long long)B * ((long long)gamma + 1) > (long long)DSSD_MAX_ROWS) return DSSD_ERR_UNSUPPORTED;
    return DSSD_OK;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace

namespace dssd {
// lets entry points defined in other files of the library report through dssd_last_cuda_error()
void set_last_cuda_error(int e) { t_last_cuda_error = e; }
}  // namespace dssd

extern "C" {

const char *dssd_status_string(int status)
{
    switch (status) {
        case DSSD_OK: return "DSSD_OK";
        case DSSD_ERR_INVALID_ARG: return "DSSD_ERR_INVALID_ARG";
        case DSSD_ERR_UNSUPPORTED: return "DSSD_ERR_UNSUPPORTED";
        case DSSD_ERR_WORKSPACE: return "DSSD_ERR_WORKSPACE";
        case DSSD_ERR_CUDA: return "DSSD_ERR_CUDA";
        default: return "DSSD_ERR_UNKNOWN";
    }
}

int dssd_version(void) { return 100; }

int dssd_last_cuda_error(void) { return t_last_cuda_error; }

size_t dssd_edge_verify_workspace_bytes(int B, int gamma, int V)
{
    if (check_sizes(B, gamma, V) != DSSD_OK) return 0;
    return dssd::edge_workspace_layout(B, gamma, dssd::edge_max_runs_per_row(V), nullptr, nullptr);
}

namespace {
dssd_status edge_verify_any(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                            const int32_t *draft_tokens, const float *draft_q_tok, const float *uniforms,
                            float temperature, int B, int gamma, int V, int32_t *accept_len, float *p_row,
                            uint16_t *p_row16, float *p_tok, float *lse, uint32_t *flags, void *workspace,
                            size_t workspace_bytes, void *cuda_stream, long long drop_row_plus1 = 0,
                            unsigned poll_limit = 0)
{
    t_last_cuda_error = 0;
    dssd_status st = check_sizes(B, gamma, V);
    if (st != DSSD_OK) return st;
    if (dtype != DSSD_F32 && dtype != DSSD_BF16) return DSSD_ERR_UNSUPPORTED;
    if (!target_logits || !accept_len || (!p_row && !p_row16)) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && (!draft_tokens || !draft_q_tok || !uniforms)) return DSSD_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !isfinite(temperature)) return DSSD_ERR_INVALID_ARG;
    if (row_stride < (int64_t)V) return DSSD_ERR_INVALID_ARG;
    const size_t esz = dtype == DSSD_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(target_logits) % esz) || (reinterpret_cast<uintptr_t>(p_row) % 4) ||
        (reinterpret_cast<uintptr_t>(p_row16) % 2))
        return DSSD_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < dssd_edge_verify_workspace_bytes(B, gamma, V))
        return DSSD_ERR_WORKSPACE;

    dssd::EdgeParams P{};
    P.logits = target_logits;
    P.row_stride = row_stride;
    P.draft_tokens = draft_tokens;
    P.draft_q_tok = draft_q_tok;
    P.uniforms = uniforms;
    P.temperature = temperature;
    P.B = B;
    P.gamma = gamma;
    P.V = V;
    P.accept_len = accept_len;
    P.p_row = p_row;
    P.p_row16 = p_row16;
    P.p_tok = p_tok;
    P.lse = lse;
    P.flags = flags;
    P.test_drop_row_plus1 = drop_row_plus1;
    P.test_poll_limit = poll_limit;
    cudaError_t e = dssd::edge_verify_launch(P, (int)dtype, workspace, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}
}  // namespace

dssd_status dssd_test_edge_verify_wait_runs_out(const void *target_logits, dssd_dtype dtype,
                                                int64_t row_stride, const int32_t *draft_tokens,
                                                const float *draft_q_tok, const float *uniforms,
                                                float temperature, int B, int gamma, int V,
                                                int32_t *accept_len, float *p_row, uint32_t *flags,
                                                void *workspace, size_t workspace_bytes,
                                                long long drop_row, unsigned poll_limit,
                                                void *cuda_stream)
{
    if (!p_row) return DSSD_ERR_INVALID_ARG;
    if (check_sizes(B, gamma, V) == DSSD_OK && (drop_row < 0 || drop_row >= (long long)B * (gamma + 1))) return DSSD_ERR_INVALID_ARG;
    return edge_verify_any(target_logits, dtype, row_stride, draft_tokens, draft_q_tok, uniforms, temperature, B, gamma,
                           V, accept_len, p_row, nullptr, nullptr, nullptr, flags, workspace, workspace_bytes, cuda_stream,
                           drop_row + 1, poll_limit);
}

dssd_status dssd_edge_verify(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                             const int32_t *draft_tokens, const float *draft_q_tok,
                             const float *uniforms, float temperature, int B, int gamma, int V,
                             int32_t *accept_len, float *p_row, float *p_tok, float *lse,
                             uint32_t *flags, void *workspace, size_t workspace_bytes,
                             void *cuda_stream)
{
    if (!p_row) return DSSD_ERR_INVALID_ARG;
    return edge_verify_any(target_logits, dtype, row_stride, draft_tokens, draft_q_tok, uniforms, temperature, B, gamma,
                           V, accept_len, p_row, nullptr, p_tok, lse, flags, workspace, workspace_bytes, cuda_stream);
}

dssd_status dssd_edge_verify_p16(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                                 const int32_t *draft_tokens, const float *draft_q_tok,
                                 const float *uniforms, float temperature, int B, int gamma, int V,
                                 int32_t *accept_len, uint16_t *p_row16, float *p_tok, float *lse,
                                 uint32_t *flags, void *workspace, size_t workspace_bytes,
                                 void *cuda_stream)
{
    if (!p_row16) return DSSD_ERR_INVALID_ARG;
    return edge_verify_any(target_logits, dtype, row_stride, draft_tokens, draft_q_tok, uniforms, temperature, B, gamma,
                           V, accept_len, nullptr, p_row16, p_tok, lse, flags, workspace, workspace_bytes, cuda_stream);
}

size_t dssd_device_resample_workspace_bytes(int B, int gamma, int V)
{
    if (check_sizes(B, gamma, V) != DSSD_OK) return 0;
    return dssd::resample_workspace_layout(B, V, nullptr, nullptr);
}

namespace {
dssd_status device_resample_any(const void *p_row, int p_half, const float *draft_q, const int32_t *accept_len,
                                const float *uniforms, int B, int gamma, int V, int32_t *token, uint32_t *flags,
                                void *workspace, size_t workspace_bytes, void *cuda_stream, int select = 0,
                                int drop_seq_plus1 = 0, unsigned poll_limit = 0)
{
    t_last_cuda_error = 0;
    dssd_status st = check_sizes(B, gamma, V);
    if (st != DSSD_OK) return st;
    if (!p_row || !accept_len || !uniforms || !token) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && !draft_q) return DSSD_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(p_row) % (p_half ? 2 : 4)) || (reinterpret_cast<uintptr_t>(draft_q) % 4))
        return DSSD_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < dssd_device_resample_workspace_bytes(B, gamma, V))
        return DSSD_ERR_WORKSPACE;

    dssd::ResampleParams P{};
    P.p_row = p_row;
    P.p_half = p_half;
    P.draft_q = draft_q;
    P.accept_len = accept_len;
    P.uniforms = uniforms;
    P.B = B;
    P.gamma = gamma;
    P.V = V;
    P.select = select;
    P.token = token;
    P.flags = flags;
    P.test_drop_seq_plus1 = drop_seq_plus1;
    P.test_poll_limit = poll_limit;
    cudaError_t e = dssd::resample_launch(P, workspace, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}
}  // namespace

dssd_status dssd_test_device_resample_wait_runs_out(const float *p_row, const float *draft_q,
                                                    const int32_t *accept_len,
                                                    const float *uniforms, int B, int gamma, int V,
                                                    int32_t *token, uint32_t *flags,
                                                    void *workspace, size_t workspace_bytes,
                                                    int drop_seq, unsigned poll_limit,
                                                    void *cuda_stream)
{
    if (B >= 1 && (drop_seq < 0 || drop_seq >= B)) return DSSD_ERR_INVALID_ARG;
    return device_resample_any(p_row, 0, draft_q, accept_len, uniforms, B, gamma, V, token, flags, workspace,
                               workspace_bytes, cuda_stream, 0, drop_seq + 1, poll_limit);
}

dssd_status dssd_device_resample(const float *p_row, const float *draft_q,
                                 const int32_t *accept_len, const float *uniforms, int B,
                                 int gamma, int V, int32_t *token, uint32_t *flags,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return device_resample_any(p_row, 0, draft_q, accept_len, uniforms, B, gamma, V, token, flags, workspace,
                               workspace_bytes, cuda_stream);
}

dssd_status dssd_device_resample_p16(const uint16_t *p_row16, const float *draft_q,
                                     const int32_t *accept_len, const float *uniforms, int B,
                                     int gamma, int V, int32_t *token, uint32_t *flags,
                                     void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    return device_resample_any(p_row16, 1, draft_q, accept_len, uniforms, B, gamma, V, token, flags, workspace,
                               workspace_bytes, cuda_stream);
}

size_t dssd_dsd_verify_workspace_bytes(int B, int gamma, int V)
{
    if (check_sizes(B, gamma, V) != DSSD_OK) return 0;
    return align256(dssd_edge_verify_workspace_bytes(B, gamma, V)) + align256(dssd_device_resample_workspace_bytes(B, gamma, V));
}

dssd_status dssd_dsd_verify(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                            const float *draft_q, const int32_t *draft_tokens, const float *uniforms,
                            const float *uniforms_rs, float temperature, int B, int gamma, int V,
                            int32_t *accept_len, int32_t *token, uint32_t *edge_flags,
                            uint32_t *rs_flags, void *workspace, size_t workspace_bytes,
                            void *cuda_stream)
{
    t_last_cuda_error = 0;
    dssd_status st = check_sizes(B, gamma, V);
    if (st != DSSD_OK) return st;
    if (dtype != DSSD_F32 && dtype != DSSD_BF16) return DSSD_ERR_UNSUPPORTED;
    if (!target_logits || !uniforms_rs || !accept_len || !token) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && (!draft_q || !draft_tokens || !uniforms)) return DSSD_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !isfinite(temperature)) return DSSD_ERR_INVALID_ARG;
    if (row_stride < (int64_t)V) return DSSD_ERR_INVALID_ARG;
    const size_t esz = dtype == DSSD_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(target_logits) % esz) || (reinterpret_cast<uintptr_t>(draft_q) % 4))
        return DSSD_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < dssd_dsd_verify_workspace_bytes(B, gamma, V))
        return DSSD_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    char *ws_edge = static_cast<char *>(workspace);
    char *ws_rs = ws_edge + align256(dssd_edge_verify_workspace_bytes(B, gamma, V));

    dssd::EdgeParams E{};
    E.logits = target_logits;
    E.row_stride = row_stride;
    E.draft_tokens = draft_tokens;
    E.draft_q_rows = draft_q;  // q_i(x_i) is read out of the uploaded rows where a sequence is folded
    E.uniforms = uniforms;
    E.temperature = temperature;
    E.B = B;
    E.gamma = gamma;
    E.V = V;
    E.accept_len = accept_len;
    E.flags = edge_flags;  // no row: nothing is emitted
    cudaError_t e = dssd::edge_verify_launch(E, (int)dtype, ws_edge, s);
    if (e != cudaSuccess) return cuda_fail(e);

    dssd::ResampleParams R{};
    R.logits = target_logits;
    R.row_stride = row_stride;
    R.logits_dtype = (int)dtype;
    R.c1 = E.c1;
    R.ready = E.ready;
    R.draft_q = draft_q;
    R.accept_len = accept_len;
    R.uniforms = uniforms_rs;
    R.B = B;
    R.gamma = gamma;
    R.V = V;
    R.token = token;
    R.flags = rs_flags;
    e = dssd::resample_launch(R, ws_rs, s);
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}

size_t dssd_edge_verify_bonus_workspace_bytes(int B, int gamma, int V)
{
    if (check_sizes(B, gamma, V) != DSSD_OK) return 0;
    return align256(dssd_edge_verify_workspace_bytes(B, gamma, V)) + align256(dssd_device_resample_workspace_bytes(B, gamma, V));
}

dssd_status dssd_edge_verify_bonus(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                                   const int32_t *draft_tokens, const float *draft_q_tok,
                                   const float *uniforms, const float *uniforms_bonus,
                                   float temperature, int B, int gamma, int V, int32_t *accept_len,
                                   float *p_row, int32_t *token, float *p_tok, float *lse,
                                   uint32_t *flags, uint32_t *token_flags, void *workspace,
                                   size_t workspace_bytes, void *cuda_stream)
{
    t_last_cuda_error = 0;
    dssd_status st = check_sizes(B, gamma, V);
    if (st != DSSD_OK) return st;
    if (dtype != DSSD_F32 && dtype != DSSD_BF16) return DSSD_ERR_UNSUPPORTED;
    if (!target_logits || !accept_len || !p_row || !token || !uniforms_bonus) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && (!draft_tokens || !draft_q_tok || !uniforms)) return DSSD_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !isfinite(temperature)) return DSSD_ERR_INVALID_ARG;
    if (row_stride < (int64_t)V) return DSSD_ERR_INVALID_ARG;
    const size_t esz = dtype == DSSD_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(target_logits) % esz) || (reinterpret_cast<uintptr_t>(p_row) % 4)) return DSSD_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < dssd_edge_verify_bonus_workspace_bytes(B, gamma, V))
        return DSSD_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    char *ws_edge = static_cast<char *>(workspace);
    char *ws_rs = ws_edge + align256(dssd_edge_verify_workspace_bytes(B, gamma, V));

    dssd::EdgeParams E{};
    E.logits = target_logits;
    E.row_stride = row_stride;
    E.draft_tokens = draft_tokens;
    E.draft_q_tok = draft_q_tok;
    E.uniforms = uniforms;
    E.temperature = temperature;
    E.B = B;
    E.gamma = gamma;
    E.V = V;
    E.accept_len = accept_len;
    E.p_row = p_row;
    E.p_tok = p_tok;
    E.lse = lse;
    E.flags = flags;
    E.skip_bonus_row = 1;  // rows of fully accepted sequences are not emitted
    cudaError_t e = dssd::edge_verify_launch(E, (int)dtype, ws_edge, s);
    if (e != cudaSuccess) return cuda_fail(e);

    // the bonus draws, from row gamma's logits and what the edge kernel left about that row
    dssd::ResampleParams R{};
    R.logits = target_logits;
    R.row_stride = row_stride;
    R.logits_dtype = (int)dtype;
    R.c1 = E.c1;
    R.ready = E.ready;
    R.accept_len = accept_len;
    R.uniforms = uniforms_bonus;
    R.B = B;
    R.gamma = gamma;
    R.V = V;
    R.select = 1;
    R.token = token;
    R.flags = token_flags;
    e = dssd::resample_launch(R, ws_rs, s);
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}

dssd_status dssd_device_resample_rejected(const float *p_row, const float *draft_q,
                                          const int32_t *accept_len, const float *uniforms, int B,
                                          int gamma, int V, int32_t *token, uint32_t *flags,
                                          void *workspace, size_t workspace_bytes,
                                          void *cuda_stream)
{
    return device_resample_any(p_row, 0, draft_q, accept_len, uniforms, B, gamma, V, token, flags, workspace,
                               workspace_bytes, cuda_stream, 2);
}

size_t dssd_edge_verify_topk_workspace_bytes(int B, int gamma, int V, int k)
{
    if (check_sizes(B, gamma, V) != DSSD_OK) return 0;
    if (k < 1 || k > V || k > DSSD_TOPK_MAX) return 0;
    return dssd::topk_workspace_layout(B, gamma, k, nullptr, nullptr);
}

dssd_status dssd_edge_verify_topk(const void *target_logits, dssd_dtype dtype, int64_t row_stride,
                                  const int32_t *draft_tokens, const float *draft_q_tok,
                                  const float *uniforms, float temperature, int B, int gamma,
                                  int V, int k, int32_t *accept_len, int32_t *p_idx, float *p_val,
                                  float *p_tok, uint32_t *flags, void *workspace,
                                  size_t workspace_bytes, void *cuda_stream)
{
    t_last_cuda_error = 0;
    dssd_status st = check_sizes(B, gamma, V);
    if (st != DSSD_OK) return st;
    if (dtype != DSSD_F32 && dtype != DSSD_BF16) return DSSD_ERR_UNSUPPORTED;
    if (k < 1 || k > V) return DSSD_ERR_INVALID_ARG;
    if (k > DSSD_TOPK_MAX) return DSSD_ERR_UNSUPPORTED;
    if (!target_logits || !accept_len || !p_idx || !p_val) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && (!draft_tokens || !draft_q_tok || !uniforms)) return DSSD_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !isfinite(temperature)) return DSSD_ERR_INVALID_ARG;
    if (row_stride < (int64_t)V) return DSSD_ERR_INVALID_ARG;
    const size_t esz = dtype == DSSD_BF16 ? 2 : 4;
    if (reinterpret_cast<uintptr_t>(target_logits) % esz) return DSSD_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < dssd_edge_verify_topk_workspace_bytes(B, gamma, V, k))
        return DSSD_ERR_WORKSPACE;

    dssd::TopkParams P{};
    P.logits = target_logits;
    P.row_stride = row_stride;
    P.draft_tokens = draft_tokens;
    P.draft_q_tok = draft_q_tok;
    P.uniforms = uniforms;
    P.temperature = temperature;
    P.B = B;
    P.gamma = gamma;
    P.V = V;
    P.k = k;
    P.accept_len = accept_len;
    P.p_idx = p_idx;
    P.p_val = p_val;
    P.p_tok = p_tok;
    P.flags = flags;
    cudaError_t e = dssd::topk_verify_launch(P, (int)dtype, workspace, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}

dssd_status dssd_device_resample_topk(const int32_t *p_idx, const float *p_val,
                                      const int32_t *q_idx, const float *q_val,
                                      const int32_t *accept_len, const float *uniforms, int B,
                                      int gamma, int k, int32_t *token, uint32_t *flags,
                                      void *cuda_stream)
{
    t_last_cuda_error = 0;
    if (B < 1 || gamma < 0 || k < 1) return DSSD_ERR_INVALID_ARG;
    if (k > DSSD_TOPK_MAX) return DSSD_ERR_UNSUPPORTED;
    if (!p_idx || !p_val || !accept_len || !uniforms || !token) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && (!q_idx || !q_val)) return DSSD_ERR_INVALID_ARG;
    dssd::TopkResampleParams P{};
    P.p_idx = p_idx;
    P.p_val = p_val;
    P.q_idx = q_idx;
    P.q_val = q_val;
    P.accept_len = accept_len;
    P.uniforms = uniforms;
    P.B = B;
    P.gamma = gamma;
    P.k = k;
    P.token = token;
    P.flags = flags;
    cudaError_t e = dssd::topk_resample_launch(P, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}

// ---- the vocabulary-sharded round ---------------------------------------------------------------

size_t dssd_edge_partial_workspace_bytes(int B, int gamma, int V_shard)
{
    return dssd_edge_verify_workspace_bytes(B, gamma, V_shard);
}

dssd_status dssd_edge_partial(const void *logits_shard, dssd_dtype dtype, int64_t row_stride,
                              const int32_t *draft_tokens, int v_begin, float temperature, int B,
                              int gamma, int V_shard, float *part_ref, double *part_sum,
                              float *tok_logit, void *workspace, size_t workspace_bytes,
                              void *cuda_stream)
{
    t_last_cuda_error = 0;
    dssd_status st = check_sizes(B, gamma, V_shard);
    if (st != DSSD_OK) return st;
    if (dtype != DSSD_F32 && dtype != DSSD_BF16) return DSSD_ERR_UNSUPPORTED;
    if (!logits_shard || !part_ref || !part_sum || v_begin < 0) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && (!draft_tokens || !tok_logit)) return DSSD_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !isfinite(temperature)) return DSSD_ERR_INVALID_ARG;
    if (row_stride < (int64_t)V_shard) return DSSD_ERR_INVALID_ARG;
    const size_t esz = dtype == DSSD_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(logits_shard) % esz) || (reinterpret_cast<uintptr_t>(part_sum) % 8) ||
        (reinterpret_cast<uintptr_t>(part_ref) % 4) || (reinterpret_cast<uintptr_t>(tok_logit) % 4))
        return DSSD_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < dssd_edge_partial_workspace_bytes(B, gamma, V_shard))
        return DSSD_ERR_WORKSPACE;
    dssd::EdgeParams P{};
    P.logits = logits_shard;
    P.row_stride = row_stride;
    P.draft_tokens = draft_tokens;
    P.temperature = temperature;
    P.B = B;
    P.gamma = gamma;
    P.V = V_shard;
    P.v_begin = v_begin;
    P.shard_ref = part_ref;
    P.shard_sum = part_sum;
    P.shard_tok_logit = tok_logit;
    cudaError_t e = dssd::edge_verify_launch(P, (int)dtype, workspace, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}

dssd_status dssd_edge_combine(const float *part_ref, const double *part_sum, const float *tok_logit,
                              int G, const int32_t *draft_tokens, const float *draft_q_tok,
                              const float *uniforms, float temperature, int B, int gamma, int V,
                              int32_t *accept_len, float *row_scale, float *p_tok, float *lse,
                              uint32_t *flags, void *cuda_stream)
{
    t_last_cuda_error = 0;
    dssd_status st = check_sizes(B, gamma, V);
    if (st != DSSD_OK) return st;
    if (G < 1) return DSSD_ERR_INVALID_ARG;
    if (G > dssd::kShardMax) return DSSD_ERR_UNSUPPORTED;
    if (!part_ref || !part_sum || !accept_len || !row_scale) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && (!tok_logit || !draft_tokens || !draft_q_tok || !uniforms)) return DSSD_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !isfinite(temperature)) return DSSD_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(part_sum) % 8) return DSSD_ERR_INVALID_ARG;
    dssd::CombineParams P{};
    P.part_ref = part_ref;
    P.part_sum = part_sum;
    P.tok_logit = tok_logit;
    P.G = G;
    P.draft_tokens = draft_tokens;
    P.draft_q_tok = draft_q_tok;
    P.uniforms = uniforms;
    P.c1 = (float)(1.4426950408889634 / (double)temperature);
    P.B = B;
    P.gamma = gamma;
    P.V = V;
    P.accept_len = accept_len;
    P.row_scale = row_scale;
    P.p_tok = p_tok;
    P.lse = lse;
    P.flags = flags;
    cudaError_t e = dssd::shard_combine_launch(P, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}

dssd_status dssd_edge_emit_shard(const void *logits_shard, dssd_dtype dtype, int64_t row_stride,
                                 const int32_t *accept_len, const float *row_scale,
                                 float temperature, int B, int gamma, int V_shard,
                                 float *p_row_shard, int64_t p_stride, void *cuda_stream)
{
    t_last_cuda_error = 0;
    dssd_status st = check_sizes(B, gamma, V_shard);
    if (st != DSSD_OK) return st;
    if (dtype != DSSD_F32 && dtype != DSSD_BF16) return DSSD_ERR_UNSUPPORTED;
    if (!logits_shard || !accept_len || !row_scale || !p_row_shard) return DSSD_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !isfinite(temperature)) return DSSD_ERR_INVALID_ARG;
    if (row_stride < (int64_t)V_shard || p_stride < (int64_t)V_shard) return DSSD_ERR_INVALID_ARG;
    const size_t esz = dtype == DSSD_BF16 ? 2 : 4;
    if ((reinterpret_cast<uintptr_t>(logits_shard) % esz) || (reinterpret_cast<uintptr_t>(p_row_shard) % 4))
        return DSSD_ERR_INVALID_ARG;
    dssd::EmitShardParams P{};
    P.logits = logits_shard;
    P.row_stride = row_stride;
    P.accept_len = accept_len;
    P.row_scale = row_scale;
    P.c1 = (float)(1.4426950408889634 / (double)temperature);
    P.B = B;
    P.gamma = gamma;
    P.V = V_shard;
    P.p_row = p_row_shard;
    P.p_stride = p_stride;
    cudaError_t e = dssd::shard_emit_launch(P, (int)dtype, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}

size_t dssd_resample_shard_workspace_bytes(int B, int gamma, int V_shard)
{
    if (check_sizes(B, gamma, V_shard) != DSSD_OK) return 0;
    return dssd::shard_resample_workspace_bytes(B, V_shard);
}

namespace {
dssd_status check_shard_rows(const float *p_row_shard, int64_t p_stride, const float *draft_q_shard, int64_t q_stride,
                             const int32_t *accept_len, int B, int gamma, int V_shard, const void *workspace,
                             size_t workspace_bytes)
{
    dssd_status st = check_sizes(B, gamma, V_shard);
    if (st != DSSD_OK) return st;
    if (!p_row_shard || !accept_len) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && !draft_q_shard) return DSSD_ERR_INVALID_ARG;
    if (p_stride < (int64_t)V_shard || (gamma > 0 && q_stride < (int64_t)V_shard)) return DSSD_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(p_row_shard) % 4) || (reinterpret_cast<uintptr_t>(draft_q_shard) % 4))
        return DSSD_ERR_INVALID_ARG;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        workspace_bytes < dssd_resample_shard_workspace_bytes(B, gamma, V_shard))
        return DSSD_ERR_WORKSPACE;
    return DSSD_OK;
}
}  // namespace

dssd_status dssd_resample_shard_mass(const float *p_row_shard, int64_t p_stride,
                                     const float *draft_q_shard, int64_t q_stride,
                                     const int32_t *accept_len, int B, int gamma, int V_shard,
                                     double *mass, void *workspace, size_t workspace_bytes,
                                     void *cuda_stream)
{
    t_last_cuda_error = 0;
    dssd_status st = check_shard_rows(p_row_shard, p_stride, draft_q_shard, q_stride, accept_len, B, gamma, V_shard,
                                      workspace, workspace_bytes);
    if (st != DSSD_OK) return st;
    if (!mass || (reinterpret_cast<uintptr_t>(mass) % 8)) return DSSD_ERR_INVALID_ARG;
    dssd::ShardResampleParams P{};
    P.p_row = p_row_shard;
    P.p_stride = p_stride;
    P.draft_q = draft_q_shard;
    P.q_stride = q_stride;
    P.accept_len = accept_len;
    P.B = B;
    P.gamma = gamma;
    P.V = V_shard;
    P.mass = mass;
    cudaError_t e = dssd::shard_mass_launch(P, workspace, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}

dssd_status dssd_resample_shard_draw(const double *masses, int G, int g, int v_begin,
                                     const float *p_row_shard, int64_t p_stride,
                                     const float *draft_q_shard, int64_t q_stride,
                                     const int32_t *accept_len, const float *uniforms, int B,
                                     int gamma, int V_shard, int32_t *token, uint32_t *flags,
                                     const void *workspace, size_t workspace_bytes,
                                     void *cuda_stream)
{
    t_last_cuda_error = 0;
    dssd_status st = check_shard_rows(p_row_shard, p_stride, draft_q_shard, q_stride, accept_len, B, gamma, V_shard,
                                      workspace, workspace_bytes);
    if (st != DSSD_OK) return st;
    if (!masses || (reinterpret_cast<uintptr_t>(masses) % 8) || !uniforms || !token) return DSSD_ERR_INVALID_ARG;
    if (G < 1 || g < 0 || g >= G || v_begin < 0) return DSSD_ERR_INVALID_ARG;
    if (G > dssd::kShardMax) return DSSD_ERR_UNSUPPORTED;
    if ((long long)v_begin + (long long)V_shard > (long long)DSSD_MAX_V) return DSSD_ERR_UNSUPPORTED;
    dssd::ShardResampleParams P{};
    P.p_row = p_row_shard;
    P.p_stride = p_stride;
    P.draft_q = draft_q_shard;
    P.q_stride = q_stride;
    P.accept_len = accept_len;
    P.B = B;
    P.gamma = gamma;
    P.V = V_shard;
    P.masses = masses;
    P.G = G;
    P.g = g;
    P.v_begin = v_begin;
    P.uniforms = uniforms;
    P.token = token;
    P.flags = flags;
    cudaError_t e = dssd::shard_draw_launch(P, workspace, static_cast<cudaStream_t>(cuda_stream));
    return e == cudaSuccess ? DSSD_OK : cuda_fail(e);
}

size_t dssd_round_host_arena_bytes(int B, int gamma, int V, dssd_dtype dtype)
{
    if (check_sizes(B, gamma, V) != DSSD_OK) return 0;
    if (dtype != DSSD_F32 && dtype != DSSD_BF16) return 0;
    const size_t esz = dtype == DSSD_BF16 ? 2 : 4;
    const size_t Bz = (size_t)B, g = (size_t)gamma, Vz = (size_t)V;
    size_t n = 0;
    n += align256(Bz * (g + 1) * Vz * esz);  // target_logits
    n += align256(Bz * g * Vz * 4);          // draft_q
    n += 3 * align256(Bz * g * 4);           // draft_tokens, draft_q_tok, uniforms
    n += align256(Bz * 4);                   // uniforms_rs
    n += align256(Bz * Vz * 4);              // p_row
    n += 4 * align256(Bz * 4);               // accept_len, token, edge flags, resample flags
    n += align256(dssd_edge_verify_workspace_bytes(B, gamma, V));
    n += align256(dssd_device_resample_workspace_bytes(B, gamma, V));
    return n;
}

dssd_status dssd_round_host(const void *target_logits, dssd_dtype dtype,
                            const int32_t *draft_tokens, const float *draft_q_tok,
                            const float *uniforms, const float *draft_q, const float *uniforms_rs,
                            float temperature, int B, int gamma, int V, int32_t *accept_len,
                            int32_t *token, uint32_t *edge_flags, uint32_t *rs_flags,
                            float *p_row, void *device_arena, size_t arena_bytes,
                            void *cuda_stream)
{
    t_last_cuda_error = 0;
    dssd_status st = check_sizes(B, gamma, V);
    if (st != DSSD_OK) return st;
    if (dtype != DSSD_F32 && dtype != DSSD_BF16) return DSSD_ERR_UNSUPPORTED;
    if (!target_logits || !uniforms_rs || !accept_len || !token) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && (!draft_tokens || !draft_q_tok || !uniforms || !draft_q)) return DSSD_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !isfinite(temperature)) return DSSD_ERR_INVALID_ARG;
    if (!device_arena || (reinterpret_cast<uintptr_t>(device_arena) & 255u) ||
        arena_bytes < dssd_round_host_arena_bytes(B, gamma, V, dtype))
        return DSSD_ERR_WORKSPACE;

    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t esz = dtype == DSSD_BF16 ? 2 : 4;
    const size_t Bz = (size_t)B, g = (size_t)gamma, Vz = (size_t)V;
    char *cur = static_cast<char *>(device_arena);
    auto take = [&](size_t bytes) {
        char *p = cur;
        cur += align256(bytes);
        return p;
    };
    void *d_logits = take(Bz * (g + 1) * Vz * esz);
    float *d_q = reinterpret_cast<float *>(take(Bz * g * Vz * 4));
    int32_t *d_tok_in = reinterpret_cast<int32_t *>(take(Bz * g * 4));
    float *d_qtok = reinterpret_cast<float *>(take(Bz * g * 4));
    float *d_u = reinterpret_cast<float *>(take(Bz * g * 4));
    float *d_urs = reinterpret_cast<float *>(take(Bz * 4));
    float *d_prow = reinterpret_cast<float *>(take(Bz * Vz * 4));
    int32_t *d_n = reinterpret_cast<int32_t *>(take(Bz * 4));
    int32_t *d_token = reinterpret_cast<int32_t *>(take(Bz * 4));
    uint32_t *d_ef = reinterpret_cast<uint32_t *>(take(Bz * 4));
    uint32_t *d_rf = reinterpret_cast<uint32_t *>(take(Bz * 4));
    const size_t ws_e = dssd_edge_verify_workspace_bytes(B, gamma, V);
    const size_t ws_r = dssd_device_resample_workspace_bytes(B, gamma, V);
    void *d_ws_e = take(ws_e);
    void *d_ws_r = take(ws_r);

    cudaError_t e;
#define DSSD_TRY(call) \
    if ((e = (call)) != cudaSuccess) return cuda_fail(e)
    DSSD_TRY(cudaMemcpyAsync(d_logits, target_logits, Bz * (g + 1) * Vz * esz, cudaMemcpyHostToDevice, s));
    if (gamma > 0) {
        DSSD_TRY(cudaMemcpyAsync(d_tok_in, draft_tokens, Bz * g * 4, cudaMemcpyHostToDevice, s));
        DSSD_TRY(cudaMemcpyAsync(d_qtok, draft_q_tok, Bz * g * 4, cudaMemcpyHostToDevice, s));
        DSSD_TRY(cudaMemcpyAsync(d_u, uniforms, Bz * g * 4, cudaMemcpyHostToDevice, s));
    }
    DSSD_TRY(cudaMemcpyAsync(d_urs, uniforms_rs, Bz * 4, cudaMemcpyHostToDevice, s));
    st = dssd_edge_verify(d_logits, dtype, (int64_t)V, gamma ? d_tok_in : nullptr, gamma ? d_qtok : nullptr,
                          gamma ? d_u : nullptr, temperature, B, gamma, V, d_n, d_prow, nullptr, nullptr,
                          d_ef, d_ws_e, ws_e, cuda_stream);
    if (st != DSSD_OK) return st;
    // The device half reads row Q_n only: wait for the accepted lengths, then upload those rows
    // (each to its place in the [B, gamma, V] array, the rest of which is never read).
    DSSD_TRY(cudaMemcpyAsync(accept_len, d_n, Bz * 4, cudaMemcpyDeviceToHost, s));
    DSSD_TRY(cudaStreamSynchronize(s));
    for (size_t b = 0; b < Bz; ++b) {
        const int n = accept_len[b];
        if (n < 0 || n >= gamma) continue;  // bonus draw (no Q row), or no draw at all
        const size_t off = (b * g + (size_t)n) * Vz;
        DSSD_TRY(cudaMemcpyAsync(d_q + off, draft_q + off, Vz * 4, cudaMemcpyHostToDevice, s));
    }
    st = dssd_device_resample(d_prow, gamma ? d_q : nullptr, d_n, d_urs, B, gamma, V, d_token, d_rf, d_ws_r,
                              ws_r, cuda_stream);
    if (st != DSSD_OK) return st;
    DSSD_TRY(cudaMemcpyAsync(token, d_token, Bz * 4, cudaMemcpyDeviceToHost, s));
    if (edge_flags) DSSD_TRY(cudaMemcpyAsync(edge_flags, d_ef, Bz * 4, cudaMemcpyDeviceToHost, s));
    if (rs_flags) DSSD_TRY(cudaMemcpyAsync(rs_flags, d_rf, Bz * 4, cudaMemcpyDeviceToHost, s));
    if (p_row) DSSD_TRY(cudaMemcpyAsync(p_row, d_prow, Bz * Vz * 4, cudaMemcpyDeviceToHost, s));
#undef DSSD_TRY
    return DSSD_OK;
}

size_t dssd_round_host_topk_arena_bytes(int B, int gamma, int V, int k, dssd_dtype dtype)
{
    if (check_sizes(B, gamma, V) != DSSD_OK) return 0;
    if (dtype != DSSD_F32 && dtype != DSSD_BF16) return 0;
    if (k < 1 || k > V || k > DSSD_TOPK_MAX) return 0;
    const size_t esz = dtype == DSSD_BF16 ? 2 : 4;
    const size_t Bz = (size_t)B, g = (size_t)gamma, Vz = (size_t)V, kz = (size_t)k;
    size_t n = 0;
    n += align256(Bz * (g + 1) * Vz * esz);  // target_logits
    n += 3 * align256(Bz * g * 4);           // draft_tokens, draft_q_tok, uniforms
    n += 2 * align256(Bz * g * kz * 4);      // q_idx, q_val
    n += align256(Bz * 4);                   // uniforms_rs
    n += 2 * align256(Bz * kz * 4);          // p_idx, p_val
    n += 4 * align256(Bz * 4);               // accept_len, token, edge flags, resample flags
    n += align256(dssd_edge_verify_topk_workspace_bytes(B, gamma, V, k));
    return n;
}

dssd_status dssd_round_host_topk(const void *target_logits, dssd_dtype dtype,
                                 const int32_t *draft_tokens, const float *draft_q_tok,
                                 const float *uniforms, const int32_t *q_idx, const float *q_val,
                                 const float *uniforms_rs, float temperature, int B, int gamma, int V,
                                 int k, int32_t *accept_len, int32_t *token, uint32_t *edge_flags,
                                 uint32_t *rs_flags, int32_t *p_idx, float *p_val, void *device_arena,
                                 size_t arena_bytes, void *cuda_stream)
{
    t_last_cuda_error = 0;
    dssd_status st = check_sizes(B, gamma, V);
    if (st != DSSD_OK) return st;
    if (dtype != DSSD_F32 && dtype != DSSD_BF16) return DSSD_ERR_UNSUPPORTED;
    if (k < 1 || k > V) return DSSD_ERR_INVALID_ARG;
    if (k > DSSD_TOPK_MAX) return DSSD_ERR_UNSUPPORTED;
    if (!target_logits || !uniforms_rs || !accept_len || !token) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && (!draft_tokens || !draft_q_tok || !uniforms || !q_idx || !q_val)) return DSSD_ERR_INVALID_ARG;
    if (!(temperature > 0.f) || !isfinite(temperature)) return DSSD_ERR_INVALID_ARG;
    if (!device_arena || (reinterpret_cast<uintptr_t>(device_arena) & 255u) ||
        arena_bytes < dssd_round_host_topk_arena_bytes(B, gamma, V, k, dtype))
        return DSSD_ERR_WORKSPACE;

    cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
    const size_t esz = dtype == DSSD_BF16 ? 2 : 4;
    const size_t Bz = (size_t)B, g = (size_t)gamma, Vz = (size_t)V, kz = (size_t)k;
    char *cur = static_cast<char *>(device_arena);
    auto take = [&](size_t bytes) {
        char *p = cur;
        cur += align256(bytes);
        return p;
    };
    void *d_logits = take(Bz * (g + 1) * Vz * esz);
    int32_t *d_tok_in = reinterpret_cast<int32_t *>(take(Bz * g * 4));
    float *d_qtok = reinterpret_cast<float *>(take(Bz * g * 4));
    float *d_u = reinterpret_cast<float *>(take(Bz * g * 4));
    int32_t *d_qidx = reinterpret_cast<int32_t *>(take(Bz * g * kz * 4));
    float *d_qval = reinterpret_cast<float *>(take(Bz * g * kz * 4));
    float *d_urs = reinterpret_cast<float *>(take(Bz * 4));
    int32_t *d_pidx = reinterpret_cast<int32_t *>(take(Bz * kz * 4));
    float *d_pval = reinterpret_cast<float *>(take(Bz * kz * 4));
    int32_t *d_n = reinterpret_cast<int32_t *>(take(Bz * 4));
    int32_t *d_token = reinterpret_cast<int32_t *>(take(Bz * 4));
    uint32_t *d_ef = reinterpret_cast<uint32_t *>(take(Bz * 4));
    uint32_t *d_rf = reinterpret_cast<uint32_t *>(take(Bz * 4));
    const size_t ws = dssd_edge_verify_topk_workspace_bytes(B, gamma, V, k);
    void *d_ws = take(ws);

    cudaError_t e;
#define DSSD_TRY(call) \
    if ((e = (call)) != cudaSuccess) return cuda_fail(e)
    DSSD_TRY(cudaMemcpyAsync(d_logits, target_logits, Bz * (g + 1) * Vz * esz, cudaMemcpyHostToDevice, s));
    if (gamma > 0) {
        DSSD_TRY(cudaMemcpyAsync(d_tok_in, draft_tokens, Bz * g * 4, cudaMemcpyHostToDevice, s));
        DSSD_TRY(cudaMemcpyAsync(d_qtok, draft_q_tok, Bz * g * 4, cudaMemcpyHostToDevice, s));
        DSSD_TRY(cudaMemcpyAsync(d_u, uniforms, Bz * g * 4, cudaMemcpyHostToDevice, s));
        DSSD_TRY(cudaMemcpyAsync(d_qidx, q_idx, Bz * g * kz * 4, cudaMemcpyHostToDevice, s));
        DSSD_TRY(cudaMemcpyAsync(d_qval, q_val, Bz * g * kz * 4, cudaMemcpyHostToDevice, s));
    }
    DSSD_TRY(cudaMemcpyAsync(d_urs, uniforms_rs, Bz * 4, cudaMemcpyHostToDevice, s));
    st = dssd_edge_verify_topk(d_logits, dtype, (int64_t)V, gamma ? d_tok_in : nullptr, gamma ? d_qtok : nullptr,
                               gamma ? d_u : nullptr, temperature, B, gamma, V, k, d_n, d_pidx, d_pval, nullptr,
                               d_ef, d_ws, ws, cuda_stream);
    if (st != DSSD_OK) return st;
    st = dssd_device_resample_topk(d_pidx, d_pval, gamma ? d_qidx : nullptr, gamma ? d_qval : nullptr, d_n, d_urs, B,
                                   gamma, k, d_token, d_rf, cuda_stream);
    if (st != DSSD_OK) return st;
    DSSD_TRY(cudaMemcpyAsync(accept_len, d_n, Bz * 4, cudaMemcpyDeviceToHost, s));
    DSSD_TRY(cudaMemcpyAsync(token, d_token, Bz * 4, cudaMemcpyDeviceToHost, s));
    if (edge_flags) DSSD_TRY(cudaMemcpyAsync(edge_flags, d_ef, Bz * 4, cudaMemcpyDeviceToHost, s));
    if (rs_flags) DSSD_TRY(cudaMemcpyAsync(rs_flags, d_rf, Bz * 4, cudaMemcpyDeviceToHost, s));
    if (p_idx) DSSD_TRY(cudaMemcpyAsync(p_idx, d_pidx, Bz * kz * 4, cudaMemcpyDeviceToHost, s));
    if (p_val) DSSD_TRY(cudaMemcpyAsync(p_val, d_pval, Bz * kz * 4, cudaMemcpyDeviceToHost, s));
#undef DSSD_TRY
    return DSSD_OK;
}

}  // extern "C"
