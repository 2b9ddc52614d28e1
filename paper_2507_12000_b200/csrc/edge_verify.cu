// Edge half of the verification round as one persistent, ticket-driven streaming kernel.
//
// Work is cut into tickets that CTAs draw from a global counter in increasing order:
//   LSE(b, i, k)  stream slice k of target row (b, i): online max / sum of exp -> one partial
//   EMIT(b, k)    stream slice k of row n_b again, write p_row[b, slice] = exp(l/T - lse)
// The CTA that completes the last slice of a row folds the row's partials (float64), evaluates
// the acceptance test for that position and bumps the sequence's counter; the CTA that completes
// the last row of a sequence runs the first-rejection scan (warp ballot) and publishes n_b.
// Nothing on that chain waits.  EMIT tickets of sequence b are placed `lag` sequences behind its
// LSE tickets, so n_b is almost always published when they are drawn; if not, one thread polls
// the sequence's ready word.  Every ticket drawn earlier is held by a CTA that is running and
// that never blocks, so the poll ends; it is bounded anyway and reports a timeout flag.
// Tickets of one sequence are adjacent, so the whole machine streams the same few rows at the
// same time and the second read of row n_b comes from L2, not from HBM.
#include "edge_verify.h"

#include <math.h>

#include "dssd_device.cuh"

namespace dssd {

namespace {

constexpr int kUnroll = 4;  // 16-byte vectors in flight per thread

struct Online {  // per-thread running max and sum of 2^((z - ref) * c1), ref = m (0 while m = -inf)
    float m;
    float s0, s1;
};

__device__ __forceinline__ float ref_of(float m) { return m == DSSD_NEG_INF ? 0.f : m; }

// fold a newly seen maximum into the running pair
__device__ __forceinline__ void raise_max(Online &o, float vmax, float c1)
{
    if (vmax > o.m) {
        float f = ex2((ref_of(o.m) - vmax) * c1);  // m = -inf: sums are 0 already
        f = (o.m == DSSD_NEG_INF) ? 0.f : f;
        o.s0 *= f;
        o.s1 *= f;
        o.m = vmax;
    }
}

template <int DT>
__device__ __forceinline__ float vec_max(const uint4 &v)
{
    float f[Elem<DT>::kVec];
    Elem<DT>::unpack(v, f);
    float m = f[0];
#pragma unroll
    for (int j = 1; j < Elem<DT>::kVec; ++j) m = fmaxf(m, f[j]);
    return m;
}

template <int DT>
__device__ __forceinline__ void vec_accum(Online &o, const uint4 &v, float ref, float c1)
{
    float f[Elem<DT>::kVec];
    Elem<DT>::unpack(v, f);
#pragma unroll
    for (int j = 0; j < Elem<DT>::kVec; j += 2) {
        o.s0 += ex2((f[j] - ref) * c1);
        o.s1 += ex2((f[j + 1] - ref) * c1);
    }
}

__device__ __forceinline__ void scalar_accum(Online &o, float z, float c1)
{
    raise_max(o, z, c1);
    o.s0 += ex2((z - ref_of(o.m)) * c1);
}

// ---- LSE ticket: one slice of one row -> (max, sum) partial --------------------------------
template <int DT>
__device__ void lse_slice(const EdgeParams &P, int64_t row, int slice, float2 *s_warp, int *s_last)
{
    using E = Elem<DT>;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float c1 = P.c1;
    const char *rowp = static_cast<const char *>(P.logits) + (size_t)row * (size_t)P.row_stride * E::kBytes;
    const int e0 = slice * P.lse_slice, e1 = min(P.V, e0 + P.lse_slice);
    // split [e0, e1) into scalar head, 16-byte aligned vector body, scalar tail
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(rowp) + (size_t)e0 * E::kBytes;
    int head = (int)(((16u - (unsigned)(a0 & 15u)) & 15u) / E::kBytes);
    head = min(head, e1 - e0);
    const int nvec = (e1 - e0 - head) / E::kVec;
    const int tail0 = e0 + head + nvec * E::kVec;
    const uint4 *body = reinterpret_cast<const uint4 *>(rowp + (size_t)(e0 + head) * E::kBytes);

    Online o{DSSD_NEG_INF, 0.f, 0.f};
    int i = tid;
    for (; i + (kUnroll - 1) * kThreads < nvec; i += kUnroll * kThreads) {
        uint4 v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) v[u] = ld_stream16(body + i + u * kThreads);
        float vm = vec_max<DT>(v[0]);
#pragma unroll
        for (int u = 1; u < kUnroll; ++u) vm = fmaxf(vm, vec_max<DT>(v[u]));
        raise_max(o, vm, c1);
        const float ref = ref_of(o.m);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) vec_accum<DT>(o, v[u], ref, c1);
    }
    for (; i < nvec; i += kThreads) {
        uint4 v = ld_stream16(body + i);
        raise_max(o, vec_max<DT>(v), c1);
        vec_accum<DT>(o, v, ref_of(o.m), c1);
    }
    if (tid < head) scalar_accum(o, E::load(rowp, e0 + tid), c1);
    if (tid < e1 - tail0) scalar_accum(o, E::load(rowp, tail0 + tid), c1);

    // CTA-wide fold of (m, s): warp shuffles, then warp 0 over the per-warp pairs
    float s = o.s0 + o.s1;
    float M = warp_max(o.m);
    s *= (o.m == DSSD_NEG_INF) ? 0.f : ex2((o.m - ref_of(M)) * c1);
    s = warp_sum(s);
    if (lane == 0) s_warp[warp] = make_float2(M, s);
    __syncthreads();
    if (warp == 0) {
        float2 w = lane < kWarps ? s_warp[lane] : make_float2(DSSD_NEG_INF, 0.f);
        float MM = warp_max(w.x);
        float ss = w.y * ((w.x == DSSD_NEG_INF) ? 0.f : ex2((w.x - ref_of(MM)) * c1));
        ss = warp_sum(ss);
        int last = 0;
        if (lane == 0) {
            P.part[(size_t)row * P.n_lse_slices + slice] = make_float2(MM, ss);
            __threadfence();
            last = (atomicAdd(&P.row_cnt[row], 1u) == (unsigned)(P.n_lse_slices - 1));
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
            // ---- this CTA finished the row: fold partials in float64, acceptance test --------
            __threadfence();
            const double T = (double)P.temperature;
            float Mr = DSSD_NEG_INF;
            for (int k = lane; k < P.n_lse_slices; k += 32)
                Mr = fmaxf(Mr, __ldcg(&P.part[(size_t)row * P.n_lse_slices + k].x));
            Mr = warp_max(Mr);
            double S = 0.0;
            bool bad = false;
            for (int k = lane; k < P.n_lse_slices; k += 32) {
                float2 pk = __ldcg(&P.part[(size_t)row * P.n_lse_slices + k]);
                if (pk.y != pk.y) bad = true;
                if (pk.x != DSSD_NEG_INF) S += (double)pk.y * exp(((double)pk.x - (double)Mr) / T);
            }
            S = warp_sum(S);
            bad = __any_sync(0xffffffffu, bad);
            const int64_t b = row / (P.gamma + 1);
            const int pos = (int)(row - b * (P.gamma + 1));
            if (lane == 0) {
                double lse = (double)Mr / T + log(S);
                bool finite = !bad && (lse == lse) && (fabs(lse) < INFINITY);
                if (!finite) lse = NAN;
                unsigned bits = finite ? 0u : 4u;
                P.row_M[row] = Mr;
                P.row_invS[row] = finite ? (float)(1.0 / S) : NAN;
                if (P.lse) P.lse[row] = (float)lse;
                if (pos < P.gamma) {
                    const size_t di = (size_t)b * P.gamma + pos;
                    const int x = P.draft_tokens[di];
                    double p = NAN;
                    bool accept = false;
                    if (x < 0 || x >= P.V) {
                        bits |= 2u;
                    } else {
                        p = exp((double)E::load(rowp, x) / T - lse);
                        const double q = (double)P.draft_q_tok[di];
                        const double u = (double)P.uniforms[di];
                        double ratio;
                        if (q != q) ratio = NAN;
                        else if (q <= 0.0) ratio = (p > 0.0) ? INFINITY : 0.0;
                        else ratio = p / q;
                        accept = (ratio == ratio) && (u < (ratio < 1.0 ? ratio : 1.0));
                    }
                    if (P.p_tok) P.p_tok[di] = (float)p;
                    bits |= accept ? 1u : 0u;
                }
                P.row_bits[row] = bits;
                __threadfence();
                last = (atomicAdd(&P.seq_cnt[b], 1u) == (unsigned)P.gamma);
            }
            last = __shfl_sync(0xffffffffu, last, 0);
            if (last) {
                // ---- this CTA finished the sequence: first-rejection scan -------------------
                __threadfence();
                int n = P.gamma;
                unsigned fl = 0;
                for (int base = 0; base <= P.gamma; base += 32) {
                    const int i2 = base + lane;
                    unsigned bits = (i2 <= P.gamma) ? __ldcg(&P.row_bits[b * (P.gamma + 1) + i2]) : 1u;
                    const unsigned rej = __ballot_sync(0xffffffffu, i2 < P.gamma && !(bits & 1u));
                    if (rej && n == P.gamma) n = base + __ffs(rej) - 1;
                    fl |= (__ballot_sync(0xffffffffu, bits & 2u) ? DSSD_EDGE_FLAG_BAD_TOKEN : 0u) |
                          (__ballot_sync(0xffffffffu, bits & 4u) ? DSSD_EDGE_FLAG_NONFINITE : 0u);
                }
                if (lane == 0) {
                    P.accept_len[b] = n;
                    if (P.flags) P.flags[b] = fl;
                    __threadfence();
                    st_release(&P.seq_ready[b], 1u);
                }
            }
        }
    }
    (void)s_last;
}

// ---- EMIT ticket: one slice of p_row[b, :] -------------------------------------------------
template <int DT>
__device__ void emit_slice(const EdgeParams &P, int64_t b, int slice, float *s_bcast)
{
    using E = Elem<DT>;
    const int tid = threadIdx.x;
    if (tid == 0) {
        unsigned ready = ld_acquire(&P.seq_ready[b]);
        for (unsigned it = 0; !ready && it < P.spin_limit; ++it) {
            __nanosleep(128);
            ready = ld_acquire(&P.seq_ready[b]);
        }
        int n = -1;
        float M = 0.f, invS = 0.f;
        if (ready) {
            n = __ldcg(&P.accept_len[b]);
            const int64_t r = b * (P.gamma + 1) + n;
            M = __ldcg(&P.row_M[r]);
            invS = __ldcg(&P.row_invS[r]);
        } else {
            atomicOr(P.error, 1u);
            if (P.flags) atomicOr(&P.flags[b], DSSD_EDGE_FLAG_TIMEOUT);
        }
        s_bcast[0] = __int_as_float(n);
        s_bcast[1] = M;
        s_bcast[2] = invS;
    }
    __syncthreads();
    const int n = __float_as_int(s_bcast[0]);
    const float M = ref_of(s_bcast[1]), invS = s_bcast[2];
    if (n < 0) return;
    const float c1 = P.c1;
    const int64_t row = b * (P.gamma + 1) + n;
    const char *rowp = static_cast<const char *>(P.logits) + (size_t)row * (size_t)P.row_stride * E::kBytes;
    float *outp = P.p_row + (size_t)b * P.V;
    const int e0 = slice * P.emit_slice, e1 = min(P.V, e0 + P.emit_slice);
    const bool aligned = (((reinterpret_cast<uintptr_t>(rowp) + (size_t)e0 * E::kBytes) |
                           reinterpret_cast<uintptr_t>(outp + e0)) & 15u) == 0;
    int done = e0;
    if (aligned) {
        const int nvec = (e1 - e0) / E::kVec;
        const uint4 *body = reinterpret_cast<const uint4 *>(rowp + (size_t)e0 * E::kBytes);
        for (int i = tid; i < nvec; i += kThreads) {
            float f[E::kVec];
            E::unpack(ld_stream16(body + i), f);
#pragma unroll
            for (int j = 0; j < E::kVec; ++j) f[j] = ex2((f[j] - M) * c1) * invS;
            float *o = outp + e0 + (size_t)i * E::kVec;
#pragma unroll
            for (int j = 0; j < E::kVec; j += 4) st_stream16(o + j, f[j], f[j + 1], f[j + 2], f[j + 3]);
        }
        done = e0 + nvec * E::kVec;
    }
    for (int e = done + tid; e < e1; e += kThreads)
        outp[e] = ex2((E::load(rowp, e) - M) * c1) * invS;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, 4) edge_verify_kernel(const EdgeParams P)
{
    __shared__ float2 s_warp[kWarps];
    __shared__ float s_bcast[4];
    __shared__ unsigned long long s_ticket;
    const int tid = threadIdx.x;
    if (tid == 0) s_ticket = atomicAdd(P.ticket, 1ull);
    __syncthreads();
    unsigned long long t = s_ticket;
    while (t < P.total_tickets) {
        __syncthreads();  // every thread has read s_ticket (and is done with the previous ticket's smem)
        unsigned long long nxt = 0;
        if (tid == 0) nxt = atomicAdd(P.ticket, 1ull);  // drawn now, needed only after this ticket
        const long long g = (long long)(t / P.tickets_per_group);
        const int idx = (int)(t - (unsigned long long)g * P.tickets_per_group);
        if (idx < P.lse_tickets) {
            if (g < P.B) {
                const int pos = idx / P.n_lse_slices;
                lse_slice<DT>(P, g * (P.gamma + 1) + pos, idx - pos * P.n_lse_slices, s_warp, nullptr);
            }
        } else if (g >= P.lag) {
            emit_slice<DT>(P, g - P.lag, idx - P.lse_tickets, s_bcast);
        }
        if (tid == 0) s_ticket = nxt;
        __syncthreads();
        t = s_ticket;
    }
}

}  // namespace

size_t edge_workspace_layout(int B, int gamma, int V, int n_lse_slices, EdgeParams *P, char *base)
{
    // [zeroed region: ticket, error, row_cnt[R], seq_cnt[B], seq_ready[B]] [row_M, row_invS, row_bits][part]
    const size_t R = (size_t)B * (size_t)(gamma + 1);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += (bytes + 255) & ~(size_t)255;
        return o;
    };
    const size_t o_ticket = take(16);
    const size_t o_rowcnt = take(R * 4);
    const size_t o_seqcnt = take((size_t)B * 4);
    const size_t o_ready = take((size_t)B * 4);
    const size_t zero_bytes = off;
    const size_t o_M = take(R * 4);
    const size_t o_invS = take(R * 4);
    const size_t o_bits = take(R * 4);
    const size_t o_part = take(R * (size_t)n_lse_slices * sizeof(float2));
    if (P) {
        P->ticket = reinterpret_cast<unsigned long long *>(base + o_ticket);
        P->error = reinterpret_cast<unsigned *>(base + o_ticket + 8);
        P->row_cnt = reinterpret_cast<unsigned *>(base + o_rowcnt);
        P->seq_cnt = reinterpret_cast<unsigned *>(base + o_seqcnt);
        P->seq_ready = reinterpret_cast<unsigned *>(base + o_ready);
        P->row_M = reinterpret_cast<float *>(base + o_M);
        P->row_invS = reinterpret_cast<float *>(base + o_invS);
        P->row_bits = reinterpret_cast<unsigned *>(base + o_bits);
        P->part = reinterpret_cast<float2 *>(base + o_part);
        P->zero_bytes = zero_bytes;
    }
    (void)V;
    return off;
}

// launch geometry per device, filled on first use (occupancy depends on the compiled kernel only)
static int g_edge_ctas_per_sm[64][2];
static int g_sm_count[64];

cudaError_t edge_verify_launch(EdgeParams &P, int dtype, void *workspace, cudaStream_t stream)
{
    cudaError_t err;
    int dev = 0;
    if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (g_sm_count[dev] == 0) {
        int sms = 0, occ0 = 0, occ1 = 0;
        if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ0, edge_verify_kernel<DSSD_F32>, kThreads, 0)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ1, edge_verify_kernel<DSSD_BF16>, kThreads, 0)) != cudaSuccess) return err;
        g_edge_ctas_per_sm[dev][0] = occ0 > 0 ? occ0 : 1;
        g_edge_ctas_per_sm[dev][1] = occ1 > 0 ? occ1 : 1;
        g_sm_count[dev] = sms;
    }
    const int esz = dtype == DSSD_BF16 ? 2 : 4;
    P.lse_slice = kEdgeLseSliceBytes / esz;
    P.emit_slice = kEdgeEmitSlice;
    P.n_lse_slices = (P.V + P.lse_slice - 1) / P.lse_slice;
    P.n_emit_slices = (P.V + P.emit_slice - 1) / P.emit_slice;
    P.lse_tickets = (P.gamma + 1) * P.n_lse_slices;
    P.tickets_per_group = (unsigned long long)P.lse_tickets + (unsigned long long)P.n_emit_slices;
    edge_workspace_layout(P.B, P.gamma, P.V, P.n_lse_slices, &P, static_cast<char *>(workspace));
    const long long resident = (long long)g_sm_count[dev] * g_edge_ctas_per_sm[dev][dtype == DSSD_BF16];
    // EMIT tickets trail their sequence's LSE tickets by `lag` sequences: enough that every LSE
    // ticket of that sequence has normally retired (all resident CTAs hold later tickets).
    P.lag = (int)((resident + P.lse_tickets - 1) / P.lse_tickets) + 2;
    P.total_tickets = ((unsigned long long)P.B + (unsigned long long)P.lag) * P.tickets_per_group;
    P.spin_limit = 1u << 22;
    P.c1 = (float)(1.4426950408889634 / (double)P.temperature);
    if ((err = cudaMemsetAsync(workspace, 0, P.zero_bytes, stream)) != cudaSuccess) return err;
    const long long grid = (long long)P.total_tickets < resident ? (long long)P.total_tickets : resident;
    if (dtype == DSSD_BF16)
        edge_verify_kernel<DSSD_BF16><<<(unsigned)grid, kThreads, 0, stream>>>(P);
    else
        edge_verify_kernel<DSSD_F32><<<(unsigned)grid, kThreads, 0, stream>>>(P);
    return cudaGetLastError();
}

}  // namespace dssd
