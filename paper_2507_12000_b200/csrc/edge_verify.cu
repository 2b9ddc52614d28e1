// Edge half of the verification round as one persistent streaming kernel.
//
// The work is an ordered list of tickets that WARPS draw from a global counter.  Group g of the list:
//   LSE(g, i, k)       stream slice k of target row (g, i): max and sum of exp -> 8-byte partial
//   EMIT(g - lag, k)   first-rejection scan over the sequence's acceptance bits (warp ballot), then
//                      slice k of row n streamed again and p_row = exp(l/T - lse) written
// A warp draws one ticket ahead and requests the first half of its next LSE slice before it works on
// the second half of the current one, so loads are always in flight.  Each LSE ticket bumps its row's
// arrival counter; the warp that brings the last slice of a row folds the row's partials (float64
// log-sum-exp) and evaluates the acceptance test for that position, at once and without waiting.
// Drawing is self-balancing: a warp that was held up simply draws fewer tickets, so the tickets
// below the counter complete within a short window, EMIT tickets (which trail their sequence by
// `lag` groups) normally find every row folded, and row n is read the second time from L2.
// An EMIT ticket whose rows are not all folded yet is parked and retried after each later ticket;
// only when a second one would have to be parked, or the list is exhausted, does a warp wait
// (bounded, with a timeout flag) - for rows whose LSE tickets were drawn by running warps.
// A warp works alone: no shared memory, no CTA barrier.  Results travel through 8-byte slots that
// the host pre-filled with all ones and that carry their own validity, so no fence is needed:
// a consumer that sees the fill pattern knows the store has not landed yet.
#include "edge_verify.h"

#include <math.h>

#include "dssd_device.cuh"

namespace dssd {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kVPL = kEdgeVecPerLane;
constexpr unsigned kBitAccept = 1u, kBitBadToken = 2u, kBitNonFinite = 4u, kBitTimeout = 8u;

enum Kind : int { kEnd = 0, kSkip = 1, kLseFast = 2, kLseSlow = 3, kEmit = 4 };

struct Ticket {
    int kind;
    int slice;
    long long index;  // LSE: row; EMIT: sequence
};

__device__ __forceinline__ float ref_of(float m) { return m == DSSD_NEG_INF ? 0.f : m; }

// counters start at all ones (the workspace fill pattern): logical value = raw + 1
__device__ __forceinline__ unsigned logical(unsigned raw) { return raw + 1u; }

template <int DT>
__device__ __forceinline__ const char *row_ptr(const EdgeParams &P, long long row)
{
    return static_cast<const char *>(P.logits) + (size_t)row * (size_t)P.row_stride * Elem<DT>::kBytes;
}

template <int DT>
__device__ __forceinline__ Ticket decode(const EdgeParams &P, unsigned t)
{
    Ticket k{kEnd, 0, 0};
    if (t >= P.total_tickets) return k;
    k.kind = kSkip;
    const unsigned g = t / P.tickets_per_group;
    const int idx = (int)(t - g * P.tickets_per_group);
    if (idx < P.lse_tickets) {
        if ((int)g >= P.B) return k;
        const int pos = idx / P.n_lse_slices;
        k.slice = idx - pos * P.n_lse_slices;
        k.index = (long long)g * (P.gamma + 1) + pos;
        const int e0 = k.slice * P.lse_slice;
        const uintptr_t a = reinterpret_cast<uintptr_t>(row_ptr<DT>(P, k.index)) + (size_t)e0 * Elem<DT>::kBytes;
        k.kind = (e0 + P.lse_slice <= P.V && (a & 15u) == 0) ? kLseFast : kLseSlow;
        return k;
    }
    const long long b = (long long)g - P.lag;
    if (b < 0 || b >= P.B) return k;
    k.kind = kEmit;
    k.index = b;
    k.slice = idx - P.lse_tickets;
    return k;
}

// one half (kVPL 16-byte vectors per lane) of a full, aligned LSE slice
template <int DT>
__device__ __forceinline__ void load_half(const EdgeParams &P, const Ticket &k, int half, uint4 (&v)[kVPL])
{
    const int lane = threadIdx.x & 31;
    const uint4 *p = reinterpret_cast<const uint4 *>(row_ptr<DT>(P, k.index) + (size_t)k.slice * kEdgeLseSliceBytes) +
                     half * (32 * kVPL) + lane;
#pragma unroll
    for (int u = 0; u < kVPL; ++u) v[u] = ld_stream16(p + u * 32);
}

struct Online {  // per-lane running max m and sum of 2^((z - ref(m)) * c1)
    float m, s0, s1;
};

template <int DT>
__device__ __forceinline__ void accum_half(Online &o, const uint4 (&v)[kVPL], float c1)
{
    using E = Elem<DT>;
    float m = o.m;
#pragma unroll
    for (int u = 0; u < kVPL; ++u) {
        float f[E::kVec];
        E::unpack(v[u], f);
#pragma unroll
        for (int j = 0; j < E::kVec; ++j) m = fmaxf(m, f[j]);
    }
    if (m > o.m) {
        const float f = (o.m == DSSD_NEG_INF) ? 0.f : ex2((o.m - m) * c1);
        o.s0 *= f;
        o.s1 *= f;
        o.m = m;
    }
    const float ref = ref_of(o.m);
#pragma unroll
    for (int u = 0; u < kVPL; ++u) {
        float f[E::kVec];
        E::unpack(v[u], f);
#pragma unroll
        for (int j = 0; j < E::kVec; j += 2) {
            o.s0 += ex2((f[j] - ref) * c1);
            o.s1 += ex2((f[j + 1] - ref) * c1);
        }
    }
}

// lane-local (m, s) -> warp-wide (M, S), one 8-byte store
__device__ __forceinline__ void publish_partial(const EdgeParams &P, const Ticket &k, float m, float s)
{
    const float M = warp_max(m);
    s *= (m == DSSD_NEG_INF) ? 0.f : ex2((m - ref_of(M)) * P.c1);
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0)
        st_relaxed_u64(&P.part[(size_t)k.index * P.n_lse_slices + k.slice],
                       (unsigned long long)__float_as_uint(M) | ((unsigned long long)__float_as_uint(s) << 32));
}

// LSE ticket, ragged or unaligned slice: scalar head, vector body, scalar tail, online max
template <int DT>
__device__ __noinline__ void lse_slow(const EdgeParams &P, const Ticket &k)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    const float c1 = P.c1;
    const char *rowp = row_ptr<DT>(P, k.index);
    const int e0 = k.slice * P.lse_slice, e1 = min(P.V, e0 + P.lse_slice);
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(rowp) + (size_t)e0 * E::kBytes;
    int head = (int)(((16u - (unsigned)(a0 & 15u)) & 15u) / E::kBytes);
    head = min(head, e1 - e0);
    const int nvec = (e1 - e0 - head) / E::kVec;
    const int tail0 = e0 + head + nvec * E::kVec;
    const uint4 *body = reinterpret_cast<const uint4 *>(rowp + (size_t)(e0 + head) * E::kBytes);
    float m = DSSD_NEG_INF, s = 0.f;
    auto add = [&](float z) {
        if (z > m) {
            s *= (m == DSSD_NEG_INF) ? 0.f : ex2((m - z) * c1);
            m = z;
        }
        s += ex2((z - ref_of(m)) * c1);
    };
    for (int i = lane; i < nvec; i += 32) {
        float f[E::kVec];
        E::unpack(ld_stream16(body + i), f);
#pragma unroll
        for (int j = 0; j < E::kVec; ++j) add(f[j]);
    }
    if (lane < head) add(E::load(rowp, e0 + lane));
    if (lane < e1 - tail0) add(E::load(rowp, tail0 + lane));
    publish_partial(P, k, m, s);
}

// Run by the warp that brought a row's last slice: the partials of the row -> log-sum-exp
// (float64), acceptance test, RowInfo.
template <int DT>
__device__ __noinline__ void fold_row(const EdgeParams &P, long long row)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    const double T = (double)P.temperature;
    const unsigned long long *part = reinterpret_cast<const unsigned long long *>(P.part) + (size_t)row * P.n_lse_slices;
    const long long b = row / (P.gamma + 1);
    const int pos = (int)(row - b * (P.gamma + 1));
    // lane 0 starts on the drafted token early: its loads overlap the partials'
    int x = -1;
    float zx = 0.f, qx = 0.f, ux = 0.f;
    if (lane == 0 && pos < P.gamma) {
        const size_t di = (size_t)b * P.gamma + pos;
        x = P.draft_tokens[di];
        qx = P.draft_q_tok[di];
        ux = P.uniforms[di];
        if (x >= 0 && x < P.V) zx = E::load(row_ptr<DT>(P, row), x);
    }
    // The arrival counter says every slice has been counted; a partial whose store has not landed
    // yet still shows the fill pattern and is polled for.
    float Mr = DSSD_NEG_INF;
    double S = 0.0;
    bool bad = false, timeout = false;
    auto fetch = [&](int k) {
        unsigned long long w = ld_relaxed_u64(part + k);
        for (unsigned it = 0; (unsigned)w == kFull && it < P.spin_limit; ++it) {
            __nanosleep(32);
            w = ld_relaxed_u64(part + k);
        }
        if ((unsigned)w == kFull) timeout = true;
        return w;
    };
    constexpr int kKeep = 4;  // partials per lane kept in registers: rows of up to 128 slices in one pass
    if (P.n_lse_slices <= 32 * kKeep) {
        unsigned long long w[kKeep];
#pragma unroll
        for (int j = 0; j < kKeep; ++j) w[j] = (lane + 32 * j < P.n_lse_slices) ? ld_relaxed_u64(part + lane + 32 * j) : 0ull;
#pragma unroll
        for (int j = 0; j < kKeep; ++j)
            if (lane + 32 * j < P.n_lse_slices) {
                if ((unsigned)w[j] == kFull) w[j] = fetch(lane + 32 * j);
                if ((unsigned)w[j] != kFull) Mr = fmaxf(Mr, __uint_as_float((unsigned)w[j]));
            }
        timeout = __any_sync(kFull, timeout);
        Mr = warp_max(Mr);
#pragma unroll
        for (int j = 0; j < kKeep; ++j)
            if (lane + 32 * j < P.n_lse_slices && !timeout) {
                const float pm = __uint_as_float((unsigned)w[j]), ps = __uint_as_float((unsigned)(w[j] >> 32));
                if (ps != ps) bad = true;
                if (pm != DSSD_NEG_INF) S += (double)ps * exp(((double)pm - (double)Mr) / T);
            }
    } else {
        for (int k = lane; k < P.n_lse_slices; k += 32) {
            const unsigned long long w = fetch(k);
            if ((unsigned)w != kFull) Mr = fmaxf(Mr, __uint_as_float((unsigned)w));
        }
        timeout = __any_sync(kFull, timeout);
        Mr = warp_max(Mr);
        if (!timeout) {
            for (int k = lane; k < P.n_lse_slices; k += 32) {
                const unsigned long long w = ld_relaxed_u64(part + k);
                const float pm = __uint_as_float((unsigned)w), ps = __uint_as_float((unsigned)(w >> 32));
                if (ps != ps) bad = true;
                if (pm != DSSD_NEG_INF) S += (double)ps * exp(((double)pm - (double)Mr) / T);
            }
        }
    }
    S = warp_sum(S);
    bad = __any_sync(kFull, bad);
    if (lane != 0) return;
    double lse = (double)Mr / T + log(S);
    const bool finite = !timeout && !bad && (lse == lse) && (fabs(lse) < INFINITY);
    if (!finite) lse = NAN;
    unsigned bits = (finite ? 0u : kBitNonFinite) | (timeout ? kBitTimeout : 0u);
    if (timeout) *P.error = 1u;
    if (P.lse) P.lse[row] = (float)lse;
    if (pos < P.gamma) {
        double p = NAN;
        bool accept = false;
        if (x < 0 || x >= P.V) {
            bits |= kBitBadToken;
        } else {
            // u < min(1, p(x)/q(x)), evaluated in float64
            p = exp((double)zx / T - lse);
            const double q = (double)qx;
            const double u = (double)ux;
            double ratio;
            if (q != q) ratio = NAN;
            else if (q <= 0.0) ratio = (p > 0.0) ? INFINITY : 0.0;
            else ratio = p / q;
            accept = (ratio == ratio) && (u < (ratio < 1.0 ? ratio : 1.0));
        }
        if (P.p_tok) P.p_tok[(size_t)b * P.gamma + pos] = (float)p;
        bits |= accept ? kBitAccept : 0u;
    }
    const float invS = finite ? (float)(1.0 / S) : NAN;
    unsigned long long *ri = reinterpret_cast<unsigned long long *>(P.row_info + row);
    st_relaxed_u64(ri, (unsigned long long)__float_as_uint(Mr) | ((unsigned long long)__float_as_uint(invS) << 32));
    st_relaxed_u64(ri + 1, (unsigned long long)bits);
}

// EMIT ticket: first-rejection scan, then one slice of p_row[b, :].
// With `wait` false it returns false, having done nothing, if some row of the sequence is not
// folded yet; with `wait` true it polls (bounded) for those rows.
template <int DT>
__device__ __noinline__ bool emit_slice(const EdgeParams &P, long long b, int slice, bool wait)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    // one row per lane: its acceptance bits and its (M, 1/S); ballot + find-first-set gives n
    int n = P.gamma;
    unsigned fl = 0;
    unsigned long long w0n = 0;
    bool timeout = false;
    for (int base = 0; base <= P.gamma; base += 32) {
        const int i = base + lane;
        unsigned bits = kBitAccept;
        unsigned long long w0 = 0;
        if (i <= P.gamma) {
            const unsigned long long *ri = reinterpret_cast<const unsigned long long *>(P.row_info + b * (P.gamma + 1) + i);
            w0 = ld_relaxed_u64(ri);
            bits = (unsigned)ld_relaxed_u64(ri + 1);
            if (wait) {
                for (unsigned it = 0; (bits == kFull || (unsigned)w0 == kFull) && it < P.spin_limit; ++it) {
                    __nanosleep(100);
                    w0 = ld_relaxed_u64(ri);
                    bits = (unsigned)ld_relaxed_u64(ri + 1);
                }
            }
            if (bits == kFull || (unsigned)w0 == kFull) { timeout = true; bits = kBitTimeout; }
        }
        if (__any_sync(kFull, timeout)) {
            if (!wait) return false;
            timeout = true;
        }
        const unsigned rej = __ballot_sync(kFull, i < P.gamma && !(bits & kBitAccept));
        if (rej && n == P.gamma) n = base + __ffs(rej) - 1;
        fl |= (__ballot_sync(kFull, bits & kBitBadToken) ? DSSD_EDGE_FLAG_BAD_TOKEN : 0u) |
              (__ballot_sync(kFull, bits & kBitNonFinite) ? DSSD_EDGE_FLAG_NONFINITE : 0u) |
              (__ballot_sync(kFull, bits & kBitTimeout) ? DSSD_EDGE_FLAG_TIMEOUT : 0u);
        if (n >= base && n < base + 32) w0n = __shfl_sync(kFull, w0, n - base);
    }
    if (slice == 0 && lane == 0) {
        P.accept_len[b] = timeout ? -1 : n;
        if (P.flags) P.flags[b] = fl;
        if (timeout) *P.error = 1u;
    }
    if (timeout) return true;
    const long long row = b * (P.gamma + 1) + n;
    const float M = ref_of(__uint_as_float((unsigned)w0n)), invS = __uint_as_float((unsigned)(w0n >> 32));
    const float c1 = P.c1;
    const char *rowp = row_ptr<DT>(P, row);
    float *outp = P.p_row + (size_t)b * P.V;
    const int e0 = slice * P.emit_slice, e1 = min(P.V, e0 + P.emit_slice);
    const bool aligned = (((reinterpret_cast<uintptr_t>(rowp) + (size_t)e0 * E::kBytes) |
                           reinterpret_cast<uintptr_t>(outp + e0)) & 15u) == 0;
    int done = e0;
    if (aligned) {
        const int nvec = (e1 - e0) / E::kVec;
        const uint4 *body = reinterpret_cast<const uint4 *>(rowp + (size_t)e0 * E::kBytes);
        constexpr int kU = 4;
        int i = lane;
        for (; i + (kU - 1) * 32 < nvec; i += kU * 32) {
            uint4 v[kU];
#pragma unroll
            for (int u = 0; u < kU; ++u) v[u] = ld_stream16(body + i + u * 32);
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                float f[E::kVec];
                E::unpack(v[u], f);
#pragma unroll
                for (int j = 0; j < E::kVec; ++j) f[j] = ex2((f[j] - M) * c1) * invS;
                float *o = outp + e0 + (size_t)(i + u * 32) * E::kVec;
#pragma unroll
                for (int j = 0; j < E::kVec; j += 4) st_stream16(o + j, f[j], f[j + 1], f[j + 2], f[j + 3]);
            }
        }
        for (; i < nvec; i += 32) {
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
    for (int e = done + lane; e < e1; e += 32) outp[e] = ex2((E::load(rowp, e) - M) * c1) * invS;
    return true;
}

template <int DT>
__global__ void __launch_bounds__(kThreads, kEdgeCtasPerSm) edge_verify_kernel(const EdgeParams P)
{
    const int lane = threadIdx.x & 31;
    const float c1 = P.c1;
    // two draws ahead: `cur` is being worked on, `nxt_no` is the number of the next ticket (drawn
    // one ticket early so that the atomic's round trip is never waited for)
    unsigned no = 0;
    if (lane == 0) no = logical(atomicAdd(P.ticket, 1u));
    Ticket cur = decode<DT>(P, __shfl_sync(kFull, no, 0));
    unsigned nxt_no = 0;
    if (lane == 0) nxt_no = logical(atomicAdd(P.ticket, 1u));
    uint4 v[kVPL], w[kVPL];
    if (cur.kind == kLseFast) load_half<DT>(P, cur, 0, v);
    Ticket parked{kEnd, 0, 0};  // an EMIT ticket whose sequence was not folded yet
    while (cur.kind != kEnd) {
        Ticket nxt;
        if (cur.kind == kLseFast) {
            load_half<DT>(P, cur, 1, w);
            // The slice is counted before its partial is stored: the count is back when the work
            // is done, and whoever folds the row polls for partials that have not landed yet.
            unsigned arrival = 0;
            if (lane == 0) arrival = logical(atomicAdd(&P.row_cnt[cur.index], 1u));
            Online o{DSSD_NEG_INF, 0.f, 0.f};
            accum_half<DT>(o, v, c1);
            // the next ticket's number is back: request its first half before the second half
            // of this slice is worked on
            nxt = decode<DT>(P, __shfl_sync(kFull, nxt_no, 0));
            if (lane == 0 && nxt.kind != kEnd) nxt_no = logical(atomicAdd(P.ticket, 1u));
            if (nxt.kind == kLseFast) load_half<DT>(P, nxt, 0, v);
            accum_half<DT>(o, w, c1);
            publish_partial(P, cur, o.m, o.s0 + o.s1);
            if (__shfl_sync(kFull, arrival, 0) == (unsigned)(P.n_lse_slices - 1)) fold_row<DT>(P, cur.index);
        } else {
            nxt = decode<DT>(P, __shfl_sync(kFull, nxt_no, 0));
            if (lane == 0 && nxt.kind != kEnd) nxt_no = logical(atomicAdd(P.ticket, 1u));
            if (nxt.kind == kLseFast) load_half<DT>(P, nxt, 0, v);
            if (cur.kind == kLseSlow) {
                unsigned arrival = 0;
                if (lane == 0) arrival = logical(atomicAdd(&P.row_cnt[cur.index], 1u));
                lse_slow<DT>(P, cur);
                if (__shfl_sync(kFull, arrival, 0) == (unsigned)(P.n_lse_slices - 1)) fold_row<DT>(P, cur.index);
            } else if (cur.kind == kEmit) {
                if (!emit_slice<DT>(P, cur.index, cur.slice, false)) {
                    if (parked.kind != kEnd) emit_slice<DT>(P, parked.index, parked.slice, true);  // older
                    parked = cur;
                }
            }
        }
        if (parked.kind != kEnd && cur.kind != kEmit && emit_slice<DT>(P, parked.index, parked.slice, false))
            parked.kind = kEnd;
        cur = nxt;
    }
    if (parked.kind != kEnd) emit_slice<DT>(P, parked.index, parked.slice, true);
}

}  // namespace

size_t edge_workspace_layout(int B, int gamma, int V, int n_lse_slices, EdgeParams *P, char *base)
{
    // all of it is filled with 0xFF before the launch: counters then read "logical 0", slots "not yet"
    const size_t R = (size_t)B * (size_t)(gamma + 1);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += (bytes + 255) & ~(size_t)255;
        return o;
    };
    const size_t o_err = take(256);  // ticket counter and error word on separate 128-byte lines
    const size_t o_rowcnt = take(R * 4);
    const size_t o_info = take(R * sizeof(RowInfo));
    const size_t o_part = take(R * (size_t)n_lse_slices * sizeof(float2));
    if (P) {
        P->ticket = reinterpret_cast<unsigned *>(base + o_err);
        P->error = reinterpret_cast<unsigned *>(base + o_err + 128);
        P->row_cnt = reinterpret_cast<unsigned *>(base + o_rowcnt);
        P->row_info = reinterpret_cast<RowInfo *>(base + o_info);
        P->part = reinterpret_cast<float2 *>(base + o_part);
        P->fill_bytes = off;
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
        if (occ0 < 1 || occ1 < 1) return cudaErrorLaunchOutOfResources;
        g_edge_ctas_per_sm[dev][0] = occ0 < kEdgeCtasPerSm ? occ0 : kEdgeCtasPerSm;
        g_edge_ctas_per_sm[dev][1] = occ1 < kEdgeCtasPerSm ? occ1 : kEdgeCtasPerSm;
        g_sm_count[dev] = sms;
    }
    const int esz = dtype == DSSD_BF16 ? 2 : 4;
    P.lse_slice = kEdgeLseSliceBytes / esz;
    P.emit_slice = kEdgeEmitSlice;
    P.n_lse_slices = (P.V + P.lse_slice - 1) / P.lse_slice;
    P.n_emit_slices = (P.V + P.emit_slice - 1) / P.emit_slice;
    P.lse_tickets = (P.gamma + 1) * P.n_lse_slices;
    const unsigned long long G = (unsigned long long)P.lse_tickets + (unsigned long long)P.n_emit_slices;
    edge_workspace_layout(P.B, P.gamma, P.V, P.n_lse_slices, &P, static_cast<char *>(workspace));
    const unsigned long long resident_ctas = (unsigned long long)g_sm_count[dev] * g_edge_ctas_per_sm[dev][dtype == DSSD_BF16];
    const unsigned long long resident_warps = resident_ctas * kWarps;
    // EMIT trails its sequence's LSE tickets by kEdgeEmitLagSweeps times the number of resident
    // warps: one such sweep covers the tickets still being worked on, the rest the fold.
    P.lag = (int)((kEdgeEmitLagSweeps * resident_warps + G - 1) / G) + 1;
    const unsigned long long total = ((unsigned long long)P.B + (unsigned long long)P.lag) * G;
    if (total + 2 * resident_warps >= 0xffffffffull) return cudaErrorInvalidValue;
    P.tickets_per_group = (unsigned)G;
    P.total_tickets = (unsigned)total;
    P.spin_limit = 1u << 20;
    P.c1 = (float)(1.4426950408889634 / (double)P.temperature);
    if ((err = cudaMemsetAsync(workspace, 0xFF, P.fill_bytes, stream)) != cudaSuccess) return err;
    const unsigned long long want = (total + 2 * kWarps - 1) / (2 * kWarps);
    const unsigned grid = (unsigned)(want < resident_ctas ? want : resident_ctas);
    void *args[] = {&P};
    const void *fn = dtype == DSSD_BF16 ? reinterpret_cast<const void *>(edge_verify_kernel<DSSD_BF16>)
                                        : reinterpret_cast<const void *>(edge_verify_kernel<DSSD_F32>);
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kThreads), args, 0, stream);
}

}  // namespace dssd
