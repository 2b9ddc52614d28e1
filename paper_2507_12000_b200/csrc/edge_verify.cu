// Edge half of the verification round as one persistent streaming kernel.
//
// Every warp is an independent worker with a private ring of shared-memory stages.  Logits
// travel global -> shared memory as bulk asynchronous copies (TMA, untiled) that the warp's
// lane 0 issues up to kEdgeStages slices ahead; a stage's arrival is signalled on an mbarrier.
// Work comes as tickets drawn from global counters:
//   LSE(row, run)    a run of consecutive slices of one target row: online maximum and sum of
//                    2^(l * c1 - ref2) in float32 -> one 8-byte partial (ref2, sum).  ref2 is an
//                    integer, so partials combine by exact power-of-two scaling.
//   EMIT(slot, run)  a run of slices of row n of a sequence taken from the `ready` queue: the row
//                    is streamed again (from L2) and p_row = 2^(l * c1 - ref2) / S is written.
// The warp that brings a row's last partial folds the row (float64 log-sum-exp, acceptance test
// of that position); the warp that folds a sequence's last row runs the first-rejection scan
// (ballot + find-first-set) and pushes the sequence to `ready`.  EMIT tickets are claimed, by
// compare-and-swap, only for sequences already pushed, and are preferred over LSE tickets, so the
// second read of row n follows the first closely and hits L2.
// Nothing on this path waits on a fence: results travel through 8-byte slots that the host
// pre-filled with all ones and that carry their own validity; a consumer that sees the fill
// pattern polls (bounded) for a store that a running warp has already issued.  A warp only ever
// waits for work held by running warps, and never while its own ring holds unprocessed slices,
// so the kernel needs no co-residency guarantee.
#include "edge_verify.h"

#include <math.h>

#include "dssd_device.cuh"

namespace dssd {

namespace {

#ifndef DSSD_EDGE_WAR
#define DSSD_EDGE_WAR 1
#endif
constexpr unsigned kFull = 0xffffffffu;
constexpr int kS = kEdgeSliceBytes;
constexpr unsigned kBitAccept = 1u, kBitBadToken = 2u, kBitNonFinite = 4u, kBitTimeout = 8u;

enum Kind : int { kEnd = 0, kIdle = 1, kLse = 2, kEmit = 3 };

// counters start at all ones (the workspace fill pattern): logical value = raw + 1
__device__ __forceinline__ unsigned logical(unsigned raw) { return raw + 1u; }
__device__ __forceinline__ unsigned long long logical(unsigned long long raw) { return raw + 1ull; }

__device__ __forceinline__ unsigned long long shfl0(unsigned long long v) { return __shfl_sync(kFull, v, 0); }
__device__ __forceinline__ int shfl0(int v) { return __shfl_sync(kFull, v, 0); }
__device__ __forceinline__ float shfl0(float v) { return __shfl_sync(kFull, v, 0); }

template <int DT>
__device__ __forceinline__ const char *row_ptr(const EdgeParams &P, long long row)
{
    return static_cast<const char *>(P.logits) + (size_t)row * (size_t)P.row_stride * Elem<DT>::kBytes;
}

// A ticket as the warp keeps it in shared memory between the moment its first copy is issued
// and the moment its last slice has been worked on.
struct Ticket {
    long long row;      // LSE: the row; EMIT: row n of the sequence
    long long out_off;  // EMIT: b * V, offset of the output row in p_row; < 0: write nothing
    int run;            // ticket index within the row (LSE: partial slot)
    int head;           // bytes before the row's first 16-byte boundary (scalar head of slice 0)
    float ref2, invS;   // EMIT
};
constexpr int kTq = 8;  // tickets a warp can have in flight (>= kEdgeStages + 1), a power of two
static_assert(kTq > kEdgeStages && (kTq & (kTq - 1)) == 0, "ticket queue too small");

// What the registers hold per ring stage: `bulk` bytes in flight and
//   meta = kind | first << 2 | last << 3 | ragged << 4 | queue slot << 5 | slice index << 8
// first/last: of its ticket; ragged: the slice has scalar elements outside the bulk copy.
constexpr unsigned kMetaFirst = 4u, kMetaLast = 8u, kMetaRagged = 16u;

// Where lane 0's copies are (the fetch side runs up to kEdgeStages slices ahead of the work),
// and what lane 0 has loaded ahead.  Values loaded ahead are kept raw (as loaded) and
// converted where they are used, so that nothing depends on a load or atomic until its round
// trip is over.
struct Fetch {
    int kind;
    int k, k_begin, k_end;  // next slice, first slice and end of the current ticket
    int slot;               // ticket queue slot of the current ticket
    int head;               // its row's head bytes
    const char *src;        // source of slice k's bulk copy
    long long remain;       // bytes of the row's body from slice k on (may be <= 0)
    unsigned issued;        // tickets started so far (next queue slot = issued % kTq)
    unsigned long long lse_raw;   // lane 0: atomic result holding the LSE ticket in hand
    unsigned long long head_raw;  // lane 0: last value loaded from emit_head
    unsigned tail_raw;            // lane 0: last value loaded from ready_tail
    unsigned long long parked;    // lane 0: EMIT ticket claimed ahead of its sequence, or kNoTicket
};
constexpr unsigned long long kNoTicket = ~0ull;

template <int DT>
__device__ __forceinline__ int row_head_bytes(const EdgeParams &P, const char *rowp)
{
    const long long rowbytes = (long long)P.V * Elem<DT>::kBytes;
    const long long h = (long long)((16u - (unsigned)(reinterpret_cast<uintptr_t>(rowp) & 15u)) & 15u);
    return (int)(h > rowbytes ? rowbytes : h);
}

// ---- per-lane online log-sum-exp state ---------------------------------------------------

struct Online {
    float m;    // running maximum of the raw logits (-inf: nothing seen)
    float ref;  // rint(m * c1), or 0 while m == -inf: terms are 2^(l * c1 - ref) <= 2^0.5
    float s0, s1, s2, s3;
};

__device__ __forceinline__ void online_reset(Online &o)
{
    o.m = DSSD_NEG_INF;
    o.ref = 0.f;
    o.s0 = o.s1 = o.s2 = o.s3 = 0.f;
}

__device__ __forceinline__ void online_raise(Online &o, float bm, float c1)
{
    if (bm > o.m) {
        const float nref = rintf(bm * c1);
        const float f = (o.m == DSSD_NEG_INF) ? 0.f : ex2(o.ref - nref);  // an exact power of two
        o.s0 *= f;
        o.s1 *= f;
        o.s2 *= f;
        o.s3 *= f;
        o.m = bm;
        o.ref = nref;
    }
}

__device__ __forceinline__ void online_add(Online &o, float z, float c1)
{
    online_raise(o, z, c1);
    o.s0 += ex2(fmaf(z, c1, -o.ref));
}

template <int DT>
__device__ __forceinline__ void accum_block(Online &o, const uint4 (&v)[4], float c1);

template <>
__device__ __forceinline__ void accum_block<DSSD_BF16>(Online &o, const uint4 (&v)[4], float c1)
{
    uint32_t mx = max_bf16x2(max_bf16x2(v[0].x, v[0].y), max_bf16x2(v[0].z, v[0].w));
#pragma unroll
    for (int u = 1; u < 4; ++u)
        mx = max_bf16x2(mx, max_bf16x2(max_bf16x2(v[u].x, v[u].y), max_bf16x2(v[u].z, v[u].w)));
    online_raise(o, fmaxf(bf16_lo(mx), bf16_hi(mx)), c1);
    const float nref = -o.ref;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        o.s0 += ex2(fmaf(bf16_lo(v[u].x), c1, nref));
        o.s1 += ex2(fmaf(bf16_hi(v[u].x), c1, nref));
        o.s2 += ex2(fmaf(bf16_lo(v[u].y), c1, nref));
        o.s3 += ex2(fmaf(bf16_hi(v[u].y), c1, nref));
        o.s0 += ex2(fmaf(bf16_lo(v[u].z), c1, nref));
        o.s1 += ex2(fmaf(bf16_hi(v[u].z), c1, nref));
        o.s2 += ex2(fmaf(bf16_lo(v[u].w), c1, nref));
        o.s3 += ex2(fmaf(bf16_hi(v[u].w), c1, nref));
    }
}

template <>
__device__ __forceinline__ void accum_block<DSSD_F32>(Online &o, const uint4 (&v)[4], float c1)
{
    float bm = DSSD_NEG_INF;
#pragma unroll
    for (int u = 0; u < 4; ++u)
        bm = fmaxf(bm, fmaxf(fmaxf(__uint_as_float(v[u].x), __uint_as_float(v[u].y)),
                             fmaxf(__uint_as_float(v[u].z), __uint_as_float(v[u].w))));
    online_raise(o, bm, c1);
    const float nref = -o.ref;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        o.s0 += ex2(fmaf(__uint_as_float(v[u].x), c1, nref));
        o.s1 += ex2(fmaf(__uint_as_float(v[u].y), c1, nref));
        o.s2 += ex2(fmaf(__uint_as_float(v[u].z), c1, nref));
        o.s3 += ex2(fmaf(__uint_as_float(v[u].w), c1, nref));
    }
}

template <int DT>
__device__ __forceinline__ uint4 neg_inf_vec()
{
    return DT == DSSD_BF16 ? make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u)
                           : make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
}

// One slice of an LSE ticket: the `bulk` bytes that the copy brought into the stage.
template <int DT>
__device__ __forceinline__ void lse_consume(uint32_t stage, uint32_t bulk, float c1, Online &o)
{
    const int lane = threadIdx.x & 31;
    const uint32_t base = stage + (uint32_t)lane * 16u;
    if (bulk == (uint32_t)kS && kS % 2048 == 0) {
#pragma unroll
        for (int blk = 0; blk < kS / 2048; ++blk) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = lds16(base + (uint32_t)(blk * 2048 + u * 512));
            accum_block<DT>(o, v, c1);
        }
        return;
    }
    const int nvec = (int)(bulk >> 4);
    int i = lane;
    for (; i + 96 < nvec; i += 128) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) v[u] = lds16(base + (uint32_t)(i - lane + 32 * u) * 16u);
        accum_block<DT>(o, v, c1);
    }
    if (i < nvec) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            v[u] = (i + 32 * u < nvec) ? lds16(base + (uint32_t)(i - lane + 32 * u) * 16u) : neg_inf_vec<DT>();
        accum_block<DT>(o, v, c1);
    }
}

// Scalar elements of slice k that lie outside its bulk copy: the head of the row (slice 0) and
// the tail of the row's last slice.  `fn(element index)` is called by one lane per element.
template <int DT, class F>
__device__ __forceinline__ void for_ragged(const EdgeParams &P, int head, int k, F fn)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    const long long rowbytes = (long long)P.V * E::kBytes;
    const long long off = (long long)k * kS;
    long long len = rowbytes - head - off;
    len = len < 0 ? 0 : (len > kS ? kS : len);
    const long long bulk = len & ~15ll;
    if (k == 0 && lane < head / E::kBytes) fn((int64_t)lane);
    const int tail = (int)((len - bulk) / E::kBytes);
    if (lane < tail) fn((int64_t)((head + off + bulk) / E::kBytes) + lane);
}

// lane-local state -> the ticket's partial (ref2, sum), one 8-byte store
__device__ __forceinline__ void publish_partial(const EdgeParams &P, long long row, int run, const Online &o)
{
    const bool empty = (o.m == DSSD_NEG_INF);
    const float R = warp_max(empty ? DSSD_NEG_INF : o.ref);
    float s = (o.s0 + o.s1) + (o.s2 + o.s3);
    s = empty ? 0.f : s * ex2(o.ref - R);  // exact scaling
    s = warp_sum(s);
    if ((threadIdx.x & 31) == 0) {
        const float Rp = (R == DSSD_NEG_INF) ? 0.f : R;
        st_relaxed_u64(&P.part[(size_t)row * P.n_lse_runs + run],
                       (unsigned long long)__float_as_uint(Rp) | ((unsigned long long)__float_as_uint(s) << 32));
    }
}

// Run by the warp that folded the last row of sequence b: first-rejection scan over the
// acceptance bits (one row per lane, ballot + find-first-set), then the push to `ready`.
__device__ __noinline__ void finish_sequence(const EdgeParams &P, long long b)
{
    const int lane = threadIdx.x & 31;
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
            for (unsigned it = 0; (bits == kFull || (unsigned)w0 == kFull) && it < P.spin_limit; ++it) {
                __nanosleep(64);
                w0 = ld_relaxed_u64(ri);
                bits = (unsigned)ld_relaxed_u64(ri + 1);
            }
            if (bits == kFull || (unsigned)w0 == kFull) {
                timeout = true;
                bits = kBitTimeout;
            }
        }
        const unsigned rej = __ballot_sync(kFull, i < P.gamma && !(bits & kBitAccept));
        if (rej && n == P.gamma) n = base + __ffs(rej) - 1;
        fl |= (__ballot_sync(kFull, bits & kBitBadToken) ? DSSD_EDGE_FLAG_BAD_TOKEN : 0u) |
              (__ballot_sync(kFull, bits & kBitNonFinite) ? DSSD_EDGE_FLAG_NONFINITE : 0u) |
              (__ballot_sync(kFull, bits & kBitTimeout) ? DSSD_EDGE_FLAG_TIMEOUT : 0u);
        if (n >= base && n < base + 32) w0n = __shfl_sync(kFull, w0, n - base);
    }
    timeout = __any_sync(kFull, timeout);
    if (lane == 0) {
        P.accept_len[b] = timeout ? -1 : n;
        if (P.flags) P.flags[b] = fl;
        if (timeout) *P.error = 1u;
        const unsigned slot = logical(atomicAdd(P.ready_tail, 1u));
        unsigned long long *rs = reinterpret_cast<unsigned long long *>(P.ready + slot);
        st_relaxed_u64(rs, (unsigned long long)(unsigned)b | ((unsigned long long)(unsigned)(timeout ? -1 : n) << 32));
        st_relaxed_u64(rs + 1, timeout ? 0ull : w0n);
    }
}

// Run by the warp that brought a row's last partial: partials -> log-sum-exp (float64),
// acceptance test of the position, RowInfo; then the sequence's arrival count.
template <int DT>
__device__ __noinline__ void fold_row(const EdgeParams &P, long long row)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    const double c1 = (double)P.c1;
    const unsigned long long *part = P.part + (size_t)row * P.n_lse_runs;
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
    // The arrival counter says every ticket of the row has been counted; a partial whose store
    // has not landed yet still shows the fill pattern and is polled for.
    float Rr = DSSD_NEG_INF;
    bool bad = false, timeout = false;
    for (int k = lane; k < P.n_lse_runs; k += 32) {
        unsigned long long w = ld_relaxed_u64(part + k);
        for (unsigned it = 0; (unsigned)w == kFull && it < P.spin_limit; ++it) {
            __nanosleep(32);
            w = ld_relaxed_u64(part + k);
        }
        if ((unsigned)w == kFull) {
            timeout = true;
        } else {
            const float ps = __uint_as_float((unsigned)(w >> 32));
            if (ps != ps) bad = true;
            if (ps > 0.f) Rr = fmaxf(Rr, __uint_as_float((unsigned)w));
        }
    }
    timeout = __any_sync(kFull, timeout);
    bad = __any_sync(kFull, bad);
    Rr = warp_max(Rr);
    double S = 0.0;
    if (!timeout && Rr != DSSD_NEG_INF) {
        for (int k = lane; k < P.n_lse_runs; k += 32) {
            const unsigned long long w = ld_relaxed_u64(part + k);
            const float pr = __uint_as_float((unsigned)w), ps = __uint_as_float((unsigned)(w >> 32));
            if (ps > 0.f) S += (double)ps * exp2((double)pr - (double)Rr);
        }
    }
    S = warp_sum(S);
    if (lane == 0) {
        double lse2 = (double)Rr + log2(S);  // log2 sum_v 2^(l_v * c1)
        const bool finite = !timeout && !bad && (lse2 == lse2) && (fabs(lse2) < INFINITY);
        if (!finite) lse2 = NAN;
        unsigned bits = (finite ? 0u : kBitNonFinite) | (timeout ? kBitTimeout : 0u);
        if (timeout) *P.error = 1u;
        if (P.lse) P.lse[row] = (float)(lse2 * 0.6931471805599453);
        if (pos < P.gamma) {
            double p = NAN;
            bool accept = false;
            if (x < 0 || x >= P.V) {
                bits |= kBitBadToken;
            } else {
                // u < min(1, p(x)/q(x)), evaluated in float64
                p = exp2((double)zx * c1 - lse2);
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
        const float Rs = finite ? Rr : 0.f;
        unsigned long long *ri = reinterpret_cast<unsigned long long *>(P.row_info + row);
        st_relaxed_u64(ri, (unsigned long long)__float_as_uint(Rs) | ((unsigned long long)__float_as_uint(invS) << 32));
        st_relaxed_u64(ri + 1, (unsigned long long)bits);
    }
    unsigned arrival = 0;
    if (lane == 0) arrival = logical(atomicAdd(&P.seq_cnt[b], 1u));
    if (__shfl_sync(kFull, arrival, 0) == (unsigned)P.gamma) finish_sequence(P, b);
}

// One slice of an EMIT ticket: body[e] = 2^(l_e * c1 - ref2) * invS for the elements of the stage.
template <int DT>
__device__ __forceinline__ void emit_consume(uint32_t stage, uint32_t bulk, float *body, float c1, float nref, float invS)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    const int nelem = (int)(bulk / E::kBytes);
    if ((reinterpret_cast<uintptr_t>(body) & 15u) == 0) {
        const int nquad = nelem >> 2;  // bulk is a multiple of 16 bytes, so nelem is a multiple of 4
        if (DT == DSSD_BF16) {
            const uint32_t base = stage + (uint32_t)lane * 8u;
#pragma unroll 4
            for (int i = lane; i < nquad; i += 32) {
                const uint2 w = lds8(base + (uint32_t)(i - lane) * 8u);
                st_stream16(body + (size_t)i * 4, ex2(fmaf(bf16_lo(w.x), c1, nref)) * invS,
                            ex2(fmaf(bf16_hi(w.x), c1, nref)) * invS, ex2(fmaf(bf16_lo(w.y), c1, nref)) * invS,
                            ex2(fmaf(bf16_hi(w.y), c1, nref)) * invS);
            }
        } else {
            const uint32_t base = stage + (uint32_t)lane * 16u;
#pragma unroll 4
            for (int i = lane; i < nquad; i += 32) {
                const uint4 w = lds16(base + (uint32_t)(i - lane) * 16u);
                st_stream16(body + (size_t)i * 4, ex2(fmaf(__uint_as_float(w.x), c1, nref)) * invS,
                            ex2(fmaf(__uint_as_float(w.y), c1, nref)) * invS,
                            ex2(fmaf(__uint_as_float(w.z), c1, nref)) * invS,
                            ex2(fmaf(__uint_as_float(w.w), c1, nref)) * invS);
            }
        }
    } else {
        // output not 16-byte aligned at this slice: coalesced 4-byte stores
        for (int i = lane; i < nelem; i += 32) {
            float z;
            if (DT == DSSD_BF16) {
                unsigned short h;
                asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(stage + (uint32_t)i * 2u));
                z = __uint_as_float((uint32_t)h << 16);
            } else {
                asm volatile("ld.shared.f32 %0, [%1];" : "=f"(z) : "r"(stage + (uint32_t)i * 4u));
            }
            body[i] = ex2(fmaf(z, c1, nref)) * invS;
        }
    }
}

// lane 0 refreshes what it knows of the EMIT queue; the values are looked at one draw later,
// so the loads' round trips are never waited for
__device__ __forceinline__ void peek_queue(const EdgeParams &P, Fetch &f)
{
    if ((threadIdx.x & 31) == 0) {
        f.tail_raw = ld_relaxed_u32(P.ready_tail);
        f.head_raw = ld_relaxed_u64(P.emit_head);
    }
}

// ticket number -> (index / per, index % per); 32-bit arithmetic whenever the number fits
__device__ __forceinline__ void split_ticket(unsigned long long t, int per, unsigned long long &q, int &r)
{
    if ((t >> 32) == 0) {
        const unsigned q32 = (unsigned)t / (unsigned)per;
        q = q32;
        r = (int)((unsigned)t - q32 * (unsigned)per);
    } else {
        q = t / (unsigned)per;
        r = (int)(t - q * (unsigned)per);
    }
}

// Starts the next ticket: an EMIT ticket if one can be had for a sequence already pushed, else
// the LSE ticket in hand.  EMIT tickets are claimed with one atomic add when the queue seems to
// hold unclaimed work; a claim that lands beyond the pushed sequences (several warps saw the same
// work) is parked and served as soon as its sequence is pushed.  Never waits for other warps'
// work: f.kind = kIdle means "nothing right now", kEnd "nothing ever again".
template <int DT>
__device__ __forceinline__ void draw(const EdgeParams &P, Fetch &f, Ticket *tq)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    int got = 0;
    unsigned long long t = 0;
    if (lane == 0) {
        const unsigned long long tail = (unsigned long long)logical(f.tail_raw);
        if (f.parked == kNoTicket) {
            const unsigned long long head = logical(f.head_raw);
            if (head < tail * (unsigned long long)P.n_emit_runs) {
                const unsigned long long claimed = logical(atomicAdd(P.emit_head, 1ull));
                if (claimed < P.total_emit) f.parked = claimed;
            }
        }
        if (f.parked != kNoTicket) {
            unsigned long long slot;
            int run;
            split_ticket(f.parked, P.n_emit_runs, slot, run);
            if (slot < tail) {
                got = 1;
                t = f.parked;
                f.parked = kNoTicket;
            }
        }
    }
    got = shfl0(got);
    Ticket tk;
    if (got) {
        t = shfl0(t);
        unsigned long long slot;
        split_ticket(t, P.n_emit_runs, slot, tk.run);
        int b = -1, n = -1;
        float ref2 = 0.f, invS = 0.f;
        if (lane == 0) {
            const unsigned long long *rs = reinterpret_cast<const unsigned long long *>(P.ready + slot);
            unsigned long long w0 = ld_relaxed_u64(rs), w1 = ld_relaxed_u64(rs + 1);
            for (unsigned it = 0; ((unsigned)w0 == kFull || (unsigned)w1 == kFull) && it < P.spin_limit; ++it) {
                __nanosleep(32);
                w0 = ld_relaxed_u64(rs);
                w1 = ld_relaxed_u64(rs + 1);
            }
            if ((unsigned)w0 == kFull || (unsigned)w1 == kFull) {
                *P.error = 1u;  // the pusher's stores never landed: nothing can be written
            } else {
                b = (int)(unsigned)w0;
                n = (int)(unsigned)(w0 >> 32);
                ref2 = __uint_as_float((unsigned)w1);
                invS = __uint_as_float((unsigned)(w1 >> 32));
            }
        }
        b = shfl0(b);
        n = shfl0(n);
        tk.ref2 = shfl0(ref2);
        tk.invS = shfl0(invS);
        tk.out_off = (b >= 0 && n >= 0) ? (long long)b * P.V : -1ll;
        tk.row = (long long)(b < 0 ? 0 : b) * (P.gamma + 1) + (n < 0 ? 0 : n);
        f.kind = kEmit;
        f.k_begin = tk.run * P.emit_run;
        f.k_end = min(P.n_slices, f.k_begin + P.emit_run);
    } else {
        const unsigned long long no = logical(shfl0(f.lse_raw));
        if (no >= P.total_lse) {
            // no LSE ticket left: done once every EMIT ticket is claimed and none is parked here
            int more = 0;
            if (lane == 0) more = (f.parked != kNoTicket) || (logical(f.head_raw) < P.total_emit);
            f.kind = shfl0(more) ? kIdle : kEnd;
            if (f.kind == kIdle) peek_queue(P, f);
            return;
        }
        unsigned long long row;
        split_ticket(no, P.n_lse_runs, row, tk.run);
        tk.row = (long long)row;
        tk.out_off = -1;
        tk.ref2 = tk.invS = 0.f;
        f.kind = kLse;
        f.k_begin = tk.run * P.lse_run;
        f.k_end = min(P.n_slices, f.k_begin + P.lse_run);
        if (lane == 0) f.lse_raw = atomicAdd(P.lse_ticket, 1ull);
    }
    peek_queue(P, f);
    const char *rowp = row_ptr<DT>(P, tk.row);
    tk.head = row_head_bytes<DT>(P, rowp);
    f.head = tk.head;
    f.k = f.k_begin;
    f.src = rowp + tk.head + (long long)f.k_begin * kS;
    f.remain = (long long)P.V * E::kBytes - tk.head - (long long)f.k_begin * kS;
    f.slot = (int)(f.issued & (kTq - 1));
    ++f.issued;
    if (lane == 0) tq[f.slot] = tk;
    __syncwarp();
}

template <int DT>
__global__ void __launch_bounds__(kEdgeThreads, 1) edge_verify_kernel(const __grid_constant__ EdgeParams P)
{
    using E = Elem<DT>;
    extern __shared__ __align__(128) unsigned char smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring = smem_addr(smem) + (uint32_t)warp * (uint32_t)(kEdgeStages * kS);
    unsigned char *after_rings = smem + (size_t)kEdgeWarps * kEdgeStages * kS;
    Ticket *tq = reinterpret_cast<Ticket *>(after_rings) + warp * kTq;
    const uint32_t bars = smem_addr(after_rings + sizeof(Ticket) * kTq * kEdgeWarps) + (uint32_t)warp * (kEdgeStages * 8u);
    if (lane == 0) {
#pragma unroll
        for (int st = 0; st < kEdgeStages; ++st) mbar_init(bars + 8u * st, 1u);
        mbar_init_fence();
    }
    __syncwarp();
    const uint64_t pol_emit = l2_policy_evict_first();
    const float c1 = P.c1;

    Fetch f;
    f.kind = kIdle;
    f.k = f.k_begin = f.k_end = f.slot = f.head = 0;
    f.src = nullptr;
    f.remain = 0;
    f.issued = 0;
    f.lse_raw = 0;
    f.head_raw = 0;
    f.tail_raw = 0;
    f.parked = kNoTicket;
    if (lane == 0) f.lse_raw = atomicAdd(P.lse_ticket, 1ull);
    peek_queue(P, f);

    // meta[0] / bulk[0] describe the oldest slice in flight, which sits in ring stage `st`; the
    // ring starts out idle and fills itself during the first kEdgeStages iterations
    unsigned meta[kEdgeStages], bulk[kEdgeStages];
#pragma unroll
    for (int j = 0; j < kEdgeStages; ++j) {
        meta[j] = kIdle;
        bulk[j] = 0;
    }
    Ticket cur;  // the ticket being worked on
    cur.row = 0;
    cur.out_off = -1;
    cur.run = cur.head = 0;
    cur.ref2 = cur.invS = 0.f;
    Online o;
    online_reset(o);
    unsigned parity = 0;  // bit s: parity of the phase that stage s completes next
    unsigned idle = 0;    // consecutive iterations without work
    int st = 0;
    bool failed = false;
    for (;;) {
        const unsigned m = meta[0], nb = bulk[0];
        const int kind = (int)(m & 3u);
        unsigned live = 0;
#pragma unroll
        for (int j = 0; j < kEdgeStages; ++j) live |= meta[j];
        if ((live & 3u) == kEnd) break;  // kinds are 0 (end) .. 3: all stages at end
        const uint32_t stage = ring + (uint32_t)st * kS, bar = bars + 8u * st;
        if (kind == kLse || kind == kEmit) {
            idle = 0;
            if (m & kMetaFirst) {
                cur = tq[(m >> 5) & (kTq - 1)];
                if (kind == kLse) online_reset(o);
            }
            const int k = (int)(m >> 8);
            unsigned arrival = 0;
            // An LSE ticket is counted before its partial is stored: the count is back by the
            // time the slice is done, and whoever folds the row polls for late partials.
            if (kind == kLse && (m & kMetaLast) && lane == 0) arrival = atomicAdd(&P.row_cnt[cur.row], 1u);  // raw
            if (!mbar_wait(bar, (parity >> st) & 1u, P.spin_limit)) {
                failed = true;  // a copy never completed
                break;
            }
            parity ^= 1u << st;
            if (kind == kLse) {
                lse_consume<DT>(stage, nb, c1, o);
                if (m & kMetaRagged) {
                    const char *rowp = row_ptr<DT>(P, cur.row);
                    for_ragged<DT>(P, cur.head, k, [&](int64_t e) { online_add(o, E::load(rowp, e), c1); });
                }
                if (m & kMetaLast) {
                    publish_partial(P, cur.row, cur.run, o);
                    if (logical(__shfl_sync(kFull, arrival, 0)) == (unsigned)(P.n_lse_runs - 1)) fold_row<DT>(P, cur.row);
                }
            } else if (cur.out_off >= 0) {
                float *outp = P.p_row + cur.out_off;
                const float nref = -cur.ref2, invS = cur.invS;
                emit_consume<DT>(stage, nb, outp + (cur.head + (long long)k * kS) / E::kBytes, c1, nref, invS);
                if (m & kMetaRagged) {
                    const char *rowp = row_ptr<DT>(P, cur.row);
                    for_ragged<DT>(P, cur.head, k, [&](int64_t e) { outp[e] = ex2(fmaf(E::load(rowp, e), c1, nref)) * invS; });
                }
            }
            __syncwarp();
#if DSSD_EDGE_WAR == 1
            fence_proxy_async();  // the stage is about to be overwritten by a bulk copy
#endif
        } else if (kind == kIdle) {
            if (++idle > P.spin_limit) {
                failed = true;
                break;
            }
            if (idle > (unsigned)kEdgeStages) __nanosleep(200);  // the whole ring is idle
        }
        // refill the stage just freed with the warp's next slice
        unsigned nm = kEnd, nbulk = 0;
        if (f.kind != kEnd) {
            if (f.kind == kIdle || f.k >= f.k_end) draw<DT>(P, f, tq);
            nm = (unsigned)f.kind;
            if (f.kind == kLse || f.kind == kEmit) {
                const long long len = f.remain < 0 ? 0 : (f.remain > kS ? kS : f.remain);
                nbulk = (unsigned)len & ~15u;
                const bool ragged = (f.k == 0 && f.head != 0) || (len & 15);
                nm |= (f.k == f.k_begin ? kMetaFirst : 0u) | (f.k + 1 == f.k_end ? kMetaLast : 0u) |
                      (ragged ? kMetaRagged : 0u) | ((unsigned)f.slot << 5) | ((unsigned)f.k << 8);
                if (lane == 0) {
                    if (nbulk) {
                        mbar_arrive_expect_tx(bar, nbulk);
                        if (f.kind == kEmit) bulk_g2s_hint(stage, f.src, nbulk, bar, pol_emit);
                        else bulk_g2s(stage, f.src, nbulk, bar);
                    } else {
                        mbar_arrive(bar);
                    }
                }
                f.src += kS;
                f.remain -= kS;
                ++f.k;
            }
        }
#pragma unroll
        for (int j = 0; j + 1 < kEdgeStages; ++j) {
            meta[j] = meta[j + 1];
            bulk[j] = bulk[j + 1];
        }
        meta[kEdgeStages - 1] = nm;
        bulk[kEdgeStages - 1] = nbulk;
        st = (st + 1 == kEdgeStages) ? 0 : st + 1;
    }
    if (failed) {
        // error exit: copies may still be in flight into this warp's ring; wait for them (bounded)
        // before the CTA's shared memory can be handed to another CTA.  Slice j sits in stage st + j;
        // the wait on slice 0 is the one that has just run out, if it was work at all.
        if (lane == 0) *P.error = 1u;
#pragma unroll
        for (int j = 0; j < kEdgeStages; ++j) {
            const int kind = (int)(meta[j] & 3u);
            if (j > 0 && (kind == kLse || kind == kEmit)) mbar_wait(bars + 8u * st, (parity >> st) & 1u, P.spin_limit);
            st = (st + 1 == kEdgeStages) ? 0 : st + 1;
        }
    }
}

constexpr size_t kEdgeSmemBytes = (size_t)kEdgeWarps * kEdgeStages * kS + sizeof(Ticket) * kTq * kEdgeWarps + (size_t)kEdgeWarps * kEdgeStages * 8;

}  // namespace

int edge_max_runs_per_row(int V)
{
    const long long n = ((long long)V * 4 + kS - 1) / kS;
    return (int)(n < 1 ? 1 : n);
}

size_t edge_workspace_layout(int B, int gamma, int runs_per_row, EdgeParams *P, char *base)
{
    // all of it is filled with 0xFF before the launch: counters then read "logical 0", slots "not yet"
    const size_t R = (size_t)B * (size_t)(gamma + 1);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += (bytes + 255) & ~(size_t)255;
        return o;
    };
    const size_t o_ctr = take(512);  // four counters, each on its own 128-byte line
    const size_t o_rowcnt = take(R * 4);
    const size_t o_seqcnt = take((size_t)B * 4);
    const size_t o_info = take(R * sizeof(RowInfo));
    const size_t o_ready = take((size_t)B * sizeof(ReadySlot));
    const size_t o_part = take(R * (size_t)runs_per_row * 8);
    if (P) {
        P->lse_ticket = reinterpret_cast<unsigned long long *>(base + o_ctr);
        P->emit_head = reinterpret_cast<unsigned long long *>(base + o_ctr + 128);
        P->ready_tail = reinterpret_cast<unsigned *>(base + o_ctr + 256);
        P->error = reinterpret_cast<unsigned *>(base + o_ctr + 384);
        P->row_cnt = reinterpret_cast<unsigned *>(base + o_rowcnt);
        P->seq_cnt = reinterpret_cast<unsigned *>(base + o_seqcnt);
        P->row_info = reinterpret_cast<RowInfo *>(base + o_info);
        P->ready = reinterpret_cast<ReadySlot *>(base + o_ready);
        P->part = reinterpret_cast<unsigned long long *>(base + o_part);
        P->fill_bytes = off;
    }
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
        if ((err = cudaFuncSetAttribute(edge_verify_kernel<DSSD_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kEdgeSmemBytes)) != cudaSuccess) return err;
        if ((err = cudaFuncSetAttribute(edge_verify_kernel<DSSD_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kEdgeSmemBytes)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ0, edge_verify_kernel<DSSD_F32>, kEdgeThreads, kEdgeSmemBytes)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ1, edge_verify_kernel<DSSD_BF16>, kEdgeThreads, kEdgeSmemBytes)) != cudaSuccess) return err;
        if (occ0 < 1 || occ1 < 1) return cudaErrorLaunchOutOfResources;
        g_edge_ctas_per_sm[dev][0] = occ0;
        g_edge_ctas_per_sm[dev][1] = occ1;
        g_sm_count[dev] = sms;
    }
    const int esz = dtype == DSSD_BF16 ? 2 : 4;
    const unsigned long long R = (unsigned long long)P.B * (unsigned long long)(P.gamma + 1);
    const long long n_slices = ((long long)P.V * esz + kS - 1) / kS;
    P.n_slices = (int)(n_slices < 1 ? 1 : n_slices);
    const unsigned long long resident_ctas = (unsigned long long)g_sm_count[dev] * g_edge_ctas_per_sm[dev][dtype == DSSD_BF16];
    const unsigned long long resident_warps = resident_ctas * kEdgeWarps;
    // run length: as long as every resident warp still gets about kEdgeTicketsPerWarp tickets
    unsigned long long run = (R * (unsigned long long)P.n_slices) / (resident_warps * kEdgeTicketsPerWarp);
    run = run < 1 ? 1 : (run > (unsigned long long)kEdgeMaxRun ? (unsigned long long)kEdgeMaxRun : run);
    P.lse_run = (int)run;
    P.emit_run = (int)run;
    P.n_lse_runs = (P.n_slices + P.lse_run - 1) / P.lse_run;
    P.n_emit_runs = (P.n_slices + P.emit_run - 1) / P.emit_run;
    P.total_lse = R * (unsigned long long)P.n_lse_runs;
    P.total_emit = (unsigned long long)P.B * (unsigned long long)P.n_emit_runs;
    P.spin_limit = 1u << 20;
    P.c1 = (float)(1.4426950408889634 / (double)P.temperature);
    edge_workspace_layout(P.B, P.gamma, P.n_lse_runs, &P, static_cast<char *>(workspace));
    if ((err = cudaMemsetAsync(workspace, 0xFF, P.fill_bytes, stream)) != cudaSuccess) return err;
    const unsigned long long tickets = P.total_lse + P.total_emit;
    const unsigned long long want = (tickets + kEdgeWarps - 1) / kEdgeWarps;
    const unsigned grid = (unsigned)(want < resident_ctas ? want : resident_ctas);
    if (dtype == DSSD_BF16) edge_verify_kernel<DSSD_BF16><<<grid, kEdgeThreads, kEdgeSmemBytes, stream>>>(P);
    else edge_verify_kernel<DSSD_F32><<<grid, kEdgeThreads, kEdgeSmemBytes, stream>>>(P);
    return cudaGetLastError();
}

}  // namespace dssd
