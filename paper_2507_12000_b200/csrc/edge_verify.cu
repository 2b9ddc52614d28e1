// Edge half of the verification round as one persistent, warp-specialised streaming kernel.
//
// One CTA per SM, launched cooperatively.  Lane 0 of warp 0 is the producer: it streams the logits
// global -> shared memory with bulk asynchronous copies (TMA, untiled) into a ring of kEdgeStages
// stages, each guarded by a "full" mbarrier (armed with the copy's bytes) and an "empty" mbarrier
// (one arrival per consumer warp).  Warps 1..kEdgeConsumers are consumers: every consumer takes a
// fixed 1/kEdgeConsumers share of each stage.  Then come the fold warp, which serves a mailbox in
// shared memory, and the scout warp, one thread of which does every round trip to global memory
// that scheduling needs (ticket draws, claims on EMIT work, look-ups of the drafted tokens) and
// hands the results to the producer through two small queues in shared memory.
//   LSE(row, run)    a run of consecutive stages of one target row (the whole row when it is
//                    short enough): every consumer keeps, per lane, an online maximum and sum of
//                    2^(l * c1 - ref2) in float32 over its shares.  At the run's last stage the
//                    consumers leave these per-lane pairs in a meeting area in shared memory
//                    (plain stores) and the last to arrive posts the ticket to the fold warp,
//                    which reduces the area to the ticket's partial (ref2, sum).  ref2 is an
//                    integer, so partials combine by exact power-of-two scaling.
//   EMIT(seq, run)   at most kEdgeEmitRun stages of row n of a folded sequence: the row is
//                    streamed again and p_row = 2^(l * c1 - ref2) / S is written.
// The fold warp stores each partial to global memory and counts it on its sequence; the fold
// warp that brings a sequence's last partial folds the sequence: one lane per position adds up
// the row's partials in float64 and evaluates the acceptance test, a ballot + find-first-set
// over the lanes gives the accepted length n, and the sequence's `ready` entry (n and row n's
// reference and 1/S) is written.  Scouts claim EMIT tickets with one atomic add when ready
// sequences have unclaimed tickets (or eagerly once their CTA has no LSE work left); an EMIT
// ticket goes before the next LSE stage, so the second read of row n follows the first as closely
// as the fold allows.
// Nothing on the global path waits on a fence: results travel through 8-byte slots that carry
// their own validity (the kernel itself sets the whole workspace to all ones before any CTA uses
// it: one grid-wide barrier at the start of the launch, overlapped with the first copies); a
// reader that sees the fill pattern asks again (bounded) for a store that a running warp has
// already issued.  The producer never touches global memory except to issue copies, so a freed
// stage of the ring is re-armed at once.  Apart from that start-up barrier, which the
// cooperative launch guarantees to complete, every wait is bounded; when one runs out the error
// word is set and the warps wind down.
#include "edge_verify.h"

#include <math.h>

#include <atomic>
#include <utility>

#include <cooperative_groups.h>

#include "dssd_device.cuh"
#include "edge_judge.cuh"

namespace dssd {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kS = kEdgeStageBytes;
constexpr int kNC = kEdgeConsumers;
constexpr int kVecPerWarp = kS / 16 / kNC;  // 16-byte vectors of a full stage per consumer warp
static_assert(kVecPerWarp >= 128 && kVecPerWarp % 128 == 0, "a consumer's share must be whole blocks of 4 vectors per lane");
constexpr int kBlocksPerWarp = kVecPerWarp / 128;
constexpr int kComb = 16;  // ticket records; tickets in flight in a CTA <= kEdgeStages + 1
static_assert(kComb >= kEdgeStages + 2 && kComb <= 16 && (kComb & (kComb - 1)) == 0, "ticket records");
constexpr int kMeet = 4;   // meeting areas where the consumers leave an LSE ticket's per-lane results for the fold warp
constexpr int kMail = 32;  // mailbox entries of the fold warp, a power of two

enum Kind : unsigned { kEnd = 0, kIdle = 1, kLse = 2, kEmit = 3 };
constexpr unsigned kMetaFirst = 4u, kMetaLast = 8u, kMetaRagged = 16u;  // first / last stage of its ticket; scalars outside the copy

// counters start at all ones (the pattern the workspace is cleared to): logical value = raw + 1
__device__ __forceinline__ unsigned logical(unsigned raw) { return raw + 1u; }
__device__ __forceinline__ unsigned long long logical(unsigned long long raw) { return raw + 1ull; }

template <int DT>
__device__ __forceinline__ const char *row_ptr(const EdgeParams &P, long long row)
{
    return static_cast<const char *>(P.logits) + (size_t)row * (size_t)P.row_stride * Elem<DT>::kBytes;
}

// A ticket as the CTA keeps it in shared memory, written by the producer before the ticket's
// first stage is armed and read by every consumer at that stage.
struct __align__(16) Ticket {
    long long row;      // LSE: the row; EMIT: row n of the sequence
    long long seq;      // the row's sequence
    long long out_off;  // EMIT: b * V, offset of the output row in p_row; < 0: write nothing
    int run;            // ticket index within the row (LSE: partial slot)
    int head;           // bytes before the row's first 16-byte boundary (scalar head of stage 0)
    float ref2, invS;   // EMIT
    int meet;           // LSE: meeting area of this ticket
    unsigned gen;       // LSE: number of earlier tickets of this CTA that used the same area
};
static_assert(sizeof(Ticket) == 48, "Ticket layout");

// What the producer writes for each stage before it arms the stage's full barrier:
//   x = kind | kMeta* | ticket slot << 5 | stage index within the row << 9
//   y = bytes that the copy brings into the stage, a multiple of 16
typedef uint2 StageDesc;
constexpr unsigned kMetaSlotShift = 5, kMetaKShift = 9;

// A ticket's partial on its way to the fold warp.
struct __align__(16) Mail {
    long long row;
    long long seq;
    int run;
    int meet;   // meeting area holding the consumers' results
    int valid;  // 0: free, 1: posted
    int pad;
};
static_assert(sizeof(Mail) == 32, "Mail layout");

// An EMIT ticket on its way from the scout to the producer.
struct __align__(16) EmitWork {
    Ticket t;
    int k_begin, k_end;
    int pad[2];
};
constexpr int kEmitQ = 2;  // powers of two
constexpr int kLseQ = 2;

struct Shared {  // carved from dynamic shared memory behind the ring
    Ticket ticket[kComb];
    StageDesc desc[kEdgeStages];
    unsigned long long full[kEdgeStages];
    unsigned long long empty[kEdgeStages];
    float2 lane_part[kMeet][kNC][32];  // per-lane (reference exponent or -inf, sum) of every consumer warp
    unsigned meet_cnt[kMeet];          // consumer warps that have left their results
    unsigned meet_gen[kMeet];          // tickets the fold warp has taken out of the area
    Mail mail[kMail];
    unsigned mail_tail;
    unsigned cons_done;
    // the scout's hand-offs to the producer (single writer, single reader each)
    EmitWork emit_q[kEmitQ];           // claimed EMIT tickets whose sequence is ready
    unsigned emit_pushed, emit_popped;
    unsigned long long lse_q[kLseQ];   // drawn LSE ticket numbers (one beyond the last ticket: no more)
    unsigned lse_pushed, lse_popped;
    unsigned lse_busy;                 // producer: it still has LSE stages to issue or LSE tickets to expect
    unsigned scout_done;               // scout: nothing further will be pushed
    unsigned abort;                    // producer: a wait ran out; everybody winds down
};

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
    f32x2 s0, s1, s2, s3;  // eight running sums, as four packed pairs
};

__device__ __forceinline__ void online_reset(Online &o)
{
    o.m = DSSD_NEG_INF;
    o.ref = 0.f;
    o.s0 = o.s1 = o.s2 = o.s3 = 0ull;
}

__device__ __forceinline__ float online_total(const Online &o)
{
    float a, b;
    unpack2(add2(add2(o.s0, o.s1), add2(o.s2, o.s3)), a, b);
    return a + b;
}

__device__ __forceinline__ void online_raise(Online &o, float bm, float c1)
{
    if (bm > o.m) {
        const float nref = rintf(bm * c1);
        const float f = (o.m == DSSD_NEG_INF) ? 0.f : ex2(o.ref - nref);  // an exact power of two
        const f32x2 ff = pack2(f, f);
        o.s0 = mul2(o.s0, ff);
        o.s1 = mul2(o.s1, ff);
        o.s2 = mul2(o.s2, ff);
        o.s3 = mul2(o.s3, ff);
        o.m = bm;
        o.ref = nref;
    }
}

__device__ __forceinline__ void online_add(Online &o, float z, float c1)
{
    online_raise(o, z, c1);
    o.s0 = add2(o.s0, pack2(ex2(fmaf(z, c1, -o.ref)), 0.f));
}

// acc += 2^(a * c1 - ref), 2^(b * c1 - ref)
__device__ __forceinline__ void add_pair(f32x2 &acc, float a, float b, f32x2 cc, f32x2 nn)
{
    float x, y;
    unpack2(fma2(pack2(a, b), cc, nn), x, y);
    acc = add2(acc, pack2(ex2(x), ex2(y)));
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
    const f32x2 cc = pack2(c1, c1), nn = pack2(-o.ref, -o.ref);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        add_pair(o.s0, bf16_lo(v[u].x), bf16_hi(v[u].x), cc, nn);
        add_pair(o.s1, bf16_lo(v[u].y), bf16_hi(v[u].y), cc, nn);
        add_pair(o.s2, bf16_lo(v[u].z), bf16_hi(v[u].z), cc, nn);
        add_pair(o.s3, bf16_lo(v[u].w), bf16_hi(v[u].w), cc, nn);
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
    const f32x2 cc = pack2(c1, c1), nn = pack2(-o.ref, -o.ref);
#pragma unroll
    for (int u = 0; u < 4; u += 2) {
        add_pair(o.s0, __uint_as_float(v[u].x), __uint_as_float(v[u].y), cc, nn);
        add_pair(o.s1, __uint_as_float(v[u].z), __uint_as_float(v[u].w), cc, nn);
        add_pair(o.s2, __uint_as_float(v[u + 1].x), __uint_as_float(v[u + 1].y), cc, nn);
        add_pair(o.s3, __uint_as_float(v[u + 1].z), __uint_as_float(v[u + 1].w), cc, nn);
    }
}

template <int DT>
__device__ __forceinline__ uint4 neg_inf_vec()
{
    return DT == DSSD_BF16 ? make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u)
                           : make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u);
}

// A consumer's share of one stage of an LSE ticket: vectors [v0, v1) of the stage.
template <int DT>
__device__ __forceinline__ void lse_consume(uint32_t stage, int v0, int v1, float c1, Online &o)
{
    const int lane = threadIdx.x & 31;
    const uint32_t base = stage + (uint32_t)(v0 + lane) * 16u;
    if (v1 - v0 == kVecPerWarp) {
#pragma unroll
        for (int blk = 0; blk < kBlocksPerWarp; ++blk) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = lds16(base + (uint32_t)(blk * 2048 + u * 512));
            accum_block<DT>(o, v, c1);
        }
        return;
    }
    const int nvec = v1 - v0;
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

// Scalar elements of stage k that lie outside its bulk copy: the head of the row (stage 0) and
// the tail of the row's last stage.  `fn(element index)` is called by one lane per element.
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

// out[0..3] = 2^(z * c1 - ref2) * invS for four logits, as two packed pairs
__device__ __forceinline__ void emit_quad(float *out, float z0, float z1, float z2, float z3, f32x2 cc, f32x2 nn, f32x2 ss)
{
    float a, b, c, d;
    unpack2(fma2(pack2(z0, z1), cc, nn), a, b);
    unpack2(fma2(pack2(z2, z3), cc, nn), c, d);
    unpack2(mul2(pack2(ex2(a), ex2(b)), ss), a, b);
    unpack2(mul2(pack2(ex2(c), ex2(d)), ss), c, d);
    st_stream16(out, a, b, c, d);
}

// A consumer's share of one stage of an EMIT ticket: body[e] = 2^(l_e * c1 - ref2) * invS for
// the `nbytes` bytes of logits at `stage`.
template <int DT>
__device__ __forceinline__ void emit_consume(uint32_t stage, int nbytes, float *body, float c1, float nref, float invS)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    const int nelem = nbytes / E::kBytes;
    const f32x2 cc = pack2(c1, c1), nn = pack2(nref, nref), ss = pack2(invS, invS);
    if ((reinterpret_cast<uintptr_t>(body) & 15u) == 0) {
        const int nquad = nelem >> 2;  // nbytes is a multiple of 16, so nelem is a multiple of 4
        if (DT == DSSD_BF16) {
            const uint32_t base = stage + (uint32_t)lane * 8u;
#pragma unroll 4
            for (int i = lane; i < nquad; i += 32) {
                const uint2 w = lds8(base + (uint32_t)(i - lane) * 8u);
                emit_quad(body + (size_t)i * 4, bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y), cc, nn, ss);
            }
        } else {
            const uint32_t base = stage + (uint32_t)lane * 16u;
#pragma unroll 4
            for (int i = lane; i < nquad; i += 32) {
                const uint4 w = lds16(base + (uint32_t)(i - lane) * 16u);
                emit_quad(body + (size_t)i * 4, __uint_as_float(w.x), __uint_as_float(w.y), __uint_as_float(w.z),
                          __uint_as_float(w.w), cc, nn, ss);
            }
        }
    } else {
        // output not 16-byte aligned here: coalesced 4-byte stores
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

// The same for the 16-bit payload: four probabilities rounded to IEEE binary16, one 8-byte store
__device__ __forceinline__ void emit_quad16(uint16_t *out, float z0, float z1, float z2, float z3, f32x2 cc, f32x2 nn, f32x2 ss)
{
    float a, b, c, d;
    unpack2(fma2(pack2(z0, z1), cc, nn), a, b);
    unpack2(fma2(pack2(z2, z3), cc, nn), c, d);
    unpack2(mul2(pack2(ex2(a), ex2(b)), ss), a, b);
    unpack2(mul2(pack2(ex2(c), ex2(d)), ss), c, d);
    st_stream8(out, pack_half2(a, b), pack_half2(c, d));
}

template <int DT>
__device__ __forceinline__ void emit_consume16(uint32_t stage, int nbytes, uint16_t *body, float c1, float nref, float invS)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    const int nelem = nbytes / E::kBytes;
    const f32x2 cc = pack2(c1, c1), nn = pack2(nref, nref), ss = pack2(invS, invS);
    if ((reinterpret_cast<uintptr_t>(body) & 7u) == 0) {
        const int nquad = nelem >> 2;
        if (DT == DSSD_BF16) {
            const uint32_t base = stage + (uint32_t)lane * 8u;
#pragma unroll 4
            for (int i = lane; i < nquad; i += 32) {
                const uint2 w = lds8(base + (uint32_t)(i - lane) * 8u);
                emit_quad16(body + (size_t)i * 4, bf16_lo(w.x), bf16_hi(w.x), bf16_lo(w.y), bf16_hi(w.y), cc, nn, ss);
            }
        } else {
            const uint32_t base = stage + (uint32_t)lane * 16u;
#pragma unroll 4
            for (int i = lane; i < nquad; i += 32) {
                const uint4 w = lds16(base + (uint32_t)(i - lane) * 16u);
                emit_quad16(body + (size_t)i * 4, __uint_as_float(w.x), __uint_as_float(w.y), __uint_as_float(w.z),
                            __uint_as_float(w.w), cc, nn, ss);
            }
        }
    } else {
        // output not 8-byte aligned here: coalesced 2-byte stores
        for (int i = lane; i < nelem; i += 32) {
            float z;
            if (DT == DSSD_BF16) {
                unsigned short h;
                asm volatile("ld.shared.u16 %0, [%1];" : "=h"(h) : "r"(stage + (uint32_t)i * 2u));
                z = __uint_as_float((uint32_t)h << 16);
            } else {
                asm volatile("ld.shared.f32 %0, [%1];" : "=f"(z) : "r"(stage + (uint32_t)i * 4u));
            }
            body[i] = to_half_bits(ex2(fmaf(z, c1, nref)) * invS);
        }
    }
}

// ---- the fold warp -------------------------------------------------------------------------

// Run by the fold warp that brought the last partial of sequence b.  One lane per position
// i = 0..gamma: the row's partials -> log-sum-exp (float64) -> acceptance test
//   u_i < min(1, p_i(x_i) / q_i(x_i));
// then the first-rejection scan over the lanes' acceptance bits (ballot + find-first-set) and
// the push of the sequence to `ready`.
template <int DT>
__device__ __noinline__ void fold_sequence(const EdgeParams &P, long long b)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    int n = P.gamma;
    unsigned fl = 0;
    float ref2_n = 0.f, invS_n = 0.f;
    bool any_timeout = false;
    for (int base = 0; base <= P.gamma; base += 32) {
        const int i = base + lane;
        const bool live = i <= P.gamma;
        const long long row = b * (P.gamma + 1) + (live ? i : 0);
        const unsigned long long *part = P.part + (size_t)row * P.n_lse_runs;
        // Everything this position needs is requested at once: the drafted token with its
        // probability and uniform, and the row's first partials; the logit of the drafted token
        // follows as soon as the token id is back.
        constexpr int kAhead = 4;
        unsigned long long pw[kAhead];
#pragma unroll
        for (int k = 0; k < kAhead; ++k) pw[k] = (live && k < P.n_lse_runs) ? ld_relaxed_u64(part + k) : 0ull;
        int x = -1;
        float zx = 0.f, qx = 0.f, ux = 0.f;
        bool owned = false;
        unsigned long long tz = 0ull, tq = 0ull;
        const bool tested = live && i < P.gamma;
        if (tested) {
            // the drafted token's logit, q_i(x_i) and u_i were looked up by the scout that drew the row's
            // first ticket and wait in the row's two slots: nothing here goes to DRAM or depends on another load
            tz = ld_relaxed_u64(P.tokz + row);
            tq = ld_relaxed_u64(P.tokq + row);
        }
        // The sequence's arrival counter says every ticket has been counted; a partial whose
        // store has not landed yet still shows the fill pattern and is polled for.
        float Rr = DSSD_NEG_INF;
        double S = 0.0;
        bool bad = false, timeout = false;
        if (tested) {
            for (unsigned it = 0; (unsigned)(tz >> 32) == kFull && it < P.spin_limit; ++it) {
                __nanosleep(32);
                tz = ld_relaxed_u64(P.tokz + row);
            }
            for (unsigned it = 0; (unsigned)(tq >> 32) == kFull && it < P.spin_limit; ++it) {
                __nanosleep(32);
                tq = ld_relaxed_u64(P.tokq + row);
            }
            if ((unsigned)(tz >> 32) == kFull || (unsigned)(tq >> 32) == kFull) timeout = true;
            owned = (unsigned)(tz >> 32) == 1u;  // the token lies in this row (this shard's slice of it)
            x = owned ? 0 : -1;                  // all that the test needs to know of the id
            zx = __uint_as_float((unsigned)tz);
            qx = __uint_as_float((unsigned)tq);
            ux = __uint_as_float((unsigned)(tq >> 32));
        }
        if (live) {
            for (int k = 0; k < P.n_lse_runs; ++k) {
                unsigned long long w = 0;
                if (k < kAhead) {
#pragma unroll
                    for (int j = 0; j < kAhead; ++j)
                        if (j == k) w = pw[j];
                } else {
                    w = ld_relaxed_u64(part + k);
                }
                const unsigned polls = row + 1 == P.test_drop_row_plus1 ? P.test_poll_limit : P.spin_limit;
                for (unsigned it = 0; (unsigned)w == kFull && it < polls; ++it) {
                    __nanosleep(32);
                    w = ld_relaxed_u64(part + k);
                }
                if ((unsigned)w == kFull) {
                    timeout = true;
                    continue;
                }
                add_partial(Rr, S, bad, __uint_as_float((unsigned)w), (double)__uint_as_float((unsigned)(w >> 32)));
            }
        }
        if (P.shard_sum) {
            // one shard of the vocabulary: the row's partial sum and the drafted token's logit (where
            // this shard holds it) go out as they are; the test is made once all shards' sums have met
            if (live) {
                P.shard_ref[row] = Rr == DSSD_NEG_INF ? 0.f : Rr;
                P.shard_sum[row] = (bad || timeout) ? (double)__int_as_float(0x7fc00000) : S;
                if (i < P.gamma) P.shard_tok_logit[(size_t)b * P.gamma + i] = owned ? zx : __int_as_float(0x7fc00000);
            }
            any_timeout = any_timeout || __any_sync(kFull, timeout);
            continue;
        }
        float Rs, invS;
        const unsigned bits = judge_position(P, b, i, live, Rr, S, bad, timeout, x, zx, qx, ux, Rs, invS);
        const unsigned rej = __ballot_sync(kFull, live && i < P.gamma && !(bits & kBitAccept));
        if (rej && n == P.gamma) n = base + __ffs(rej) - 1;
        fl |= (__ballot_sync(kFull, bits & kBitBadToken) ? DSSD_EDGE_FLAG_BAD_TOKEN : 0u) |
              (__ballot_sync(kFull, bits & kBitNonFinite) ? DSSD_EDGE_FLAG_NONFINITE : 0u) |
              (__ballot_sync(kFull, bits & kBitTimeout) ? DSSD_EDGE_FLAG_TIMEOUT : 0u);
        any_timeout = any_timeout || __any_sync(kFull, timeout);
        if (n >= base && n < base + 32) {
            ref2_n = __shfl_sync(kFull, Rs, n - base);
            invS_n = __shfl_sync(kFull, invS, n - base);
        }
    }
    if (P.shard_sum) {
        if (lane == 0 && any_timeout) *P.error = 1u;
        return;
    }
    if (lane == 0) {
        P.accept_len[b] = any_timeout ? -1 : n;
        if (P.flags) P.flags[b] = fl;
        if (any_timeout) *P.error = 1u;
        // the sequence's entry, then the count of ready sequences (nobody waits for either)
        unsigned long long *rs = reinterpret_cast<unsigned long long *>(P.ready + b);
        st_relaxed_u64(rs, (unsigned long long)(unsigned)b | ((unsigned long long)(unsigned)(any_timeout ? -1 : n) << 32));
        st_relaxed_u64(rs + 1, any_timeout ? 0ull
                                           : ((unsigned long long)__float_as_uint(ref2_n) |
                                              ((unsigned long long)__float_as_uint(invS_n) << 32)));
        atomicAdd(P.ready_count, 1u);
    }
}

// Serves the CTA's mailbox.  For each posted ticket: reduce the meeting area to the ticket's
// partial (ref2, sum), store it to global memory and count it on its sequence.  The count's
// result is not waited for: up to two are in flight, and they are looked at when no mail is
// waiting (or a third count is due), so posting partials always comes before folding.  Whoever
// brought a sequence's last partial folds it.
template <int DT>
__device__ __forceinline__ void fold_warp(const EdgeParams &P, Shared *sh)
{
    const int lane = threadIdx.x & 31;
    const unsigned per_seq = (unsigned)(P.gamma + 1) * (unsigned)P.n_lse_runs;
    int npend = 0;
    long long pend_b0 = 0, pend_b1 = 0;
    unsigned pend_raw0 = 0, pend_raw1 = 0;  // lane 0: raw results of the counts, oldest first
    auto resolve_oldest = [&]() {
        const bool last = logical(__shfl_sync(kFull, pend_raw0, 0)) == per_seq - 1u;
        const long long b = pend_b0;
        pend_b0 = pend_b1;
        pend_raw0 = pend_raw1;
        --npend;
        if (last) fold_sequence<DT>(P, b);
    };
    unsigned idle = 0;
    for (unsigned head = 0;;) {
        Mail *e = &sh->mail[head & (kMail - 1)];
        volatile int *valid = &e->valid;
        if (*valid) {
            idle = 0;
            if (npend == 2) resolve_oldest();
            __threadfence_block();
            const long long row = e->row, b = e->seq;
            const int run = e->run, meet = e->meet;
            // this lane's column of the meeting area, then across the lanes: the ticket's (ref2, sum)
            float2 c[kNC];
#pragma unroll
            for (int w = 0; w < kNC; ++w) {
                const volatile float *cp = reinterpret_cast<const volatile float *>(&sh->lane_part[meet][w][lane]);
                c[w].x = cp[0];
                c[w].y = cp[1];
            }
            float R = DSSD_NEG_INF;
            bool nan = false;
#pragma unroll
            for (int w = 0; w < kNC; ++w) {
                nan = nan || (c[w].y != c[w].y);
                if (c[w].y > 0.f) R = fmaxf(R, c[w].x);
            }
            float S = 0.f;
#pragma unroll
            for (int w = 0; w < kNC; ++w)
                if (c[w].y > 0.f) S += c[w].y * ex2(c[w].x - R);  // exact scaling
            const float Rt = warp_max(R);
            float sum = warp_sum(R == DSSD_NEG_INF ? 0.f : S * ex2(R - Rt));
            if (__any_sync(kFull, nan)) sum = __int_as_float(0x7fc00000);
            const float ref2 = Rt == DSSD_NEG_INF ? 0.f : Rt;
            __syncwarp();
            unsigned raw = 0;
            if (lane == 0) {
                __threadfence_block();
                *valid = 0;
                ++*(volatile unsigned *)&sh->meet_gen[meet];  // the area may be used again
                if (row + 1 != P.test_drop_row_plus1)  // (the test hook withholds this one store)
                    st_relaxed_u64(&P.part[(size_t)row * P.n_lse_runs + run],
                                   (unsigned long long)__float_as_uint(ref2) | ((unsigned long long)__float_as_uint(sum) << 32));
                raw = atomicAdd(&P.seq_cnt[b], 1u);
            }
            if (npend == 0) {
                pend_b0 = b;
                pend_raw0 = raw;
            } else {
                pend_b1 = b;
                pend_raw1 = raw;
            }
            ++npend;
            ++head;
            continue;
        }
        if (npend) {
            resolve_oldest();
            continue;
        }
        if (*(volatile unsigned *)&sh->cons_done == (unsigned)kNC) {
            // every consumer has left; anything they posted is visible by now
            __threadfence_block();
            if (*valid) continue;
            return;
        }
        if (++idle > P.spin_limit) {
            if (lane == 0) *P.error = 1u;  // waited too long
            return;
        }
        __nanosleep(200);
    }
}

// ---- the consumers -------------------------------------------------------------------------

// At an LSE ticket's last stage every consumer warp leaves its lanes' running (reference, sum)
// pairs in the ticket's meeting area - plain stores, no shuffles on the streaming warps - and the
// last warp to arrive posts the ticket to the fold warp, which does the reduction.
__device__ __forceinline__ void leave_and_post(const EdgeParams &P, Shared *sh, int w, const Ticket &t, const Online &o)
{
    const int lane = threadIdx.x & 31;
    // the area is free once the fold warp has taken out every earlier ticket that used it
    volatile unsigned *gen = &sh->meet_gen[t.meet];
    for (unsigned it = 0; *gen != t.gen && it < P.spin_limit; ++it) __nanosleep(64);
    if (*gen != t.gen) {
        if (lane == 0) *P.error = 1u;  // the fold warp is not keeping up: this ticket's partial is lost
        return;
    }
    sh->lane_part[t.meet][w][lane] = make_float2(o.m == DSSD_NEG_INF ? DSSD_NEG_INF : o.ref, online_total(o));
    __syncwarp();
    if (lane == 0) {
        __threadfence_block();
        if (atomicAdd(&sh->meet_cnt[t.meet], 1u) == (unsigned)(kNC - 1)) {
            sh->meet_cnt[t.meet] = 0;
            const unsigned ms = atomicAdd(&sh->mail_tail, 1u) & (kMail - 1);
            Mail *e = &sh->mail[ms];
            volatile int *valid = &e->valid;
            unsigned it = 0;
            while (*valid && it < P.spin_limit) {  // the fold warp is a whole mailbox behind
                __nanosleep(100);
                ++it;
            }
            if (*valid) {
                *P.error = 1u;
            } else {
                e->row = t.row;
                e->seq = t.seq;
                e->run = t.run;
                e->meet = t.meet;
                __threadfence_block();
                *valid = 1;
            }
        }
    }
}

template <int DT>
__device__ __forceinline__ void consumer_warp(const EdgeParams &P, Shared *sh, uint32_t ring, int w)
{
    using E = Elem<DT>;
    const int lane = threadIdx.x & 31;
    const float c1 = P.c1;
    const int v0 = w * kVecPerWarp;
    Online o;
    online_reset(o);
    // the LSE and the EMIT ticket in progress: an EMIT ticket may run between two stages of an LSE ticket
    Ticket lt, et;
    lt.row = lt.seq = 0;
    lt.out_off = -1;
    lt.run = lt.head = lt.meet = 0;
    lt.gen = 0;
    lt.ref2 = lt.invS = 0.f;
    et = lt;
    unsigned st = 0, par = 0;
    for (;;) {
        if (!mbar_wait(smem_addr(&sh->full[st]), par, P.spin_limit)) {
            if (lane == 0) *P.error = 1u;  // the producer went silent
            break;
        }
        const StageDesc d = sh->desc[st];
        const unsigned meta = d.x;
        const unsigned kind = meta & 3u;
        if (kind == kEnd) break;
        const unsigned slot = (meta >> kMetaSlotShift) & (kComb - 1);
        if (meta & kMetaFirst) {
            if (kind == kLse) {
                lt = sh->ticket[slot];
                online_reset(o);
            } else {
                et = sh->ticket[slot];
            }
        }
        const uint32_t stage = ring + st * (uint32_t)kS;
        const int k = (int)(meta >> kMetaKShift);
        const int nvec = (int)(d.y >> 4);
        const int v1 = min(nvec, v0 + kVecPerWarp);
        if (kind == kLse) {
            if (v1 > v0) lse_consume<DT>(stage, v0, v1, c1, o);
            if ((meta & kMetaRagged) && w == 0) {
                const char *rowp = row_ptr<DT>(P, lt.row);
                for_ragged<DT>(P, lt.head, k, [&](int64_t e) { online_add(o, E::load(rowp, e), c1); });
            }
        } else if (et.out_off >= 0) {
            const float nref = -et.ref2, invS = et.invS;
            const long long first = (et.head + (long long)k * kS + (long long)v0 * 16) / E::kBytes;
            if (P.p_row16) {
                uint16_t *outp = P.p_row16 + et.out_off;
                if (v1 > v0) emit_consume16<DT>(stage + (uint32_t)v0 * 16u, (v1 - v0) * 16, outp + first, c1, nref, invS);
                if ((meta & kMetaRagged) && w == 0) {
                    const char *rowp = row_ptr<DT>(P, et.row);
                    for_ragged<DT>(P, et.head, k,
                                   [&](int64_t e) { outp[e] = to_half_bits(ex2(fmaf(E::load(rowp, e), c1, nref)) * invS); });
                }
            } else {
                float *outp = P.p_row + et.out_off;
                if (v1 > v0) emit_consume<DT>(stage + (uint32_t)v0 * 16u, (v1 - v0) * 16, outp + first, c1, nref, invS);
                if ((meta & kMetaRagged) && w == 0) {
                    const char *rowp = row_ptr<DT>(P, et.row);
                    for_ragged<DT>(P, et.head, k, [&](int64_t e) { outp[e] = ex2(fmaf(E::load(rowp, e), c1, nref)) * invS; });
                }
            }
        }
        // release the stage: the arrival orders this warp's reads before the producer's next copy
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_addr(&sh->empty[st]));
        if (kind == kLse && (meta & kMetaLast)) leave_and_post(P, sh, w, lt, o);
        if (++st == (unsigned)kEdgeStages) {
            st = 0;
            par ^= 1u;
        }
    }
    __syncwarp();
    if (lane == 0) {
        __threadfence_block();
        atomicAdd(&sh->cons_done, 1u);
    }
}

// ---- the producer --------------------------------------------------------------------------

// ticket number -> (t / per, t % per).  `magic` = ceil(2^64 / per) when the host has checked
// that the multiply-high is exact for every ticket number of this launch, else 0.
__device__ __forceinline__ void split_ticket(unsigned long long t, int per, unsigned long long magic,
                                             unsigned long long &q, int &r)
{
    if (per == 1) {
        q = t;
        r = 0;
        return;
    }
    q = magic ? __umul64hi(t, magic) : t / (unsigned)per;
    r = (int)(t - q * (unsigned)per);
}

// A run of stages that the producer is issuing.
struct Run {
    unsigned kind;  // kEnd: none
    unsigned slot;  // ticket record
    int k, k_begin, k_end;
    const char *src;   // source of stage k's copy
    long long remain;  // bytes of the row's body from stage k on (may be <= 0)
    int head;
    bool evict_first;  // the copies carry the L2 evict_first hint
};

// The producer's claim on EMIT work advances one step per stage issued, and no step waits for
// memory: a value requested in one step is looked at in the next.
//   kWatch    nothing claimed; the counters of ready sequences and of claimed tickets are watched
//   kClaimed  one atomic add on emit_head is in flight
//   kLooking  the ticket is known; its sequence's `ready` entry has been requested
// A ticket whose sequence is not ready yet (claims are handed out in sequence order, sequences
// become ready in any order) simply stays in kLooking while the LSE work goes on.
enum ClaimState : int { kWatch = 0, kClaimed = 1, kLooking = 2 };
struct Claim {
    int state;
    unsigned ready_raw;           // last value loaded from ready_count
    unsigned long long head_raw;  // last value loaded from emit_head
    unsigned long long claim_raw; // result of the atomic add in flight
    unsigned long long ticket;    // kLooking: the claimed ticket
    unsigned long long w0, w1;    // kLooking: the two words of ready[sequence], as loaded
    bool exhausted;               // a claim came back beyond the last EMIT ticket
};

__device__ __forceinline__ void claim_watch(const EdgeParams &P, Claim &c)
{
    c.ready_raw = ld_relaxed_u32(P.ready_count);
    c.head_raw = ld_relaxed_u64(P.emit_head);
}

__device__ __forceinline__ void claim_look(const EdgeParams &P, Claim &c)
{
    unsigned long long b;
    int run;
    split_ticket(c.ticket, P.n_emit_runs, P.emit_magic, b, run);
    const unsigned long long *rs = reinterpret_cast<const unsigned long long *>(P.ready + b);
    c.w0 = ld_relaxed_u64(rs);
    c.w1 = ld_relaxed_u64(rs + 1);
}

// One step of the claim.  Returns true, with the ticket's fields of `t` and its stage range
// filled in, when an EMIT ticket can start now.
__device__ __forceinline__ bool claim_step(const EdgeParams &P, Claim &c, Ticket &t, int &k_begin, int &k_end, bool eager)
{
    if (c.state == kWatch) {
        const unsigned long long ready = (unsigned long long)logical(c.ready_raw);
        const unsigned long long head = logical(c.head_raw);
        // `eager` (nothing else left to do): claim the next ticket even before its sequence is
        // ready and watch its entry, which saves the round trips of noticing and claiming later
        if (!c.exhausted && (head < ready * (unsigned long long)P.n_emit_runs || (eager && head < P.total_emit))) {
            c.claim_raw = atomicAdd(P.emit_head, 1ull);
            c.state = kClaimed;
        } else {
            claim_watch(P, c);
        }
        return false;
    }
    if (c.state == kClaimed) {
        c.ticket = logical(c.claim_raw);
        if (c.ticket >= P.total_emit) {
            c.exhausted = true;
            c.state = kWatch;
            claim_watch(P, c);
            return false;
        }
        c.state = kLooking;
        claim_look(P, c);
        return false;
    }
    // kLooking
    if ((unsigned)c.w0 == kFull || (unsigned)c.w1 == kFull) {
        claim_look(P, c);  // not ready (or a store still on its way): ask again
        return false;
    }
    unsigned long long b;
    split_ticket(c.ticket, P.n_emit_runs, P.emit_magic, b, t.run);
    const int n = (int)(unsigned)(c.w0 >> 32);
    if (P.skip_bonus_row && n == P.gamma) {  // the bonus token is drawn from the logits: no row to emit
        c.state = kWatch;
        claim_watch(P, c);
        return false;
    }
    t.ref2 = __uint_as_float((unsigned)c.w1);
    t.invS = __uint_as_float((unsigned)(c.w1 >> 32));
    t.seq = (long long)b;
    t.out_off = n >= 0 ? (long long)b * P.V : -1ll;  // n < 0: a wait ran out while folding, nothing can be written
    t.row = t.seq * (P.gamma + 1) + (n < 0 ? 0 : n);
    k_begin = t.run * P.emit_run;
    k_end = min(P.n_slices, k_begin + P.emit_run);
    c.state = kWatch;
    claim_watch(P, c);
    return true;
}

template <int DT>
__device__ __forceinline__ void start_run(const EdgeParams &P, Shared *sh, Run &r, unsigned kind, Ticket &t, int k_begin,
                                          int k_end, unsigned &tickets, unsigned &lse_tickets)
{
    using E = Elem<DT>;
    const char *rowp = row_ptr<DT>(P, t.row);
    t.head = row_head_bytes<DT>(P, rowp);
    t.meet = 0;
    t.gen = 0;
    if (kind == kLse) {
        t.meet = (int)(lse_tickets % kMeet);
        t.gen = lse_tickets / kMeet;
        ++lse_tickets;
    }
    r.kind = kind;
    r.evict_first = kind == kEmit;  // an emitted row is never read again
    r.slot = tickets++ & (kComb - 1);
    // The record's previous ticket was started kComb tickets ago; every consumer read it at that
    // ticket's first stage, which has been released since (more than kEdgeStages stages ago).
    sh->ticket[r.slot] = t;
    r.k = r.k_begin = k_begin;
    r.k_end = k_end;
    r.head = t.head;
    r.src = rowp + t.head + (long long)k_begin * kS;
    r.remain = (long long)P.V * E::kBytes - t.head - (long long)k_begin * kS;
}

// The producer's position in the ring and in its tickets.  The first part of it is set up before
// the grid-wide barrier (see producer_prologue), the rest by producer_thread.
struct ProducerState {
    Run lr;  // the LSE run in progress
    unsigned st, par;
    unsigned issued, tickets, lse_tickets;
    bool lse_left;
};

// LSE ticket number `no` (< total_lse) -> its ticket record and stage range; starts the run
template <int DT>
__device__ __forceinline__ void start_lse_ticket(const EdgeParams &P, Shared *sh, Run &lr, unsigned long long no,
                                                 unsigned &tickets, unsigned &lse_tickets)
{
    Ticket t;
    unsigned long long row;
    split_ticket(no, P.n_lse_runs, P.lse_magic, row, t.run);
    t.row = (long long)row;
    t.seq = (row >> 32) == 0 ? (long long)((unsigned)row / (unsigned)(P.gamma + 1))
                             : (long long)(row / (unsigned)(P.gamma + 1));
    t.out_off = -1;
    t.ref2 = t.invS = 0.f;
    const int k_begin = t.run * P.lse_run;
    const int k_end = min(P.n_slices, k_begin + P.lse_run);
    start_run<DT>(P, sh, lr, kLse, t, k_begin, k_end, tickets, lse_tickets);
    // First reads leave L2 early too, so that the stream does not push the workspace's lines (the
    // counters and slots that every hand-off goes through) out of it.  The exception is the last
    // row of a short sequence, the likeliest one to be read again (with probability alpha^gamma).
    if (P.first_read_hint) {
        const unsigned pos = (unsigned)(row - (unsigned long long)t.seq * (unsigned)(P.gamma + 1));
        lr.evict_first = !(pos == (unsigned)P.gamma && P.gamma <= kEdgeKeepLastRowGamma);
    }
}

// Arms ring stage `st` with the next stage of run r and issues its copy.  The stage must be free.
__device__ __forceinline__ void issue_stage(Shared *sh, uint32_t ring, Run &r, unsigned &st, unsigned &par,
                                            unsigned &issued)
{
    const unsigned len = r.remain <= 0 ? 0u : (r.remain >= kS ? (unsigned)kS : (unsigned)r.remain);
    const unsigned bulk = len & ~15u;
    const bool ragged = (r.k == 0 && r.head != 0) || (len & 15u);
    const unsigned meta = r.kind | (r.k == r.k_begin ? kMetaFirst : 0u) | (r.k + 1 == r.k_end ? kMetaLast : 0u) |
                          (ragged ? kMetaRagged : 0u) | (r.slot << kMetaSlotShift) | ((unsigned)r.k << kMetaKShift);
    sh->desc[st] = make_uint2(meta, bulk);
    const uint32_t bar = smem_addr(&sh->full[st]);
    if (bulk) {
        mbar_arrive_expect_tx(bar, bulk);
        if (r.evict_first) bulk_g2s_hint(ring + st * (uint32_t)kS, r.src, bulk, bar, l2_policy_evict_first());
        else bulk_g2s(ring + st * (uint32_t)kS, r.src, bulk, bar);
    } else {
        mbar_arrive(bar);
    }
    ++issued;
    r.src += kS;
    r.remain -= kS;
    if (++r.k == r.k_end) r.kind = kEnd;
    if (++st == (unsigned)kEdgeStages) {
        st = 0;
        par ^= 1u;
    }
}

// Before the grid-wide barrier that follows the clearing of the workspace nothing of the workspace
// may be touched, but the logits may be read: every CTA's first LSE ticket is its own number
// (the ticket counter starts at the number of CTAs), and its first stages go out at once, into
// the still empty ring, so that the copies are in flight while the barrier completes.
template <int DT>
__device__ __forceinline__ void producer_prologue(const EdgeParams &P, Shared *sh, uint32_t ring, ProducerState &s)
{
    s.lr.kind = kEnd;
    s.st = 0;
    s.par = 1;  // a fresh barrier passes a wait on parity 1: the ring starts out empty
    s.issued = s.tickets = s.lse_tickets = 0;
    s.lse_left = true;
    const unsigned long long no = blockIdx.x;
    if (no >= P.total_lse) {
        s.lse_left = false;
        return;
    }
    start_lse_ticket<DT>(P, sh, s.lr, no, s.tickets, s.lse_tickets);
    for (int j = 0; j < kEdgeStages && s.lr.kind != kEnd; ++j) issue_stage(sh, ring, s.lr, s.st, s.par, s.issued);
}

// The producer issues stages and nothing else: which ticket comes next it learns from two small
// queues in shared memory that the scout fills, so no round trip to global memory ever stands
// between a freed stage of the ring and the next copy.
template <int DT>
__device__ __forceinline__ void producer_thread(const EdgeParams &P, Shared *sh, uint32_t ring, ProducerState &s)
{
    bool lse_left = s.lse_left;
    Run lr = s.lr, er;  // the LSE and the EMIT run in progress; an EMIT run goes first
    er.kind = kEnd;
    unsigned st = s.st, par = s.par;
    unsigned issued = s.issued, tickets = s.tickets, lse_tickets = s.lse_tickets, idle = 0;
    unsigned emit_popped = 0, lse_popped = 0;
    bool failed = false;
    volatile unsigned *emit_pushed = &sh->emit_pushed, *lse_pushed = &sh->lse_pushed, *scout_done = &sh->scout_done;
    for (;;) {
        if (er.kind == kEnd && *emit_pushed != emit_popped) {
            __threadfence_block();
            EmitWork w = sh->emit_q[emit_popped & (kEmitQ - 1)];
            ++emit_popped;
            __threadfence_block();
            *(volatile unsigned *)&sh->emit_popped = emit_popped;
            start_run<DT>(P, sh, er, kEmit, w.t, w.k_begin, w.k_end, tickets, lse_tickets);
        }
        if (er.kind == kEnd && lr.kind == kEnd && lse_left && *lse_pushed != lse_popped) {
            __threadfence_block();
            const unsigned long long no = sh->lse_q[lse_popped & (kLseQ - 1)];
            ++lse_popped;
            __threadfence_block();
            *(volatile unsigned *)&sh->lse_popped = lse_popped;
            if (no < P.total_lse) start_lse_ticket<DT>(P, sh, lr, no, tickets, lse_tickets);
            else lse_left = false;
        }
        {
            const unsigned busy = (lse_left || lr.kind != kEnd) ? 1u : 0u;
            if (*(volatile unsigned *)&sh->lse_busy != busy) *(volatile unsigned *)&sh->lse_busy = busy;
        }
        Run &r = er.kind != kEnd ? er : lr;
        if (r.kind == kEnd) {
            // nothing to issue: done once no LSE ticket is left and the scout has nothing more to hand over
            if (!lse_left && *scout_done && *emit_pushed == emit_popped) break;
            if (++idle > P.spin_limit) {
                failed = true;
                break;
            }
            __nanosleep(100);
            continue;
        }
        idle = 0;
        if (!mbar_wait(smem_addr(&sh->empty[st]), par, P.spin_limit)) {
            failed = true;  // the consumers went silent
            break;
        }
        issue_stage(sh, ring, r, st, par, issued);
    }
    if (!failed && mbar_wait(smem_addr(&sh->empty[st]), par, P.spin_limit)) {
        // tell the consumers that nothing follows
        sh->desc[st] = make_uint2(kEnd, 0u);
        mbar_arrive(smem_addr(&sh->full[st]));
        return;
    }
    // error exit: the consumers will run out of patience on their own.  Copies may still be in
    // flight into the ring; wait for them (bounded) before the CTA's shared memory can be handed
    // to another CTA.  The last min(issued, kEdgeStages) stages armed are st - 1, st - 2, ...
    *P.error = 1u;
    *(volatile unsigned *)&sh->abort = 1u;
    unsigned s2 = st, p2 = par;
    for (unsigned j = 0; j < (unsigned)kEdgeStages && j < issued; ++j) {
        if (s2 == 0) {
            s2 = kEdgeStages;
            p2 ^= 1u;
        }
        --s2;
        mbar_wait(smem_addr(&sh->full[s2]), p2 ^ 1u, P.spin_limit);  // armed in the pass whose empty parity was p2
    }
}


// The scout (one thread) does everything that needs a round trip to global memory on the
// producer's behalf: it draws the CTA's next LSE ticket (one ticket ahead) and runs the claim on
// EMIT work - watch the counters, claim a ticket, look up its sequence's `ready` entry - and
// pushes what it gets into the two queues.  Its loop runs at the pace of those round trips, which
// no longer matters to the stream.
template <int DT>
__device__ __forceinline__ void scout_thread(const EdgeParams &P, Shared *sh)
{
    using E = Elem<DT>;
    Claim c;
    c.state = kWatch;
    c.exhausted = false;
    c.claim_raw = c.ticket = c.w0 = c.w1 = 0;
    claim_watch(P, c);
    bool more_lse = (unsigned long long)blockIdx.x < P.total_lse;  // else the CTA never had an LSE ticket
    bool lse_pending = false;
    unsigned long long lse_raw = 0;
    // Towards the end of the launch no new EMIT ticket is claimed while LSE work is left: the last
    // waves of LSE tickets then finish sooner (their sequences complete sooner) and the rows held
    // back fill the time in which the final sequences complete, on all CTAs, in short tickets.
    bool endgame = (unsigned long long)blockIdx.x + P.endgame_tickets >= P.total_lse;
    unsigned emit_pushed = 0, lse_pushed = 0, idle = 0;
    volatile unsigned *emit_popped = &sh->emit_popped, *lse_popped = &sh->lse_popped, *lse_busy = &sh->lse_busy,
                      *abort = &sh->abort;
    EmitWork w;
    bool have = false;  // a claimed, ready EMIT ticket waiting for room in the queue
    // Whoever draws the first ticket of a row also looks up the row's drafted token and that token's
    // logit (and, when the draft rows are given, its probability) and leaves them in the row's slots,
    // long before the sequence is folded.  One look-up at a time: 0 idle, 1 the token id has been
    // asked for, 2 the values have been asked for.
    int pf = 0, pf_x = 0;
    long long pf_row = 0;
    size_t pf_di = 0;
    float pf_z = 0.f, pf_q = 0.f, pf_u = 0.f;
    bool pf_owned = false;
    auto pf_advance = [&]() {
        if (pf == 1) {
            // (a shard of the vocabulary holds entries v_begin .. v_begin + V - 1; v_begin is 0 otherwise)
            const long long xl = (long long)pf_x - (long long)P.v_begin;
            pf_owned = xl >= 0 && xl < (long long)P.V;
            pf_z = pf_owned ? E::load(row_ptr<DT>(P, pf_row), xl) : 0.f;
            // a token id outside the vocabulary has no q: NaN (the id itself gets the position rejected and flagged)
            if (P.draft_q_rows)
                pf_q = (pf_x >= 0 && pf_x < P.V) ? __ldg(P.draft_q_rows + pf_di * (size_t)P.V + (size_t)pf_x) : __int_as_float(0x7fc00000);
            pf = 2;
        } else if (pf == 2) {
            st_relaxed_u64(P.tokz + pf_row, (unsigned long long)__float_as_uint(pf_z) | ((unsigned long long)(pf_owned ? 1u : 0u) << 32));
            // (q_i(x_i), u_i): a NaN is stored as the canonical one, so that the pair never equals the all-ones pattern
            const float qs = pf_q != pf_q ? __int_as_float(0x7fc00000) : pf_q, us = pf_u != pf_u ? __int_as_float(0x7fc00000) : pf_u;
            st_relaxed_u64(P.tokq + pf_row, (unsigned long long)__float_as_uint(qs) | ((unsigned long long)__float_as_uint(us) << 32));
            pf = 0;
        }
    };
    auto pf_start = [&](unsigned long long no) {
        unsigned long long row;
        int run;
        split_ticket(no, P.n_lse_runs, P.lse_magic, row, run);
        const unsigned i = (unsigned)(row % (unsigned)(P.gamma + 1));
        if (run != 0 || (int)i >= P.gamma) return;
        while (pf) pf_advance();
        pf_row = (long long)row;
        pf_di = (size_t)(row / (unsigned)(P.gamma + 1)) * (size_t)P.gamma + i;
        pf_x = P.draft_tokens[pf_di];
        pf_u = P.uniforms ? P.uniforms[pf_di] : 0.f;
        if (P.draft_q_tok) pf_q = P.draft_q_tok[pf_di];
        pf = 1;
    };
    if (more_lse) pf_start(blockIdx.x);
    for (;;) {
        if (*abort) {
            while (pf) pf_advance();
            return;
        }
        pf_advance();
        // the next LSE ticket: drawn as soon as the producer has taken the one before
        if (more_lse && !lse_pending && lse_pushed == *lse_popped) {
            lse_raw = atomicAdd(P.lse_ticket, 1ull);
            lse_pending = true;
        }
        const bool busy = *lse_busy != 0u || more_lse;
        if (have) {
            if (emit_pushed - *emit_popped < (unsigned)kEmitQ) {
                sh->emit_q[emit_pushed & (kEmitQ - 1)] = w;
                __threadfence_block();
                *(volatile unsigned *)&sh->emit_pushed = ++emit_pushed;
                have = false;
                idle = 0;
            }
        } else {
            const bool hold = endgame && busy && c.state == kWatch;
            if (!hold) {
                const int before = c.state;
                have = claim_step(P, c, w.t, w.k_begin, w.k_end, !busy);
                if (have || c.state != before) idle = 0;
            } else if (!lse_pending) {
                __nanosleep(200);  // nothing to ask memory for: do not take issue slots from the working warps
            }
        }
        if (lse_pending) {  // asked for at the top of this pass, or earlier: by now it is usually back
            const unsigned long long no = logical(lse_raw);
            lse_pending = false;
            endgame = no + P.endgame_tickets >= P.total_lse;
            if (no >= P.total_lse) more_lse = false;
            else pf_start(no);
            sh->lse_q[lse_pushed & (kLseQ - 1)] = no;  // a number beyond the last ticket tells the producer that none is left
            __threadfence_block();
            *(volatile unsigned *)&sh->lse_pushed = ++lse_pushed;
            idle = 0;
        }
        // done once no LSE ticket is left anywhere, no claim is under way, nothing waits here and every
        // EMIT ticket has been claimed by someone
        if (!more_lse && !have && pf == 0 && c.state == kWatch && (c.exhausted || logical(c.head_raw) >= P.total_emit)) {
            __threadfence_block();
            *(volatile unsigned *)&sh->scout_done = 1u;
            return;
        }
        if (++idle > P.spin_limit) {
            while (pf) pf_advance();
            *P.error = 1u;  // waited too long (for a sequence to become ready, or for the producer)
            *(volatile unsigned *)&sh->scout_done = 1u;
            return;
        }
        if (have || (c.state == kWatch && !busy)) __nanosleep(100);
    }
}

// ---- small launches: one thread-block cluster per sequence, no workspace -----------------------
//
// When the whole batch fits one CTA per SM with a small share each, the hand-offs of the streaming
// kernel (tickets, partials in global memory, the workspace fill) cost more than the streaming
// itself.  Here a cluster of 1, 2, 4 or 8 CTAs of 1024 threads does a whole sequence: every CTA
// streams its share of every row with 16-byte loads into the same per-lane online sums, the
// CTAs' per-row results meet in the shared memory of the cluster's first CTA (distributed shared
// memory, hardware cluster barrier), whose warp 0 judges the positions (same arithmetic as the
// fold warp) and finds n; then every CTA streams its share of row n again (from L2) and writes
// p_row.  Same results as the streaming kernel up to the order of the float32 sums.

constexpr int kSmallThreads = 1024;
constexpr int kSmallWarps = kSmallThreads / 32;
constexpr int kSmallMaxRows = 64;                 // gamma + 1 at most
constexpr int kSmallMaxCluster = 8;               // CTAs per sequence at most (the portable cluster size)
constexpr long long kSmallCtaBytes = 32 << 10;                        // share of a sequence aimed at per CTA
constexpr long long kSmallMaxCtaBytes = 128 << 10;   // ... and the most a CTA takes

template <int DT>
__global__ void __launch_bounds__(kSmallThreads, 1) edge_small_kernel(const __grid_constant__ EdgeParams P)
{
    using E = Elem<DT>;
    namespace cg = cooperative_groups;
    cg::cluster_group cluster = cg::this_cluster();
    const int crank = (int)cluster.block_rank(), csize = (int)cluster.num_blocks();  // CTAs sharing this sequence
    __shared__ float2 s_part[kSmallMaxRows][kSmallWarps];
    __shared__ float2 s_clu[kSmallMaxRows][kSmallMaxCluster];  // rank 0: every CTA's (ref2, sum) per row
    __shared__ int s_x[kSmallMaxRows];
    __shared__ float s_zx[kSmallMaxRows], s_q[kSmallMaxRows], s_u[kSmallMaxRows];
    __shared__ int s_n;
    __shared__ float s_ref2, s_invS;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long b = blockIdx.x / csize;
    const float c1 = P.c1;
    const long long rowbytes = (long long)P.V * E::kBytes;
    // A CTA's shared memory may be written by its peers only once it is known to have started:
    // every CTA announces itself here, and the matching wait stands before the first remote
    // store (the streaming loop lies between the two, so the wait costs nothing).
    if (csize > 1) (void)cluster.barrier_arrive();
    // Every CTA of the cluster takes a contiguous 1/csize of each row's 16-byte vectors.
    // The rows are streamed side by side, a group of `wpr` warps per row, so that the loads of
    // all rows are in flight together; the first lane of each group also fetches the row's
    // drafted token, its probability and uniform, and (once the token id is back) its logit.
    const int rows = P.gamma + 1;
    const int wpr = rows >= kSmallWarps ? 1 : kSmallWarps / rows;  // warps per row
    const int groups = kSmallWarps / wpr;                           // rows in flight at once
    const int g = warp / wpr, wi = warp - g * wpr, gthreads = wpr * 32, t = wi * 32 + lane;
    for (int i = g; i < rows && g < groups; i += groups) {
        const char *rowp = row_ptr<DT>(P, b * rows + i);
        const int head = row_head_bytes<DT>(P, rowp);
        const long long body = rowbytes - head;
        const int nvec = (int)(body >> 4);
        const uint4 *v4 = reinterpret_cast<const uint4 *>(rowp + head);
        const int vbeg = (int)((long long)nvec * crank / csize), vend = (int)((long long)nvec * (crank + 1) / csize);
        const bool scout = t == 0 && i < P.gamma && crank == 0;
        int x = -1;
        float qx = 0.f, ux = 0.f, zx = 0.f;
        if (scout) {
            const size_t di = (size_t)b * P.gamma + i;
            x = P.draft_tokens[di];
            qx = P.draft_q_tok[di];
            ux = P.uniforms[di];
        }
        Online o;
        online_reset(o);
        bool asked = false;
        for (int j = vbeg + t; j < vend; j += 4 * gthreads) {
            uint4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = (j + u * gthreads < vend) ? ld_stream16(v4 + j + u * gthreads) : neg_inf_vec<DT>();
            if (scout && !asked) {  // the token id is back by now: its logit travels with the next loads
                if (x >= 0 && x < P.V) zx = E::load(rowp, x);
                asked = true;
            }
            accum_block<DT>(o, v, c1);
        }
        if (scout && !asked && x >= 0 && x < P.V) zx = E::load(rowp, x);
        if (wi == 0 && crank == 0) {  // the scalars before the first and after the last 16-byte vector
            if (lane < head / E::kBytes) online_add(o, E::load(rowp, lane), c1);
            const int tail = (int)((body - ((long long)nvec << 4)) / E::kBytes);
            if (lane < tail) online_add(o, E::load(rowp, (int64_t)((head + ((long long)nvec << 4)) / E::kBytes) + lane), c1);
        }
        const bool empty = (o.m == DSSD_NEG_INF);
        const float R = warp_max(empty ? DSSD_NEG_INF : o.ref);
        float sum = online_total(o);
        sum = warp_sum(empty ? 0.f : sum * ex2(o.ref - R));  // exact scaling
        if (lane == 0) s_part[i][wi] = make_float2(R == DSSD_NEG_INF ? 0.f : R, sum);
        if (scout) {
            s_x[i] = x;
            s_zx[i] = zx;
            s_q[i] = qx;
            s_u[i] = ux;
        }
    }
    __syncthreads();
    if (csize > 1) cluster.barrier_wait();  // every CTA of the cluster is running
    // each CTA's result per row goes to rank 0's shared memory (distributed shared memory)
    if (tid < rows) {
        float R = DSSD_NEG_INF;
        bool nan = false;
        for (int k = 0; k < wpr; ++k) {
            const float2 c = s_part[tid][k];
            nan = nan || (c.y != c.y);
            if (c.y > 0.f) R = fmaxf(R, c.x);
        }
        float S = 0.f;
        for (int k = 0; k < wpr; ++k) {
            const float2 c = s_part[tid][k];
            if (c.y > 0.f) S += c.y * ex2(c.x - R);  // exact scaling
        }
        if (nan) S = __int_as_float(0x7fc00000);
        float2 *dst = cluster.map_shared_rank(&s_clu[tid][crank], 0);
        *dst = make_float2(R == DSSD_NEG_INF ? 0.f : R, S);
    }
    if (csize == 1) __syncthreads();
    else cluster.sync();
    if (warp == 0 && crank == 0) {
        int n = P.gamma;
        unsigned fl = 0;
        float ref2_n = 0.f, invS_n = 0.f;
        for (int base = 0; base <= P.gamma; base += 32) {
            const int i = base + lane;
            const bool live = i <= P.gamma;
            int x = -1;
            float zx = 0.f, qx = 0.f, ux = 0.f;
            if (live && i < P.gamma) {
                x = s_x[i];
                zx = s_zx[i];
                qx = s_q[i];
                ux = s_u[i];
            }
            float Rr = DSSD_NEG_INF;
            double S = 0.0;
            bool bad = false;
            if (live) {
                for (int k = 0; k < csize; ++k) {
                    const float2 c = s_clu[i][k];
                    add_partial(Rr, S, bad, c.x, (double)c.y);
                }
            }
            float Rs, invS;
            const unsigned bits = judge_position(P, b, i, live, Rr, S, bad, false, x, zx, qx, ux, Rs, invS);
            const unsigned rej = __ballot_sync(kFull, live && i < P.gamma && !(bits & kBitAccept));
            if (rej && n == P.gamma) n = base + __ffs(rej) - 1;
            fl |= (__ballot_sync(kFull, bits & kBitBadToken) ? DSSD_EDGE_FLAG_BAD_TOKEN : 0u) |
                  (__ballot_sync(kFull, bits & kBitNonFinite) ? DSSD_EDGE_FLAG_NONFINITE : 0u);
            if (n >= base && n < base + 32) {
                ref2_n = __shfl_sync(kFull, Rs, n - base);
                invS_n = __shfl_sync(kFull, invS, n - base);
            }
        }
        if (lane == 0) {
            P.accept_len[b] = n;
            if (P.flags) P.flags[b] = fl;
            for (int r = 0; r < csize; ++r) {  // the verdict goes to every CTA of the cluster
                *cluster.map_shared_rank(&s_n, r) = n;
                *cluster.map_shared_rank(&s_ref2, r) = ref2_n;
                *cluster.map_shared_rank(&s_invS, r) = invS_n;
            }
        }
    }
    if (csize == 1) __syncthreads();
    else cluster.sync();
    // row n once more, every CTA its share: p_row[b, v] = 2^(l_v * c1 - ref2) / S.  No CTA reads
    // another CTA's shared memory from here on, so the CTAs may leave in any order.
    {
        const int n = s_n;
        const float ref2 = s_ref2, invS = s_invS;
        const char *rowp = row_ptr<DT>(P, b * (P.gamma + 1) + n);
        const int head = row_head_bytes<DT>(P, rowp);
        const long long body = rowbytes - head;
        const int nvec = (int)(body >> 4);
        const uint4 *v4 = reinterpret_cast<const uint4 *>(rowp + head);
        const float nref = -ref2;
        const f32x2 cc = pack2(c1, c1), nn = pack2(nref, nref), ss = pack2(invS, invS);
        const int vbeg = (int)((long long)nvec * crank / csize), vend = (int)((long long)nvec * (crank + 1) / csize);
        if (P.p_row16) {
            uint16_t *outp = P.p_row16 + (size_t)b * P.V;
            uint16_t *bodyp = outp + head / E::kBytes;
            const bool vec_out = (reinterpret_cast<uintptr_t>(bodyp) & 7u) == 0;
            for (int j = vbeg + tid; j < vend; j += kSmallThreads) {
                float f[E::kVec];
                E::unpack(ld_stream16(v4 + j), f);
                uint16_t *o = bodyp + (size_t)j * E::kVec;
                if (vec_out) {
#pragma unroll
                    for (int q = 0; q < E::kVec; q += 4) emit_quad16(o + q, f[q], f[q + 1], f[q + 2], f[q + 3], cc, nn, ss);
                } else {
#pragma unroll
                    for (int q = 0; q < E::kVec; ++q) o[q] = to_half_bits(ex2(fmaf(f[q], c1, nref)) * invS);
                }
            }
            if (warp == 0 && crank == 0) {
                if (lane < head / E::kBytes) outp[lane] = to_half_bits(ex2(fmaf(E::load(rowp, lane), c1, nref)) * invS);
                const int tail = (int)((body - ((long long)nvec << 4)) / E::kBytes);
                const int64_t e = (int64_t)((head + ((long long)nvec << 4)) / E::kBytes) + lane;
                if (lane < tail) outp[e] = to_half_bits(ex2(fmaf(E::load(rowp, e), c1, nref)) * invS);
            }
            return;
        }
        float *outp = P.p_row + (size_t)b * P.V;
        float *bodyp = outp + head / E::kBytes;
        const bool vec_out = (reinterpret_cast<uintptr_t>(bodyp) & 15u) == 0;
        for (int j = vbeg + tid; j < vend; j += kSmallThreads) {
            float f[E::kVec];
            E::unpack(ld_stream16(v4 + j), f);
            float *o = bodyp + (size_t)j * E::kVec;
            if (vec_out) {
#pragma unroll
                for (int q = 0; q < E::kVec; q += 4) emit_quad(o + q, f[q], f[q + 1], f[q + 2], f[q + 3], cc, nn, ss);
            } else {
#pragma unroll
                for (int q = 0; q < E::kVec; ++q) o[q] = ex2(fmaf(f[q], c1, nref)) * invS;
            }
        }
        if (warp == 0 && crank == 0) {
            if (lane < head / E::kBytes) outp[lane] = ex2(fmaf(E::load(rowp, lane), c1, nref)) * invS;
            const int tail = (int)((body - ((long long)nvec << 4)) / E::kBytes);
            const int64_t e = (int64_t)((head + ((long long)nvec << 4)) / E::kBytes) + lane;
            if (lane < tail) outp[e] = ex2(fmaf(E::load(rowp, e), c1, nref)) * invS;
        }
    }
}

constexpr size_t kEdgeSmemBytes = (size_t)kEdgeStages * kS + sizeof(Shared);

// The workspace is cleared inside the kernel: every slot and counter to all ones, except the LSE
// ticket counter, which starts at the number of CTAs (every CTA's first ticket is its own number).
__device__ __forceinline__ void clear_workspace(const EdgeParams &P)
{
    uint4 *w = reinterpret_cast<uint4 *>(P.lse_ticket);  // the workspace starts with the counters
    const size_t n = P.fill_bytes / 16;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        uint4 v = make_uint4(kFull, kFull, kFull, kFull);
        if (i == 0) {  // raw value of the 64-bit counter: logical value - 1
            v.x = gridDim.x - 1u;
            v.y = 0u;
        }
        w[i] = v;
    }
}

// Launched cooperatively (all CTAs resident), which is what allows the one grid-wide barrier
// between the clearing of the workspace and its first use.  The barrier is split: every CTA
// arrives once its share of the workspace is cleared, its producer sends the first copies on their
// way, and only then does the CTA wait for the others; no CTA waits for anything before it has
// arrived, so the barrier always completes.
template <int DT>
__global__ void __launch_bounds__(kEdgeThreads, 1) edge_verify_kernel(const __grid_constant__ EdgeParams P)
{
    extern __shared__ __align__(128) unsigned char smem[];
    namespace cg = cooperative_groups;
    cg::grid_group grid = cg::this_grid();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t ring = smem_addr(smem);
    Shared *sh = reinterpret_cast<Shared *>(smem + (size_t)kEdgeStages * kS);
    if (threadIdx.x == 0) {
#pragma unroll
        for (int st = 0; st < kEdgeStages; ++st) {
            mbar_init(smem_addr(&sh->full[st]), 1u);
            mbar_init(smem_addr(&sh->empty[st]), (unsigned)kNC);
        }
        for (int i = 0; i < kMeet; ++i) sh->meet_cnt[i] = sh->meet_gen[i] = 0;
        for (int i = 0; i < kMail; ++i) sh->mail[i].valid = 0;
        sh->mail_tail = 0;
        sh->cons_done = 0;
        sh->emit_pushed = sh->emit_popped = sh->lse_pushed = sh->lse_popped = 0;
        sh->lse_busy = 1;
        sh->scout_done = sh->abort = 0;
        mbar_init_fence();
    }
    clear_workspace(P);
    auto arrived = grid.barrier_arrive();  // (a CTA-wide barrier is part of it)
    ProducerState ps;
    if (threadIdx.x == 0) producer_prologue<DT>(P, sh, ring, ps);
    grid.barrier_wait(std::move(arrived));
    if (warp == 0) {
        if (lane == 0) producer_thread<DT>(P, sh, ring, ps);
    } else if (warp <= kNC) {
        consumer_warp<DT>(P, sh, ring, warp - 1);
    } else if (warp == kNC + 1) {
        fold_warp<DT>(P, sh);
    } else {
        if (lane == 0) scout_thread<DT>(P, sh);
    }
}

}  // namespace

int edge_max_runs_per_row(int V)
{
    const long long n = ((long long)V * 4 + kS - 1) / kS;
    return (int)(n < 1 ? 1 : n);
}

size_t edge_workspace_layout(int B, int gamma, int runs_per_row, EdgeParams *P, char *base)
{
    // the kernel sets all of it to 0xFF before use: counters then read "logical 0", slots "not yet"
    const size_t R = (size_t)B * (size_t)(gamma + 1);
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += (bytes + 255) & ~(size_t)255;
        return o;
    };
    const size_t o_ctr = take(512);  // four counters, each on its own 128-byte line
    const size_t o_seqcnt = take((size_t)B * 4);
    const size_t o_ready = take((size_t)B * sizeof(ReadySlot));
    const size_t o_part = take(R * (size_t)runs_per_row * 8);
    const size_t o_tokz = take(R * 8);
    const size_t o_tokq = take(R * 8);
    if (P) {
        P->tokz = reinterpret_cast<unsigned long long *>(base + o_tokz);
        P->tokq = reinterpret_cast<unsigned long long *>(base + o_tokq);
        P->lse_ticket = reinterpret_cast<unsigned long long *>(base + o_ctr);
        P->emit_head = reinterpret_cast<unsigned long long *>(base + o_ctr + 128);
        P->ready_count = reinterpret_cast<unsigned *>(base + o_ctr + 256);
        P->error = reinterpret_cast<unsigned *>(base + o_ctr + 384);
        P->seq_cnt = reinterpret_cast<unsigned *>(base + o_seqcnt);
        P->ready = reinterpret_cast<ReadySlot *>(base + o_ready);
        P->part = reinterpret_cast<unsigned long long *>(base + o_part);
        P->fill_bytes = off;
    }
    return off;
}

// launch geometry per device, filled on first use (occupancy depends on the compiled kernel only).
// g_sm_count is published last (release) and read first (acquire): a concurrent first call finds
// either 0 and looks the constants up itself, or the complete set.
static std::atomic<int> g_edge_ctas_per_sm[64][2];
static std::atomic<int> g_sm_count[64];

cudaError_t edge_verify_launch(EdgeParams &P, int dtype, void *workspace, cudaStream_t stream)
{
    cudaError_t err;
    int dev = 0;
    if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    int sm_count = g_sm_count[dev].load(std::memory_order_acquire);
    if (sm_count == 0) {
        int sms = 0, occ0 = 0, occ1 = 0;
        if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
        if ((err = cudaFuncSetAttribute(edge_verify_kernel<DSSD_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kEdgeSmemBytes)) != cudaSuccess) return err;
        if ((err = cudaFuncSetAttribute(edge_verify_kernel<DSSD_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kEdgeSmemBytes)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ0, edge_verify_kernel<DSSD_F32>, kEdgeThreads, kEdgeSmemBytes)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ1, edge_verify_kernel<DSSD_BF16>, kEdgeThreads, kEdgeSmemBytes)) != cudaSuccess) return err;
        if (occ0 < 1 || occ1 < 1) return cudaErrorLaunchOutOfResources;
        g_edge_ctas_per_sm[dev][0].store(occ0, std::memory_order_relaxed);
        g_edge_ctas_per_sm[dev][1].store(occ1, std::memory_order_relaxed);
        g_sm_count[dev].store(sms, std::memory_order_release);
        sm_count = sms;
    }
    const int ctas_per_sm = g_edge_ctas_per_sm[dev][dtype == DSSD_BF16].load(std::memory_order_relaxed);
    const int esz = dtype == DSSD_BF16 ? 2 : 4;
    P.c1 = (float)(1.4426950408889634 / (double)P.temperature);
    // Without an output row (the fused verification of Algorithm 1) nothing is emitted: there are no
    // EMIT tickets, and what the draw needs about row n stays in the workspace (`ready`).
    const bool no_emit = !P.p_row && !P.p_row16;
    // small launches: a cluster of 1..8 CTAs per sequence, no workspace, one launch
    if (!no_emit && !P.skip_bonus_row && !P.draft_q_rows && !P.shard_sum && !P.test_drop_row_plus1) {
        const long long seq_bytes = (long long)(P.gamma + 1) * P.V * esz;
        int csize = 1;
        while (csize < kSmallMaxCluster && seq_bytes / csize > kSmallCtaBytes) csize *= 2;
        while (csize > 1 && (long long)P.B * csize > sm_count) csize /= 2;
        if (P.gamma + 1 <= kSmallMaxRows && seq_bytes / csize <= kSmallMaxCtaBytes &&
            (long long)P.B * csize <= sm_count) {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3((unsigned)(P.B * csize));
            cfg.blockDim = dim3(kSmallThreads);
            cfg.dynamicSmemBytes = 0;
            cfg.stream = stream;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeClusterDimension;
            attr[0].val.clusterDim.x = (unsigned)csize;
            attr[0].val.clusterDim.y = 1;
            attr[0].val.clusterDim.z = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            if (dtype == DSSD_BF16) return cudaLaunchKernelEx(&cfg, edge_small_kernel<DSSD_BF16>, P);
            return cudaLaunchKernelEx(&cfg, edge_small_kernel<DSSD_F32>, P);
        }
    }
    const unsigned long long R = (unsigned long long)P.B * (unsigned long long)(P.gamma + 1);
    const long long n_slices = ((long long)P.V * esz + kS - 1) / kS;
    P.n_slices = (int)(n_slices < 1 ? 1 : n_slices);
    const unsigned long long resident_ctas = (unsigned long long)sm_count * (unsigned long long)ctas_per_sm;
    // Stages per ticket: as long as every resident CTA still gets about kEdgeTicketsPerCta
    // tickets, at most kEdgeMaxRun, and then evened out so that a row splits into equal tickets.
    unsigned long long run = (R * (unsigned long long)P.n_slices) / (resident_ctas * kEdgeTicketsPerCta);
    run = run < 1 ? 1 : (run > (unsigned long long)kEdgeMaxRun ? (unsigned long long)kEdgeMaxRun : run);
    const int runs_per_row = (int)((P.n_slices + run - 1) / run);
    run = (unsigned long long)((P.n_slices + runs_per_row - 1) / runs_per_row);
    P.lse_run = (int)run;
    // EMIT tickets stay short: they cost the consumers nothing per ticket, and at the end of the
    // launch the last sequences' rows are then written by several CTAs at once
    P.emit_run = (int)(run < (unsigned long long)kEdgeEmitRun ? run : (unsigned long long)kEdgeEmitRun);
    P.n_lse_runs = (P.n_slices + P.lse_run - 1) / P.lse_run;
    P.n_emit_runs = (P.n_slices + P.emit_run - 1) / P.emit_run;
    P.total_lse = R * (unsigned long long)P.n_lse_runs;
    {
        // the last kEdgeEndgameWaves waves of LSE tickets; in long launches with many positions per
        // sequence (the rows to emit are a small share of the bytes, and a stream of reads alone runs
        // faster than one with writes mixed in) all but the first eighth of the waves
        const unsigned long long waves = (P.total_lse + resident_ctas - 1) / resident_ctas;
        unsigned long long hold = (unsigned long long)kEdgeEndgameWaves;
        if (waves >= (unsigned long long)kEdgeEndgameLongWaves && P.gamma + 1 >= kEdgeEndgameLongRows)
            hold = waves * (unsigned long long)kEdgeEndgameLongEighths / 8;
        P.endgame_tickets = hold * resident_ctas;
        // (a launch that holds its EMIT tickets back almost throughout streams reads alone: there
        // the hint gains nothing and was measured to cost 2 %)
        P.first_read_hint = hold == (unsigned long long)kEdgeEndgameWaves ? 1 : 0;
    }
    P.total_emit = no_emit ? 0ull : (unsigned long long)P.B * (unsigned long long)P.n_emit_runs;
    // t / d == mulhi64(t, ceil(2^64 / d)) for every t with t * d * d < 2^64
    auto magic = [](unsigned long long total, int d) -> unsigned long long {
        if (d < 2 || d > (1 << 15) || total > (1ull << 33)) return 0ull;
        return ~0ull / (unsigned long long)d + 1ull;
    };
    P.lse_magic = magic(P.total_lse, P.n_lse_runs);
    P.emit_magic = magic(P.total_emit, P.n_emit_runs);
    P.spin_limit = 1u << 20;
    P.c1 = (float)(1.4426950408889634 / (double)P.temperature);
    edge_workspace_layout(P.B, P.gamma, P.n_lse_runs, &P, static_cast<char *>(workspace));
    const unsigned long long tickets = P.total_lse + P.total_emit;
    const unsigned grid = (unsigned)(tickets < resident_ctas ? tickets : resident_ctas);
    // a cooperative launch: all CTAs are resident at once (grid <= resident_ctas), which the kernel's
    // grid-wide barrier after the clearing of the workspace relies on
    void *args[] = {&P};
    const void *fn = dtype == DSSD_BF16 ? reinterpret_cast<const void *>(edge_verify_kernel<DSSD_BF16>)
                                        : reinterpret_cast<const void *>(edge_verify_kernel<DSSD_F32>);
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kEdgeThreads), args, kEdgeSmemBytes, stream);
}

}  // namespace dssd
