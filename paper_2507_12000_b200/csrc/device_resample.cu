// Device half of the verification round: residual (or bonus) inverse-CDF draw.
//
// Pass A, ticket (b, c): stream chunk c of p_row[b] and of Q_n[b], form r = max(0, p - q) (or
// r = p for the bonus draw) and add it up in float64 -> one or two chunk sums, 8-byte slots that are
// valid once they differ from the all-ones pattern that the kernel itself clears its scratch to
// (a cooperative launch; one grid-wide barrier, split around the first ticket's loads, separates
// the clearing from the first use).  A ticket costs one barrier and waits for no round trip.
// Pass B, ticket b, taken by a CTA once no chunk is left for it: a block-wide float64 prefix over
// the sequence's chunk sums gives Z and the chunk holding u' * Z; every thread fetches its run of
// that chunk (from L2 or HBM), a second prefix finds the thread, and the thread walks its run.
// The draws run after the streams because their dependent round trips are several times longer
// while the memory system is saturated.
// All sums are float64, so the token differs from an index-order float64 scan only when u' * Z
// lies within rounding (about 1e-13 relative) of a CDF step.
#include "device_resample.h"
#include "edge_verify.h"

#include <atomic>
#include <mutex>

#include <limits.h>
#include <math.h>

#include <utility>

#include <cooperative_groups.h>

#include "dssd_device.cuh"

namespace dssd {

namespace {

constexpr bool kWideTickets = true;  // whole tickets request all their loads at once (ticket_mass2)
constexpr int kResampleCtas = 4;      // resident CTAs per SM aimed at
constexpr int kSub = kResampleSub;         // entries per chunk sum: a ticket covers P.subs of them
constexpr int kRun = kSub / kThreads;      // contiguous entries per thread in pass B
static_assert(kRun == 16, "pass B fetches a run as one group of 16 entries");

__device__ __forceinline__ double res(float p, float q) { return fmax(0.0, (double)p - (double)q); }

__device__ __forceinline__ float4 as_f4(const uint4 &v)
{
    return make_float4(__uint_as_float(v.x), __uint_as_float(v.y), __uint_as_float(v.z), __uint_as_float(v.w));
}

// The row p comes as float32, as IEEE binary16 bit patterns (the 16-bit payload), or - for the
// fused verification of Algorithm 1, where no row is ever written - as the target logits of row n
// together with the row's reference exponent and 1 / sum, from which p_v = 2^(l_v c1 - ref2) / S is
// formed on the fly exactly as the edge kernel forms it when it emits a row.  The kernel is
// written once over these views.  A "quad" is four consecutive entries.
__device__ __forceinline__ float half_bits_to_float(unsigned short h) { return __half2float(__ushort_as_half(h)); }
__device__ __forceinline__ float4 half_quad(uint2 v)
{
    const float2 a = __half22float2(*reinterpret_cast<const __half2 *>(&v.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2 *>(&v.y));
    return make_float4(a.x, a.y, b.x, b.y);
}
__device__ __forceinline__ uint2 ld_stream8(const void *p)
{
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
}

struct RowF32 {  // p_row as float32
    typedef uint4 Raw;
    const float *p;
    __device__ static __forceinline__ RowF32 make(const ResampleParams &P, int64_t b, int)
    {
        RowF32 r;
        r.p = reinterpret_cast<const float *>(P.p_row) + (size_t)b * P.V;
        return r;
    }
    __device__ __forceinline__ bool aligned(int e) const { return (reinterpret_cast<uintptr_t>(p + e) & 15u) == 0; }
    __device__ __forceinline__ float ld(int64_t e) const { return __ldg(p + e); }
    __device__ __forceinline__ Raw ld_quad_stream(int e0, int64_t quad) const
    {
        return ld_stream16(reinterpret_cast<const uint4 *>(p + e0) + quad);
    }
    __device__ __forceinline__ float4 quad(const Raw &v) const { return as_f4(v); }
    __device__ __forceinline__ float4 ld_quad(int e0, int64_t quad) const
    {
        return __ldg(reinterpret_cast<const float4 *>(p + e0) + quad);
    }
};

struct RowF16 {  // p_row as binary16 bit patterns
    typedef uint2 Raw;
    const uint16_t *p;
    __device__ static __forceinline__ RowF16 make(const ResampleParams &P, int64_t b, int)
    {
        RowF16 r;
        r.p = reinterpret_cast<const uint16_t *>(P.p_row) + (size_t)b * P.V;
        return r;
    }
    __device__ __forceinline__ bool aligned(int e) const { return (reinterpret_cast<uintptr_t>(p + e) & 7u) == 0; }
    __device__ __forceinline__ float ld(int64_t e) const { return half_bits_to_float(__ldg(p + e)); }
    __device__ __forceinline__ Raw ld_quad_stream(int e0, int64_t quad) const
    {
        return ld_stream8(reinterpret_cast<const uint2 *>(p + e0) + quad);
    }
    __device__ __forceinline__ float4 quad(const Raw &v) const { return half_quad(v); }
    __device__ __forceinline__ float4 ld_quad(int e0, int64_t quad) const
    {
        return half_quad(__ldg(reinterpret_cast<const uint2 *>(p + e0) + quad));
    }
};

// four consecutive logits: how they are loaded and widened
template <int DT>
struct LogitQuad;
template <>
struct LogitQuad<DSSD_F32> {
    typedef uint4 Raw;
    __device__ static __forceinline__ Raw ld_stream(const void *p) { return ld_stream16(p); }
    __device__ static __forceinline__ float4 widen(const Raw &v) { return as_f4(v); }
};
template <>
struct LogitQuad<DSSD_BF16> {
    typedef uint2 Raw;
    __device__ static __forceinline__ Raw ld_stream(const void *p) { return ld_stream8(p); }
    __device__ static __forceinline__ float4 widen(const Raw &v)
    {
        return make_float4(bf16_lo(v.x), bf16_hi(v.x), bf16_lo(v.y), bf16_hi(v.y));
    }
};

template <int DT>
struct RowLogits {  // row n of the target logits, turned into probabilities on the fly
    typedef typename LogitQuad<DT>::Raw Raw;
    const char *row;
    float c1, nref, invS;
    __device__ static __forceinline__ RowLogits make(const ResampleParams &P, int64_t b, int n)
    {
        RowLogits r;
        r.row = reinterpret_cast<const char *>(P.logits) +
                ((size_t)b * (size_t)(P.gamma + 1) + (size_t)n) * (size_t)P.row_stride * Elem<DT>::kBytes;
        const ReadySlot s = reinterpret_cast<const ReadySlot *>(P.ready)[b];
        r.c1 = P.c1;
        r.nref = -s.ref2;
        r.invS = s.invS;
        return r;
    }
    __device__ __forceinline__ float prob(float l) const { return ex2(fmaf(l, c1, nref)) * invS; }
    __device__ __forceinline__ bool aligned(int e) const
    {
        return (reinterpret_cast<uintptr_t>(row + (size_t)e * Elem<DT>::kBytes) & (4u * Elem<DT>::kBytes - 1u)) == 0;
    }
    __device__ __forceinline__ float ld(int64_t e) const { return prob(Elem<DT>::load(row, e)); }
    __device__ __forceinline__ Raw ld_quad_stream(int e0, int64_t quad) const
    {
        return LogitQuad<DT>::ld_stream(row + ((size_t)e0 + 4 * (size_t)quad) * Elem<DT>::kBytes);
    }
    __device__ __forceinline__ float4 quad(const Raw &v) const
    {
        const float4 l = LogitQuad<DT>::widen(v);
        return make_float4(prob(l.x), prob(l.y), prob(l.z), prob(l.w));
    }
    __device__ __forceinline__ float4 ld_quad(int e0, int64_t quad) const { return this->quad(ld_quad_stream(e0, quad)); }
};

// per-thread part of sum_{e in [e0,e1)} r_e ; q == nullptr means r = p
template <typename RV>
__device__ __forceinline__ double chunk_mass(const RV &row, const float *q, int e0, int e1)
{
    const int tid = threadIdx.x;
    double acc = 0.0;
    int done = e0;
    const bool aligned = row.aligned(e0) && (!q || (reinterpret_cast<uintptr_t>(q + e0) & 15u) == 0);
    if (aligned) {
        const int nvec = (e1 - e0) / 4;
        if (q) {
            const uint4 *q4 = reinterpret_cast<const uint4 *>(q + e0);
            int i = tid;
            for (; i + 3 * kThreads < nvec; i += 4 * kThreads) {
                typename RV::Raw a[4];
                uint4 b[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    a[u] = row.ld_quad_stream(e0, i + u * kThreads);
                    b[u] = ld_stream16(q4 + i + u * kThreads);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float4 x = row.quad(a[u]), y = as_f4(b[u]);
                    acc += (res(x.x, y.x) + res(x.y, y.y)) + (res(x.z, y.z) + res(x.w, y.w));
                }
            }
            for (; i < nvec; i += kThreads) {
                const float4 x = row.quad(row.ld_quad_stream(e0, i)), y = as_f4(ld_stream16(q4 + i));
                acc += (res(x.x, y.x) + res(x.y, y.y)) + (res(x.z, y.z) + res(x.w, y.w));
            }
        } else {
            int i = tid;
            for (; i + 3 * kThreads < nvec; i += 4 * kThreads) {
                typename RV::Raw a[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) a[u] = row.ld_quad_stream(e0, i + u * kThreads);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float4 x = row.quad(a[u]);
                    acc += ((double)x.x + (double)x.y) + ((double)x.z + (double)x.w);
                }
            }
            for (; i < nvec; i += kThreads) {
                const float4 x = row.quad(row.ld_quad_stream(e0, i));
                acc += ((double)x.x + (double)x.y) + ((double)x.z + (double)x.w);
            }
        }
        done = e0 + nvec * 4;
    }
    for (int e = done + tid; e < e1; e += kThreads) acc += q ? res(row.ld(e), __ldg(q + e)) : (double)row.ld(e);
    return acc;
}

// A whole ticket of two full chunk sums whose rows are 16-byte aligned: all of a thread's loads
// (eight quads of p and of q) are requested before the first is used.  Quads u < 4 of a thread
// belong to the first chunk sum, the others to the second; the order of addition within each is
// the one chunk_mass uses, so both give the same bits.
template <typename RV>
__device__ __forceinline__ void ticket_mass2(const RV &row, const float *q, int e0, double &acc0, double &acc1)
{
    const int tid = threadIdx.x;
    typename RV::Raw a[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) a[u] = row.ld_quad_stream(e0, tid + u * kThreads);
    if (q) {
        const uint4 *q4 = reinterpret_cast<const uint4 *>(q + e0);
        uint4 b[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) b[u] = ld_stream16(q4 + tid + u * kThreads);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float4 x = row.quad(a[u]), y = as_f4(b[u]);
            const double t = (res(x.x, y.x) + res(x.y, y.y)) + (res(x.z, y.z) + res(x.w, y.w));
            if (u < 4) acc0 += t;
            else acc1 += t;
        }
    } else {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const float4 x = row.quad(a[u]);
            const double t = ((double)x.x + (double)x.y) + ((double)x.z + (double)x.w);
            if (u < 4) acc0 += t;
            else acc1 += t;
        }
    }
}

// CTA-wide sum in a fixed order; result valid in thread 0
__device__ __forceinline__ double block_sum(double x, double *s_w)
{
    x = warp_sum(x);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) s_w[threadIdx.x >> 5] = x;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0) {
#pragma unroll
        for (int w = 0; w < kWarps; ++w) t += s_w[w];
    }
    return t;
}

struct Pick {  // what thread 0 hands to the CTA for pass B
    int ok;        // Z > 0 and finite
    int chunk;     // chunk holding the target
    int beyond;    // no chunk prefix exceeds the target: take the last positive entry
    double base;   // mass before that chunk
    double target; // u' * Z
};

constexpr unsigned long long kFill64 = ~0ull;

// is a sequence with accepted length n (0 <= n <= gamma) one this launch draws for?
__device__ __forceinline__ bool selected(const ResampleParams &P, int n)
{
    return P.select == 0 || (P.select == 1 ? n == P.gamma : n < P.gamma);
}

__device__ __forceinline__ unsigned long long logical(unsigned long long raw) { return raw + 1ull; }

// chunk sum (b, c); a sum whose store has not landed yet still shows the fill pattern and is
// polled for (bounded); when the wait runs out the fill pattern itself comes back (see timed_out)
__device__ __forceinline__ double load_chunk_sum(const ResampleParams &P, const unsigned long long *cs, int c, unsigned polls)
{
    unsigned long long w = ld_relaxed_u64(cs + c);
    for (unsigned it = 0; w == kFill64 && it < polls; ++it) {
        __nanosleep(32);
        w = ld_relaxed_u64(cs + c);
    }
    return __longlong_as_double((long long)w);
}

__device__ __forceinline__ bool timed_out(double m) { return (unsigned long long)__double_as_longlong(m) == kFill64; }

// every thread's verdict on its chunk sums; on a timeout the sequence gets no token
__device__ __forceinline__ bool give_up(const ResampleParams &P, int64_t b, bool mine, unsigned fl)
{
    if (!__syncthreads_or(mine)) return false;
    if (threadIdx.x == 0) {
        P.token[b] = -1;
        if (P.flags) P.flags[b] = fl | DSSD_RS_FLAG_INVALID | DSSD_RS_FLAG_TIMEOUT;
    }
    return true;
}

// CTA-wide inclusive prefix sum in index order of the threads; `total` is the sum over the CTA
__device__ __forceinline__ double block_scan(double x, double *s_scan, double &total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    __syncthreads();
    if (lane == 31) s_scan[warp] = incl;
    __syncthreads();
    double before = 0.0, all = 0.0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        const double v = s_scan[w];
        if (w < warp) before += v;
        all += v;
    }
    total = all;
    return before + incl;
}

// The draw inside the chunk that `pk` names: every thread fetches its run of the chunk, a prefix over
// the CTA finds the thread whose run holds the target, and that thread walks its run.  The token
// (its index in the row plus tok_base, or -1 when the chunk has no positive entry) and the flags
// go to *token_out / *flags_out.  q == nullptr means r = p.
template <typename RV>
__device__ __forceinline__ void walk_chunk(const Pick &pk, int V, const RV &row, const float *q, unsigned fl, int tok_base,
                                           int32_t *token_out, uint32_t *flags_out, double *s_w, int *s_i)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int e0 = pk.chunk * kSub, e1 = min(V, e0 + kSub);
    const int r0 = min(e1, e0 + tid * kRun), r1 = min(e1, r0 + kRun);
    double mine = 0.0;
    int last_pos = -1;
    // The run's 16 entries are all requested before the first is used (one round trip for the
    // run, not one per entry); entries past the row's end read as 0.
    const bool vec = (r1 - r0 == kRun) && row.aligned(r0) && (!q || (reinterpret_cast<uintptr_t>(q + r0) & 15u) == 0);
#pragma unroll
    for (int g = 0; g < kRun; g += 16) {
        float pv[16], qv[16];
        if (vec) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float4 a = row.ld_quad(r0 + g, j);
                pv[4 * j] = a.x, pv[4 * j + 1] = a.y, pv[4 * j + 2] = a.z, pv[4 * j + 3] = a.w;
                float4 c = make_float4(0.f, 0.f, 0.f, 0.f);
                if (q) c = __ldg(reinterpret_cast<const float4 *>(q + r0 + g) + j);
                qv[4 * j] = c.x, qv[4 * j + 1] = c.y, qv[4 * j + 2] = c.z, qv[4 * j + 3] = c.w;
            }
        } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
                const int e = r0 + g + j;
                pv[j] = e < r1 ? row.ld(e) : 0.f;
                qv[j] = (q && e < r1) ? __ldg(q + e) : 0.f;
            }
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
            const double r = q ? res(pv[j], qv[j]) : (double)pv[j];
            mine += r;
            if (r > 0.0) last_pos = r0 + g + j;
        }
    }
    // exclusive prefix of the per-thread run sums across the CTA
    double incl = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
    __syncthreads();
    if (lane == 31) s_w[warp] = incl;
    __syncthreads();
    double before = pk.base;
    for (int w = 0; w < warp; ++w) before += s_w[w];
    before += incl - mine;
    const bool crosses = !pk.beyond && (before + mine > pk.target);
    const unsigned bal = __ballot_sync(0xffffffffu, crosses);
    if (tid == 0) { s_i[0] = 0x7fffffff; s_i[1] = -1; }
    __syncthreads();
    if (lane == 0 && bal) atomicMin(&s_i[0], warp * 32 + __ffs(bal) - 1);
    if (last_pos >= 0) atomicMax(&s_i[1], last_pos);
    __syncthreads();
    const int first = s_i[0];
    if (first == 0x7fffffff) {
        if (tid == 0) {
            *token_out = s_i[1] < 0 ? -1 : tok_base + s_i[1];
            if (flags_out) *flags_out = fl | (s_i[1] < 0 ? DSSD_RS_FLAG_INVALID : 0u);
        }
    } else if (tid == first) {
        double C = before;
        int tok = last_pos;
        for (int e = r0; e < r1; ++e) {
            C += q ? res(row.ld(e), __ldg(q + e)) : (double)row.ld(e);
            if (C > pk.target) { tok = e; break; }
        }
        tok = tok >= 0 ? tok : s_i[1];
        *token_out = tok < 0 ? -1 : tok_base + tok;
        if (flags_out) *flags_out = fl;
    }
}

// pass B for sequence b; q == nullptr means r = p
template <typename RV>
__device__ void draw(const ResampleParams &P, int64_t b, const RV &row, const float *q, unsigned fl, float u,
                     double *s_w, Pick *s_pick, int *s_i)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    unsigned long long *cs = reinterpret_cast<unsigned long long *>(P.chunk_sum) + (size_t)b * P.n_sub;
    const unsigned polls = b + 1 == (int64_t)P.test_drop_seq_plus1 ? P.test_poll_limit : P.spin_limit;
    for (int attempt = 0; attempt < 2; ++attempt) {
        bool ok;
        if (P.n_sub <= kThreads) {
            // one chunk per thread: a single scan gives Z and every inclusive prefix
            const double m = tid < P.n_sub ? load_chunk_sum(P, cs, tid, polls) : 0.0;
            if (give_up(P, b, timed_out(m), fl)) return;
            double Z;
            const double incl = block_scan(m, s_w, Z);
            ok = (Z > 0.0) && (Z < INFINITY);
            if (ok) {
                const double target = (double)u * Z;
                if (tid == 0) {
                    s_i[0] = 0x7fffffff;
                    s_i[1] = -1;
                }
                __syncthreads();
                const bool crosses = tid < P.n_sub && incl > target;
                const unsigned bal = __ballot_sync(0xffffffffu, crosses);
                if (lane == 0 && bal) atomicMin(&s_i[0], warp * 32 + __ffs(bal) - 1);
                const unsigned pos = __ballot_sync(0xffffffffu, tid < P.n_sub && m > 0.0);
                if (lane == 0 && pos) atomicMax(&s_i[1], warp * 32 + 31 - __clz(pos));
                __syncthreads();
                const int first = s_i[0], last = s_i[1];
                if (tid == (first != 0x7fffffff ? first : last)) {
                    Pick pk;
                    pk.ok = 1;
                    pk.beyond = first == 0x7fffffff;
                    pk.chunk = tid;
                    pk.base = incl - m;
                    pk.target = target;
                    *s_pick = pk;
                }
                __syncthreads();
                break;
            }
        } else {
        // Z = sum of the chunk sums, in groups of one chunk per thread
        double Z = 0.0;
        bool late = false;
        for (int base = 0; base < P.n_sub; base += kThreads) {
            const int c = base + tid;
            const double m = c < P.n_sub ? load_chunk_sum(P, cs, c, polls) : 0.0;
            late |= timed_out(m);
            double tot;
            block_scan(m, s_w, tot);
            Z += tot;
            __syncthreads();
        }
        if (give_up(P, b, late, fl)) return;
        ok = (Z > 0.0) && (Z < INFINITY);
        if (ok) {
            // the first chunk whose inclusive prefix exceeds the target, else the last chunk with mass
            const double target = (double)u * Z;
            if (tid == 0) {
                s_i[0] = 0x7fffffff;
                s_i[1] = -1;
            }
            __syncthreads();
            double carry = 0.0;
            double my_base_first = 0.0, my_base_last = 0.0;
            int my_first = 0x7fffffff, my_last = -1;
            for (int base = 0; base < P.n_sub; base += kThreads) {
                const int c = base + tid;
                const double m = c < P.n_sub ? load_chunk_sum(P, cs, c, polls) : 0.0;
                double tot;
                const double incl = carry + block_scan(m, s_w, tot);
                if (c < P.n_sub && incl > target && my_first == 0x7fffffff) {
                    my_first = c;
                    my_base_first = incl - m;
                }
                if (c < P.n_sub && m > 0.0) {
                    my_last = c;
                    my_base_last = incl - m;
                }
                carry += tot;
                __syncthreads();
            }
            if (my_first != 0x7fffffff) atomicMin(&s_i[0], my_first);
            if (my_last >= 0) atomicMax(&s_i[1], my_last);
            __syncthreads();
            const int first = s_i[0], last = s_i[1];
            if (first != 0x7fffffff ? (my_first == first) : (my_last == last && last >= 0)) {
                Pick pk;
                pk.ok = 1;
                pk.beyond = first == 0x7fffffff;
                pk.chunk = pk.beyond ? last : first;
                pk.base = pk.beyond ? my_base_last : my_base_first;
                pk.target = target;
                *s_pick = pk;
            }
            __syncthreads();
            break;
        }
        }
        if (q == nullptr) {  // already drawing from p: the row has no usable mass
            if (tid == 0) {
                P.token[b] = -1;
                if (P.flags) P.flags[b] = fl | DSSD_RS_FLAG_INVALID;
            }
            return;
        }
        // residual has no mass (p == q): draw from p instead
        q = nullptr;
        fl |= DSSD_RS_FLAG_FALLBACK;
        for (int c = 0; c < P.n_sub; ++c) {
            const int e0 = c * kSub, e1 = min(P.V, e0 + kSub);
            const double tot = block_sum(chunk_mass(row, nullptr, e0, e1), s_w);
            if (tid == 0) st_relaxed_u64(cs + c, (unsigned long long)__double_as_longlong(tot));
        }
        __syncthreads();
    }
    const Pick pk = *s_pick;
    walk_chunk<RV>(pk, P.V, row, q, fl, 0, P.token + b, P.flags ? P.flags + b : nullptr, s_w, s_i);
}

template <typename RV>
__global__ void __launch_bounds__(kThreads, kResampleCtas) resample_kernel(const __grid_constant__ ResampleParams P)
{
    __shared__ double s_w[2][kWarps][2];
    __shared__ double s_scan[kWarps];
    __shared__ Pick s_pick;
    __shared__ int s_i[2];
    __shared__ unsigned long long s_ticket[2];
    __shared__ float s_first_u;
    __shared__ int s_first_n;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // ---- the scratch is cleared here, by the kernel itself: every chunk sum to the all-ones pattern,
    // the ticket counter to twice the number of CTAs (every CTA's first two tickets are its own
    // number and that plus the number of CTAs), the draw counter to the number of CTAs when every
    // sequence has a CTA of its own.  One grid-wide barrier (a cooperative launch: all CTAs are
    // resident) separates the clearing from the first use; it is split around the first ticket's
    // loads, which need nothing of the scratch. ----
    namespace cg = cooperative_groups;
    cg::grid_group grid = cg::this_grid();
    const bool early = (unsigned long long)P.B <= (unsigned long long)gridDim.x;
    {
        uint4 *w = reinterpret_cast<uint4 *>(P.ticket);  // the scratch starts with the counters
        const size_t nw = P.fill_bytes / 16;
        for (size_t i = (size_t)blockIdx.x * kThreads + tid; i < nw; i += (size_t)gridDim.x * kThreads) {
            uint4 v = make_uint4(~0u, ~0u, ~0u, ~0u);
            if (i == 0) {  // raw value of a 64-bit counter: logical value - 1
                const unsigned long long raw = 2ull * gridDim.x - 1ull;
                v.x = (unsigned)raw;
                v.y = (unsigned)(raw >> 32);
            }
            if (i == 8 && early) {  // the draw counter, 128 bytes on
                v.x = gridDim.x - 1u;
                v.y = 0u;
            }
            w[i] = v;
        }
    }
    auto arrived = grid.barrier_arrive();
    bool waited = false;

    // ---- pass A: chunk sums.  One barrier per ticket, no round trip waited for. ----
    unsigned long long next_raw = 0;  // thread 0: the ticket after the next one, drawn early
    // when there is at most one draw per CTA, a CTA's draw is the sequence of its own number, so
    // that neither a ticket nor the sequence's accepted length and uniform are waited for when the
    // draws begin (with more draws than CTAs the first ticket is taken when the draws begin, by
    // whoever gets there first)
    const unsigned long long my_draw = blockIdx.x;
    int first_n = INT_MIN;  // not loaded
    float first_u = 0.f;
    unsigned long long t = blockIdx.x;
    for (int it = 0; t < P.total_tickets; ++it) {
        const int buf = it & 1;
        // tickets run from the last sequence's last chunk backwards: when the rows were written by a
        // kernel just before this one, the end of the array is the part most likely still in L2
        const unsigned long long tr = P.total_tickets - 1ull - t;
        const int64_t b = (int64_t)(tr / (unsigned)P.n_chunks);
        const int c = (int)(tr - (unsigned long long)b * (unsigned)P.n_chunks);
        const int n = __ldg(P.accept_len + b);
        double acc0 = 0.0, acc1 = 0.0;  // the ticket's chunk sums
        if (n >= 0 && n <= P.gamma && selected(P, n)) {
            const RV row = RV::make(P, b, n);
            const float *q = n < P.gamma ? P.draft_q + ((size_t)b * P.gamma + n) * (size_t)P.V : nullptr;
            const int e0 = c * P.subs * kSub, e1 = min(P.V, e0 + kSub), e2 = min(P.V, e0 + P.subs * kSub);
            static_assert(kSub == 4 * 4 * kThreads, "a thread's four quads per chunk sum");
            if (kWideTickets && e2 - e0 == 2 * kSub && row.aligned(e0) && (!q || (reinterpret_cast<uintptr_t>(q + e0) & 15u) == 0)) {
                ticket_mass2(row, q, e0, acc0, acc1);
            } else {
                acc0 = chunk_mass(row, q, e0, e1);
                if (e2 > e1) acc1 = chunk_mass(row, q, e1, e2);
            }
        }
        acc0 = warp_sum(acc0);
        acc1 = warp_sum(acc1);
        if (lane == 0) {
            s_w[buf][warp][0] = acc0;
            s_w[buf][warp][1] = acc1;
        }
        if (it == 0) {  // the first ticket's loads are done: from here on the scratch is used
            grid.barrier_wait(std::move(arrived));
            waited = true;
        }
        if (tid == 0) {
            s_ticket[buf] = it == 0 ? t + gridDim.x : logical(next_raw);
            next_raw = atomicAdd(P.ticket, 1ull);
            if (it == 0 && early && my_draw < (unsigned long long)P.B) {
                first_n = __ldg(P.accept_len + ((unsigned long long)P.B - 1ull - my_draw));
                first_u = __ldg(P.uniforms + ((unsigned long long)P.B - 1ull - my_draw));
            }
        }
        __syncthreads();
        if (tid == 0) {
            double tot0 = 0.0, tot1 = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                tot0 += s_w[buf][w][0];
                tot1 += s_w[buf][w][1];
            }
            unsigned long long *cs = reinterpret_cast<unsigned long long *>(P.chunk_sum) + (size_t)b * P.n_sub + P.subs * c;
            if (b + 1 != (int64_t)P.test_drop_seq_plus1) {  // (the test hook withholds these stores)
                st_relaxed_u64(cs, (unsigned long long)__double_as_longlong(tot0));
                if (P.subs == 2 && 2 * c + 1 < P.n_sub) st_relaxed_u64(cs + 1, (unsigned long long)__double_as_longlong(tot1));
            }
        }
        t = s_ticket[buf];
    }

    // ---- pass B: the draws, one sequence per ticket, once this CTA has no chunk left.  By then
    // the memory system is no longer saturated by the streams, so a draw's two round trips are
    // short; a chunk sum that has not landed yet is polled for (its CTA is still running). ----
    if (!waited) grid.barrier_wait(std::move(arrived));
    __syncthreads();
    if (tid == 0) {
        s_ticket[0] = early ? my_draw : logical(atomicAdd(P.draw_ticket, 1ull));
        s_first_n = first_n;
        s_first_u = first_u;
        next_raw = atomicAdd(P.draw_ticket, 1ull);
    }
    __syncthreads();
    unsigned long long d = s_ticket[0];
    const bool prefetched = s_first_n != INT_MIN;
    for (int it = 1; d < (unsigned long long)P.B; ++it) {
        const int buf = it & 1;
        if (tid == 0) {
            s_ticket[buf] = logical(next_raw);
            next_raw = atomicAdd(P.draw_ticket, 1ull);
        }
        const int64_t b = (int64_t)P.B - 1 - (int64_t)d;  // in the order in which pass A completes the sequences
        const int n = (it == 1 && prefetched) ? s_first_n : __ldg(P.accept_len + b);
        const float u = (it == 1 && prefetched) ? s_first_u : __ldg(P.uniforms + b);
        if (n < 0 || n > P.gamma) {
            if (tid == 0) {
                P.token[b] = -1;
                if (P.flags) P.flags[b] = DSSD_RS_FLAG_INVALID;
            }
        } else if (!selected(P, n)) {
            if (P.select == 1 && tid == 0) {  // a rejected sequence: its token comes from the device half
                P.token[b] = -1;
                if (P.flags) P.flags[b] = 0u;
            }
        } else {
            const RV row = RV::make(P, b, n);
            const float *q = n < P.gamma ? P.draft_q + ((size_t)b * P.gamma + n) * (size_t)P.V : nullptr;
            draw<RV>(P, b, row, q, q ? 0u : DSSD_RS_FLAG_BONUS, u, s_scan, &s_pick, s_i);
        }
        __syncthreads();
        d = s_ticket[buf];
    }
}

// ---- one shard of the vocabulary ---------------------------------------------------------------
//
// The draw over a row that is spread over G shards takes two steps with one small exchange
// between them.  shard_mass_kernel streams this shard's slice of p_row and of Q_n once and leaves,
// per chunk of kSub entries, the residual mass sum max(0, p - q) (sum p for a bonus draw) and the
// plain mass sum p (needed if the residual turns out to have no mass anywhere);
// shard_total_kernel adds a sequence's chunks up.  After the masses of all shards have been
// gathered, shard_draw_kernel - one CTA per sequence - takes the same decisions on every shard
// (Z, fall-back, the shard that holds u' Z) and the owning shard walks its slice exactly as the
// dense kernel walks a row.  Plain stores and stream order connect the launches: no slot is read
// before the launch that wrote it has ended, so the scratch needs no fill.

template <typename RV>
__device__ __forceinline__ void chunk_mass2(const RV &row, const float *q, int e0, int e1, double &acc_r, double &acc_p)
{
    const int tid = threadIdx.x;
    int done = e0;
    const bool aligned = row.aligned(e0) && (!q || (reinterpret_cast<uintptr_t>(q + e0) & 15u) == 0);
    if (aligned) {
        const int nvec = (e1 - e0) / 4;
        const uint4 *q4 = reinterpret_cast<const uint4 *>(q + e0);
        for (int i = tid; i < nvec; i += 4 * kThreads) {
            typename RV::Raw a[4];
            uint4 c[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const bool in = i + u * kThreads < nvec;
                a[u] = in ? row.ld_quad_stream(e0, i + u * kThreads) : typename RV::Raw();
                c[u] = (in && q) ? ld_stream16(q4 + i + u * kThreads) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (i + u * kThreads >= nvec) continue;
                const float4 x = row.quad(a[u]), y = as_f4(c[u]);
                acc_p += ((double)x.x + (double)x.y) + ((double)x.z + (double)x.w);
                if (q) acc_r += (res(x.x, y.x) + res(x.y, y.y)) + (res(x.z, y.z) + res(x.w, y.w));
            }
        }
        done = e0 + nvec * 4;
    }
    for (int e = done + tid; e < e1; e += kThreads) {
        const float pv = row.ld(e);
        acc_p += (double)pv;
        if (q) acc_r += res(pv, __ldg(q + e));
    }
    if (!q) acc_r = acc_p;
}

__device__ __forceinline__ RowF32 shard_row(const ShardResampleParams &P, int64_t b)
{
    RowF32 r;
    r.p = P.p_row + (size_t)b * (size_t)P.p_stride;
    return r;
}

__global__ void __launch_bounds__(kThreads, kResampleCtas) shard_mass_kernel(const __grid_constant__ ShardResampleParams P)
{
    __shared__ double s_w[kWarps][2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long total = (long long)P.B * P.n_sub;
    for (long long t = blockIdx.x; t < total; t += gridDim.x) {
        const int64_t b = t / P.n_sub;
        const int c = (int)(t - b * P.n_sub);
        const int n = __ldg(P.accept_len + b);
        double acc_r = 0.0, acc_p = 0.0;
        const bool valid = n >= 0 && n <= P.gamma;
        if (valid) {
            const RowF32 row = shard_row(P, b);
            const float *q = n < P.gamma ? P.draft_q + ((size_t)b * P.gamma + n) * (size_t)P.q_stride : nullptr;
            const int e0 = c * kSub, e1 = min(P.V, e0 + kSub);
            chunk_mass2(row, q, e0, e1, acc_r, acc_p);
        }
        acc_r = warp_sum(acc_r);
        acc_p = warp_sum(acc_p);
        __syncthreads();  // the previous ticket's sums have been read
        if (lane == 0) {
            s_w[warp][0] = acc_r;
            s_w[warp][1] = acc_p;
        }
        __syncthreads();
        if (tid == 0) {
            double tr = 0.0, tp = 0.0;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) {
                tr += s_w[w][0];
                tp += s_w[w][1];
            }
            const double nan = __longlong_as_double(0x7ff8000000000000ll);
            double *cs = P.chunk_sum + ((size_t)b * P.n_sub + c) * 2;
            cs[0] = valid ? tr : nan;
            cs[1] = valid ? tp : nan;
        }
    }
}

// one warp per sequence: the chunk sums in a fixed order
__global__ void __launch_bounds__(kThreads) shard_total_kernel(const __grid_constant__ ShardResampleParams P)
{
    const int lane = threadIdx.x & 31;
    const long long b = (long long)blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (b >= P.B) return;
    const double *cs = P.chunk_sum + (size_t)b * P.n_sub * 2;
    double r = 0.0, p = 0.0;
    for (int c = lane; c < P.n_sub; c += 32) {
        r += cs[2 * c];
        p += cs[2 * c + 1];
    }
    r = warp_sum(r);
    p = warp_sum(p);
    if (lane == 0) {
        P.mass[2 * b] = r;
        P.mass[2 * b + 1] = p;
    }
}

__global__ void __launch_bounds__(kThreads) shard_draw_kernel(const __grid_constant__ ShardResampleParams P)
{
    __shared__ double s_scan[kWarps];
    __shared__ Pick s_pick;
    __shared__ int s_i[2];
    const int tid = threadIdx.x;
    const int64_t b = blockIdx.x;
    const int n = __ldg(P.accept_len + b);
    int32_t *token_out = P.token + b;
    uint32_t *flags_out = P.flags ? P.flags + b : nullptr;
    if (n < 0 || n > P.gamma) {
        if (tid == 0) {
            *token_out = -1;
            if (flags_out) *flags_out = DSSD_RS_FLAG_INVALID;
        }
        return;
    }
    // The verdict on the sequence, from all shards' masses: every thread of every shard takes the
    // same steps in the same order.
    unsigned fl = n == P.gamma ? DSSD_RS_FLAG_BONUS : 0u;
    int col = 0;
    double Z = 0.0;
    for (int h = 0; h < P.G; ++h) Z += __ldg(P.masses + ((size_t)h * P.B + b) * 2);
    bool ok = (Z > 0.0) && (Z < INFINITY);
    if (!ok && n < P.gamma) {  // no residual mass anywhere: draw from p instead
        fl |= DSSD_RS_FLAG_FALLBACK;
        col = 1;
        Z = 0.0;
        for (int h = 0; h < P.G; ++h) Z += __ldg(P.masses + ((size_t)h * P.B + b) * 2 + 1);
        ok = (Z > 0.0) && (Z < INFINITY);
    }
    if (!ok) {
        if (tid == 0) {
            *token_out = -1;
            if (flags_out) *flags_out = fl | DSSD_RS_FLAG_INVALID;
        }
        return;
    }
    const double t = (double)__ldg(P.uniforms + b) * Z;
    double C = 0.0, before = 0.0;
    int owner = -1, last_mass = -1;
    for (int h = 0; h < P.G; ++h) {
        const double m = __ldg(P.masses + ((size_t)h * P.B + b) * 2 + col);
        if (m > 0.0) last_mass = h;
        if (owner < 0 && C + m > t) {
            owner = h;
            before = C;
        }
        C += m;
    }
    const bool beyond = owner < 0;  // rounding left no shard above t: the last shard with mass, its last positive entry
    if (beyond) owner = last_mass;
    if (owner != P.g) {
        if (tid == 0) {
            *token_out = -1;
            if (flags_out) *flags_out = fl;
        }
        return;
    }
    // this shard holds the target: the chunk first, then the walk inside it
    const double target = t - before;
    const double *cs = P.chunk_sum + (size_t)b * P.n_sub * 2 + col;
    if (tid == 0) {
        s_i[0] = 0x7fffffff;
        s_i[1] = -1;
    }
    __syncthreads();
    double carry = 0.0, my_base_first = 0.0, my_base_last = 0.0;
    int my_first = 0x7fffffff, my_last = -1;
    for (int base = 0; base < P.n_sub; base += kThreads) {
        const int c = base + tid;
        const double m = c < P.n_sub ? cs[2 * c] : 0.0;
        double tot;
        const double incl = carry + block_scan(m, s_scan, tot);
        if (!beyond && c < P.n_sub && incl > target && my_first == 0x7fffffff) {
            my_first = c;
            my_base_first = incl - m;
        }
        if (c < P.n_sub && m > 0.0) {
            my_last = c;
            my_base_last = incl - m;
        }
        carry += tot;
        __syncthreads();
    }
    if (my_first != 0x7fffffff) atomicMin(&s_i[0], my_first);
    if (my_last >= 0) atomicMax(&s_i[1], my_last);
    __syncthreads();
    const int first = s_i[0], last = s_i[1];
    if (first == 0x7fffffff && last < 0) {  // cannot happen while this shard's mass is positive
        if (tid == 0) {
            *token_out = -1;
            if (flags_out) *flags_out = fl | DSSD_RS_FLAG_INVALID;
        }
        return;
    }
    if (first != 0x7fffffff ? (my_first == first) : (my_last == last)) {
        Pick pk;
        pk.ok = 1;
        pk.beyond = first == 0x7fffffff;
        pk.chunk = pk.beyond ? last : first;
        pk.base = pk.beyond ? my_base_last : my_base_first;
        pk.target = target;
        s_pick = pk;
    }
    __syncthreads();
    const Pick pk = s_pick;
    const RowF32 row = shard_row(P, b);
    const float *q = (col == 0 && n < P.gamma) ? P.draft_q + ((size_t)b * P.gamma + n) * (size_t)P.q_stride : nullptr;
    walk_chunk<RowF32>(pk, P.V, row, q, fl, P.v_begin, token_out, flags_out, s_scan, s_i);
}


}  // namespace

size_t resample_workspace_layout(int B, int V, ResampleParams *P, char *base)
{
    // the kernel sets all of it to 0xFF before use: counters then read "logical 0" (raw + 1) and
    // the chunk sums read "not yet"
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += (bytes + 255) & ~(size_t)255;
        return o;
    };
    const size_t o_ticket = take(256);  // the two ticket counters, on separate 128-byte lines
    const int n_sub = (V + kResampleSub - 1) / kResampleSub;
    const size_t o_sum = take((size_t)B * (size_t)n_sub * sizeof(double));
    if (P) {
        P->ticket = reinterpret_cast<unsigned long long *>(base + o_ticket);
        P->draw_ticket = reinterpret_cast<unsigned long long *>(base + o_ticket + 128);
        P->chunk_sum = reinterpret_cast<double *>(base + o_sum);
        P->fill_bytes = off;
        if (P->subs != 1) P->subs = 2;
        P->n_chunks = (n_sub + P->subs - 1) / P->subs;
        P->n_sub = n_sub;
        P->total_tickets = (unsigned long long)B * (unsigned long long)P->n_chunks;
    }
    return off;
}

// resident CTAs per device, looked up on the first launch made with that device current (the
// occupancy depends on the compiled kernels only); 0: not looked up yet
static std::atomic<int> g_resample_resident[64];  // published last (release), read first (acquire)
static std::atomic<int> g_resample_sms[64];

cudaError_t resample_launch(ResampleParams &P, void *workspace, cudaStream_t stream)
{
    cudaError_t err;
    int dev = 0, sms = 0, occ = 0;
    if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    occ = g_resample_resident[dev].load(std::memory_order_acquire);
    if (occ == 0) {
        if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
        int o[4] = {0, 0, 0, 0};
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o[0], resample_kernel<RowF32>, kThreads, 0)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o[1], resample_kernel<RowF16>, kThreads, 0)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o[2], resample_kernel<RowLogits<DSSD_F32>>, kThreads, 0)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&o[3], resample_kernel<RowLogits<DSSD_BF16>>, kThreads, 0)) != cudaSuccess) return err;
        occ = o[0];
        for (int i = 1; i < 4; ++i) occ = o[i] < occ ? o[i] : occ;
        if (occ < 1) occ = 1;
        g_resample_sms[dev].store(sms, std::memory_order_relaxed);
        g_resample_resident[dev].store(occ, std::memory_order_release);  // a concurrent first call finds either 0 or the final pair
    }
    sms = g_resample_sms[dev].load(std::memory_order_relaxed);
    // two chunk sums per ticket halve the barriers; one per ticket evens out the CTAs' shares when
    // there are only a few tickets for each
    {
        const unsigned long long pairs = (unsigned long long)P.B * (unsigned long long)(((P.V + kResampleSub - 1) / kResampleSub + 1) / 2);
        P.subs = pairs < 4ull * (unsigned long long)sms * (unsigned long long)occ ? 1 : 2;
    }
    resample_workspace_layout(P.B, P.V, &P, static_cast<char *>(workspace));
    P.spin_limit = 1u << 20;
    const unsigned long long resident = (unsigned long long)sms * (unsigned long long)occ;
    const unsigned grid = (unsigned)(P.total_tickets < resident ? P.total_tickets : resident);
    // a cooperative launch: all CTAs are resident at once (grid <= resident), which the kernel's
    // grid-wide barrier after the clearing of the scratch relies on
    const void *fn;
    if (P.logits) {
        fn = P.logits_dtype == DSSD_BF16 ? reinterpret_cast<const void *>(resample_kernel<RowLogits<DSSD_BF16>>)
                                         : reinterpret_cast<const void *>(resample_kernel<RowLogits<DSSD_F32>>);
    } else if (P.p_half) {
        fn = reinterpret_cast<const void *>(resample_kernel<RowF16>);
    } else {
        fn = reinterpret_cast<const void *>(resample_kernel<RowF32>);
    }
    void *args[] = {&P};
    return cudaLaunchCooperativeKernel(fn, dim3(grid), dim3(kThreads), args, 0, stream);
}

size_t shard_resample_workspace_bytes(int B, int V)
{
    const size_t n_sub = (size_t)((V + kResampleSub - 1) / kResampleSub);
    return (((size_t)B * n_sub * 2 * sizeof(double)) + 255) & ~(size_t)255;
}

cudaError_t shard_mass_launch(ShardResampleParams &P, void *workspace, cudaStream_t stream)
{
    cudaError_t err;
    int dev = 0, sms = 0;
    if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
    if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
    P.n_sub = (P.V + kResampleSub - 1) / kResampleSub;
    P.chunk_sum = static_cast<double *>(workspace);
    const long long total = (long long)P.B * P.n_sub;
    const long long resident = (long long)(sms < 1 ? 1 : sms) * kResampleCtas;
    shard_mass_kernel<<<(unsigned)(total < resident ? total : resident), kThreads, 0, stream>>>(P);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
    shard_total_kernel<<<(unsigned)((P.B + kWarps - 1) / kWarps), kThreads, 0, stream>>>(P);
    return cudaGetLastError();
}

cudaError_t shard_draw_launch(ShardResampleParams &P, const void *workspace, cudaStream_t stream)
{
    P.n_sub = (P.V + kResampleSub - 1) / kResampleSub;
    P.chunk_sum = const_cast<double *>(static_cast<const double *>(workspace));
    shard_draw_kernel<<<(unsigned)P.B, kThreads, 0, stream>>>(P);
    return cudaGetLastError();
}

}  // namespace dssd

// ---- dssd_device_resample_static: the same draw, with its scratch inside the library ----------
//
// The scratch of this entry point is a fixed array in the library's device image.  Host code
// cannot use the array's name as an address: the address is looked up once per device with
// cudaGetSymbolAddress, with that device current, and handed to the kernel like any workspace.

static __device__ __align__(256) unsigned char g_static_scratch[DSSD_STATIC_SCRATCH_BYTES];

namespace {
std::mutex g_static_mutex;
void *g_static_ptr[64];  // per device, filled on the first call made with that device current
}  // namespace

extern "C" dssd_status dssd_device_resample_static(const float *p_row, const float *draft_q,
                                                   const int32_t *accept_len, const float *uniforms, int B,
                                                   int gamma, int V, int32_t *token, uint32_t *flags,
                                                   void *cuda_stream)
{
    dssd::set_last_cuda_error(0);
    if (B < 1 || gamma < 0 || V < 1) return DSSD_ERR_INVALID_ARG;
    if (V > DSSD_MAX_V || (long long)B * ((long long)gamma + 1) > (long long)DSSD_MAX_ROWS) return DSSD_ERR_UNSUPPORTED;
    if (!p_row || !accept_len || !uniforms || !token) return DSSD_ERR_INVALID_ARG;
    if (gamma > 0 && !draft_q) return DSSD_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(p_row) % 4) || (reinterpret_cast<uintptr_t>(draft_q) % 4)) return DSSD_ERR_INVALID_ARG;
    // the built-in scratch has a fixed size: larger batches must use dssd_device_resample
    if (dssd::resample_workspace_layout(B, V, nullptr, nullptr) > (size_t)DSSD_STATIC_SCRATCH_BYTES) return DSSD_ERR_UNSUPPORTED;

    cudaError_t e;
    int dev = 0;
    if ((e = cudaGetDevice(&dev)) != cudaSuccess) {
        dssd::set_last_cuda_error((int)e);
        return DSSD_ERR_CUDA;
    }
    if (dev < 0 || dev >= 64) return DSSD_ERR_UNSUPPORTED;
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ptr[dev]) {
            void *ptr = nullptr;
            e = cudaGetSymbolAddress(&ptr, g_static_scratch);
            if (e == cudaSuccess && !ptr) e = cudaErrorInvalidSymbol;  // a look-up that gives no address is a failed one
            if (e != cudaSuccess) {
                dssd::set_last_cuda_error((int)e);
                return DSSD_ERR_CUDA;
            }
            g_static_ptr[dev] = ptr;
        }
        scratch = g_static_ptr[dev];
    }

    dssd::ResampleParams P{};
    P.p_row = p_row;
    P.draft_q = draft_q;
    P.accept_len = accept_len;
    P.uniforms = uniforms;
    P.B = B;
    P.gamma = gamma;
    P.V = V;
    P.token = token;
    P.flags = flags;
    // resample_launch refills the part of the scratch it uses (counters and validity patterns),
    // so what the previous call left behind does not matter
    e = dssd::resample_launch(P, scratch, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) {
        dssd::set_last_cuda_error((int)e);
        return DSSD_ERR_CUDA;
    }
    return DSSD_OK;
}
