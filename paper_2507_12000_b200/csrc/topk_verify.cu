// Truncated-support (top-k) verification round for sm_100a: the sampler of the paper's
// experiments (Section 4) applied to Algorithm 2.
//
// Edge kernel.  The work is one pass over the logits, so the kernel is a pure HBM read stream
// with a selection riding on it:
//
//   * Rows are cut into blocks of kTopkBlock entries; the blocks of all rows are numbered row
//     by row and divided evenly over the resident CTAs, each CTA owning one contiguous span.
//     A span crosses row boundaries, so a CTA works through a few "pieces" (row, first block,
//     last block); no tickets, no atomics on the streaming path, every CTA ends at the same time.
//   * Warp specialisation.  One producer thread streams the CTA's span through a ring of
//     kStages shared-memory stages with bulk asynchronous copies (TMA, untiled) that complete
//     on "full" mbarriers; the consumer warps read a stage into registers (kU vectors of 16
//     bytes per thread), scan them and release the stage through an "empty" mbarrier.  Memory
//     latency is hidden by the rings, not by the consumers; several small CTAs share an SM so
//     that one CTA's selection work overlaps with the others' streaming.
//   * Each vector is reduced to its maximum with NaN-propagating max instructions and compared
//     with the warp's threshold tau, a lower bound on the piece's k-th largest logit.  A vector
//     that reaches tau is taken apart by the whole warp: its 16 bytes are broadcast and lane j
//     judges element j; the elements that beat the threshold key go into the warp's own ring of
//     keys in shared memory (no atomics).  One vote per stage settles the common case that
//     nothing reaches tau.  The consumers never meet at a barrier within a piece.
//   * A key is 64 bits: the logit mapped to an unsigned integer that sorts like the float
//     (with -0 folded into +0), then the complemented index - larger key = earlier in the order
//     (logit descending, index ascending), and all keys of a row are distinct.
//   * A selection warp drains the rings.  Lane r holds entry r of the piece's list, best first;
//     a candidate is inserted with one ballot (its position) and one shuffle (the shift), and
//     the k-th key is published in shared memory, where the consumers pick it up at their next
//     stage.  No sorting network, no merge rounds.
//   * tau starts from the piece's first stage: the consumer threads form 32 groups, each
//     group's maximum is one distinct element, so the k-th largest group maximum (k <= 32) is a
//     valid lower bound.  On input that defeats the threshold (an ascending row) every element
//     goes through the rings: slow, never wrong; a full ring makes its warp wait.
//   * Pieces alternate between two channels (rings, threshold, counters), so the consumers
//     scan a piece while the selection warp still finishes the one before.  At the end of a
//     piece the selection warp frees its channel and then settles the row: a row that was one
//     piece is judged on the spot, from the registers (its k logits become probabilities in
//     float64, the acceptance test runs, the k pairs and a verdict word go to the workspace);
//     a piece of a shared row is published and counted on the row, and the CTA that completes
//     the row merges the pieces by rank counting and judges it.  Judged rows are counted on
//     their sequence; the CTA that completes a sequence finds the first rejection among the
//     verdict words and copies row n's pairs out: two small batches of loads.  So the float64
//     work of a sequence is spread over the CTAs that scanned its rows and overlaps the stream,
//     instead of following it in one warp.  No counter's answer is waited for: it is looked at
//     one piece later.
//   * Every wait (mbarrier, ring, channel hand-off) is bounded; a wait that runs out raises an
//     error word in the workspace, the kernel runs to its end without faulting and every
//     sequence folded after that carries DSSD_EDGE_FLAG_TIMEOUT.
//
// Device kernel: one warp per sequence, everything in registers and shuffles, sums strictly
// sequential in float64 so that the draw is reproducible bit for bit.
#include <atomic>
#include <utility>

#include <cooperative_groups.h>
#include "topk_verify.h"

#include <math.h>

#include "dssd_device.cuh"

namespace dssd {
namespace {

constexpr int kConsWarps = 4;      // consumer warps per CTA (a power of two, 4..16)
constexpr int kConsThreads = 32 * kConsWarps;
constexpr int kTkThreads = kConsThreads + 64;        // + the producer warp and the selection warp
constexpr int kStages = 3;            // ring stages per CTA
constexpr int kStageBytes = 16384;   // logits bytes per stage (one bulk copy)
constexpr int kStageVecs = kStageBytes / 16;         // 16-byte vectors per stage
constexpr int kU = kStageVecs / kConsThreads;        // vectors per consumer thread per stage
constexpr int kGroup = kConsThreads / 32;            // threads per group of the first threshold
static_assert(kU >= 1 && kU * kConsThreads == kStageVecs && kGroup >= 4 && kGroup <= 16, "stage / consumer shape");
constexpr int kCap = 32;                // candidate keys per consumer warp and channel (32: one batch of the selection warp)
constexpr unsigned kSpinLimit = 1u << 16;            // tries of a bounded wait (about 4 us each)
constexpr unsigned kSpinLimitAborted = 8u;           // after a wait has run out
constexpr unsigned long long kBadList = ~0ull;  // first key of a piece that held a NaN or +inf
constexpr unsigned kFullMask = 0xffffffffu;

__device__ __forceinline__ float max_nan(float a, float b)
{
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

__device__ __forceinline__ uint32_t max_nan_bf16x2(uint32_t a, uint32_t b)
{
    uint32_t r;
    asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
    return r;
}

// unsigned integers that sort like the floats they come from (NaN excluded by the callers)
__device__ __forceinline__ uint32_t ord(float f)
{
    uint32_t b = __float_as_uint(f);
    if (b == 0x80000000u) b = 0u;  // -0 and +0 are the same logit
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__device__ __forceinline__ float unord(uint32_t o)
{
    return __uint_as_float((o & 0x80000000u) ? (o & 0x7fffffffu) : ~o);
}

__device__ __forceinline__ unsigned long long make_key(float f, int idx)
{
    return ((unsigned long long)ord(f) << 32) | (unsigned long long)(~(uint32_t)idx);
}

__device__ __forceinline__ int key_index(unsigned long long key) { return (int)(~(uint32_t)key); }
__device__ __forceinline__ float key_value(unsigned long long key) { return unord((uint32_t)(key >> 32)); }

template <int DT>
struct Vec;
template <>
struct Vec<DSSD_F32> {
    static constexpr int E = 4;
    static constexpr int kEsz = 4;
    __device__ static __forceinline__ uint4 fill() { return make_uint4(0xff800000u, 0xff800000u, 0xff800000u, 0xff800000u); }
    __device__ static __forceinline__ float vmax(const uint4 &v)
    {
        return max_nan(max_nan(__uint_as_float(v.x), __uint_as_float(v.y)),
                       max_nan(__uint_as_float(v.z), __uint_as_float(v.w)));
    }
    __device__ static __forceinline__ float load(const void *row, int64_t i) { return reinterpret_cast<const float *>(row)[i]; }
    // element j of the vector (j < E)
    __device__ static __forceinline__ float elem(const uint4 &v, int j)
    {
        return __uint_as_float(j < 2 ? (j == 0 ? v.x : v.y) : (j == 2 ? v.z : v.w));
    }
};
template <>
struct Vec<DSSD_BF16> {
    static constexpr int E = 8;
    static constexpr int kEsz = 2;
    __device__ static __forceinline__ uint4 fill() { return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u); }
    __device__ static __forceinline__ float vmax(const uint4 &v)
    {
        const uint32_t w = max_nan_bf16x2(max_nan_bf16x2(v.x, v.y), max_nan_bf16x2(v.z, v.w));
        return max_nan(bf16_lo(w), bf16_hi(w));
    }
    __device__ static __forceinline__ float load(const void *row, int64_t i)
    {
        return __uint_as_float((uint32_t)reinterpret_cast<const unsigned short *>(row)[i] << 16);
    }
    __device__ static __forceinline__ float elem(const uint4 &v, int j)
    {
        const uint32_t w = j < 4 ? (j < 2 ? v.x : v.y) : (j < 6 ? v.z : v.w);
        return (j & 1) ? bf16_hi(w) : bf16_lo(w);
    }
};

// What the consumers and the selection warp share for one piece.  There are two of them, used
// by even and odd pieces, so that the consumers can scan a piece while the selection warp is
// still finishing the one before.
struct Channel {
    unsigned long long keys[kConsWarps][kCap];  // candidate keys of consumer warp w on their way to the selection warp
    unsigned head[kConsWarps];          // keys warp w has written (counts up for the kernel's life)
    unsigned tail[kConsWarps];          // keys the selection warp has taken from warp w
    unsigned long long taukey;          // the selection warp's current k-th key (0: list not full yet)
    unsigned done;                      // consumer warps that have finished the piece
    int bad;                            // the piece holds a NaN or +inf
};

struct Smem {
    unsigned long long full[kStages];   // mbarriers: stage filled by the copy engine
    unsigned long long empty[kStages];  // mbarriers: stage read by all consumer warps
    Channel ch[2];
    float grp[2][32];                   // group maxima of a piece's first stage (by piece parity)
    int abort;                          // a bounded wait ran out
    unsigned long long fold_keys[kTopkMergeKeys];  // fold: one row's pieces
    unsigned long long fold_top[32];               // fold: the row's top-k, best first
};

// Piece boundary (one named barrier per piece parity): before scanning piece j the consumers
// wait here for each other and for the selection warp to have finished piece j - 2, which used
// the same channel; the selection warp only arrives and goes on.
__device__ __forceinline__ void boundary_sync(int parity)
{
    if (parity) asm volatile("bar.sync 2, %0;" ::"n"(kConsThreads + 32) : "memory");
    else asm volatile("bar.sync 1, %0;" ::"n"(kConsThreads + 32) : "memory");
}
__device__ __forceinline__ void boundary_arrive(int parity)
{
    if (parity) asm volatile("bar.arrive 2, %0;" ::"n"(kConsThreads + 32) : "memory");
    else asm volatile("bar.arrive 1, %0;" ::"n"(kConsThreads + 32) : "memory");
}

// acquire-release fences (the sequentially consistent ones that __threadfence*() emit cost a
// pipeline drain each, which the selection warp cannot afford once per batch)
__device__ __forceinline__ void fence_cta() { asm volatile("fence.acq_rel.cta;" ::: "memory"); }
__device__ __forceinline__ void fence_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }

// release / acquire on a shared-memory word at CTA scope: what the hand-offs between the
// consumer warps and the selection warp are built from
__device__ __forceinline__ void st_release_shared(unsigned *p, unsigned v)
{
    asm volatile("st.release.cta.shared.u32 [%0], %1;" ::"r"(smem_addr(p)), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned ld_acquire_shared(const unsigned *p)
{
    unsigned v;
    asm volatile("ld.acquire.cta.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_addr(p)) : "memory");
    return v;
}

__device__ __forceinline__ unsigned ld_shared_volatile_u32(const unsigned *p) { return *reinterpret_cast<const volatile unsigned *>(p); }
__device__ __forceinline__ unsigned long long ld_shared_volatile_u64(const unsigned long long *p)
{
    return *reinterpret_cast<const volatile unsigned long long *>(p);
}

__device__ __forceinline__ void raise_abort(const TopkParams &P, Smem &S)
{
    *reinterpret_cast<volatile int *>(&S.abort) = 1;
    atomicExch(P.error, 1u);
}

// A consumer warp's end of its key ring (the same values in all lanes)
struct Outbox {
    unsigned head;   // keys written so far
    unsigned tail;   // the selection warp's progress as last read
};

// Hands the keys of the lanes in `wm` (at most kCap of them) to the selection warp through the
// warp's own ring: no atomic, no other consumer warp involved.  Waits, bounded, while the ring
// is full; keys that cannot be delivered are dropped and the error word is raised.
__device__ __forceinline__ void push_keys(const TopkParams &P, Smem &S, Channel &C, int warp, Outbox &ob, unsigned wm,
                                          unsigned long long key)
{
    const int lane = threadIdx.x & 31;
    const unsigned n = (unsigned)__popc(wm);
    unsigned it = 0;
    while (ob.head + n - ob.tail > (unsigned)kCap) {
        ob.tail = ld_acquire_shared(&C.tail[warp]);
        if (ob.head + n - ob.tail <= (unsigned)kCap) break;
        if (++it > kSpinLimit * 64u || *reinterpret_cast<volatile int *>(&S.abort)) {
            raise_abort(P, S);
            return;
        }
        __nanosleep(32);
    }
    if ((wm >> lane) & 1u)
        *reinterpret_cast<volatile unsigned long long *>(&C.keys[warp][(ob.head + (unsigned)__popc(wm & ((1u << lane) - 1u))) % kCap]) = key;
    ob.head += n;
    __syncwarp();
    if (lane == 0) st_release_shared(&C.head[warp], ob.head);
}

// The ragged ends of a piece: lane e < count judges element first + e
template <int DT>
__device__ __forceinline__ void offer_ragged(const TopkParams &P, Smem &S, Channel &C, int warp, Outbox &ob, const char *rowp,
                                             int first, int count, unsigned long long taukey)
{
    const int lane = threadIdx.x & 31;
    bool want = false;
    unsigned long long key = 0ull;
    if (lane < count) {
        const float f = Vec<DT>::load(rowp, first + lane);
        if (f != f || f == INFINITY) {
            C.bad = 1;
        } else {
            key = make_key(f, first + lane);
            want = key > taukey;
        }
    }
    const unsigned wm = __ballot_sync(kFullMask, want);
    if (wm) push_keys(P, S, C, warp, ob, wm, key);
}

// Scans the warp's kU x 32 vectors of one stage.  One vote settles the common case that nothing
// reaches tau.  Otherwise a vector whose maximum (NaN-propagating) reaches tau is taken apart
// by the whole warp: its 16 bytes are broadcast and lane j judges element j; the keys that pass
// go into the warp's own ring.  vi0 = this lane's first vector within
// the piece's vector body, idx0 = vocabulary index of the body's first element.
template <int DT>
__device__ __forceinline__ void scan(const TopkParams &P, const uint4 (&a)[kU], int vi0, int nvec, int idx0, float tau,
                                     unsigned long long taukey, Smem &S, Channel &C, int warp, Outbox &ob)
{
    constexpr int E = Vec<DT>::E;
    const int lane = threadIdx.x & 31;
    float vm[kU];
#pragma unroll
    for (int u = 0; u < kU; ++u) vm[u] = Vec<DT>::vmax(a[u]);
    float top = vm[0];
#pragma unroll
    for (int u = 1; u < kU; ++u) top = max_nan(top, vm[u]);
    if (!__any_sync(kFullMask, !(top < tau))) return;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const int vi = vi0 + u * kConsThreads;
        unsigned hot = __ballot_sync(kFullMask, vi < nvec && !(vm[u] < tau));
        while (hot) {
            const int src = __ffs(hot) - 1;
            uint4 v;
            v.x = __shfl_sync(kFullMask, a[u].x, src);
            v.y = __shfl_sync(kFullMask, a[u].y, src);
            v.z = __shfl_sync(kFullMask, a[u].z, src);
            v.w = __shfl_sync(kFullMask, a[u].w, src);
            const float f = Vec<DT>::elem(v, lane);
            bool want = false;
            unsigned long long key = 0ull;
            if (lane < E && !(f < tau)) {
                if (f != f || f == INFINITY) {
                    C.bad = 1;
                } else {
                    key = make_key(f, idx0 + (vi - lane + src) * E + lane);
                    want = key > taukey;
                }
            }
            const unsigned wm = __ballot_sync(kFullMask, want);
            if (wm) push_keys(P, S, C, warp, ob, wm, key);
            hot &= hot - 1u;
        }
    }
}

// Geometry of one piece: elements [e0, e1) of a row = ragged head (up to the first 16-byte
// boundary), `nvec` whole vectors streamed through the ring in `stages` bulk copies, ragged tail.
struct Piece {
    const char *rowp;
    const uint4 *vp;   // first whole vector
    int64_t row;
    int fb, lb;        // blocks [fb, lb) of the row
    int e0, e1, head, nvec, idx0, tail0, stages;
};

template <int DT>
__device__ __forceinline__ Piece piece_at(const TopkParams &P, unsigned long long blk, unsigned long long blk_end)
{
    constexpr int E = Vec<DT>::E;
    constexpr int kEsz = Vec<DT>::kEsz;
    Piece pc;
    pc.row = (int64_t)(blk / (unsigned long long)P.nb);
    pc.fb = (int)(blk - (unsigned long long)pc.row * P.nb);
    pc.lb = (int)min((unsigned long long)P.nb, pc.fb + (blk_end - blk));
    pc.e0 = pc.fb * kTopkBlock;
    pc.e1 = (int)min((long long)P.V, (long long)pc.lb * kTopkBlock);
    pc.rowp = reinterpret_cast<const char *>(P.logits) + (size_t)pc.row * (size_t)P.row_stride * kEsz;
    const uintptr_t addr = reinterpret_cast<uintptr_t>(pc.rowp) + (uintptr_t)pc.e0 * kEsz;
    pc.head = min(pc.e1 - pc.e0, (int)(((16u - (unsigned)(addr & 15u)) & 15u) / kEsz));
    pc.nvec = (pc.e1 - pc.e0 - pc.head) / E;
    pc.idx0 = pc.e0 + pc.head;
    pc.tail0 = pc.idx0 + pc.nvec * E;
    pc.vp = reinterpret_cast<const uint4 *>(pc.rowp + (size_t)pc.idx0 * kEsz);
    pc.stages = (pc.nvec + kStageVecs - 1) / kStageVecs;
    return pc;
}

// Bounded wait on a ring barrier.  Once a wait has run out the CTA keeps going with short
// waits, so that it still ends, and reports through the error word.
__device__ __forceinline__ void ring_wait(const TopkParams &P, Smem &S, unsigned long long *bar, uint32_t parity)
{
    const unsigned limit = *reinterpret_cast<volatile int *>(&S.abort) ? kSpinLimitAborted : kSpinLimit;
    if (!mbar_wait(smem_addr(bar), parity, limit)) raise_abort(P, S);
}

// The producer thread: streams the CTA's span, stage by stage, in the order the consumers read it.
// It can stop after a given number of stages and be resumed (the first stages go out before the
// grid-wide barrier at the start of the kernel, the rest after it).
struct ProducerPos {
    unsigned long long blk;  // first block of the piece in progress
    int s;                   // next stage of that piece
    unsigned q;              // stages issued so far
};

template <int DT>
__device__ void producer(const TopkParams &P, Smem &S, uint32_t ring, ProducerPos &pos, unsigned long long blk_end,
                         unsigned q_stop)
{
    while (pos.blk < blk_end) {
        const Piece pc = piece_at<DT>(P, pos.blk, blk_end);
        for (; pos.s < pc.stages; ++pos.s, ++pos.q) {
            if (pos.q == q_stop) return;
            const unsigned slot = pos.q % kStages, pass = pos.q / kStages;
            if (pass > 0) ring_wait(P, S, &S.empty[slot], (pass - 1u) & 1u);
            const uint32_t bytes = (uint32_t)min(kStageVecs, pc.nvec - pos.s * kStageVecs) * 16u;
            const uint32_t bar = smem_addr(&S.full[slot]);
            mbar_arrive_expect_tx(bar, bytes);
            // no logit is read twice: the evict_first hint keeps the stream from pushing the
            // workspace's lines (partial results, counters) out of L2
            bulk_g2s_hint(ring + slot * (uint32_t)kStageBytes, pc.vp + (size_t)pos.s * kStageVecs, bytes, bar,
                          l2_policy_evict_first());
        }
        pos.s = 0;
        pos.blk += (unsigned long long)(pc.lb - pc.fb);
    }
}

// The consumers' part of one piece.  `q` counts the stages consumed so far (the ring position),
// as the producer counts them; `parity` is the piece's parity within this CTA.
template <int DT>
__device__ void consume_piece(const TopkParams &P, const Piece &pc, int k, int parity, Smem &S, uint32_t ring, unsigned &q)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    Channel &C = S.ch[parity];
    uint4 a[kU];
    unsigned slot = 0;
    const uint32_t lane_off = (uint32_t)tid * 16u;
    if (pc.stages > 0) {
        slot = q % kStages;
        ring_wait(P, S, &S.full[slot], (q / kStages) & 1u);
#pragma unroll
        for (int u = 0; u < kU; ++u)
            a[u] = tid + u * kConsThreads < pc.nvec ? lds16(ring + slot * (uint32_t)kStageBytes + lane_off + (uint32_t)u * kConsThreads * 16u)
                                                    : Vec<DT>::fill();
    } else {
#pragma unroll
        for (int u = 0; u < kU; ++u) a[u] = Vec<DT>::fill();
    }
    // tau from the first stage: k-th largest of the 32 group maxima
    float tm = -INFINITY;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        const float v = Vec<DT>::vmax(a[u]);
        tm = fmaxf(tm, v == v ? v : -INFINITY);
    }
#pragma unroll
    for (int o = 1; o < kGroup; o <<= 1) tm = fmaxf(tm, __shfl_xor_sync(kFullMask, tm, o));
    if ((tid & (kGroup - 1)) == 0) S.grp[parity][tid / kGroup] = tm;
    boundary_sync(parity);  // the channel is free: the selection warp has finished the piece before the last
    float tau;
    {
        const float g = S.grp[parity][lane];
        int rank = 0;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            const float o = __shfl_sync(kFullMask, g, j);
            rank += (o > g) || (o == g && j < lane);
        }
        const unsigned hit = __ballot_sync(kFullMask, rank == k - 1);
        tau = __shfl_sync(kFullMask, g, __ffs(hit) - 1);
    }
    unsigned long long taukey = (unsigned long long)ord(tau) << 32;
    Outbox ob;
    ob.head = C.head[warp];  // only this warp writes it
    ob.tail = ob.head;       // the ring is empty: the selection warp finished with this channel
    // the ragged ends of the piece (warp 0: before the first whole vector, warp 1: after the last)
    if (warp == 0 && pc.head > 0) offer_ragged<DT>(P, S, C, warp, ob, pc.rowp, pc.e0, pc.head, taukey);
    if (warp == 1 % kConsWarps && pc.e1 > pc.tail0) offer_ragged<DT>(P, S, C, warp, ob, pc.rowp, pc.tail0, pc.e1 - pc.tail0, taukey);
    for (int s = 0; s < pc.stages; ++s, ++q) {
        if (s > 0) {
            slot = q % kStages;
            ring_wait(P, S, &S.full[slot], (q / kStages) & 1u);
#pragma unroll
            for (int u = 0; u < kU; ++u)
                a[u] = s * kStageVecs + tid + u * kConsThreads < pc.nvec
                           ? lds16(ring + slot * (uint32_t)kStageBytes + lane_off + (uint32_t)u * kConsThreads * 16u)
                           : Vec<DT>::fill();
            // the selection warp's k-th key, once it beats what this warp filters with
            const unsigned long long pub = ld_shared_volatile_u64(&C.taukey);
            if (pub > taukey) {
                taukey = pub;
                tau = key_value(pub);
            }
        }
        scan<DT>(P, a, s * kStageVecs + tid, pc.nvec, pc.idx0, tau, taukey, S, C, warp, ob);
        // the stage has been consumed from registers: hand the buffer back to the producer
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_addr(&S.empty[slot]));
    }
    // this warp's candidates of the piece are all in its ring
    __syncwarp();
    if (lane == 0) {
        fence_cta();
        atomicAdd(&C.done, 1u);
    }
}

// CTA that owns block `blk` when `total` blocks are divided over `grid` CTAs
__device__ __forceinline__ unsigned long long owner_of(unsigned long long blk, unsigned long long grid, unsigned long long total)
{
    return ((blk + 1ull) * grid - 1ull) / total;
}

struct RowDist {   // per lane r < k: entry r of the row's support, best first
    int idx;
    double prob;
    bool bad;      // the row has no distribution (warp-uniform)
};

// pieces that share `row`
__device__ __forceinline__ int pieces_of(const TopkParams &P, int64_t row)
{
    const unsigned long long first_blk = (unsigned long long)row * (unsigned long long)P.nb;
    return (int)(owner_of(first_blk + P.nb - 1, P.grid, P.total_blocks) - owner_of(first_blk, P.grid, P.total_blocks)) + 1;
}

// One warp: lane r < k holds key r of a row's support (best first; kBadList in lane 0 marks a
// row with a NaN or +inf).  Turns the k logits into probabilities in float64, summed in rank order.
__device__ __forceinline__ RowDist dist_from_keys(const TopkParams &P, unsigned long long key)
{
    const int lane = threadIdx.x & 31, k = P.k;
    RowDist d;
    d.idx = -1;
    d.prob = NAN;
    const float val = key_value(key);
    const float best = __shfl_sync(kFullMask, val, 0);
    d.bad = __shfl_sync(kFullMask, key, 0) == kBadList || !(best > -INFINITY);  // nothing above -inf
    if (d.bad) return d;
    const double T = (double)P.temperature;
    const double z = (double)val / T;
    const double mx = __shfl_sync(kFullMask, z, 0);
    const double e = lane < k ? exp(z - mx) : 0.0;
    double S = 0.0;
    for (int r = 0; r < k; ++r) S += __shfl_sync(kFullMask, e, r);
    d.idx = lane < k ? key_index(key) : -1;
    d.prob = e / S;
    return d;
}

// One warp: merges the `pieces` lists of `row` by rank counting; returns key r in lane r.
__device__ unsigned long long merged_keys(const TopkParams &P, int64_t row, int pieces, unsigned long long *keys,
                                          unsigned long long *top)
{
    const int lane = threadIdx.x & 31, k = P.k;
    const int m = pieces * k;
    const unsigned long long *src = P.lists + (size_t)row * P.max_pieces * k;
    bool bad = false;
    __syncwarp();
    for (int i = lane; i < m; i += 32) {
        const unsigned long long x = __ldcg(src + i);
        bad |= (x == kBadList);
        keys[i] = x;
    }
    bad = __any_sync(kFullMask, bad);
    __syncwarp();
    if (bad) return lane == 0 ? kBadList : 0ull;
    for (int i = lane; i < m; i += 32) {
        const unsigned long long x = keys[i];
        int rank = 0;
        for (int j = 0; j < m; ++j) rank += keys[j] > x;
        if (rank < k) top[rank] = x;  // keys below rank k include every empty slot
    }
    __syncwarp();
    return lane < k ? top[lane] : 0ull;
}

// The acceptance test of one position, as the oracle states it (float64 throughout)
__device__ __forceinline__ bool judge(const TopkParams &P, const RowDist &d, int x, double u, double q, unsigned &fl,
                                      double &p)
{
    const int lane = threadIdx.x & 31;
    const unsigned holds = __ballot_sync(kFullMask, lane < P.k && !d.bad && d.idx == x);
    const double p_in = __shfl_sync(kFullMask, d.prob, holds ? __ffs(holds) - 1 : 0);
    if (x < 0 || x >= P.V) {
        fl |= DSSD_EDGE_FLAG_BAD_TOKEN;
        p = NAN;
        return false;
    }
    p = d.bad ? NAN : (holds ? p_in : 0.0);
    double ratio;
    if (q != q || p != p) ratio = NAN;
    else if (q <= 0.0) ratio = p > 0.0 ? INFINITY : 0.0;
    else ratio = p / q;
    return (ratio == ratio) && (u < (ratio < 1.0 ? ratio : 1.0));
}

// A position's draft (token, uniform, q of the token), requested when its row's piece starts
struct Draft {
    int x;
    float u, q;
};

__device__ __forceinline__ Draft load_draft(const TopkParams &P, int64_t row)
{
    Draft d;
    d.x = 0;
    d.u = d.q = 0.f;
    const int b = (int)(row / (P.gamma + 1)), j = (int)(row - (int64_t)b * (P.gamma + 1));
    if (j < P.gamma) {
        const size_t o = (size_t)b * P.gamma + j;
        d.x = __ldg(P.draft_tokens + o);
        d.u = __ldg(P.uniforms + o);
        d.q = __ldg(P.draft_q_tok + o);
    }
    return d;
}

// verdict word of a row: bit 0 = the position was accepted (always set for the bonus row), the
// row's flag bits above it
constexpr unsigned kVerdictAccept = 1u;
constexpr int kVerdictFlagShift = 8;

// One warp, lane r < k holding key r of `row`'s support: the row's k pairs (index, probability)
// go to the first list slot of the row, its verdict word to `verdict`; counts the row on its
// sequence and returns the count including this row (lane 0; the caller decides when to look).
__device__ __forceinline__ unsigned judge_row(const TopkParams &P, int64_t row, unsigned long long key, const Draft &dr)
{
    const int lane = threadIdx.x & 31, k = P.k;
    const int b = (int)(row / (P.gamma + 1)), j = (int)(row - (int64_t)b * (P.gamma + 1));
    const RowDist d = dist_from_keys(P, key);
    unsigned fl = d.bad ? DSSD_EDGE_FLAG_NONFINITE : 0u;
    bool accept = true;
    if (j < P.gamma) {
        double p;
        accept = judge(P, d, dr.x, (double)dr.u, (double)dr.q, fl, p);
        if (lane == 0 && P.p_tok) P.p_tok[(size_t)b * P.gamma + j] = (float)p;
    }
    if (lane < k) {
        const unsigned long long pair = (unsigned long long)(uint32_t)(d.bad ? -1 : d.idx) |
                                        ((unsigned long long)__float_as_uint(d.bad ? NAN : (float)d.prob) << 32);
        __stcg(P.lists + (size_t)row * P.max_pieces * k + lane, pair);
    }
    if (lane == 0) __stcg(P.verdict + row, (accept ? kVerdictAccept : 0u) | (fl << kVerdictFlagShift));
    fence_gpu();
    __syncwarp();
    unsigned cnt = 0;
    if (lane == 0) cnt = atomicAdd(P.seq_done + b, 1u) + 1u;
    return cnt;
}

// The selection warp of the CTA that judged a sequence's last row: first rejection over the
// rows' verdict words (one batch of loads), then row n's pairs (a second one).
__device__ __noinline__ void fold_sequence(const TopkParams &P, int b)
{
    const int lane = threadIdx.x & 31;
    const int gamma = P.gamma, k = P.k;
    unsigned fl = ld_relaxed_u32(P.error) ? DSSD_EDGE_FLAG_TIMEOUT : 0u;
    const int64_t row0 = (int64_t)b * (gamma + 1);
    int n = gamma;
    for (int base = 0; base <= gamma; base += 32) {
        const int j = base + lane;
        const unsigned v = j <= gamma ? __ldcg(P.verdict + row0 + j) : kVerdictAccept;
        fl |= v >> kVerdictFlagShift;
        const unsigned rej = __ballot_sync(kFullMask, !(v & kVerdictAccept));
        if (rej && n == gamma) n = base + __ffs(rej) - 1;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) fl |= __shfl_xor_sync(kFullMask, fl, o);
    if (lane < k) {
        const unsigned long long pair = __ldcg(P.lists + (size_t)(row0 + n) * P.max_pieces * k + lane);
        P.p_idx[(size_t)b * k + lane] = (int)(uint32_t)pair;
        P.p_val[(size_t)b * k + lane] = __uint_as_float((uint32_t)(pair >> 32));
    }
    if (lane == 0) {
        P.accept_len[b] = n;
        if (P.flags) P.flags[b] = fl;
    }
}

// The selection warp.  Lane r holds entry r of the current piece's list, best first; candidates
// arrive through the consumer warps' rings in shared memory and are inserted by a ballot and a shuffle;
// the k-th key is published for the consumers to filter with.  At the end of a piece the warp
// frees the channel (boundary_arrive) before it writes the list out, counts the piece's
// blocks and, when that completes a sequence, folds it; the other channel's rings buffer the
// next piece's candidates meanwhile.
template <int DT>
__device__ void selection_warp(const TopkParams &P, Smem &S, unsigned long long blk, unsigned long long blk_end)
{
    const int lane = threadIdx.x & 31, k = P.k;
    const unsigned long long G = (unsigned long long)P.grid, TB = P.total_blocks, c = blockIdx.x;
    const unsigned per_seq = (unsigned)(P.gamma + 1);
    unsigned tails[2] = {0u, 0u};  // lane w < kConsWarps: keys taken from warp w's ring, per channel
    // No counter's answer is waited for: it is looked at one piece later (or after the last piece).
    //   seq_b[i], seq_cnt[i]   a sequence and (lane 0) its count of judged rows after a row of it
    //                          was judged here: i = 0 a row that was one piece, i = 1 a merged row
    //   def_row, def_cnt, ...  a row of several pieces and (lane 0) its count of published pieces
    int seq_b[2] = {-1, -1};
    unsigned seq_cnt[2] = {0u, 0u};
    int64_t def_row = -1;
    unsigned def_cnt = 0u;
    int def_pcs = 0;
    Draft def_draft = {0, 0.f, 0.f};
    auto settle = [&]() {
#pragma unroll
        for (int i = 0; i < 2; ++i) {
            if (seq_b[i] < 0) continue;
            const bool last = __shfl_sync(kFullMask, (int)(seq_cnt[i] == per_seq), 0);
            if (last) {
                fence_gpu();
                fold_sequence(P, seq_b[i]);
            }
            seq_b[i] = -1;
        }
        if (def_row >= 0) {
            const bool last = __shfl_sync(kFullMask, (int)(def_cnt == (unsigned)def_pcs), 0);
            if (last) {
                fence_gpu();
                const unsigned long long key = merged_keys(P, def_row, def_pcs, S.fold_keys, S.fold_top);
                seq_cnt[1] = judge_row(P, def_row, key, def_draft);
                seq_b[1] = (int)(def_row / (P.gamma + 1));
            }
            def_row = -1;
        }
    };
    boundary_arrive(0);  // both channels start free
    boundary_arrive(1);
    int parity = 0;
    while (blk < blk_end) {
        const Piece pc = piece_at<DT>(P, blk, blk_end);
        const Draft draft = load_draft(P, pc.row);  // used when the piece ends
        Channel &C = S.ch[parity];
        unsigned tl = parity ? tails[1] : tails[0];
        // empty slots hold distinct small keys (k - r in slot r), below every real key
        unsigned long long key = lane < k ? (unsigned long long)(k - lane) : 0ull;
        unsigned long long tkey = 0ull;
        unsigned idle = 0;
        for (;;) {
            const bool last_look = ld_shared_volatile_u32(&C.done) == (unsigned)kConsWarps;  // read before the heads
            const unsigned h = lane < kConsWarps ? ld_acquire_shared(&C.head[lane]) : 0u;
            unsigned pend = __ballot_sync(kFullMask, lane < kConsWarps && h != tl);
            if (!pend) {
                if (last_look) break;
                if (++idle > kSpinLimit * 256u) {
                    raise_abort(P, S);
                    break;
                }
                continue;
            }
            idle = 0;
            while (pend) {
                const int w = __ffs(pend) - 1;
                pend &= pend - 1u;
                const unsigned hw = __shfl_sync(kFullMask, h, w), tw = __shfl_sync(kFullMask, tl, w);
                const unsigned long long v =
                    (unsigned)lane < hw - tw ? ld_shared_volatile_u64(&C.keys[w][(tw + (unsigned)lane) % kCap]) : 0ull;
                // insert the candidates that beat the k-th key as it stood when the batch was taken; one
                // that has been overtaken within the batch lands beyond lane k - 1 and is never read
                unsigned want = __ballot_sync(kFullMask, v > tkey);
                // the keys are in registers: give the slots back
                if (lane == w) {
                    tl = hw;
                    st_release_shared(&C.tail[w], hw);
                }
                while (want) {
                    const int src = __ffs(want) - 1;
                    want &= want - 1u;
                    const unsigned long long x = __shfl_sync(kFullMask, v, src);
                    const unsigned long long up = __shfl_up_sync(kFullMask, key, 1);
                    const int pos = __popc(__ballot_sync(kFullMask, key > x));  // keys above x form a prefix
                    key = lane == pos ? x : (lane > pos ? up : key);
                }
            }
            const unsigned long long kth = __shfl_sync(kFullMask, key, k - 1);
            if (kth > (unsigned long long)k && kth != tkey) {  // the list is full of real keys
                tkey = kth;
                if (lane == 0) *reinterpret_cast<volatile unsigned long long *>(&C.taukey) = tkey;
            }
        }
        if (parity) tails[1] = tl;
        else tails[0] = tl;
        // the piece is complete: take what the consumers left, reset the channel and free it
        const int bad = *reinterpret_cast<volatile int *>(&C.bad);
        __syncwarp();
        if (lane == 0) {
            *reinterpret_cast<volatile int *>(&C.bad) = 0;
            *reinterpret_cast<volatile unsigned *>(&C.done) = 0u;
            *reinterpret_cast<volatile unsigned long long *>(&C.taukey) = 0ull;
            fence_cta();
        }
        __syncwarp();
        boundary_arrive(parity);
        settle();  // what the piece before this one asked for
        const int pcs = pieces_of(P, pc.row);
        unsigned long long out = key;
        if (bad) out = lane == 0 ? kBadList : 0ull;
        if (pcs == 1) {
            // the whole row: judged from the registers
            seq_cnt[0] = judge_row(P, pc.row, lane < k ? out : 0ull, draft);
            seq_b[0] = (int)(pc.row / (P.gamma + 1));
        } else {
            // publish the list, then count the piece on its row
            const int slot = (int)(c - owner_of((unsigned long long)pc.row * P.nb, G, TB));
            if (lane < k) __stcg(P.lists + ((size_t)pc.row * P.max_pieces + slot) * k + lane, out);
            fence_gpu();
            __syncwarp();
            if (lane == 0) def_cnt = atomicAdd(P.row_done + pc.row, 1u) + 1u;
            def_row = pc.row;
            def_pcs = pcs;
            def_draft = draft;
        }
        blk += (unsigned long long)(pc.lb - pc.fb);
        parity ^= 1;
    }
    settle();  // the last piece's row or sequence ...
    settle();  // ... and the sequence of a row merged just now
}

template <int DT>
__global__ void __launch_bounds__(kTkThreads, 4) topk_verify_kernel(const __grid_constant__ TopkParams P)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem &S = *reinterpret_cast<Smem *>(smem_raw + (size_t)kStages * kStageBytes);
    const uint32_t ring = smem_addr(smem_raw);
    const int tid = threadIdx.x;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_addr(&S.full[s]), 1u);
            mbar_init(smem_addr(&S.empty[s]), (uint32_t)kConsWarps);
        }
        for (int h = 0; h < 2; ++h) {
            S.ch[h].taukey = 0ull;
            S.ch[h].done = 0u;
            S.ch[h].bad = 0;
            for (int w = 0; w < kConsWarps; ++w) {
                S.ch[h].head[w] = 0u;
                S.ch[h].tail[w] = 0u;
            }
        }
        S.abort = 0;
        mbar_init_fence();
    }
    // The error word and the sequences' block counters are zeroed here, by the kernel itself: one
    // grid-wide barrier (a cooperative launch: all CTAs are resident) separates that from their first
    // use, and it is split around the producer's first copies, which need nothing of the workspace.
    namespace cg = cooperative_groups;
    cg::grid_group grid = cg::this_grid();
    {
        unsigned long long *z = reinterpret_cast<unsigned long long *>(P.error);
        const size_t nz = P.zero_bytes / 8;
        for (size_t i = (size_t)blockIdx.x * kTkThreads + tid; i < nz; i += (size_t)gridDim.x * kTkThreads) z[i] = 0ull;
    }
    auto arrived = grid.barrier_arrive();  // (a CTA-wide barrier is part of it)
    const unsigned long long G = (unsigned long long)P.grid, TB = P.total_blocks, c = blockIdx.x;
    const unsigned long long blk_end = (c + 1ull) * TB / G;
    unsigned long long blk = c * TB / G;
    ProducerPos pos;
    pos.blk = blk;
    pos.s = 0;
    pos.q = 0;
    if (tid == kConsThreads) producer<DT>(P, S, ring, pos, blk_end, (unsigned)kStages);  // the ring is empty: nothing is waited for
    grid.barrier_wait(std::move(arrived));
    if (tid >= kConsThreads + 32) {
        selection_warp<DT>(P, S, blk, blk_end);
        return;
    }
    if (tid >= kConsThreads) {
        if (tid == kConsThreads) producer<DT>(P, S, ring, pos, blk_end, ~0u);
        return;
    }
    unsigned q = 0;
    int parity = 0;
    while (blk < blk_end) {
        const Piece pc = piece_at<DT>(P, blk, blk_end);
        consume_piece<DT>(P, pc, P.k, parity, S, ring, q);
        parity ^= 1;
        blk += (unsigned long long)(pc.lb - pc.fb);
    }
}

// ---------------------------------------------------------------------------------------------
// device half: one warp per sequence

__device__ __forceinline__ double shfl_f64(double v, int src) { return __shfl_sync(kFullMask, v, src); }

// inverse CDF over the warp's k entries (lane e holds r_e, entries in increasing index);
// returns the position, or -1 when the mass is not positive and finite
__device__ __forceinline__ int warp_inverse_cdf(double r, int k, double u)
{
    double Z = 0.0;
    for (int e = 0; e < k; ++e) Z += shfl_f64(r, e);
    if (!(Z > 0.0) || !(Z < INFINITY)) return -1;
    const double t = u * Z;
    double C = 0.0;
    int last_pos = -1, hit = -1;
    for (int e = 0; e < k; ++e) {
        const double re = shfl_f64(r, e);
        C += re;
        if (re > 0.0) last_pos = e;
        if (hit < 0 && C > t) hit = e;
    }
    return hit >= 0 ? hit : last_pos;
}

__global__ void __launch_bounds__(kThreads) topk_resample_kernel(const TopkResampleParams P)
{
    __shared__ int s_idx[kWarps][32];
    __shared__ float s_val[kWarps][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, k = P.k;
    const int b = blockIdx.x * kWarps + warp;
    if (b >= P.B) return;
    const int n = __ldg(P.accept_len + b);
    const double u = (double)__ldg(P.uniforms + b);
    const int pi = lane < k ? __ldg(P.p_idx + (size_t)b * k + lane) : 0;
    const float pv = lane < k ? __ldg(P.p_val + (size_t)b * k + lane) : 0.f;
    const bool has_row = !__any_sync(kFullMask, lane < k && pi < 0);
    unsigned fl = 0u;
    int tok = -1;
    if (n < 0 || n > P.gamma || !has_row) {
        fl = DSSD_RS_FLAG_INVALID;
    } else {
        // P's entries in increasing vocabulary index (indices are distinct)
        int rank = 0;
        for (int e = 0; e < k; ++e) rank += __shfl_sync(kFullMask, pi, e) < pi;
        if (lane < k) {
            s_idx[warp][rank] = pi;
            s_val[warp][rank] = pv;
        }
        __syncwarp();
        const int sid = lane < k ? s_idx[warp][lane] : -1;
        const double sp = lane < k ? (double)s_val[warp][lane] : 0.0;
        int pos;
        if (n == P.gamma) {
            fl |= DSSD_RS_FLAG_BONUS;
            pos = warp_inverse_cdf(sp, k, u);
        } else {
            const size_t qo = ((size_t)b * P.gamma + n) * (size_t)k;
            const int qi = lane < k ? __ldg(P.q_idx + qo + lane) : -1;
            const float qv = lane < k ? __ldg(P.q_val + qo + lane) : 0.f;
            float sq = 0.f;
            for (int f = k - 1; f >= 0; --f) {  // the first listed match wins
                const int fi = __shfl_sync(kFullMask, qi, f);
                const float fv = __shfl_sync(kFullMask, qv, f);
                if (fi == sid) sq = fv;
            }
            const double r = lane < k ? fmax(0.0, sp - (double)sq) : 0.0;
            pos = warp_inverse_cdf(r, k, u);
            if (pos < 0) {
                fl |= DSSD_RS_FLAG_FALLBACK;
                pos = warp_inverse_cdf(sp, k, u);
            }
        }
        if (pos < 0) fl |= DSSD_RS_FLAG_INVALID;
        else tok = __shfl_sync(kFullMask, sid, pos);
    }
    if (lane == 0) {
        P.token[b] = tok;
        if (P.flags) P.flags[b] = fl;
    }
}

}  // namespace

int topk_max_pieces(int k)
{
    const int byk = kTopkMergeKeys / (k < 1 ? 1 : k);
    return byk < kTopkMaxPieces ? byk : kTopkMaxPieces;
}

size_t topk_workspace_layout(int B, int gamma, int k, TopkParams *P, char *base)
{
    const size_t rows = (size_t)B * (size_t)(gamma + 1);
    const size_t zero = (8 + ((size_t)B + rows) * 4 + 7) & ~(size_t)7;  // error word, seq_done, row_done
    const size_t cnt = (zero + rows * 4 + 255) & ~(size_t)255;          // ... and verdict
    const size_t lists = rows * (size_t)topk_max_pieces(k) * (size_t)k * 8;
    if (P) {
        P->error = reinterpret_cast<unsigned *>(base);
        P->seq_done = reinterpret_cast<unsigned *>(base + 8);
        P->row_done = P->seq_done + B;
        P->verdict = reinterpret_cast<unsigned *>(base + zero);
        P->lists = reinterpret_cast<unsigned long long *>(base + cnt);
        P->zero_bytes = zero;
        P->max_pieces = topk_max_pieces(k);
    }
    return cnt + ((lists + 255) & ~(size_t)255);
}

static std::atomic<int> g_topk_ctas[64];  // CTAs resident on the device at once (0 = not asked yet)
constexpr size_t kTopkSmemBytes = (size_t)kStages * kStageBytes + sizeof(Smem);

cudaError_t topk_verify_launch(TopkParams &P, int dtype, void *workspace, cudaStream_t stream)
{
    cudaError_t err;
    int dev = 0;
    if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
    int ctas = (dev >= 0 && dev < 64) ? g_topk_ctas[dev].load(std::memory_order_acquire) : 0;
    if (ctas == 0) {
        int sms = 0;
        if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
        if ((err = cudaFuncSetAttribute(topk_verify_kernel<DSSD_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTopkSmemBytes)) != cudaSuccess) return err;
        if ((err = cudaFuncSetAttribute(topk_verify_kernel<DSSD_BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kTopkSmemBytes)) != cudaSuccess) return err;
        int occ0 = 0, occ1 = 0;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ0, topk_verify_kernel<DSSD_F32>, kTkThreads, kTopkSmemBytes)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ1, topk_verify_kernel<DSSD_BF16>, kTkThreads, kTopkSmemBytes)) != cudaSuccess) return err;
        const int occ = occ0 < occ1 ? occ0 : occ1;
        ctas = (sms < 1 ? 1 : sms) * (occ < 1 ? 1 : occ);
        if (dev >= 0 && dev < 64) g_topk_ctas[dev].store(ctas, std::memory_order_release);
    }
    topk_workspace_layout(P.B, P.gamma, P.k, &P, static_cast<char *>(workspace));
    const unsigned long long rows = (unsigned long long)P.B * (unsigned long long)(P.gamma + 1);
    P.nb = (P.V + kTopkBlock - 1) / kTopkBlock;
    P.total_blocks = rows * (unsigned long long)P.nb;
    // every span must hold at least ceil(nb / (max_pieces - 1)) blocks, so that no row is shared
    // by more than max_pieces CTAs
    unsigned long long wmin = ((unsigned long long)P.nb + P.max_pieces - 2) / (unsigned long long)(P.max_pieces - 1);
    // a span below about 32 KB is not worth a CTA of its own: small launches get fewer, larger pieces
    const unsigned long long worth = 32768ull / ((unsigned long long)kTopkBlock * (dtype == DSSD_BF16 ? 2u : 4u));
    if (wmin < worth) wmin = worth;
    unsigned long long grid = P.total_blocks / wmin;
    if (grid > (unsigned long long)ctas) grid = (unsigned long long)ctas;
    if (grid < 1) grid = 1;
    P.grid = (int)grid;
    // a cooperative launch: all CTAs are resident at once (grid <= ctas), which the kernel's grid-wide
    // barrier after the zeroing of the counters relies on
    void *args[] = {&P};
    const void *fn = dtype == DSSD_BF16 ? reinterpret_cast<const void *>(topk_verify_kernel<DSSD_BF16>)
                                        : reinterpret_cast<const void *>(topk_verify_kernel<DSSD_F32>);
    return cudaLaunchCooperativeKernel(fn, dim3((unsigned)P.grid), dim3(kTkThreads), args, kTopkSmemBytes, stream);
}

cudaError_t topk_resample_launch(const TopkResampleParams &P, cudaStream_t stream)
{
    const int grid = (P.B + kWarps - 1) / kWarps;
    topk_resample_kernel<<<grid, kThreads, 0, stream>>>(P);
    return cudaGetLastError();
}

}  // namespace dssd
