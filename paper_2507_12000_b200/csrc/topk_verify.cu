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
//     latency is hidden by the rings, not by the consumers; several CTAs share an SM so that
//     one CTA's barriers and merges overlap with the others' streaming.
//   * Each vector is reduced to its maximum with NaN-propagating max instructions and compared
//     with the CTA's threshold tau, a lower bound on the piece's k-th largest logit.  A vector
//     that reaches tau is taken apart by the whole warp: its 16 bytes are broadcast and lane j
//     judges element j; the elements that beat the current k-th key are appended to a candidate
//     buffer in shared memory (one atomic per vector).
//   * A key is 64 bits: the logit mapped to an unsigned integer that sorts like the float
//     (with -0 folded into +0), then the complemented index - larger key = earlier in the order
//     (logit descending, index ascending), and all keys of a row are distinct.
//   * After every stage the consumers meet at a named barrier; when enough candidates have
//     gathered they merge them with the current list by rank counting (each key counts the keys
//     above it; rank < k writes itself to that slot), which needs no sorting network.  The
//     threshold lives in registers and is refreshed from the new list.
//   * tau starts from the piece's first stage: the consumer threads form 32 groups,
//     each group's maximum is one distinct element, so the k-th largest group maximum (k <= 32)
//     is a valid lower bound.  A candidate buffer that overflows anyway (ascending input) is
//     handled by merging and resuming the same registers from where each warp stopped.
//   * The piece's list goes to the workspace; the CTA that completes a sequence (a counter of
//     scanned blocks per sequence tells) folds it: one warp per row merges the row's pieces,
//     turns the k logits into probabilities in float64, applies the acceptance test; the first
//     rejection is an atomicMin in shared memory; warp 0 then writes row n's k pairs.
//   * Every wait on an mbarrier is bounded; a wait that runs out raises an error word in the
//     workspace, the kernel runs to its end without faulting and every sequence folded after
//     that carries DSSD_EDGE_FLAG_TIMEOUT.
//
// Device kernel: one warp per sequence, everything in registers and shuffles, sums strictly
// sequential in float64 so that the draw is reproducible bit for bit.
#include "topk_verify.h"

#include <math.h>

#include "dssd_device.cuh"

namespace dssd {
namespace {

#ifndef DSSD_TOPK_CONS_WARPS
#define DSSD_TOPK_CONS_WARPS 8
#endif
#ifndef DSSD_TOPK_STAGE_BYTES
#define DSSD_TOPK_STAGE_BYTES 32768
#endif
#ifndef DSSD_TOPK_STAGES
#define DSSD_TOPK_STAGES 3
#endif
#ifndef DSSD_TOPK_MIN_CTAS
#define DSSD_TOPK_MIN_CTAS 2
#endif
#ifndef DSSD_TOPK_MERGE_AT
#define DSSD_TOPK_MERGE_AT 24
#endif
constexpr int kConsWarps = DSSD_TOPK_CONS_WARPS;      // consumer warps per CTA (a power of two, 4..16)
constexpr int kConsThreads = 32 * kConsWarps;
constexpr int kTkThreads = kConsThreads + 32;        // + the producer warp
constexpr int kStages = DSSD_TOPK_STAGES;            // ring stages per CTA
constexpr int kStageBytes = DSSD_TOPK_STAGE_BYTES;   // logits bytes per stage (one bulk copy)
constexpr int kStageVecs = kStageBytes / 16;         // 16-byte vectors per stage
constexpr int kU = kStageVecs / kConsThreads;        // vectors per consumer thread per stage
constexpr int kGroup = kConsThreads / 32;            // threads per group of the first threshold
static_assert(kU >= 1 && kU * kConsThreads == kStageVecs && kGroup >= 4 && kGroup <= 16, "stage / consumer shape");
constexpr int kCap = 512;                            // candidate buffer entries
constexpr int kMergeAt = DSSD_TOPK_MERGE_AT;         // merge once this many candidates wait
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
    __device__ static __forceinline__ void unpack(const uint4 &v, float *f)
    {
        f[0] = __uint_as_float(v.x), f[1] = __uint_as_float(v.y);
        f[2] = __uint_as_float(v.z), f[3] = __uint_as_float(v.w);
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
    __device__ static __forceinline__ void unpack(const uint4 &v, float *f)
    {
        f[0] = bf16_lo(v.x), f[1] = bf16_hi(v.x), f[2] = bf16_lo(v.y), f[3] = bf16_hi(v.y);
        f[4] = bf16_lo(v.z), f[5] = bf16_hi(v.z), f[6] = bf16_lo(v.w), f[7] = bf16_hi(v.w);
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

struct Smem {
    unsigned long long full[kStages];  // mbarriers: stage filled by the copy engine
    unsigned long long empty[kStages]; // mbarriers: stage read by all consumer warps
    unsigned long long list[2][32];    // the piece's current top-k, best first; two buffers, swapped by each merge
    unsigned long long cand[kCap + 8]; // candidates since the last merge (a vector reserved below kCap may end past it)
    float grp[32];                     // group maxima of the piece's first stage
    int n[2];                          // candidate slots reserved (runs past kCap on overflow)
    int nvalid[2];                     // first slot of the first refused reservation (INT_MAX: none)
    int bad;                           // the piece holds a NaN or +inf
    int fold_b;                        // sequence that this CTA completed and now folds (-1: none)
    int abort;                         // a bounded wait ran out
    int first_reject;                  // fold: first rejected position
    unsigned fl;                       // fold: flags of the sequence
    unsigned long long fold_keys[kConsWarps][kTopkMergeKeys];  // fold: one row's pieces, per warp
    unsigned long long fold_top[kConsWarps][32];               // fold: the row's top-k, best first
};

// barrier among the consumer warps only (the producer warp never joins)
__device__ __forceinline__ void cons_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kConsThreads) : "memory"); }

// the same barrier, returning to every consumer the number of them that passed a true predicate
__device__ __forceinline__ int cons_sync_count(bool pred)
{
    unsigned r;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.u32 p, %1, 0;\n\t"
        "bar.red.popc.u32 %0, 1, %2, p;\n\t}"
        : "=r"(r)
        : "r"((unsigned)pred), "n"(kConsThreads)
        : "memory");
    return (int)r;
}

constexpr int kNone = 0x7fffffff;

// One element of a piece's ragged ends (called before the first scan, when the buffer is empty)
__device__ __forceinline__ void offer(Smem &S, int nbuf, float f, int idx, unsigned long long taukey)
{
    if (f != f || f == INFINITY) {
        S.bad = 1;
        return;
    }
    const unsigned long long key = make_key(f, idx);
    if (key > taukey) S.cand[atomicAdd(&S.n[nbuf], 1)] = key;
}

// Where a warp stopped when the candidate buffer was full
struct Resume {
    int u;          // vector of the iteration (kU: the warp is done)
    unsigned hot;   // lanes of that vector still to be taken apart
};

// Scans the warp's kU x 32 vectors.  A vector whose maximum reaches tau is taken apart by the
// whole warp: its 16 bytes are broadcast and lane j judges element j, so a hit costs a few
// instructions instead of a divergent per-element loop; the slots of a vector are reserved with
// one shared-memory atomic.  Returns false when a reservation was refused (buffer full): `r`
// then tells where to resume after the merge.  `asked` grows by the slots the warp asked for.  vi0 = this lane's first vector within the
// piece's vector body, idx0 = vocabulary index of the body's first element.
template <int DT>
__device__ __forceinline__ bool scan(const uint4 (&a)[kU], Resume &r, bool resuming, int vi0, int nvec, int idx0,
                                     float tau, unsigned long long taukey, Smem &S, int nbuf, int &asked)
{
    constexpr int E = Vec<DT>::E;
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int u = 0; u < kU; ++u) {
        if (u < r.u) continue;
        const int vi = vi0 + u * kConsThreads;
        unsigned hot = __ballot_sync(kFullMask, vi < nvec && !(Vec<DT>::vmax(a[u]) < tau));
        if (resuming && u == r.u) hot = r.hot;
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
                    S.bad = 1;
                } else {
                    key = make_key(f, idx0 + (vi - lane + src) * E + lane);
                    want = key > taukey;
                }
            }
            const unsigned wm = __ballot_sync(kFullMask, want);
            if (wm) {
                asked += __popc(wm);
                int base = 0;
                if (lane == 0) base = atomicAdd(&S.n[nbuf], __popc(wm));
                base = __shfl_sync(kFullMask, base, 0);
                if (base >= kCap) {
                    if (lane == 0) atomicMin(&S.nvalid[nbuf], base);
                    r.u = u;
                    r.hot = hot;
                    return false;
                }
                if (want) S.cand[base + __popc(wm & ((1u << lane) - 1u))] = key;
            }
            hot &= hot - 1u;
        }
    }
    r.u = kU;
    return true;
}

// Merges n candidates with the current list by rank counting; the new list lands in the other
// buffer.  All keys involved are distinct.  One warp per key: the lanes compare 32 keys at a time
// with it and a ballot counts the larger ones, so there is no chain of dependent loads.  Called
// by all consumers; ends with their barrier.
__device__ __forceinline__ void merge(Smem &S, int cur, int nbuf, int n, int k)
{
    const int m = k + n, lane = threadIdx.x & 31;
    const unsigned long long *top = S.list[cur];
    unsigned long long *out = S.list[cur ^ 1];
    if (threadIdx.x == 0) {
        S.n[nbuf ^ 1] = 0;
        S.nvalid[nbuf ^ 1] = kNone;
    }
    for (int i = threadIdx.x >> 5; i < m; i += kConsWarps) {
        const unsigned long long x = i < k ? top[i] : S.cand[i - k];
        int rank = 0;
        for (int j0 = 0; j0 < m; j0 += 32) {
            const int j = j0 + lane;
            const unsigned long long y = j < k ? top[j] : (j < m ? S.cand[j - k] : 0ull);
            rank += __popc(__ballot_sync(kFullMask, y > x));
        }
        if (lane == 0 && rank < k) out[rank] = x;
    }
    cons_sync();
}

// State of a piece's scan that the iterations share
struct PieceState {
    int cur, nbuf;              // list / counter buffers in use
    float tau;                  // value of the threshold key
    unsigned long long taukey;  // a key must exceed this to be a candidate
    int pending;                // slots asked for since the last merge (the same in every consumer)
};

// One stage: scan the registers, meet, merge when worthwhile; repeats while the buffer overflows.
// Every decision that the consumers must take alike comes out of the barrier itself (the count
// of slots asked for, capped at 32 per warp, summed by the barrier) or is read from shared
// memory at a point where no consumer can be writing it, so that a fast warp that has moved on
// to the next stage never changes what a slow warp sees.  A refused reservation implies that
// at least kCap slots were asked for since the last merge, so it always falls in a merge round.
template <int DT>
__device__ __forceinline__ void iteration(const uint4 (&a)[kU], int vi0, int nvec, int idx0, bool last_it, int k,
                                          PieceState &st, Smem &S)
{
    const int lane = threadIdx.x & 31;
    Resume r;
    r.u = 0;
    r.hot = 0u;
    bool resuming = false;
    for (;;) {
        int asked = 0;
        resuming = !scan<DT>(a, r, resuming, vi0, nvec, idx0, st.tau, st.taukey, S, st.nbuf, asked);
        st.pending += cons_sync_count(lane < asked);
        if (st.pending < kMergeAt && !last_it) break;
        const int n_raw = S.n[st.nbuf], n_ok = S.nvalid[st.nbuf];
        const bool overflow = n_ok != kNone;
        merge(S, st.cur, st.nbuf, overflow ? n_ok : n_raw, k);
        st.cur ^= 1;
        st.nbuf ^= 1;
        st.pending = 0;
        const unsigned long long kth = S.list[st.cur][k - 1];
        if (kth > st.taukey) {
            st.taukey = kth;
            st.tau = key_value(kth);
        }
        if (!overflow) break;
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
    if (!mbar_wait(smem_addr(bar), parity, limit)) {
        *reinterpret_cast<volatile int *>(&S.abort) = 1;
        atomicExch(P.error, 1u);
    }
}

// The producer thread: streams the CTA's span, stage by stage, in the order the consumers read it.
template <int DT>
__device__ void producer(const TopkParams &P, Smem &S, uint32_t ring, unsigned long long blk, unsigned long long blk_end)
{
    unsigned q = 0;  // stages issued so far
    while (blk < blk_end) {
        const Piece pc = piece_at<DT>(P, blk, blk_end);
        for (int s = 0; s < pc.stages; ++s, ++q) {
            const unsigned slot = q % kStages, pass = q / kStages;
            if (pass > 0) ring_wait(P, S, &S.empty[slot], (pass - 1u) & 1u);
            const uint32_t bytes = (uint32_t)min(kStageVecs, pc.nvec - s * kStageVecs) * 16u;
            const uint32_t bar = smem_addr(&S.full[slot]);
            mbar_arrive_expect_tx(bar, bytes);
            bulk_g2s(ring + slot * (uint32_t)kStageBytes, pc.vp + (size_t)s * kStageVecs, bytes, bar);
        }
        blk += (unsigned long long)(pc.lb - pc.fb);
    }
}

// Top-k of one piece into S.list[returned buffer]; S.bad tells whether the piece held a NaN or
// +inf.  Called by all consumers, which have met at their barrier since they last touched S.
// `q` counts the stages consumed so far (the ring position), as the producer counts them.
template <int DT>
__device__ int piece_topk(const TopkParams &P, const Piece &pc, int k, Smem &S, uint32_t ring, unsigned &q)
{
    const int tid = threadIdx.x, lane = tid & 31;
    // empty slots hold distinct small keys (k - r in slot r), below every real key
    if (tid < 32) S.list[0][tid] = tid < k ? (unsigned long long)(k - tid) : 0ull;
    if (tid == 0) {
        S.n[0] = 0;
        S.n[1] = 0;
        S.nvalid[0] = kNone;
        S.nvalid[1] = kNone;
        S.bad = 0;
    }
    PieceState st;
    st.cur = 0;
    st.nbuf = 0;
    st.pending = 0;
    st.tau = -INFINITY;
    for (int s = 0; s < pc.stages; ++s, ++q) {
        const unsigned slot = q % kStages, pass = q / kStages;
        ring_wait(P, S, &S.full[slot], pass & 1u);
        uint4 a[kU];
        const int vi0 = s * kStageVecs + tid;
        const uint32_t src = ring + slot * (uint32_t)kStageBytes + (uint32_t)tid * 16u;
#pragma unroll
        for (int u = 0; u < kU; ++u)
            a[u] = vi0 + u * kConsThreads < pc.nvec ? lds16(src + (uint32_t)u * kConsThreads * 16u) : Vec<DT>::fill();
        if (s == 0) {
            // tau from the first stage: k-th largest of the 32 group maxima
            float tm = -INFINITY;
#pragma unroll
            for (int u = 0; u < kU; ++u) {
                const float v = Vec<DT>::vmax(a[u]);
                tm = fmaxf(tm, v == v ? v : -INFINITY);
            }
#pragma unroll
            for (int o = 1; o < kGroup; o <<= 1) tm = fmaxf(tm, __shfl_xor_sync(kFullMask, tm, o));
            if ((tid & (kGroup - 1)) == 0) S.grp[tid / kGroup] = tm;
            cons_sync();
            const float g = S.grp[lane];
            int rank = 0;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
                const float o = __shfl_sync(kFullMask, g, j);
                rank += (o > g) || (o == g && j < lane);
            }
            const unsigned hit = __ballot_sync(kFullMask, rank == k - 1);
            st.tau = __shfl_sync(kFullMask, g, __ffs(hit) - 1);
            st.taukey = (unsigned long long)ord(st.tau) << 32;
            // the ragged ends of the piece, one element per thread
            if (tid < pc.head) offer(S, 0, Vec<DT>::load(pc.rowp, pc.e0 + tid), pc.e0 + tid, st.taukey);
            if (tid >= 32 && tid - 32 < pc.e1 - pc.tail0)
                offer(S, 0, Vec<DT>::load(pc.rowp, pc.tail0 + tid - 32), pc.tail0 + tid - 32, st.taukey);
        }
        iteration<DT>(a, vi0, pc.nvec, pc.idx0, s + 1 == pc.stages, k, st, S);
        // the stage has been consumed from registers: hand the buffer back to the producer
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_addr(&S.empty[slot]));
    }
    if (pc.stages == 0) {  // only ragged elements
        cons_sync();
        st.taukey = 0ull;
        if (tid < pc.head) offer(S, 0, Vec<DT>::load(pc.rowp, pc.e0 + tid), pc.e0 + tid, st.taukey);
        if (tid >= 32 && tid - 32 < pc.e1 - pc.tail0)
            offer(S, 0, Vec<DT>::load(pc.rowp, pc.tail0 + tid - 32), pc.tail0 + tid - 32, st.taukey);
        cons_sync();
        merge(S, st.cur, st.nbuf, S.n[st.nbuf], k);
        st.cur ^= 1;
    }
    return st.cur;
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

// One warp: merges the pieces of `row`, then turns the k logits into probabilities (float64,
// summed in rank order).
__device__ RowDist row_dist(const TopkParams &P, int64_t row, unsigned long long *keys, unsigned long long *top)
{
    const int lane = threadIdx.x & 31, k = P.k;
    const unsigned long long first_blk = (unsigned long long)row * (unsigned long long)P.nb;
    const int pieces = (int)(owner_of(first_blk + P.nb - 1, P.grid, P.total_blocks) - owner_of(first_blk, P.grid, P.total_blocks)) + 1;
    const int m = pieces * k;
    const unsigned long long *src = P.lists + (size_t)row * P.max_pieces * k;
    bool bad = false;
    for (int i = lane; i < m; i += 32) {
        const unsigned long long x = __ldcg(src + i);
        bad |= (x == kBadList);
        keys[i] = x;
    }
    bad = __any_sync(kFullMask, bad);
    __syncwarp();
    RowDist d;
    d.idx = -1;
    d.prob = NAN;
    d.bad = bad;
    if (bad) return d;
    if (pieces == 1) {
        if (lane < k) top[lane] = keys[lane];
    } else {
        for (int i = lane; i < m; i += 32) {
            const unsigned long long x = keys[i];
            int rank = 0;
            for (int j = 0; j < m; ++j) rank += keys[j] > x;
            if (rank < k) top[rank] = x;  // keys below rank k include every empty slot
        }
    }
    __syncwarp();
    const unsigned long long key = lane < k ? top[lane] : 0ull;
    __syncwarp();
    const float val = key_value(key);
    const float best = __shfl_sync(kFullMask, val, 0);
    if (!(best > -INFINITY)) {  // nothing above -inf
        d.bad = true;
        return d;
    }
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

// The CTA that scanned a sequence's last block: acceptance tests, first rejection, row n's pairs.
// Called by all consumers.
__device__ __noinline__ void fold_sequence(const TopkParams &P, int b, Smem &S)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int gamma = P.gamma, k = P.k;
    if (tid == 0) {
        S.first_reject = gamma;
        S.fl = ld_relaxed_u32(P.error) ? DSSD_EDGE_FLAG_TIMEOUT : 0u;
    }
    cons_sync();
    for (int j = warp; j <= gamma; j += kConsWarps) {
        const RowDist d = row_dist(P, (int64_t)b * (gamma + 1) + j, S.fold_keys[warp], S.fold_top[warp]);
        if (d.bad && lane == 0) atomicOr(&S.fl, DSSD_EDGE_FLAG_NONFINITE);
        if (j == gamma) continue;
        const size_t o = (size_t)b * gamma + j;
        const int x = __ldg(P.draft_tokens + o);
        const unsigned holds = __ballot_sync(kFullMask, lane < k && !d.bad && d.idx == x);
        const double p_in = __shfl_sync(kFullMask, d.prob, holds ? __ffs(holds) - 1 : 0);
        if (lane == 0) {
            const double u = (double)__ldg(P.uniforms + o), q = (double)__ldg(P.draft_q_tok + o);
            double p;
            bool accept = false;
            if (x < 0 || x >= P.V) {
                atomicOr(&S.fl, DSSD_EDGE_FLAG_BAD_TOKEN);
                p = NAN;
            } else {
                p = d.bad ? NAN : (holds ? p_in : 0.0);
                double ratio;
                if (q != q || p != p) ratio = NAN;
                else if (q <= 0.0) ratio = p > 0.0 ? INFINITY : 0.0;
                else ratio = p / q;
                accept = (ratio == ratio) && (u < (ratio < 1.0 ? ratio : 1.0));
            }
            if (P.p_tok) P.p_tok[o] = (float)p;
            if (!accept) atomicMin(&S.first_reject, j);
        }
    }
    cons_sync();
    const int n = S.first_reject;
    if (warp == 0) {
        const RowDist d = row_dist(P, (int64_t)b * (gamma + 1) + n, S.fold_keys[0], S.fold_top[0]);
        if (lane < k) {
            P.p_idx[(size_t)b * k + lane] = d.bad ? -1 : d.idx;
            P.p_val[(size_t)b * k + lane] = d.bad ? NAN : (float)d.prob;
        }
        if (lane == 0) {
            P.accept_len[b] = n;
            if (P.flags) P.flags[b] = S.fl;
        }
    }
}

template <int DT>
__global__ void __launch_bounds__(kTkThreads, DSSD_TOPK_MIN_CTAS) topk_verify_kernel(const __grid_constant__ TopkParams P)
{
    extern __shared__ __align__(128) unsigned char smem_raw[];
    Smem &S = *reinterpret_cast<Smem *>(smem_raw + (size_t)kStages * kStageBytes);
    const uint32_t ring = smem_addr(smem_raw);
    const int tid = threadIdx.x, k = P.k;
    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_addr(&S.full[s]), 1u);
            mbar_init(smem_addr(&S.empty[s]), (uint32_t)kConsWarps);
        }
        S.abort = 0;
        mbar_init_fence();
    }
    __syncthreads();
    const unsigned long long G = (unsigned long long)P.grid, TB = P.total_blocks, c = blockIdx.x;
    const unsigned long long blk_end = (c + 1ull) * TB / G;
    unsigned long long blk = c * TB / G;
    if (tid >= kConsThreads) {
        if (tid == kConsThreads) producer<DT>(P, S, ring, blk, blk_end);
        return;
    }
    const unsigned long long per_seq = (unsigned long long)(P.gamma + 1) * (unsigned long long)P.nb;
    unsigned q = 0;
    // The sequence counter's answer is not waited for: thread 0 looks at it one piece later.
    unsigned long long prev_sum = 0ull;  // thread 0: counter value after the previous piece's blocks
    int prev_b = -1;
    while (blk < blk_end) {
        const Piece pc = piece_at<DT>(P, blk, blk_end);
        const int cur = piece_topk<DT>(P, pc, k, S, ring, q);
        const int b = (int)(pc.row / (P.gamma + 1));
        if (tid < 32) {
            // warp 0 publishes the piece: list, fence, then the blocks are counted
            const int slot = (int)(c - owner_of((unsigned long long)pc.row * P.nb, G, TB));
            if (tid < k) {
                unsigned long long key = S.list[cur][tid];
                if (S.bad) key = tid == 0 ? kBadList : 0ull;
                __stcg(P.lists + ((size_t)pc.row * P.max_pieces + slot) * k + tid, key);
            }
            __threadfence();
            __syncwarp();
            if (tid == 0) {
                S.fold_b = (prev_b >= 0 && prev_sum == per_seq) ? prev_b : -1;
                const unsigned long long done = (unsigned long long)(pc.lb - pc.fb);
                prev_sum = atomicAdd(P.seq_done + b, done) + done;
                prev_b = b;
            }
        }
        cons_sync();
        const int fb = S.fold_b;
        if (fb >= 0) {
            __threadfence();
            fold_sequence(P, fb, S);
            cons_sync();
        }
        blk += (unsigned long long)(pc.lb - pc.fb);
    }
    if (tid == 0) S.fold_b = (prev_b >= 0 && prev_sum == per_seq) ? prev_b : -1;
    cons_sync();
    if (S.fold_b >= 0) {
        __threadfence();
        fold_sequence(P, S.fold_b, S);
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
    const size_t cnt = (8 + (size_t)B * 8 + 255) & ~(size_t)255;
    const size_t lists = rows * (size_t)topk_max_pieces(k) * (size_t)k * 8;
    if (P) {
        P->error = reinterpret_cast<unsigned *>(base);
        P->seq_done = reinterpret_cast<unsigned long long *>(base + 8);
        P->lists = reinterpret_cast<unsigned long long *>(base + cnt);
        P->zero_bytes = 8 + (size_t)B * 8;
        P->max_pieces = topk_max_pieces(k);
    }
    return cnt + ((lists + 255) & ~(size_t)255);
}

static int g_topk_ctas[64];  // CTAs resident on the device at once (0 = not asked yet)
constexpr size_t kTopkSmemBytes = (size_t)kStages * kStageBytes + sizeof(Smem);

cudaError_t topk_verify_launch(TopkParams &P, int dtype, void *workspace, cudaStream_t stream)
{
    cudaError_t err;
    int dev = 0;
    if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
    int ctas = (dev >= 0 && dev < 64) ? g_topk_ctas[dev] : 0;
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
        if (dev >= 0 && dev < 64) g_topk_ctas[dev] = ctas;
    }
    topk_workspace_layout(P.B, P.gamma, P.k, &P, static_cast<char *>(workspace));
    const unsigned long long rows = (unsigned long long)P.B * (unsigned long long)(P.gamma + 1);
    P.nb = (P.V + kTopkBlock - 1) / kTopkBlock;
    P.total_blocks = rows * (unsigned long long)P.nb;
    // every span must hold at least ceil(nb / (max_pieces - 1)) blocks, so that no row is shared
    // by more than max_pieces CTAs
    const unsigned long long wmin = ((unsigned long long)P.nb + P.max_pieces - 2) / (unsigned long long)(P.max_pieces - 1);
    unsigned long long grid = P.total_blocks / wmin;
    if (grid > (unsigned long long)ctas) grid = (unsigned long long)ctas;
    if (grid < 1) grid = 1;
    P.grid = (int)grid;
    if ((err = cudaMemsetAsync(P.error, 0, P.zero_bytes, stream)) != cudaSuccess) return err;
    if (dtype == DSSD_BF16)
        topk_verify_kernel<DSSD_BF16><<<P.grid, kTkThreads, kTopkSmemBytes, stream>>>(P);
    else
        topk_verify_kernel<DSSD_F32><<<P.grid, kTkThreads, kTopkSmemBytes, stream>>>(P);
    return cudaGetLastError();
}

cudaError_t topk_resample_launch(const TopkResampleParams &P, cudaStream_t stream)
{
    const int grid = (P.B + kWarps - 1) / kWarps;
    topk_resample_kernel<<<grid, kThreads, 0, stream>>>(P);
    return cudaGetLastError();
}

}  // namespace dssd
