// The vocabulary-sharded round: what happens between and after the shards' partial sums.
//
// Every shard runs the streaming edge kernel on its slice of the logits in "partial" mode and
// gets, per row, sum_v 2^(l_v c1) = part_sum * 2^part_ref over its slice, plus the logits of the
// drafted tokens it holds.  Once these small arrays have been exchanged (an all-gather of a few
// bytes per row), shard_combine_kernel - one warp per sequence, one lane per position - adds the
// shards' sums by exact power-of-two rescaling and evaluates the acceptance test and the
// first-rejection scan with the same arithmetic as the dense kernel's fold.  shard_emit_kernel
// then writes this shard's slice of row P_n.
#include "shard_verify.h"

#include <atomic>

#include "dssd_device.cuh"
#include "edge_judge.cuh"

namespace dssd {

namespace {

constexpr unsigned kFull = 0xffffffffu;

__global__ void __launch_bounds__(kThreads) shard_combine_kernel(const __grid_constant__ CombineParams P)
{
    const int lane = threadIdx.x & 31;
    const long long b = (long long)blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (b >= P.B) return;
    const size_t rows = (size_t)P.B * (size_t)(P.gamma + 1), toks = (size_t)P.B * (size_t)P.gamma;
    int n = P.gamma;
    unsigned fl = 0;
    float ref2_n = 0.f, invS_n = 0.f;
    for (int base = 0; base <= P.gamma; base += 32) {
        const int i = base + lane;
        const bool live = i <= P.gamma;
        const size_t row = (size_t)b * (size_t)(P.gamma + 1) + (size_t)(live ? i : 0);
        int x = -1;
        float zx = __int_as_float(0x7fc00000), qx = 0.f, ux = 0.f;
        if (live && i < P.gamma) {
            const size_t di = (size_t)b * P.gamma + i;
            x = P.draft_tokens[di];
            qx = P.draft_q_tok[di];
            ux = P.uniforms[di];
            // the one shard that holds x reports its logit, the others NaN
            for (int g = 0; g < P.G; ++g) {
                const float z = __ldg(P.tok_logit + (size_t)g * toks + di);
                if (z == z) zx = z;
            }
        }
        float Rr = DSSD_NEG_INF;
        double S = 0.0;
        bool bad = false;
        if (live) {
            for (int g = 0; g < P.G; ++g)  // shard order
                add_partial(Rr, S, bad, __ldg(P.part_ref + (size_t)g * rows + row), __ldg(P.part_sum + (size_t)g * rows + row));
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
        P.row_scale[2 * b] = ref2_n;
        P.row_scale[2 * b + 1] = invS_n;
    }
}

// p_row[b, v] = 2^(l_{b,n,v} c1 - ref2) / S over this shard's slice of row n.  Work is cut into
// tiles of kTile entries handed out round robin; 16-byte loads and stores where the row's body
// and its output are aligned, element-wise otherwise (a slice may start anywhere in a row).
constexpr int kTile = 8192;

template <int DT>
__global__ void __launch_bounds__(kThreads) shard_emit_kernel(const __grid_constant__ EmitShardParams P)
{
    using E = Elem<DT>;
    const int tiles_per_row = (P.V + kTile - 1) / kTile;
    const long long total = (long long)P.B * tiles_per_row;
    for (long long t = blockIdx.x; t < total; t += gridDim.x) {
        const long long b = t / tiles_per_row;
        const int tile = (int)(t - b * tiles_per_row);
        const int n = P.accept_len[b];
        if (n < 0 || n > P.gamma) continue;
        const float nref = -P.row_scale[2 * b], invS = P.row_scale[2 * b + 1];
        const char *rowp = static_cast<const char *>(P.logits) +
                           ((size_t)b * (size_t)(P.gamma + 1) + (size_t)n) * (size_t)P.row_stride * E::kBytes;
        float *outp = P.p_row + (size_t)b * (size_t)P.p_stride;
        // the row's body starts at its first 16-byte boundary, `head` entries in
        const int head_bytes = (int)((16u - (unsigned)(reinterpret_cast<uintptr_t>(rowp) & 15u)) & 15u);
        int head = head_bytes / E::kBytes;
        if (head > P.V) head = P.V;
        const int nvec = (P.V - head) / E::kVec;
        const int e0 = tile * kTile, e1 = min(P.V, e0 + kTile);
        const bool vec_out = (reinterpret_cast<uintptr_t>(outp + head) & 15u) == 0;
        // vectors of the body that lie wholly inside this tile
        const int j0 = e0 <= head ? 0 : (e0 - head + E::kVec - 1) / E::kVec;
        const int j1 = min(nvec, e1 <= head ? 0 : (e1 - head) / E::kVec);
        const f32x2 cc = pack2(P.c1, P.c1), nn = pack2(nref, nref), ss = pack2(invS, invS);
        for (int j = j0 + (int)threadIdx.x; j < j1; j += kThreads) {
            float f[E::kVec];
            E::unpack(ld_stream16(rowp + (size_t)head * E::kBytes + (size_t)j * 16), f);
            float *o = outp + head + (size_t)j * E::kVec;
#pragma unroll
            for (int q = 0; q < E::kVec; q += 4) {
                float a, b2, c, d;
                unpack2(fma2(pack2(f[q], f[q + 1]), cc, nn), a, b2);
                unpack2(fma2(pack2(f[q + 2], f[q + 3]), cc, nn), c, d);
                unpack2(mul2(pack2(ex2(a), ex2(b2)), ss), a, b2);
                unpack2(mul2(pack2(ex2(c), ex2(d)), ss), c, d);
                if (vec_out) {
                    st_stream16(o + q, a, b2, c, d);
                } else {
                    o[q] = a, o[q + 1] = b2, o[q + 2] = c, o[q + 3] = d;
                }
            }
        }
        // entries of the tile outside those vectors: the row's head, its tail, and the ends of a
        // tile that cuts a vector (at most a few per tile)
        const int v_lo = head + j0 * E::kVec, v_hi = head + (j1 > j0 ? j1 : j0) * E::kVec;
        for (int e = e0 + (int)threadIdx.x; e < min(e1, v_lo); e += kThreads)
            outp[e] = ex2(fmaf(E::load(rowp, e), P.c1, nref)) * invS;
        for (int e = max(e0, v_hi) + (int)threadIdx.x; e < e1; e += kThreads)
            outp[e] = ex2(fmaf(E::load(rowp, e), P.c1, nref)) * invS;
    }
}

std::atomic<int> g_emit_ctas[64];  // resident CTAs of the emission kernel per device (0: not asked yet)

}  // namespace

cudaError_t shard_combine_launch(const CombineParams &P, cudaStream_t stream)
{
    const unsigned grid = (unsigned)((P.B + kWarps - 1) / kWarps);
    shard_combine_kernel<<<grid, kThreads, 0, stream>>>(P);
    return cudaGetLastError();
}

cudaError_t shard_emit_launch(const EmitShardParams &P, int dtype, cudaStream_t stream)
{
    cudaError_t err;
    int dev = 0;
    if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
    int ctas = (dev >= 0 && dev < 64) ? g_emit_ctas[dev].load(std::memory_order_acquire) : 0;
    if (ctas == 0) {
        int sms = 0, occ0 = 0, occ1 = 0;
        if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ0, shard_emit_kernel<DSSD_F32>, kThreads, 0)) != cudaSuccess) return err;
        if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ1, shard_emit_kernel<DSSD_BF16>, kThreads, 0)) != cudaSuccess) return err;
        const int occ = occ0 < occ1 ? occ0 : occ1;
        ctas = (sms < 1 ? 1 : sms) * (occ < 1 ? 1 : occ);
        if (dev >= 0 && dev < 64) g_emit_ctas[dev].store(ctas, std::memory_order_release);
    }
    const long long total = (long long)P.B * ((P.V + kTile - 1) / kTile);
    const unsigned grid = (unsigned)(total < ctas ? total : ctas);
    if (dtype == DSSD_BF16) shard_emit_kernel<DSSD_BF16><<<grid, kThreads, 0, stream>>>(P);
    else shard_emit_kernel<DSSD_F32><<<grid, kThreads, 0, stream>>>(P);
    return cudaGetLastError();
}

}  // namespace dssd
