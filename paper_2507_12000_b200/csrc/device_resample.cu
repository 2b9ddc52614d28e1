// Device half of the verification round: residual (or bonus) inverse-CDF draw.
//
// Pass A, ticket (b, c): stream chunk c of p_row[b] and of Q_n[b], form r = max(0, p - q) (or
// r = p for the bonus draw) and add it up in float64 -> chunk_sum[b, c].
// Pass B, run by the CTA that completes the last chunk of sequence b: prefix over the chunk sums
// gives Z and the chunk holding u' * Z; that one chunk is read again (from L2), a block-wide
// prefix sum over per-thread runs finds the thread, and the thread walks its run.
// All sums are float64, so the token differs from an index-order float64 scan only when u' * Z
// lies within rounding (about 1e-13 relative) of a CDF step.
#include "device_resample.h"

#include <mutex>

#include <math.h>

#include "dssd_device.cuh"

namespace dssd {

namespace {

constexpr int kRun = kResampleChunk / kThreads;  // contiguous entries per thread in pass B

__device__ __forceinline__ double res(float p, float q) { return fmax(0.0, (double)p - (double)q); }

__device__ __forceinline__ float4 as_f4(const uint4 &v)
{
    return make_float4(__uint_as_float(v.x), __uint_as_float(v.y), __uint_as_float(v.z), __uint_as_float(v.w));
}

// per-thread part of sum_{e in [e0,e1)} r_e ; q == nullptr means r = p
__device__ __forceinline__ double chunk_mass(const float *p, const float *q, int e0, int e1)
{
    const int tid = threadIdx.x;
    double acc = 0.0;
    int done = e0;
    const bool aligned =
        ((reinterpret_cast<uintptr_t>(p + e0) | (q ? reinterpret_cast<uintptr_t>(q + e0) : 0)) & 15u) == 0;
    if (aligned) {
        const int nvec = (e1 - e0) / 4;
        const uint4 *p4 = reinterpret_cast<const uint4 *>(p + e0);
        if (q) {
            const uint4 *q4 = reinterpret_cast<const uint4 *>(q + e0);
            int i = tid;
            for (; i + 3 * kThreads < nvec; i += 4 * kThreads) {
                uint4 a[4], b[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    a[u] = ld_stream16(p4 + i + u * kThreads);
                    b[u] = ld_stream16(q4 + i + u * kThreads);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float4 x = as_f4(a[u]), y = as_f4(b[u]);
                    acc += (res(x.x, y.x) + res(x.y, y.y)) + (res(x.z, y.z) + res(x.w, y.w));
                }
            }
            for (; i < nvec; i += kThreads) {
                const float4 x = as_f4(ld_stream16(p4 + i)), y = as_f4(ld_stream16(q4 + i));
                acc += (res(x.x, y.x) + res(x.y, y.y)) + (res(x.z, y.z) + res(x.w, y.w));
            }
        } else {
            int i = tid;
            for (; i + 3 * kThreads < nvec; i += 4 * kThreads) {
                uint4 a[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) a[u] = ld_stream16(p4 + i + u * kThreads);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const float4 x = as_f4(a[u]);
                    acc += ((double)x.x + (double)x.y) + ((double)x.z + (double)x.w);
                }
            }
            for (; i < nvec; i += kThreads) {
                const float4 x = as_f4(ld_stream16(p4 + i));
                acc += ((double)x.x + (double)x.y) + ((double)x.z + (double)x.w);
            }
        }
        done = e0 + nvec * 4;
    }
    for (int e = done + tid; e < e1; e += kThreads) acc += q ? res(__ldg(p + e), __ldg(q + e)) : (double)__ldg(p + e);
    return acc;
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

// pass B for sequence b; q == nullptr means r = p
__device__ void draw(const ResampleParams &P, int64_t b, const float *p, const float *q, unsigned fl,
                     double *s_w, Pick *s_pick, int *s_i)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    double *cs = P.chunk_sum + (size_t)b * P.n_chunks;
    for (int attempt = 0; attempt < 2; ++attempt) {
        if (tid == 0) {
            double Z = 0.0;
            for (int c = 0; c < P.n_chunks; ++c) Z += __ldcg(cs + c);
            Pick pk;
            pk.ok = (Z > 0.0) && (Z < INFINITY);
            pk.chunk = 0;
            pk.beyond = 1;
            pk.base = 0.0;
            pk.target = (double)__ldg(P.uniforms + b) * Z;
            if (pk.ok) {
                double C = 0.0;
                int last_pos = 0;
                double last_base = 0.0;
                for (int c = 0; c < P.n_chunks; ++c) {
                    const double m = __ldcg(cs + c);
                    if (m > 0.0) { last_pos = c; last_base = C; }
                    if (C + m > pk.target) { pk.chunk = c; pk.base = C; pk.beyond = 0; break; }
                    C += m;
                }
                if (pk.beyond) { pk.chunk = last_pos; pk.base = last_base; }
            }
            *s_pick = pk;
        }
        __syncthreads();
        if (s_pick->ok) break;
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
        for (int c = 0; c < P.n_chunks; ++c) {
            const int e0 = c * kResampleChunk, e1 = min(P.V, e0 + kResampleChunk);
            const double tot = block_sum(chunk_mass(p, nullptr, e0, e1), s_w);
            if (tid == 0) cs[c] = tot;
        }
        __threadfence();
        __syncthreads();
    }
    const Pick pk = *s_pick;
    const int e0 = pk.chunk * kResampleChunk, e1 = min(P.V, e0 + kResampleChunk);
    const int r0 = min(e1, e0 + tid * kRun), r1 = min(e1, r0 + kRun);
    double mine = 0.0;
    int last_pos = -1;
    for (int e = r0; e < r1; ++e) {
        const double r = q ? res(__ldg(p + e), __ldg(q + e)) : (double)__ldg(p + e);
        mine += r;
        if (r > 0.0) last_pos = e;
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
            P.token[b] = s_i[1];
            if (P.flags) P.flags[b] = fl | (s_i[1] < 0 ? DSSD_RS_FLAG_INVALID : 0u);
        }
    } else if (tid == first) {
        double C = before;
        int tok = last_pos;
        for (int e = r0; e < r1; ++e) {
            C += q ? res(__ldg(p + e), __ldg(q + e)) : (double)__ldg(p + e);
            if (C > pk.target) { tok = e; break; }
        }
        P.token[b] = tok >= 0 ? tok : s_i[1];
        if (P.flags) P.flags[b] = fl;
    }
}

__global__ void __launch_bounds__(kThreads, 4) resample_kernel(const ResampleParams P)
{
    __shared__ double s_w[kWarps];
    __shared__ Pick s_pick;
    __shared__ int s_i[2];
    __shared__ int s_last;
    __shared__ unsigned long long s_ticket;
    const int tid = threadIdx.x;
    if (tid == 0) s_ticket = atomicAdd(P.ticket, 1ull);
    __syncthreads();
    unsigned long long t = s_ticket;
    while (t < P.total_tickets) {
        __syncthreads();
        unsigned long long nxt = 0;
        if (tid == 0) nxt = atomicAdd(P.ticket, 1ull);
        const int64_t b = (int64_t)(t / (unsigned)P.n_chunks);
        const int c = (int)(t - (unsigned long long)b * (unsigned)P.n_chunks);
        const int n = __ldg(P.accept_len + b);
        const bool valid = n >= 0 && n <= P.gamma;
        const float *p = P.p_row + (size_t)b * P.V;
        const float *q = (valid && n < P.gamma) ? P.draft_q + ((size_t)b * P.gamma + n) * (size_t)P.V : nullptr;
        const int e0 = c * kResampleChunk, e1 = min(P.V, e0 + kResampleChunk);
        const double tot = block_sum(valid ? chunk_mass(p, q, e0, e1) : 0.0, s_w);
        if (tid == 0) {
            P.chunk_sum[(size_t)b * P.n_chunks + c] = tot;
            __threadfence();
            s_last = (atomicAdd(&P.seq_cnt[b], 1u) == (unsigned)(P.n_chunks - 1));
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            if (!valid) {
                if (tid == 0) {
                    P.token[b] = -1;
                    if (P.flags) P.flags[b] = DSSD_RS_FLAG_INVALID;
                }
            } else {
                draw(P, b, p, q, q ? 0u : DSSD_RS_FLAG_BONUS, s_w, &s_pick, s_i);
            }
        }
        if (tid == 0) s_ticket = nxt;
        __syncthreads();
        t = s_ticket;
    }
}

}  // namespace

size_t resample_workspace_layout(int B, int V, ResampleParams *P, char *base)
{
    const int n_chunks = (V + kResampleChunk - 1) / kResampleChunk;
    size_t off = 0;
    auto take = [&](size_t bytes) {
        size_t o = off;
        off += (bytes + 255) & ~(size_t)255;
        return o;
    };
    const size_t o_ticket = take(16);
    const size_t o_cnt = take((size_t)B * 4);
    const size_t zero_bytes = off;
    const size_t o_sum = take((size_t)B * (size_t)n_chunks * sizeof(double));
    if (P) {
        P->ticket = reinterpret_cast<unsigned long long *>(base + o_ticket);
        P->seq_cnt = reinterpret_cast<unsigned *>(base + o_cnt);
        P->chunk_sum = reinterpret_cast<double *>(base + o_sum);
        P->zero_bytes = zero_bytes;
        P->n_chunks = n_chunks;
        P->total_tickets = (unsigned long long)B * (unsigned long long)n_chunks;
    }
    return off;
}

cudaError_t resample_launch(ResampleParams &P, void *workspace, cudaStream_t stream)
{
    cudaError_t err;
    int dev = 0, sms = 0, occ = 0;
    if ((err = cudaGetDevice(&dev)) != cudaSuccess) return err;
    if ((err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return err;
    if ((err = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, resample_kernel, kThreads, 0)) != cudaSuccess) return err;
    if (occ < 1) occ = 1;
    resample_workspace_layout(P.B, P.V, &P, static_cast<char *>(workspace));
    if ((err = cudaMemsetAsync(workspace, 0, P.zero_bytes, stream)) != cudaSuccess) return err;
    const unsigned long long resident = (unsigned long long)sms * (unsigned long long)occ;
    const unsigned grid = (unsigned)(P.total_tickets < resident ? P.total_tickets : resident);
    resample_kernel<<<grid, kThreads, 0, stream>>>(P);
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
            if ((e = cudaGetSymbolAddress(&ptr, g_static_scratch)) != cudaSuccess || !ptr) {
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
    // resample_launch clears the counters that must start at zero; the rest of the scratch is
    // written before it is read, so what the previous call left behind does not matter
    e = dssd::resample_launch(P, scratch, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) {
        dssd::set_last_cuda_error((int)e);
        return DSSD_ERR_CUDA;
    }
    return DSSD_OK;
}
