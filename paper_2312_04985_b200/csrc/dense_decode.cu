// dense_decode: dense single-token decode attention, Eq. (2), the comparison kernel for the
// speed-up figure.  One CTA per (split, KV head, batch): a CTA covers one slice of the sequence of one KV head
// for all (up to 8 at a time) query heads of its group, so K and V are read once per KV head;
// half-warp per cache row, 128-bit loads, online softmax in fp32.  With more than one split the
// per-split softmax states go through a scratch buffer and a small merge kernel.
#include <mutex>

#include "common.cuh"
#include "kernels.h"

namespace sparq {
namespace {

// Scratch of dense_decode_static: lives in the library's device image, so every GPU that loads the
// library carries these 8 MiB until the process exits, and every call on a device shares them.
constexpr size_t kStaticScratchBytes = SPARQ_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_dense_scratch[kStaticScratchBytes];
constexpr int kMaxDevices = 64;
float* g_dense_scratch_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal
std::mutex g_dense_scratch_mutex;

constexpr int NT = 256;             // threads per CTA
constexpr int NHW = NT / 16;        // half-warps per CTA (one K/V row each)

// One CTA per (split, KV head, batch).  A CTA covers positions [split*chunk, (split+1)*chunk) of one KV head
// for all G query heads of the group; half-warp per cache row, online softmax in fp32.
template <int G>
__global__ void __launch_bounds__(NT)
dense_decode_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                    const sparq_half* __restrict__ V, const int32_t* __restrict__ seq_lens,
                    int Hq, int Hkv, int S_max, int g_total, int g_base, int splits,
                    sparq_half* __restrict__ out, float* __restrict__ ws, int32_t* status) {
    __shared__ float merge[NHW * (D + 2)];
    const int tid = threadIdx.x, hw = tid >> 4, l16 = tid & 15;
    // one-dimensional grid: split fastest, then KV head, then batch (no 65535 limit on the batch)
    const int split = (int)(blockIdx.x % (unsigned)splits);
    const int hkv = (int)((blockIdx.x / (unsigned)splits) % (unsigned)Hkv), b = (int)(blockIdx.x / ((unsigned)splits * (unsigned)Hkv));
    const int n = seq_lens[b];
    const int h0 = hkv * g_total + g_base;                    // first query head served here
    if (n < 1 || n > S_max) {
        if (split == 0) {
            if (tid == 0) raise_status(status, SPARQ_DEV_BAD_SEQ_LEN);
            for (int i = tid; i < G * D; i += NT) out[((size_t)b * Hq + h0 + i / D) * D + (i % D)] = 0;
        }
        return;                                               // merge kernel skips this sequence too
    }
    int chunk = (n + splits - 1) / splits;
    chunk = (chunk + 15) & ~15;
    const int t_begin = split * chunk, t_end = min(n, t_begin + chunk);

    const float qscale = rsqrtf((float)D) * LOG2E;
    // this lane's 8 query components per head, as stored (fp16): q . k is a chain of mixed-precision
    // FMAs on exact fp16 x fp16 products, scaled once at the end
    uint32_t qw[G][4];
    float acc[G][8], m[G], l[G];
#pragma unroll
    for (int gi = 0; gi < G; ++gi) {
        m[gi] = -CUDART_INF_F; l[gi] = 0.f;
        const uint4 q8 = *reinterpret_cast<const uint4*>(q + ((size_t)b * Hq + h0 + gi) * D + l16 * 8);
        qw[gi][0] = q8.x; qw[gi][1] = q8.y; qw[gi][2] = q8.z; qw[gi][3] = q8.w;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[gi][e] = 0.f;
    }
    const size_t kv_head = (size_t)b * Hkv + hkv;
    const uint4* Kh = reinterpret_cast<const uint4*>(K + kv_head * (size_t)S_max * D);
    const uint4* Vh = reinterpret_cast<const uint4*>(V + kv_head * (size_t)S_max * D);
    constexpr int RG = 4;
    for (int tb = t_begin; tb < t_end; tb += NHW * RG) {      // trip count uniform across the CTA
        const int t0 = tb + hw;
        uint4 kv[RG], vv[RG];
#pragma unroll
        for (int u = 0; u < RG; ++u) {
            int t = min(t0 + u * NHW, t_end - 1);
            kv[u] = ld_stream(Kh + (size_t)t * (D / 8) + l16);
            vv[u] = ld_stream(Vh + (size_t)t * (D / 8) + l16);
        }
#pragma unroll
        for (int gi = 0; gi < G; ++gi) {
            // the RG rows' logits for this head, then ONE rescale of the running state per batch of rows
            float z[RG], bmax = -CUDART_INF_F;
#pragma unroll
            for (int u = 0; u < RG; ++u) {
                const uint32_t kw[4] = {kv[u].x, kv[u].y, kv[u].z, kv[u].w};
                float za = 0.f, zb = 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(za) : "h"((uint16_t)(kw[e] & 0xffffu)), "h"((uint16_t)(qw[gi][e] & 0xffffu)));
                    asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(zb) : "h"((uint16_t)(kw[e] >> 16)), "h"((uint16_t)(qw[gi][e] >> 16)));
                }
                float zz = (za + zb) * qscale;
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) zz += __shfl_xor_sync(FULL, zz, o);
                z[u] = (t0 + u * NHW < t_end) ? zz : -CUDART_INF_F;        // uniform within the half-warp
                bmax = fmaxf(bmax, z[u]);
            }
            const float mn = fmaxf(m[gi], bmax);
            if (mn > -CUDART_INF_F) {
                const float sc = exp2f(m[gi] - mn);
                float lsum = l[gi] * sc;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[gi][e] *= sc;
#pragma unroll
                for (int u = 0; u < RG; ++u) {
                    const float p = exp2f(z[u] - mn);
                    lsum += p;
                    const __half2* vh = reinterpret_cast<const __half2*>(&vv[u]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 w = __half22float2(vh[e]);
                        acc[gi][2 * e] = fmaf(p, w.x, acc[gi][2 * e]);
                        acc[gi][2 * e + 1] = fmaf(p, w.y, acc[gi][2 * e + 1]);
                    }
                }
                l[gi] = lsum;
                m[gi] = mn;
            }
        }
    }
    // merge the CTA's half-warps, one query head at a time
#pragma unroll
    for (int gi = 0; gi < G; ++gi) {
        __syncthreads();
        float* mg = merge + hw * (D + 2);
#pragma unroll
        for (int e = 0; e < 8; ++e) mg[l16 * 8 + e] = acc[gi][e];
        if (l16 == 0) { mg[D] = m[gi]; mg[D + 1] = l[gi]; }
        __syncthreads();
        if (tid < D) {
            float M = -CUDART_INF_F;
#pragma unroll
            for (int w = 0; w < NHW; ++w) M = fmaxf(M, merge[w * (D + 2) + D]);
            float L = 0.f, s = 0.f;
            if (M > -CUDART_INF_F) {
#pragma unroll
                for (int w = 0; w < NHW; ++w) {
                    float sc = exp2f(merge[w * (D + 2) + D] - M);
                    L = fmaf(merge[w * (D + 2) + D + 1], sc, L);
                    s = fmaf(merge[w * (D + 2) + tid], sc, s);
                }
            }
            const size_t bhq = (size_t)b * Hq + h0 + gi;
            if (splits == 1) {
                out[bhq * D + tid] = __half_as_ushort(__float2half_rn(s / L));
            } else {
                float* p = ws + (bhq * splits + split) * (D + 2);
                p[tid] = s;
                if (tid == 0) { p[D] = M; p[D + 1] = L; }
            }
        }
    }
}

// grid B*Hq, D threads: combine the per-split partial states.
__global__ void __launch_bounds__(D)
dense_merge_kernel(const float* __restrict__ ws, const int32_t* __restrict__ seq_lens, int Hq, int S_max,
                   int splits, sparq_half* __restrict__ out) {
    const int bh = blockIdx.x, tid = threadIdx.x;
    const int n = seq_lens[bh / Hq];
    if (n < 1 || n > S_max) return;                           // already zeroed by the main kernel
    const float* p = ws + (size_t)bh * splits * (D + 2);
    float M = -CUDART_INF_F;
    for (int s = 0; s < splits; ++s) M = fmaxf(M, p[s * (D + 2) + D]);
    float L = 0.f, y = 0.f;
    for (int s = 0; s < splits; ++s) {
        float ms = p[s * (D + 2) + D];
        if (ms > -CUDART_INF_F) {                             // empty splits carry m = -inf, l = 0
            float sc = exp2f(ms - M);
            L = fmaf(p[s * (D + 2) + D + 1], sc, L);
            y = fmaf(p[s * (D + 2) + tid], sc, y);
        }
    }
    out[(size_t)bh * D + tid] = __half_as_ushort(__float2half_rn(y / L));
}

}  // namespace

int dense_splits(int B, int Hkv, int S_max) {
    long ctas = (long)B * Hkv;
    long want = (4L * 148 + ctas - 1) / ctas;                 // aim for >= 4 CTAs per SM
    long cap = (S_max + 255) / 256;                           // at least 256 positions per split
    long s = want < cap ? want : cap;
    return (int)(s < 1 ? 1 : s);
}

size_t dense_scratch_bytes(int B, int Hq, int Hkv, int S_max) {
    int splits = dense_splits(B, Hkv, S_max);
    return splits == 1 ? 0 : (size_t)B * Hq * splits * (D + 2) * sizeof(float);
}

// Device address of the static scratch on the current device.  In host code the array's name is only
// a handle of the symbol, not an address a kernel could use: the address comes from the runtime, once
// per device, with that device current.
cudaError_t dense_static_scratch(float** ptr, size_t* bytes) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_dense_scratch_mutex);
    if (!g_dense_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_dense_scratch);
        if (e != cudaSuccess) return e;
        g_dense_scratch_ptr[dev] = static_cast<float*>(p);
    }
    *ptr = g_dense_scratch_ptr[dev];
    *bytes = kStaticScratchBytes;
    return cudaSuccess;
}

cudaError_t launch_dense_decode(const sparq_half* q, const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                                int B, int Hq, int Hkv, int S_max, sparq_half* out, float* ws, int32_t* status,
                                cudaStream_t st) {
    const int splits = dense_splits(B, Hkv, S_max);
    const int g = Hq / Hkv;
    const unsigned grid = (unsigned)splits * (unsigned)Hkv * (unsigned)B;
    // the group's query heads are served G at a time by one pass over K and V
    for (int g_base = 0; g_base < g;) {
        int left = g - g_base;
        if (left >= 8) { dense_decode_kernel<8><<<grid, NT, 0, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status); g_base += 8; }
        else if (left >= 4) { dense_decode_kernel<4><<<grid, NT, 0, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status); g_base += 4; }
        else if (left >= 2) { dense_decode_kernel<2><<<grid, NT, 0, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status); g_base += 2; }
        else { dense_decode_kernel<1><<<grid, NT, 0, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status); g_base += 1; }
    }
    if (splits > 1) dense_merge_kernel<<<B * Hq, D, 0, st>>>(ws, seq_lens, Hq, S_max, splits, out);
    return cudaGetLastError();
}

}  // namespace sparq
