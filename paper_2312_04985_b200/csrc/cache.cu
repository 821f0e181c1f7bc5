// Cache maintenance: the per-step append (K, Kt, V, running value sum and mean) and the
// prefill-side builder that derives Kt and v_bar from a filled K, V.
#include "common.cuh"
#include "kernels.h"

namespace sparq {
namespace {

// One CTA per sequence, one warp per KV head (warps stride over the heads when there are more than
// 32 of them); lane l owns components 4l .. 4l+3 of the new token.  Every thread reads the old
// length before the CTA-wide barrier and thread 0 stores the new one after it, so the whole append
// is one launch.
__global__ void __launch_bounds__(1024)
cache_append_kernel(const sparq_half* __restrict__ k_new, const sparq_half* __restrict__ v_new,
                    sparq_half* __restrict__ K, sparq_half* __restrict__ Kt, sparq_half* __restrict__ V,
                    float* __restrict__ vsum, sparq_half* __restrict__ vbar,
                    int32_t* __restrict__ seq_lens, int Hkv, int S_max, int32_t* status) {
    static_assert(D == 128, "one warp covers a token: 32 lanes x 4 components");
    const int b = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
    const int c0 = lane * 4;
    const int n = *reinterpret_cast<volatile const int32_t*>(seq_lens + b);
    const bool ok = n >= 0 && n < S_max;
    if (ok) {
        for (int h = warp; h < Hkv; h += nw) {
            const size_t bh = (size_t)b * Hkv + h, head = bh * S_max * D;
            const uint2 kraw = *reinterpret_cast<const uint2*>(k_new + bh * D + c0);
            const uint2 vraw = *reinterpret_cast<const uint2*>(v_new + bh * D + c0);
            float4 s = *reinterpret_cast<const float4*>(vsum + bh * D + c0);
            *reinterpret_cast<uint2*>(K + head + (size_t)n * D + c0) = kraw;
            *reinterpret_cast<uint2*>(V + head + (size_t)n * D + c0) = vraw;
            // the small non-contiguous writes.  Invariant of the layout: the rest of the 16-byte vector
            // that holds the last valid position is zero, so readers may take whole vectors without masking.
            const uint16_t kc[4] = {(uint16_t)(kraw.x & 0xffffu), (uint16_t)(kraw.x >> 16),
                                    (uint16_t)(kraw.y & 0xffffu), (uint16_t)(kraw.y >> 16)};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                sparq_half* dst = Kt + head + (size_t)(c0 + u) * S_max + n;
                if ((n & 7) == 0) *reinterpret_cast<uint4*>(dst) = make_uint4(kc[u], 0u, 0u, 0u);
                else *dst = kc[u];
            }
            s.x += __half2float(__ushort_as_half((uint16_t)(vraw.x & 0xffffu)));
            s.y += __half2float(__ushort_as_half((uint16_t)(vraw.x >> 16)));
            s.z += __half2float(__ushort_as_half((uint16_t)(vraw.y & 0xffffu)));
            s.w += __half2float(__ushort_as_half((uint16_t)(vraw.y >> 16)));
            *reinterpret_cast<float4*>(vsum + bh * D + c0) = s;
            const float inv = (float)(n + 1);
            uint2 m;
            m.x = (uint32_t)__half_as_ushort(__float2half_rn(s.x / inv)) | ((uint32_t)__half_as_ushort(__float2half_rn(s.y / inv)) << 16);
            m.y = (uint32_t)__half_as_ushort(__float2half_rn(s.z / inv)) | ((uint32_t)__half_as_ushort(__float2half_rn(s.w / inv)) << 16);
            *reinterpret_cast<uint2*>(vbar + bh * D + c0) = m;
        }
    }
    __syncthreads();                                           // every thread has read the old length
    if (threadIdx.x == 0) {
        if (ok) seq_lens[b] = n + 1;
        else raise_status(status, SPARQ_DEV_CACHE_FULL);
    }
}

// one CTA of 256 threads per (KV head, block of 64 positions), one-dimensional grid:
// Kt[:, t0:t0+64] = K[t0:t0+64, :]^T for t < n.
__global__ void __launch_bounds__(256)
cache_transpose_kernel(const sparq_half* __restrict__ K, sparq_half* __restrict__ Kt,
                       const int32_t* __restrict__ seq_lens, int Hkv, int S_max) {
    __shared__ uint16_t tile[64][D + 2];
    const unsigned tblocks = (unsigned)(S_max + 63) / 64u;
    const int bh = (int)(blockIdx.x / tblocks), t0 = (int)(blockIdx.x % tblocks) * 64, tid = threadIdx.x;
    const int n = min(seq_lens[bh / Hkv], S_max);
    if (t0 >= n) return;
    const size_t head = (size_t)bh * S_max * D;
    for (int i = tid; i < 64 * D; i += 256) {
        int tt = i / D, c = i % D;
        tile[tt][c] = (t0 + tt < n) ? K[head + (size_t)(t0 + tt) * D + c] : (uint16_t)0;
    }
    __syncthreads();
    const int n8 = (n + 7) & ~7;                               // zero fill up to the end of the last 16-byte vector
    for (int i = tid; i < 64 * D; i += 256) {
        int c = i / 64, tt = i % 64;
        if (t0 + tt < n8) Kt[head + (size_t)c * S_max + t0 + tt] = tile[tt][c];
    }
}

// grid B*Hkv, 1024 threads = 8 row groups x D components: fp32 sum of the valid rows of V.
__global__ void __launch_bounds__(1024)
cache_vsum_kernel(const sparq_half* __restrict__ V, const int32_t* __restrict__ seq_lens,
                  float* __restrict__ vsum, sparq_half* __restrict__ vbar, int Hkv, int S_max, int32_t* status) {
    __shared__ float part[8][D];
    const int bh = blockIdx.x, c = threadIdx.x % D, grp = threadIdx.x / D;
    int n = seq_lens[bh / Hkv];
    if (n < 0 || n > S_max) { if (threadIdx.x == 0) raise_status(status, SPARQ_DEV_BAD_SEQ_LEN); n = 0; }
    const sparq_half* Vh = V + (size_t)bh * S_max * D;
    float s = 0.f;
    for (int t = grp; t < n; t += 8) s += __half2float(__ushort_as_half(Vh[(size_t)t * D + c]));
    part[grp][c] = s;
    __syncthreads();
    if (grp == 0) {
        float tot = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) tot += part[i][c];
        vsum[(size_t)bh * D + c] = tot;
        vbar[(size_t)bh * D + c] = __half_as_ushort(__float2half_rn(n > 0 ? tot / (float)n : 0.f));
    }
}

}  // namespace

cudaError_t launch_cache_build(const sparq_half* K, const sparq_half* V, const int32_t* seq_lens, sparq_half* Kt,
                               float* vsum, sparq_half* vbar, int B, int Hkv, int S_max, int32_t* status,
                               cudaStream_t st) {
    const unsigned tblocks = (unsigned)(S_max + 63) / 64u;
    cache_transpose_kernel<<<tblocks * (unsigned)(B * Hkv), 256, 0, st>>>(K, Kt, seq_lens, Hkv, S_max);
    cache_vsum_kernel<<<B * Hkv, 1024, 0, st>>>(V, seq_lens, vsum, vbar, Hkv, S_max, status);
    return cudaGetLastError();
}

cudaError_t launch_cache_append(const sparq_half* k_new, const sparq_half* v_new, sparq_half* K, sparq_half* Kt,
                                sparq_half* V, float* vsum, sparq_half* vbar, int32_t* seq_lens, int B, int Hkv,
                                int S_max, int32_t* status, cudaStream_t st) {
    const int threads = 32 * (Hkv < 32 ? Hkv : 32);
    cache_append_kernel<<<B, threads, 0, st>>>(k_new, v_new, K, Kt, V, vsum, vbar, seq_lens, Hkv, S_max, status);
    return cudaGetLastError();
}

}  // namespace sparq
