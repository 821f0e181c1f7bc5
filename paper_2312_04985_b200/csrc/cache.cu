// Cache maintenance: the per-step append (K, Kt, V, running value sum and mean) and the
// prefill-side builder that derives Kt and v_bar from a filled K, V.
#include "common.cuh"
#include "kernels.h"

namespace sparq {
namespace {

// grid B*Hkv, D threads: thread c owns component c of the new token.
__global__ void __launch_bounds__(D)
cache_append_kernel(const sparq_half* __restrict__ k_new, const sparq_half* __restrict__ v_new,
                    sparq_half* __restrict__ K, sparq_half* __restrict__ Kt, sparq_half* __restrict__ V,
                    float* __restrict__ vsum, sparq_half* __restrict__ vbar,
                    const int32_t* __restrict__ seq_lens, int Hkv, int S_max, int32_t* status) {
    const int bh = blockIdx.x, c = threadIdx.x, b = bh / Hkv;
    const int n = seq_lens[b];
    if (n < 0 || n >= S_max) { if (c == 0) raise_status(status, SPARQ_DEV_CACHE_FULL); return; }
    const uint16_t kc = k_new[(size_t)bh * D + c], vc = v_new[(size_t)bh * D + c];
    const size_t head = (size_t)bh * S_max * D;
    K[head + (size_t)n * D + c] = kc;
    V[head + (size_t)n * D + c] = vc;
    // the small non-contiguous write.  Invariant of the layout: the rest of the 16-byte vector that
    // holds the last valid position is zero, so readers may take whole vectors without masking.
    if ((n & 7) == 0) *reinterpret_cast<uint4*>(Kt + head + (size_t)c * S_max + n) = make_uint4(kc, 0u, 0u, 0u);
    else Kt[head + (size_t)c * S_max + n] = kc;
    float s = vsum[(size_t)bh * D + c] + __half2float(__ushort_as_half(vc));
    vsum[(size_t)bh * D + c] = s;
    vbar[(size_t)bh * D + c] = __half_as_ushort(__float2half_rn(s / (float)(n + 1)));
}

// runs after every head of every sequence has written at the old length
__global__ void seq_bump_kernel(int32_t* seq_lens, int B, int S_max) {
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b < B) { int n = seq_lens[b]; if (n >= 0 && n < S_max) seq_lens[b] = n + 1; }
}

// grid (ceil(S_max/64), B*Hkv), 256 threads: Kt[:, t0:t0+64] = K[t0:t0+64, :]^T for t < n.
__global__ void __launch_bounds__(256)
cache_transpose_kernel(const sparq_half* __restrict__ K, sparq_half* __restrict__ Kt,
                       const int32_t* __restrict__ seq_lens, int Hkv, int S_max) {
    __shared__ uint16_t tile[64][D + 2];
    const int bh = blockIdx.y, t0 = blockIdx.x * 64, tid = threadIdx.x;
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
    dim3 grid((S_max + 63) / 64, B * Hkv);
    cache_transpose_kernel<<<grid, 256, 0, st>>>(K, Kt, seq_lens, Hkv, S_max);
    cache_vsum_kernel<<<B * Hkv, 1024, 0, st>>>(V, seq_lens, vsum, vbar, Hkv, S_max, status);
    return cudaGetLastError();
}

cudaError_t launch_cache_append(const sparq_half* k_new, const sparq_half* v_new, sparq_half* K, sparq_half* Kt,
                                sparq_half* V, float* vsum, sparq_half* vbar, int32_t* seq_lens, int B, int Hkv,
                                int S_max, int32_t* status, cudaStream_t st) {
    cache_append_kernel<<<B * Hkv, D, 0, st>>>(k_new, v_new, K, Kt, V, vsum, vbar, seq_lens, Hkv, S_max, status);
    seq_bump_kernel<<<(B + 255) / 256, 256, 0, st>>>(seq_lens, B, S_max);
    return cudaGetLastError();
}

}  // namespace sparq
