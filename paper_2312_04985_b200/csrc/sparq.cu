// SparQ decode attention for NVIDIA B200 (sm_100a): kernels and the C ABI of include/sparq.h.
//
// The path is HBM-bound gather/scan work (about one FMA per byte read), so everything here
// runs on the CUDA cores with 128-bit coalesced loads; no stage is a dense contraction.
//
//   sparq_decode_kernel   one CTA per (batch, query head), all stages fused:
//       a1  top-r of |q| by rank counting on integer keys, tau                (Step 1, Eq. (9))
//       a2  stream the r selected rows of Kt, fp64-accumulated dot products   (Eq. (7))
//           kept on chip as order-preserving 32-bit keys (4 bytes/position in shared memory)
//       a3  softmax statistics of the approximate logits                      (Eq. (7))
//       a4  MSB radix select of the k largest keys; exact fp64 tie refinement; index-ordered
//           compaction; alpha                                                 (Step 2/3)
//       a5  gather of the k selected K and V rows, online softmax in fp32     (Eq. (8))
//       a6  out = alpha y3 + (1 - alpha) v_bar                                (Eq. (10))
//   dense_decode_kernel / dense_merge_kernel    split-sequence dense attention (Eq. (2))
//   cache_append_kernel / seq_bump_kernel       K, Kt, V, vsum, vbar update
//   cache_transpose_kernel / cache_vsum_kernel  Kt and v_bar from a prefilled K, V
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "sparq.h"

namespace {

constexpr int D = SPARQ_HEAD_DIM;   // head dimension d_h
constexpr int NT = 256;             // threads per CTA (decode kernels)
constexpr int NW = NT / 32;         // warps per CTA
constexpr int NHW = NT / 16;        // half-warps per CTA (one K/V row each)
constexpr int RB = 8;               // Kt rows loaded per batch in the stream stage
constexpr int MERGE_FLOATS = NHW * (D + 2);
constexpr unsigned FULL = 0xffffffffu;

__device__ __forceinline__ void raise_status(int32_t* status, int code) {
    if (status) atomicMax(status, code);
}

// ---- fp16 -> fp64 without the slow 64-bit conversion pipe -------------------------------
// The 15 exponent+mantissa bits of a binary16 value, placed at bits 24..10 of the high word
// of a binary64, give exactly value * 2^-1008 (subnormals included: they land on binary64
// subnormals with the same scaling).  The query side carries the factor 2^+1008, so every
// product q_j * K[t, j] is formed exactly and the fp64 FMA chain equals the plain fp64 sum.
__device__ __forceinline__ double h2d_lo(uint32_t w) {   // low half of a packed half2
    return __hiloint2double((int)(((w & 0x8000u) << 16) | ((w & 0x7fffu) << 10)), 0);
}
__device__ __forceinline__ double h2d_hi(uint32_t w) {   // high half of a packed half2
    return __hiloint2double((int)((w & 0x80000000u) | ((w >> 6) & 0x01fffc00u)), 0);
}
__device__ __forceinline__ double h2d_scalar(uint16_t h) { return h2d_lo((uint32_t)h); }

// order-preserving integer keys (larger value <-> larger key); -0 is folded into +0 first
__device__ __forceinline__ uint32_t key32(float f) {
    uint32_t b = __float_as_uint(f + 0.0f);
    return b ^ ((uint32_t)((int32_t)b >> 31) | 0x80000000u);
}
__device__ __forceinline__ float unkey32(uint32_t u) {
    return __uint_as_float((u & 0x80000000u) ? (u ^ 0x80000000u) : ~u);
}
__device__ __forceinline__ unsigned long long key64(double f) {
    unsigned long long b = (unsigned long long)__double_as_longlong(f + 0.0);
    return b ^ ((unsigned long long)((long long)b >> 63) | 0x8000000000000000ull);
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {   // read-once data: keep it out of L1
    uint4 v;
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(FULL, v, o));
    return v;
}

// Block-wide sum / max in a fixed order (bitwise reproducible run to run).  red: NW floats.
__device__ __forceinline__ float block_sum(float v, float* red) {
    v = warp_sum(v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) t += red[w];
    return t;
}
__device__ __forceinline__ uint32_t block_max_u32(uint32_t v, uint32_t* red) {
    v = __reduce_max_sync(FULL, v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    uint32_t t = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) t = max(t, red[w]);
    return t;
}

// Warp 0: walk a 256-bucket histogram from the top and find the bucket that holds the
// need-th largest candidate.  res[0] = bucket, res[1] = candidates above it, res[2] = its count.
__device__ __forceinline__ void find_bucket(const uint32_t* hist, uint32_t need, uint32_t* res) {
    const int lane = threadIdx.x & 31;
    uint32_t c[8], s = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) { c[i] = hist[255 - (lane * 8 + i)]; s += c[i]; }
    uint32_t incl = s;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t v = __shfl_up_sync(FULL, incl, o);
        if (lane >= o) incl += v;
    }
    uint32_t run = incl - s;
    if (run < need && need <= incl) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (run + c[i] >= need) { res[0] = 255 - (lane * 8 + i); res[1] = run; res[2] = c[i]; break; }
            run += c[i];
        }
    }
}

// Add 1 to hist[digit] for every active lane, one shared-memory atomic per distinct digit.
__device__ __forceinline__ void hist_add(uint32_t* hist, bool active, uint32_t digit) {
    unsigned am = __ballot_sync(FULL, active);
    if (active) {
        unsigned peers = __match_any_sync(am, digit);
        if ((int)(threadIdx.x & 31) == __ffs(peers) - 1) atomicAdd(&hist[digit], (uint32_t)__popc(peers));
    }
}

struct DecodeShared {
    double qd[D + RB];          // selected query components * 2^1008, in i1 order, zero padded
    float qf[D];                // q as fp32
    uint32_t rowoff[D + RB];    // i1[j] * (S_max / 8): row offset in 16-byte units
    uint32_t rkey[D];           // top-r ranking keys
    int32_t i1[D];
    uint32_t hist[256];
    int32_t i2[SPARQ_K_MAX];
    float red[NW];
    uint32_t redu[NW];
    uint32_t wcnt[2 * NW];
    uint32_t res[4];
    unsigned long long res64[2];
    float inv_tau;
};

// fp64 dot product of the selected query components with position t of the r selected Kt rows,
// in the same order as the stream stage (so it reproduces that stage's value bit for bit).
__device__ __forceinline__ double dot64_at(const sparq_half* Kt_head, const DecodeShared& sh, int S_max, int r, int t) {
    double acc = 0.0;
    for (int j = 0; j < r; ++j)
        acc = fma(sh.qd[j], h2d_scalar(Kt_head[(size_t)sh.i1[j] * S_max + t]), acc);
    return acc;
}

__global__ void __launch_bounds__(NT)
sparq_decode_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                    const sparq_half* __restrict__ Kt, const sparq_half* __restrict__ V,
                    const sparq_half* __restrict__ vbar, const int32_t* __restrict__ seq_lens,
                    int Hq, int Hkv, int S_max, int r, int k,
                    sparq_half* __restrict__ out, int32_t* __restrict__ idx_r, int32_t* __restrict__ idx_k,
                    float* __restrict__ alpha_out, int32_t* status) {
    extern __shared__ __align__(16) unsigned char dyn_smem[];
    uint32_t* keys = reinterpret_cast<uint32_t*>(dyn_smem);   // [n] approximate-logit keys
    float* merge = reinterpret_cast<float*>(dyn_smem);        // reused by stage a5 once keys are dead
    __shared__ DecodeShared sh;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bh = blockIdx.x, b = bh / Hq, h = bh % Hq, hkv = h / (Hq / Hkv);
    const int n = seq_lens[b];
    const size_t kv_head = (size_t)b * Hkv + hkv;
    sparq_half* out_row = out + (size_t)bh * D;

    if (n < 1 || n > S_max) {            // defined result, no trap
        if (tid == 0) { raise_status(status, SPARQ_DEV_BAD_SEQ_LEN); if (alpha_out) alpha_out[bh] = 0.f; }
        if (tid < D) out_row[tid] = 0;
        if (idx_r) for (int j = tid; j < r; j += NT) idx_r[(size_t)bh * r + j] = -1;
        if (idx_k) for (int j = tid; j < k; j += NT) idx_k[(size_t)bh * k + j] = -1;
        return;
    }
    const int k_eff = min(k, n);

    // ------------------------------------------------------------------ a1: top-r of |q|
    // key = |q_j| bit pattern above (127 - j): distinct keys, larger |q| first, then smaller j.
    float aq = 0.f;
    if (tid < D) {
        uint16_t hb = q[(size_t)bh * D + tid];
        float f = __half2float(__ushort_as_half(hb));
        sh.qf[tid] = f;
        aq = fabsf(f);
        sh.rkey[tid] = ((uint32_t)(hb & 0x7fffu) << 7) | (uint32_t)(D - 1 - tid);
    }
    __syncthreads();
    bool sel = false;
    if (tid < D) {
        uint32_t mine = sh.rkey[tid];
        int rank = 0;
#pragma unroll 8
        for (int j = 0; j < D; ++j) rank += (sh.rkey[j] > mine);
        sel = rank < r;
    }
    unsigned bal = __ballot_sync(FULL, sel);
    if (lane == 0) sh.wcnt[warp] = __popc(bal);
    float l1_all = block_sum(aq, sh.red);                    // contains the barriers wcnt needs
    float l1_sel = block_sum(sel ? aq : 0.f, sh.red);
    if (sel) {
        int slot = __popc(bal & ((1u << lane) - 1));
        for (int w = 0; w < warp; ++w) slot += sh.wcnt[w];
        sh.i1[slot] = tid;                                   // ascending by construction
        sh.qd[slot] = ldexp((double)sh.qf[tid], 1008);
        sh.rowoff[slot] = (uint32_t)tid * (uint32_t)(S_max >> 3);
    }
    if (tid == 0) sh.inv_tau = (l1_all > 0.f) ? rsqrtf((float)D * l1_sel / l1_all) : 1.0f;
    __syncthreads();
    const int r_pad = (r + RB - 1) / RB * RB;
    if (tid >= r && tid < r_pad) { sh.qd[tid] = 0.0; sh.rowoff[tid] = sh.rowoff[0]; }
    if (idx_r) for (int j = tid; j < r; j += NT) idx_r[(size_t)bh * r + j] = sh.i1[j];
    __syncthreads();
    const float inv_tau = sh.inv_tau;

    float alpha = 0.f;
    if (k_eff > 0) {
        // -------------------------------------------------------------- a2: stream r rows of Kt
        const sparq_half* Kt_head = Kt + kv_head * (size_t)D * S_max;
        const uint4* Kt_vec = reinterpret_cast<const uint4*>(Kt_head);
        const int n_vec = (n + 7) >> 3;
        for (int c8 = tid; c8 < n_vec; c8 += NT) {
            double acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.0;
            for (int jb = 0; jb < r_pad; jb += RB) {
                uint4 v[RB];
#pragma unroll
                for (int u = 0; u < RB; ++u) v[u] = ld_stream(Kt_vec + sh.rowoff[jb + u] + c8);
#pragma unroll
                for (int u = 0; u < RB; ++u) {
                    const double qj = sh.qd[jb + u];
                    acc[0] = fma(qj, h2d_lo(v[u].x), acc[0]); acc[1] = fma(qj, h2d_hi(v[u].x), acc[1]);
                    acc[2] = fma(qj, h2d_lo(v[u].y), acc[2]); acc[3] = fma(qj, h2d_hi(v[u].y), acc[3]);
                    acc[4] = fma(qj, h2d_lo(v[u].z), acc[4]); acc[5] = fma(qj, h2d_hi(v[u].z), acc[5]);
                    acc[6] = fma(qj, h2d_lo(v[u].w), acc[6]); acc[7] = fma(qj, h2d_hi(v[u].w), acc[7]);
                }
            }
            uint32_t kk[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) kk[e] = key32((float)acc[e]);
            const int t0 = c8 << 3;
            if (t0 + 8 <= n) {
                *reinterpret_cast<uint4*>(keys + t0) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
                *reinterpret_cast<uint4*>(keys + t0 + 4) = make_uint4(kk[4], kk[5], kk[6], kk[7]);
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) if (t0 + e < n) keys[t0 + e] = kk[e];
            }
        }
        __syncthreads();

        // -------------------------------------------------------------- a3: softmax statistics
        uint32_t kmax = 0;
        for (int t = tid; t < n; t += NT) kmax = max(kmax, keys[t]);
        kmax = block_max_u32(kmax, sh.redu);
        const float vmax = unkey32(kmax);
        float zpart = 0.f;
        for (int t = tid; t < n; t += NT) zpart += __expf((unkey32(keys[t]) - vmax) * inv_tau);
        const float Z = block_sum(zpart, sh.red);

        // -------------------------------------------------------------- a4: top-k select
        // 4 passes of 8 bits from the top: afterwards `prefix` is the k_eff-th largest key T,
        // `need` of the `ceq` keys equal to T are wanted and every key > T is selected.
        uint32_t prefix = 0, mask = 0, need = (uint32_t)k_eff, ceq = 0;
        for (int shift = 24; shift >= 0; shift -= 8) {
            sh.hist[tid] = 0;                                // NT == 256 buckets
            __syncthreads();
            for (int base = 0; base < n; base += NT) {
                int t = base + tid;
                uint32_t u = (t < n) ? keys[t] : 0u;
                hist_add(sh.hist, t < n && (u & mask) == prefix, (u >> shift) & 255u);
            }
            __syncthreads();
            if (warp == 0) find_bucket(sh.hist, need, sh.res);
            __syncthreads();
            prefix |= sh.res[0] << shift;
            mask |= 255u << shift;
            need -= sh.res[1];
            ceq = sh.res[2];
        }
        const uint32_t T = prefix;

        if (ceq > need) {
            // Rare: several positions round to the same fp32 key at the threshold.  Decide among
            // them by their fp64 values (recomputed from Kt), 8 passes of 8 bits, then re-key the
            // winners just above T and the losers just below it.  Equal fp64 values stay at T and
            // the compaction takes the lowest positions.
            unsigned long long p64 = 0, m64 = 0;
            uint32_t need64 = need;
            for (int shift = 56; shift >= 0; shift -= 8) {
                sh.hist[tid] = 0;
                __syncthreads();
                for (int base = 0; base < n; base += NT) {
                    int t = base + tid;
                    bool act = t < n && keys[t] == T;
                    unsigned long long u = 0;
                    if (act) { u = key64(dot64_at(Kt_head, sh, S_max, r, t)); act = (u & m64) == p64; }
                    hist_add(sh.hist, act, (uint32_t)(u >> shift) & 255u);
                }
                __syncthreads();
                if (warp == 0) find_bucket(sh.hist, need64, sh.res);
                __syncthreads();
                p64 |= (unsigned long long)sh.res[0] << shift;
                m64 |= 255ull << shift;
                need64 -= sh.res[1];
            }
            for (int t = tid; t < n; t += NT) {
                if (keys[t] == T) {
                    unsigned long long u = key64(dot64_at(Kt_head, sh, S_max, r, t));
                    if (u > p64) keys[t] = T + 1; else if (u < p64) keys[t] = T - 1;
                }
            }
            need = need64;
            __syncthreads();
        }

        // index-ordered compaction: warp w owns a contiguous segment of positions
        const int seg = ((n + NW - 1) / NW + 31) & ~31;
        const int t_begin = warp * seg, t_end = min(n, t_begin + seg);
        uint32_t cg = 0, ce = 0;
        for (int t0 = t_begin; t0 < t_end; t0 += 32) {
            int t = t0 + lane;
            uint32_t u = (t < t_end) ? keys[t] : 0u;
            cg += __popc(__ballot_sync(FULL, t < t_end && u > T));
            ce += __popc(__ballot_sync(FULL, t < t_end && u == T));
        }
        if (lane == 0) { sh.wcnt[warp] = cg; sh.wcnt[NW + warp] = ce; }
        __syncthreads();
        uint32_t g_run = 0, e_run = 0;
        for (int w = 0; w < warp; ++w) { g_run += sh.wcnt[w]; e_run += sh.wcnt[NW + w]; }
        float a_part = 0.f;
        const unsigned lt = (1u << lane) - 1;
        for (int t0 = t_begin; t0 < t_end; t0 += 32) {
            int t = t0 + lane;
            uint32_t u = (t < t_end) ? keys[t] : 0u;
            bool gt = t < t_end && u > T, eq = t < t_end && u == T;
            unsigned bg = __ballot_sync(FULL, gt), be = __ballot_sync(FULL, eq);
            uint32_t gb = g_run + __popc(bg & lt), eb = e_run + __popc(be & lt);
            if (gt || (eq && eb < need)) {
                sh.i2[gb + min(eb, need)] = t;
                a_part += __expf((unkey32(u) - vmax) * inv_tau);
            }
            g_run += __popc(bg);
            e_run += __popc(be);
        }
        alpha = block_sum(a_part, sh.red) / Z;               // barriers also publish sh.i2; keys are dead

        // -------------------------------------------------------------- a5: gather k rows of K and V
        const int hw = tid >> 4, l16 = tid & 15;
        const float qscale = rsqrtf((float)D) * 1.4426950408889634f;   // 1/sqrt(d_h) * log2(e)
        float qs[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) qs[e] = sh.qf[l16 * 8 + e] * qscale;
        const uint4* Kh = reinterpret_cast<const uint4*>(K + kv_head * (size_t)S_max * D);
        const uint4* Vh = reinterpret_cast<const uint4*>(V + kv_head * (size_t)S_max * D);
        float m = -CUDART_INF_F, l = 0.f, acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        constexpr int RG = 4;
        for (int jb = 0; jb < k_eff; jb += NHW * RG) {       // trip count uniform across the CTA
            const int j0 = jb + hw;
            uint4 kv[RG], vv[RG];
#pragma unroll
            for (int u = 0; u < RG; ++u) {
                int j = j0 + u * NHW;
                int t = sh.i2[min(j, k_eff - 1)];
                kv[u] = ld_stream(Kh + (size_t)t * (D / 8) + l16);
                vv[u] = ld_stream(Vh + (size_t)t * (D / 8) + l16);
            }
#pragma unroll
            for (int u = 0; u < RG; ++u) {
                const __half2* kh = reinterpret_cast<const __half2*>(&kv[u]);
                float z = 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    float2 f = __half22float2(kh[e]);
                    z = fmaf(f.x, qs[2 * e], z);
                    z = fmaf(f.y, qs[2 * e + 1], z);
                }
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) z += __shfl_xor_sync(FULL, z, o);
                if (j0 + u * NHW < k_eff) {                  // uniform within the half-warp
                    float mn = fmaxf(m, z);
                    float sc = exp2f(m - mn), p = exp2f(z - mn);
                    l = l * sc + p;
                    const __half2* vh = reinterpret_cast<const __half2*>(&vv[u]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        float2 f = __half22float2(vh[e]);
                        acc[2 * e] = fmaf(p, f.x, acc[2 * e] * sc);
                        acc[2 * e + 1] = fmaf(p, f.y, acc[2 * e + 1] * sc);
                    }
                    m = mn;
                }
            }
        }
        // merge the half-warps' partial softmax states
        float* mg = merge + hw * (D + 2);
#pragma unroll
        for (int e = 0; e < 8; ++e) mg[l16 * 8 + e] = acc[e];
        if (l16 == 0) { mg[D] = m; mg[D + 1] = l; }
        __syncthreads();
    }

    // ------------------------------------------------------------------ a6: combine with v_bar
    if (tid < D) {
        float vb = __half2float(__ushort_as_half(vbar[kv_head * D + tid]));
        float y = vb;
        if (k_eff > 0) {
            float M = -CUDART_INF_F;
#pragma unroll
            for (int w = 0; w < NHW; ++w) M = fmaxf(M, merge[w * (D + 2) + D]);
            float L = 0.f, s = 0.f;
#pragma unroll
            for (int w = 0; w < NHW; ++w) {
                float sc = exp2f(merge[w * (D + 2) + D] - M);
                L = fmaf(merge[w * (D + 2) + D + 1], sc, L);
                s = fmaf(merge[w * (D + 2) + tid], sc, s);
            }
            y = alpha * (s / L) + (1.f - alpha) * vb;
        }
        out_row[tid] = __half_as_ushort(__float2half_rn(y));
    }
    if (tid == 0 && alpha_out) alpha_out[bh] = alpha;
    if (idx_k) for (int j = tid; j < k; j += NT) idx_k[(size_t)bh * k + j] = (j < k_eff) ? sh.i2[j] : -1;
}

// =========================================================================== dense attention
// grid (splits, Hkv, B).  A CTA covers positions [split*chunk, (split+1)*chunk) of one KV head
// for all G query heads of the group; half-warp per cache row, online softmax in fp32.
template <int G>
__global__ void __launch_bounds__(NT)
dense_decode_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                    const sparq_half* __restrict__ V, const int32_t* __restrict__ seq_lens,
                    int Hq, int Hkv, int S_max, int g_total, int g_base, int splits,
                    sparq_half* __restrict__ out, float* __restrict__ ws, int32_t* status) {
    __shared__ float merge[NHW * (D + 2)];
    const int tid = threadIdx.x, hw = tid >> 4, l16 = tid & 15;
    const int split = blockIdx.x, hkv = blockIdx.y, b = blockIdx.z;
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

    const float qscale = rsqrtf((float)D) * 1.4426950408889634f;
    float qs[G][8], acc[G][8], m[G], l[G];
#pragma unroll
    for (int gi = 0; gi < G; ++gi) {
        m[gi] = -CUDART_INF_F; l[gi] = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            qs[gi][e] = __half2float(__ushort_as_half(q[((size_t)b * Hq + h0 + gi) * D + l16 * 8 + e])) * qscale;
            acc[gi][e] = 0.f;
        }
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
        for (int u = 0; u < RG; ++u) {
            const __half2* kh = reinterpret_cast<const __half2*>(&kv[u]);
            const __half2* vh = reinterpret_cast<const __half2*>(&vv[u]);
            float kf[8], vf[8];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                float2 f = __half22float2(kh[e]); kf[2 * e] = f.x; kf[2 * e + 1] = f.y;
                float2 w = __half22float2(vh[e]); vf[2 * e] = w.x; vf[2 * e + 1] = w.y;
            }
            const bool valid = t0 + u * NHW < t_end;          // uniform within the half-warp
#pragma unroll
            for (int gi = 0; gi < G; ++gi) {
                float z = 0.f;
#pragma unroll
                for (int e = 0; e < 8; ++e) z = fmaf(kf[e], qs[gi][e], z);
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) z += __shfl_xor_sync(FULL, z, o);
                if (valid) {
                    float mn = fmaxf(m[gi], z);
                    float sc = exp2f(m[gi] - mn), p = exp2f(z - mn);
                    l[gi] = l[gi] * sc + p;
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc[gi][e] = fmaf(p, vf[e], acc[gi][e] * sc);
                    m[gi] = mn;
                }
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

// =========================================================================== cache maintenance
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
    Kt[head + (size_t)c * S_max + n] = kc;                    // the small non-contiguous write
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
    for (int i = tid; i < 64 * D; i += 256) {
        int c = i / 64, tt = i % 64;
        if (t0 + tt < n) Kt[head + (size_t)c * S_max + t0 + tt] = tile[tt][c];
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

// =========================================================================== host side
constexpr size_t kDecodeStaticSmem = sizeof(DecodeShared);

int device_smem_optin() {
    int dev = 0, v = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 0;
    if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return 0;
    return v;
}

size_t decode_dyn_smem(int S_max) {
    size_t keys = (size_t)S_max * sizeof(uint32_t);
    size_t mrg = (size_t)MERGE_FLOATS * sizeof(float);
    return keys > mrg ? keys : mrg;
}

int dense_splits(int B, int Hkv, int S_max) {
    long ctas = (long)B * Hkv;
    long want = (4L * 148 + ctas - 1) / ctas;                 // aim for >= 4 CTAs per SM
    long cap = (S_max + 255) / 256;                           // at least 256 positions per split
    long s = want < cap ? want : cap;
    return (int)(s < 1 ? 1 : s);
}

bool bad_common(int B, int Hq, int Hkv, int d, int S_max) {
    return B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || d != D || S_max < 8 || S_max % 8 != 0;
}

int launch_ok() { return cudaGetLastError() == cudaSuccess ? SPARQ_OK : SPARQ_ERR_CUDA; }

}  // namespace

extern "C" {

const char* sparq_status_string(int code) {
    switch (code) {
        case SPARQ_OK: return "SPARQ_OK";
        case SPARQ_ERR_NULL_POINTER: return "SPARQ_ERR_NULL_POINTER";
        case SPARQ_ERR_BAD_SHAPE: return "SPARQ_ERR_BAD_SHAPE";
        case SPARQ_ERR_BAD_RK: return "SPARQ_ERR_BAD_RK";
        case SPARQ_ERR_WORKSPACE: return "SPARQ_ERR_WORKSPACE";
        case SPARQ_ERR_TOO_LONG: return "SPARQ_ERR_TOO_LONG";
        case SPARQ_ERR_CUDA: return "SPARQ_ERR_CUDA";
        case SPARQ_DEV_BAD_SEQ_LEN: return "SPARQ_DEV_BAD_SEQ_LEN";
        case SPARQ_DEV_CACHE_FULL: return "SPARQ_DEV_CACHE_FULL";
        default: return "SPARQ_UNKNOWN_STATUS";
    }
}

int sparq_max_seq_len(void) {
    long avail = (long)device_smem_optin() - (long)kDecodeStaticSmem - 1024;
    if (avail <= 0) return 0;
    return (int)((avail / 4) & ~7L);
}

int sparq_cache_build(const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                      sparq_half* Kt, float* vsum, sparq_half* vbar,
                      int B, int Hkv, int d, int S_max, int32_t* status, void* stream) {
    if (!K || !V || !seq_lens || !Kt || !vsum || !vbar) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hkv, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    dim3 grid((S_max + 63) / 64, B * Hkv);
    cache_transpose_kernel<<<grid, 256, 0, st>>>(K, Kt, seq_lens, Hkv, S_max);
    cache_vsum_kernel<<<B * Hkv, 1024, 0, st>>>(V, seq_lens, vsum, vbar, Hkv, S_max, status);
    return launch_ok();
}

int sparq_cache_append(const sparq_half* k_new, const sparq_half* v_new,
                       sparq_half* K, sparq_half* Kt, sparq_half* V, float* vsum, sparq_half* vbar,
                       int32_t* seq_lens, int B, int Hkv, int d, int S_max, int32_t* status, void* stream) {
    if (!k_new || !v_new || !K || !Kt || !V || !vsum || !vbar || !seq_lens) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hkv, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    cache_append_kernel<<<B * Hkv, D, 0, st>>>(k_new, v_new, K, Kt, V, vsum, vbar, seq_lens, Hkv, S_max, status);
    seq_bump_kernel<<<(B + 255) / 256, 256, 0, st>>>(seq_lens, B, S_max);
    return launch_ok();
}

size_t sparq_workspace_bytes(int, int, int, int, int, int, int) { return 0; }

int sparq_decode(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                 const sparq_half* vbar, const int32_t* seq_lens,
                 int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                 sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                 void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    (void)workspace; (void)workspace_bytes;
    if (!q || !K || !Kt || !V || !vbar || !seq_lens || !out) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hq, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    if (r < 1 || r > d || k < 0 || k > SPARQ_K_MAX) return SPARQ_ERR_BAD_RK;
    const size_t dyn = decode_dyn_smem(S_max);
    if (dyn + kDecodeStaticSmem + 1024 > (size_t)device_smem_optin()) return SPARQ_ERR_TOO_LONG;
    if (cudaFuncSetAttribute(sparq_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn) != cudaSuccess)
        return SPARQ_ERR_CUDA;
    sparq_decode_kernel<<<B * Hq, NT, dyn, (cudaStream_t)stream>>>(q, K, Kt, V, vbar, seq_lens, Hq, Hkv, S_max, r, k,
                                                                    out, idx_r, idx_k, alpha, status);
    return launch_ok();
}

size_t dense_workspace_bytes(int B, int Hq, int Hkv, int d, int S_max) {
    if (bad_common(B, Hq, Hkv, d, S_max)) return 0;
    int splits = dense_splits(B, Hkv, S_max);
    return splits == 1 ? 0 : (size_t)B * Hq * splits * (D + 2) * sizeof(float);
}

int dense_decode(const sparq_half* q, const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                 int B, int Hq, int Hkv, int d, int S_max, sparq_half* out,
                 void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    if (!q || !K || !V || !seq_lens || !out) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hq, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    const int splits = dense_splits(B, Hkv, S_max);
    const size_t need = dense_workspace_bytes(B, Hq, Hkv, d, S_max);
    if (need && (!workspace || workspace_bytes < need)) return SPARQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    float* ws = (float*)workspace;
    const int g = Hq / Hkv;
    dim3 grid(splits, Hkv, B);
    // the group's query heads are served G at a time by one pass over K and V
    for (int g_base = 0; g_base < g;) {
        int left = g - g_base;
        if (left >= 8) { dense_decode_kernel<8><<<grid, NT, 0, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status); g_base += 8; }
        else if (left >= 4) { dense_decode_kernel<4><<<grid, NT, 0, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status); g_base += 4; }
        else if (left >= 2) { dense_decode_kernel<2><<<grid, NT, 0, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status); g_base += 2; }
        else { dense_decode_kernel<1><<<grid, NT, 0, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status); g_base += 1; }
    }
    if (splits > 1) dense_merge_kernel<<<B * Hq, D, 0, st>>>(ws, seq_lens, Hq, S_max, splits, out);
    return launch_ok();
}

size_t sparq_step_host_staging_bytes(int B, int Hq, int Hkv, int d) {
    if (B < 1 || Hq < 1 || Hkv < 1 || d < 1) return 0;
    return ((size_t)2 * B * Hq * d + (size_t)2 * B * Hkv * d) * sizeof(sparq_half);
}

int sparq_step_host(const sparq_half* q_host, const sparq_half* k_new_host, const sparq_half* v_new_host,
                    sparq_half* K, sparq_half* Kt, sparq_half* V, float* vsum, sparq_half* vbar,
                    int32_t* seq_lens, int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                    sparq_half* out_host, void* staging, size_t staging_bytes, int32_t* status, void* stream) {
    if (!q_host || !k_new_host || !v_new_host || !out_host) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hq, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    if (!staging || staging_bytes < sparq_step_host_staging_bytes(B, Hq, Hkv, d)) return SPARQ_ERR_WORKSPACE;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t nq = (size_t)B * Hq * d, nkv = (size_t)B * Hkv * d;
    sparq_half* q_dev = (sparq_half*)staging;
    sparq_half* out_dev = q_dev + nq;
    sparq_half* k_dev = out_dev + nq;
    sparq_half* v_dev = k_dev + nkv;
    if (cudaMemcpyAsync(q_dev, q_host, nq * sizeof(sparq_half), cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(k_dev, k_new_host, nkv * sizeof(sparq_half), cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(v_dev, v_new_host, nkv * sizeof(sparq_half), cudaMemcpyHostToDevice, st) != cudaSuccess)
        return SPARQ_ERR_CUDA;
    int rc = sparq_cache_append(k_dev, v_dev, K, Kt, V, vsum, vbar, seq_lens, B, Hkv, d, S_max, status, stream);
    if (rc != SPARQ_OK) return rc;
    rc = sparq_decode(q_dev, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, d, S_max, r, k, out_dev, nullptr, nullptr, nullptr,
                      nullptr, 0, status, stream);
    if (rc != SPARQ_OK) return rc;
    if (cudaMemcpyAsync(out_host, out_dev, nq * sizeof(sparq_half), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return SPARQ_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? SPARQ_OK : SPARQ_ERR_CUDA;
}

}  // extern "C"
