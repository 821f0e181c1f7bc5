// sparq_decode for a handful of (batch, query head) units -- batch-1 decoding: one CTA of 512
// threads per unit, so that every stage of the unit's latency chain runs wide.
// With fewer units than SMs nothing overlaps one unit's stages with another's; what counts is how
// long each stage takes, and the persistent kernel's one-warp top-r and 256-thread select and gather
// stages are built for throughput, not for that.
//
//   a1  top-r of |q| by rank counting, one component per thread                  (Step 1, Eq. (9))
//   a2  the r selected rows of Kt by plain 128-bit loads: the CTA covers 4096 positions at a time,
//       a vector of 8 positions per thread, sixteen rows in flight per thread.  Keys (4 bytes per
//       position) stay in shared memory; the first-digit histogram, the largest key, the largest
//       |K| and the softmax denominator are accumulated on the way                       (Eq. (7))
//   a3-a6  decode_common.cuh: select from the prefilled histogram, fp64 re-decision of the band,
//       alpha, gather of the K and V rows (32 half-warps, four rows in flight each: one round for
//       k = 128), combine                                           (Steps 2-3, Eqs. (8), (10))
#include "decode_common.cuh"
#include "kernels.h"

namespace sparq {
namespace {

constexpr int WROWS = 16;                // Kt rows in flight per thread

template <int WNT>
struct WideShared {
    HeadMeta hm;
    int32_t i2[SPARQ_K_MAX];
    float red[2 * (WNT / 32)];
    uint32_t redu[2 * (WNT / 32)];
    uint32_t res[4];
    uint32_t band[4];
    uint32_t cnt[4];
};

__host__ __device__ constexpr int wide_bm_words(int S_max) { return (S_max + 127) / 128 * 4; }
__host__ __device__ constexpr size_t wide_keys_bytes(int S_max) { return ((size_t)S_max * 4 + 127) & ~(size_t)127; }

// WNT = 512: one CTA per SM (the latency form).  WNT = 256: two CTAs per SM where their keys fit, so that
// one unit's select and gather overlap another's stream (many units on a long cache).
template <int WNT>
__global__ void __launch_bounds__(WNT, WNT == 512 ? 1 : 2)
sparq_decode_wide_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                         const sparq_half* __restrict__ Kt, const sparq_half* __restrict__ V,
                         const sparq_half* __restrict__ vbar, const int32_t* __restrict__ seq_lens,
                         int Hq, int Hkv, int S_max, int r, int k, uint32_t opts,
                         sparq_half* __restrict__ out, int32_t* __restrict__ idx_r, int32_t* __restrict__ idx_k,
                         float* __restrict__ alpha_out, int32_t* status) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    uint32_t* keys = reinterpret_cast<uint32_t*>(dyn_smem);                           // [S_max] approximate-score keys
    uint32_t* hist1 = reinterpret_cast<uint32_t*>(dyn_smem + wide_keys_bytes(S_max));  // [FBINS] histogram of the keys' top bits
    unsigned char* scratch = reinterpret_cast<unsigned char*>(hist1 + FBINS);         // the post phase's scratch
    using WCTA = Group<WNT, 0>;
    constexpr int WCH = WNT * 8;                             // positions per pass: a vector of 8 per thread
    __shared__ WideShared<WNT> sh;
    HeadMeta& hm = sh.hm;

    const int tid = threadIdx.x;
    const int bh = blockIdx.x, b = bh / Hq, h = bh % Hq, hkv = h / (Hq / Hkv);
    const int n = seq_lens[b];
    const size_t kv_head = (size_t)b * Hkv + hkv;
    sparq_half* out_row = out + (size_t)bh * D;

    if (n < 1 || n > S_max) {            // defined result, no trap
        if (tid == 0) { raise_status(status, SPARQ_DEV_BAD_SEQ_LEN); if (alpha_out) alpha_out[bh] = 0.f; }
        if (tid < D) out_row[tid] = 0;
        if (idx_r) for (int j = tid; j < r; j += WNT) idx_r[(size_t)bh * r + j] = -1;
        if (idx_k) for (int j = tid; j < k; j += WNT) idx_k[(size_t)bh * k + j] = -1;
        return;
    }
    const int k_eff = min(k, n);
    for (int i = tid; i < FBINS; i += WNT) hist1[i] = 0;
    if (tid == 0) { hm.bh = bh; hm.n = n; hm.k_eff = k_eff; hm.valid = 1; opt_set_window(hm, n, k_eff, opts); }
    top_r_block<WCTA, 8>(tid, q + (size_t)bh * D, r, hm, sh.red, sh.cnt, opts);        // a1; its barriers publish the cleared histogram
    if (idx_r) for (int j = tid; j < r; j += WNT) idx_r[(size_t)bh * r + j] = hm.i1[j];
    if (k_eff == 0) {                    // nothing to select: the output is the mean value vector
        if (tid < D) out_row[tid] = vbar[kv_head * D + tid];
        if (tid == 0 && alpha_out) alpha_out[bh] = 0.f;
        return;
    }

    // ------------------------------------------------------------------ a2 (+ a3 statistics)
    const sparq_half* Kt_head = Kt + kv_head * (size_t)D * S_max;
    const uint4* Kt_vec = reinterpret_cast<const uint4*>(Kt_head);
    const int row_vecs = S_max >> 3;
    const float c1 = hm.inv_tau * LOG2E;
    uint32_t kmax = 0;
    float zm = -CUDART_INF_F, zs = 0.f;                      // running max (log2 units) and sum of 2^(x - zm)
    __half2 mx[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) mx[e] = __float2half2_rn(0.f);
    const int n_pass = (n + WCH - 1) / WCH;
    for (int c = 0; c < n_pass; ++c) {
        const int t0 = c * WCH + tid * 8;
        const int nvalid = min(8, n - t0);                   // (the layout keeps zeros up to the end of the last vector)
        if (nvalid <= 0) continue;
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        for (int jb = 0; jb < r; jb += WROWS) {
            uint4 v[WROWS];
#pragma unroll
            for (int u = 0; u < WROWS; ++u) v[u] = ld_stream(Kt_vec + (size_t)hm.i1[min(jb + u, r - 1)] * row_vecs + (t0 >> 3));
#pragma unroll
            for (int u = 0; u < WROWS; ++u)
                if (jb + u < r) row_fma(acc, mx, v[u], hm.qh[jb + u]);
        }
        float cm = -CUDART_INF_F;                            // softmax statistics of these keys, online
#pragma unroll
        for (int e = 0; e < 8; ++e) if (e < nvalid) cm = fmaxf(cm, acc[e] * c1);
        const float nm = fmaxf(zm, cm);
        zs *= ex2(zm - nm);
#pragma unroll
        for (int e = 0; e < 8; ++e) if (e < nvalid) zs += ex2(acc[e] * c1 - nm);
        zm = nm;
#pragma unroll
        for (int e = 0; e < 8; ++e)
            if (e < nvalid) {
                const uint32_t kk = key32(acc[e]);
                keys[t0 + e] = kk;
                kmax = max(kmax, kk);
                atomicAdd(&hist1[kk >> FSH], 1u);
            }
    }
    uint32_t kabs_bits = __float_as_uint(mx_to_float(mx));
    group_max2_u32<WCTA>(kmax, kabs_bits, sh.redu, tid);     // barriers: the keys and the histogram are complete
    const float Z = group_sum<WCTA>(zs > 0.f ? zs * ex2(zm - unkey32(kmax) * c1) : 0.f, sh.red, tid);

    // ------------------------------------------------------------------ a3-a6
    PostScratch sc;
    carve_post_scratch(sc, scratch, WCTA::NHW, wide_bm_words(S_max));
    sc.i2 = sh.i2; sc.red = sh.red; sc.redu = sh.redu; sc.res = sh.res; sc.band = sh.band;
    const float kabs = __uint_as_float(kabs_bits);
    SelectResult sel;
    const bool windowed = hm.n_sel != hm.n;                  // (uniform) a local window is reserved inside the budget
    if (hm.k_sel == 0) {
        sel = select_nothing<WCTA>(tid, hm, keys, kmax, sc);
    } else {
        if (windowed) window_unhist<WCTA>(tid, hm, keys, hist1);
        if (!select_prefilled<WCTA>(tid, hm, keys, kmax, kabs, Z, sc, hist1, r, S_max, Kt_head, sel))
            sel = select_generic<WCTA>(tid, hm, keys, kmax, kabs, sc, r, S_max, Kt_head);
    }
    if (windowed) window_mark<WCTA>(tid, hm, sc);
    finish<WCTA, 4>(tid, hm, keys, kmax, sel, sc, k, K + kv_head * (size_t)S_max * D, V + kv_head * (size_t)S_max * D,
                    vbar + kv_head * D, out_row, idx_k ? idx_k + (size_t)bh * k : nullptr, alpha_out ? alpha_out + bh : nullptr,
                    true, opt_realloc(opts));
}

size_t wide_dynamic_smem(int S_max, int nt) {
    return wide_keys_bytes(S_max) + (size_t)FBINS * 4 +
           ((post_scratch_bytes(nt / 16, wide_bm_words(S_max)) + 127) & ~(size_t)127);
}

}  // namespace

bool wide_fits(int S_max, int smem_optin) {
    return wide_dynamic_smem(S_max, 512) + sizeof(WideShared<512>) + 1024 <= (size_t)smem_optin;
}
// two 256-thread CTAs of this S_max per SM (each CTA also costs 1 KB of the SM's shared memory)
bool wide_pair_fits(int S_max, int smem_per_sm) {
    return 2 * (wide_dynamic_smem(S_max, 256) + sizeof(WideShared<256>) + 1024) <= (size_t)smem_per_sm;
}

cudaError_t launch_sparq_decode_wide(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                     const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                     int r, int k, uint32_t opts, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                     int32_t* status, bool pairs, cudaStream_t stream) {
    const int nt = pairs ? 256 : 512;
    const size_t dyn = wide_dynamic_smem(S_max, nt);
    auto kernel = pairs ? sparq_decode_wide_kernel<256> : sparq_decode_wide_kernel<512>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    if (e != cudaSuccess) return e;
    kernel<<<B * Hq, nt, dyn, stream>>>(q, K, Kt, V, vbar, seq_lens, Hq, Hkv, S_max, r, k, opts, out, idx_r, idx_k, alpha, status);
    return cudaGetLastError();
}

}  // namespace sparq
