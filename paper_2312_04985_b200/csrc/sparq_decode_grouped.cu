// sparq_decode_grouped: the paper's grouped-query variant (Section 4, "Grouped query attention").
// The g query heads that share a KV head select together: Step 1 takes the top-r of |q| summed
// over the group, Step 2 the top-k of the approximate scores summed over the group; temperature,
// scores, attention and alpha stay per query head.  Grid (slices, batch x KV heads): the sequence of
// a group is cut into interleaved slices streamed by different CTAs (g1-g2); the CTA that draws the
// group's last ticket runs g3-g5 for the whole group.
//
//   g1  sum of |q| over the group per component, as exact integers (fp16 magnitudes in units of
//       2^-24), ranked by counting: ties go to the smaller component by construction
//   g2  the r selected Kt rows are streamed ONCE for the whole group; every position gets g fp32
//       chains of exact fp16 x fp16 products.  The chains go to a scratch buffer as order-preserving
//       keys (g x 4 bytes per position); each head's maximum and softmax denominator are
//       accumulated on the way (online, per thread)                                    (Eq. (7))
//   g3  every thread reads the chains back, forms log2 sum_h s_hat[h, t] (a log-sum-exp: scores below
//       fp32's range keep their order) and writes it as the position's selection key, filling the
//       histogram of the keys' top bits
//   g4  top-k of the summed scores (decode_common.cuh; equal keys go to the lowest positions)
//   g5  per head: alpha, gather of the k selected K/V rows (from L1/L2 after the first head),
//       exact attention, Step 3 (or not)                                        (Eqs. (8), (10))
//
// The summed scores are evaluated in fp32, so unlike the per-head path the selection is not re-decided
// in fp64: positions whose summed scores differ by less than the fp32 evaluation error (the chains'
// rounding bound over tau plus a few ulps of the logit's distance from the maximum) may swap against a
// float64 evaluation.
#include "decode_common.cuh"
#include "kernels.h"

namespace sparq {
namespace {

constexpr int NT = 256;
constexpr int CHG = NT * 8;              // positions a CTA covers per pass: 8 per thread
constexpr int GFB = 11;                  // first digit of the selection keys
constexpr int GFBINS = 1 << GFB;
using CTA = Group<NT, 0>;

// Optional per-stage cycle counters (thread 0 of every CTA, summed); compiled in only with
// -DSPARQ_PHASE_CLOCKS for tuning, never in the shipped library.
#ifdef SPARQ_PHASE_CLOCKS
__device__ unsigned long long g_group_clocks[16];
#define GCLK_INIT() long long gc_prev_ = clock64()
#define GCLK(i) do { if (threadIdx.x == 0) { long long gc_now_ = clock64(); atomicAdd(&g_group_clocks[i], (unsigned long long)(gc_now_ - gc_prev_)); gc_prev_ = gc_now_; } } while (0)
#else
#define GCLK_INIT()
#define GCLK(i)
#endif

struct GroupShared {
    HeadMeta hm;                          // the head being finished (g5); i1 and n are the group's
    int32_t i2[SPARQ_K_MAX];
    unsigned long long gkey[D];           // g1: ranking keys
    uint16_t qh[SPARQ_G_MAX][D + 8];      // per head: selected components' fp16 bits in i1 order
    alignas(16) uint16_t q16[SPARQ_G_MAX][D];   // per head: the whole query, fp16 bits (g5)
    float pL[SPARQ_G_MAX];                // per head: sum of the exact attention's softmax weights (g5)
    float inv_tau[SPARQ_G_MAX];
    uint32_t kmax[SPARQ_G_MAX];           // per head: largest chain, as a key
    float zsum[SPARQ_G_MAX];              // per head: softmax denominator relative to it
    float red[2 * CTA::NW];
    uint32_t redu[2 * CTA::NW];
    uint32_t res[4];
    uint32_t band[4];
    uint32_t cnt[4];
};

// |x| of an fp16 bit pattern in units of 2^-24, exactly (subnormals included)
__device__ __forceinline__ unsigned long long fixed_abs(uint16_t h) {
    const uint32_t e = (h >> 10) & 31u, m = h & 0x3ffu;
    return e ? (unsigned long long)(0x400u | m) << (e - 1) : (unsigned long long)m;
}

__device__ __forceinline__ void row_fma_plain(float (&acc)[8], uint4 v, uint16_t qj) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        fma_h(acc[2 * e], qj, (uint16_t)(w[e] & 0xffffu));
        fma_h(acc[2 * e + 1], qj, (uint16_t)(w[e] >> 16));
    }
}

template <int G>
__global__ void __launch_bounds__(NT, G >= 8 ? 1 : 2)
sparq_grouped_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                     const sparq_half* __restrict__ Kt, const sparq_half* __restrict__ V,
                     const sparq_half* __restrict__ vbar, const int32_t* __restrict__ seq_lens,
                     int Hkv, int S_max, int r, int k, uint32_t opts, int bm_words, int slices,
                     sparq_half* __restrict__ out, int32_t* __restrict__ idx_r, int32_t* __restrict__ idx_k,
                     float* __restrict__ alpha_out, int32_t* status, uint32_t* ws, uint32_t* ws_part,
                     unsigned int* ws_count) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    uint32_t* hist1 = reinterpret_cast<uint32_t*>(dyn_smem);              // later the select stage's list
    static_assert(GFBINS <= HIST_BINS, "the first-digit histogram aliases the select scratch's histogram");
    __shared__ GroupShared sh;
    HeadMeta& hm = sh.hm;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // one-dimensional grid: (batch, KV head) and slice, the slices of a group neighbours in launch order
    const int bk = (int)(blockIdx.x / (unsigned)slices), b = bk / Hkv, p = (int)(blockIdx.x % (unsigned)slices);
    const int Hq = Hkv * G;
    const size_t q_row0 = ((size_t)b * Hq + (size_t)(bk % Hkv) * G) * D;  // first query head of the group
    const int n = seq_lens[b];
    sparq_half* out0 = out + q_row0;
    float* alpha0 = alpha_out ? alpha_out + q_row0 / D : nullptr;

    if (n < 1 || n > S_max) {            // defined result, no trap (slice 0 writes it)
        if (p != 0) return;
        if (tid == 0) raise_status(status, SPARQ_DEV_BAD_SEQ_LEN);
        for (int i = tid; i < G * D; i += NT) out0[i] = 0;
        if (alpha0 && tid < G) alpha0[tid] = 0.f;
        if (idx_r) for (int j = tid; j < r; j += NT) idx_r[(size_t)bk * r + j] = -1;
        if (idx_k) for (int j = tid; j < k; j += NT) idx_k[(size_t)bk * k + j] = -1;
        return;
    }
    const int k_eff = min(k, n);
    GCLK_INIT();
    for (int i = tid; i < GFBINS / 4; i += NT) reinterpret_cast<uint4*>(hist1)[i] = make_uint4(0, 0, 0, 0);

    // ------------------------------------------------------------------ g1: group top-r, per-head tau
    uint16_t qbits[G];
    float aq[G];
    bool sel = false;
    if (tid < D) {
        unsigned long long sum = 0;
#pragma unroll
        for (int h = 0; h < G; ++h) {
            qbits[h] = q[q_row0 + (size_t)h * D + tid];
            sh.q16[h][tid] = qbits[h];
            aq[h] = fabsf(__half2float(__ushort_as_half(qbits[h])));
            sum += fixed_abs(qbits[h]);
        }
        sh.gkey[tid] = (sum << 7) | (unsigned long long)(D - 1 - tid);    // distinct keys: larger sum first, then smaller index
    } else {
#pragma unroll
        for (int h = 0; h < G; ++h) { qbits[h] = 0; aq[h] = 0.f; }
    }
    __syncthreads();
    if (tid < D) {
        const unsigned long long mine = sh.gkey[tid];
        int rank = 0;
#pragma unroll 8
        for (int j = 0; j < D; ++j) rank += sh.gkey[j] > mine;
        sel = rank < r;
    }
    const unsigned bal = __ballot_sync(FULL, sel);
    if (lane == 0 && warp < 4) sh.cnt[warp] = __popc(bal);
    __syncthreads();
    int slot = -1;
    if (sel) {
        slot = __popc(bal & ((1u << lane) - 1));
        for (int w = 0; w < warp; ++w) slot += sh.cnt[w];
        hm.i1[slot] = tid;                                   // ascending by construction
    }
    const int r_pad = (r + 7) & ~7;
#pragma unroll
    for (int h = 0; h < G; ++h) {
        if (sel) sh.qh[h][slot] = qbits[h];
        if (tid >= r && tid < r_pad) sh.qh[h][tid] = 0;
        float l1_all = aq[h], l1_sel = sel ? aq[h] : 0.f;
        group_sum2<CTA>(l1_all, l1_sel, sh.red, tid);
        // (a head with no weight on the group's components has all-zero approximate logits: tau := 1)
        if (tid == 0) sh.inv_tau[h] = opt_inv_tau(opts, l1_all, l1_sel, r);
    }
    if (tid == 0) { hm.bh = bk; hm.n = n; hm.k_eff = k_eff; hm.valid = 1; hm.l1_sel = 0.f; hm.inv_tau = 1.f; opt_set_window(hm, n, k_eff, opts); }
    __syncthreads();
    if (p == 0 && idx_r) for (int j = tid; j < r; j += NT) idx_r[(size_t)bk * r + j] = hm.i1[j];

    const sparq_half* vbar_head = vbar + (size_t)bk * D;
    if (k_eff == 0) {                    // nothing to select: every head's output is the mean value vector
        if (p != 0) return;
        for (int i = tid; i < G * D; i += NT) out0[i] = vbar_head[i % D];
        if (alpha0 && tid < G) alpha0[tid] = 0.f;
        return;
    }

    GCLK(0);
    // ------------------------------------------------------------------ g2: one stream for the whole group
    const sparq_half* Kt_head = Kt + (size_t)bk * D * S_max;
    uint32_t* ws_unit = ws + (size_t)bk * (G + 1) * S_max;                // [G][S_max] chains, then [S_max] selection keys
    uint32_t* keys_sum = ws_unit + (size_t)G * S_max;
    float c1[G], zm[G], zs[G];
    uint32_t kmx[G];
#pragma unroll
    for (int h = 0; h < G; ++h) { c1[h] = sh.inv_tau[h] * LOG2E; zm[h] = -CUDART_INF_F; zs[h] = 0.f; kmx[h] = 0; }
    const uint4* Kt_vec = reinterpret_cast<const uint4*>(Kt_head);
    const int row_vecs = S_max >> 3;
    const int n_pass = ((n + 7) / 8 + NT - 1) / NT;
    for (int c = p; c < n_pass; c += slices) {               // this CTA's passes: c = p, p + slices, ...
        const int t0 = c * CHG + tid * 8;
        const int nvalid = min(8, n - t0);
        if (nvalid <= 0) continue;                           // (the layout keeps zeros up to the end of the last vector)
        float acc[G][8];
#pragma unroll
        for (int h = 0; h < G; ++h)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[h][e] = 0.f;
        for (int jb = 0; jb < r; jb += 8) {
            uint4 v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = ld_stream(Kt_vec + (size_t)hm.i1[min(jb + u, r - 1)] * row_vecs + (t0 >> 3));
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (jb + u < r) {
#pragma unroll
                    for (int h = 0; h < G; ++h) row_fma_plain(acc[h], v[u], sh.qh[h][jb + u]);
                }
            }
        }
#pragma unroll
        for (int h = 0; h < G; ++h) {
            float cm = -CUDART_INF_F;
#pragma unroll
            for (int e = 0; e < 8; ++e) if (e < nvalid) cm = fmaxf(cm, acc[h][e] * c1[h]);
            const float nm = fmaxf(zm[h], cm);
            zs[h] *= ex2(zm[h] - nm);
#pragma unroll
            for (int e = 0; e < 8; ++e) if (e < nvalid) zs[h] += ex2(acc[h][e] * c1[h] - nm);
            zm[h] = nm;
            uint32_t kk[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) { kk[e] = key32(acc[h][e]); if (e < nvalid) kmx[h] = max(kmx[h], kk[e]); }
            uint32_t* dst = ws_unit + (size_t)h * S_max + t0;             // whole vectors: S_max is a multiple of 8
            *reinterpret_cast<uint4*>(dst) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
            *reinterpret_cast<uint4*>(dst + 4) = make_uint4(kk[4], kk[5], kk[6], kk[7]);
        }
    }
    GCLK(1);
    // per head: the CTA-wide maximum and the denominator relative to it
    float lz[G], vmax[G];                                    // per head: log2 of the denominator, the largest chain
#pragma unroll
    for (int h = 0; h < G; ++h) {
        uint32_t km = kmx[h], dummy = 0;
        group_max2_u32<CTA>(km, dummy, sh.redu, tid);
        const float Z = group_sum<CTA>(zs[h] > 0.f ? zs[h] * ex2(zm[h] - unkey32(km) * c1[h]) : 0.f, sh.red, tid);
        if (tid == 0) { sh.kmax[h] = km; sh.zsum[h] = Z; }
    }
    if (slices > 1) {
        // leave this slice's statistics, take a ticket; only the last CTA of the group goes on
        uint32_t* part = ws_part + ((size_t)bk * slices + p) * (2 * G);
        __syncthreads();
        if (tid < G) { part[2 * tid] = sh.kmax[tid]; part[2 * tid + 1] = __float_as_uint(sh.zsum[tid]); }
        __threadfence();                                     // this thread's chains and statistics: device-visible
        __syncthreads();
        if (tid == 0) sh.cnt[0] = atomicAdd(&ws_count[bk], 1u);
        __syncthreads();
        if (sh.cnt[0] != (uint32_t)(slices - 1)) return;
        __threadfence();
        if (tid < G) {                                       // merge the slices' statistics for head tid
            const uint32_t* p0 = ws_part + (size_t)bk * slices * (2 * G);
            uint32_t km = 0;
            for (int s_ = 0; s_ < slices; ++s_) km = max(km, __ldcg(p0 + (size_t)s_ * 2 * G + 2 * tid));
            const float vm = unkey32(km), cc = sh.inv_tau[tid] * LOG2E;
            float Z = 0.f;
            for (int s_ = 0; s_ < slices; ++s_) {
                const uint32_t ks = __ldcg(p0 + (size_t)s_ * 2 * G + 2 * tid);
                const float zp = __uint_as_float(__ldcg(p0 + (size_t)s_ * 2 * G + 2 * tid + 1));
                if (zp > 0.f) Z += zp * ex2((unkey32(ks) - vm) * cc);
            }
            sh.kmax[tid] = km; sh.zsum[tid] = Z;
        }
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < G; ++h) { vmax[h] = unkey32(sh.kmax[h]); lz[h] = __log2f(sh.zsum[h]); }

    GCLK(2);
    // ------------------------------------------------------------------ g3: summed scores as selection keys
    uint32_t smax = 0;
    for (int c = 0; c < n_pass; ++c) {                       // every position of the group, whoever streamed it
        const int t0 = c * CHG + tid * 8;
        const int nvalid = min(8, n - t0);
        if (nvalid <= 0) continue;
        // log2 of the summed scores: x_h = log2 s_hat[h, t], then max_h x_h + log2 sum_h 2^(x_h - max).  Ranking
        // the logarithm keeps the order of scores that would underflow as plain exponentials; for a group
        // of one it is the logit itself.
        float x[G][8], ssum[8];
#pragma unroll
        for (int h = 0; h < G; ++h) {
            const uint32_t* src = ws_unit + (size_t)h * S_max + t0;
            const uint4 a = __ldcg(reinterpret_cast<const uint4*>(src)), bq = __ldcg(reinterpret_cast<const uint4*>(src + 4));
            const uint32_t kk[8] = {a.x, a.y, a.z, a.w, bq.x, bq.y, bq.z, bq.w};
#pragma unroll
            for (int e = 0; e < 8; ++e) x[h][e] = (unkey32(kk[e]) - vmax[h]) * c1[h] - lz[h];
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            float mxe = x[0][e];
#pragma unroll
            for (int h = 1; h < G; ++h) mxe = fmaxf(mxe, x[h][e]);
            if constexpr (G == 1) {
                ssum[e] = mxe;
            } else {
                float acc2 = 0.f;
#pragma unroll
                for (int h = 0; h < G; ++h) acc2 += ex2(x[h][e] - mxe);
                ssum[e] = mxe + __log2f(acc2);
            }
        }
        uint32_t ks[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) ks[e] = key32(ssum[e]);
        *reinterpret_cast<uint4*>(keys_sum + t0) = make_uint4(ks[0], ks[1], ks[2], ks[3]);
        *reinterpret_cast<uint4*>(keys_sum + t0 + 4) = make_uint4(ks[4], ks[5], ks[6], ks[7]);
#pragma unroll
        for (int e = 0; e < 8; ++e)
            if (e < nvalid) { smax = max(smax, ks[e]); atomicAdd(&hist1[ks[e] >> (32 - GFB)], 1u); }
    }
    {
        uint32_t dummy = 0;
        group_max2_u32<CTA>(smax, dummy, sh.redu, tid);      // barriers: histogram and selection keys complete
    }

    GCLK(3);
    // ------------------------------------------------------------------ g4: top-k of the summed scores
    PostScratch sc;
    carve_post_scratch(sc, dyn_smem, CTA::NHW, bm_words);
    sc.i2 = sh.i2; sc.red = sh.red; sc.redu = sh.redu; sc.res = sh.res; sc.band = sh.band;
    SelectResult sel_res;
    // kabs = 0: no rounding-error band, only exactly equal keys compete (lowest positions win)
    const bool windowed = hm.n_sel != hm.n;                  // (uniform) a local window is reserved inside the budget
    if (hm.k_sel == 0) {                                     // the window takes the whole budget: nothing to rank
        sel_res = select_nothing<CTA>(tid, hm, keys_sum, smax, sc);
    } else {
        if (windowed) window_unhist<CTA, GFB>(tid, hm, keys_sum, hist1);
        if (!select_prefilled<CTA, GFB, true, true>(tid, hm, keys_sum, smax, 0.f, 1.f, sc, hist1, r, S_max, Kt_head, sel_res))
            sel_res = select_generic<CTA, true>(tid, hm, keys_sum, smax, 0.f, sc, r, S_max, Kt_head);
    }
    if (windowed) window_mark<CTA>(tid, hm, sc);

    GCLK(4);
    // ------------------------------------------------------------------ g5: alpha, exact attention, Step 3 -- all heads at once
    // Every selected K and V row is gathered once and serves the g heads: q.K for all heads per row
    // (scores to shared memory), per-head softmax weights, then the weighted V sums.
    const sparq_half* K_head = K + (size_t)bk * S_max * D;
    const sparq_half* V_head = V + (size_t)bk * S_max * D;
    build_index_list<CTA>(tid, hm, sel_res, sc);             // sc.i2 ascending; the select stage's scratch is dead from here
    for (int i = tid; i < 4 * k_eff; i += NT) {              // the rows on their way from HBM to L2 meanwhile
        const int t = min(max(sc.i2[i >> 2], 0), n - 1);
        const sparq_half* row = ((i & 2) ? V_head : K_head) + (size_t)t * D + (i & 1) * (D / 2);
        asm volatile("prefetch.global.L2 [%0];" ::"l"(row));
    }
    float* zsc = reinterpret_cast<float*>(dyn_smem);                      // [G][k_eff] scores, then weights
    float* slab = zsc + ((G * k_eff + 3) & ~3);                           // [warps][G][D] partial V sums
    float alpha[G];                                          // per head: approximate-score mass of the selected set (Step 3)
#pragma unroll
    for (int h = 0; h < G; ++h) {
        float part = 0.f;
        for (int j = tid; j < k_eff; j += NT)
            part += ex2((unkey32(__ldcg(ws_unit + (size_t)h * S_max + min(max(sc.i2[j], 0), n - 1))) - vmax[h]) * c1[h]);
        // (numerator and denominator are fp32 sums taken in different orders: keep the mass a probability)
        alpha[h] = fminf(group_sum<CTA>(part, sh.red, tid) / sh.zsum[h], 1.0f);
    }
    const int hw = tid >> 4, l16 = tid & 15;
    constexpr int RG = G >= 8 ? 2 : 4;                       // gathered rows in flight per half-warp
    {
        const float qscale = rsqrtf((float)D) * LOG2E;
        const uint4* Kh = reinterpret_cast<const uint4*>(K_head);
        for (int jb = 0; jb < k_eff; jb += CTA::NHW * RG) {  // trip count uniform across the CTA
            uint4 kv[RG];
#pragma unroll
            for (int u = 0; u < RG; ++u) {
                const int t = min(max(sc.i2[min(jb + u * CTA::NHW + hw, k_eff - 1)], 0), n - 1);
                kv[u] = ld_stream(Kh + (size_t)t * (D / 8) + l16);
            }
#pragma unroll
            for (int u = 0; u < RG; ++u) {
                const int j = jb + u * CTA::NHW + hw;
                const uint32_t kw[4] = {kv[u].x, kv[u].y, kv[u].z, kv[u].w};
#pragma unroll
                for (int h = 0; h < G; ++h) {
                    const uint4 q8 = *reinterpret_cast<const uint4*>(&sh.q16[h][l16 * 8]);
                    const uint32_t qw[4] = {q8.x, q8.y, q8.z, q8.w};
                    float zz = 0.f, zz2 = 0.f;               // exact fp16 products, two fp32 chains
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        fma_h(zz, (uint16_t)(kw[e] & 0xffffu), (uint16_t)(qw[e] & 0xffffu));
                        fma_h(zz2, (uint16_t)(kw[e] >> 16), (uint16_t)(qw[e] >> 16));
                    }
                    zz = (zz + zz2) * qscale;
#pragma unroll
                    for (int o = 8; o > 0; o >>= 1) zz += __shfl_xor_sync(FULL, zz, o);
                    if (l16 == 0 && j < k_eff) zsc[h * k_eff + j] = zz;
                }
            }
        }
    }
    __syncthreads();
    for (int h = warp; h < G; h += CTA::NW) {                // per head: maximum, weights in place, their sum
        float mx = -CUDART_INF_F;
        for (int j = lane; j < k_eff; j += 32) mx = fmaxf(mx, zsc[h * k_eff + j]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(FULL, mx, o));
        float l_ = 0.f;
        for (int j = lane; j < k_eff; j += 32) { const float w_ = ex2(zsc[h * k_eff + j] - mx); zsc[h * k_eff + j] = w_; l_ += w_; }
        l_ = warp_sum(l_);
        if (lane == 0) sh.pL[h] = l_;
    }
    __syncthreads();
    {
        float acc[G][8];
#pragma unroll
        for (int h = 0; h < G; ++h)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[h][e] = 0.f;
        const uint4* Vh = reinterpret_cast<const uint4*>(V_head);
        for (int jb = 0; jb < k_eff; jb += CTA::NHW * RG) {
            uint4 vv[RG];
#pragma unroll
            for (int u = 0; u < RG; ++u) {
                const int t = min(max(sc.i2[min(jb + u * CTA::NHW + hw, k_eff - 1)], 0), n - 1);
                vv[u] = ld_stream(Vh + (size_t)t * (D / 8) + l16);
            }
#pragma unroll
            for (int u = 0; u < RG; ++u) {
                const int j = jb + u * CTA::NHW + hw;
                if (j < k_eff) {
                    const __half2* vh = reinterpret_cast<const __half2*>(&vv[u]);
                    float2 f[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) f[e] = __half22float2(vh[e]);
#pragma unroll
                    for (int h = 0; h < G; ++h) {
                        const float w_ = zsc[h * k_eff + j];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            acc[h][2 * e] = fmaf(w_, f[e].x, acc[h][2 * e]);
                            acc[h][2 * e + 1] = fmaf(w_, f[e].y, acc[h][2 * e + 1]);
                        }
                    }
                }
            }
        }
        // the two half-warps of a warp, then the warps through shared memory (fixed order: reproducible)
#pragma unroll
        for (int h = 0; h < G; ++h)
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[h][e] += __shfl_xor_sync(FULL, acc[h][e], 16);
        if (lane < 16) {
#pragma unroll
            for (int h = 0; h < G; ++h) {
                float4* dst = reinterpret_cast<float4*>(slab + ((size_t)warp * G + h) * D + l16 * 8);
                dst[0] = make_float4(acc[h][0], acc[h][1], acc[h][2], acc[h][3]);
                dst[1] = make_float4(acc[h][4], acc[h][5], acc[h][6], acc[h][7]);
            }
        }
    }
    __syncthreads();
    for (int i = tid; i < G * D; i += NT) {                  // Eq. (10) per head (or Eq. (8) alone)
        const int h = i / D, c = i % D;
        float s_ = 0.f;
#pragma unroll
        for (int w = 0; w < CTA::NW; ++w) s_ += slab[((size_t)w * G + h) * D + c];
        const float y3 = s_ / sh.pL[h];
        float a_ = alpha[0];
#pragma unroll
        for (int hh = 1; hh < G; ++hh) a_ = (h == hh) ? alpha[hh] : a_;
        const float vb = __half2float(__ushort_as_half(vbar_head[c]));
        out0[i] = __half_as_ushort(__float2half_rn(opt_realloc(opts) ? a_ * y3 + (1.f - a_) * vb : y3));
        if (c == 0 && alpha0) alpha0[h] = a_;
    }
    if (idx_k) for (int j = tid; j < k; j += NT) idx_k[(size_t)bk * k + j] = (j < k_eff) ? sc.i2[j] : -1;
    GCLK(5);
}

int grouped_bm_words(int S_max) { return (S_max + 127) / 128 * 4; }

template <int G>
cudaError_t launch_g(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                     const sparq_half* vbar, const int32_t* seq_lens, int B, int Hkv, int S_max, int r, int k, uint32_t opts,
                     sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha, int32_t* status, uint32_t* ws,
                     int slices, cudaStream_t stream) {
    const int groups = B * Hkv;
    uint32_t* ws_part = ws + (size_t)groups * (G + 1) * S_max;
    unsigned int* ws_count = ws_part + (size_t)groups * slices * 2 * G;
    const size_t dyn = grouped_dynamic_smem(S_max, G, k);
    cudaError_t e = cudaFuncSetAttribute(sparq_grouped_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    if (e != cudaSuccess) return e;
    if (slices > 1) {
        e = cudaMemsetAsync(ws_count, 0, (size_t)groups * sizeof(unsigned int), stream);
        if (e != cudaSuccess) return e;
    }
    sparq_grouped_kernel<G><<<(unsigned)slices * (unsigned)groups, NT, dyn, stream>>>(q, K, Kt, V, vbar, seq_lens, Hkv, S_max, r, k, opts,
                                                                      grouped_bm_words(S_max), slices, out, idx_r, idx_k,
                                                                      alpha, status, ws, ws_part, ws_count);
    return cudaGetLastError();
}

}  // namespace

#ifdef SPARQ_PHASE_CLOCKS
extern "C" int sparq_debug_group_clocks(unsigned long long* out16, int reset) {
    cudaDeviceSynchronize();
    if (out16 && cudaMemcpyFromSymbol(out16, g_group_clocks, sizeof(unsigned long long) * 16) != cudaSuccess) return 1;
    if (reset) { unsigned long long z[16] = {0}; if (cudaMemcpyToSymbol(g_group_clocks, z, sizeof(z)) != cudaSuccess) return 1; }
    return 0;
}
#endif

// The select stages' scratch, or -- later, in the same space -- the fused last stage's scores [g][k]
// and partial V sums [warps][g][d_h], whichever is larger.
size_t grouped_dynamic_smem(int S_max, int g, int k) {
    const size_t select_bytes = post_scratch_bytes(CTA::NHW, grouped_bm_words(S_max));
    const size_t fused_bytes = ((((size_t)g * k + 3) & ~(size_t)3) + (size_t)CTA::NW * g * D) * sizeof(float);
    return ((select_bytes > fused_bytes ? select_bytes : fused_bytes) + 127) & ~(size_t)127;
}

// Slices per group.  With at least one group per SM the groups are left whole: the stages after the
// stream (one CTA per group) weigh too much for slicing to pay (measured on 256 groups: 84 us whole,
// 121 us in three slices).  Fewer groups than SMs: about two waves of resident CTAs (two per SM), at
// least one pass of CHG positions per slice (128 groups: 173 us in five slices, 207 us whole).
int grouped_slices(int groups, int S_max, int n_sm) {
    if (n_sm <= 0 || groups >= n_sm) return 1;
    const int want = (4 * n_sm + groups - 1) / groups;
    const int cap = (S_max + CHG - 1) / CHG;
    const int s = want < cap ? want : cap;
    return s < 1 ? 1 : s;
}

// chains [g][S_max] and selection keys [S_max] per group; per-slice statistics; ticket counters
size_t grouped_scratch_bytes(int B, int Hq, int Hkv, int S_max, int slices) {
    const size_t groups = (size_t)B * Hkv, g = (size_t)(Hq / Hkv);
    return (groups * (g + 1) * S_max + groups * slices * 2 * g + groups) * sizeof(uint32_t);
}

cudaError_t launch_sparq_decode_grouped(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                        const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                        int r, int k, uint32_t opts, sparq_half* out, int32_t* idx_r, int32_t* idx_k,
                                        float* alpha, int32_t* status, void* scratch, int slices, cudaStream_t stream) {
    uint32_t* ws = static_cast<uint32_t*>(scratch);
    switch (Hq / Hkv) {
        case 1: return launch_g<1>(q, K, Kt, V, vbar, seq_lens, B, Hkv, S_max, r, k, opts, out, idx_r, idx_k, alpha, status, ws, slices, stream);
        case 2: return launch_g<2>(q, K, Kt, V, vbar, seq_lens, B, Hkv, S_max, r, k, opts, out, idx_r, idx_k, alpha, status, ws, slices, stream);
        case 4: return launch_g<4>(q, K, Kt, V, vbar, seq_lens, B, Hkv, S_max, r, k, opts, out, idx_r, idx_k, alpha, status, ws, slices, stream);
        case 8: return launch_g<8>(q, K, Kt, V, vbar, seq_lens, B, Hkv, S_max, r, k, opts, out, idx_r, idx_k, alpha, status, ws, slices, stream);
        default: return cudaErrorInvalidValue;
    }
}

}  // namespace sparq
