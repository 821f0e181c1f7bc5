// sparq_decode, one CTA per (batch, query head) fed by a ring of bulk copies (any S_max whose score
// keys fit in shared memory beside the ring), and -- further down -- the split plan for caches
// beyond shared memory.  Every stage is fused so that only the compulsory bytes touch HBM.  (The
// ring kernel runs only when forced: the wide kernel of sparq_decode_wide.cu is faster at every
// shape; it stays as an independent implementation for the tests to compare the others with.)
//
//   a1  top-r of |q| by rank counting on integer keys; tau                    (Step 1, Eq. (9))
//   a2  stream the r selected rows of Kt through a ring of bulk asynchronous copies
//       (cp.async.bulk + mbarrier, no multicast).  Each position's sum over the r components
//       is an fp32 chain of mixed-precision FMAs (fp16 x fp16 products are exact in fp32), kept
//       on chip as an order-preserving 32-bit key: 4 bytes/position of shared memory.  The
//       largest |K| seen gives a rigorous bound B on every sum's rounding error   (Eq. (7))
//   a3-a6  post phase (decode_common.cuh): radix select of the k largest keys with fp64
//       re-decision of the positions within 2B of the threshold, softmax statistics and alpha,
//       K/V row gather with online softmax, combine with v_bar          (Steps 2-3, Eqs. (8), (10))
#include "decode_common.cuh"
#include "kernels.h"

namespace sparq {
namespace {

constexpr int NT = 256;                  // threads per CTA
constexpr int CH = NT * 8;               // positions per chunk: 8 per thread (one 16-byte vector)
constexpr int RB = 4;                    // Kt rows per pipeline stage
constexpr int STAGES = 3;
constexpr int STAGE_BYTES = RB * CH * 2;
constexpr int RING_BYTES = STAGES * STAGE_BYTES;
constexpr int BM_WORDS = 2048;           // bitmap capacity: 65536 positions
using CTA = Group<NT, 0>;

static_assert(post_scratch_bytes(CTA::NHW, BM_WORDS) <= RING_BYTES, "post-phase scratch must fit the dead ring");
static_assert(RB <= 8, "HeadMeta::qh padding");


// Optional per-phase cycle counters (thread 0 of every CTA, summed over CTAs); compiled in only
// with -DSPARQ_PHASE_CLOCKS for tuning, never in the shipped library.
#ifdef SPARQ_PHASE_CLOCKS
__device__ unsigned long long g_phase_clocks[16];
#define PHASE_INIT() long long t_prev_ = clock64()
#define PHASE_MARK(i)                                                                     \
    do {                                                                                  \
        if (threadIdx.x == 0) {                                                           \
            long long t_now_ = clock64();                                                 \
            atomicAdd(&g_phase_clocks[i], (unsigned long long)(t_now_ - t_prev_));        \
            t_prev_ = t_now_;                                                             \
        }                                                                                 \
    } while (0)
#else
#define PHASE_INIT()
#define PHASE_MARK(i)
#endif

struct DecodeShared {
    HeadMeta hm;
    int32_t i2[SPARQ_K_MAX];
    uint64_t full[STAGES];        // mbarriers: stage s has landed
    float red[2 * CTA::NW];
    uint32_t redu[2 * CTA::NW];
    uint32_t res[4];
    uint32_t band[4];
};

__global__ void __launch_bounds__(NT, 3)
sparq_decode_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                    const sparq_half* __restrict__ Kt, const sparq_half* __restrict__ V,
                    const sparq_half* __restrict__ vbar, const int32_t* __restrict__ seq_lens,
                    int Hq, int Hkv, int S_max, int r, int k,
                    sparq_half* __restrict__ out, int32_t* __restrict__ idx_r, int32_t* __restrict__ idx_k,
                    float* __restrict__ alpha_out, int32_t* status, uint32_t opts) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    unsigned char* ring = dyn_smem;                                       // a2: STAGES x [RB rows x CH positions] fp16
    uint32_t* keys = reinterpret_cast<uint32_t*>(dyn_smem + RING_BYTES);  // [n] approximate-score keys
    __shared__ DecodeShared sh;
    HeadMeta& hm = sh.hm;

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
    PHASE_INIT();
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) mbar_init(&sh.full[s], 1);
        mbar_init_fence();
        hm.bh = bh; hm.n = n; hm.k_eff = k_eff; hm.valid = 1;
        opt_set_window(hm, n, k_eff, opts);
    }

    top_r_block<CTA, RB>(tid, q + (size_t)bh * D, r, hm, sh.red, sh.res, opts);  // a1
    const int r_pad = (r + RB - 1) / RB * RB;
    if (idx_r) for (int j = tid; j < r; j += NT) idx_r[(size_t)bh * r + j] = hm.i1[j];

    PHASE_MARK(0);
    if (k_eff == 0) {                    // nothing to select: the output is the mean value vector
        if (tid < D) out_row[tid] = vbar[kv_head * D + tid];
        if (tid == 0 && alpha_out) alpha_out[bh] = 0.f;
        return;
    }

    const sparq_half* Kt_head = Kt + kv_head * (size_t)D * S_max;
    uint32_t kmax = 0, kabs_bits = 0;
    // ------------------------------------------------------------------ a2: stream r rows of Kt
    const int n8 = (n + 7) & ~7;                             // whole 16-byte vectors; n8 <= S_max
    const int n_chunks = (n8 + CH - 1) / CH;
    const int nb = r_pad / RB;
    const int total = n_chunks * nb;
    // Warp 0 refills a slot: lane 0 arms the barrier, then lanes 0..rows-1 each issue one row's
    // copy (one thread can only start a bulk copy every few hundred cycles; lanes overlap).
    auto issue = [&](int it, int s) {
        const int c = it / nb, jb = (it - c * nb) * RB;
        const uint32_t bytes = (uint32_t)min(CH, n8 - c * CH) * 2u;
        const int rows = min(RB, r - jb);
        if (lane == 0) mbar_expect_tx(&sh.full[s], bytes * rows);
        __syncwarp();
        if (lane < rows)
            bulk_g2s(ring + s * STAGE_BYTES + lane * (CH * 2), Kt_head + (size_t)hm.i1[jb + lane] * S_max + c * CH, bytes,
                     &sh.full[s]);
    };
    if (warp == 0) for (int it = 0; it < min(STAGES, total); ++it) issue(it, it);

    __half2 mx[4];                                           // largest |K| among the valid streamed values
#pragma unroll
    for (int e = 0; e < 4; ++e) mx[e] = __float2half2_rn(0.f);
    bool ok = true;
    int it = 0, s = 0;
    uint32_t parity = 0;
    for (int c = 0; c < n_chunks; ++c) {
        float acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        const int t0 = c * CH + tid * 8;
        const int nvalid = min(8, n - t0);                   // positions of this thread's vector inside the sequence
        __half2 mxc[4];                                      // |K| maximum of this chunk, kept only if the vector is inside
#pragma unroll
        for (int e = 0; e < 4; ++e) mxc[e] = __float2half2_rn(0.f);
        for (int jb = 0; jb < r_pad; jb += RB, ++it) {
            ok = mbar_wait_bounded(&sh.full[s], parity, WAIT_LIMIT);
            stage_fma<RB, CH / 8>(acc, mxc, reinterpret_cast<const uint4*>(ring + s * STAGE_BYTES) + tid, hm.qh + jb, r - jb);
            ok = __syncthreads_and(ok);                      // slot s fully consumed (or a wait gave up)
            if (!ok) break;
            if (warp == 0 && it + STAGES < total) issue(it + STAGES, s);
            if (++s == STAGES) { s = 0; parity ^= 1u; }
        }
        if (!ok) break;
        if (nvalid > 0) {
#pragma unroll
            for (int e = 0; e < 4; ++e) mx[e] = __hmax2(mx[e], mxc[e]);
        }
        uint32_t kk[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) kk[e] = key32(acc[e]);
        if (nvalid >= 8) {
            *reinterpret_cast<uint4*>(keys + t0) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
            *reinterpret_cast<uint4*>(keys + t0 + 4) = make_uint4(kk[4], kk[5], kk[6], kk[7]);
#pragma unroll
            for (int e = 0; e < 8; ++e) kmax = max(kmax, kk[e]);
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) if (e < nvalid) { keys[t0 + e] = kk[e]; kmax = max(kmax, kk[e]); }
        }
    }
    if (!ok) {                           // a bulk copy never landed: report, define the output, leave
        if (tid == 0) { raise_status(status, SPARQ_DEV_TIMEOUT); if (alpha_out) alpha_out[bh] = 0.f; }
        if (tid < D) out_row[tid] = 0;
        if (idx_k) for (int j = tid; j < k; j += NT) idx_k[(size_t)bh * k + j] = -1;
        return;
    }
    PHASE_MARK(1);
    kabs_bits = __float_as_uint(mx_to_float(mx));
    group_max2_u32<CTA>(kmax, kabs_bits, sh.redu, tid);      // barriers: keys complete, ring is dead

    // ------------------------------------------------------------------ a3-a6 (scratch in the dead ring)
    PostScratch sc;
    carve_post_scratch(sc, ring, CTA::NHW, BM_WORDS);
    sc.i2 = sh.i2; sc.red = sh.red; sc.redu = sh.redu; sc.res = sh.res; sc.band = sh.band;
    const SelectResult sel_res = hm.k_sel == 0 ? select_nothing<CTA>(tid, hm, keys, kmax, sc)
                                               : select_generic<CTA>(tid, hm, keys, kmax, __uint_as_float(kabs_bits), sc, r, S_max, Kt_head);
    if (hm.n_sel != hm.n) window_mark<CTA>(tid, hm, sc);
    finish<CTA, 8>(tid, hm, keys, kmax, sel_res, sc, k, K + kv_head * (size_t)S_max * D, V + kv_head * (size_t)S_max * D,
                   vbar + kv_head * D, out_row, idx_k ? idx_k + (size_t)bh * k : nullptr, alpha_out ? alpha_out + bh : nullptr,
                   true, opt_realloc(opts));
    PHASE_MARK(2);
}

// ---------------------------------------------------------------------------------- split-S plan
// For fewer (batch, head) units than SMs (batch-1 decode over a long cache) and for caches whose
// keys do not fit the persistent kernel's shared memory: one CTA per (unit, slice), 128 threads, five
// CTAs per SM.  Every unit's sequence is cut into `splits` interleaved slices; each CTA repeats
// a1 (cheap) and streams its slice of the r selected Kt rows with plain 128-bit loads (16 rows in
// flight per thread).  The keys go to a scratch buffer in global memory; the histogram of their top
// SPLIT_FB bits, the largest key, the largest |K| and the softmax denominator stay in the CTA.
//   splits == 1: the CTA goes straight on to a3-a6 with the keys it just wrote (they are read back
//     out of the L2 while other CTAs of the SM stream: occupancy overlaps the two kinds of work).
//   splits > 1: every CTA also leaves its histogram and statistics in the scratch buffer and takes a
//     ticket from the unit's counter; the CTA that draws the last ticket sums the slices' histograms
//     and runs a3-a6 for the unit.
// The selection runs on the same keys with the same rules as in the other plans, so the selected
// set is exactly theirs.
constexpr int FNT = 128;                 // threads of a split-plan CTA
constexpr int SCH = FNT * 8;             // positions a CTA covers per pass
constexpr int SROWS = 16;                // Kt rows in flight per thread (16 with five CTAs per SM measured best)
constexpr int SPLIT_CTAS = 5;            // resident CTAs per SM the kernel is compiled for
constexpr int SPLIT_FB = 11;             // long sequences: a finer first digit keeps the threshold bin's list short
constexpr int SPLIT_FBINS = 1 << SPLIT_FB;
constexpr int PART_WORDS = 4;            // per (unit, slice): largest key, largest |K| bits, Z bits, unused
using FCTA = Group<FNT, 0>;

struct SplitShared {
    HeadMeta hm;
    int32_t i2[SPARQ_K_MAX];
    float red[2 * FCTA::NW];
    uint32_t redu[2 * FCTA::NW];
    uint32_t res[4];
    uint32_t band[4];
    uint32_t cnt[4];
    uint32_t ticket;
    alignas(16) uint16_t qmask[D];   // ONE_K: q with the components outside i1 zeroed (read as 16-byte vectors)
};

// ONE_K: the variant that stores K once (no transposed copy): stage a2 reads whole rows of K, a
// half-warp per position, and multiplies by the masked query; everything after it is unchanged.
template <bool ONE_K>
__global__ void __launch_bounds__(FNT, SPLIT_CTAS)
sparq_split_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                   const sparq_half* __restrict__ Kt, const sparq_half* __restrict__ V,
                   const sparq_half* __restrict__ vbar, const int32_t* __restrict__ seq_lens,
                   int Hq, int Hkv, int S_max, int r, int k, int splits, int bm_words,
                   sparq_half* __restrict__ out, int32_t* __restrict__ idx_r, int32_t* __restrict__ idx_k,
                   float* __restrict__ alpha_out, int32_t* status,
                   uint32_t* ws_keys, uint32_t* ws_part, uint32_t* ws_hist, unsigned int* ws_count, uint32_t opts) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    // histogram of the keys' top bits; once the threshold bin is known the space becomes the select stage's list
    uint32_t* hist1 = reinterpret_cast<uint32_t*>(dyn_smem);
    static_assert(SPLIT_FBINS <= HIST_BINS, "the first-digit histogram aliases the select scratch's histogram");
    __shared__ SplitShared sh;
    HeadMeta& hm = sh.hm;
    // one-dimensional grid (no 65535 limit on the units): the slices of a unit are neighbours in launch order
    const int tid = threadIdx.x, p = (int)(blockIdx.x % (unsigned)splits), bh = (int)(blockIdx.x / (unsigned)splits);
    const int b = bh / Hq, h = bh % Hq, hkv = h / (Hq / Hkv);
    const int n = seq_lens[b];
    const size_t kv_head = (size_t)b * Hkv + hkv;
    sparq_half* out_row = out + (size_t)bh * D;

    if (n < 1 || n > S_max) {            // defined result, no trap (slice 0 writes it)
        if (p == 0) {
            if (tid == 0) { raise_status(status, SPARQ_DEV_BAD_SEQ_LEN); if (alpha_out) alpha_out[bh] = 0.f; }
            if (tid < D) out_row[tid] = 0;
            if (idx_r) for (int j = tid; j < r; j += FNT) idx_r[(size_t)bh * r + j] = -1;
            if (idx_k) for (int j = tid; j < k; j += FNT) idx_k[(size_t)bh * k + j] = -1;
        }
        return;
    }
    const int k_eff = min(k, n);
    PHASE_INIT();
    for (int i = tid; i < SPLIT_FBINS / 4; i += FNT) reinterpret_cast<uint4*>(hist1)[i] = make_uint4(0, 0, 0, 0);
    if (tid == 0) { hm.bh = bh; hm.n = n; hm.k_eff = k_eff; hm.valid = 1; opt_set_window(hm, n, k_eff, opts); }
    top_r_block<FCTA, 8>(tid, q + (size_t)bh * D, r, hm, sh.red, sh.cnt, opts);   // a1; its barriers also publish the cleared histogram
    if (p == 0 && idx_r) for (int j = tid; j < r; j += FNT) idx_r[(size_t)bh * r + j] = hm.i1[j];
    if (k_eff == 0) {                    // nothing to select: the output is the mean value vector
        if (p == 0) {
            if (tid < D) out_row[tid] = vbar[kv_head * D + tid];
            if (tid == 0 && alpha_out) alpha_out[bh] = 0.f;
        }
        return;
    }
    PHASE_MARK(0);

    // ------------------------------------------------------------------ a2 (+ a3 statistics) over this CTA's slice
    const sparq_half* Kt_head = ONE_K ? nullptr : Kt + kv_head * (size_t)D * S_max;
    uint32_t* keys = ws_keys + (size_t)bh * S_max;
    const float c1 = hm.inv_tau * LOG2E;
    uint32_t kmax = 0;
    float zm = -CUDART_INF_F, zs = 0.f;                      // running max (log2 units) and sum of 2^(x - zm)
    __half2 mx[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) mx[e] = __float2half2_rn(0.f);
    if constexpr (ONE_K) {
        // the masked query, then rows of K: lane l of a half-warp owns components 8l .. 8l+7
        if (tid < D) sh.qmask[tid] = 0;
        __syncthreads();
        if (tid < r) sh.qmask[hm.i1[tid]] = hm.qh[tid];
        __syncthreads();
        const int hw = tid >> 4, l16 = tid & 15;
        const uint4 qm = *reinterpret_cast<const uint4*>(sh.qmask + l16 * 8);
        const uint32_t qw[4] = {qm.x, qm.y, qm.z, qm.w};
        const uint4* Kh = reinterpret_cast<const uint4*>(K + kv_head * (size_t)S_max * D);
        const int n_pass = (n + SCH - 1) / SCH;
        for (int c = p; c < n_pass; c += splits) {
            for (int i0 = 0; i0 < SCH / (FNT / 16); i0 += 4) {           // four rows in flight per half-warp
                uint4 v[4];
                int t[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    t[u] = c * SCH + (i0 + u) * (FNT / 16) + hw;
                    v[u] = t[u] < n ? ld_stream(Kh + (size_t)t[u] * (D / 8) + l16) : make_uint4(0u, 0u, 0u, 0u);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const uint32_t w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
                    float part = 0.f;
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        fma_h(part, (uint16_t)(qw[e] & 0xffffu), (uint16_t)(w[e] & 0xffffu));
                        fma_h(part, (uint16_t)(qw[e] >> 16), (uint16_t)(w[e] >> 16));
                        mx[e] = __hmax2(mx[e], __habs2(*reinterpret_cast<const __half2*>(&w[e])));
                    }
#pragma unroll
                    for (int o = 8; o > 0; o >>= 1) part += __shfl_xor_sync(FULL, part, o, 16);
                    if (l16 == 0 && t[u] < n) {
                        const uint32_t kk = key32(part);
                        keys[t[u]] = kk;
                        kmax = max(kmax, kk);
                        atomicAdd(&hist1[kk >> (32 - SPLIT_FB)], 1u);
                        const float cm = part * c1;
                        if (cm > zm) { zs *= ex2(zm - cm); zm = cm; }
                        zs += ex2(cm - zm);
                    }
                }
            }
        }
    } else
    {
        const uint4* Kt_vec = reinterpret_cast<const uint4*>(Kt_head);
        const int row_vecs = S_max >> 3;
        const int n_pass = ((n + 7) / 8 + FNT - 1) / FNT;    // passes of SCH positions over the whole sequence
        for (int c = p; c < n_pass; c += splits) {           // this CTA's passes: c = p, p + splits, ...
            const int t0 = c * SCH + tid * 8;
            const int nvalid = min(8, n - t0);
            if (nvalid <= 0) continue;                       // (the layout keeps zeros up to the end of the last vector)
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
            for (int jb = 0; jb < r; jb += SROWS) {
                uint4 v[SROWS];
#pragma unroll
                for (int u = 0; u < SROWS; ++u) v[u] = ld_stream(Kt_vec + (size_t)hm.i1[min(jb + u, r - 1)] * row_vecs + (t0 >> 3));
#pragma unroll
                for (int u = 0; u < SROWS; ++u)
                    if (jb + u < r) row_fma(acc, mx, v[u], hm.qh[jb + u]);
            }
            float cm = -CUDART_INF_F;                        // softmax statistics of these keys, online
#pragma unroll
            for (int e = 0; e < 8; ++e) if (e < nvalid) cm = fmaxf(cm, acc[e] * c1);
            const float nm = fmaxf(zm, cm);
            zs *= ex2(zm - nm);
#pragma unroll
            for (int e = 0; e < 8; ++e) if (e < nvalid) zs += ex2(acc[e] * c1 - nm);
            zm = nm;
            uint32_t kk[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) kk[e] = key32(acc[e]);
            if (nvalid >= 8) {
                *reinterpret_cast<uint4*>(keys + t0) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
                *reinterpret_cast<uint4*>(keys + t0 + 4) = make_uint4(kk[4], kk[5], kk[6], kk[7]);
            }
#pragma unroll
            for (int e = 0; e < 8; ++e)
                if (e < nvalid) {
                    if (nvalid < 8) keys[t0 + e] = kk[e];
                    kmax = max(kmax, kk[e]);
                    atomicAdd(&hist1[kk[e] >> (32 - SPLIT_FB)], 1u);
                }
        }
    }
    uint32_t kabs_bits = __float_as_uint(mx_to_float(mx));
    group_max2_u32<FCTA>(kmax, kabs_bits, sh.redu, tid);     // barriers: the histogram and this CTA's keys are complete
    // the slice's denominator relative to its own largest key
    float Z = group_sum<FCTA>(zs > 0.f ? zs * ex2(zm - unkey32(kmax) * c1) : 0.f, sh.red, tid);
    PHASE_MARK(1);

    if (splits > 1) {
        // leave this slice's results, take a ticket; only the last CTA of the unit goes on
        const size_t slice0 = (size_t)bh * splits;
        if (tid == 0)
            *reinterpret_cast<uint4*>(ws_part + (slice0 + p) * PART_WORDS) = make_uint4(kmax, kabs_bits, __float_as_uint(Z), 0u);
        uint4* hdst = reinterpret_cast<uint4*>(ws_hist + (slice0 + p) * SPLIT_FBINS);
        for (int i = tid; i < SPLIT_FBINS / 4; i += FNT) hdst[i] = reinterpret_cast<const uint4*>(hist1)[i];
        __threadfence();                                     // this thread's keys, histogram words, statistics: device-visible
        __syncthreads();
        if (tid == 0) sh.ticket = atomicAdd(&ws_count[bh], 1u);
        __syncthreads();
        if (sh.ticket != (uint32_t)(splits - 1)) return;
        __threadfence();
        // the unit's histogram: all slices summed (L2 reads: other SMs wrote them)
        const uint4* hsrc = reinterpret_cast<const uint4*>(ws_hist + slice0 * SPLIT_FBINS);
        for (int i = tid; i < SPLIT_FBINS / 4; i += FNT) {
            uint4 s4 = __ldcg(hsrc + i);
            for (int pp = 1; pp < splits; ++pp) {
                const uint4 o = __ldcg(hsrc + (size_t)pp * (SPLIT_FBINS / 4) + i);
                s4.x += o.x; s4.y += o.y; s4.z += o.z; s4.w += o.w;
            }
            reinterpret_cast<uint4*>(hist1)[i] = s4;
        }
        // largest key and |K| over the slices, then the denominators rescaled to the largest key
        kmax = 0; kabs_bits = 0;
        for (int pp = tid; pp < splits; pp += FNT) {
            const uint4 part = __ldcg(reinterpret_cast<const uint4*>(ws_part + (slice0 + pp) * PART_WORDS));
            kmax = max(kmax, part.x);
            kabs_bits = max(kabs_bits, part.y);
        }
        group_max2_u32<FCTA>(kmax, kabs_bits, sh.redu, tid);
        const float vmax = unkey32(kmax);
        float zpart = 0.f;
        for (int pp = tid; pp < splits; pp += FNT) {
            const uint4 part = __ldcg(reinterpret_cast<const uint4*>(ws_part + (slice0 + pp) * PART_WORDS));
            const float zp = __uint_as_float(part.z);
            if (zp > 0.f) zpart += zp * ex2((unkey32(part.x) - vmax) * c1);
        }
        Z = group_sum<FCTA>(zpart, sh.red, tid);             // barriers: the summed histogram is complete as well
    }

    // ------------------------------------------------------------------ a3-a6 with the keys in global memory
    PostScratch sc;
    carve_post_scratch(sc, dyn_smem, FCTA::NHW, bm_words);
    sc.i2 = sh.i2; sc.red = sh.red; sc.redu = sh.redu; sc.res = sh.res; sc.band = sh.band;
    const float kabs = __uint_as_float(kabs_bits);
    SelectResult sel;
    // where the fp64 re-decision finds component c of position t: Kt[c * S_max + t], or K[t * d_h + c]
    const sparq_half* band_src = ONE_K ? K + kv_head * (size_t)S_max * D : Kt_head;
    const int c_stride = ONE_K ? 1 : S_max, t_stride = ONE_K ? D : 1;
    const bool windowed = hm.n_sel != hm.n;                  // (uniform) a local window is reserved inside the budget
    if (hm.k_sel == 0) {
        sel = select_nothing<FCTA>(tid, hm, keys, kmax, sc);
    } else {
        if (windowed) window_unhist<FCTA, SPLIT_FB>(tid, hm, keys, hist1);
        if (!select_prefilled<FCTA, SPLIT_FB, true>(tid, hm, keys, kmax, kabs, Z, sc, hist1, r, c_stride, band_src, sel, t_stride)) {
#ifdef SPARQ_PHASE_CLOCKS
            if (tid == 0) atomicAdd(&g_phase_clocks[7], 1ull);
#endif
            sel = select_generic<FCTA>(tid, hm, keys, kmax, kabs, sc, r, c_stride, band_src, t_stride);
        }
    }
    if (windowed) window_mark<FCTA>(tid, hm, sc);
    PHASE_MARK(2);
    finish<FCTA, 4>(tid, hm, keys, kmax, sel, sc, k, K + kv_head * (size_t)S_max * D, V + kv_head * (size_t)S_max * D,
                    vbar + kv_head * D, out_row, idx_k ? idx_k + (size_t)bh * k : nullptr, alpha_out ? alpha_out + bh : nullptr,
                    true, opt_realloc(opts));
    PHASE_MARK(3);
}

}  // namespace

#ifdef SPARQ_PHASE_CLOCKS
extern "C" int sparq_debug_phase_clocks(unsigned long long* out16, int reset) {
    cudaDeviceSynchronize();
    if (out16 && cudaMemcpyFromSymbol(out16, g_phase_clocks, sizeof(unsigned long long) * 16) != cudaSuccess) return 1;
    if (reset) { unsigned long long z[16] = {0}; if (cudaMemcpyToSymbol(g_phase_clocks, z, sizeof(z)) != cudaSuccess) return 1; }
    return 0;
}
#endif

#ifdef SPARQ_PHASE_CLOCKS
extern "C" int sparq_debug_post_clocks_split(unsigned long long* out16, int reset) {
    cudaDeviceSynchronize();
    if (out16 && cudaMemcpyFromSymbol(out16, g_post_clocks, sizeof(unsigned long long) * 16) != cudaSuccess) return 1;
    if (reset) { unsigned long long z[16] = {0}; if (cudaMemcpyToSymbol(g_post_clocks, z, sizeof(z)) != cudaSuccess) return 1; }
    return 0;
}
#endif

size_t decode_static_smem() { return sizeof(DecodeShared); }
size_t decode_dynamic_smem(int S_max) { return (size_t)RING_BYTES + (size_t)S_max * sizeof(uint32_t); }
static int post_bm_words(int S_max) { return (S_max + 127) / 128 * 4; }      // whole 16-byte groups of bitmap words
static size_t post_dynamic_smem(int S_max) {
    return (post_scratch_bytes(FCTA::NHW, post_bm_words(S_max)) + 127) & ~(size_t)127;
}
int decode_max_positions() { return BM_WORDS * 32; }

cudaError_t launch_sparq_decode(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                int r, int k, uint32_t opts, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                int32_t* status, cudaStream_t stream) {
    const size_t dyn = decode_dynamic_smem(S_max);
    cudaError_t e = cudaFuncSetAttribute(sparq_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    if (e != cudaSuccess) return e;
    sparq_decode_kernel<<<B * Hq, NT, dyn, stream>>>(q, K, Kt, V, vbar, seq_lens, Hq, Hkv, S_max, r, k, out, idx_r,
                                                            idx_k, alpha, status, opts);
    return cudaGetLastError();
}

// Slices per unit of the split plan: enough CTAs for about two waves of resident CTAs, at least
// one pass of SCH positions per slice; 0 when the plan does not apply (a short cache).  With two
// or more whole units per SM the units are left whole: slicing then only adds the repeated top-r
// and the merge of the slices (1024 units of 16384 positions: 146 us whole, 154 us in two slices,
// 151 in three; 512 units of up to 32800: 287 whole, 290 in three).
// (The variant that stores K once reads d_h / r times the bytes per unit and keeps the slices:
// 1024 such units took 1121 us whole against 885 us in two slices.)
int split_count(int units, int S_max, int n_sm, bool one_k) {
    if (n_sm <= 0 || S_max < 2 * SCH) return 0;
    if (!one_k && units >= 2 * n_sm) return 1;
    const int want = (2 * SPLIT_CTAS * n_sm + units - 1) / units;      // about two waves of resident CTAs
    const int cap = (S_max + SCH - 1) / SCH;
    const int s = want < cap ? want : cap;
    return s < 1 ? 1 : s;
}

size_t split_scratch_bytes(int units, int S_max, int splits) {
    // keys; with slicing also per-slice statistics and histograms and the units' ticket counters
    const size_t sliced = splits > 1 ? (size_t)units * splits * (PART_WORDS + SPLIT_FBINS) + (size_t)units : 0;
    return ((size_t)units * S_max + sliced) * sizeof(uint32_t);
}

cudaError_t launch_sparq_decode_split(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                      const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                      int r, int k, uint32_t opts, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                      int32_t* status, int splits, void* scratch, bool one_k, cudaStream_t stream) {
    const int units = B * Hq;
    uint32_t* ws_keys = static_cast<uint32_t*>(scratch);
    uint32_t* ws_part = ws_keys + (size_t)units * S_max;
    uint32_t* ws_hist = ws_part + (size_t)units * splits * PART_WORDS;
    unsigned int* ws_count = ws_hist + (size_t)units * splits * SPLIT_FBINS;
    const size_t dyn = post_dynamic_smem(S_max);
    auto kernel = one_k ? sparq_split_kernel<true> : sparq_split_kernel<false>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    if (e != cudaSuccess) return e;
    // Half of the SM's memory as shared memory holds the five CTAs; the other half stays L1, whose
    // size bounds how many of the streaming loads can be in flight (measured: 50 % beats both 62 % and
    // the driver's own choice).
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, 50);
    if (e != cudaSuccess) return e;
    if (splits > 1) {
        e = cudaMemsetAsync(ws_count, 0, (size_t)units * sizeof(unsigned int), stream);
        if (e != cudaSuccess) return e;
    }
    kernel<<<(unsigned)splits * (unsigned)units, FNT, dyn, stream>>>(q, K, Kt, V, vbar, seq_lens, Hq, Hkv, S_max, r, k, splits,
                                                     post_bm_words(S_max), out, idx_r, idx_k, alpha, status,
                                                     ws_keys, ws_part, ws_hist, ws_count, opts);
    return cudaGetLastError();
}

}  // namespace sparq
