// sparq_decode, one CTA per (batch, query head): the kernel for long sequences (any S_max whose
// score keys fit in shared memory).  Every stage is fused so that only the compulsory bytes touch
// HBM.
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
constexpr int SCRATCH_ONLY_BYTES = (int)((post_scratch_bytes(CTA::NHW, BM_WORDS) + 127) & ~(size_t)127);
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

// Stage a1 by a whole CTA (G::NT >= 128 threads): the r largest |q_j| by rank counting.
// key = |q_j| bit pattern above (127 - j): distinct keys, larger |q| first, then smaller j.
// Fills hm.qf, q16, i1 (ascending), qh (zero padded to a multiple of RB_), inv_tau, l1_sel.
// red: 2*NW floats, cnt: 4 words.  Ends with a barrier.
template <class G, int RB_>
__device__ __forceinline__ void top_r_block(int tid, const sparq_half* __restrict__ q_row, int r, HeadMeta& hm, float* red,
                                            uint32_t* cnt) {
    const int lane = tid & 31, warp = tid >> 5;
    uint16_t hb = 0;
    float qf = 0.f, aq = 0.f;
    uint32_t mine = 0;
    if (tid < D) {
        hb = q_row[tid];
        qf = __half2float(__ushort_as_half(hb));
        aq = fabsf(qf);
        mine = ((uint32_t)(hb & 0x7fffu) << 7) | (uint32_t)(D - 1 - tid);
        hm.qf[tid] = qf;
        hm.q16[tid] = hb;
        hm.rkey[tid] = mine;
    }
    G::sync();
    bool sel = false;
    if (tid < D) {
        int rank = 0;
        const uint4* rk4 = reinterpret_cast<const uint4*>(hm.rkey);
#pragma unroll 8
        for (int j = 0; j < D / 4; ++j) {
            uint4 o = rk4[j];
            rank += (o.x > mine) + (o.y > mine) + (o.z > mine) + (o.w > mine);
        }
        sel = rank < r;
    }
    const unsigned bal = __ballot_sync(FULL, sel);
    if (lane == 0 && warp < 4) cnt[warp] = __popc(bal);      // warps 0..3 hold the D components
    float l1_all = aq, l1_sel = sel ? aq : 0.f;
    group_sum2<G>(l1_all, l1_sel, red, tid);                 // its barriers also publish cnt
    if (sel) {
        int slot = __popc(bal & ((1u << lane) - 1));
        for (int w = 0; w < warp; ++w) slot += cnt[w];
        hm.i1[slot] = tid;                                   // ascending by construction
        hm.qh[slot] = hb;
    }
    const int r_pad = (r + RB_ - 1) / RB_ * RB_;
    if (tid >= r && tid < r_pad) hm.qh[tid] = 0;
    if (tid == 0) { hm.inv_tau = (l1_all > 0.f) ? rsqrtf((float)D * l1_sel / l1_all) : 1.0f; hm.l1_sel = l1_sel; }
    G::sync();
}

struct DecodeShared {
    HeadMeta hm;
    int32_t i2[SPARQ_K_MAX];
    uint64_t full[STAGES];        // mbarriers: stage s has landed
    float red[2 * CTA::NW];
    uint32_t redu[2 * CTA::NW];
    uint32_t res[4];
    uint32_t band[4];
};

// FROM_SCRATCH = false: the whole step.  FROM_SCRATCH = true: the second kernel of the split-S plan;
// the keys of this unit were written to ws_keys by sparq_split_scores_kernel (with per-split maxima
// in ws_part), so a2 is replaced by a copy of the keys into shared memory.
template <bool FROM_SCRATCH>
__global__ void __launch_bounds__(NT, 3)
sparq_decode_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                    const sparq_half* __restrict__ Kt, const sparq_half* __restrict__ V,
                    const sparq_half* __restrict__ vbar, const int32_t* __restrict__ seq_lens,
                    int Hq, int Hkv, int S_max, int r, int k,
                    sparq_half* __restrict__ out, int32_t* __restrict__ idx_r, int32_t* __restrict__ idx_k,
                    float* __restrict__ alpha_out, int32_t* status,
                    const uint32_t* __restrict__ ws_keys, const uint32_t* __restrict__ ws_part, int splits) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    unsigned char* ring = dyn_smem;                                       // a2: STAGES x [RB rows x CH positions] fp16
    // [n] approximate-score keys, after the ring (or, without a2, after the post-phase scratch alone)
    uint32_t* keys = reinterpret_cast<uint32_t*>(dyn_smem + (FROM_SCRATCH ? SCRATCH_ONLY_BYTES : RING_BYTES));
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
    }

    top_r_block<CTA, RB>(tid, q + (size_t)bh * D, r, hm, sh.red, sh.res);        // a1
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
    if constexpr (FROM_SCRATCH) {
        // ---------------------------------------------------------------- a2 was done by the split kernel
        const uint4* src = reinterpret_cast<const uint4*>(ws_keys + (size_t)bh * S_max);
        for (int i = tid; i < (n + 3) / 4; i += NT) reinterpret_cast<uint4*>(keys)[i] = src[i];
        for (int p = tid; p < splits; p += NT) {
            kmax = max(kmax, ws_part[((size_t)bh * splits + p) * 2]);
            kabs_bits = max(kabs_bits, ws_part[((size_t)bh * splits + p) * 2 + 1]);
        }
    } else {
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
    }
    group_max2_u32<CTA>(kmax, kabs_bits, sh.redu, tid);      // barriers: keys complete, ring is dead

    // ------------------------------------------------------------------ a3-a6 (scratch in the dead ring)
    PostScratch sc;
    carve_post_scratch(sc, ring, CTA::NHW, BM_WORDS);
    sc.i2 = sh.i2; sc.red = sh.red; sc.redu = sh.redu; sc.res = sh.res; sc.band = sh.band;
    const SelectResult sel_res = select_generic<CTA>(tid, hm, keys, kmax, __uint_as_float(kabs_bits), sc, r, S_max, Kt_head);
    finish<CTA, 8>(tid, hm, keys, kmax, sel_res, sc, k, K + kv_head * (size_t)S_max * D, V + kv_head * (size_t)S_max * D,
                   vbar + kv_head * D, out_row, idx_k ? idx_k + (size_t)bh * k : nullptr, alpha_out ? alpha_out + bh : nullptr);
    PHASE_MARK(2);
}

// ---------------------------------------------------------------------------------- split-S plan
// When there are fewer (batch, head) units than SMs (batch-1 decode over a long cache), one CTA
// per unit leaves most of the GPU idle.  The split plan cuts every unit's sequence into `splits`
// slices: grid (splits, units), 128 threads, each CTA repeats a1 (cheap) and streams its slice of
// the r selected Kt rows with plain 128-bit loads (8 rows in flight per thread), writing the
// slice's keys to a scratch buffer and its largest key / largest |K| beside them.  The second
// kernel, sparq_decode_kernel<true>, one CTA per unit, picks the keys up and runs a3-a6 unchanged,
// so the selected set is exactly the one of the unsplit plans.
constexpr int SNT = 128;                 // threads of a scores CTA
constexpr int SCH = SNT * 8;             // positions a scores CTA covers per pass
using SCTA = Group<SNT, 0>;

__global__ void __launch_bounds__(SNT)
sparq_split_scores_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ Kt,
                          const int32_t* __restrict__ seq_lens, int Hq, int Hkv, int S_max, int r, int k, int splits,
                          uint32_t* __restrict__ ws_keys, uint32_t* __restrict__ ws_part, int32_t* __restrict__ idx_r) {
    __shared__ HeadMeta hm;
    __shared__ float red[2 * SCTA::NW];
    __shared__ uint32_t redu[2 * SCTA::NW];
    __shared__ uint32_t cnt[4];
    const int tid = threadIdx.x, p = blockIdx.x, bh = blockIdx.y;
    const int b = bh / Hq, h = bh % Hq, hkv = h / (Hq / Hkv);
    const int n = seq_lens[b];
    uint32_t kmax = 0;
    __half2 mx[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) mx[e] = __float2half2_rn(0.f);
    if (n >= 1 && n <= S_max && k > 0) {                     // otherwise the second kernel reports / returns v_bar
        top_r_block<SCTA, 8>(tid, q + (size_t)bh * D, r, hm, red, cnt);
        if (p == 0 && idx_r) for (int j = tid; j < r; j += SNT) idx_r[(size_t)bh * r + j] = hm.i1[j];
        const uint4* Kt_vec = reinterpret_cast<const uint4*>(Kt + ((size_t)b * Hkv + hkv) * (size_t)D * S_max);
        const int row_vecs = S_max >> 3;
        const int n_pass = ((n + 7) / 8 + SNT - 1) / SNT;    // passes of SCH positions over the whole sequence
        uint32_t* keys = ws_keys + (size_t)bh * S_max;
        for (int c = p; c < n_pass; c += splits) {           // this CTA's passes: c = p, p + splits, ...
            const int t0 = c * SCH + tid * 8;
            const int nvalid = min(8, n - t0);
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
            if (nvalid > 0) {                                // (the layout keeps zeros up to the end of the last vector)
                for (int jb = 0; jb < r; jb += 8) {
                    uint4 v[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) v[u] = ld_stream(Kt_vec + (size_t)hm.i1[min(jb + u, r - 1)] * row_vecs + (t0 >> 3));
#pragma unroll
                    for (int u = 0; u < 8; ++u)
                        if (jb + u < r) row_fma(acc, mx, v[u], hm.qh[jb + u]);
                }
#pragma unroll
                for (int e = 0; e < 8; ++e)
                    if (e < nvalid) { const uint32_t kk = key32(acc[e]); keys[t0 + e] = kk; kmax = max(kmax, kk); }
            }
        }
    }
    else if (p == 0 && idx_r && (n < 1 || n > S_max)) {
        for (int j = tid; j < r; j += SNT) idx_r[(size_t)bh * r + j] = -1;
    }
    uint32_t kabs_bits = __float_as_uint(mx_to_float(mx));
    group_max2_u32<SCTA>(kmax, kabs_bits, redu, tid);
    if (tid == 0) { ws_part[((size_t)bh * splits + p) * 2] = kmax; ws_part[((size_t)bh * splits + p) * 2 + 1] = kabs_bits; }
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

size_t decode_static_smem() { return sizeof(DecodeShared); }
size_t decode_dynamic_smem(int S_max) { return (size_t)RING_BYTES + (size_t)S_max * sizeof(uint32_t); }
static size_t decode_dynamic_smem_from_scratch(int S_max) { return (size_t)SCRATCH_ONLY_BYTES + (size_t)S_max * sizeof(uint32_t); }
int decode_max_positions() { return BM_WORDS * 32; }

cudaError_t launch_sparq_decode(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                int r, int k, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                int32_t* status, cudaStream_t stream) {
    const size_t dyn = decode_dynamic_smem(S_max);
    cudaError_t e = cudaFuncSetAttribute(sparq_decode_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    if (e != cudaSuccess) return e;
    sparq_decode_kernel<false><<<B * Hq, NT, dyn, stream>>>(q, K, Kt, V, vbar, seq_lens, Hq, Hkv, S_max, r, k, out, idx_r,
                                                            idx_k, alpha, status, nullptr, nullptr, 0);
    return cudaGetLastError();
}

// Slices per unit of the split plan: enough CTAs for about two per SM, at least one pass of SCH
// positions per slice; 0 when the plan does not apply (a short cache).  With at least as many
// units as SMs the answer is 1: no slicing, but still two kernels -- a pure streaming kernel at
// high occupancy, then the latency-bound stages with the keys read back from the workspace --
// which pays off when the keys of one unit fill most of an SM's shared memory.
int split_count(int units, int S_max, int n_sm) {
    if (n_sm <= 0 || S_max < 2 * SCH) return 0;
    if (units >= n_sm) return 1;
    const int want = (2 * n_sm + units - 1) / units;
    const int cap = (S_max + SCH - 1) / SCH;
    const int s = want < cap ? want : cap;
    return s < 1 ? 1 : s;
}

size_t split_scratch_bytes(int units, int S_max, int splits) {
    return ((size_t)units * S_max + (size_t)units * splits * 2) * sizeof(uint32_t);
}

cudaError_t launch_sparq_decode_split(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                      const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                      int r, int k, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                      int32_t* status, int splits, void* scratch, cudaStream_t stream) {
    const int units = B * Hq;
    uint32_t* ws_keys = static_cast<uint32_t*>(scratch);
    uint32_t* ws_part = ws_keys + (size_t)units * S_max;
    const size_t dyn = decode_dynamic_smem_from_scratch(S_max);
    cudaError_t e = cudaFuncSetAttribute(sparq_decode_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    if (e != cudaSuccess) return e;
    sparq_split_scores_kernel<<<dim3(splits, units), SNT, 0, stream>>>(q, Kt, seq_lens, Hq, Hkv, S_max, r, k, splits,
                                                                       ws_keys, ws_part, idx_r);
    sparq_decode_kernel<true><<<units, NT, dyn, stream>>>(q, K, Kt, V, vbar, seq_lens, Hq, Hkv, S_max, r, k, out, nullptr,
                                                          idx_k, alpha, status, ws_keys, ws_part, splits);
    return cudaGetLastError();
}

}  // namespace sparq
