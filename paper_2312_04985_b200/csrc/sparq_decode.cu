// sparq_decode: the SparQ attention step (Section 4, Steps 1-3), one CTA per (batch, query head),
// every stage fused so that only the compulsory bytes touch HBM.
//
//   a1  top-r of |q| by rank counting on integer keys; tau                    (Step 1, Eq. (9))
//   a2  stream the r selected rows of Kt through a ring of bulk asynchronous copies
//       (cp.async.bulk + mbarrier, no multicast).  Each position's sum over the r components
//       is an fp32 chain of mixed-precision FMAs (fp16 x fp16 products are exact in fp32), kept
//       on chip as an order-preserving 32-bit key: 4 bytes/position of shared memory.  The
//       largest |K| seen gives a rigorous bound B on every sum's rounding error   (Eq. (7))
//   a4  MSB radix select (11+11+10 bits, early exit) of the k largest keys.  If fp32 sums within
//       2B of the threshold lie on both sides of it (or tie), those few positions are re-decided by
//       their exact-product fp64 sums, so the selected set equals the float64 one.   (Step 2)
//   a3  softmax statistics of the approximate logits, fused with the pass that turns the
//       selection into a ballot bitmap -> ascending i2; alpha                   (Eq. (7), Step 3)
//   a5  gather of the k selected K and V rows (128-bit loads, half-warp per row), online
//       softmax in fp32                                                        (Eq. (8))
//   a6  out = alpha y3 + (1 - alpha) v_bar                                     (Eq. (10))
#include "common.cuh"
#include "kernels.h"

namespace sparq {
namespace {

constexpr int NT = 256;                  // threads per CTA
constexpr int NW = NT / 32;
constexpr int NHW = NT / 16;             // half-warps: one gathered K/V row each
constexpr int CH = NT * 8;               // positions per chunk: 8 per thread (one 16-byte vector)
constexpr int RB = 4;                    // Kt rows per pipeline stage
constexpr int STAGES = 3;
constexpr int STAGE_BYTES = RB * CH * 2;
constexpr int RING_BYTES = STAGES * STAGE_BYTES;
constexpr int HIST_BINS = 2048;
constexpr int BM_WORDS = 2048;           // bitmap capacity: 65536 positions
constexpr int RG = 8;                    // gathered rows in flight per half-warp
constexpr int CAND_MAX = 256;            // threshold-band positions the quick fp64 re-decision handles
constexpr int WAIT_LIMIT = 1 << 22;      // polls before a copy is declared lost

static_assert(HIST_BINS * 4 + 2 * BM_WORDS * 4 + NHW * (D + 2) * 4 + CAND_MAX * 12 <= RING_BYTES, "a4/a5 scratch must fit the ring");
static_assert(CAND_MAX <= NT, "one thread per band candidate");
static_assert(NT >= D && HIST_BINS % NT == 0, "thread mapping");

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
    double qd[D];                 // tie path only: selected query components * 2^1008, in i1 order
    float qf[D];                  // q as fp32
    uint32_t rkey[D];             // top-r ranking keys
    int32_t i1[D];
    uint16_t qh[D + RB];          // selected query components (fp16 bits) in i1 order
    int32_t i2[SPARQ_K_MAX];
    uint64_t full[STAGES];        // mbarriers: stage s has landed
    float red[2 * NW];
    uint32_t redu[2 * NW];
    uint32_t res[4];
    uint32_t band[4];             // [0] keys in [lo, edge), [1] keys in [edge, hi], [2] candidate list length
    float inv_tau, l1_sel;
};

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
// Two block-wide maxima with one pair of barriers.  red: 2*NW words.
__device__ __forceinline__ void block_max2_u32(uint32_t& a, uint32_t& b, uint32_t* red) {
    a = __reduce_max_sync(FULL, a);
    b = __reduce_max_sync(FULL, b);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { red[threadIdx.x >> 5] = a; red[NW + (threadIdx.x >> 5)] = b; }
    __syncthreads();
    a = 0; b = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) { a = max(a, red[w]); b = max(b, red[NW + w]); }
}
__device__ __forceinline__ uint32_t block_sum_u32(uint32_t v, uint32_t* red) {
    v = __reduce_add_sync(FULL, v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = v;
    __syncthreads();
    uint32_t t = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) t += red[w];
    return t;
}
// Inclusive prefix sum over the CTA in thread order; *total receives the CTA-wide sum.
__device__ __forceinline__ uint32_t block_scan_incl(uint32_t v, uint32_t* red, uint32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t x = __shfl_up_sync(FULL, v, o);
        if (lane >= o) v += x;
    }
    __syncthreads();
    if (lane == 31) red[warp] = v;
    __syncthreads();
    uint32_t before = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < NW; ++w) { if (w < warp) before += red[w]; tot += red[w]; }
    *total = tot;
    return v + before;
}

// One radix-select pass over an already filled histogram of HIST_BINS bins: find, from the top,
// the bin holding the need-th largest candidate.  res[0] = bin, res[1] = candidates above it,
// res[2] = candidates in it.  All threads call; the result is valid after the trailing barrier.
__device__ __forceinline__ void find_bin(const uint32_t* hist, uint32_t need, uint32_t* red, uint32_t* res) {
    constexpr int PER = HIST_BINS / NT;
    const int top = HIST_BINS - 1 - (int)threadIdx.x * PER;   // this thread's bins: top, top-1, ...
    uint32_t c[PER], s = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) { c[i] = hist[top - i]; s += c[i]; }
    uint32_t total;
    uint32_t incl = block_scan_incl(s, red, &total);
    uint32_t run = incl - s;
    if (run < need && need <= incl) {
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            if (run + c[i] >= need) { res[0] = top - i; res[1] = run; res[2] = c[i]; break; }
            run += c[i];
        }
    }
    __syncthreads();
}

__device__ __forceinline__ void zero_hist(uint32_t* hist) {
    uint4* h4 = reinterpret_cast<uint4*>(hist);
    for (int i = threadIdx.x; i < HIST_BINS / 4; i += NT) h4[i] = make_uint4(0, 0, 0, 0);
}

__device__ __forceinline__ float ex2(float x) {            // 2^x, 2 ulp; exact enough for softmax weights
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// d = a * b + d with fp16 a, b and fp32 d: the product is exact, one rounding (sm_100 mixed FMA).
__device__ __forceinline__ void fma_h(float& d, uint16_t a, uint16_t b) {
    asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(d) : "h"(a), "h"(b));
}

// One Kt row vector (8 positions) times one query component into the 8 running sums.
__device__ __forceinline__ void row_fma(float (&acc)[8], __half2& mx, uint4 v, uint16_t qj) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        fma_h(acc[2 * e], (uint16_t)(w[e] & 0xffffu), qj);
        fma_h(acc[2 * e + 1], (uint16_t)(w[e] >> 16), qj);
        mx = __hmax2(mx, __habs2(*reinterpret_cast<const __half2*>(&w[e])));
    }
}

// fp64 sum of the exact products of the selected query components with position t of the r
// selected Kt rows, in i1 order: bit for bit the float64 oracle's accumulation.
__device__ __forceinline__ double dot64_at(const sparq_half* Kt_head, const DecodeShared& sh, int S_max, int r, int t) {
    double acc = 0.0;
    for (int j = 0; j < r; ++j)
        acc = fma(sh.qd[j], h2d_scalar(Kt_head[(size_t)sh.i1[j] * S_max + t]), acc);
    return acc;
}

__global__ void __launch_bounds__(NT, 3)
sparq_decode_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                    const sparq_half* __restrict__ Kt, const sparq_half* __restrict__ V,
                    const sparq_half* __restrict__ vbar, const int32_t* __restrict__ seq_lens,
                    int Hq, int Hkv, int S_max, int r, int k,
                    sparq_half* __restrict__ out, int32_t* __restrict__ idx_r, int32_t* __restrict__ idx_k,
                    float* __restrict__ alpha_out, int32_t* status) {
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    unsigned char* ring = dyn_smem;                                       // a2: STAGES x [RB rows x CH positions] fp16
    uint32_t* keys = reinterpret_cast<uint32_t*>(dyn_smem + RING_BYTES);  // [n] approximate-logit keys
    // the ring is dead after a2; a4/a5 scratch lives there
    uint32_t* hist = reinterpret_cast<uint32_t*>(ring);
    uint32_t* bm_sel = hist + HIST_BINS;                                  // bit t: position t is selected
    uint32_t* bm_tie = bm_sel + BM_WORDS;                                 // bit t: exact fp64 tie at the threshold
    float* merge = reinterpret_cast<float*>(bm_tie + BM_WORDS);
    unsigned long long* cand_val = reinterpret_cast<unsigned long long*>(merge + NHW * (D + 2));   // band candidates' fp64 keys
    int32_t* cand_pos = reinterpret_cast<int32_t*>(cand_val + CAND_MAX);                           // and positions
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
    PHASE_INIT();
    if (tid == 0) {
#pragma unroll
        for (int s = 0; s < STAGES; ++s) mbar_init(&sh.full[s], 1);
        mbar_init_fence();
    }

    // ------------------------------------------------------------------ a1: top-r of |q|
    // key = |q_j| bit pattern above (127 - j): distinct keys, larger |q| first, then smaller j.
    uint16_t hb = 0;
    float qf = 0.f, aq = 0.f;
    uint32_t mine = 0;
    if (tid < D) {
        hb = q[(size_t)bh * D + tid];
        qf = __half2float(__ushort_as_half(hb));
        aq = fabsf(qf);
        mine = ((uint32_t)(hb & 0x7fffu) << 7) | (uint32_t)(D - 1 - tid);
        sh.qf[tid] = qf;
        sh.rkey[tid] = mine;
    }
    __syncthreads();
    bool sel = false;
    if (tid < D) {
        int rank = 0;
        const uint4* rk4 = reinterpret_cast<const uint4*>(sh.rkey);
#pragma unroll 8
        for (int j = 0; j < D / 4; ++j) {
            uint4 o = rk4[j];
            rank += (o.x > mine) + (o.y > mine) + (o.z > mine) + (o.w > mine);
        }
        sel = rank < r;
    }
    const unsigned bal = __ballot_sync(FULL, sel);
    if (lane == 0) sh.redu[warp] = __popc(bal);
    const float l1_all = block_sum(aq, sh.red);              // its barriers also publish redu
    int slot = __popc(bal & ((1u << lane) - 1));
    for (int w = 0; w < warp; ++w) slot += sh.redu[w];
    const float l1_sel = block_sum(sel ? aq : 0.f, sh.red);
    if (sel) {
        sh.i1[slot] = tid;                                   // ascending by construction
        sh.qh[slot] = hb;
        sh.qd[slot] = ldexp((double)qf, 1008);
    }
    const int r_pad = (r + RB - 1) / RB * RB;
    if (tid >= r && tid < r_pad) sh.qh[tid] = 0;
    if (tid == 0) { sh.inv_tau = (l1_all > 0.f) ? rsqrtf((float)D * l1_sel / l1_all) : 1.0f; sh.l1_sel = l1_sel; }
    __syncthreads();
    if (idx_r) for (int j = tid; j < r; j += NT) idx_r[(size_t)bh * r + j] = sh.i1[j];
    const float inv_tau = sh.inv_tau;

    float alpha = 0.f;
    PHASE_MARK(0);
    if (k_eff > 0) {
        // -------------------------------------------------------------- a2: stream r rows of Kt
        const sparq_half* Kt_head = Kt + kv_head * (size_t)D * S_max;
        const int n8 = (n + 7) & ~7;                         // whole 16-byte vectors; n8 <= S_max
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
                bulk_g2s(ring + s * STAGE_BYTES + lane * (CH * 2), Kt_head + (size_t)sh.i1[jb + lane] * S_max + c * CH, bytes,
                         &sh.full[s]);
        };
        if (warp == 0) for (int it = 0; it < min(STAGES, total); ++it) issue(it, it);

        uint32_t kmax = 0;
        __half2 mx = __float2half2_rn(0.f);                  // largest |K| among the valid streamed values
        bool ok = true;
        int it = 0, s = 0;
        uint32_t parity = 0;
        for (int c = 0; c < n_chunks; ++c) {
            float acc[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] = 0.f;
            const int t0 = c * CH + tid * 8;
            const int nvalid = min(8, n - t0);               // positions of this thread's vector inside the sequence
            // positions past n in the straddling vector hold whatever the caller's memory holds: mask them
            uint32_t msk[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) msk[e] = (nvalid >= 2 * e + 2) ? 0xffffffffu : (nvalid == 2 * e + 1 ? 0x0000ffffu : 0u);
            for (int jb = 0; jb < r_pad; jb += RB, ++it) {
                ok = mbar_wait_bounded(&sh.full[s], parity, WAIT_LIMIT);
                const uint4* src = reinterpret_cast<const uint4*>(ring + s * STAGE_BYTES) + tid;
                if (nvalid >= 8) {
#pragma unroll
                    for (int u = 0; u < RB; ++u)
                        if (jb + u < r) row_fma(acc, mx, src[u * (CH / 8)], sh.qh[jb + u]);   // uniform; padded rows were not copied
                } else if (nvalid > 0) {
#pragma unroll
                    for (int u = 0; u < RB; ++u)
                        if (jb + u < r) {
                            uint4 v = src[u * (CH / 8)];
                            v.x &= msk[0]; v.y &= msk[1]; v.z &= msk[2]; v.w &= msk[3];
                            row_fma(acc, mx, v, sh.qh[jb + u]);
                        }
                }
                ok = __syncthreads_and(ok);                  // slot s fully consumed (or a wait gave up)
                if (!ok) break;
                if (warp == 0 && it + STAGES < total) issue(it + STAGES, s);
                if (++s == STAGES) { s = 0; parity ^= 1u; }
            }
            if (!ok) break;
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
        if (!ok) {                       // a bulk copy never landed: report, define the output, leave
            if (tid == 0) { raise_status(status, SPARQ_DEV_TIMEOUT); if (alpha_out) alpha_out[bh] = 0.f; }
            if (tid < D) out_row[tid] = 0;
            if (idx_k) for (int j = tid; j < k; j += NT) idx_k[(size_t)bh * k + j] = -1;
            return;
        }
        PHASE_MARK(1);
        uint32_t kabs_bits = __float_as_uint(fmaxf(__low2float(mx), __high2float(mx)));
        block_max2_u32(kmax, kabs_bits, sh.redu);            // barriers: keys complete, ring is dead
        const float vmax = unkey32(kmax);
        const float kabs = __uint_as_float(kabs_bits);
        // |fp32 chain - exact sum| <= ((1+u)^r - 1) sum_j |q_j K_tj| <= 1.02 r u ||q[i1]||_1 max|K|,  u = 2^-24
        const float twoB = 2.f * (1.02f * (float)r * 5.9604645e-8f * sh.l1_sel * kabs) + 1e-37f * (float)(kabs > 0.f);

        // -------------------------------------------------------------- a4: top-k select
        // MSB radix select, 11 + 11 + 10 bits, leaving the loop as soon as a whole bin is wanted.
        // Afterwards the k_eff largest keys are those >= edge, except that `over` too many keys
        // equal edge when the fp32 sums tie at the threshold.
        uint32_t prefix = 0, mask = 0, need = (uint32_t)k_eff, ceq = 0;
        {
            int shift = 32;
#pragma unroll 1
            for (int pass = 0; pass < 3; ++pass) {
                const int bits = pass < 2 ? 11 : 10;
                shift -= bits;
                zero_hist(hist);
                __syncthreads();
                for (int t = tid; t < n; t += NT) {
                    const uint32_t u = keys[t];
                    if ((u & mask) == prefix) atomicAdd(&hist[(u >> shift) & ((1u << bits) - 1)], 1u);
                }
                __syncthreads();
                find_bin(hist, need, sh.redu, sh.res);
                prefix |= sh.res[0] << shift;
                mask |= ((1u << bits) - 1) << shift;
                need -= sh.res[1];
                ceq = sh.res[2];
                if (ceq == need) break;                      // the whole bin is selected: no need to split it
            }
        }
        PHASE_MARK(2);
        const uint32_t edge = prefix;                        // unprocessed low bits are zero
        const uint32_t over = ceq - need;
        const float edge_val = unkey32(edge);
        const uint32_t lo_key = key32(__fadd_rd(edge_val, -twoB)), hi_key = key32(__fadd_ru(edge_val, twoB));

        // -------------------------------------------------------------- a3 + bitmap of the selection
        // Softmax denominator, the speculative selection key >= edge as a bitmap, and the positions
        // whose key lies within 2B of the edge (counted on each side, listed while the list has room).
        const int nwords = (n + 31) >> 5;
        const float c1 = inv_tau * LOG2E;
        if (tid < 4) sh.band[tid] = 0;
        __syncthreads();
        float zpart = 0.f;
        for (int wi = warp; wi < nwords; wi += NW) {
            const int t = (wi << 5) + lane;
            const bool valid = t < n;
            const uint32_t u = valid ? keys[t] : 0u;
            zpart += valid ? ex2((unkey32(u) - vmax) * c1) : 0.f;
            const bool ge = valid && u >= edge;
            const unsigned g = __ballot_sync(FULL, ge);
            if (lane == 0) bm_sel[wi] = g;
            if (valid && u >= lo_key && u <= hi_key) {       // rare
                atomicAdd(&sh.band[ge ? 1 : 0], 1u);
                const uint32_t slot = atomicAdd(&sh.band[2], 1u);
                if (slot < CAND_MAX) cand_pos[slot] = t;
            }
        }
        const float Z = block_sum(zpart, sh.red);            // barriers also publish the bitmap and the band
        const uint32_t cnt_lo = sh.band[0], cnt_hi = sh.band[1], n_cand = sh.band[2];
        PHASE_MARK(3);
        uint32_t need_tie = 0;
        if (over > 0 || (cnt_lo > 0 && cnt_hi > 0)) {
            // fp32 sums on both sides of the threshold are closer to it than their error bound (or
            // tie).  The n_cand positions in the band compete for cnt_hi - over places by their fp64
            // sums of exact products; equal fp64 sums go to the lowest positions.
            const uint32_t need64 = cnt_hi - over;
            if (n_cand <= CAND_MAX) {
                // few candidates: one thread each, rank by counting, then patch their bitmap bits
                unsigned long long v = 0;
                int t = 0;
                if (tid < n_cand) { t = cand_pos[tid]; v = key64(dot64_at(Kt_head, sh, S_max, r, t)); cand_val[tid] = v; }
                __syncthreads();
                if (tid < n_cand) {
                    uint32_t rank = 0;
                    for (uint32_t i = 0; i < n_cand; ++i) {
                        const unsigned long long vi = cand_val[i];
                        rank += (vi > v) || (vi == v && cand_pos[i] < t);
                    }
                    if (rank < need64) atomicOr(&bm_sel[t >> 5], 1u << (t & 31));
                    else atomicAnd(&bm_sel[t >> 5], ~(1u << (t & 31)));
                }
                __syncthreads();
            } else {
                // many candidates (degenerate inputs, e.g. constant keys): radix select over their
                // 64-bit keys, 8 passes of 8 bits, then rebuild the bitmap
                unsigned long long p64 = 0, m64 = 0;
                uint32_t left = need64;
#pragma unroll 1
                for (int shift = 56; shift >= 0; shift -= 8) {
                    zero_hist(hist);
                    __syncthreads();
                    for (int t = tid; t < n; t += NT) {
                        const uint32_t u = keys[t];
                        if (u >= lo_key && u <= hi_key) {
                            const unsigned long long v = key64(dot64_at(Kt_head, sh, S_max, r, t));
                            if ((v & m64) == p64) atomicAdd(&hist[(uint32_t)(v >> shift) & 255u], 1u);
                        }
                    }
                    __syncthreads();
                    find_bin(hist, left, sh.redu, sh.res);
                    p64 |= (unsigned long long)sh.res[0] << shift;
                    m64 |= 255ull << shift;
                    left -= sh.res[1];
                }
                need_tie = left;
                for (int wi = warp; wi < nwords; wi += NW) {
                    const int t = (wi << 5) + lane;
                    const uint32_t u = t < n ? keys[t] : 0u;
                    bool s_ = t < n && u > hi_key, tie = false;
                    if (t < n && u >= lo_key && u <= hi_key) {
                        const unsigned long long v = key64(dot64_at(Kt_head, sh, S_max, r, t));
                        s_ = v > p64;
                        tie = v == p64;
                    }
                    const unsigned g = __ballot_sync(FULL, s_), te = __ballot_sync(FULL, tie);
                    if (lane == 0) { bm_sel[wi] = g; bm_tie[wi] = te; }
                }
                __syncthreads();
            }
        }

        PHASE_MARK(4);
        // ascending list of selected positions from the bitmap(s)
        uint32_t carry_tie = 0, carry_sel = 0;
        for (int base = 0; base < nwords; base += NT) {
            const int wi = base + tid;
            uint32_t g = wi < nwords ? bm_sel[wi] : 0u;
            if (need_tie) {                                  // add the first need_tie tied positions
                uint32_t e = wi < nwords ? bm_tie[wi] : 0u, tot;
                const uint32_t ce = __popc(e);
                const uint32_t before = carry_tie + block_scan_incl(ce, sh.redu, &tot) - ce;
                const uint32_t allowed = before >= need_tie ? 0u : min(ce, need_tie - before);
                while ((uint32_t)__popc(e) > allowed) e &= ~(0x80000000u >> __clz(e));
                g |= e;
                carry_tie += tot;
            }
            uint32_t tot;
            const uint32_t cs = __popc(g);
            uint32_t off = carry_sel + block_scan_incl(cs, sh.redu, &tot) - cs;
            while (g) {
                const int bit = __ffs(g) - 1;
                if (off < (uint32_t)k_eff) sh.i2[off] = (wi << 5) + bit;
                ++off;
                g &= g - 1;
            }
            carry_sel += tot;
        }
        __syncthreads();
        // alpha = approximate-score mass of the selected set (Step 3)
        float apart = 0.f;
        for (int j = tid; j < k_eff; j += NT) apart += ex2((unkey32(keys[sh.i2[j]]) - vmax) * c1);
        alpha = block_sum(apart, sh.red) / Z;

        PHASE_MARK(5);
        // -------------------------------------------------------------- a5: gather k rows of K and V
        const int hw = tid >> 4, l16 = tid & 15;
        const float qscale = rsqrtf((float)D) * LOG2E;
        float qs[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) qs[e] = sh.qf[l16 * 8 + e] * qscale;
        const uint4* Kh = reinterpret_cast<const uint4*>(K + kv_head * (size_t)S_max * D);
        const uint4* Vh = reinterpret_cast<const uint4*>(V + kv_head * (size_t)S_max * D);
        float m = -CUDART_INF_F, l = 0.f, acc[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] = 0.f;
        for (int jb = 0; jb < k_eff; jb += NHW * RG) {       // trip count uniform across the CTA
            uint4 kv[RG], vv[RG];
#pragma unroll
            for (int u = 0; u < RG; ++u) {
                const int t = sh.i2[min(jb + u * NHW + hw, k_eff - 1)];
                kv[u] = ld_stream(Kh + (size_t)t * (D / 8) + l16);
                vv[u] = ld_stream(Vh + (size_t)t * (D / 8) + l16);
            }
            float z[RG], bmax = -CUDART_INF_F;
#pragma unroll
            for (int u = 0; u < RG; ++u) {
                const __half2* kh = reinterpret_cast<const __half2*>(&kv[u]);
                float zz = 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const float2 f = __half22float2(kh[e]);
                    zz = fmaf(f.x, qs[2 * e], zz);
                    zz = fmaf(f.y, qs[2 * e + 1], zz);
                }
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) zz += __shfl_xor_sync(FULL, zz, o);
                z[u] = (jb + u * NHW + hw < k_eff) ? zz : -CUDART_INF_F;   // uniform within the half-warp
                bmax = fmaxf(bmax, z[u]);
            }
            const float mn = fmaxf(m, bmax);
            if (mn > -CUDART_INF_F) {
                const float sc = ex2(m - mn);
                l *= sc;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] *= sc;
#pragma unroll
                for (int u = 0; u < RG; ++u) {
                    const float p = ex2(z[u] - mn);
                    l += p;
                    const __half2* vh = reinterpret_cast<const __half2*>(&vv[u]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __half22float2(vh[e]);
                        acc[2 * e] = fmaf(p, f.x, acc[2 * e]);
                        acc[2 * e + 1] = fmaf(p, f.y, acc[2 * e + 1]);
                    }
                }
                m = mn;
            }
        }
        PHASE_MARK(6);
        // merge the half-warps' partial softmax states
        float* mg = merge + hw * (D + 2);
#pragma unroll
        for (int e = 0; e < 8; ++e) mg[l16 * 8 + e] = acc[e];
        if (l16 == 0) { mg[D] = m; mg[D + 1] = l; }
        __syncthreads();
    }

    // ------------------------------------------------------------------ a6: combine with v_bar
    if (tid < D) {
        const float vb = __half2float(__ushort_as_half(vbar[kv_head * D + tid]));
        float y = vb;
        if (k_eff > 0) {
            float M = -CUDART_INF_F;
#pragma unroll
            for (int w = 0; w < NHW; ++w) M = fmaxf(M, merge[w * (D + 2) + D]);
            float L = 0.f, s = 0.f;
#pragma unroll
            for (int w = 0; w < NHW; ++w) {
                const float sc = ex2(merge[w * (D + 2) + D] - M);
                L = fmaf(merge[w * (D + 2) + D + 1], sc, L);
                s = fmaf(merge[w * (D + 2) + tid], sc, s);
            }
            y = alpha * (s / L) + (1.f - alpha) * vb;
        }
        out_row[tid] = __half_as_ushort(__float2half_rn(y));
    }
    if (tid == 0 && alpha_out) alpha_out[bh] = alpha;
    if (idx_k) for (int j = tid; j < k; j += NT) idx_k[(size_t)bh * k + j] = (j < k_eff) ? sh.i2[j] : -1;
    PHASE_MARK(7);
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
int decode_max_positions() { return BM_WORDS * 32; }

cudaError_t launch_sparq_decode(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                int r, int k, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                int32_t* status, cudaStream_t stream) {
    const size_t dyn = decode_dynamic_smem(S_max);
    cudaError_t e = cudaFuncSetAttribute(sparq_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    if (e != cudaSuccess) return e;
    sparq_decode_kernel<<<B * Hq, NT, dyn, stream>>>(q, K, Kt, V, vbar, seq_lens, Hq, Hkv, S_max, r, k, out, idx_r,
                                                     idx_k, alpha, status);
    return cudaGetLastError();
}

}  // namespace sparq
