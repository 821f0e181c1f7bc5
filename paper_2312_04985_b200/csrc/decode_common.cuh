// Building blocks shared by the two sparq_decode kernels (the one-CTA-per-head kernel and the
// persistent warp-specialised one): thread-group reductions, the streamed fp32 score chain, and
// the whole "post" phase -- top-k select with exact re-decision of the threshold band, softmax
// statistics, ascending index list, K/V row gather with online softmax, and the v_bar combine.
#pragma once
#include "common.cuh"

namespace sparq {

#ifdef SPARQ_PHASE_CLOCKS
__device__ unsigned long long g_post_clocks[16];
#define POST_CLK_INIT() long long pc_prev_ = clock64()
#define POST_CLK(i) do { if (gtid == 0) { long long pc_now_ = clock64(); atomicAdd(&g_post_clocks[i], (unsigned long long)(pc_now_ - pc_prev_)); pc_prev_ = pc_now_; } } while (0)
#else
#define POST_CLK_INIT()
#define POST_CLK(i)
#endif

constexpr int HIST_BINS = 2048;
constexpr int CAND_MAX = 256;            // threshold-band positions the quick fp64 re-decision handles
constexpr int WAIT_LIMIT = 1 << 22;      // polls before an asynchronous copy is declared lost

// A group of NT_ consecutive threads (whole warps) that synchronises on its own barrier.
// BAR_ == 0: the whole CTA (__syncthreads); otherwise named barrier BAR_.
template <int NT_, int BAR_>
struct Group {
    static constexpr int NT = NT_, NW = NT_ / 32, NHW = NT_ / 16;
    static __device__ __forceinline__ void sync() {
        if constexpr (BAR_ == 0) __syncthreads();
        else asm volatile("bar.sync %0, %1;" ::"n"(BAR_), "n"(NT_) : "memory");
    }
};

// What the later stages need to know about one (batch, query head) unit; filled by stage a1.
struct alignas(16) HeadMeta {
    uint16_t q16[D];              // q as stored (fp16 bits)
    int32_t i1[D];                // selected components, ascending
    uint32_t rkey[D];             // a1 scratch: ranking keys
    uint16_t qh[D + 8];           // selected components' fp16 bits in i1 order, zero padded
    int32_t bh, n, k_eff, valid;
    float inv_tau, l1_sel;
    int32_t n_sel, k_sel;         // Step 2 ranks positions [0, n_sel) for k_sel places; [n_sel, n) is the local window
};

// Settings of a decode call packed into one word (0 = the paper's algorithm as Section 4 states it):
// bits 0-1 the approximate softmax's temperature (0: Eq. (9), 1: sqrt(d_h), 2: sqrt(r); Section 5.3),
// bit 2 set: Step 3 left out (the output is Eq. (8)'s y3), bits 16-31: local window l.  Packed on the
// host by pack_opts() (kernels.h).
__device__ __forceinline__ bool opt_realloc(uint32_t opts) { return (opts & 4u) == 0u; }
// 1 / tau.  Eq. (9) with tau := 1 where it is 0/0 (no weight on the kept components: every approximate logit is 0).
__device__ __forceinline__ float opt_inv_tau(uint32_t opts, float l1_all, float l1_sel, int r) {
    const uint32_t mode = opts & 3u;
    if (mode == 1u) return rsqrtf((float)D);
    if (mode == 2u) return rsqrtf((float)r);
    return (l1_all > 0.f && l1_sel > 0.f) ? rsqrtf((float)D * l1_sel / l1_all) : 1.0f;
}
// The l = min(window, k_eff) most recent positions are selected outright; the other places are ranked.
__device__ __forceinline__ void opt_set_window(HeadMeta& hm, int n, int k_eff, uint32_t opts) {
    const int l = min((int)(opts >> 16), k_eff);
    hm.n_sel = n - l;
    hm.k_sel = k_eff - l;
}

// Shared-memory scratch of one post phase.
struct PostScratch {
    uint32_t* hist;               // [HIST_BINS]
    uint32_t* bm_sel;             // [ceil(n/32)] bit t: position t is selected
    uint32_t* bm_tie;             // [ceil(n/32)] bit t: exact fp64 tie at the threshold (degenerate path)
    float* merge;                 // [NHW * (D + 2)]
    unsigned long long* cand_val; // [CAND_MAX]
    int32_t* cand_pos;            // [CAND_MAX]
    int32_t* i2;                  // [SPARQ_K_MAX]
    float* red;                   // [2 * NW]
    uint32_t* redu;               // [2 * NW]
    uint32_t* res;                // [4]
    uint32_t* band;               // [4]
};
// Bytes of the scratch that may alias a dead buffer (everything except i2 and the small arrays).
// The half-warp merge area of stage a5 reuses the select stage's histogram/list and the head of
// the bitmaps, all dead by then, so it costs no space of its own.
__host__ __device__ constexpr size_t post_scratch_bytes(int nhw, int bm_words) {
    const size_t select_part = (size_t)HIST_BINS * 4 + 2 * (size_t)bm_words * 4;
    const size_t merge_part = (size_t)nhw * (D + 2) * 4;
    return (((select_part > merge_part ? select_part : merge_part) + 7) & ~(size_t)7) + (size_t)CAND_MAX * 12;
}
__device__ __forceinline__ void carve_post_scratch(PostScratch& sc, unsigned char* base, int nhw, int bm_words) {
    const size_t select_part = (size_t)HIST_BINS * 4 + 2 * (size_t)bm_words * 4;
    const size_t merge_part = (size_t)nhw * (D + 2) * 4;
    sc.hist = reinterpret_cast<uint32_t*>(base);
    sc.bm_sel = sc.hist + HIST_BINS;
    sc.bm_tie = sc.bm_sel + bm_words;
    sc.merge = reinterpret_cast<float*>(base);               // live only after the index list is built
    sc.cand_val = reinterpret_cast<unsigned long long*>(base + (((select_part > merge_part ? select_part : merge_part) + 7) & ~(size_t)7));
    sc.cand_pos = reinterpret_cast<int32_t*>(sc.cand_val + CAND_MAX);
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

// One Kt row vector (8 positions) times one query component into the 8 running sums; mx tracks
// the largest |K| seen (four independent chains).
__device__ __forceinline__ void row_fma(float (&acc)[8], __half2 (&mx)[4], uint4 v, uint16_t qj) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        fma_h(acc[2 * e], (uint16_t)(w[e] & 0xffffu), qj);
        fma_h(acc[2 * e + 1], (uint16_t)(w[e] >> 16), qj);
        mx[e] = __hmax2(mx[e], __habs2(*reinterpret_cast<const __half2*>(&w[e])));
    }
}
__device__ __forceinline__ float mx_to_float(const __half2 (&mx)[4]) {
    const __half2 a = __hmax2(__hmax2(mx[0], mx[1]), __hmax2(mx[2], mx[3]));
    return fmaxf(__low2float(a), __high2float(a));
}

// One ring stage (RB rows of CH8 16-byte vectors each) into a thread's 8 running sums.
//   src: the thread's vector in row 0 of the stage; qh_jb: the RB query components of these rows
//   (16-byte aligned); rows_left: selected rows not yet consumed (>= 1).
// No masking here.  The Kt layout guarantees zeros between the sequence end and the end of its
// 16-byte vector, and a thread whose whole vector lies past the end works on whatever the stage
// holds there; the caller throws that thread's sums and |K| maximum away (it keeps the maximum
// per chunk for that).
template <int RB, int CH8>
__device__ __forceinline__ void stage_fma(float (&acc)[8], __half2 (&mx)[4], const uint4* src, const uint16_t* qh_jb,
                                          int rows_left) {
    static_assert(RB == 4 || RB == 8, "query components are fetched as one 8- or 16-byte vector");
    if (rows_left >= RB) {                                   // uniform; the common case, no predicates at all
        uint32_t qw[RB / 2];
        if constexpr (RB == 8) { const uint4 q8 = *reinterpret_cast<const uint4*>(qh_jb); qw[0] = q8.x; qw[1] = q8.y; qw[2] = q8.z; qw[3] = q8.w; }
        else { const uint2 q4 = *reinterpret_cast<const uint2*>(qh_jb); qw[0] = q4.x; qw[1] = q4.y; }
#pragma unroll
        for (int u = 0; u < RB; ++u)
            row_fma(acc, mx, src[u * CH8], (uint16_t)((u & 1) ? (qw[u >> 1] >> 16) : (qw[u >> 1] & 0xffffu)));
    } else {                                                 // the last, partial batch of rows: the rest was not copied
#pragma unroll
        for (int u = 0; u < RB; ++u)
            if (u < rows_left) row_fma(acc, mx, src[u * CH8], qh_jb[u]);
    }
}

// ---- group-wide reductions in a fixed order (bitwise reproducible run to run) -------------
template <class G>
__device__ __forceinline__ float group_sum(float v, float* red, int gtid) {
    v = warp_sum(v);
    G::sync();
    if ((gtid & 31) == 0) red[gtid >> 5] = v;
    G::sync();
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < G::NW; ++w) t += red[w];
    return t;
}
template <class G>
__device__ __forceinline__ void group_sum2(float& a, float& b, float* red, int gtid) {
    a = warp_sum(a);
    b = warp_sum(b);
    G::sync();
    if ((gtid & 31) == 0) { red[gtid >> 5] = a; red[G::NW + (gtid >> 5)] = b; }
    G::sync();
    a = 0.f; b = 0.f;
#pragma unroll
    for (int w = 0; w < G::NW; ++w) { a += red[w]; b += red[G::NW + w]; }
}
template <class G>
__device__ __forceinline__ void group_max2_u32(uint32_t& a, uint32_t& b, uint32_t* red, int gtid) {
    a = __reduce_max_sync(FULL, a);
    b = __reduce_max_sync(FULL, b);
    G::sync();
    if ((gtid & 31) == 0) { red[gtid >> 5] = a; red[G::NW + (gtid >> 5)] = b; }
    G::sync();
    a = 0; b = 0;
#pragma unroll
    for (int w = 0; w < G::NW; ++w) { a = max(a, red[w]); b = max(b, red[G::NW + w]); }
}
// Inclusive prefix sum over the group in thread order; *total receives the group-wide sum.
template <class G>
__device__ __forceinline__ uint32_t group_scan_incl(uint32_t v, uint32_t* red, uint32_t* total, int gtid) {
    const int lane = gtid & 31, warp = gtid >> 5;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t x = __shfl_up_sync(FULL, v, o);
        if (lane >= o) v += x;
    }
    G::sync();
    if (lane == 31) red[warp] = v;
    G::sync();
    uint32_t before = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < G::NW; ++w) { if (w < warp) before += red[w]; tot += red[w]; }
    *total = tot;
    return v + before;
}

// Stage a1 by a whole CTA (G::NT >= 128 threads): the r largest |q_j| by rank counting.
// key = |q_j| bit pattern above (127 - j): distinct keys, larger |q| first, then smaller j.
// Fills hm.q16, i1 (ascending), qh (zero padded to a multiple of RB_), inv_tau, l1_sel.
// red: 2*NW floats, cnt: 4 words.  Ends with a barrier.
template <class G, int RB_>
__device__ __forceinline__ void top_r_block(int tid, const sparq_half* __restrict__ q_row, int r, HeadMeta& hm, float* red,
                                            uint32_t* cnt, uint32_t opts) {
    const int lane = tid & 31, warp = tid >> 5;
    uint16_t hb = 0;
    float qf = 0.f, aq = 0.f;
    uint32_t mine = 0;
    if (tid < D) {
        hb = q_row[tid];
        qf = __half2float(__ushort_as_half(hb));
        aq = fabsf(qf);
        mine = ((uint32_t)(hb & 0x7fffu) << 7) | (uint32_t)(D - 1 - tid);
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
    if (tid == 0) { hm.inv_tau = opt_inv_tau(opts, l1_all, l1_sel, r); hm.l1_sel = l1_sel; }
    G::sync();
}

// One radix-select pass over an already filled histogram: find, from the top, the bin holding the
// need-th largest candidate.  res[0] = bin, res[1] = candidates above it, res[2] = candidates in
// it.  All threads of the group call; the result is valid after the trailing barrier.
template <class G, int NBINS>
__device__ __forceinline__ void find_bin(const uint32_t* hist, uint32_t need, uint32_t* red, uint32_t* res, int gtid) {
    constexpr int PER = NBINS / G::NT;
    static_assert(NBINS % G::NT == 0 && PER >= 1, "bins per thread");
    const int top = NBINS - 1 - gtid * PER;                  // this thread's bins: top, top-1, ...
    uint32_t c[PER], s = 0;
#pragma unroll
    for (int i = 0; i < PER; ++i) { c[i] = hist[top - i]; s += c[i]; }
    uint32_t total;
    uint32_t incl = group_scan_incl<G>(s, red, &total, gtid);
    uint32_t run = incl - s;
    if (run < need && need <= incl) {
#pragma unroll
        for (int i = 0; i < PER; ++i) {
            if (run + c[i] >= need) { res[0] = top - i; res[1] = run; res[2] = c[i]; break; }
            run += c[i];
        }
    }
    G::sync();
}
template <class G>
__device__ __forceinline__ void zero_hist(uint32_t* hist, int gtid) {
    uint4* h4 = reinterpret_cast<uint4*>(hist);
    for (int i = gtid; i < HIST_BINS / 4; i += G::NT) h4[i] = make_uint4(0, 0, 0, 0);
}

// fp64 sum of the exact products of the selected query components with position t of the r
// selected Kt rows, in i1 order: bit for bit the float64 oracle's accumulation.
// Element (component c, position t) is Kt_head[c * S_max + t * t_stride]: the transposed cache with t_stride = 1, or
// the row-major K with S_max := 1 and t_stride := d_h (the variant that stores K once).
__device__ __forceinline__ double dot64_at(const sparq_half* Kt_head, const HeadMeta& hm, int S_max, int r, int t,
                                           int t_stride = 1) {
    double acc = 0.0;
    for (int j = 0; j < r; ++j) {
        const int c = hm.i1[j];
        acc = fma(ldexp((double)__half2float(__ushort_as_half(hm.q16[c])), 1008), h2d_scalar(Kt_head[(size_t)c * S_max + (size_t)t * t_stride]), acc);
    }
    return acc;
}
// The same sum with 16 loads in flight at a time, for callers whose Kt reads come from far away
// (long caches: every load a miss).  Not inlined: its registers stay out of the callers' hot loops.
static __device__ __noinline__ double dot64_at_batched(const sparq_half* Kt_head, const HeadMeta& hm, int S_max, int r, int t,
                                                       int t_stride = 1) {
    double acc = 0.0;
    for (int j0 = 0; j0 < r; j0 += 16) {
        uint16_t kv[16];
#pragma unroll
        for (int u = 0; u < 16; ++u)
            kv[u] = j0 + u < r ? Kt_head[(size_t)hm.i1[j0 + u] * S_max + (size_t)t * t_stride] : (uint16_t)0;
#pragma unroll
        for (int u = 0; u < 16; ++u)
            if (j0 + u < r) acc = fma(ldexp((double)__half2float(__ushort_as_half(hm.q16[hm.i1[j0 + u]])), 1008), h2d_scalar(kv[u]), acc);
    }
    return acc;
}

// The approximate-score keys of a unit as the post stages see them: one array of 32-bit keys, or the
// keys' upper halves in one array (shared memory) and their lower halves in another (global memory,
// read around the L1).  key_coarse: the key with at least its upper 16 bits right and the rest zero or
// right -- enough for the first digit; key_full: all 32 bits.
struct SplitKeys {
    const uint16_t* hi;
    const uint16_t* lo;
};
__device__ __forceinline__ uint32_t key_full(const uint32_t* keys, int t) { return keys[t]; }
__device__ __forceinline__ uint32_t key_coarse(const uint32_t* keys, int t) { return keys[t]; }
__device__ __forceinline__ uint32_t key_coarse(SplitKeys keys, int t) { return (uint32_t)keys.hi[t] << 16; }
__device__ __forceinline__ uint32_t key_full(SplitKeys keys, int t) {
    return ((uint32_t)keys.hi[t] << 16) | (uint32_t)__ldcg(keys.lo + t);
}
template <class T> struct keys_split { static constexpr bool value = false; };
template <> struct keys_split<SplitKeys> { static constexpr bool value = true; };

// What a select variant hands to finish(): the selection bitmap sc.bm_sel (and, in the degenerate
// path, the tie bitmap sc.bm_tie with need_tie of its lowest positions wanted) and the softmax
// denominator of the approximate scores relative to the largest key.
struct SelectResult {
    float Z;
    uint32_t need_tie;
};

// |fp32 chain - exact sum| <= ((1+u)^r - 1) sum_j |q_j K_tj| <= 1.02 r u ||q[i1]||_1 max|K|,  u = 2^-24
__device__ __forceinline__ float two_b(int r, float l1_sel, float kabs) {
    return 2.f * (1.02f * (float)r * 5.9604645e-8f * l1_sel * kabs);
}

// Re-decide the positions listed in sc.cand_pos[0..n_cand) (all keys within 2B of the threshold) by
// their fp64 sums of exact products: the need64 largest (ties to the lowest position) get their
// bitmap bit set, the others cleared.  n_cand <= CAND_MAX.
// BY_POS: the keys are final (no rounding-error band); the listed positions hold equal keys and the
// lowest positions win.
template <class G, bool BATCHED = false, bool BY_POS = false>
__device__ __forceinline__ void redecide_band(int gtid, const HeadMeta& hm, const PostScratch& sc, uint32_t n_cand,
                                              uint32_t need64, const sparq_half* Kt_head, int S_max, int r,
                                              int t_stride = 1) {
    constexpr int PER = (CAND_MAX + G::NT - 1) / G::NT;      // candidates per thread (1 for groups of 256)
    unsigned long long v[PER];
    int t[PER];
#pragma unroll
    for (int x = 0; x < PER; ++x) {
        const uint32_t c = gtid + x * G::NT;
        v[x] = 0; t[x] = 0;
        if (c < n_cand) {
            t[x] = sc.cand_pos[c];
            if constexpr (!BY_POS)
                v[x] = key64(BATCHED ? dot64_at_batched(Kt_head, hm, S_max, r, t[x], t_stride)
                                     : dot64_at(Kt_head, hm, S_max, r, t[x], t_stride));
            sc.cand_val[c] = v[x];
        }
    }
    G::sync();
#pragma unroll
    for (int x = 0; x < PER; ++x) {
        if (gtid + x * G::NT < n_cand) {
            uint32_t rank = 0;
            for (uint32_t i = 0; i < n_cand; ++i) {
                const unsigned long long vi = sc.cand_val[i];
                rank += (vi > v[x]) || (vi == v[x] && sc.cand_pos[i] < t[x]);
            }
            if (rank < need64) atomicOr(&sc.bm_sel[t[x] >> 5], 1u << (t[x] & 31));
            else atomicAnd(&sc.bm_sel[t[x] >> 5], ~(1u << (t[x] & 31)));
        }
    }
    G::sync();
}

// Stages a4 + a3 from the keys alone (any n): MSB radix select over all keys, 11 + 11 + 10 bits,
// then one pass for the softmax denominator, the bitmap and the threshold band.
template <class G, bool BY_POS = false, class KeysT>
__device__ __forceinline__ SelectResult select_generic(int gtid, const HeadMeta& hm, KeysT keys, uint32_t kmax,
                                                       float kabs, const PostScratch& sc, int r, int S_max,
                                                       const sparq_half* __restrict__ Kt_head, int t_stride = 1) {
    const int lane = gtid & 31, warp = gtid >> 5;
    const int n = hm.n_sel, k_eff = hm.k_sel;                // the ranked positions and places (all of them without a window)
    const float inv_tau = hm.inv_tau;
    const float vmax = unkey32(kmax);
    const float twoB = two_b(r, hm.l1_sel, kabs);

    // -------------------------------------------------------------- a4: top-k select
    // MSB radix select, 11 + 11 + 10 bits, leaving the loop as soon as a whole bin is wanted.
    // Afterwards the k_eff largest keys are those >= edge, except that `over` too many keys equal
    // edge when the fp32 sums tie at the threshold.
    uint32_t prefix = 0, mask = 0, need = (uint32_t)k_eff, ceq = 0;
    {
        int shift = 32;
#pragma unroll 1
        for (int pass = 0; pass < 3; ++pass) {
            const int bits = pass < 2 ? 11 : 10;
            shift -= bits;
            zero_hist<G>(sc.hist, gtid);
            G::sync();
            for (int t = gtid; t < n; t += G::NT) {
                const uint32_t u = key_full(keys, t);
                if ((u & mask) == prefix) atomicAdd(&sc.hist[(u >> shift) & ((1u << bits) - 1)], 1u);
            }
            G::sync();
            find_bin<G, HIST_BINS>(sc.hist, need, sc.redu, sc.res, gtid);
            prefix |= sc.res[0] << shift;
            mask |= ((1u << bits) - 1) << shift;
            need -= sc.res[1];
            ceq = sc.res[2];
            if (ceq == need) break;                          // the whole bin is selected: no need to split it
        }
    }
    const uint32_t edge = prefix;                            // unprocessed low bits are zero
    const uint32_t over = ceq - need;
    const float edge_val = unkey32(edge);
    const uint32_t lo_key = key32(__fadd_rd(edge_val, -twoB)), hi_key = key32(__fadd_ru(edge_val, twoB));

    // -------------------------------------------------------------- a3 + bitmap of the selection
    // Softmax denominator, the speculative selection key >= edge as a bitmap, and the positions
    // whose key lies within 2B of the edge (counted on each side, listed while the list has room).
    const int nwords = (hm.n + 31) >> 5;                     // the denominator runs over the window too
    const float c1 = inv_tau * LOG2E;
    if (gtid < 4) sc.band[gtid] = 0;
    G::sync();
    float zpart = 0.f;
    for (int wi = warp; wi < nwords; wi += G::NW) {
        const int t = (wi << 5) + lane;
        const uint32_t u = t < hm.n ? key_full(keys, t) : 0u;
        zpart += t < hm.n ? ex2((unkey32(u) - vmax) * c1) : 0.f;
        const bool valid = t < n;
        const bool ge = valid && u >= edge;
        const unsigned g = __ballot_sync(FULL, ge);
        if (lane == 0) sc.bm_sel[wi] = g;
        if (valid && u >= lo_key && u <= hi_key) {           // rare
            atomicAdd(&sc.band[ge ? 1 : 0], 1u);
            const uint32_t slot = atomicAdd(&sc.band[2], 1u);
            if (slot < CAND_MAX) sc.cand_pos[slot] = t;
        }
    }
    const float Z = group_sum<G>(zpart, sc.red, gtid);       // barriers also publish the bitmap and the band
    const uint32_t cnt_lo = sc.band[0], cnt_hi = sc.band[1], n_cand = sc.band[2];
    uint32_t need_tie = 0;
    if (over > 0 || (cnt_lo > 0 && cnt_hi > 0)) {
        // fp32 sums on both sides of the threshold are closer to it than their error bound (or
        // tie).  The n_cand positions in the band compete for cnt_hi - over places by their fp64
        // sums of exact products; equal fp64 sums go to the lowest positions.
        const uint32_t need64 = cnt_hi - over;
        if (n_cand <= CAND_MAX) {
            redecide_band<G, false, BY_POS>(gtid, hm, sc, n_cand, need64, Kt_head, S_max, r, t_stride);
        } else if constexpr (BY_POS) {
            // many equal keys at the threshold: all of them tie, the first need64 positions are taken
            need_tie = need64;
            for (int wi = warp; wi < nwords; wi += G::NW) {
                const int t = (wi << 5) + lane;
                const uint32_t u = t < n ? key_full(keys, t) : 0u;
                const unsigned g = __ballot_sync(FULL, t < n && u > hi_key);
                const unsigned te = __ballot_sync(FULL, t < n && u >= lo_key && u <= hi_key);
                if (lane == 0) { sc.bm_sel[wi] = g; sc.bm_tie[wi] = te; }
            }
            G::sync();
        } else {
            // many candidates (degenerate inputs, e.g. constant keys): radix select over their
            // 64-bit keys, 8 passes of 8 bits, then rebuild the bitmap
            unsigned long long p64 = 0, m64 = 0;
            uint32_t left = need64;
#pragma unroll 1
            for (int shift = 56; shift >= 0; shift -= 8) {
                zero_hist<G>(sc.hist, gtid);
                G::sync();
                for (int t = gtid; t < n; t += G::NT) {
                    const uint32_t u = key_full(keys, t);
                    if (u >= lo_key && u <= hi_key) {
                        const unsigned long long v = key64(dot64_at(Kt_head, hm, S_max, r, t, t_stride));
                        if ((v & m64) == p64) atomicAdd(&sc.hist[(uint32_t)(v >> shift) & 255u], 1u);
                    }
                }
                G::sync();
                find_bin<G, HIST_BINS>(sc.hist, left, sc.redu, sc.res, gtid);
                p64 |= (unsigned long long)sc.res[0] << shift;
                m64 |= 255ull << shift;
                left -= sc.res[1];
            }
            need_tie = left;
            for (int wi = warp; wi < nwords; wi += G::NW) {
                const int t = (wi << 5) + lane;
                const uint32_t u = t < n ? key_full(keys, t) : 0u;
                bool s_ = t < n && u > hi_key, tie = false;
                if (t < n && u >= lo_key && u <= hi_key) {
                    const unsigned long long v = key64(dot64_at(Kt_head, hm, S_max, r, t, t_stride));
                    s_ = v > p64;
                    tie = v == p64;
                }
                const unsigned g = __ballot_sync(FULL, s_), te = __ballot_sync(FULL, tie);
                if (lane == 0) { sc.bm_sel[wi] = g; sc.bm_tie[wi] = te; }
            }
            G::sync();
        }
    }

    SelectResult res;
    res.Z = Z;
    res.need_tie = need_tie;
    return res;
}

// First-digit histogram the stream stage fills while the keys are still in registers.
constexpr int FB = 10, FSH = 32 - FB, FBINS = 1 << FB;
constexpr int WIDE_DEPTH = 4;            // 256-position steps in flight per warp in the scan of keys in global memory (2: 2 % slower on c3; 8: no better)
constexpr int LIST_MAX = HIST_BINS / 2;  // (key, position) pairs of the threshold bin; the list lives in sc.hist

// Stages a4 + a3 when hist1 already holds the histogram of the keys' top FB bits.  One scan of the
// keys builds the bitmap of everything above the threshold bin, the softmax denominator and the list
// of the bin's own keys; the threshold is then resolved inside that short list, and the 2B band
// around it re-decided in fp64 as in select_generic.  Clears hist1 for its next user (not with WIDE).
// Returns false (for every thread of the group alike) when the short-cut does not apply -- the bin
// holds more keys than the list (with WIDE) or a warp's segment of it (without) has room for, or the
// band reaches outside the bin or holds too many keys -- and the caller runs select_generic instead.
// Z_stream: the softmax denominator relative to the largest key, accumulated by the stream stage.
template <class G, int FB_ = FB, bool WIDE = false, bool BY_POS = false, class KeysT>
__device__ __forceinline__ bool select_prefilled(int gtid, const HeadMeta& hm, KeysT keys, uint32_t kmax,
                                                 float kabs, float Z_stream, const PostScratch& sc, uint32_t* hist1, int r,
                                                 int S_max, const sparq_half* __restrict__ Kt_head, SelectResult& out,
                                                 int t_stride = 1) {
    constexpr int FSH_ = 32 - FB_, FBINS_ = 1 << FB_;         // first digit: the keys' top FB_ bits
    static_assert(FSH_ > 16 && FSH_ <= 24, "the bin's remaining bits resolve as 8 + 8 + (FSH_ - 16)");
    const int lane = gtid & 31, warp = gtid >> 5;
    const int n = hm.n_sel, k_eff = hm.k_sel;                // the ranked positions and places (all of them without a window)
    (void)kmax;

    POST_CLK_INIT();
    if (gtid < 4) sc.band[gtid] = 0;     // [0] band keys below the edge, [1] at/above it, [2] band list length
    find_bin<G, FBINS_>(hist1, (uint32_t)k_eff, sc.redu, sc.res, gtid);
    POST_CLK(0);
    const uint32_t b1 = sc.res[0], above = sc.res[1];
    if constexpr (!WIDE)                                     // (WIDE callers use a histogram once and may alias it with sc.hist)
        for (int i = gtid; i < FBINS_ / 4; i += G::NT) reinterpret_cast<uint4*>(hist1)[i] = make_uint4(0, 0, 0, 0);
    // the bin's own keys: every warp appends to its own segment of the list (no atomics), in the
    // order it meets them
    constexpr int SEG = LIST_MAX / G::NW;                    // (key, position) pairs per warp
    uint32_t* seg_key = sc.hist + warp * SEG;
    int32_t* seg_pos = reinterpret_cast<int32_t*>(sc.hist + LIST_MAX) + warp * SEG;
    const unsigned lt = (1u << lane) - 1;

    const int nwords = (n + 31) >> 5;
    uint32_t wcount = 0;                                     // this warp's list length (warp-uniform)
    if constexpr (WIDE) {
        // Keys in global memory.  A lane owns eight consecutive positions -- two 16-byte loads and one
        // whole byte of the bitmap, so no lane talks to another -- and a warp 256 positions per step,
        // WIDE_DEPTH steps in flight.  The bin's own keys are rare: a lane that meets some reserves their
        // places in the one list of the group with a single shared-memory atomic.  (With one warp
        // per scheduler, as in the 128-thread kernels, this scan is bound by its own instruction
        // stream, not by the loads: issuing every load twice changed its time by 5 %.)
        unsigned char* bm8 = reinterpret_cast<unsigned char*>(sc.bm_sel);
        uint32_t* list_key = sc.hist;
        int32_t* list_pos = reinterpret_cast<int32_t*>(sc.hist + LIST_MAX);
        const int nblocks = (n + 255) >> 8;
        for (int b0 = warp; b0 < nblocks; b0 += WIDE_DEPTH * G::NW) {
            uint4 kv[WIDE_DEPTH][2];
#pragma unroll
            for (int x = 0; x < WIDE_DEPTH; ++x) {
                const int t = ((b0 + x * G::NW) << 8) + lane * 8;        // a multiple of 8: both vectors lie inside the buffer
                kv[x][0] = t < n ? *reinterpret_cast<const uint4*>(keys + t) : make_uint4(0u, 0u, 0u, 0u);
                kv[x][1] = t < n ? *reinterpret_cast<const uint4*>(keys + t + 4) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int x = 0; x < WIDE_DEPTH; ++x) {
                const int t = ((b0 + x * G::NW) << 8) + lane * 8;
                if (t < nwords * 32) {                       // (the bytes of the last word past n are written too, as zeros)
                    const uint32_t u[8] = {kv[x][0].x, kv[x][0].y, kv[x][0].z, kv[x][0].w, kv[x][1].x, kv[x][1].y, kv[x][1].z, kv[x][1].w};
                    uint32_t sel8 = 0, inb = 0;
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        const uint32_t dig = u[e] >> FSH_;
                        sel8 |= (dig > b1) ? 1u << e : 0u;
                        inb |= (dig == b1) ? 1u << e : 0u;
                    }
                    const int rem = n - t;                   // valid positions among the eight
                    if (rem < 8) { const uint32_t vm = rem > 0 ? (1u << rem) - 1u : 0u; sel8 &= vm; inb &= vm; }
                    bm8[t >> 3] = (unsigned char)sel8;
                    if (inb) {
                        uint32_t slot = atomicAdd(&sc.band[3], (uint32_t)__popc(inb));
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            if ((inb >> e) & 1u) {
                                if (slot < (uint32_t)LIST_MAX) { list_key[slot] = u[e]; list_pos[slot] = t + e; }
                                ++slot;
                            }
                        }
                    }
                }
            }
        }
    } else if constexpr (keys_split<KeysT>::value) {
        // Split keys: the upper halves of eight consecutive keys are one 16-byte vector of shared memory.
        // A lane owns such a vector -- one load, one whole byte of the bitmap -- and the bin's own keys
        // go to the one list of the group, as above; their lower halves are fetched after the scan.
        unsigned char* bm8 = reinterpret_cast<unsigned char*>(sc.bm_sel);
        uint32_t* list_key = sc.hist;
        int32_t* list_pos = reinterpret_cast<int32_t*>(sc.hist + LIST_MAX);
        constexpr int HSH = FSH_ - 16;                       // the first digit inside an upper half
        for (int v = gtid; v < nwords * 4; v += G::NT) {     // (the bytes of the last word past n are written too, as zeros)
            const int t = v << 3;
            const uint4 kv = t < n ? *reinterpret_cast<const uint4*>(keys.hi + t) : make_uint4(0u, 0u, 0u, 0u);
            const uint32_t w[4] = {kv.x, kv.y, kv.z, kv.w};
            uint32_t sel8 = 0, inb = 0;
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const uint32_t dig = ((e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xffffu)) >> HSH;
                sel8 |= (dig > b1) ? 1u << e : 0u;
                inb |= (dig == b1) ? 1u << e : 0u;
            }
            const int rem = n - t;                           // valid positions among the eight
            if (rem < 8) { const uint32_t vm = rem > 0 ? (1u << rem) - 1u : 0u; sel8 &= vm; inb &= vm; }
            bm8[v] = (unsigned char)sel8;
            if (inb) {
                uint32_t slot = atomicAdd(&sc.band[3], (uint32_t)__popc(inb));
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    if ((inb >> e) & 1u) {
                        if (slot < (uint32_t)LIST_MAX) {
                            list_key[slot] = ((e & 1) ? (w[e >> 1] >> 16) : (w[e >> 1] & 0xffffu)) << 16;
                            list_pos[slot] = t + e;
                        }
                        ++slot;
                    }
                }
            }
        }
    } else {
        for (int w0 = warp; w0 < nwords; w0 += 4 * G::NW) {      // four words in flight per warp
            uint32_t u[4];
            bool valid[4];
    #pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int t = ((w0 + x * G::NW) << 5) + lane;
                valid[x] = t < n;                                // also false for words past the end
                u[x] = valid[x] ? key_coarse(keys, t) : 0u;
            }
    #pragma unroll
            for (int x = 0; x < 4; ++x) {
                const int wi = w0 + x * G::NW;
                if (wi < nwords) {                               // warp-uniform
                    const uint32_t dig = u[x] >> FSH_;
                    const unsigned g = __ballot_sync(FULL, valid[x] && dig > b1);
                    const unsigned inb = __ballot_sync(FULL, valid[x] && dig == b1);
                    if (lane == 0) sc.bm_sel[wi] = g;
                    if (inb) {
                        const uint32_t slot = wcount + __popc(inb & lt);
                        if ((inb >> lane & 1u) && slot < SEG) { seg_key[slot] = u[x]; seg_pos[slot] = (wi << 5) + lane; }
                        wcount += __popc(inb);
                    }
                }
            }
        }

    }
    if (lane == 0) sc.redu[G::NW + warp] = wcount;
    G::sync();                                               // publishes the bitmap and the lists
    out.Z = Z_stream;
    out.need_tie = 0;
    POST_CLK(1);
    constexpr bool ONE_LIST = WIDE || keys_split<KeysT>::value;   // one list of the group, or a segment per warp
    uint32_t m = 0;
    bool fits = true;
    if constexpr (ONE_LIST) {
        m = sc.band[3];
        fits = m <= (uint32_t)LIST_MAX;
    } else {
#pragma unroll
        for (int w = 0; w < G::NW; ++w) { const uint32_t c = sc.redu[G::NW + w]; m += c; fits = fits && c <= SEG; }
    }
    if (!fits) return false;
    // this thread's walk over the list(s): its warp's segment, or its share of the group's one list
    uint32_t* my_key = ONE_LIST ? sc.hist : seg_key;
    const int32_t* my_pos = ONE_LIST ? reinterpret_cast<const int32_t*>(sc.hist + LIST_MAX) : seg_pos;
    const uint32_t my_first = ONE_LIST ? (uint32_t)gtid : (uint32_t)lane, my_step = ONE_LIST ? (uint32_t)G::NT : 32u;
    const uint32_t my_n = ONE_LIST ? m : min(wcount, (uint32_t)SEG);
    if constexpr (keys_split<KeysT>::value) {
        // the scan listed the keys' upper halves; every thread completes the entries it walks below
        for (uint32_t i = my_first; i < my_n; i += my_step) my_key[i] |= (uint32_t)__ldcg(keys.lo + my_pos[i]);
    }

    // the threshold among the bin's m keys: `need` of them are wanted; remaining bits as 8 + 8 + the rest
    uint32_t need = (uint32_t)k_eff - above, prefix = b1 << FSH_, mask = ~0u << FSH_, ceq = m;
    // One 256-bin histogram per pass, all cleared up front, and every warp scanning the finished
    // histogram for itself: one barrier per pass instead of three.
    static_assert(CAND_MAX * 12 >= 3 * 256 * 4, "three histograms fit cand_val + cand_pos, free until the band step");
    uint32_t* h256 = reinterpret_cast<uint32_t*>(sc.cand_val);
    const float twoB = two_b(r, hm.l1_sel, kabs);
    int shift = FSH_, pass = 0;
    bool cleared = ceq != need;
    if (cleared) {
        for (int i = gtid; i < 3 * 256; i += G::NT) h256[i] = 0;
        G::sync();
    }
    // The first go stops as soon as a whole (sub-)bin is wanted: `prefix` is then that bin's lower edge, not a
    // key.  If that edge lies so low in the first-digit bin that the 2B band below it would leave the
    // bin (typically: every key of the bin is wanted, one unit in a few hundred), a second go carries on to the
    // exact smallest wanted key, whose band almost surely stays inside.
#pragma unroll 1
    for (int go = 0; go < 2; ++go) {
#pragma unroll 1
        for (; pass < 3 && (go == 1 || ceq != need); ++pass) {
            const int bits = pass < 2 ? 8 : FSH_ - 16;
            shift -= bits;
            uint32_t* hcur = h256 + pass * 256;
            for (uint32_t i = my_first; i < my_n; i += my_step) {
                const uint32_t u = my_key[i];
                if ((u & mask) == prefix) atomicAdd(&hcur[(u >> shift) & ((1u << bits) - 1)], 1u);
            }
            G::sync();
            // 8 bins per lane, from the top; the lane whose range holds the need-th key knows the answer
            uint32_t c[8], sum = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { c[i] = hcur[255 - (lane * 8 + i)]; sum += c[i]; }
            uint32_t incl = sum;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const uint32_t x = __shfl_up_sync(FULL, incl, o); if (lane >= o) incl += x; }
            uint32_t run = incl - sum, bin = 0, cnt = 0;
            const bool mine = run < need && need <= incl;
            if (mine) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (run + c[i] >= need) { bin = 255 - (lane * 8 + i); cnt = c[i]; break; }
                    run += c[i];
                }
            }
            const int src = __ffs(__ballot_sync(FULL, mine)) - 1;    // exactly one lane
            bin = __shfl_sync(FULL, bin, src);
            run = __shfl_sync(FULL, run, src);
            cnt = __shfl_sync(FULL, cnt, src);
            prefix |= bin << shift;
            mask |= ((1u << bits) - 1) << shift;
            need -= run;
            ceq = cnt;
        }
        if (pass == 3 || (key32(__fadd_rd(unkey32(prefix), -twoB)) >> FSH_) == b1) break;   // (uniform)
        if (go == 0 && !cleared) {
            for (int i = gtid; i < 3 * 256; i += G::NT) h256[i] = 0;
            G::sync();
        }
    }
    POST_CLK(2);
    const uint32_t edge = prefix;                            // unprocessed low bits are zero
    const uint32_t over = ceq - need;
    const float edge_val = unkey32(edge);
    const uint32_t lo_key = key32(__fadd_rd(edge_val, -twoB)), hi_key = key32(__fadd_ru(edge_val, twoB));
    if ((lo_key >> FSH_) != b1 || (hi_key >> FSH_) != b1) return false;   // keys outside the list may be in the band

    for (uint32_t i = my_first; i < my_n; i += my_step) {
        const uint32_t u = my_key[i];
        const int t = my_pos[i];
        if (u >= edge) atomicOr(&sc.bm_sel[t >> 5], 1u << (t & 31));
        if (u >= lo_key && u <= hi_key) {
            atomicAdd(&sc.band[u >= edge ? 1 : 0], 1u);
            const uint32_t slot = atomicAdd(&sc.band[2], 1u);
            if (slot < CAND_MAX) sc.cand_pos[slot] = t;
        }
    }
    G::sync();
    const uint32_t cnt_lo = sc.band[0], cnt_hi = sc.band[1], n_cand = sc.band[2];
    if (over > 0 || (cnt_lo > 0 && cnt_hi > 0)) {
        if (n_cand > CAND_MAX) return false;
        redecide_band<G, WIDE, BY_POS>(gtid, hm, sc, n_cand, cnt_hi - over, Kt_head, S_max, r, t_stride);
    }
    POST_CLK(3);
    return true;
}

// Local window, before a select that starts from a first-digit histogram of all n keys: take the
// window's keys out of it again (at most SPARQ_K_MAX of them).  Ends with a barrier.
template <class G, int FB_ = FB, class KeysT>
__device__ __forceinline__ void window_unhist(int gtid, const HeadMeta& hm, KeysT keys, uint32_t* hist1) {
    for (int t = hm.n_sel + gtid; t < hm.n; t += G::NT) atomicSub(&hist1[key_coarse(keys, t) >> (32 - FB_)], 1u);
    G::sync();
}

// Local window, after the select: positions [n_sel, n) join the selection.  The select wrote the
// bitmap words that hold ranked positions; the words above them are set here.  Ends with a barrier.
template <class G>
__device__ __forceinline__ void window_mark(int gtid, const HeadMeta& hm, const PostScratch& sc) {
    const int n_sel = hm.n_sel, n = hm.n;
    const int ranked_words = (n_sel + 31) >> 5;
    for (int wi = (n_sel >> 5) + gtid; wi <= ((n - 1) >> 5); wi += G::NT) {
        const int lo = max(n_sel - (wi << 5), 0), hi = min(n - (wi << 5), 32);       // bits [lo, hi) of this word
        const uint32_t mask = (hi == 32 ? ~0u : (1u << hi) - 1u) & ~((1u << lo) - 1u);
        sc.bm_sel[wi] = (wi < ranked_words ? sc.bm_sel[wi] : 0u) | mask;
    }
    G::sync();
}

// Local window as large as the budget (k_sel = 0): nothing is ranked.  Clears the bitmap words of the
// older positions; Z = the softmax denominator relative to the largest key, from the keys.
template <class G, class KeysT>
__device__ __forceinline__ SelectResult select_nothing(int gtid, const HeadMeta& hm, KeysT keys, uint32_t kmax,
                                                       const PostScratch& sc) {
    const float vmax = unkey32(kmax), c1 = hm.inv_tau * LOG2E;
    for (int wi = gtid; wi < ((hm.n_sel + 31) >> 5); wi += G::NT) sc.bm_sel[wi] = 0u;
    float zpart = 0.f;
    for (int t = gtid; t < hm.n; t += G::NT) zpart += ex2((unkey32(key_full(keys, t)) - vmax) * c1);
    SelectResult res;
    res.Z = group_sum<G>(zpart, sc.red, gtid);               // its barriers publish the bitmap
    res.need_tie = 0;
    return res;
}

// The ascending list sc.i2 of the k_eff selected positions from the selection bitmap (plus, in the
// degenerate path, the first need_tie positions of the tie bitmap).  Ends with a barrier.
template <class G>
__device__ __forceinline__ void build_index_list(int gtid, const HeadMeta& hm, SelectResult sel, const PostScratch& sc) {
    const int n = hm.n, k_eff = hm.k_eff;
    const int nwords = (n + 31) >> 5;
    const uint32_t need_tie = sel.need_tie;
    uint32_t carry_tie = 0, carry_sel = 0;
    for (int base = 0; base < nwords; base += G::NT) {
        const int wi = base + gtid;
        uint32_t g = wi < nwords ? sc.bm_sel[wi] : 0u;
        if (need_tie) {                                      // add the first need_tie tied positions
            uint32_t e = wi < nwords ? sc.bm_tie[wi] : 0u, tot;
            const uint32_t ce = __popc(e);
            const uint32_t before = carry_tie + group_scan_incl<G>(ce, sc.redu, &tot, gtid) - ce;
            const uint32_t allowed = before >= need_tie ? 0u : min(ce, need_tie - before);
            while ((uint32_t)__popc(e) > allowed) e &= ~(0x80000000u >> __clz(e));
            g |= e;
            carry_tie += tot;
        }
        uint32_t tot;
        const uint32_t cs = __popc(g);
        uint32_t off = carry_sel + group_scan_incl<G>(cs, sc.redu, &tot, gtid) - cs;
        while (g) {
            const int bit = __ffs(g) - 1;
            if (off < (uint32_t)k_eff) sc.i2[off] = (wi << 5) + bit;
            ++off;
            g &= g - 1;
        }
        carry_sel += tot;
    }
    G::sync();
}

// Stages a5 and a6 for one unit from a finished selection: ascending index list from the bitmap(s),
// alpha, gather of the selected K and V rows with online softmax, combine with v_bar.
// RG: gathered K and V rows in flight per half-warp (register budget of the calling kernel).
// realloc = false leaves Step 3 out (out = the restricted attention; alpha is still reported).
// Writes out_row (fp16), alpha_out and idx_k_row when not NULL.  Ends with every thread of the
// group past its last read of keys and scratch except sc.i2 (read by the idx_k copy at the end).
template <class G, int RG, class KeysT>
__device__ __forceinline__ void finish(int gtid, const HeadMeta& hm, KeysT keys, uint32_t kmax, SelectResult sel,
                                       const PostScratch& sc, int k, const sparq_half* __restrict__ K_head,
                                       const sparq_half* __restrict__ V_head, const sparq_half* __restrict__ vbar_head,
                                       sparq_half* __restrict__ out_row, int32_t* __restrict__ idx_k_row,
                                       float* __restrict__ alpha_out, bool build_list = true, bool realloc = true) {
    const int n = hm.n, k_eff = hm.k_eff;
    const float vmax = unkey32(kmax);
    const float c1 = hm.inv_tau * LOG2E;
    const float Z = sel.Z;
    POST_CLK_INIT();
    if (build_list) build_index_list<G>(gtid, hm, sel, sc);  // (a caller that kept sc.i2 from an earlier call skips the rebuild)
    else G::sync();
    // start the selected rows on their way from HBM to L2 now; the gather below reads them a few
    // barriers later (two 128-byte lines per row and tensor)
    for (int i = gtid; i < 4 * k_eff; i += G::NT) {
        const int t = min(max(sc.i2[i >> 2], 0), n - 1);
        const sparq_half* row = ((i & 2) ? V_head : K_head) + (size_t)t * D + (i & 1) * (D / 2);
        asm volatile("prefetch.global.L2 [%0];" ::"l"(row));
    }
    // alpha = approximate-score mass of the selected set (Step 3)
    float apart = 0.f;
    for (int j = gtid; j < k_eff; j += G::NT) apart += ex2((unkey32(key_full(keys, min(max(sc.i2[j], 0), n - 1))) - vmax) * c1);
    // (numerator and denominator are fp32 sums taken in different orders: keep the mass a probability)
    const float alpha = fminf(group_sum<G>(apart, sc.red, gtid) / Z, 1.0f);
    POST_CLK(4);

    // -------------------------------------------------------------- a5: gather k rows of K and V
    const int hw = gtid >> 4, l16 = gtid & 15;
    const float qscale = rsqrtf((float)D) * LOG2E;
    const uint4 q8 = *reinterpret_cast<const uint4*>(hm.q16 + l16 * 8);   // this lane's 8 query components, fp16
    const uint32_t qw[4] = {q8.x, q8.y, q8.z, q8.w};
    const uint4* Kh = reinterpret_cast<const uint4*>(K_head);
    const uint4* Vh = reinterpret_cast<const uint4*>(V_head);
    float m = -CUDART_INF_F, l = 0.f, acc[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) acc[e] = 0.f;
    for (int jb = 0; jb < k_eff; jb += G::NHW * RG) {        // trip count uniform across the group
        uint4 kv[RG], vv[RG];
#pragma unroll
        for (int u = 0; u < RG; ++u) {
            // (the clamp keeps the address inside the head even if the list were ever corrupt)
            const int t = min(max(sc.i2[min(jb + u * G::NHW + hw, k_eff - 1)], 0), n - 1);
            kv[u] = ld_stream(Kh + (size_t)t * (D / 8) + l16);
            vv[u] = ld_stream(Vh + (size_t)t * (D / 8) + l16);
        }
        float z[RG], bmax = -CUDART_INF_F;
#pragma unroll
        for (int u = 0; u < RG; ++u) {
            const uint32_t kw[4] = {kv[u].x, kv[u].y, kv[u].z, kv[u].w};
            float zz = 0.f, zz2 = 0.f;                       // exact fp16 products, two fp32 chains
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                fma_h(zz, (uint16_t)(kw[e] & 0xffffu), (uint16_t)(qw[e] & 0xffffu));
                fma_h(zz2, (uint16_t)(kw[e] >> 16), (uint16_t)(qw[e] >> 16));
            }
            zz = (zz + zz2) * qscale;
#pragma unroll
            for (int o = 8; o > 0; o >>= 1) zz += __shfl_xor_sync(FULL, zz, o);
            z[u] = (jb + u * G::NHW + hw < k_eff) ? zz : -CUDART_INF_F;   // uniform within the half-warp
            bmax = fmaxf(bmax, z[u]);
        }
        const float mn = fmaxf(m, bmax);
        if (mn > -CUDART_INF_F) {
            const float scl = ex2(m - mn);
            l *= scl;
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[e] *= scl;
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
    POST_CLK(5);
    // merge the half-warps' partial softmax states
    float* mg = sc.merge + hw * (D + 2);
#pragma unroll
    for (int e = 0; e < 8; ++e) mg[l16 * 8 + e] = acc[e];
    if (l16 == 0) { mg[D] = m; mg[D + 1] = l; }
    G::sync();

    // -------------------------------------------------------------- a6: combine with v_bar
    if (gtid < D) {
        const float vb = __half2float(__ushort_as_half(vbar_head[gtid]));
        float M = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < G::NHW; ++w) M = fmaxf(M, sc.merge[w * (D + 2) + D]);
        float L = 0.f, s = 0.f;
#pragma unroll
        for (int w = 0; w < G::NHW; ++w) {
            const float scl = ex2(sc.merge[w * (D + 2) + D] - M);
            L = fmaf(sc.merge[w * (D + 2) + D + 1], scl, L);
            s = fmaf(sc.merge[w * (D + 2) + gtid], scl, s);
        }
        out_row[gtid] = __half_as_ushort(__float2half_rn(realloc ? alpha * (s / L) + (1.f - alpha) * vb : s / L));
    }
    if (gtid == 0 && alpha_out) *alpha_out = alpha;
    if (idx_k_row) for (int j = gtid; j < k; j += G::NT) idx_k_row[j] = (j < k_eff) ? sc.i2[j] : -1;
    POST_CLK(6);
}

}  // namespace sparq
