// sparq_decode, persistent warp-specialised kernel: one CTA per SM walks over (batch, query head)
// units, and the three kinds of work of a unit run on different warps so that the HBM stream
// never waits for the latency-bound stages:
//
//   a1 warp           top-r of |q| and tau for the units ahead (metadata slots), off everyone's path
//   producer warps    the bulk asynchronous copies (cp.async.bulk + mbarrier, no multicast) of the
//                     r selected Kt rows into a ring of shared-memory stages; two warps take
//                     alternate stages and lanes issue one row each, because one thread (and even
//                     one warp) can only start a copy every few hundred cycles
//   stream group      a2: consumes the ring, fp32 mixed-precision FMA chain per position, writes the
//                     order-preserving keys of unit j into key buffer j mod NKB (4 where they fit, else 3)
//   post groups 0/1   a3-a6 of units j = 0,2,4,.. / 1,3,5,.. (decode_common.cuh): radix select with
//                     exact re-decision of the threshold band, alpha, K/V row gather, combine
//
// Hand-offs are mbarriers (ring full/empty, unit metadata full/free, key buffer full/free); every
// wait is bounded: a wait that gives up raises SPARQ_DEV_TIMEOUT and sets a CTA-wide flag after
// which no wait blocks any more, so the kernel always terminates.
#include "decode_common.cuh"
#include "kernels.h"

namespace sparq {
namespace {

constexpr int SNT = 256;                 // stream-group threads
constexpr int GNT = 256;                 // threads of one post group
constexpr int NPOST = 2;
constexpr int NPROD = 2;                 // producer warps (one warp alone cannot start copies fast enough)
constexpr int LEAD = 32 * (NPROD + 1);   // producer warps + a1 warp
constexpr int NT = LEAD + SNT + NPOST * GNT;
constexpr int CH = SNT * 8;              // positions per chunk: 8 per stream thread (one 16-byte vector)
// The ring: RB Kt rows per stage.  3 stages of 8 rows (32 KB stages: fewer hand-offs beat a deeper ring,
// measured), or, where the longest caches of the split-key form leave less room, 4 stages of 4 rows (64 KB).
// Split keys (K16): the keys' upper halves in shared memory, the lower halves in the caller's workspace,
// where the L2 keeps them; for caches whose 32-bit keys do not fit three times beside the ring.
// RING: 0 = 3 x 32 KB, 1 = 4 x 16 KB, 2 = 5 x 16 KB (the split-key form's longest caches, when the budget k is
// small enough for the fifth stage to fit beside the index lists).
template <int RING>
struct Ring {
    static constexpr int RB = RING ? 4 : 8;
    static constexpr int STAGES = RING == 0 ? 3 : RING == 1 ? 4 : 5;
    static constexpr int STAGE_BYTES = RB * CH * 2;
    static constexpr int BYTES = STAGES * STAGE_BYTES;
};
constexpr int STAGES_MAX = 5;
// entries of one post group's index list i2 in dynamic shared memory (k rounded up to whole 128-byte lines)
__host__ __device__ constexpr int i2_pad(int k) { return ((k > 0 ? k : 1) + 31) & ~31; }
__host__ __device__ constexpr size_t post_scratch_aligned(int S_cap) { return (post_scratch_bytes(GNT / 16, S_cap / 32) + 127) & ~(size_t)127; }
constexpr int NKB_MAX = 4;               // key buffers: one being written, the others waiting for or in the post groups;
                                         // four where they fit (1.7 us faster on the bench shape), else three
constexpr int NMETA = 4;                 // unit metadata slots in flight
using SG = Group<SNT, 1>;
using PG0 = Group<GNT, 2>;
using PG1 = Group<GNT, 3>;

// Optional cycle counters for tuning (-DSPARQ_PHASE_CLOCKS): [0] post phase, [1] post waiting for keys,
// [2] stream waiting for a free key buffer, [3] stream waiting for ring data, [4] stream total per unit,
// [5] producer waiting for a free ring slot, [6] producer a1, [7] units that took the generic select (a count)
#ifdef SPARQ_PHASE_CLOCKS
__device__ unsigned long long g_cta_end[256];
__device__ unsigned long long g_cta_begin[256];
__device__ unsigned long long g_pipe_clocks[16];
#define CLK_BEGIN(var) long long var = clock64()
#define CLK_ADD(i, var, cond) do { if (cond) atomicAdd(&g_pipe_clocks[i], (unsigned long long)(clock64() - var)); } while (0)
#else
#define CLK_BEGIN(var)
#define CLK_ADD(i, var, cond)
#endif

template <bool K16>
struct PipeSharedT {
    HeadMeta meta[NMETA];
    int32_t i2[NPOST][K16 ? 8 : SPARQ_K_MAX];     // (split keys: the lists live in dynamic shared memory)
    uint64_t full[STAGES_MAX], empty[STAGES_MAX];          // ring stage landed / consumed
    uint64_t meta_full[NMETA], meta_free[NMETA];   // a1 done / unit finished
    uint64_t keys_full[NKB_MAX], keys_free[NKB_MAX];   // keys of a unit complete / post-processed
    uint32_t kmax[NKB_MAX];
    float kabs[NKB_MAX];
    float zsum[NKB_MAX];                              // softmax denominator of the unit's approximate scores
    float sred[2 * (SNT / 32)];
    float red[NPOST][2 * (GNT / 32)];
    uint32_t redu[NPOST][2 * (GNT / 32)];
    uint32_t res[NPOST][4];
    uint32_t band[NPOST][4];
    uint32_t sredu[2 * (SNT / 32)];
    int abort_flag;
};

constexpr size_t SPLIT_LO_OFFSET = 256;
struct Args {
    const sparq_half *q, *K, *Kt, *V, *vbar;
    const int32_t* seq_lens;
    int n_units, Hq, Hkv, S_max, S_cap, r, k;
    sparq_half* out;
    int32_t *idx_r, *idx_k;
    float* alpha;
    int32_t* status;
    unsigned int* unit_counter;   // zeroed device word for dynamic unit assignment, or NULL: static stride; with split
                                  // keys their lower halves follow SPLIT_LO_OFFSET bytes behind it, [gridDim.x][NKB][S_cap]
};

// (A member of its own for this pointer made the struct larger and every instantiation of the kernel
// spill a few registers, the ones that never use it included.)
template <int NKB>
__device__ __forceinline__ uint16_t* split_lo(const Args& a, int kb) {
    return reinterpret_cast<uint16_t*>(reinterpret_cast<unsigned char*>(a.unit_counter) + SPLIT_LO_OFFSET) +
           ((size_t)blockIdx.x * NKB + kb) * a.S_cap;
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// Bounded wait.  Between polls the warp sleeps NS nanoseconds so that waiting warps leave the issue
// slots to the working ones.  Gives up after WAIT_LIMIT polls, or at once when another thread
// already gave up; from then on no wait in this CTA blocks.
template <int NS, class SH>
__device__ __forceinline__ void wait_or_abort(uint64_t* bar, uint32_t parity, SH& sh, int32_t* status) {
    volatile int* flag = &sh.abort_flag;
    for (int i = 0; i < WAIT_LIMIT; ++i) {
        if (mbar_try_wait(bar, parity)) return;
        if ((i & 63) == 63 && *flag) return;
        __nanosleep(NS);
    }
    *flag = 1;
    raise_status(status, SPARQ_DEV_TIMEOUT);
}

// The same for a whole thread group: its first warp polls, the other warps sleep in the group's
// hardware barrier instead of spending issue slots on polls.
template <class G, int NS, class SH>
__device__ __forceinline__ void group_wait(int gtid, uint64_t* bar, uint32_t parity, SH& sh, int32_t* status) {
    if (gtid < 32) wait_or_abort<NS>(bar, parity, sh, status);
    G::sync();
}

// ---------------------------------------------------------------------------------- a1 warp
// Units are handed out first come, first served when a zeroed counter is available (CTAs differ by
// 10-20 % in how fast they get through a unit, so a fixed share per CTA leaves the last ones
// running alone); without a counter CTA i takes units i, i + gridDim.x, ...  After the last unit
// the a1 warp publishes NPOST end markers (bh = -1), one for each post group.
__device__ __forceinline__ int next_unit(const Args& a, int bh, int lane) {
    int u = bh + (int)gridDim.x;
    if (a.unit_counter) {
        if (lane == 0) u = (int)gridDim.x + (int)atomicAdd(a.unit_counter, 1u);
        u = __shfl_sync(FULL, u, 0);
    }
    return u < a.n_units ? u : -1;
}

template <int RB, class SH>
__device__ __forceinline__ void a1_role(const Args& a, SH& sh, const uint32_t opts) {
    const int lane = threadIdx.x & 31;
    int bh = (int)blockIdx.x < a.n_units ? (int)blockIdx.x : -1;
    uint2 qraw = make_uint2(0, 0);                           // components 4*lane .. 4*lane+3 of the unit's q
    int n_next = 0;
    if (bh >= 0) {
        qraw = *reinterpret_cast<const uint2*>(a.q + (size_t)bh * D + lane * 4);
        n_next = a.seq_lens[bh / a.Hq];
    }
    int markers = 0;
    for (int j = 0; markers < NPOST; ++j) {
        const int m = j % NMETA;
        HeadMeta& hm = sh.meta[m];
        if (bh < 0) {                                        // no unit left: an end marker for one post group
            wait_or_abort<200>(&sh.meta_free[m], (((uint32_t)(j / NMETA)) & 1u) ^ 1u, sh, a.status);
            if (lane == 0) { hm.bh = -1; hm.n = 0; hm.k_eff = 0; hm.valid = 0; hm.n_sel = 0; hm.k_sel = 0; }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh.meta_full[m]);
            ++markers;
            continue;
        }
        // key = |q_c| bits above (127 - c): distinct keys, larger |q| first, then smaller c
        const int n = n_next;
        const bool valid = n >= 1 && n <= a.S_max;
        const int k_eff = valid ? min(a.k, n) : 0;
        const uint16_t hb[4] = {(uint16_t)(qraw.x & 0xffffu), (uint16_t)(qraw.x >> 16), (uint16_t)(qraw.y & 0xffffu),
                                (uint16_t)(qraw.y >> 16)};
        wait_or_abort<200>(&sh.meta_free[m], (((uint32_t)(j / NMETA)) & 1u) ^ 1u, sh, a.status);
        CLK_BEGIN(t_a1);
        float qf[4], l1_all = 0.f;
        uint32_t mine[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int c = lane * 4 + e;
            qf[e] = __half2float(__ushort_as_half(hb[e]));
            l1_all += fabsf(qf[e]);
            mine[e] = ((uint32_t)(hb[e] & 0x7fffu) << 7) | (uint32_t)(D - 1 - c);
            hm.q16[c] = hb[e];
            hm.rkey[c] = mine[e];
        }
        __syncwarp();
        int rank[4] = {0, 0, 0, 0};
        const uint4* rk4 = reinterpret_cast<const uint4*>(hm.rkey);
#pragma unroll 4
        for (int i = 0; i < D / 4; ++i) {
            const uint4 o = rk4[i];
#pragma unroll
            for (int e = 0; e < 4; ++e) rank[e] += (o.x > mine[e]) + (o.y > mine[e]) + (o.z > mine[e]) + (o.w > mine[e]);
        }
        int cnt = 0;
        float l1_sel = 0.f;
        bool sel[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) { sel[e] = rank[e] < a.r; cnt += sel[e]; l1_sel += sel[e] ? fabsf(qf[e]) : 0.f; }
        int incl = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const int x = __shfl_up_sync(FULL, incl, o); if (lane >= o) incl += x; }
        int slot = incl - cnt;                               // ascending component order: by lane, then e
#pragma unroll
        for (int e = 0; e < 4; ++e) if (sel[e]) { hm.i1[slot] = lane * 4 + e; hm.qh[slot] = hb[e]; ++slot; }
        l1_all = warp_sum(l1_all);
        l1_sel = warp_sum(l1_sel);
        const int r_pad = (a.r + RB - 1) / RB * RB;
        for (int c = a.r + lane; c < r_pad; c += 32) hm.qh[c] = 0;
        if (lane == 0) {
            hm.bh = bh; hm.n = n; hm.k_eff = k_eff; hm.valid = valid;
            hm.inv_tau = opt_inv_tau(opts, l1_all, l1_sel, a.r);
            hm.l1_sel = l1_sel;
            opt_set_window(hm, n, k_eff, opts);
        }
        __syncwarp();
        if (a.idx_r) for (int c = lane; c < a.r; c += 32) a.idx_r[(size_t)bh * a.r + c] = valid ? hm.i1[c] : -1;
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh.meta_full[m]);
        CLK_ADD(6, t_a1, lane == 0);
        // Only now draw the next unit and fetch its query and length: the stream group has a whole unit
        // to work on meanwhile, and the first unit of the launch is not held up by the draw.  (Drawing
        // later still -- once the stream group has started on this unit -- would leave fewer drawn but
        // unstarted units per CTA at the end of the launch; it measured slower, the draw landing on the
        // critical path.)
        bh = next_unit(a, bh, lane);
        if (bh >= 0) {
            qraw = *reinterpret_cast<const uint2*>(a.q + (size_t)bh * D + lane * 4);
            n_next = a.seq_lens[bh / a.Hq];
        }
    }
}

// ---------------------------------------------------------------------------------- producer
template <int RING, class SH>
__device__ __forceinline__ void producer_role(const Args& a, SH& sh, unsigned char* ring, int p) {
    constexpr int RB = Ring<RING>::RB, STAGES = Ring<RING>::STAGES, STAGE_BYTES = Ring<RING>::STAGE_BYTES;
    const int lane = threadIdx.x & 31;
    const int g_heads = a.Hq / a.Hkv;
    uint32_t g = 0;                                          // ring stages issued so far
    for (int j = 0, markers = 0; markers < NPOST; ++j) {
        const int m = j % NMETA;
        const HeadMeta& hm = sh.meta[m];
        wait_or_abort<100>(&sh.meta_full[m], ((uint32_t)(j / NMETA)) & 1u, sh, a.status);
        if (hm.bh < 0 || sh.abort_flag) { ++markers; continue; }
        // the unit's ring stages: [chunk c][row batch jb] -> RB rows x CH positions
        if (hm.k_eff > 0) {
            const int bh = hm.bh, b = bh / a.Hq, h = bh % a.Hq, n = hm.n;
            const sparq_half* Kt_head = a.Kt + ((size_t)b * a.Hkv + h / g_heads) * (size_t)D * a.S_max;
            const int n8 = (n + 7) & ~7;
            const int n_chunks = (n8 + CH - 1) / CH;
            for (int c = 0; c < n_chunks; ++c) {
                const uint32_t bytes = (uint32_t)min(CH, n8 - c * CH) * 2u;
                for (int jb = 0; jb < a.r; jb += RB, ++g) {
                    if ((int)(g % NPROD) != p) continue;     // the other producer warp's stage
                    const int s = g % STAGES;
                    const int rows = min(RB, a.r - jb);
                    wait_or_abort<40>(&sh.empty[s], ((g / STAGES) & 1u) ^ 1u, sh, a.status);
                    if (lane == 0) mbar_expect_tx(&sh.full[s], bytes * rows);
                    __syncwarp();
                    if (lane < rows)
                        bulk_g2s(ring + s * STAGE_BYTES + lane * (CH * 2),
                                 Kt_head + (size_t)hm.i1[jb + lane] * a.S_max + c * CH, bytes, &sh.full[s]);
                }
            }
        }
    }
}

// ---------------------------------------------------------------------------------- stream group
template <int NKB, bool K16, int RING, class SH>
__device__ __forceinline__ void stream_role(const Args& a, SH& sh, const unsigned char* ring, uint32_t* keys_all,
                                            uint32_t* hist1_all) {
    constexpr int RB = Ring<RING>::RB, STAGES = Ring<RING>::STAGES, STAGE_BYTES = Ring<RING>::STAGE_BYTES;
    const int gtid = threadIdx.x - LEAD, lane = gtid & 31;
    int s = 0;                                               // ring slot and its phase parity
    uint32_t parity = 0;
    for (int j = 0, markers = 0; markers < NPOST; ++j) {
        const int m = j % NMETA, kb = j % NKB;
        const HeadMeta& hm = sh.meta[m];
        uint32_t* keys = keys_all + (size_t)kb * a.S_cap / (K16 ? 2 : 1);     // split keys: the upper halves, 2 bytes each
        uint32_t* hist1 = hist1_all + kb * FBINS;
        CLK_BEGIN(t_unit);
#ifdef SPARQ_PHASE_CLOCKS
        long long ring_wait = 0;
#endif
        if (gtid < 32) wait_or_abort<100>(&sh.meta_full[m], ((uint32_t)(j / NMETA)) & 1u, sh, a.status);
        CLK_BEGIN(t_kf);
        group_wait<SG, 100>(gtid, &sh.keys_free[kb], (((uint32_t)(j / NKB)) & 1u) ^ 1u, sh, a.status);
        CLK_ADD(2, t_kf, gtid == 0);
        const int n = hm.n, r = a.r;
        if (hm.bh < 0 || sh.abort_flag) ++markers;           // forwarded to the post group below (group-uniform)
        if (hm.k_eff > 0) {
            uint32_t kmax = 0;
            float zm = -CUDART_INF_F, zs = 0.f;              // this thread's running max (in log2 units) and sum of 2^(x - zm)
            const float c1 = hm.inv_tau * LOG2E;
            __half2 mx[4];                                   // largest |K| among the valid streamed values
#pragma unroll
            for (int e = 0; e < 4; ++e) mx[e] = __float2half2_rn(0.f);
            const int n8 = (n + 7) & ~7;
            const int n_chunks = (n8 + CH - 1) / CH;
            for (int c = 0; c < n_chunks; ++c) {
                float acc[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[e] = 0.f;
                const int t0 = c * CH + gtid * 8;
                const int nvalid = min(8, n - t0);           // positions of this thread's vector inside the sequence
                __half2 mxc[4];                              // |K| maximum of this chunk, kept only if the vector is inside
#pragma unroll
                for (int e = 0; e < 4; ++e) mxc[e] = __float2half2_rn(0.f);
                for (int jb = 0; jb < r; jb += RB) {
#ifdef SPARQ_PHASE_CLOCKS
                    const long long t_f0 = clock64();
#endif
                    wait_or_abort<20>(&sh.full[s], parity, sh, a.status);
#ifdef SPARQ_PHASE_CLOCKS
                    ring_wait += clock64() - t_f0;
#endif
                    stage_fma<RB, CH / 8>(acc, mxc, reinterpret_cast<const uint4*>(ring + s * STAGE_BYTES) + gtid, hm.qh + jb, r - jb);
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh.empty[s]);   // this warp is done with slot s
                    if (++s == STAGES) { s = 0; parity ^= 1u; }
                }
                uint32_t kk[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) kk[e] = key32(acc[e]);
                if (nvalid > 0) {
#pragma unroll
                    for (int e = 0; e < 4; ++e) mx[e] = __hmax2(mx[e], mxc[e]);
                }
                if (nvalid > 0) {                            // softmax statistics of this thread's keys (a3), online
                    float cm = -CUDART_INF_F;
#pragma unroll
                    for (int e = 0; e < 8; ++e) if (e < nvalid) cm = fmaxf(cm, acc[e] * c1);
                    const float nm = fmaxf(zm, cm);
                    zs *= ex2(zm - nm);
#pragma unroll
                    for (int e = 0; e < 8; ++e) if (e < nvalid) zs += ex2(acc[e] * c1 - nm);
                    zm = nm;
                }
                if (nvalid >= 8) {
                    if constexpr (K16) {
                        uint16_t* keys_hi = reinterpret_cast<uint16_t*>(keys);
                        uint16_t* keys_lo = split_lo<NKB>(a, kb);
                        *reinterpret_cast<uint4*>(keys_hi + t0) =
                            make_uint4(__byte_perm(kk[0], kk[1], 0x7632), __byte_perm(kk[2], kk[3], 0x7632),
                                       __byte_perm(kk[4], kk[5], 0x7632), __byte_perm(kk[6], kk[7], 0x7632));
                        __stcg(reinterpret_cast<uint4*>(keys_lo + t0),
                               make_uint4(__byte_perm(kk[0], kk[1], 0x5410), __byte_perm(kk[2], kk[3], 0x5410),
                                          __byte_perm(kk[4], kk[5], 0x5410), __byte_perm(kk[6], kk[7], 0x5410)));
                    } else {
                        *reinterpret_cast<uint4*>(keys + t0) = make_uint4(kk[0], kk[1], kk[2], kk[3]);
                        *reinterpret_cast<uint4*>(keys + t0 + 4) = make_uint4(kk[4], kk[5], kk[6], kk[7]);
                    }
#pragma unroll
                    for (int e = 0; e < 8; ++e) { kmax = max(kmax, kk[e]); atomicAdd(&hist1[kk[e] >> FSH], 1u); }
                } else {
#pragma unroll
                    for (int e = 0; e < 8; ++e)
                        if (e < nvalid) {
                            if constexpr (K16) {
                                reinterpret_cast<uint16_t*>(keys)[t0 + e] = (uint16_t)(kk[e] >> 16);
                                __stcg(split_lo<NKB>(a, kb) + t0 + e, (uint16_t)(kk[e] & 0xffffu));
                            }
                            else keys[t0 + e] = kk[e];
                            kmax = max(kmax, kk[e]);
                            atomicAdd(&hist1[kk[e] >> FSH], 1u);
                        }
                }
            }
            uint32_t kabs_bits = __float_as_uint(mx_to_float(mx));
            group_max2_u32<SG>(kmax, kabs_bits, sh.sredu, gtid);
            // Z = sum over threads of zs * 2^(zm - max), max = the largest logit in log2 units
            const float Z = group_sum<SG>(zs > 0.f ? zs * ex2(zm - unkey32(kmax) * c1) : 0.f, sh.sred, gtid);
            if (gtid == 0) { sh.kmax[kb] = kmax; sh.kabs[kb] = __uint_as_float(kabs_bits); sh.zsum[kb] = Z; }
        }
        SG::sync();                                          // every key of the unit is written
        if (gtid == 0) mbar_arrive(&sh.keys_full[kb]);
        CLK_ADD(4, t_unit, gtid == 0);
#ifdef SPARQ_PHASE_CLOCKS
        if (gtid == 0) atomicAdd(&g_pipe_clocks[3], (unsigned long long)ring_wait);
#endif
    }
}

// ---------------------------------------------------------------------------------- post groups
template <class PG, int NKB, bool K16, class SH>
__device__ __forceinline__ void post_role(const Args& a, SH& sh, const uint32_t* keys_all, uint32_t* hist1_all,
                                          unsigned char* scratch, int32_t* i2, int p, const uint32_t opts) {
    const int gtid = threadIdx.x - LEAD - SNT - p * GNT;
    PostScratch sc;
    carve_post_scratch(sc, scratch, PG::NHW, a.S_cap / 32);
    sc.i2 = i2; sc.red = sh.red[p]; sc.redu = sh.redu[p]; sc.res = sh.res[p]; sc.band = sh.band[p];
    const int g_heads = a.Hq / a.Hkv;
    for (int j = p;; j += NPOST) {
        const int m = j % NMETA, kb = j % NKB;
        const HeadMeta& hm = sh.meta[m];
        CLK_BEGIN(t_w);
        group_wait<PG, 100>(gtid, &sh.keys_full[kb], ((uint32_t)(j / NKB)) & 1u, sh, a.status);
        CLK_ADD(1, t_w, gtid == 0);
        CLK_BEGIN(t_p);
        if (hm.bh < 0 || sh.abort_flag) {                    // end marker (or a wait gave up): this group is done
#ifdef SPARQ_PHASE_CLOCKS
            if (gtid == 0) { unsigned long long gt; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt)); atomicMax(&g_cta_end[blockIdx.x], gt); }
#endif
            break;
        }
        const int bh = hm.bh, b = bh / a.Hq, h = bh % a.Hq;
        const size_t kv_head = (size_t)b * a.Hkv + h / g_heads;
        sparq_half* out_row = a.out + (size_t)bh * D;
        if (!hm.valid) {                                     // defined result, no trap
            if (gtid == 0) { raise_status(a.status, SPARQ_DEV_BAD_SEQ_LEN); if (a.alpha) a.alpha[bh] = 0.f; }
            if (gtid < D) out_row[gtid] = 0;
            if (a.idx_k) for (int i = gtid; i < a.k; i += GNT) a.idx_k[(size_t)bh * a.k + i] = -1;
        } else if (hm.k_eff == 0) {                          // nothing to select: the mean value vector
            if (gtid < D) out_row[gtid] = a.vbar[kv_head * D + gtid];
            if (gtid == 0 && a.alpha) a.alpha[bh] = 0.f;
        } else {
            const sparq_half* Kt_head = a.Kt + kv_head * (size_t)D * a.S_max;
            auto keys = [&] {
                if constexpr (K16) {
                    return SplitKeys{reinterpret_cast<const uint16_t*>(keys_all) + (size_t)kb * a.S_cap,
                                     split_lo<NKB>(a, kb)};
                } else {
                    return keys_all + (size_t)kb * a.S_cap;
                }
            }();
            SelectResult sel;
            const bool windowed = (opts >> 16) != 0u && hm.n_sel != hm.n;   // (uniform) a local window is reserved inside the budget
            if (windowed && hm.k_sel == 0) {                 // the window takes the whole budget: nothing to rank
                for (int i = gtid; i < FBINS; i += GNT) hist1_all[kb * FBINS + i] = 0;   // left clear for the buffer's next unit
                sel = select_nothing<PG>(gtid, hm, keys, sh.kmax[kb], sc);
            } else {
                if (windowed) window_unhist<PG>(gtid, hm, keys, hist1_all + kb * FBINS);
                if (!select_prefilled<PG>(gtid, hm, keys, sh.kmax[kb], sh.kabs[kb], sh.zsum[kb], sc, hist1_all + kb * FBINS, a.r,
                                          a.S_max, Kt_head, sel)) {
#ifdef SPARQ_PHASE_CLOCKS
                    if (gtid == 0) atomicAdd(&g_pipe_clocks[7], 1ull);
#endif
                    sel = select_generic<PG>(gtid, hm, keys, sh.kmax[kb], sh.kabs[kb], sc, a.r, a.S_max, Kt_head);
                }
            }
            if (windowed) window_mark<PG>(gtid, hm, sc);
            finish<PG, 4>(gtid, hm, keys, sh.kmax[kb], sel, sc, a.k, a.K + kv_head * (size_t)a.S_max * D,
                          a.V + kv_head * (size_t)a.S_max * D, a.vbar + kv_head * D, out_row,
                          a.idx_k ? a.idx_k + (size_t)bh * a.k : nullptr, a.alpha ? a.alpha + bh : nullptr, true,
                          opt_realloc(opts));
        }
        PG::sync();                                          // the group is done with the keys, the metadata, i2
        CLK_ADD(0, t_p, gtid == 0);
        if (gtid == 0) { mbar_arrive(&sh.keys_free[kb]); mbar_arrive(&sh.meta_free[m]); }
    }
}

// OPT = false: the paper's algorithm as stated, the settings word known to be 0 at compile time (the
// instantiation the plain decode call runs); OPT = true: settings taken from `opts_arg`.
template <int NKB, bool OPT, bool K16, int RING>
__global__ void __launch_bounds__(NT, 1) sparq_decode_pipe_kernel(const Args a, const uint32_t opts_arg) {
    using R = Ring<RING>;
    const uint32_t opts = OPT ? opts_arg : 0u;
    extern __shared__ __align__(128) unsigned char dyn_smem[];
    unsigned char* ring = dyn_smem;
    uint32_t* keys_all = reinterpret_cast<uint32_t*>(dyn_smem + R::BYTES);     // NKB buffers of S_cap keys (split keys: their upper halves)
    uint32_t* hist1_all = keys_all + (size_t)NKB * a.S_cap / (K16 ? 2 : 1);   // per key buffer: histogram of the keys' top bits
    unsigned char* scratch0 = reinterpret_cast<unsigned char*>(hist1_all + NKB * FBINS);
    const size_t scratch_bytes = post_scratch_aligned(a.S_cap);
    // the post groups' index lists: SPARQ_K_MAX entries each in static shared memory, or, with split keys (whose
    // longest caches need the room), i2_pad(k) entries each behind the scratch areas
    int32_t* i2_dyn = reinterpret_cast<int32_t*>(scratch0 + NPOST * scratch_bytes);
    __shared__ PipeSharedT<K16> sh;

    if (threadIdx.x == 0) {
        for (int s = 0; s < R::STAGES; ++s) { mbar_init(&sh.full[s], 1); mbar_init(&sh.empty[s], SNT / 32); }
        for (int m = 0; m < NMETA; ++m) { mbar_init(&sh.meta_full[m], 1); mbar_init(&sh.meta_free[m], 1); }
        for (int b = 0; b < NKB; ++b) { mbar_init(&sh.keys_full[b], 1); mbar_init(&sh.keys_free[b], 1); }
        sh.abort_flag = 0;
        mbar_init_fence();
    }
    for (int i = threadIdx.x; i < NKB * FBINS; i += NT) hist1_all[i] = 0;
    __syncthreads();
#ifdef SPARQ_PHASE_CLOCKS
    if (threadIdx.x == 0) { unsigned long long gt; asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(gt)); g_cta_begin[blockIdx.x] = gt; g_cta_end[blockIdx.x] = 0; }
#endif
    const int warp = threadIdx.x >> 5;
    if (warp < NPROD) producer_role<RING>(a, sh, ring, warp);
    else if (warp == NPROD) a1_role<R::RB>(a, sh, opts);
    else if (warp < LEAD / 32 + SNT / 32) stream_role<NKB, K16, RING>(a, sh, ring, keys_all, hist1_all);
    else if (warp < LEAD / 32 + SNT / 32 + GNT / 32) post_role<PG0, NKB, K16>(a, sh, keys_all, hist1_all, scratch0, K16 ? i2_dyn : sh.i2[0], 0, opts);
    else post_role<PG1, NKB, K16>(a, sh, keys_all, hist1_all, scratch0 + scratch_bytes, K16 ? i2_dyn + i2_pad(a.k) : sh.i2[1], 1, opts);
}

size_t pipe_dynamic_smem(int S_cap, int NKB, bool k16, int ring, int k) {
    const size_t scratch = post_scratch_aligned(S_cap);
    const size_t ring_bytes = ring == 0 ? Ring<0>::BYTES : ring == 1 ? Ring<1>::BYTES : Ring<2>::BYTES;
    return ring_bytes + (size_t)NKB * S_cap * (k16 ? 2 : 4) + (size_t)NKB * FBINS * 4 + NPOST * scratch +
           (k16 ? (size_t)NPOST * i2_pad(k) * 4 : 0);
}
constexpr int NKB_SPLIT = 3;             // key buffers of the split-key form

}  // namespace

#ifdef SPARQ_PHASE_CLOCKS
extern "C" int sparq_debug_pipe_clocks(unsigned long long* out16, int reset) {
    cudaDeviceSynchronize();
    if (out16 && cudaMemcpyFromSymbol(out16, g_pipe_clocks, sizeof(unsigned long long) * 16) != cudaSuccess) return 1;
    if (reset) { unsigned long long z[16] = {0}; if (cudaMemcpyToSymbol(g_pipe_clocks, z, sizeof(z)) != cudaSuccess) return 1; }
    return 0;
}
extern "C" int sparq_debug_cta_times(unsigned long long* begin256, unsigned long long* end256) {
    cudaDeviceSynchronize();
    if (cudaMemcpyFromSymbol(begin256, g_cta_begin, sizeof(unsigned long long) * 256) != cudaSuccess) return 1;
    if (cudaMemcpyFromSymbol(end256, g_cta_end, sizeof(unsigned long long) * 256) != cudaSuccess) return 1;
    return 0;
}
extern "C" int sparq_debug_post_clocks(unsigned long long* out16, int reset) {
    cudaDeviceSynchronize();
    if (out16 && cudaMemcpyFromSymbol(out16, g_post_clocks, sizeof(unsigned long long) * 16) != cudaSuccess) return 1;
    if (reset) { unsigned long long z[16] = {0}; if (cudaMemcpyToSymbol(g_post_clocks, z, sizeof(z)) != cudaSuccess) return 1; }
    return 0;
}
#endif

// S_max rounded up so that bitmap words and 16-byte key vectors stay whole
static int pipe_s_cap(int S_max) { return (S_max + 127) & ~127; }

// (the plan selection asks without knowing k: the largest budget's index lists are assumed)
static bool pipe_fits_nkb(int S_max, int smem_optin, int nkb, bool k16, int ring, int k = SPARQ_K_MAX) {
    return pipe_dynamic_smem(pipe_s_cap(S_max), nkb, k16, ring, k) + (k16 ? sizeof(PipeSharedT<true>) : sizeof(PipeSharedT<false>)) + 1024 <= (size_t)smem_optin;
}
bool pipe_fits(int S_max, int smem_optin) { return pipe_fits_nkb(S_max, smem_optin, 3, false, 0); }
bool pipe_split_fits(int S_max, int smem_optin) { return pipe_fits_nkb(S_max, smem_optin, NKB_SPLIT, true, 1); }
bool pipe_split_thin_ring(int S_max, int smem_optin) { return !pipe_fits_nkb(S_max, smem_optin, NKB_SPLIT, true, 0); }
// Workspace of the split-key form: the unit counter, then the keys' lower halves.
size_t pipe_split_workspace(int S_max, int n_sm) { return SPLIT_LO_OFFSET + (size_t)n_sm * NKB_SPLIT * pipe_s_cap(S_max) * 2; }

// split_keys: unit_counter heads a workspace of pipe_split_workspace() bytes; else 32-bit keys in shared memory.
cudaError_t launch_sparq_decode_pipe(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                     const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                     int r, int k, uint32_t opts, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                     int32_t* status, int n_sm, unsigned int* unit_counter, bool split_keys,
                                     cudaStream_t stream) {
    Args a;
    a.q = q; a.K = K; a.Kt = Kt; a.V = V; a.vbar = vbar; a.seq_lens = seq_lens;
    a.n_units = B * Hq; a.Hq = Hq; a.Hkv = Hkv; a.S_max = S_max; a.S_cap = pipe_s_cap(S_max); a.r = r; a.k = k;
    a.out = out; a.idx_r = idx_r; a.idx_k = idx_k; a.alpha = alpha; a.status = status; a.unit_counter = unit_counter;
    const int smem_optin = device_info().smem_optin;
    const bool k16 = split_keys && unit_counter;
    const bool four = !k16 && pipe_fits_nkb(S_max, smem_optin, 4, false, 0);
    // split keys: the 96 KB ring where it fits whatever the budget; else five 16 KB stages if this call's k leaves room, else four
    const int ring = !k16 ? 0 : pipe_fits_nkb(S_max, smem_optin, NKB_SPLIT, true, 0) ? 0
                                : pipe_fits_nkb(S_max, smem_optin, NKB_SPLIT, true, 2, k) ? 2 : 1;
    const size_t dyn = pipe_dynamic_smem(a.S_cap, k16 ? NKB_SPLIT : (four ? 4 : 3), k16, ring, k);
    auto kernel = k16 ? (ring == 0 ? (opts ? sparq_decode_pipe_kernel<NKB_SPLIT, true, true, 0> : sparq_decode_pipe_kernel<NKB_SPLIT, false, true, 0>)
                       : ring == 1 ? (opts ? sparq_decode_pipe_kernel<NKB_SPLIT, true, true, 1> : sparq_decode_pipe_kernel<NKB_SPLIT, false, true, 1>)
                                   : (opts ? sparq_decode_pipe_kernel<NKB_SPLIT, true, true, 2> : sparq_decode_pipe_kernel<NKB_SPLIT, false, true, 2>))
                : opts ? (four ? sparq_decode_pipe_kernel<4, true, false, 0> : sparq_decode_pipe_kernel<3, true, false, 0>)
                       : (four ? sparq_decode_pipe_kernel<4, false, false, 0> : sparq_decode_pipe_kernel<3, false, false, 0>);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dyn);
    if (e != cudaSuccess) return e;
    const int grid = a.n_units < n_sm ? a.n_units : n_sm;
    if (unit_counter) {
        e = cudaMemsetAsync(unit_counter, 0, sizeof(unsigned int), stream);
        if (e != cudaSuccess) return e;
    }
    kernel<<<grid, NT, dyn, stream>>>(a, opts);
    return cudaGetLastError();
}

}  // namespace sparq
