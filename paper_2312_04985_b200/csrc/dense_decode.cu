// dense_decode: dense single-token decode attention, Eq. (2), the comparison kernel for the
// speed-up figure.  One CTA per (split, KV head, batch): a CTA covers one slice of the sequence of one KV head
// for all (up to 8 at a time) query heads of its group, so K and V are read once per KV head.
// One or two heads at a time: half-warp per cache row, 128-bit loads, online softmax in fp32, on the
// CUDA cores.  Four or eight at a time: the pass is a small dense contraction and runs on the tensor
// cores (further down).  With more than one split the per-split softmax states go through a scratch
// buffer and a small merge kernel.
#include <mutex>

#include "common.cuh"
#include "kernels.h"

namespace sparq {
namespace {

// Scratch of dense_decode_static: lives in the library's device image, so every GPU that loads the
// library carries these 8 MiB until the process exits, and every call on a device shares them.
constexpr size_t kStaticScratchBytes = SPARQ_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_dense_scratch[kStaticScratchBytes];
constexpr int kMaxDevices = 64;
float* g_dense_scratch_ptr[kMaxDevices] = {};   // device address of the array, per device ordinal
std::mutex g_dense_scratch_mutex;

constexpr int NT = 256;             // threads per CTA
constexpr int NHW = NT / 16;        // half-warps per CTA (one K/V row each)

// One CTA per (split, KV head, batch).  A CTA covers positions [split*chunk, (split+1)*chunk) of one KV head
// for all G query heads of the group; half-warp per cache row, online softmax in fp32.
template <int G>
__global__ void __launch_bounds__(NT)
dense_decode_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                    const sparq_half* __restrict__ V, const int32_t* __restrict__ seq_lens,
                    int Hq, int Hkv, int S_max, int g_total, int g_base, int splits,
                    sparq_half* __restrict__ out, float* __restrict__ ws, int32_t* status) {
    __shared__ float merge[NHW * (D + 2)];
    const int tid = threadIdx.x, hw = tid >> 4, l16 = tid & 15;
    // one-dimensional grid: split fastest, then KV head, then batch (no 65535 limit on the batch)
    const int split = (int)(blockIdx.x % (unsigned)splits);
    const int hkv = (int)((blockIdx.x / (unsigned)splits) % (unsigned)Hkv), b = (int)(blockIdx.x / ((unsigned)splits * (unsigned)Hkv));
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

    const float qscale = rsqrtf((float)D) * LOG2E;
    // this lane's 8 query components per head, as stored (fp16): q . k is a chain of mixed-precision
    // FMAs on exact fp16 x fp16 products, scaled once at the end
    uint32_t qw[G][4];
    float acc[G][8], m[G], l[G];
#pragma unroll
    for (int gi = 0; gi < G; ++gi) {
        m[gi] = -CUDART_INF_F; l[gi] = 0.f;
        const uint4 q8 = *reinterpret_cast<const uint4*>(q + ((size_t)b * Hq + h0 + gi) * D + l16 * 8);
        qw[gi][0] = q8.x; qw[gi][1] = q8.y; qw[gi][2] = q8.z; qw[gi][3] = q8.w;
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[gi][e] = 0.f;
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
        for (int gi = 0; gi < G; ++gi) {
            // the RG rows' logits for this head, then ONE rescale of the running state per batch of rows
            float z[RG], bmax = -CUDART_INF_F;
#pragma unroll
            for (int u = 0; u < RG; ++u) {
                const uint32_t kw[4] = {kv[u].x, kv[u].y, kv[u].z, kv[u].w};
                float za = 0.f, zb = 0.f;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(za) : "h"((uint16_t)(kw[e] & 0xffffu)), "h"((uint16_t)(qw[gi][e] & 0xffffu)));
                    asm("fma.rn.f32.f16 %0, %1, %2, %0;" : "+f"(zb) : "h"((uint16_t)(kw[e] >> 16)), "h"((uint16_t)(qw[gi][e] >> 16)));
                }
                float zz = (za + zb) * qscale;
#pragma unroll
                for (int o = 8; o > 0; o >>= 1) zz += __shfl_xor_sync(FULL, zz, o);
                z[u] = (t0 + u * NHW < t_end) ? zz : -CUDART_INF_F;        // uniform within the half-warp
                bmax = fmaxf(bmax, z[u]);
            }
            const float mn = fmaxf(m[gi], bmax);
            if (mn > -CUDART_INF_F) {
                const float sc = exp2f(m[gi] - mn);
                float lsum = l[gi] * sc;
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[gi][e] *= sc;
#pragma unroll
                for (int u = 0; u < RG; ++u) {
                    const float p = exp2f(z[u] - mn);
                    lsum += p;
                    const __half2* vh = reinterpret_cast<const __half2*>(&vv[u]);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 w = __half22float2(vh[e]);
                        acc[gi][2 * e] = fmaf(p, w.x, acc[gi][2 * e]);
                        acc[gi][2 * e + 1] = fmaf(p, w.y, acc[gi][2 * e + 1]);
                    }
                }
                l[gi] = lsum;
                m[gi] = mn;
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

// ---------------------------------------------------------------------------------- grouped heads on the tensor cores
// With four or eight query heads per KV head the pass over K and V is a small dense contraction
// (heads x d_h times d_h x positions, then heads x positions times positions x d_h), and on the CUDA cores
// it is bound by instruction issue at half the memory bandwidth.  Here a warp takes 16 positions at a
// time: their K and V rows go through shared memory into mma.sync m16n8k16 fragments (fp16 operands,
// fp32 accumulators), the query heads are rows 0..GH-1 of the 16-row A operand (the others zero), and
// the softmax runs online on the accumulator fragments.  The weights are rounded to fp16 for the
// second product, as every tensor-core attention kernel does.
constexpr int TCW = 4;                   // warps per CTA, each with its own tiles and softmax state
constexpr int TCT = 16;                  // positions per warp tile
constexpr int TROW = D * 2 + 16;         // bytes per staged row: 16 bytes of padding keep ldmatrix free of bank conflicts

// 16 bytes global -> shared without passing through registers (both addresses 16-byte aligned)
__device__ __forceinline__ void cp_async16(unsigned char* dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const unsigned char* row) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(row)));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t (&r)[4], const unsigned char* row) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(row)));
}
// c += a (16x16, rows 8..15 zero: a1 = a3 = 0) * b (16x8)
__device__ __forceinline__ void mma_16816(float& c0, float& c1, float& c2, float& c3, uint32_t a0, uint32_t a2, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c0), "+f"(c1), "+f"(c2), "+f"(c3) : "r"(a0), "r"(0u), "r"(a2), "r"(0u), "r"(b0), "r"(b1));
}

template <int GH>
__global__ void __launch_bounds__(TCW * 32)
dense_decode_tc_kernel(const sparq_half* __restrict__ q, const sparq_half* __restrict__ K,
                       const sparq_half* __restrict__ V, const int32_t* __restrict__ seq_lens,
                       int Hq, int Hkv, int S_max, int g_total, int g_base, int splits,
                       sparq_half* __restrict__ out, float* __restrict__ ws, int32_t* status) {
    static_assert(GH == 4 || GH == 8, "rows 0..GH-1 of the A operand");
    extern __shared__ __align__(128) unsigned char tc_smem[];
    // per warp: two buffers of a K tile and a V tile each (the next tile's rows are on their way while this one is used)
    unsigned char (*tiles)[2][2][TCT * TROW] = reinterpret_cast<unsigned char (*)[2][2][TCT * TROW]>(tc_smem);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, c = lane & 3;                   // fragment row (query head) and column pair of this lane
    const int split = (int)(blockIdx.x % (unsigned)splits);
    const int hkv = (int)((blockIdx.x / (unsigned)splits) % (unsigned)Hkv), b = (int)(blockIdx.x / ((unsigned)splits * (unsigned)Hkv));
    const int n = seq_lens[b];
    const int h0 = hkv * g_total + g_base;                    // first query head served here
    if (n < 1 || n > S_max) {
        if (split == 0) {
            if (tid == 0) raise_status(status, SPARQ_DEV_BAD_SEQ_LEN);
            for (int i = tid; i < GH * D; i += TCW * 32) out[((size_t)b * Hq + h0 + i / D) * D + (i % D)] = 0;
        }
        return;                                               // merge kernel skips this sequence too
    }
    int chunk = (n + splits - 1) / splits;
    chunk = (chunk + 15) & ~15;
    const int t_begin = split * chunk, t_end = min(n, t_begin + chunk);
    const float qscale = rsqrtf((float)D) * LOG2E;

    // A fragments of the queries: for k-slab ks, a0 = (row g, columns 16 ks + 2c, +1), a2 = (row g, 16 ks + 8 + 2c, +1)
    uint32_t qa0[8], qa2[8];
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
        qa0[ks] = 0; qa2[ks] = 0;
        if (g < GH) {
            const sparq_half* qrow = q + ((size_t)b * Hq + h0 + g) * D;
            qa0[ks] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 2 * c);
            qa2[ks] = *reinterpret_cast<const uint32_t*>(qrow + ks * 16 + 8 + 2 * c);
        }
    }
    // accumulators of the output: n-tile nt holds (row g, dims 8 nt + 2c, +1); rows 8..15 stay zero
    float o0[16], o1[16], z2 = 0.f, z3 = 0.f;
#pragma unroll
    for (int nt = 0; nt < 16; ++nt) { o0[nt] = 0.f; o1[nt] = 0.f; }
    float m = -CUDART_INF_F, l = 0.f;                         // this row's running maximum (log2 units) and sum

    const size_t kv_head = (size_t)b * Hkv + hkv;
    const uint4* Kh = reinterpret_cast<const uint4*>(K + kv_head * (size_t)S_max * D);
    const uint4* Vh = reinterpret_cast<const uint4*>(V + kv_head * (size_t)S_max * D);
    // stage 16 rows of K and of V: 256 16-byte pieces each, 8 per lane; rows past the end repeat the last one
    auto stage = [&](int buf, int tb) {
#pragma unroll
        for (int jj = 0; jj < 8; ++jj) {
            const int id = lane + 32 * jj, row = id >> 4, col = id & 15;
            const int t = min(tb + row, t_end - 1);
            cp_async16(tiles[warp][buf][0] + row * TROW + col * 16, Kh + (size_t)t * (D / 8) + col);
            cp_async16(tiles[warp][buf][1] + row * TROW + col * 16, Vh + (size_t)t * (D / 8) + col);
        }
        cp_async_commit();
    };
    int buf = 0;
    if (t_begin + warp * TCT < t_end) stage(0, t_begin + warp * TCT);
    for (int tb = t_begin + warp * TCT; tb < t_end; tb += TCW * TCT, buf ^= 1) {
        const unsigned char* kt = tiles[warp][buf][0];
        const unsigned char* vt = tiles[warp][buf][1];
        if (tb + TCW * TCT < t_end) { stage(buf ^ 1, tb + TCW * TCT); cp_async_wait<1>(); }   // all but the newest group have landed
        else cp_async_wait<0>();
        __syncwarp();

        // scores of the 16 positions: two n-tiles of 8
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
        {
            const int mat = lane >> 3, row = lane & 7;       // this lane's row address for ldmatrix
            const unsigned char* base = kt + ((mat >> 1) * 8 + row) * TROW + (mat & 1) * 16;
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                uint32_t r[4];
                ldsm_x4(r, base + ks * 32);
                mma_16816(s0[0], s0[1], s0[2], s0[3], qa0[ks], qa2[ks], r[0], r[1]);
                mma_16816(s1[0], s1[1], s1[2], s1[3], qa0[ks], qa2[ks], r[2], r[3]);
            }
        }
        // online softmax on row g: this lane holds positions 2c, 2c+1, 8+2c, 9+2c of the tile
        float x[4] = {s0[0] * qscale, s0[1] * qscale, s1[0] * qscale, s1[1] * qscale};
        const int p0 = tb + 2 * c;
        if (p0 >= t_end) x[0] = -CUDART_INF_F;
        if (p0 + 1 >= t_end) x[1] = -CUDART_INF_F;
        if (p0 + 8 >= t_end) x[2] = -CUDART_INF_F;
        if (p0 + 9 >= t_end) x[3] = -CUDART_INF_F;
        float tm = fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3]));
        tm = fmaxf(tm, __shfl_xor_sync(FULL, tm, 1));
        tm = fmaxf(tm, __shfl_xor_sync(FULL, tm, 2));
        const float mn = fmaxf(m, tm);                        // finite: the tile's first position is valid
        const float sc = exp2f(m - mn);
        float p[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) p[i] = exp2f(x[i] - mn);
        // the weights as the kernel uses them: rounded to fp16; their sum is taken of the rounded values
        const __half2 pa = __floats2half2_rn(p[0], p[1]), pb = __floats2half2_rn(p[2], p[3]);
        const float2 fa = __half22float2(pa), fb = __half22float2(pb);
        float ps = (fa.x + fa.y) + (fb.x + fb.y);
        ps += __shfl_xor_sync(FULL, ps, 1);
        ps += __shfl_xor_sync(FULL, ps, 2);
        l = l * sc + ps;
        m = mn;
        if (__any_sync(FULL, sc != 1.0f)) {
#pragma unroll
            for (int nt = 0; nt < 16; ++nt) { o0[nt] *= sc; o1[nt] *= sc; }
        }
        const uint32_t a0 = *reinterpret_cast<const uint32_t*>(&pa), a2 = *reinterpret_cast<const uint32_t*>(&pb);
        {
            const int mat = lane >> 3, row = lane & 7;
            const unsigned char* base = vt + ((mat & 1) * 8 + row) * TROW + (mat >> 1) * 16;
#pragma unroll
            for (int j = 0; j < 8; ++j) {                    // two n-tiles (16 dims) per ldmatrix
                uint32_t r[4];
                ldsm_x4_trans(r, base + j * 32);
                mma_16816(o0[2 * j], o1[2 * j], z2, z3, a0, a2, r[0], r[1]);
                mma_16816(o0[2 * j + 1], o1[2 * j + 1], z2, z3, a0, a2, r[2], r[3]);
            }
        }
        __syncwarp();                                         // this buffer is refilled by the next iteration's copies
    }
    // merge the warps' states, one (head, dim) per output element
    __syncthreads();                                          // every warp is done with its tiles
    float* mg = reinterpret_cast<float*>(tc_smem);            // [TCW][GH][D + 2]
    if (g < GH) {
        float* row = mg + ((size_t)warp * GH + g) * (D + 2);
#pragma unroll
        for (int nt = 0; nt < 16; ++nt) { row[nt * 8 + 2 * c] = o0[nt]; row[nt * 8 + 2 * c + 1] = o1[nt]; }
        if (c == 0) { row[D] = m; row[D + 1] = l; }
    }
    __syncthreads();
    for (int i = tid; i < GH * D; i += TCW * 32) {
        const int gi = i / D, dim = i % D;
        float M = -CUDART_INF_F;
#pragma unroll
        for (int w = 0; w < TCW; ++w) M = fmaxf(M, mg[((size_t)w * GH + gi) * (D + 2) + D]);
        float L = 0.f, y = 0.f;
        if (M > -CUDART_INF_F) {
#pragma unroll
            for (int w = 0; w < TCW; ++w) {
                const float* row = mg + ((size_t)w * GH + gi) * (D + 2);
                const float scw = exp2f(row[D] - M);          // (a warp without a tile carries m = -inf, l = 0)
                L = fmaf(row[D + 1], scw, L);
                y = fmaf(row[dim], scw, y);
            }
        }
        const size_t bhq = (size_t)b * Hq + h0 + gi;
        if (splits == 1) {
            out[bhq * D + dim] = __half_as_ushort(__float2half_rn(y / L));
        } else {
            float* pw = ws + (bhq * splits + split) * (D + 2);
            pw[dim] = y;
            if (dim == 0) { pw[D] = M; pw[D + 1] = L; }
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

}  // namespace

int dense_splits(int B, int Hkv, int S_max) {
    long ctas = (long)B * Hkv;
    long want = (4L * 148 + ctas - 1) / ctas;                 // aim for >= 4 CTAs per SM
    long cap = (S_max + 255) / 256;                           // at least 256 positions per split
    long s = want < cap ? want : cap;
    return (int)(s < 1 ? 1 : s);
}

size_t dense_scratch_bytes(int B, int Hq, int Hkv, int S_max) {
    int splits = dense_splits(B, Hkv, S_max);
    return splits == 1 ? 0 : (size_t)B * Hq * splits * (D + 2) * sizeof(float);
}

// Device address of the static scratch on the current device.  In host code the array's name is only
// a handle of the symbol, not an address a kernel could use: the address comes from the runtime, once
// per device, with that device current.
cudaError_t dense_static_scratch(float** ptr, size_t* bytes) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_dense_scratch_mutex);
    if (!g_dense_scratch_ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_dense_scratch);
        if (e != cudaSuccess) return e;
        g_dense_scratch_ptr[dev] = static_cast<float*>(p);
    }
    *ptr = g_dense_scratch_ptr[dev];
    *bytes = kStaticScratchBytes;
    return cudaSuccess;
}

cudaError_t launch_dense_decode(const sparq_half* q, const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                                int B, int Hq, int Hkv, int S_max, sparq_half* out, float* ws, int32_t* status,
                                cudaStream_t st) {
    const int splits = dense_splits(B, Hkv, S_max);
    const int g = Hq / Hkv;
    const unsigned grid = (unsigned)splits * (unsigned)Hkv * (unsigned)B;
    // the group's query heads are served G at a time by one pass over K and V
    for (int g_base = 0; g_base < g;) {
        int left = g - g_base;
        if (left >= 4) {
            constexpr size_t tc_dyn = (size_t)TCW * 2 * 2 * TCT * TROW;
            auto kernel = left >= 8 ? dense_decode_tc_kernel<8> : dense_decode_tc_kernel<4>;
            cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc_dyn);
            if (e != cudaSuccess) return e;
            kernel<<<grid, TCW * 32, tc_dyn, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status);
            g_base += left >= 8 ? 8 : 4;
        }
        else if (left >= 2) { dense_decode_kernel<2><<<grid, NT, 0, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status); g_base += 2; }
        else { dense_decode_kernel<1><<<grid, NT, 0, st>>>(q, K, V, seq_lens, Hq, Hkv, S_max, g, g_base, splits, out, ws, status); g_base += 1; }
    }
    if (splits > 1) dense_merge_kernel<<<B * Hq, D, 0, st>>>(ws, seq_lens, Hq, S_max, splits, out);
    return cudaGetLastError();
}

}  // namespace sparq
