// The C ABI of include/sparq.h: argument validation and kernel launches.  Nothing here
// allocates device memory or synchronises, except sparq_step_host which waits for its stream.
#include <stdlib.h>
#include <string.h>

#include <atomic>

#include "kernels.h"

namespace sparq {

// The current device's figures the plan selection needs, queried once per device: the attribute
// queries cost more than the rest of a call's host work (batch-1 decoding is host-bound without
// CUDA graphs).  Zeros when there is no device (the host-side checks still work).
DeviceInfo device_info() {
    constexpr int kMax = 64;
    static DeviceInfo table[kMax];
    static std::atomic<int> ready[kMax];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return DeviceInfo{0, 0, 0};
    const bool cached = dev >= 0 && dev < kMax;
    if (cached && ready[dev].load(std::memory_order_acquire)) return table[dev];
    DeviceInfo d{0, 0, 0};
    if (cudaDeviceGetAttribute(&d.sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&d.smem_per_sm, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) != cudaSuccess)
        return DeviceInfo{0, 0, 0};
    if (cached) { table[dev] = d; ready[dev].store(1, std::memory_order_release); }   // (racing threads store the same values)
    return d;
}

}  // namespace sparq

namespace {

using namespace sparq;

int device_smem_optin() { return device_info().smem_optin; }

bool bad_common(int B, int Hq, int Hkv, int d, int S_max) {
    return B < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || d != SPARQ_HEAD_DIM || S_max < 8 || S_max % 8 != 0;
}

int device_sm_count() { return device_info().sm_count; }

// SPARQ_DECODE_PLAN=simple|pipe|pipe16|split|wide forces one of the sparq_decode plans (tests and tuning).
// Unset or anything else: the wide kernel (one CTA of 512 threads, or two of 256, per SM; a unit's
// keys in shared memory) for up to two units per SM and for caches too long for the persistent
// kernel; the persistent pipelined kernel wherever else one unit's keys fit its shared memory, and in
// its split-key form (pipe16) for four or more units per SM on caches up to about 17,800 positions;
// beyond the wide kernel's reach (about 44,000 positions) the split plan if the caller passed its
// workspace; else one CTA per unit.
int forced_plan() {
    const char* e = getenv("SPARQ_DECODE_PLAN");
    if (!e) return 0;
    if (!strcmp(e, "simple")) return 1;
    if (!strcmp(e, "pipe")) return 2;
    if (!strcmp(e, "split")) return 3;
    if (!strcmp(e, "wide")) return 4;
    if (!strcmp(e, "pipe16")) return 5;
    return 0;
}

constexpr size_t SPARQ_PIPE_WORKSPACE_BYTES = 64;
static size_t pipe_split_bytes(int S_max, int n_sm) { return pipe_split_workspace(S_max, n_sm); }

int rc(cudaError_t e) { return e == cudaSuccess ? SPARQ_OK : SPARQ_ERR_CUDA; }

// true when any of the given pointers (NULL allowed: optional arguments) is not 16-byte aligned
template <class... P>
bool misaligned(P... ptrs) {
    return (((reinterpret_cast<uintptr_t>((const void*)ptrs) & 15u) != 0) || ...);
}

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
        case SPARQ_ERR_STATIC_SCRATCH: return "SPARQ_ERR_STATIC_SCRATCH";
        case SPARQ_ERR_ALIGNMENT: return "SPARQ_ERR_ALIGNMENT";
        case SPARQ_ERR_BAD_OPTION: return "SPARQ_ERR_BAD_OPTION";
        case SPARQ_DEV_BAD_SEQ_LEN: return "SPARQ_DEV_BAD_SEQ_LEN";
        case SPARQ_DEV_CACHE_FULL: return "SPARQ_DEV_CACHE_FULL";
        case SPARQ_DEV_TIMEOUT: return "SPARQ_DEV_TIMEOUT";
        default: return "SPARQ_UNKNOWN_STATUS";
    }
}

// largest S_max of the one-CTA-per-unit kernel with the bulk-copy ring (a forced plan "simple")
static int simple_max_seq_len() {
    long avail = (long)device_smem_optin() - (long)decode_static_smem() - (long)decode_dynamic_smem(0) - 1024;
    if (avail <= 0) return 0;
    long s = (avail / 4) & ~7L;
    long cap = decode_max_positions();
    return (int)(s < cap ? s : cap);
}

// largest S_max of the wide kernel: its shared memory grows with S_max, so bisect on multiples of 8
static int wide_max_seq_len() {
    const int optin = device_smem_optin();
    int lo = 0, hi = SPARQ_S_MAX_WORKSPACE / 8;              // in units of 8 positions; lo fits (or is 0), hi may not
    if (wide_fits(hi * 8, optin)) return hi * 8;
    while (hi - lo > 1) {
        const int mid = (lo + hi) / 2;
        if (wide_fits(mid * 8, optin)) lo = mid; else hi = mid;
    }
    return lo * 8;
}

int sparq_max_seq_len(void) {
    const int a = simple_max_seq_len(), b = wide_max_seq_len();
    return a > b ? a : b;
}

int sparq_cache_build(const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                      sparq_half* Kt, float* vsum, sparq_half* vbar,
                      int B, int Hkv, int d, int S_max, int32_t* status, void* stream) {
    if (!K || !V || !seq_lens || !Kt || !vsum || !vbar) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hkv, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    if (misaligned(K, V, Kt, vsum, vbar)) return SPARQ_ERR_ALIGNMENT;
    return rc(launch_cache_build(K, V, seq_lens, Kt, vsum, vbar, B, Hkv, S_max, status, (cudaStream_t)stream));
}

int sparq_cache_append(const sparq_half* k_new, const sparq_half* v_new,
                       sparq_half* K, sparq_half* Kt, sparq_half* V, float* vsum, sparq_half* vbar,
                       int32_t* seq_lens, int B, int Hkv, int d, int S_max, int32_t* status, void* stream) {
    if (!k_new || !v_new || !K || !Kt || !V || !vsum || !vbar || !seq_lens) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hkv, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    if (misaligned(k_new, v_new, K, Kt, V, vsum, vbar)) return SPARQ_ERR_ALIGNMENT;
    return rc(launch_cache_append(k_new, v_new, K, Kt, V, vsum, vbar, seq_lens, B, Hkv, S_max, status,
                                  (cudaStream_t)stream));
}

// The split plan against the persistent kernel where the wide kernel does not apply (a forced plan,
// or a cache beyond the wide kernel's shared memory): wherever the persistent kernel does not fit,
// and for a few units (fewer than SMs) with a lot to stream each, which it slices over all SMs.
static bool split_preferred(int units, int S_max, int r, int n_sm, bool pipe_ok) {
    if (!pipe_ok) return true;
    return units < n_sm && (size_t)2 * S_max * r > ((size_t)512 << 10);
}

// The wide kernel against the others, where its keys fit in shared memory.  Up to one unit per SM it
// is the fastest at any length (32 units of 4096 positions: 19.8 us, persistent kernel 22.7, sliced
// plan 27.6; 128 units of 16384 at r = 16: 28.6 against the sliced plan's 58.2).  Beyond that the
// persistent kernel wins wherever it fits (2048 units of 4096: 128 against 161 us), and the wide
// kernel wins on the longer caches (1024 units of 16384, r = 16, two CTAs per SM: 141 against the
// split plan's 147 us; 256 units: 43 against 71; 512 units of up to 32800 positions at r = 64, one
// CTA per SM: 260 against 289).
// Up to two units per SM all of them are resident at once as two CTAs per SM, and the wide kernel still
// wins (4096 positions, r = 32: 160 units 25.3 against the persistent kernel's 28.6 us, 256 units 29.1
// against 32.2; 320 units 40.2 against 37.9, 1024 units 86.9 against 73.2).
static bool wide_preferred(int units, int n_sm, bool pipe_ok) { return units <= 2 * n_sm || !pipe_ok; }

// The persistent kernel's split-key form against the wide kernel, for caches too long for the persistent
// kernel's 32-bit keys: with four or more units per SM its hand-built overlap of one unit's stream with
// the others' select and gather beats the wide kernel's two CTAs per SM (1024 units of 16384 positions
// at r = 16: 116 against 142 us; 2048 units of 8192 at r = 16: 125 against 156; 1024 units of 8192 at
// r = 32: 117 against 132), with fewer it loses (256 units of 16384: 48 against 41).  Beyond about 12,700
// positions only a ring of four or five 16 KB stages fits beside the keys, which holds the stream back when the rows are many
// (1024 units of 16384 at r = 32: 201 against 195; 512 units at r = 64: 223 against 175): there only up to r = 16.
static bool pipe16_preferred(int units, int S_max, int r, int n_sm) {
    const int smem = device_info().smem_optin;
    if (units < 4 * n_sm || pipe_fits(S_max, smem) || !pipe_split_fits(S_max, smem)) return false;
    return !pipe_split_thin_ring(S_max, smem) || r <= 16;
}

// Two 256-thread CTAs per SM instead of one of 512 threads: with more units than SMs, where both fit.
// SPARQ_WIDE_PAIRS=0|1 overrides (tuning).
static bool wide_pairs(int units, int S_max, int n_sm) {
    const int per_sm = device_info().smem_per_sm;
    if (per_sm <= 0) return false;
    bool pairs = units > n_sm && wide_pair_fits(S_max, per_sm);
    if (const char* e = getenv("SPARQ_WIDE_PAIRS")) pairs = (e[0] == '1') && wide_pair_fits(S_max, per_sm);
    return pairs;
}

size_t sparq_workspace_bytes(int B, int Hq, int Hkv, int d, int S_max, int r, int k) {
    (void)k;
    if (bad_common(B, Hq, Hkv, d, S_max)) return 0;
    const int n_sm = device_sm_count();
    const int splits = S_max <= SPARQ_S_MAX_WORKSPACE ? split_count(B * Hq, S_max, n_sm) : 0;
    const bool pipe_ok = pipe_fits(S_max, device_smem_optin());
    const int plan = forced_plan();                          // a plan forced through the environment gets what it needs
    if (plan == 5) return pipe_split_fits(S_max, device_smem_optin()) ? pipe_split_bytes(S_max, n_sm) : 0;
    if (plan == 0 && pipe16_preferred(B * Hq, S_max, r, n_sm)) return pipe_split_bytes(S_max, n_sm);
    if (plan == 4 || (plan == 0 && wide_fits(S_max, device_smem_optin()) && wide_preferred(B * Hq, n_sm, pipe_ok)))
        return 0;
    if (splits && (plan == 3 || (plan == 0 && split_preferred(B * Hq, S_max, r, n_sm, pipe_ok))))
        return split_scratch_bytes(B * Hq, S_max, splits);
    if (pipe_ok) return B * Hq > n_sm ? SPARQ_PIPE_WORKSPACE_BYTES : 0;   // the persistent kernel's unit counter
    return 0;
}

// sparq_decode and sparq_decode_opt: one plan selection, the settings travel as one packed word
static int decode_with(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                       const sparq_half* vbar, const int32_t* seq_lens,
                       int B, int Hq, int Hkv, int d, int S_max, int r, int k, uint32_t opts,
                       sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                       void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    if (!q || !K || !Kt || !V || !vbar || !seq_lens || !out) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hq, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    if (r < 1 || r > d || k < 0 || k > SPARQ_K_MAX) return SPARQ_ERR_BAD_RK;
    if (misaligned(q, K, Kt, V, vbar, out, workspace)) return SPARQ_ERR_ALIGNMENT;
    const int plan = forced_plan();
    const int n_sm = device_sm_count();
    const int splits = S_max <= SPARQ_S_MAX_WORKSPACE ? split_count(B * Hq, S_max, n_sm) : 0;
    const bool ws_ok = splits && workspace && workspace_bytes >= split_scratch_bytes(B * Hq, S_max, splits);
    const bool too_long = S_max > sparq_max_seq_len();       // beyond shared memory only the split plan's scratch buffer helps
    if (too_long && !ws_ok)
        return S_max <= SPARQ_S_MAX_WORKSPACE && (plan == 0 || plan == 3) ? SPARQ_ERR_WORKSPACE : SPARQ_ERR_TOO_LONG;
    if (plan == 3 && !ws_ok) return SPARQ_ERR_WORKSPACE;
    // one 512-thread CTA per unit with the keys in shared memory: the choice for a handful of units whatever
    // their length, and beside the split plan for caches the persistent kernel cannot hold
    // the persistent kernel's split-key form: the library's choice only with its workspace (without, the wide kernel)
    const bool p16_ws = workspace && workspace_bytes >= pipe_split_bytes(S_max, n_sm);
    if (plan == 5 || (plan == 0 && p16_ws && pipe16_preferred(B * Hq, S_max, r, n_sm))) {
        if (!pipe_split_fits(S_max, device_smem_optin())) return SPARQ_ERR_TOO_LONG;
        if (!p16_ws) return SPARQ_ERR_WORKSPACE;
        return rc(launch_sparq_decode_pipe(q, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, S_max, r, k, opts, out, idx_r, idx_k,
                                           alpha, status, n_sm, static_cast<unsigned int*>(workspace), true,
                                           (cudaStream_t)stream));
    }
    const bool wide_ok = wide_fits(S_max, device_smem_optin());
    if (plan == 4 && !wide_ok) return SPARQ_ERR_TOO_LONG;
    if (wide_ok && (plan == 4 || (plan == 0 && wide_preferred(B * Hq, n_sm, pipe_fits(S_max, device_smem_optin())))))
        return rc(launch_sparq_decode_wide(q, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, S_max, r, k, opts, out, idx_r, idx_k, alpha,
                                           status, wide_pairs(B * Hq, S_max, n_sm), (cudaStream_t)stream));
    const bool split_pays = split_preferred(B * Hq, S_max, r, n_sm, pipe_fits(S_max, device_smem_optin()));
    if (ws_ok && (plan == 3 || (plan == 0 && split_pays)))
        return rc(launch_sparq_decode_split(q, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, S_max, r, k, opts, out, idx_r, idx_k,
                                            alpha, status, splits, workspace, false, (cudaStream_t)stream));
    if (too_long) return SPARQ_ERR_TOO_LONG;                 // a plan without scratch was forced
    const bool fits = pipe_fits(S_max, device_smem_optin());
    if (plan == 2 && !fits) return SPARQ_ERR_TOO_LONG;
    if (plan == 1 && S_max > simple_max_seq_len()) return SPARQ_ERR_TOO_LONG;
    if (fits && plan != 1) {
        // with a workspace the persistent CTAs draw their units from a counter instead of a fixed share
        unsigned int* counter = (workspace && workspace_bytes >= SPARQ_PIPE_WORKSPACE_BYTES && B * Hq > n_sm)
                                    ? static_cast<unsigned int*>(workspace) : nullptr;
        return rc(launch_sparq_decode_pipe(q, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, S_max, r, k, opts, out, idx_r, idx_k,
                                           alpha, status, n_sm, counter, false, (cudaStream_t)stream));
    }
    return rc(launch_sparq_decode(q, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, S_max, r, k, opts, out, idx_r, idx_k, alpha,
                                  status, (cudaStream_t)stream));
}

int sparq_decode(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                 const sparq_half* vbar, const int32_t* seq_lens,
                 int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                 sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                 void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    return decode_with(q, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, d, S_max, r, k, 0u, out, idx_r, idx_k, alpha, workspace,
                       workspace_bytes, status, stream);
}

int sparq_decode_opt(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                     const sparq_half* vbar, const int32_t* seq_lens,
                     int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                     int tau_mode, int realloc, int window,
                     sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                     void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    if (tau_mode < SPARQ_TAU_L1 || tau_mode > SPARQ_TAU_SQRT_R || window < 0 || window > SPARQ_K_MAX)
        return SPARQ_ERR_BAD_OPTION;
    return decode_with(q, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, d, S_max, r, k, pack_opts(tau_mode, realloc != 0, window),
                       out, idx_r, idx_k, alpha, workspace, workspace_bytes, status, stream);
}

static int one_k_splits(int units, int S_max) {
    const int s = split_count(units, S_max, device_sm_count(), /*one_k=*/true);
    return s < 1 ? 1 : s;
}

size_t sparq_1xk_workspace_bytes(int B, int Hq, int Hkv, int d, int S_max) {
    if (bad_common(B, Hq, Hkv, d, S_max)) return 0;
    return split_scratch_bytes(B * Hq, S_max, one_k_splits(B * Hq, S_max));
}

int sparq_decode_1xk(const sparq_half* q, const sparq_half* K, const sparq_half* V, const sparq_half* vbar,
                     const int32_t* seq_lens, int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                     sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                     void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    if (!q || !K || !V || !vbar || !seq_lens || !out) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hq, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    if (r < 1 || r > d || k < 0 || k > SPARQ_K_MAX) return SPARQ_ERR_BAD_RK;
    if (S_max > SPARQ_S_MAX_WORKSPACE) return SPARQ_ERR_TOO_LONG;
    if (misaligned(q, K, V, vbar, out, workspace)) return SPARQ_ERR_ALIGNMENT;
    const int splits = one_k_splits(B * Hq, S_max);
    if (!workspace || workspace_bytes < split_scratch_bytes(B * Hq, S_max, splits)) return SPARQ_ERR_WORKSPACE;
    return rc(launch_sparq_decode_split(q, K, nullptr, V, vbar, seq_lens, B, Hq, Hkv, S_max, r, k, 0u, out, idx_r, idx_k, alpha,
                                        status, splits, workspace, true, (cudaStream_t)stream));
}

size_t sparq_grouped_workspace_bytes(int B, int Hq, int Hkv, int d, int S_max) {
    if (bad_common(B, Hq, Hkv, d, S_max)) return 0;
    return grouped_scratch_bytes(B, Hq, Hkv, S_max, grouped_slices(B * Hkv, S_max, device_sm_count()));
}

static int grouped_with(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                        const sparq_half* vbar, const int32_t* seq_lens,
                        int B, int Hq, int Hkv, int d, int S_max, int r, int k, uint32_t opts,
                        sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                        void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    if (!q || !K || !Kt || !V || !vbar || !seq_lens || !out) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hq, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    const int g = Hq / Hkv;
    if (g != 1 && g != 2 && g != 4 && g != 8) return SPARQ_ERR_BAD_SHAPE;
    if (r < 1 || r > d || k < 0 || k > SPARQ_K_MAX) return SPARQ_ERR_BAD_RK;
    if (misaligned(q, K, Kt, V, vbar, out, workspace)) return SPARQ_ERR_ALIGNMENT;
    if (S_max > SPARQ_S_MAX_WORKSPACE || grouped_dynamic_smem(S_max, Hq / Hkv, k) + 16384 > (size_t)device_smem_optin()) return SPARQ_ERR_TOO_LONG;
    const int slices = grouped_slices(B * Hkv, S_max, device_sm_count());
    if (!workspace || workspace_bytes < grouped_scratch_bytes(B, Hq, Hkv, S_max, slices)) return SPARQ_ERR_WORKSPACE;
    return rc(launch_sparq_decode_grouped(q, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, S_max, r, k, opts, out, idx_r, idx_k,
                                          alpha, status, workspace, slices, (cudaStream_t)stream));
}

int sparq_decode_grouped(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                         const sparq_half* vbar, const int32_t* seq_lens,
                         int B, int Hq, int Hkv, int d, int S_max, int r, int k, int realloc,
                         sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                         void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    return grouped_with(q, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, d, S_max, r, k, pack_opts(SPARQ_TAU_L1, realloc != 0, 0), out,
                        idx_r, idx_k, alpha, workspace, workspace_bytes, status, stream);
}

int sparq_decode_grouped_opt(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                             const sparq_half* vbar, const int32_t* seq_lens,
                             int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                             int tau_mode, int realloc, int window,
                             sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                             void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    if (tau_mode < SPARQ_TAU_L1 || tau_mode > SPARQ_TAU_SQRT_R || window < 0 || window > SPARQ_K_MAX)
        return SPARQ_ERR_BAD_OPTION;
    return grouped_with(q, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, d, S_max, r, k, pack_opts(tau_mode, realloc != 0, window), out,
                        idx_r, idx_k, alpha, workspace, workspace_bytes, status, stream);
}

size_t dense_workspace_bytes(int B, int Hq, int Hkv, int d, int S_max) {
    if (bad_common(B, Hq, Hkv, d, S_max)) return 0;
    return dense_scratch_bytes(B, Hq, Hkv, S_max);
}

int dense_decode(const sparq_half* q, const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                 int B, int Hq, int Hkv, int d, int S_max, sparq_half* out,
                 void* workspace, size_t workspace_bytes, int32_t* status, void* stream) {
    if (!q || !K || !V || !seq_lens || !out) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hq, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    if (misaligned(q, K, V, out, workspace)) return SPARQ_ERR_ALIGNMENT;
    const size_t need = dense_scratch_bytes(B, Hq, Hkv, S_max);
    if (need && (!workspace || workspace_bytes < need)) return SPARQ_ERR_WORKSPACE;
    return rc(launch_dense_decode(q, K, V, seq_lens, B, Hq, Hkv, S_max, out, (float*)workspace, status,
                                  (cudaStream_t)stream));
}

int dense_decode_static(const sparq_half* q, const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                        int B, int Hq, int Hkv, int d, int S_max, sparq_half* out, int32_t* status, void* stream) {
    if (!q || !K || !V || !seq_lens || !out) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hq, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    if (misaligned(q, K, V, out)) return SPARQ_ERR_ALIGNMENT;
    if (dense_scratch_bytes(B, Hq, Hkv, S_max) > SPARQ_STATIC_SCRATCH_BYTES) return SPARQ_ERR_STATIC_SCRATCH;
    float* scratch = nullptr;
    size_t bytes = 0;
    if (dense_static_scratch(&scratch, &bytes) != cudaSuccess) return SPARQ_ERR_CUDA;
    return rc(launch_dense_decode(q, K, V, seq_lens, B, Hq, Hkv, S_max, out, scratch, status, (cudaStream_t)stream));
}

// device copies of q, out, k_new, v_new, then the workspace sparq_decode would like for these shapes
static size_t step_host_ws_bytes(int B, int Hq, int Hkv, int d, int S_max, int r, int k) {
    const size_t want = sparq_workspace_bytes(B, Hq, Hkv, d, S_max, r, k);
    return want > SPARQ_PIPE_WORKSPACE_BYTES ? want : SPARQ_PIPE_WORKSPACE_BYTES;
}
size_t sparq_step_host_staging_bytes(int B, int Hq, int Hkv, int d, int S_max, int r, int k) {
    if (bad_common(B, Hq, Hkv, d, S_max)) return 0;
    return ((size_t)2 * B * Hq * d + (size_t)2 * B * Hkv * d) * sizeof(sparq_half) + step_host_ws_bytes(B, Hq, Hkv, d, S_max, r, k);
}

int sparq_step_host(const sparq_half* q_host, const sparq_half* k_new_host, const sparq_half* v_new_host,
                    sparq_half* K, sparq_half* Kt, sparq_half* V, float* vsum, sparq_half* vbar,
                    int32_t* seq_lens, int B, int Hq, int Hkv, int d, int S_max, int r, int k,
                    sparq_half* out_host, void* staging, size_t staging_bytes, int32_t* status, void* stream) {
    const bool packed = !k_new_host && !v_new_host;          // q_host holds q, k_new, v_new back to back
    if (!q_host || !out_host || (!packed && (!k_new_host || !v_new_host))) return SPARQ_ERR_NULL_POINTER;
    if (bad_common(B, Hq, Hkv, d, S_max)) return SPARQ_ERR_BAD_SHAPE;
    if (!staging || staging_bytes < sparq_step_host_staging_bytes(B, Hq, Hkv, d, S_max, r, k)) return SPARQ_ERR_WORKSPACE;
    if (misaligned(staging)) return SPARQ_ERR_ALIGNMENT;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t nq = (size_t)B * Hq * d, nkv = (size_t)B * Hkv * d;
    sparq_half* q_dev = (sparq_half*)staging;                // device copies: q | k_new | v_new | out
    sparq_half* k_dev = q_dev + nq;
    sparq_half* v_dev = k_dev + nkv;
    sparq_half* out_dev = v_dev + nkv;
    if (packed) {                                            // one copy instead of three
        if (cudaMemcpyAsync(q_dev, q_host, (nq + 2 * nkv) * sizeof(sparq_half), cudaMemcpyHostToDevice, st) != cudaSuccess)
            return SPARQ_ERR_CUDA;
    } else if (cudaMemcpyAsync(q_dev, q_host, nq * sizeof(sparq_half), cudaMemcpyHostToDevice, st) != cudaSuccess ||
               cudaMemcpyAsync(k_dev, k_new_host, nkv * sizeof(sparq_half), cudaMemcpyHostToDevice, st) != cudaSuccess ||
               cudaMemcpyAsync(v_dev, v_new_host, nkv * sizeof(sparq_half), cudaMemcpyHostToDevice, st) != cudaSuccess) {
        return SPARQ_ERR_CUDA;
    }
    int code = sparq_cache_append(k_dev, v_dev, K, Kt, V, vsum, vbar, seq_lens, B, Hkv, d, S_max, status, stream);
    if (code != SPARQ_OK) return code;
    void* ws = out_dev + nq;                                 // the tail of the staging area: the decode's workspace
    code = sparq_decode(q_dev, K, Kt, V, vbar, seq_lens, B, Hq, Hkv, d, S_max, r, k, out_dev, nullptr, nullptr, nullptr,
                        ws, step_host_ws_bytes(B, Hq, Hkv, d, S_max, r, k), status, stream);
    if (code != SPARQ_OK) return code;
    if (cudaMemcpyAsync(out_host, out_dev, nq * sizeof(sparq_half), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return SPARQ_ERR_CUDA;
    return cudaStreamSynchronize(st) == cudaSuccess ? SPARQ_OK : SPARQ_ERR_CUDA;
}

}  // extern "C"
