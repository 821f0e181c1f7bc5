// Internal launch interfaces between the kernel files and the C ABI (api.cu).
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "sparq.h"

namespace sparq {

// api.cu: multiprocessors, largest opt-in shared memory per block, shared memory per multiprocessor of
// the current device (cached per device; zeros without a device)
struct DeviceInfo { int sm_count, smem_optin, smem_per_sm; };
DeviceInfo device_info();

// `opts` of the decode launchers: the call's settings in one word (0 = Eq. (9) temperature, Step 3
// applied, no local window).  Bits 0-1: temperature (SPARQ_TAU_*), bit 2: Step 3 left out,
// bits 16-31: local window.
inline uint32_t pack_opts(int tau_mode, int realloc, int window) {
    return (uint32_t)tau_mode | (realloc ? 0u : 4u) | ((uint32_t)window << 16);
}

// sparq_decode.cu
size_t decode_static_smem();
size_t decode_dynamic_smem(int S_max);
int decode_max_positions();
cudaError_t launch_sparq_decode(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                int r, int k, uint32_t opts, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                int32_t* status, cudaStream_t stream);

// split-S plan (sparq_decode.cu): one CTA per (slice, unit) with the keys in a scratch buffer, for
// caches too long for the persistent kernel and for few units with long sequences
int split_count(int units, int S_max, int n_sm, bool one_k = false);
size_t split_scratch_bytes(int units, int S_max, int splits);
cudaError_t launch_sparq_decode_split(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                      const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                      int r, int k, uint32_t opts, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                      int32_t* status, int splits, void* scratch, bool one_k, cudaStream_t stream);

// sparq_decode_pipe.cu: persistent warp-specialised variant for S_max small enough that three key
// buffers, the copy ring and two post-phase scratch areas fit in shared memory
// Split-key form (the keys' upper halves in shared memory, the lower halves in pipe_split_workspace()
// bytes of the caller's workspace): reaches caches about three times as long.
bool pipe_fits(int S_max, int smem_optin);
bool pipe_split_fits(int S_max, int smem_optin);
bool pipe_split_thin_ring(int S_max, int smem_optin);    // only a ring of 16 KB stages fits beside the keys (S_max beyond about 12,700)
size_t pipe_split_workspace(int S_max, int n_sm);
cudaError_t launch_sparq_decode_pipe(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                     const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                     int r, int k, uint32_t opts, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                     int32_t* status, int n_sm, unsigned int* unit_counter, bool split_keys,
                                     cudaStream_t stream);

// sparq_decode_wide.cu: one CTA of 512 threads per unit, for a handful of units (batch-1 latency)
bool wide_fits(int S_max, int smem_optin);
bool wide_pair_fits(int S_max, int smem_per_sm);
cudaError_t launch_sparq_decode_wide(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                     const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                     int r, int k, uint32_t opts, sparq_half* out, int32_t* idx_r, int32_t* idx_k, float* alpha,
                                     int32_t* status, bool pairs, cudaStream_t stream);

// sparq_decode_grouped.cu: group-shared selection (one CTA per KV head)
int grouped_slices(int groups, int S_max, int n_sm);
size_t grouped_scratch_bytes(int B, int Hq, int Hkv, int S_max, int slices);
size_t grouped_dynamic_smem(int S_max, int g, int k);
cudaError_t launch_sparq_decode_grouped(const sparq_half* q, const sparq_half* K, const sparq_half* Kt, const sparq_half* V,
                                        const sparq_half* vbar, const int32_t* seq_lens, int B, int Hq, int Hkv, int S_max,
                                        int r, int k, uint32_t opts, sparq_half* out, int32_t* idx_r, int32_t* idx_k,
                                        float* alpha, int32_t* status, void* scratch, int slices, cudaStream_t stream);

// dense_decode.cu
int dense_splits(int B, int Hkv, int S_max);
size_t dense_scratch_bytes(int B, int Hq, int Hkv, int S_max);
cudaError_t launch_dense_decode(const sparq_half* q, const sparq_half* K, const sparq_half* V, const int32_t* seq_lens,
                                int B, int Hq, int Hkv, int S_max, sparq_half* out, float* scratch, int32_t* status,
                                cudaStream_t stream);

cudaError_t dense_static_scratch(float** ptr, size_t* bytes);   // library-owned scratch on the current device

// cache.cu
cudaError_t launch_cache_build(const sparq_half* K, const sparq_half* V, const int32_t* seq_lens, sparq_half* Kt,
                               float* vsum, sparq_half* vbar, int B, int Hkv, int S_max, int32_t* status,
                               cudaStream_t stream);
cudaError_t launch_cache_append(const sparq_half* k_new, const sparq_half* v_new, sparq_half* K, sparq_half* Kt,
                                sparq_half* V, float* vsum, sparq_half* vbar, int32_t* seq_lens, int B, int Hkv,
                                int S_max, int32_t* status, cudaStream_t stream);

}  // namespace sparq
