// Host-side launchers of the kernels (one translation unit per kernel family).
#pragma once

#include "st_common.cuh"

namespace st {

// Applies page-table updates on the stream (append-only tables; entries in use are never rewritten).
cudaError_t launch_page_update(const PageUpdateParams &p, cudaStream_t stream);

// RoPE at the streaming position ids + paged append of K and V + rotated queries to scratch.
cudaError_t launch_rope_append(const AppendParams &p, int total_blocks, cudaStream_t stream);

// Slow, simple attention over the generic two-range form (one warp per row and q head).
cudaError_t launch_attn_reference(const AttnParams &p, int total_rows, cudaStream_t stream);

// Dual-cache decode: one row per sequence, split-K over both caches, then the LSE merge.
// Returns the number of launches in *n_launches.
// t0/t1 (optional) are recorded immediately before and after the main kernel.
cudaError_t launch_decode(AttnParams &p, int num_sms, cudaStream_t stream, int *n_launches,
                          cudaEvent_t t0 = nullptr, cudaEvent_t t1 = nullptr);
// Workspace floats needed by launch_decode for up to n_seq sequences per launch.
size_t decode_partial_floats(int n_seq_per_launch, int n_kv_heads, int num_sms);

// Multi-row attention on tensor cores (chunk prefill and reasoning spans).
// precise: probabilities as two bf16 terms (one more P V product per key tile), for values of large magnitude.
cudaError_t launch_attn_tc(AttnParams &p, bool precise, int num_sms, cudaStream_t stream, int *n_launches,
                           cudaEvent_t t0 = nullptr, cudaEvent_t t1 = nullptr);
int attn_tc_rows_per_cta();

// Gathers tokens [tok0, tok0+ntok) of one sequence into plain [ntok][Hkv][128] K and V buffers.
cudaError_t launch_cache_gather(const uint8_t *pool, const int32_t *ptab_row, int n_kv_heads, int tok0, int ntok,
                                __nv_bfloat16 *k_out, __nv_bfloat16 *v_out, cudaStream_t stream);

// Launch with programmatic stream serialisation: the kernel may begin while its predecessor in the stream drains
// (see grid_dep_launch / grid_dep_wait). Launch latency and kernel prologues then overlap the previous kernel's tail,
// which matters for the decode step's chain of short kernels.
template <typename P>
inline cudaError_t launch_dependent(void (*kernel)(const P), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                    const P &params) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, params);
}

// Fills table[i][c] = (cos, sin)(i * step * inv_freq[c]), i < n, c < 64 (rotation tables of the fused decode append).
cudaError_t launch_rope_table(const double *inv_freq, double2 *table, int n, int step, cudaStream_t stream);

// Test surface: one warp waits (at most limit_ns) for a barrier that nothing arrives at, then records kDevTimeoutProbe.
cudaError_t launch_wait_expiry(int32_t *status, uint64_t limit_ns, cudaStream_t stream);

// Fills n 16-bit words with `value` (debug contexts: the sentinel of free pages).
cudaError_t launch_fill_u16(void *dst, size_t n, uint16_t value, cudaStream_t stream);
constexpr uint16_t kPoisonBf16 = 0x7149;   // bf16 0x7149 = 9.96e29: large, finite, and finite after 128-term dot products

// One-time per-process function attribute set-up (dynamic shared memory opt-in).
cudaError_t init_kernels();

}  // namespace st
