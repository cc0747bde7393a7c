// Shared definitions of the streaming dual-KV-cache kernels: cache page layout, launch
// parameter blocks and small PTX wrappers (mbarrier, bulk copies, bounded waits).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace st {

// ------------------------------------------------------------------------------------------
// Page layout in HBM.
//
// A page holds 64 tokens. For one (layer, page, kv head) the pool stores one 32 KiB block:
//
//   bytes [0, 16384)      rotated keys K, as two panels (channels 0..63, 64..127); a panel is
//                         64 rows (tokens) of 128 bytes (64 bf16 channels);
//   bytes [16384, 32768)  values, TRANSPOSED: one panel of 128 rows (channels) of 128 bytes
//                         (64 bf16 tokens).
//
// Inside every panel the eight 16-byte chunks of a row are permuted: chunk c of row r is stored
// at chunk position c ^ (r & 7). This is the 128-byte swizzle pattern of the sm_100 tensor-core
// shared-memory operand format, so a block copied verbatim to 1024-byte aligned shared memory
// (one bulk copy, no tensor map) is directly a K-major MMA operand: K for Q K^T (rows = keys,
// contraction over channels) and V^T for P V (rows = channels, contraction over keys). The same
// permutation makes ldmatrix reads of the decode kernel bank-conflict free.
// ------------------------------------------------------------------------------------------
constexpr int kHeadDim = 128;
constexpr int kPageTokens = 64;
constexpr int kBlockBytes = 32768;
constexpr int kKeyBytes = 16384;
constexpr int kPanelBytesK = 8192;
constexpr int kRopeLoSteps = 1024;      // positions covered by the fine rotation table
constexpr int kMaxSplitItems = 74;     // work items of one tensor-core attention launch that may be split by keys
constexpr int kMaxSeqPerLaunch = 112;   // keeps every parameter block under the 4 KiB limit
constexpr int kMaxGroup = 8;            // q heads per kv head

__host__ __device__ __forceinline__ uint32_t k_byte_offset(int tok, int c) {
  return (uint32_t)((c >> 6) * kPanelBytesK + tok * 128 + ((((c & 63) >> 3) ^ (tok & 7)) << 4) + ((c & 7) << 1));
}
__host__ __device__ __forceinline__ uint32_t vt_byte_offset(int tok, int c) {
  return (uint32_t)(kKeyBytes + c * 128 + (((tok >> 3) ^ (c & 7)) << 4) + ((tok & 7) << 1));
}

// Device status word values (written by a kernel that gave up a bounded wait).
constexpr int kDevOk = 0;
constexpr int kDevTimeoutDecode = 1;
constexpr int kDevTimeoutPrefill = 2;
constexpr int kDevTimeoutProbe = 3;     // the wait-expiry test kernel
constexpr int kDevTimeoutLinear = 5;    // the projection kernel
constexpr int kDevBadPage = 4;          // a page id read from a page table lies outside its pool: the access was skipped

// ------------------------------------------------------------------------------------------
// Launch parameter blocks (passed by value: stream ordered, no staging buffers).
// ------------------------------------------------------------------------------------------
struct AppendSeq {
  int32_t slot;       // sequence slot = page-table row
  int32_t pos0;       // position id of the sequence's first new token (= tokens already cached)
  int32_t n;          // new tokens of this sequence
  int32_t q_begin;    // first packed row of this sequence in q/k/v
  int32_t blk_begin;  // first thread block of this sequence (blocks cover aligned groups of 8 positions)
  int32_t rope_off;   // position id of a token = its index in the cache + rope_off (0 with the streaming position encoding)
};

struct AppendParams {
  const __nv_bfloat16 *q, *k, *v;  // packed [tokens][heads][128]
  __nv_bfloat16 *qhat;             // rotated queries, packed [tokens][n_q_heads][128]
  uint8_t *pool;                   // layer base of the pool written to
  const int32_t *ptab;             // [max_batch][ptab_stride] page ids
  int32_t ptab_stride;
  int32_t n_pages;                 // pages of the pool: a page id outside [0, n_pages) is reported, not used
  int32_t *status;                 // device status word
  // per-head RMS normalisation of q and k before the rotation (nullptr: none): weights of this layer, [128] each
  const float *norm_q, *norm_k;
  float norm_eps;
  int32_t n_seq, n_q_heads, n_kv_heads;
  double inv_freq[64];             // theta^(-2c/128), c = 0..63
  AppendSeq seq[kMaxSeqPerLaunch];
};

// Generic two-range attention: row i of a sequence (i = 0..n_rows-1) attends to
//   range A: keys [0, a_len) of cache A, no mask inside the range;
//   range B: keys [0, b_base + i] of cache B (causal).
// Chunk prefill: A empty, B = source cache. Decode / extend: A = source prefix, B = reasoning cache.
struct AttnSeq {
  int32_t slot;
  int32_t a_len;
  int32_t b_base;
  int32_t n_rows;
  int32_t q_begin;    // first packed row in qhat / out
  int32_t work_begin; // kernel specific prefix (tiles or blocks)
  int32_t rope_off;   // position id of row i = b_base + i + rope_off (kernels that rotate their own queries or keys)
};

struct AttnParams {
  const uint8_t *pool_a, *pool_b;  // layer bases
  const int32_t *ptab_a, *ptab_b;
  int32_t ptab_stride_a, ptab_stride_b;
  int32_t n_pages_a, n_pages_b;    // pages of each pool: a page id outside [0, n_pages) is reported, not used
  const __nv_bfloat16 *qhat;
  // Un-rotated inputs of the call, packed [tokens][heads][128]. Decode with the append fused in (q_raw != nullptr):
  // the kernel rotates q and k, writes the new token into cache B and does not read qhat. Tensor-core kernel: q_raw
  // only (always set); it rotates the rows of its Q tiles while staging them and never reads qhat.
  const __nv_bfloat16 *q_raw, *k_raw, *v_raw;
  float *out;                      // [rows][n_q_heads][128]
  float *partial;                  // split-K workspace (decode)
  int32_t *status;                 // device status word
  int32_t n_seq, n_q_heads, n_kv_heads, group;
  int32_t total_work;              // total tiles (decode) / blocks (prefill)
  int32_t work_per_cta;            // decode: tiles per CTA
  int32_t reverse;                 // decode: every CTA walks its slice of the tile list from the end to the start
  int32_t n_cta;
  float scale_log2;                // softmax scale * log2(e)
  double inv_freq[64];             // theta^(-2c/128): the tensor-core kernel rotates its queries itself (from q_raw)
  // per-head RMS normalisation of q and k before the rotation, for the kernels that rotate their own (nullptr: none)
  const float *norm_q, *norm_k;
  float norm_eps;
  // decode with the append fused in: (cos, sin) of k * 1024 * inv_freq[c] and of j * inv_freq[c], j < 1024, as [.][64]
  const double2 *rope_hi, *rope_lo;
  // Tensor-core kernel, key split of the last work items of a launch (see st_k_attn_tc): the last n_split items are
  // run by two CTAs each, one per half of the keys; whichever finishes second merges. Workspace per split item and
  // half: 256 rows x 128 un-normalised outputs, 256 x (reference maximum, row sum); one ticket per item and M-tile.
  float *split_o;
  float2 *split_ml;
  int32_t *split_ticket;
  int32_t n_split;
  AttnSeq seq[kMaxSeqPerLaunch];
};
static_assert(sizeof(AttnParams) <= 4096, "kernel parameter space");

struct PageUpdate {
  int32_t slot_which;  // slot * 2 + which
  int32_t index;
  int32_t page;
};
constexpr int kMaxPageUpdates = 320;
struct PageUpdateParams {
  int32_t *ptab[2];
  int32_t stride[2];
  int32_t n;
  PageUpdate upd[kMaxPageUpdates];
};

// Split-K partial record (decode): per (pair, cta) slot, for 8 head columns:
//   float o[8][128] (unnormalised), float m[8] (log2 domain), float l[8].
constexpr int kPartialFloats = 8 * 128 + 16;

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
#ifdef __CUDACC__

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\n"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Page id check of every page-table read that turns into an address: an id outside the pool is recorded in the status
// word and the caller skips the access (no trap, no fault). One compare in one lane per 32 KiB block.
__device__ __forceinline__ bool page_ok(int page, int n_pages, volatile int *abort_flag, int32_t *status) {
  if ((unsigned)page < (unsigned)n_pages) return true;
  *abort_flag = 1;
  atomicExch(status, kDevBadPage);
  return false;
}

// Bounded wait on an mbarrier phase. Gives up after kWaitLimitNs of wall time (or when another
// thread of the CTA has already given up), records `code` in the global status word, raises the
// CTA's abort flag and returns false. Callers leave their loops and go to the common exit path.
// The wall clock is looked at only every 256 failed polls (a poll itself suspends the thread for
// a while), so a wait that is satisfied quickly never pays for reading the timer.
constexpr uint64_t kWaitLimitNs = 2000000000ull;
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int *abort_flag,
                                          int32_t *status, int code, uint64_t limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  uint64_t t0 = 0;
  uint32_t polls = 0;
  while (true) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((++polls & 255u) == 0u) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > limit_ns) {
        *abort_flag = 1;
        atomicExch(status, code);
        return false;
      }
    }
  }
}

// One contiguous bulk copy global -> shared, completion counted in bytes on an mbarrier.
// Both addresses and the size are multiples of 16 bytes by construction (whole cache blocks).
__device__ __forceinline__ void bulk_load(uint32_t dst_smem, const void *src, uint32_t bytes, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst_smem),
      "l"(src), "r"(bytes), "r"(bar)
      : "memory");
}

// Largest i in [0, n) with key(i) <= target, for a non-decreasing key with key(0) <= target: the work item ->
// sequence look-up of the kernels (a linear scan over 32 entries of the parameter block cost ~1,000 cycles).
template <typename F>
__device__ __forceinline__ int last_not_above(int n, int target, F key) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (key(mid) <= target) lo = mid;
    else hi = mid - 1;
  }
  return lo;
}

// 16-byte asynchronous copy global -> shared (L2 only); src_bytes = 0 writes zeros and reads nothing.
__device__ __forceinline__ void cp_async16(uint32_t dst_smem, const void *src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Programmatic dependent launch: a kernel launched with launch_dependent() may start before the kernel in front
// of it in the stream has finished. grid_dep_launch() (early in every kernel) lets the next kernel's blocks
// become resident while this grid drains; grid_dep_wait() (before the first access to global memory) holds them
// until the previous grid has completed and its writes are visible. Both are no-ops in an ordinary launch.
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// generic-proxy writes (any state space) before later async-proxy reads (bulk copies) of this thread
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

__device__ __forceinline__ float exp2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&t);
}

#endif  // __CUDACC__

}  // namespace st
