// Multi-row attention on the 5th-generation tensor cores (tcgen05 + tensor memory): chunk prefill of
// source units and multi-token reasoning spans.
//
// What it computes. For every packed row (token i of a sequence, q head h) the generic two-range form
//   O = softmax( scale * q^ . [K_A[0:a_len] ; K_B[0 : b_base+i+1]] ) [V_A ; V_B]
// Chunk prefill (Algorithm 1, prefill loop): range A is empty and range B is the source cache, i.e.
// the ordinary causal mask that Eq. 2 keeps for input rows; a source row never sees a reasoning token.
// Reasoning span (Algorithm 1, last step / teacher forcing): range A is the visible source prefix
// (Eq. 1, Eq. 2's streaming region), range B the reasoning cache, causal.
//
// Shape of the kernel. One CTA owns one (sequence, kv head) and up to 256 packed rows, row = token*G + g,
// so the G q heads that share a kv head share every K/V tile (GQA packing). The rows form two 128-row
// M-tiles. Key tiles are 128 keys = two cache pages, so that S = Q K^T is an N = 128 MMA chain (measured here:
// an N = 64 MMA takes 48 cycles, bound by operand reads from shared memory, i.e. 1.5x per flop, and while such
// MMAs run every other shared-memory access of the SM - mbarrier polls included - takes hundreds of cycles).
// Warp roles (10 warps):
//   warps 0-3 / 4-7  softmax + epilogue of M-tile 0 / 1 (one thread per row; TMEM lane = row)
//   warp 8           producer: bulk copies (TMA, no tensor map) of the pages' K panels and V^T panels
//   warp 9           MMA issuer and TMEM allocator. It runs its loop with all 32 lanes and predicates the
//                    instructions on an elected lane, so that descriptors stay warp-uniform values (an issuer that
//                    was a single diverged lane needed ~100 cycles per MMA against 64 of execution).
// Operands. The cache block layout in HBM already is the 128-byte-swizzled K-major shared-memory operand
// format, so panels are used as landed: the two pages' K panels of one channel half are placed one after the
// other and form a 128-key operand; every V^T panel (channels x 64 keys) serves four 16-key steps of P V.
// Q tiles are copied into the same format by the softmax warps with asynchronous 16-byte copies (whole rows per copy
// instruction) from the caller's un-rotated queries, and rotated in place at their position ids (the two-term variant
// takes them rotated from the append kernel's scratch instead).
// Tensor memory (512 columns): S[t] (128 fp32 columns per M-tile) and O[t] (128 columns per M-tile).
// Schedule per M-tile and key tile j (the MMA pipe executes in issue order, which is what the aliasing relies on):
//   the softmax warps work S(j) off as two 64-key online-softmax steps (one cache page each);
//   P of the first half overwrites the first 32 score columns as packed bf16 pairs and P V (j, 0) takes it as its
//   A operand straight from tensor memory;
//   as soon as the second half's scores are in registers the score columns are free: Q K^T (j+1) is issued (after
//   P V (j, 0)) and runs while the softmax warps are in the second half's exponentials, so S(j+1) is complete
//   when they come round; P of the second half therefore goes through shared memory (16 KiB per M-tile) and
//   P V (j, 1) reads both operands from there.
// The issuer serves M-tile 0 and M-tile 1 alternately (P V (j, 0) and Q K^T (j+1) of one, then of the other, then
// the two P V (j, 1)), which is the order in which the events arrive when tile 1 runs a little behind tile 0.
// Softmax is online with a lazily updated reference maximum: O is rescaled (TMEM load, multiply, store)
// only when a row's maximum grew by more than 2^8 since the last rescale, which keeps P within bf16/fp32
// range and leaves the result exact (the same reference is used for P, l and O). The row sum adds the
// bf16-rounded probabilities, i.e. exactly the weights the tensor core applies to V.
// Grid. One CTA per work item (sequence, kv head, 256 packed rows), one CTA per SM at a time, items in launch order
// (the host lists the longest sequences first). When the last wave of items would fill at most half of the SMs, each of
// its items that is long enough is run by two CTAs, one per half of the keys; each leaves its un-normalised share in a
// workspace and whichever finishes second (a ticket per item and M-tile; nobody waits) adds the two shares and writes
// the rows. Measured on 32 sequences x 8 kv heads x 2 row pairs (512 items on 148 SMs, 68 of them cut): 6.8 us per key
// tile and launch against 7.5 without the cut, for 5 us more of fixed cost.
// Every mbarrier wait is bounded; on expiry the CTA records a status word, stops and frees its TMEM.
#include <algorithm>
#include <cstddef>

#include "st_internal.h"

namespace st {

namespace {

constexpr int kKStagesFast = 2;             // K ring depth (32 KiB per stage: 128 keys x 128 channels); the two-term
                                            // variant gives its second stage to the low-order P of the second key half
constexpr int kVStages = 2;                 // V ring depth (32 KiB per stage: two V^T page panels)
constexpr int kProducerWarp = 8, kMmaWarp = 9;
constexpr int kThreads = 320;               // 8 softmax warps, producer, MMA issuer
constexpr int kRowsPerTile = 128;
constexpr int kRowsPerCta = 256;
constexpr int kQTileBytes = 32768;          // 2 channel halves x 128 rows x 128 B
constexpr int kKStageBytes = 32768;         // 2 channel halves x 128 keys x 128 B
constexpr int kVStageBytes = 32768;         // 2 pages x 128 channels x 128 B (64 keys)
constexpr int kHalfPanel = 16384;           // one channel half of a 128-row tile / one V^T page panel
constexpr float kRescaleThreshold = 8.0f;   // log2 units
constexpr int kMinCutPages = 20;             // key split: items of fewer cache pages are not cut (below about ten key
                                            // tiles the merge costs more than the shorter last wave saves)
#ifndef ST_ATTN_POLY_PAIRS
#define ST_ATTN_POLY_PAIRS 0x92u
#endif
constexpr uint32_t kPolyPairs = ST_ATTN_POLY_PAIRS;   // of every 8 score pairs, those whose bit is set take the polynomial exp2

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;
constexpr int kOffK = kOffQ + 2 * kQTileBytes;
constexpr int kOffP1Lo = kOffK + kKStageBytes;            // two-term variant only: low-order P of the second key half, per M-tile
constexpr int kOffV = kOffK + kKStagesFast * kKStageBytes;
constexpr int kOffP1 = kOffV + kVStages * kVStageBytes;   // P of the second key half, per M-tile: 128 rows x 64 keys bf16
constexpr int kP1Bytes = 16384;
constexpr int kOffBar = kOffP1 + 2 * kP1Bytes;
// epilogue staging (over the Q buffers and the start of the first K stage): one line per row
constexpr int kOutStageLine = 272, kOutStageTile = 36864;
static_assert(kOutStageTile >= kRowsPerTile * kOutStageLine && kOutStageTile + kRowsPerTile * kOutStageLine <= kOffK + kKStageBytes, "epilogue staging");
constexpr int kSmemBytes = kOffBar + 256;
static_assert(kSmemBytes + 1024 <= 232448, "shared memory budget of one CTA");

struct Barriers {
  uint64_t q_full[2];
  uint64_t k_full[kKStagesFast];
  uint64_t k_empty[kKStagesFast];
  uint64_t v_full[kVStages];
  uint64_t v_empty[kVStages];
  uint64_t s_full[2];     // S[t](j) complete
  uint64_t p_full[2][2];  // P[t](j), key half h, published by the tile's four softmax warps (half 0 in tensor memory,
                          // half 1 in shared memory)
  uint64_t y_loaded[2];   // the tile's softmax warps hold all scores of S[t](j) in registers or have used them:
                          // the score columns may be overwritten once P V (j, half 0) has been issued
  uint64_t pv0_done[2];   // P V [t](j) of key half 0 complete (O may be rescaled before half 1 is published)
  uint64_t p1_free[2];    // P V [t](j) of key half 1 complete: its shared-memory P may be overwritten, O rescaled
  uint64_t o_final[2];    // the last P V of M-tile t is complete: O[t] may be read
  uint32_t tmem_base;
  int abort_flag;
};
static_assert(sizeof(Barriers) <= 256, "barrier block too large");

// TMEM column map
constexpr uint32_t kColS = 0;      // S[t] at kColS + t*128; P of key half h aliases columns 64h .. 64h+31
constexpr uint32_t kColO = 256;    // O[t] at kColO + t*128

// ---- tcgen05 wrappers ----------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// The MMA warp runs its loop with all 32 lanes, so that addresses and descriptors stay warp-uniform values
// (an issuer that is a single diverged lane needed about 100 cycles per instruction, against 64 of execution);
// the instructions themselves are issued by one elected lane (`issue` != 0 in that lane only).
__device__ __forceinline__ uint32_t elect_one() {
  uint32_t pred;
  asm volatile("{\n.reg .pred P;\nelect.sync _|P, 0xffffffff;\nselp.u32 %0, 1, 0, P;\n}\n" : "=r"(pred));
  return pred;
}
__device__ __forceinline__ void tc_commit(uint32_t bar, uint32_t issue) {
  asm volatile(
      "{\n.reg .pred q;\n"
      "setp.ne.b32 q, %1, 0;\n"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}\n" ::"r"(bar), "r"(issue)
      : "memory");
}
// D[tmem] (+)= A[smem] . B[smem]^T
__device__ __forceinline__ void tc_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate, uint32_t issue) {
  asm volatile(
      "{\n.reg .pred p, q;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "setp.ne.b32 q, %5, 0;\n"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(issue)
      : "memory");
}
// D[tmem] (+)= A[tmem] . B[smem]^T  (A: row = lane, two bf16 of consecutive k per 32-bit column)
__device__ __forceinline__ void tc_mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate, uint32_t issue) {
  asm volatile(
      "{\n.reg .pred p, q;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "setp.ne.b32 q, %5, 0;\n"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n}\n" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(issue)
      : "memory");
}
// One bulk store shared -> global (TMA, no tensor map): both addresses 16-byte aligned, size a multiple of 16.
__device__ __forceinline__ void bulk_store(void *dst, uint32_t src_smem, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src_smem), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// until the bulk stores of this thread have read their shared-memory source
__device__ __forceinline__ void bulk_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 consecutive columns of this thread's TMEM lane (warp w reads lanes 32*(w%4) .. +31)
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float *r) {
  uint32_t *u = reinterpret_cast<uint32_t *>(r);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]),
        "=r"(u[9]), "=r"(u[10]), "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]),
        "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]), "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]),
        "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]), "=r"(u[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t *u) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "r"(u[0]), "r"(u[1]), "r"(u[2]), "r"(u[3]), "r"(u[4]), "r"(u[5]), "r"(u[6]), "r"(u[7]), "r"(u[8]), "r"(u[9]),
      "r"(u[10]), "r"(u[11]), "r"(u[12]), "r"(u[13]), "r"(u[14]), "r"(u[15]), "r"(u[16]), "r"(u[17]), "r"(u[18]),
      "r"(u[19]), "r"(u[20]), "r"(u[21]), "r"(u[22]), "r"(u[23]), "r"(u[24]), "r"(u[25]), "r"(u[26]), "r"(u[27]),
      "r"(u[28]), "r"(u[29]), "r"(u[30]), "r"(u[31])
      : "memory");
}

// Shared-memory operand descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
//   bits 0-13 start address >> 4, 16-29 leading offset >> 4 (unused with swizzle: 1), 32-45 stride
//   offset >> 4 (1024 B), 46-47 descriptor version 1, 61-63 layout 2 = 128-byte swizzle.
// Adding (byte offset >> 4) to a descriptor moves its start address (no carry leaves the 14-bit field here).
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulator, bf16 x bf16, both operands K-major, M = 128.
__host__ __device__ constexpr uint32_t make_idesc(int n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// Barrier among the four softmax warps of M-tile t (named barriers 1 and 2; 0 is __syncthreads).
__device__ __forceinline__ void tile_sync(int t) {
  if (t == 0) asm volatile("bar.sync 1, 128;" ::: "memory");
  else asm volatile("bar.sync 2, 128;" ::: "memory");
}

// ---- arithmetic helpers -------------------------------------------------------------------
__device__ __forceinline__ uint32_t cvt_bf16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// two-wide fp32 arithmetic on register pairs
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) {
  float2 d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;"
      : "=l"(reinterpret_cast<uint64_t &>(d))
      : "l"(reinterpret_cast<const uint64_t &>(a)), "l"(reinterpret_cast<const uint64_t &>(b)),
        "l"(reinterpret_cast<const uint64_t &>(c)));
  return d;
}
__device__ __forceinline__ float2 fmul2(float2 a, float2 b) {
  float2 d;
  asm("mul.rn.f32x2 %0, %1, %2;"
      : "=l"(reinterpret_cast<uint64_t &>(d))
      : "l"(reinterpret_cast<const uint64_t &>(a)), "l"(reinterpret_cast<const uint64_t &>(b)));
  return d;
}
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) {
  float2 d;
  asm("add.rn.f32x2 %0, %1, %2;"
      : "=l"(reinterpret_cast<uint64_t &>(d))
      : "l"(reinterpret_cast<const uint64_t &>(a)), "l"(reinterpret_cast<const uint64_t &>(b)));
  return d;
}
// 2^x for a pair, on the FMA pipe: x = n + f with n = round(x) and f in [-1/2, 1/2]; 2^f by a cubic with
// relative error 7.6e-5 (the result is rounded to bf16, half an ulp of which is 2e-3), then n is added to
// the exponent field. Inputs below -126 (masked scores are -inf) give 2^-126 instead of 0.
__device__ __forceinline__ float2 exp2_poly2(float2 x) {
  const float2 magic = make_float2(12582912.f, 12582912.f);          // 1.5 * 2^23: x + magic has round(x) in its low bits
  const float2 neg_magic = make_float2(-12582912.f, -12582912.f);
  x.x = fmaxf(x.x, -126.f);
  x.y = fmaxf(x.y, -126.f);
  const float2 t = fadd2(x, magic);
  const float2 n = fadd2(t, neg_magic);
  const float2 f = ffma2(n, make_float2(-1.f, -1.f), x);
  float2 q = ffma2(f, make_float2(0.05520550534f, 0.05520550534f), make_float2(0.2426139712f, 0.2426139712f));
  q = ffma2(q, f, make_float2(0.6932547688f, 0.6932547688f));
  q = ffma2(q, f, make_float2(0.9999276996f, 0.9999276996f));
  return make_float2(__int_as_float(__float_as_int(q.x) + (__float_as_int(t.x) << 23)),
                     __int_as_float(__float_as_int(q.y) + (__float_as_int(t.y) << 23)));
}
__device__ __forceinline__ float sin_approx(float x) {
  float y;
  asm("sin.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float cos_approx(float x) {
  float y;
  asm("cos.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// acc_lo += low bf16 of pk, acc_hi += high bf16 of pk (fp32 accumulation of bf16 terms)
__device__ __forceinline__ void add_bf16x2(float &acc_lo, float &acc_hi, uint32_t pk) {
  asm("{\n.reg .b16 lo, hi;\n"
      "mov.b32 {lo, hi}, %2;\n"
      "add.rn.f32.bf16 %0, lo, %0;\n"
      "add.rn.f32.bf16 %1, hi, %1;\n}\n"
      : "+f"(acc_lo), "+f"(acc_hi)
      : "r"(pk));
}

}  // namespace

// kPrecise: the probabilities enter P V as two bf16 terms (p = hi + lo, 16 significant bits) instead of one. One bf16
// term bounds a row's error by about 2^-9 times the largest |v| it mixes, which leaves the 1e-2 tolerance when values
// reach a few tens (outlier channels); the second term costs one more P V product per key tile.
// kNorm (one-term variant only): per-head RMS normalisation of the query rows in front of their rotation. A template
// parameter because the same code as a run-time option cost the kernel 6 us per launch with the option off (788 against
// 820 TFLOP/s on the appends of the benchmark workload).
template <bool kPrecise, bool kNorm>
__global__ void __launch_bounds__(kThreads, 1) st_k_attn_tc(const __grid_constant__ AttnParams p) {
  constexpr int kKStages = kPrecise ? 1 : kKStagesFast;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  Barriers &bar = *reinterpret_cast<Barriers *>(smem + kOffBar);
  volatile int *abort_flag = &bar.abort_flag;
  // warp index broadcast from lane 0, so that the compiler knows the role branches are warp-uniform
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const int G = p.group, Hkv = p.n_kv_heads, Hq = p.n_q_heads;
  // packed row -> token: row / G by multiplication (G <= 8, rows < 2^24: exact); the generic division is ~30 instructions
  const uint32_t g_magic = (uint32_t)((0x100000000ull + (uint32_t)G - 1u) / (uint32_t)G);
  auto div_g = [&](int row) { return G == 1 ? row : (int)__umulhi((uint32_t)row, g_magic); };

  // ---- which work item (sequence, kv head, row pair) is this CTA, and which part of its keys.
  // The last n_split items of the launch are run by two CTAs each (CTA indices from first_split on, two per item).
  const int first_split = p.total_work - p.n_split;
  int item = (int)blockIdx.x, part = -1;                     // part -1: all keys of the item
  if (item >= first_split) {
    const int k = item - first_split;
    item = first_split + (k >> 1);
    part = k & 1;
  }
  const int split_idx = item - first_split;
  const int s = last_not_above(p.n_seq, item, [&](int i) { return p.seq[i].work_begin; });
  const AttnSeq sq = p.seq[s];
  const int packed_rows = sq.n_rows * G;
  const int pairs = (packed_rows + kRowsPerCta - 1) / kRowsPerCta;
  const int rel = item - sq.work_begin;
  const int kvh = rel / pairs, pair = rel - kvh * pairs;
  const int row0 = pair * kRowsPerCta;                       // first packed row of the CTA

  // per M-tile geometry: pages (range A pages, then range B pages) and 128-key tiles
  const int nA = (sq.a_len + 63) >> 6;
  int np_all[2], n_pages_all = 0;                            // pages each M-tile looks at, over all keys of the item
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    const int r_lo = row0 + t * kRowsPerTile;
    const int r_hi = min(r_lo + kRowsPerTile, packed_rows) - 1;
    np_all[t] = r_lo < packed_rows ? nA + ((sq.b_base + r_hi / G) >> 6) + 1 : 0;
    n_pages_all = max(n_pages_all, np_all[t]);
  }
  // Key split. An item of at least kMinCutPages pages is cut at a tile boundary near its middle: part 0 takes the pages in
  // front of page_mid, part 1 those from page_mid on (M-tile 0 looks at no less than the item's page count minus two,
  // so both parts of both M-tiles are non-empty). Each part leaves un-normalised outputs with its reference maxima and
  // row sums in the workspace; whichever part of an M-tile finishes second adds the two and writes the rows out. A
  // shorter item is not cut: part 0 does all of it, part 1 has nothing to do.
  const bool cut = part >= 0 && n_pages_all >= kMinCutPages;
  const int page_mid = 2 * (((n_pages_all + 1) >> 1) >> 1);
  const int pg0 = cut && part == 1 ? page_mid : 0;           // first page of this CTA's share
  int n_tiles[2];
  bool active[2];
  int n_pages = 0;
#pragma unroll
  for (int t = 0; t < 2; ++t) {
    int np = np_all[t];
    if (cut) np = part == 0 ? min(np, page_mid) : max(np - page_mid, 0);
    if (!cut && part == 1) np = 0;
    active[t] = np > 0;
    n_tiles[t] = (np + 1) >> 1;
    n_pages = max(n_pages, np);
  }
  const int n_max = (n_pages + 1) >> 1;

  // Q rows of M-tile t into the swizzled operand layout, by asynchronous 16-byte copies: the tile's 128 threads copy it
  // 8 rows at a time, 16 lanes take the 16 chunks of one row, so every copy instruction reads whole 256-byte rows; rows
  // past the end of the sequence are zero-filled (source size 0, nothing is read).
  // `between(i)` runs behind copy i: the copy instructions stall at issue once enough of them are in flight, so work that
  // needs no memory is placed between them instead of behind them.
  auto issue_q_copies = [&](int t, int r_local, auto between) {
    const __nv_bfloat16 *q_src = kPrecise ? p.qhat : p.q_raw;
    const int c = r_local & 15;                            // chunk of the row
    const uint32_t q_smem = smem_u32(smem + kOffQ + t * kQTileBytes);
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int rr = i * 8 + (r_local >> 4);                // row of the tile
      const int grow = row0 + t * kRowsPerTile + rr;
      const int gt = div_g(grow), gh = kvh * G + (grow - gt * G);
      const bool in = grow < packed_rows;
      const __nv_bfloat16 *src = in ? q_src + ((size_t)(sq.q_begin + gt) * Hq + gh) * kHeadDim + c * 8 : q_src;
      cp_async16(q_smem + (c >> 3) * kHalfPanel + rr * 128 + (((c & 7) ^ (rr & 7)) << 4), src, in ? 16u : 0u);
      between(i);
    }
  };
  // The one-term variant reads the caller's un-rotated queries, which no kernel in front of this one writes: their
  // copies start at once and fly while the barriers and the tensor memory are set up. Between the copies each thread
  // computes the rotation angles of its first two work items of the rotation pass below (item = (token, chunk c): 8
  // angles; all items up to 32 tokens per M-tile, i.e. from 4 query heads per kv head on): the copy instructions of
  // a thread take ~3,000 cycles to issue (per-CTA trace), and the angles ride along for a few hundred more.
  float cs_pre[2][8], sn_pre[2][8];
  if constexpr (!kPrecise) {
    if (warp < 8 && active[warp >> 2]) {
      const int t = warp >> 2, r_local = (warp & 3) * 32 + lane;
      const int tok_first = div_g(row0 + t * kRowsPerTile);
      issue_q_copies(t, r_local, [&](int i) {
        const int it = r_local + (i >> 3) * kRowsPerTile, e = i & 7;   // angle e of item `it` (see the rotation pass)
        const double pos = (double)(sq.b_base + tok_first + (it >> 3) + sq.rope_off);
        const double turns = pos * p.inv_freq[8 * (it & 7) + e] * 0.15915494309189535;   // angle / 2 pi
        const float r = (float)(turns - rint(turns)) * 6.2831853071795865f;              // in [-pi, pi]
        sn_pre[i >> 3][e] = sin_approx(r);
        cs_pre[i >> 3][e] = cos_approx(r);
      });
    }
  }

  // one thread per barrier (24 of them: a single thread took ~600 cycles over this). Barriers that the four softmax
  // warps of an M-tile arrive at count 4, those completed by tcgen05.commit or a bulk copy count 1.
  constexpr int kNumBarriers = (int)(offsetof(Barriers, tmem_base) / sizeof(uint64_t));
  if (threadIdx.x < kNumBarriers) {
    const uint64_t *b = reinterpret_cast<const uint64_t *>(&bar) + threadIdx.x;
    const bool by_warps = (b >= bar.q_full && b < bar.q_full + 2) || (b >= &bar.p_full[0][0] && b < &bar.p_full[0][0] + 4) ||
                          (b >= bar.y_loaded && b < bar.y_loaded + 2);
    mbar_init(smem_u32(b), by_warps ? 4 : 1);
    if (threadIdx.x == 0) bar.abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(&bar.tmem_base), 512);
    tmem_relinquish();
  }
  grid_dep_launch();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bar.tmem_base;
  grid_dep_wait();   // set-up above touches no global memory; the cache pages come from earlier kernels

  if (warp < 8) {
    // =========================================================== softmax + epilogue warps
    const int t = warp >> 2;                                  // M-tile
    if (active[t]) {
      const int r_local = (warp & 3) * 32 + lane;             // row inside the tile = TMEM lane
      const int row = row0 + t * kRowsPerTile + r_local;      // packed row inside the sequence
      const int tok = div_g(row);
      const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
      const uint32_t s_base = lane_addr + kColS + (uint32_t)(t * 128);
      const uint32_t o_addr = lane_addr + kColO + (uint32_t)(t * 128);

      // ---- Q tile into the swizzled K-major operand layout, by asynchronous 16-byte copies. The tile's 128 threads
      // copy it 8 rows at a time: 16 lanes take the 16 chunks of one row, so every copy instruction reads whole
      // 256-byte rows; rows past the end of the sequence are zero-filled (source size 0, nothing is read).
      // Two-term variant: the rows come rotated from the append kernel's scratch (fp64 rotation, exactly the rounding
      // bf16(RoPE(q)); needed when channels of large magnitude make a one-ulp difference in a rotated query visible).
      // One-term variant: the rows come un-rotated from the caller's buffer and are rotated in place below.
      uint8_t *q_tile = smem + kOffQ + t * kQTileBytes;
      // Rotation pass of the one-term variant, at the streaming position ids (position of token tk of the call = tokens
      // already in the cache + tk), in place. One work item = (token, 16-byte chunk c and its partner c + 8, i.e.
      // channels 8c..8c+7 and 64+8c..): its cos/sin are computed once and serve the G query heads of the token. The
      // angle pos * inv_freq is formed and reduced to a fraction of a turn in fp64 (an fp32 angle would be off by a bf16
      // ulp of the result at positions of a few 10^4); sine, cosine and the rotation run in fp32, whose error (1e-6 of
      // |q|) is three orders below the bf16 rounding that follows: about one rotated element in 10^4 lands on the other
      // side of a rounding boundary than the fp64 rotation would put it.
      const int r_lo = row0 + t * kRowsPerTile;              // first packed row of the tile
      const int r_end = min(r_lo + kRowsPerTile, packed_rows);
      const int tok_lo = div_g(r_lo), tok_hi = div_g(r_end - 1);
      const int n_items = (tok_hi - tok_lo + 1) * 8;
      auto item_angles = [&](int it, float *cs, float *sn) {
        const int tk = tok_lo + (it >> 3), c = it & 7;
        const double pos = (double)(sq.b_base + tk + sq.rope_off);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const double turns = pos * p.inv_freq[8 * c + e] * 0.15915494309189535;   // angle / 2 pi
          const float r = (float)(turns - rint(turns)) * 6.2831853071795865f;       // in [-pi, pi]
          sn[e] = sin_approx(r);
          cs[e] = cos_approx(r);
        }
      };
      // (the angles of this thread's first two items were computed between the query copies, before the set-up)
      {
        if constexpr (kPrecise) issue_q_copies(t, r_local, [](int) {});   // (the one-term variant issued them before the set-up)
        cp_async_wait_all();
      }
      if constexpr (!kPrecise) {
        tile_sync(t);                                          // every thread's copies have landed
        constexpr bool norm = kNorm;
        // (with the normalisation the whole warp walks the items together, for the shuffles: the 8 items of a token sit
        // in 8 neighbouring lanes, all of them in range or none)
        auto rotate_item = [&](int it, const float *cs, const float *sn) {
          unsigned lanes = 0xffffffffu;
          if constexpr (kNorm) {
            lanes = __ballot_sync(0xffffffffu, it < n_items);
            if (it >= n_items) return;
          }
          const int tk = tok_lo + (it >> 3), c = it & 7;
          // all rows of the item are read before the first is written back (the compiler cannot move a shared-memory
        // load over a store of the row before it, and with two warps per scheduler nothing else hides that latency)
        uint4 lo_raw[kMaxGroup], hi_raw[kMaxGroup];
#pragma unroll
        for (int g = 0; g < kMaxGroup; ++g) {
          const int rr = tk * G + g - r_lo;
          if (g < G && rr >= 0 && rr < r_end - r_lo) {
            const uint8_t *ptr = q_tile + rr * 128 + ((c ^ (rr & 7)) << 4);
            lo_raw[g] = *reinterpret_cast<const uint4 *>(ptr);
            hi_raw[g] = *reinterpret_cast<const uint4 *>(ptr + kHalfPanel);
          }
        }
#pragma unroll
        for (int g = 0; g < kMaxGroup; ++g) {
          const int rr = tk * G + g - r_lo;
          const bool valid = g < G && rr >= 0 && rr < r_end - r_lo;
          unsigned row_lanes = 0u;
          if constexpr (kNorm) row_lanes = __ballot_sync(lanes, valid);   // the lanes that take part in this row's shuffles
          if (valid) {
            const uint32_t *lo_w = reinterpret_cast<const uint32_t *>(&lo_raw[g]);
            const uint32_t *hi_w = reinterpret_cast<const uint32_t *>(&hi_raw[g]);
            uint32_t lo_out[4], hi_out[4];
            // optional RMS normalisation of the row over its 128 channels: the 8 lanes of the token add their squares
            float rs = 1.f;
            if constexpr (norm) {
              float ss = 0.f;
#pragma unroll
              for (int e = 0; e < 4; ++e) {
                const float a0 = __uint_as_float(lo_w[e] << 16), a1 = __uint_as_float(lo_w[e] & 0xffff0000u);
                const float b0 = __uint_as_float(hi_w[e] << 16), b1 = __uint_as_float(hi_w[e] & 0xffff0000u);
                ss += a0 * a0 + a1 * a1 + b0 * b0 + b1 * b1;
              }
              ss += __shfl_xor_sync(row_lanes, ss, 1);
              ss += __shfl_xor_sync(row_lanes, ss, 2);
              ss += __shfl_xor_sync(row_lanes, ss, 4);
              rs = rsqrtf(ss * (1.f / kHeadDim) + p.norm_eps);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              // two channels per word: x = channels 8c+2e, 8c+2e+1, y = their partners 64 channels on
              float2 x = make_float2(__uint_as_float(lo_w[e] << 16), __uint_as_float(lo_w[e] & 0xffff0000u));
              float2 y = make_float2(__uint_as_float(hi_w[e] << 16), __uint_as_float(hi_w[e] & 0xffff0000u));
              if constexpr (norm) {
                x.x *= rs * p.norm_q[8 * c + 2 * e];
                x.y *= rs * p.norm_q[8 * c + 2 * e + 1];
                y.x *= rs * p.norm_q[64 + 8 * c + 2 * e];
                y.y *= rs * p.norm_q[64 + 8 * c + 2 * e + 1];
              }
              const float2 c2 = make_float2(cs[2 * e], cs[2 * e + 1]), s2 = make_float2(sn[2 * e], sn[2 * e + 1]);
              const float2 ns2 = make_float2(-sn[2 * e], -sn[2 * e + 1]);
              const float2 lo_r = ffma2(x, c2, fmul2(y, ns2));          // x cos - y sin
              const float2 hi_r = ffma2(y, c2, fmul2(x, s2));           // y cos + x sin
              lo_out[e] = cvt_bf16x2(lo_r.x, lo_r.y);
              hi_out[e] = cvt_bf16x2(hi_r.x, hi_r.y);
            }
            uint8_t *ptr = q_tile + rr * 128 + ((c ^ (rr & 7)) << 4);
            *reinterpret_cast<uint4 *>(ptr) = make_uint4(lo_out[0], lo_out[1], lo_out[2], lo_out[3]);
            *reinterpret_cast<uint4 *>(ptr + kHalfPanel) = make_uint4(hi_out[0], hi_out[1], hi_out[2], hi_out[3]);
          }
        }
        };
        const int span = kNorm ? n_items + r_local : n_items;   // item index bound of this thread's walk
        if (r_local < span) rotate_item(r_local, cs_pre[0], sn_pre[0]);
        if (r_local + kRowsPerTile < span) rotate_item(r_local + kRowsPerTile, cs_pre[1], sn_pre[1]);
        for (int it = r_local + 2 * kRowsPerTile; it < span; it += kRowsPerTile) {
          float cs[8], sn[8];
          item_angles(it, cs, sn);
          rotate_item(it, cs, sn);
        }
      }
      fence_proxy_async_smem();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bar.q_full[t]));

      const float c_log2 = p.scale_log2;
      float m_ref = -INFINITY, l_sum = 0.f;                   // m_ref in scaled (log2) units
      const int nt = n_tiles[t];
      bool ok = true;
      uint8_t *p1_row = smem + kOffP1 + t * kP1Bytes + r_local * 128;   // this row of the shared-memory P (64 keys, 128 bytes)
      for (int j = 0; j < nt && ok; ++j) {
        if (!mbar_wait(smem_u32(&bar.s_full[t]), j & 1, abort_flag, p.status, kDevTimeoutPrefill)) { ok = false; break; }
        tc_fence_after();
        // The 128-key score tile is worked off as two 64-key online-softmax steps (one cache page each). P of the
        // first half goes back into tensor memory (over its own scores) and P V of it runs at once. As soon as the
        // second half's scores are in registers the whole score tile is free, and the tensor core computes the next
        // tile's scores while this thread is still in the second half's exponentials; P of the second half therefore
        // goes to shared memory. In steady state the next scores are complete when this loop comes round.
        const int halves = (2 * j + 1 < n_pages) ? 2 : 1;
        for (int h = 0; h < halves; ++h) {
          const uint32_t s_addr = s_base + (uint32_t)(h * 64);
          float sv[64];
          tmem_ld32(s_addr, &sv[0]);
          tmem_ld32(s_addr + 32, &sv[32]);
          tmem_wait_ld();
          if (h == 1) {
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&bar.y_loaded[t]));
          }

          // visible columns of this row in this page: column c is visible iff c <= lim
          const int pg = pg0 + 2 * j + h;
          const int lim = pg < nA ? sq.a_len - (pg << 6) - 1 : sq.b_base + tok - ((pg - nA) << 6);
          if (lim < 63) {
#pragma unroll
            for (int c = 0; c < 64; ++c) sv[c] = c <= lim ? sv[c] : -INFINITY;
          }
          float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int c = 0; c < 64; c += 8) {
            mx[0] = max3(mx[0], sv[c], sv[c + 1]);
            mx[1] = max3(mx[1], sv[c + 2], sv[c + 3]);
            mx[2] = max3(mx[2], sv[c + 4], sv[c + 5]);
            mx[3] = max3(mx[3], sv[c + 6], sv[c + 7]);
          }
          const float m_tile = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * c_log2;   // scale > 0

          // lazily updated reference maximum
          float alpha = 1.f;
          const bool grow = m_tile > m_ref + kRescaleThreshold;   // also true while m_ref is -inf and a key is visible
          if (grow) {
            alpha = exp2_approx(m_ref - m_tile);               // 0 on the first visible tile
            l_sum *= alpha;
            m_ref = m_tile;
          }
          const float neg_m = m_ref == -INFINITY ? 0.f : -m_ref;
          float acc[4] = {0.f, 0.f, 0.f, 0.f};
          uint32_t packed[32];
          uint32_t packed_lo[kPrecise ? 32 : 1];
#pragma unroll
          for (int c = 0; c < 32; ++c) {
            // The special-function unit does 16 exp2 per clock and SM, exactly the rate at which the tensor core
            // consumes probabilities; a fixed share of the pairs takes a polynomial on the FMA pipe instead.
            float e0, e1;
            const float2 x = ffma2(make_float2(sv[2 * c], sv[2 * c + 1]), make_float2(c_log2, c_log2), make_float2(neg_m, neg_m));
            if ((kPolyPairs >> (c & 7)) & 1u) {
              const float2 e = exp2_poly2(x);
              e0 = e.x;
              e1 = e.y;
            } else {
              e0 = exp2_approx(x.x);
              e1 = exp2_approx(x.y);
            }
            const uint32_t pk = cvt_bf16x2(e0, e1);
            packed[c] = pk;
            if constexpr (kPrecise) {
              // second term: what the first left over; hi + lo carries 16 bits of p, so the row sum takes p itself
              packed_lo[c] = cvt_bf16x2(e0 - __uint_as_float(pk << 16), e1 - __uint_as_float(pk & 0xffff0000u));
              acc[2 * (c & 1)] += e0;
              acc[2 * (c & 1) + 1] += e1;
            } else {
              add_bf16x2(acc[2 * (c & 1)], acc[2 * (c & 1) + 1], pk);   // sum what the tensor core will use
            }
          }
          l_sum += (acc[0] + acc[1]) + (acc[2] + acc[3]);

          // The P V before this one must be complete before O is rescaled, and (second half) before the shared-memory
          // P is overwritten. First half: that is P V (j-1, half 1), whose barrier is in phase j-1 (pending) or j
          // (done) here; second half: P V (j, half 0), barrier in phase j or j+1. Neither parity test can alias.
          const bool rescale = (j > 0 || h > 0) && __any_sync(0xffffffffu, grow);
          if (h == 0) {
            tmem_st32(s_addr, packed);                          // P: 64 keys as 32 packed columns, over the scores
            if constexpr (kPrecise) tmem_st32(s_addr + 32, packed_lo);   // (columns 32-63 of the half were read above)
            if (rescale && !mbar_wait(smem_u32(&bar.p1_free[t]), (j - 1) & 1, abort_flag, p.status, kDevTimeoutPrefill)) { ok = false; break; }
          } else {
            if (j > 0 && !mbar_wait(smem_u32(&bar.p1_free[t]), (j - 1) & 1, abort_flag, p.status, kDevTimeoutPrefill)) { ok = false; break; }
#pragma unroll
            for (int c8 = 0; c8 < 8; ++c8)                      // K-major operand layout, 128-byte swizzle
              *reinterpret_cast<uint4 *>(p1_row + ((c8 ^ (r_local & 7)) << 4)) =
                  make_uint4(packed[c8 * 4], packed[c8 * 4 + 1], packed[c8 * 4 + 2], packed[c8 * 4 + 3]);
            if constexpr (kPrecise) {
              uint8_t *lo_row = smem + kOffP1Lo + t * kP1Bytes + r_local * 128;
#pragma unroll
              for (int c8 = 0; c8 < 8; ++c8)
                *reinterpret_cast<uint4 *>(lo_row + ((c8 ^ (r_local & 7)) << 4)) =
                    make_uint4(packed_lo[c8 * 4], packed_lo[c8 * 4 + 1], packed_lo[c8 * 4 + 2], packed_lo[c8 * 4 + 3]);
            }
            fence_proxy_async_smem();
            if (rescale && !mbar_wait(smem_u32(&bar.pv0_done[t]), j & 1, abort_flag, p.status, kDevTimeoutPrefill)) { ok = false; break; }
          }
          if (rescale) {
            tc_fence_after();
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) {
              float ov[32];
              tmem_ld32(o_addr + c0, ov);
              tmem_wait_ld();
#pragma unroll
              for (int c = 0; c < 32; ++c) ov[c] *= alpha;
              tmem_st32(o_addr + c0, reinterpret_cast<const uint32_t *>(ov));
            }
          }
          tmem_wait_st();
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bar.p_full[t][h]));
        }
      }

      // ---- epilogue: O / l to global memory (write_rows below). All four warps of the tile take the same path whatever
      // happened before.
      const bool fin = ok && mbar_wait(smem_u32(&bar.o_final[t]), 0, abort_flag, p.status, kDevTimeoutPrefill);
      tc_fence_after();
      // The tile's accumulator to the output rows: this thread's row times `mul`; with `other` set, plus the other
      // part's share of the row (workspace, in the layout of write_share below) times `other_mul`. Thread = row: the
      // thread lays 64 channels of its row (256 bytes) into its own line of a staging area and hands the line to the
      // TMA unit as one bulk store, so the rows leave in 256-byte pieces without a transpose between threads, without
      // group barriers and without store instructions of the warps. Lines are 272 bytes apart (the 32 lanes of a
      // 16-byte store then hit every bank group four times, the minimum). The staging area lies over shared memory
      // that no MMA reads any more once the tile's last P V is complete: M-tile 0 its own Q buffer and the first 2 KiB
      // of M-tile 1's (whose last score product was issued in front of this tile's last P V), M-tile 1 the rest of
      // its Q buffer and the start of the first K stage.
      uint8_t *my_line = smem + kOffQ + t * kOutStageTile + r_local * kOutStageLine;
      float *out_row = p.out + ((size_t)(sq.q_begin + tok) * Hq + (size_t)(kvh * G + (row - tok * G))) * kHeadDim;
      const bool store_row = fin && row < packed_rows;
      auto write_rows = [&](float mul, const float4 *other, float other_mul) {
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          float ov[32];
#pragma unroll
          for (int c0 = 0; c0 < 64; c0 += 32) {
            tmem_ld32(o_addr + half * 64 + c0, ov);
            float4 o[8];
            if (other) {
#pragma unroll
              for (int c = 0; c < 8; ++c) o[c] = __ldcg(other + (size_t)((half * 64 + c0) / 4 + c) * kRowsPerTile + r_local);
            }
            tmem_wait_ld();
            if (half == 1 && c0 == 0) bulk_store_wait_read();   // the line is free again once the first half has been read
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
              // (each product is rounded on its own - no fused multiply-add - and the sum commutes: the bits do not
              // depend on which part merges)
              float4 v = make_float4(__fmul_rn(ov[c], mul), __fmul_rn(ov[c + 1], mul), __fmul_rn(ov[c + 2], mul), __fmul_rn(ov[c + 3], mul));
              if (other) {
                const float4 w = o[c >> 2];
                v = make_float4(__fadd_rn(v.x, __fmul_rn(w.x, other_mul)), __fadd_rn(v.y, __fmul_rn(w.y, other_mul)),
                                __fadd_rn(v.z, __fmul_rn(w.z, other_mul)), __fadd_rn(v.w, __fmul_rn(w.w, other_mul)));
              }
              *reinterpret_cast<float4 *>(my_line + (c0 + c) * 4) = v;
            }
          }
          fence_proxy_async_smem();
          if (store_row) bulk_store(out_row + half * 64, smem_u32(my_line), 256);
          bulk_store_commit();
        }
        bulk_store_wait_read();
      };
      // This part's un-normalised share of the tile to the workspace, straight from tensor memory: 16-byte chunk q of
      // row r at [q][r], so that a warp's 32 rows write (and the merging part reads) 512 contiguous bytes.
      auto write_share = [&](float4 *share) {
#pragma unroll
        for (int c0 = 0; c0 < kHeadDim; c0 += 32) {
          float ov[32];
          tmem_ld32(o_addr + c0, ov);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; c += 4)
            share[(size_t)((c0 + c) >> 2) * kRowsPerTile + r_local] = make_float4(ov[c], ov[c + 1], ov[c + 2], ov[c + 3]);
        }
      };
      if (!cut) {
        write_rows(1.f / l_sum, nullptr, 0.f);
      } else {
        // This part's share goes to the workspace; the ticket of (item, M-tile) then tells whether the other part was
        // there first (odd count: tickets are never reset, each launch adds two).
        const size_t mine = (size_t)(split_idx * 2 + part) * kRowsPerCta + t * kRowsPerTile;
        const size_t theirs = (size_t)(split_idx * 2 + (part ^ 1)) * kRowsPerCta + t * kRowsPerTile;
        float4 *share = reinterpret_cast<float4 *>(p.split_o);
        if (fin) {
          p.split_ml[mine + r_local] = make_float2(m_ref, l_sum);
          write_share(share + mine * (kHeadDim / 4));
        }
        __threadfence();
        tile_sync(t);
        // (all four warps of the tile take the same path from here whatever happened before: the group barriers
        // cannot be left waiting; a tile that gave up takes no ticket and writes nothing)
        int *second = reinterpret_cast<int *>(smem + kOffP1 + t * kP1Bytes);   // free: the last P V is complete
        if (r_local == 0) *second = fin ? atomicAdd(p.split_ticket + split_idx * 2 + t, 1) & 1 : 0;
        tile_sync(t);
        if (*second) {
          __threadfence();
          const float2 o_ml = __ldcg(p.split_ml + theirs + r_local);
          // (a part in which this row saw no key has maximum -inf and weight 0; part 0 always sees the first key)
          const float m_all = fmaxf(m_ref, o_ml.x);
          const float w_mine = exp2_approx(m_ref - m_all), w_theirs = exp2_approx(o_ml.x - m_all);
          const float inv = __frcp_rn(__fadd_rn(__fmul_rn(l_sum, w_mine), __fmul_rn(o_ml.y, w_theirs)));
          write_rows(__fmul_rn(w_mine, inv), share + theirs * (kHeadDim / 4), __fmul_rn(w_theirs, inv));
        }
      }
      tc_fence_before();
    }
  } else if (warp == kProducerWarp) {
    // =========================================================== producer
    if (lane == 0) {
      // blocks of the (one or two) pages of key tile j; false if a page id lies outside its pool
      auto tile_pages = [&](int j, const uint8_t *(&src)[2]) -> bool {
        bool pages_ok = true;
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int pg = pg0 + min(2 * j + h, n_pages - 1);
          const bool in_a = pg < nA;
          const int page = in_a ? p.ptab_a[(size_t)sq.slot * p.ptab_stride_a + pg]
                                : p.ptab_b[(size_t)sq.slot * p.ptab_stride_b + (pg - nA)];
          pages_ok = pages_ok && page_ok(page, in_a ? p.n_pages_a : p.n_pages_b, abort_flag, p.status);
          src[h] = (in_a ? p.pool_a : p.pool_b) + ((size_t)page * Hkv + kvh) * kBlockBytes;
        }
        return pages_ok;   // nothing is copied from an address built on a bad page id
      };
      auto pages_of = [&](int j) { return min(2, n_pages - 2 * j); };   // 2, or 1 in an odd tail
      auto wait_k_stage = [&](int j) {
        const uint32_t use = (uint32_t)(j / kKStages);
        return mbar_wait(smem_u32(&bar.k_empty[j % kKStages]), (use & 1u) ^ 1u, abort_flag, p.status, kDevTimeoutPrefill);
      };
      auto wait_v_stage = [&](int j) {
        const uint32_t use = (uint32_t)(j / kVStages);
        return mbar_wait(smem_u32(&bar.v_empty[j % kVStages]), (use & 1u) ^ 1u, abort_flag, p.status, kDevTimeoutPrefill);
      };
      auto copy_k = [&](int j, const uint8_t *const (&src)[2], uint32_t full) {
        const uint32_t dst = smem_u32(smem + kOffK + (j % kKStages) * kKStageBytes);
        for (int h = 0; h < pages_of(j); ++h) {
          // channel half c of page h -> rows 64h .. 64h+63 of the stage's panel c
          bulk_load(dst + h * kPanelBytesK, src[h], kPanelBytesK, full);
          bulk_load(dst + kHalfPanel + h * kPanelBytesK, src[h] + kPanelBytesK, kPanelBytesK, full);
        }
      };
      auto copy_v = [&](int j, const uint8_t *const (&src)[2], uint32_t full) {
        const uint32_t dst = smem_u32(smem + kOffV + (j % kVStages) * kVStageBytes);
        for (int h = 0; h < pages_of(j); ++h) bulk_load(dst + h * kHalfPanel, src[h] + kKeyBytes, kHalfPanel, full);
      };
      if constexpr (kPrecise) {
        // one K stage: K(j) and V(j) of a tile, each on its own barrier
        for (int j = 0; j < n_max; ++j) {
          const uint8_t *src[2];
          if (!tile_pages(j, src)) break;
          if (!wait_k_stage(j)) break;
          mbar_arrive_expect_tx(smem_u32(&bar.k_full[j % kKStages]), (uint32_t)(pages_of(j) * kKeyBytes));
          copy_k(j, src, smem_u32(&bar.k_full[j % kKStages]));
          if (!wait_v_stage(j)) break;
          mbar_arrive_expect_tx(smem_u32(&bar.v_full[j % kVStages]), (uint32_t)(pages_of(j) * kHalfPanel));
          copy_v(j, src, smem_u32(&bar.v_full[j % kVStages]));
        }
      } else {
        // K(0) on its own barrier; then V(j) and K(j+1) together on v_full[j % 2]: the issuer needs both at the same
        // point of tile j (P V (j, 0), then Q K^T (j+1)), and every wait it does not have to make is ~400 cycles.
        const uint8_t *cur[2], *nxt[2];
        bool ok = n_max > 0 && tile_pages(0, cur) && wait_k_stage(0);
        if (ok) {
          mbar_arrive_expect_tx(smem_u32(&bar.k_full[0]), (uint32_t)(pages_of(0) * kKeyBytes));
          copy_k(0, cur, smem_u32(&bar.k_full[0]));
        }
        for (int j = 0; ok && j < n_max; ++j) {
          const bool more = j + 1 < n_max;
          if (more && !tile_pages(j + 1, nxt)) break;
          if (!wait_v_stage(j) || (more && !wait_k_stage(j + 1))) break;
          const uint32_t full = smem_u32(&bar.v_full[j % kVStages]);
          mbar_arrive_expect_tx(full, (uint32_t)(pages_of(j) * kHalfPanel + (more ? pages_of(j + 1) * kKeyBytes : 0)));
          copy_v(j, cur, full);
          if (more) copy_k(j + 1, nxt, full);
          cur[0] = nxt[0];
          cur[1] = nxt[1];
        }
      }
    }
  } else {
    // =========================================================== MMA issuer
    const uint32_t issue = elect_one();
    const uint32_t q_addr = smem_u32(smem + kOffQ), k_addr = smem_u32(smem + kOffK), v_addr = smem_u32(smem + kOffV);
    bool ok = true;

    auto issue_qk = [&](int t, int j) {
      // S[t] = Q_t (128 x 128 channels) . K_j^T: 8 steps of 16 channels; N = 128 keys (64 in an odd tail)
      const uint32_t idesc = (2 * j + 1 < n_pages) ? make_idesc(128) : make_idesc(64);
      const uint32_t d = tmem + kColS + (uint32_t)(t * 128);
      const uint64_t qd = make_desc(q_addr + t * kQTileBytes), kd = make_desc(k_addr + (j % kKStages) * kKStageBytes);
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        const uint64_t off = (uint64_t)(((ks >> 2) * kHalfPanel + (ks & 3) * 32) >> 4);
        tc_mma_ss(d, qd + off, kd + off, idesc, ks > 0, issue);
      }
      tc_commit(smem_u32(&bar.s_full[t]), issue);
    };
    const uint32_t p1_addr = smem_u32(smem + kOffP1);
    auto issue_pv = [&](int t, int j, int h) {
      // O[t] += P_t (128 x 64 keys of page 2j+h) . V: 4 steps of 16 keys, the V^T panel is K-major.
      // P of half 0 is read from tensor memory (the first 32 score columns), P of half 1 from shared memory.
      constexpr uint32_t idesc = make_idesc(128);
      const uint32_t d = tmem + kColO + (uint32_t)(t * 128);
      const uint64_t vd = make_desc(v_addr + (j % kVStages) * kVStageBytes + h * kHalfPanel);
      if (h == 0) {
        const uint32_t pa = tmem + kColS + (uint32_t)(t * 128);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          tc_mma_ts(d, pa + ks * 8, vd + (uint64_t)((ks * 32) >> 4), idesc, (j > 0 || ks > 0) ? 1u : 0u, issue);
        if constexpr (kPrecise) {
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            tc_mma_ts(d, pa + 32 + ks * 8, vd + (uint64_t)((ks * 32) >> 4), idesc, 1u, issue);
        }
      } else {
        const uint64_t pd = make_desc(p1_addr + t * kP1Bytes);
#pragma unroll
        for (int ks = 0; ks < 4; ++ks)
          tc_mma_ss(d, pd + (uint64_t)((ks * 32) >> 4), vd + (uint64_t)((ks * 32) >> 4), idesc, 1u, issue);
        if constexpr (kPrecise) {
          const uint64_t pl = make_desc(smem_u32(smem + kOffP1Lo) + t * kP1Bytes);
#pragma unroll
          for (int ks = 0; ks < 4; ++ks)
            tc_mma_ss(d, pl + (uint64_t)((ks * 32) >> 4), vd + (uint64_t)((ks * 32) >> 4), idesc, 1u, issue);
        }
      }
    };

    // first score tiles: each M-tile's as soon as its own Q rows and the first key tile have landed
    bool have_k0 = false;
    for (int t = 0; t < 2 && ok; ++t) {
      if (!active[t]) continue;
      ok = mbar_wait(smem_u32(&bar.q_full[t]), 0, abort_flag, p.status, kDevTimeoutPrefill);
      if (ok && !have_k0) {
        ok = mbar_wait(smem_u32(&bar.k_full[0]), 0, abort_flag, p.status, kDevTimeoutPrefill);
        have_k0 = true;
      }
      if (!ok) break;
      tc_fence_after();
      issue_qk(t, 0);
    }
    if (ok) tc_commit(smem_u32(&bar.k_empty[0]), issue);
    // Per key tile j, in the order in which the events arrive when M-tile 1 runs a little behind M-tile 0:
    //   for each M-tile: P of half 0 published -> P V (j, 0); all scores of the tile consumed -> Q K^T (j+1)
    //                    (issued after P V (j, 0), which reads the same columns);
    //   for each M-tile: P of half 1 published -> P V (j, 1).
    for (int j = 0; j < n_max && ok; ++j) {
      const int halves = (2 * j + 1 < n_pages) ? 2 : 1;
      bool have_k = false;
      for (int t = 0; t < 2 && ok; ++t) {
        if (j >= n_tiles[t]) continue;
        // With two key halves one wait serves P V (j, 0) and Q K^T (j+1): every softmax warp arrives at y_loaded
        // behind its arrival at p_full[0] (program order, both releases), so a complete y_loaded phase means that P of
        // half 0 is published as well. Every wait of this warp costs ~400 cycles while MMAs run (its polls are
        // shared-memory accesses in competition with the operand reads), and the issuer's chain of waits was the
        // longest path through a key tile (per-CTA trace: nine steps of 370-400 cycles).
        ok = halves == 2 ? mbar_wait(smem_u32(&bar.y_loaded[t]), (uint32_t)j & 1u, abort_flag, p.status, kDevTimeoutPrefill)
                         : mbar_wait(smem_u32(&bar.p_full[t][0]), (uint32_t)j & 1u, abort_flag, p.status, kDevTimeoutPrefill);
        if (ok && t == (n_tiles[0] > j ? 0 : 1))
          ok = mbar_wait(smem_u32(&bar.v_full[j % kVStages]), (uint32_t)(j / kVStages) & 1u, abort_flag, p.status, kDevTimeoutPrefill);
        if (!ok) break;
        tc_fence_after();
        issue_pv(t, j, 0);
        tc_commit(smem_u32(&bar.pv0_done[t]), issue);
        if (halves == 1 && j == n_tiles[t] - 1) tc_commit(smem_u32(&bar.o_final[t]), issue);
        if (halves == 2) {
          if (j + 1 < n_tiles[t]) {
            if (kPrecise && !have_k) {   // (one-term variant: K(j+1) came with V(j), on the barrier waited for above)
              ok = mbar_wait(smem_u32(&bar.k_full[(j + 1) % kKStages]), (uint32_t)((j + 1) / kKStages) & 1u, abort_flag, p.status, kDevTimeoutPrefill);
              have_k = true;
              if (!ok) break;
            }
            tc_fence_after();
            issue_qk(t, j + 1);
          }
        }
      }
      if (ok && halves == 2) {
        if (j + 1 < n_max) tc_commit(smem_u32(&bar.k_empty[(j + 1) % kKStages]), issue);
        for (int t = 0; t < 2 && ok; ++t) {
          if (j >= n_tiles[t]) continue;
          ok = mbar_wait(smem_u32(&bar.p_full[t][1]), (uint32_t)j & 1u, abort_flag, p.status, kDevTimeoutPrefill);
          if (!ok) break;
          tc_fence_after();
          issue_pv(t, j, 1);
          tc_commit(smem_u32(&bar.p1_free[t]), issue);
          if (j == n_tiles[t] - 1) tc_commit(smem_u32(&bar.o_final[t]), issue);
        }
      }
      // V(j) is free once every P V that reads it is complete
      if (ok) tc_commit(smem_u32(&bar.v_empty[j % kVStages]), issue);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

cudaError_t init_attn_tc_kernels() {
  cudaError_t e = cudaFuncSetAttribute(st_k_attn_tc<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes + 1024);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(st_k_attn_tc<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes + 1024);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(st_k_attn_tc<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes + 1024);
}

int attn_tc_rows_per_cta() { return kRowsPerCta; }

cudaError_t launch_attn_tc(AttnParams &p, bool precise, int num_sms, cudaStream_t stream, int *n_launches, cudaEvent_t t0,
                           cudaEvent_t t1) {
  *n_launches = 0;
  int total = 0;
  for (int i = 0; i < p.n_seq; ++i) {
    p.seq[i].work_begin = total;
    total += p.n_kv_heads * ((p.seq[i].n_rows * p.group + kRowsPerCta - 1) / kRowsPerCta);
  }
  if (total == 0) return cudaSuccess;
  p.total_work = total;
  // One CTA per SM at a time: the items run in waves of num_sms. When the last wave would fill at most half of the
  // SMs, its items are cut in two by keys (two CTAs each), so that it takes about half as long.
  const int tail = total % num_sms;
  p.n_split = (p.split_o != nullptr && tail > 0 && 2 * tail <= num_sms) ? std::min(tail, kMaxSplitItems) : 0;
  if (p.n_split > 0) {   // ... unless none of them is long enough to be cut (the kernel decides per item, by the same count)
    int longest = 0;
    for (int i = p.n_seq - 1; i >= 0; --i) {
      const AttnSeq &sq = p.seq[i];
      if (sq.n_rows > 0) longest = std::max(longest, ((sq.a_len + 63) >> 6) + ((sq.b_base + sq.n_rows - 1) >> 6) + 1);
      if (sq.work_begin <= total - p.n_split) break;
    }
    if (longest < kMinCutPages) p.n_split = 0;
  }
  p.n_cta = total + p.n_split;
  if (t0) cudaEventRecord(t0, stream);
  // (the two-term variant takes queries that the append kernel has normalised and rotated)
  auto kernel = precise ? st_k_attn_tc<true, false> : p.norm_q != nullptr ? st_k_attn_tc<false, true> : st_k_attn_tc<false, false>;
  cudaError_t e = launch_dependent(kernel, dim3(p.n_cta), dim3(kThreads), kSmemBytes + 1024, stream, p);
  if (e != cudaSuccess) return e;
  if (t1) cudaEventRecord(t1, stream);
  *n_launches = 1;
  return cudaSuccess;
}

}  // namespace st
