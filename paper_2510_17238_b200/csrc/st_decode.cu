// Dual-cache decode (one new reasoning token per sequence) with split-K over both caches.
//
// What it computes (Section 3.3 / Algorithm 1, decode loop): for every listed sequence and q head,
//   O = softmax( scale * q^ . [K_src[0:vis] ; K_rsn[0:r+1]] ) [V_src[0:vis] ; V_rsn[0:r+1]],
// i.e. attention over the visible source prefix and the reasoning cache including the new token.
// The paper merges the two caches into one before decoding and splits them afterwards; here the
// kernel simply walks two page tables, so "merge" and "split" cost nothing.
//
// Shape of the kernel. The work is HBM-bound (every K/V byte is read once, ~G flop per byte).
// The key tiles (one page = 64 tokens = one 32 KiB block per kv head) of all (sequence, kv head)
// pairs form one global list; CTA c takes the contiguous slice [c*L, (c+1)*L) of it, whatever
// pair boundaries it crosses, so all CTAs stream the same number of bytes. A producer warp feeds a
// shared-memory ring with one 32 KiB bulk copy (TMA, no tensor map) per tile; a tile is worked off by four
// consumer warps, each of which owns 16 of its 64 keys and keeps an independent online-softmax state, so the
// only per-tile synchronisation is the ring's full/empty mbarriers. There are two such groups of four warps;
// consecutive tiles of the walk go to them alternately, so that two tiles are in work at a time (the chains of
// ldmatrix and mma.sync of one tile hide behind the other's: 152.7 -> 151.8 us per launch on the benchmark
// workload, 141.2 -> 139.2 us on the long-context one). The products run on
// mma.sync.m16n8k16 in transposed form:
//     S^T[16 keys x 8 heads]   = K[16 x 128]   . Q^T[128 x 8]      (A = K via ldmatrix)
//     O^T[128 ch  x 8 heads]  += V^T[128 x 16] . P^T[16 x 8]       (A = V^T via ldmatrix)
// so the padded dimension is the 8-wide head axis (G <= 8 q heads share a kv head), not M.
// P^T goes from accumulator to B-operand layout with movmatrix, split into bf16 hi + lo parts
// so that the rounding of P does not limit accuracy. Per pair slice the four warps combine their
// states (all eight warps') through shared memory (log-sum-exp merge); a slice that covers its pair completely
// writes the final rows, otherwise it writes an (m, l, O) partial that a second small kernel
// merges across CTAs. All waits are bounded.
//
// The step's append (Algorithm 1: the new reasoning token enters the reasoning cache before it is attended to)
// runs inside this kernel when the call hands over the un-rotated q/k/v (q_raw != nullptr): a sixth warp walks
// the CTA's pairs ahead of the consumers, rotates the pair's G query rows at the token's position into shared
// memory (every CTA that holds a slice of the pair does this for itself), and -- in the one CTA that holds the
// pair's last tile -- rotates the new key and writes key and value into the cache page before the producer
// fetches that tile (release by fence + a shared-memory counter, then a proxy fence before the bulk copy). The
// rotation is the append kernel's (fp64, one rounding to bf16); cos and sin come from two fp64 tables
// (positions 1024 a + b, one angle addition) because a sincos per channel and pair was far too slow for one warp.
// A decode step is then two kernels (this one and the merge) instead of three.
//
// Direction of the walk. Consecutive decode steps read the same caches (plus one token), more than L2 holds; what is
// left in L2 after a step is the end of every CTA's slice. With `reverse` set every role walks the CTA's slice from
// its last tile to its first (the pairs in reverse order, the tiles of a pair from the one that holds the new token
// down), so a step that runs in the opposite direction of the one before it starts on the ~50 MB that are still in
// L2. The host alternates the direction step by step. A plain streaming probe (148 CTAs, the same bulk copies and
// ring) measured 37.0 -> 29.0 us per pass over 242 MB and 136.3 -> 129.6 us over 970 MB.
#include "st_internal.h"

namespace st {

namespace {

constexpr int kStages = 4;
constexpr int kTileWarps = 4;                 // warps that share a tile: 16 of its 64 keys each
constexpr int kConsumerGroups = 2;            // groups of kTileWarps warps; consecutive tiles of the walk alternate between them
constexpr int kConsumerWarps = kTileWarps * kConsumerGroups;
constexpr int kThreads = (kConsumerWarps + 2) * 32;   // two consumer groups, producer, append warp
// Per warp: o[8][128] with the head rows kMergeRow floats apart (132: the four lanes of a quad write heads 2 tq, i.e.
// rows 264 tq floats = 8 tq banks apart, and the stores are conflict-free; with rows of 128 they were 4-way conflicts),
// then m[8], l[8].
constexpr int kMergeRow = 132;
constexpr int kMergeM = 8 * kMergeRow, kMergeL = kMergeM + 8;
constexpr int kMergeFloats = kMergeL + 8;

struct __align__(1024) DecodeSmem {
  uint8_t ring[kStages][kBlockBytes];
  float merge[kConsumerWarps][kMergeFloats];
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t group_bar;
  uint64_t q_ready[2];   // fused append: rotated queries of a pair are in qhat[slot]
  uint64_t q_free[2];    // fused append: the consumers have taken them
  __nv_bfloat16 qhat[2][8][kHeadDim];
  int pairs_prepared;    // fused append: pairs of this CTA whose queries and new token are in place (monotonic)
  int abort_flag;
};

// The part of one (sequence, kv head) pair's tiles that lies inside a CTA's slice [tile_begin, tile_end) of the global
// tile list, and the walk of a CTA over its pairs. Tile t of a pair: [0, nA) source pages, [nA, nA + nB) reasoning
// pages; the last one holds the step's token.
struct PairSlice {
  int seq;       // index into params.seq
  int kvh;
  int nA, nB;
  int pair_first;  // global index of the pair's tile 0
  int t_lo, t_hi;  // tiles t_lo .. t_hi (inclusive) of the pair are this CTA's

  __device__ __forceinline__ int tiles() const { return t_hi - t_lo + 1; }
  __device__ __forceinline__ bool owns_token_tile() const { return t_hi == nA + nB - 1; }
  // k-th tile of the slice in walk order. Forwards: ascending. Backwards: descending, except that the tile with the
  // step's token comes last (it can only be fetched once the append warp has written the token, which must not hold
  // up the start of the CTA's walk).
  __device__ __forceinline__ int tile_at(int k, bool rev) const {
    if (!rev) return t_lo + k;
    if (!owns_token_tile()) return t_hi - k;
    return k == t_hi - t_lo ? t_hi : t_hi - 1 - k;
  }
  __device__ __forceinline__ void load(const AttnParams &p, int tile_begin, int tile_end) {
    nA = (p.seq[seq].a_len + 63) >> 6;
    nB = (p.seq[seq].b_base + 1 + 63) >> 6;
    pair_first = p.seq[seq].work_begin * p.n_kv_heads + kvh * (nA + nB);
    t_lo = max(0, tile_begin - pair_first);
    t_hi = min(nA + nB, tile_end - pair_first) - 1;
  }
  // first pair of the walk: the one that holds tile_begin (forwards) or tile_end - 1 (backwards)
  __device__ __forceinline__ void first(const AttnParams &p, int tile_begin, int tile_end, bool rev) {
    const int Hkv = p.n_kv_heads, gt = rev ? tile_end - 1 : tile_begin;
    seq = last_not_above(p.n_seq, gt, [&](int i) { return p.seq[i].work_begin * Hkv; });
    const int nt = ((p.seq[seq].a_len + 63) >> 6) + ((p.seq[seq].b_base + 1 + 63) >> 6);
    kvh = (gt - p.seq[seq].work_begin * Hkv) / nt;
    load(p, tile_begin, tile_end);
  }
  // next pair of the walk; false when the walk has left the CTA's slice
  __device__ __forceinline__ bool next(const AttnParams &p, int tile_begin, int tile_end, bool rev) {
    if (rev) {
      if (pair_first <= tile_begin) return false;
      if (kvh-- == 0) { kvh = p.n_kv_heads - 1; --seq; }
    } else {
      if (pair_first + nA + nB >= tile_end) return false;
      if (++kvh == p.n_kv_heads) { kvh = 0; ++seq; }
    }
    load(p, tile_begin, tile_end);
    return true;
  }
};

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// Bounded wait until a monotonic shared-memory counter exceeds `below` (same time limit and abort protocol as mbar_wait).
__device__ __forceinline__ bool wait_counter_above(const int *counter, int below, volatile int *abort_flag, int32_t *status,
                                                   int code) {
  uint64_t t0 = 0;
  for (uint32_t polls = 1;; ++polls) {
    if (*(const volatile int *)counter > below) return true;
    if ((polls & 255u) == 0u) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      if (now - t0 > kWaitLimitNs) {
        *abort_flag = 1;
        atomicExch(status, code);
        return false;
      }
    }
  }
}

}  // namespace

__global__ void __launch_bounds__(kThreads, 1) st_k_decode(const __grid_constant__ AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  DecodeSmem &sm = *reinterpret_cast<DecodeSmem *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int *abort_flag = &sm.abort_flag;

  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(smem_u32(&sm.full[i]), 1);
      mbar_init(smem_u32(&sm.empty[i]), kTileWarps);
    }
    mbar_init(smem_u32(&sm.group_bar), kConsumerWarps);
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&sm.q_ready[i]), 1);
      mbar_init(smem_u32(&sm.q_free[i]), kConsumerWarps);
    }
    sm.pairs_prepared = 0;
    sm.abort_flag = 0;
    mbar_fence_init();
  }
  grid_dep_launch();
  __syncthreads();
  grid_dep_wait();

  const int tile_begin = blockIdx.x * p.work_per_cta;
  const int tile_end = min(tile_begin + p.work_per_cta, p.total_work);
  const int Hkv = p.n_kv_heads;

  const bool fused = p.q_raw != nullptr;
  const bool rev = p.reverse != 0;
  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------ producer
    if (lane == 0 && tile_begin < tile_end) {
      PairSlice ps;
      ps.first(p, tile_begin, tile_end, rev);
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int ord = 0; ok; ++ord) {   // ord: ordinal of the pair within this CTA's walk
        const AttnSeq &sq = p.seq[ps.seq];
        for (int k = 0; k < ps.tiles(); ++k) {
          const int t = ps.tile_at(k, rev);
          const bool in_a = t < ps.nA;
          const bool token_tile = t == ps.nA + ps.nB - 1;       // the tile that holds the step's token
          const int page = in_a ? p.ptab_a[(size_t)sq.slot * p.ptab_stride_a + t]
                                : p.ptab_b[(size_t)sq.slot * p.ptab_stride_b + (t - ps.nA)];
          if (!page_ok(page, in_a ? p.n_pages_a : p.n_pages_b, abort_flag, p.status)) { ok = false; break; }
          const uint8_t *src = (in_a ? p.pool_a : p.pool_b) + ((size_t)page * Hkv + ps.kvh) * kBlockBytes;
          if (!mbar_wait(smem_u32(&sm.empty[stage]), phase ^ 1u, abort_flag, p.status, kDevTimeoutDecode)) { ok = false; break; }
          if (fused && token_tile) {
            // the tile that holds the step's token is fetched after the append warp has written the token
            if (!wait_counter_above(&sm.pairs_prepared, ord, abort_flag, p.status, kDevTimeoutDecode)) { ok = false; break; }
            fence_proxy_async_all();
          }
          mbar_arrive_expect_tx(smem_u32(&sm.full[stage]), kBlockBytes);
          bulk_load(smem_u32(sm.ring[stage]), src, kBlockBytes, smem_u32(&sm.full[stage]));
          if (++stage == kStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok || !ps.next(p, tile_begin, tile_end, rev)) break;
      }
    }
  } else if (warp == kConsumerWarps + 1) {
    // ------------------------------------------------------------------ append warp (only with the append fused in)
    // Walks the pairs of this CTA in order, up to two ahead of the consumers. For every pair it rotates the G
    // query rows of the step at the new token's position into shared memory; if this CTA holds the pair's last tile
    // it also rotates the new key and writes it and the new value into the cache page (one CTA per pair does).
    // Arithmetic as in the append kernel (fp64 rotation, one rounding to bf16); cos and sin of the angle come from
    // two fp64 tables by one angle addition instead of a sincos per channel.
    if (fused && tile_begin < tile_end) {
      PairSlice ps;
      ps.first(p, tile_begin, tile_end, rev);
      const int G = p.group;
      for (int n = 0;; ++n) {
        const AttnSeq &sq = p.seq[ps.seq];
        const int kvh = ps.kvh;
        const bool owns_last = ps.owns_token_tile();
        const int slot = n & 1, use = n >> 1;
        if (use > 0) {                              // the consumers must have taken the slot's previous contents
          int good = 1;
          if (lane == 0) good = mbar_wait(smem_u32(&sm.q_free[slot]), (uint32_t)(use - 1) & 1u, abort_flag, p.status, kDevTimeoutDecode);
          if (!__shfl_sync(0xffffffffu, good, 0)) break;
        }
        const int pos = sq.b_base;                  // index of the step's token in the reasoning cache
        const int rpos = pos + sq.rope_off;         // its position id
        // every global load of the pair is issued before the first value is used: one round trip, not five
        double2 hi[2], lo[2];
        __nv_bfloat16 qx[8][2], qy[8][2], kx[2], ky[2], vv[4];
        int page = 0;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          hi[i] = p.rope_hi[(size_t)(rpos / kRopeLoSteps) * 64 + lane + 32 * i];
          lo[i] = p.rope_lo[(size_t)(rpos % kRopeLoSteps) * 64 + lane + 32 * i];
        }
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          if (g < G) {
            const __nv_bfloat16 *src = p.q_raw + ((size_t)sq.q_begin * p.n_q_heads + (size_t)kvh * G + g) * kHeadDim;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
              qx[g][i] = src[lane + 32 * i];
              qy[g][i] = src[lane + 32 * i + 64];
            }
          }
        }
        if (owns_last) {
          page = p.ptab_b[(size_t)sq.slot * p.ptab_stride_b + (pos >> 6)];
          const __nv_bfloat16 *ksrc = p.k_raw + ((size_t)sq.q_begin * Hkv + kvh) * kHeadDim;
          const __nv_bfloat16 *vsrc = p.v_raw + ((size_t)sq.q_begin * Hkv + kvh) * kHeadDim;
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            kx[i] = ksrc[lane + 32 * i];
            ky[i] = ksrc[lane + 32 * i + 64];
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) vv[i] = vsrc[lane + 32 * i];
        }
        // optional RMS normalisation of the query rows and of the new key over their 128 channels (fp64, as in the
        // append kernel): every lane holds 4 channels of a row, the warp adds the squares
        const bool norm = p.norm_k != nullptr;
        double wq[2][2] = {{1.0, 1.0}, {1.0, 1.0}}, wk[2][2] = {{1.0, 1.0}, {1.0, 1.0}};   // [i][low/high half]
        if (norm) {
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            wq[i][0] = (double)p.norm_q[lane + 32 * i];
            wq[i][1] = (double)p.norm_q[lane + 32 * i + 64];
            wk[i][0] = (double)p.norm_k[lane + 32 * i];
            wk[i][1] = (double)p.norm_k[lane + 32 * i + 64];
          }
        }
        auto row_scale = [&](const __nv_bfloat16 (&x)[2], const __nv_bfloat16 (&y)[2]) -> double {
          double ss = 0.0;
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const double a = (double)__bfloat162float(x[i]), b = (double)__bfloat162float(y[i]);
            ss += a * a + b * b;
          }
#pragma unroll
          for (int off = 1; off < 32; off <<= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
          return 1.0 / sqrt(ss * (1.0 / kHeadDim) + (double)p.norm_eps);
        };
        double cs[2], sn[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {              // angle addition from the two rotation tables
          cs[i] = hi[i].x * lo[i].x - hi[i].y * lo[i].y;
          sn[i] = hi[i].y * lo[i].x + hi[i].x * lo[i].y;
        }
#pragma unroll
        for (int g = 0; g < 8; ++g) {
          if (g < G) {
            const double rs = norm ? row_scale(qx[g], qy[g]) : 1.0;
#pragma unroll
            for (int i = 0; i < 2; ++i) {
              const int c = lane + 32 * i;
              double x = (double)__bfloat162float(qx[g][i]), y = (double)__bfloat162float(qy[g][i]);
              if (norm) {
                x = x * rs * wq[i][0];
                y = y * rs * wq[i][1];
              }
              sm.qhat[slot][g][c] = __double2bfloat16(x * cs[i] - y * sn[i]);
              sm.qhat[slot][g][c + 64] = __double2bfloat16(y * cs[i] + x * sn[i]);
            }
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sm.q_ready[slot]));     // to the consumers: the pair's queries are in place
        if (owns_last && !page_ok(page, p.n_pages_b, abort_flag, p.status)) break;   // (warp-uniform) nothing is written
        if (owns_last) {
          uint8_t *blk = const_cast<uint8_t *>(p.pool_b) + ((size_t)page * Hkv + kvh) * kBlockBytes;
          const int tok = pos & 63;
          const double rs = norm ? row_scale(kx, ky) : 1.0;
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const int c = lane + 32 * i;
            double x = (double)__bfloat162float(kx[i]), y = (double)__bfloat162float(ky[i]);
            if (norm) {
              x = x * rs * wk[i][0];
              y = y * rs * wk[i][1];
            }
            *reinterpret_cast<__nv_bfloat16 *>(blk + k_byte_offset(tok, c)) = __double2bfloat16(x * cs[i] - y * sn[i]);
            *reinterpret_cast<__nv_bfloat16 *>(blk + k_byte_offset(tok, c + 64)) = __double2bfloat16(y * cs[i] + x * sn[i]);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i)
            *reinterpret_cast<__nv_bfloat16 *>(blk + vt_byte_offset(tok, lane + 32 * i)) = vv[i];
          __threadfence();                          // the new token is in the page before the producer is told so
        }
        __syncwarp();
        if (lane == 0) {
          fence_proxy_async_all();
          *(volatile int *)&sm.pairs_prepared = n + 1;               // to the producer: the pair's new token is in the cache
        }
        if (!ps.next(p, tile_begin, tile_end, rev)) break;
      }
    }
  } else if (warp < kConsumerWarps && tile_begin < tile_end) {
    // ------------------------------------------------------------------ consumers
    const int g = lane >> 2, tq = lane & 3;
    const int G = p.group;
    PairSlice ps;
    ps.first(p, tile_begin, tile_end, rev);
    uint32_t group_phase = 0;
    bool ok = true;
    int ord = 0;   // ordinal of the slice (pair) within this CTA's walk, as counted by the producer warp
    const int wq = warp % kTileWarps;    // this warp's quarter of a tile's keys
    const int grp = warp / kTileWarps;   // its group: it works on the tiles whose ring index is congruent to grp
    int ring_index = 0;                  // tiles of the walk in front of the current slice

    for (bool more = true; more && ok; more = ps.next(p, tile_begin, tile_end, rev)) {
      // ---- one slice of one (sequence, kv head) pair
      const AttnSeq sq = p.seq[ps.seq];
      const int kvh = ps.kvh, slice_seq = ps.seq;
      const int pair_tiles = ps.nA + ps.nB;
      const int pair_first = ps.pair_first;                   // global index of the pair's first tile

      // Q^T fragments of the pair: column n = g is q head kvh*G + g (zero beyond the group)
      uint32_t bq[8][2];
      if (fused) {
        // rotated by the producer warp into shared memory
        if (!mbar_wait(smem_u32(&sm.q_ready[ord & 1]), (uint32_t)(ord >> 1) & 1u, abort_flag, p.status, kDevTimeoutDecode)) break;
        const uint32_t *qrow = reinterpret_cast<const uint32_t *>(sm.qhat[ord & 1][g < G ? g : 0]);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          bq[ks][0] = g < G ? qrow[ks * 8 + tq] : 0u;
          bq[ks][1] = g < G ? qrow[ks * 8 + 4 + tq] : 0u;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sm.q_free[ord & 1]));
        ++ord;
      } else {
        const uint32_t *qrow = reinterpret_cast<const uint32_t *>(
            p.qhat + ((size_t)sq.q_begin * p.n_q_heads + (size_t)kvh * G + (g < G ? g : 0)) * kHeadDim);
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
          bq[ks][0] = g < G ? qrow[ks * 8 + tq] : 0u;
          bq[ks][1] = g < G ? qrow[ks * 8 + 4 + tq] : 0u;
        }
      }
      float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
      float o[8][4];
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) o[mt][0] = o[mt][1] = o[mt][2] = o[mt][3] = 0.f;

      for (int k = 0; k < ps.tiles(); ++k) {
        const int ri = ring_index + k;
        if (ri % kConsumerGroups != grp) continue;            // the other group's tile
        const int stage = ri % kStages;
        const uint32_t phase = (uint32_t)(ri / kStages) & 1u;
        const int t = ps.tile_at(k, rev);
        if (!mbar_wait(smem_u32(&sm.full[stage]), phase, abort_flag, p.status, kDevTimeoutDecode)) { ok = false; break; }
        const uint32_t sb = smem_u32(sm.ring[stage]);
        // valid keys in this tile
        const bool in_a = t < ps.nA;
        const int range_len = in_a ? sq.a_len : sq.b_base + 1;
        const int valid = min(64, range_len - ((in_a ? t : t - ps.nA) << 6));

        // S^T = K . Q^T for this warp's 16 keys
        // (two accumulators over alternate channel steps: a chain of four dependent MMAs instead of eight)
        float c[4] = {0.f, 0.f, 0.f, 0.f};
        {
          float c_odd[4] = {0.f, 0.f, 0.f, 0.f};
          const int key = wq * 16 + (lane & 7) + ((lane >> 3) & 1) * 8;
#pragma unroll
          for (int ks = 0; ks < 8; ++ks) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(sb + k_byte_offset(key, (2 * ks + (lane >> 4)) * 8), a0, a1, a2, a3);
            if (ks & 1) mma_bf16(c_odd, a0, a1, a2, a3, bq[ks][0], bq[ks][1]);
            else mma_bf16(c, a0, a1, a2, a3, bq[ks][0], bq[ks][1]);
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) c[i] += c_odd[i];
        }
        const int key0 = wq * 16 + g;
        const float NEG = -INFINITY;
        c[0] = key0 < valid ? c[0] * p.scale_log2 : NEG;
        c[1] = key0 < valid ? c[1] * p.scale_log2 : NEG;
        c[2] = key0 + 8 < valid ? c[2] * p.scale_log2 : NEG;
        c[3] = key0 + 8 < valid ? c[3] * p.scale_log2 : NEG;

        float mx0 = fmaxf(c[0], c[2]), mx1 = fmaxf(c[1], c[3]);
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
          mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
        }
        const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
        const float ms0 = mn0 == NEG ? 0.f : mn0, ms1 = mn1 == NEG ? 0.f : mn1;
        const float al0 = exp2_approx(m0 - ms0), al1 = exp2_approx(m1 - ms1);
        m0 = mn0;
        m1 = mn1;
        const float p0 = exp2_approx(c[0] - ms0), p1 = exp2_approx(c[1] - ms1);
        const float p2 = exp2_approx(c[2] - ms0), p3 = exp2_approx(c[3] - ms1);
        l0 = l0 * al0 + p0 + p2;   // per-thread share; reduced over the quad column at the end
        l1 = l1 * al1 + p1 + p3;
        if (__any_sync(0xffffffffu, al0 != 1.f || al1 != 1.f)) {
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) {
            o[mt][0] *= al0; o[mt][1] *= al1; o[mt][2] *= al0; o[mt][3] *= al1;
          }
        }
        // P^T as bf16 hi + lo, moved from accumulator layout to B-operand layout
        const uint32_t h01 = pack_bf16x2(p0, p1), h23 = pack_bf16x2(p2, p3);
        const __nv_bfloat162 h01v = *reinterpret_cast<const __nv_bfloat162 *>(&h01);
        const __nv_bfloat162 h23v = *reinterpret_cast<const __nv_bfloat162 *>(&h23);
        const uint32_t l01 = pack_bf16x2(p0 - __low2float(h01v), p1 - __high2float(h01v));
        const uint32_t l23 = pack_bf16x2(p2 - __low2float(h23v), p3 - __high2float(h23v));
        const uint32_t bh0 = movmatrix_trans(h01), bh1 = movmatrix_trans(h23);
        const uint32_t bl0 = movmatrix_trans(l01), bl1 = movmatrix_trans(l23);

        // O^T += V^T . P^T
        {
          const int ch = (lane & 7) + ((lane >> 3) & 1) * 8;
          const int tok = wq * 16 + (lane >> 4) * 8;
#pragma unroll
          for (int mt = 0; mt < 8; ++mt) {
            uint32_t a0, a1, a2, a3;
            ldmatrix_x4(sb + vt_byte_offset(tok, mt * 16 + ch), a0, a1, a2, a3);
            mma_bf16(o[mt], a0, a1, a2, a3, bh0, bh1);
            mma_bf16(o[mt], a0, a1, a2, a3, bl0, bl1);
          }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(smem_u32(&sm.empty[stage]));
      }
      if (!ok) break;
      ring_index += ps.tiles();

      // ---- combine the four warps' states (log-sum-exp merge through shared memory)
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, off);
        l1 += __shfl_xor_sync(0xffffffffu, l1, off);
      }
      float *mg = sm.merge[warp];
#pragma unroll
      for (int mt = 0; mt < 8; ++mt) {
        mg[(2 * tq) * kMergeRow + mt * 16 + g] = o[mt][0];
        mg[(2 * tq + 1) * kMergeRow + mt * 16 + g] = o[mt][1];
        mg[(2 * tq) * kMergeRow + mt * 16 + g + 8] = o[mt][2];
        mg[(2 * tq + 1) * kMergeRow + mt * 16 + g + 8] = o[mt][3];
      }
      if (g == 0) {
        mg[kMergeM + 2 * tq] = m0;
        mg[kMergeM + 2 * tq + 1] = m1;
        mg[kMergeL + 2 * tq] = l0;
        mg[kMergeL + 2 * tq + 1] = l1;
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sm.group_bar));
      if (!mbar_wait(smem_u32(&sm.group_bar), group_phase, abort_flag, p.status, kDevTimeoutDecode)) break;
      group_phase ^= 1u;

      const bool whole_pair = (pair_first >= tile_begin) && (pair_first + pair_tiles <= tile_end);
      const int d = threadIdx.x % 128;   // output channel; the two halves of the consumer threads take alternate heads
      {
        // pair index in launch order and partial slot of this (pair, CTA)
        const int pidx = slice_seq * Hkv + kvh;   // (cur has already advanced past the slice)
        float *rec = p.partial + (size_t)(pidx + blockIdx.x) * kPartialFloats;
        for (int h = threadIdx.x / 128; h < G; h += kConsumerWarps * 32 / 128) {
          float M = -INFINITY;
#pragma unroll
          for (int w = 0; w < kConsumerWarps; ++w) M = fmaxf(M, sm.merge[w][kMergeM + h]);
          float L = 0.f, O = 0.f;
#pragma unroll
          for (int w = 0; w < kConsumerWarps; ++w) {
            const float f = exp2f(sm.merge[w][kMergeM + h] - M);   // a warp that saw no valid key has m = -inf -> 0
            L += sm.merge[w][kMergeL + h] * f;
            O += sm.merge[w][h * kMergeRow + d] * f;
          }
          if (whole_pair) {
            p.out[((size_t)sq.q_begin * p.n_q_heads + (size_t)kvh * G + h) * kHeadDim + d] = O / L;
          } else {
            rec[h * 128 + d] = O;
            if (d == 0) { rec[1024 + h] = M; rec[1032 + h] = L; }
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sm.group_bar));
      if (!mbar_wait(smem_u32(&sm.group_bar), group_phase, abort_flag, p.status, kDevTimeoutDecode)) break;
      group_phase ^= 1u;
    }
  }
  __syncthreads();
}

// Merge of the split-K partials of one (sequence, q head): exact log-sum-exp combination.
__global__ void __launch_bounds__(128) st_k_decode_merge(const __grid_constant__ AttnParams p) {
  grid_dep_launch();
  grid_dep_wait();
  // a decode kernel that gave up (expired wait, page id outside the pool) left partial records unwritten: merge nothing
  if (*(volatile const int32_t *)p.status != kDevOk) return;
  const int Hkv = p.n_kv_heads, G = p.group;
  const int seq_i = blockIdx.x / p.n_q_heads, qh = blockIdx.x % p.n_q_heads;
  const int kvh = qh / G, h = qh % G;
  const AttnSeq sq = p.seq[seq_i];
  const int pair_tiles = ((sq.a_len + 63) >> 6) + ((sq.b_base + 1 + 63) >> 6);
  const int first = sq.work_begin * Hkv + kvh * pair_tiles;
  const int c_first = first / p.work_per_cta, c_last = (first + pair_tiles - 1) / p.work_per_cta;
  if (c_first == c_last) return;  // the decode kernel wrote the final row itself
  const int pidx = seq_i * Hkv + kvh;
  const int d = threadIdx.x;
  float M = -INFINITY;
  for (int c = c_first; c <= c_last; ++c) M = fmaxf(M, p.partial[(size_t)(pidx + c) * kPartialFloats + 1024 + h]);
  float L = 0.f, O = 0.f;
  for (int c = c_first; c <= c_last; ++c) {
    const float *rec = p.partial + (size_t)(pidx + c) * kPartialFloats;
    const float f = exp2f(rec[1024 + h] - M);
    L += rec[1032 + h] * f;
    O += rec[h * 128 + d] * f;
  }
  p.out[((size_t)sq.q_begin * p.n_q_heads + qh) * kHeadDim + d] = O / L;
}

size_t decode_partial_floats(int n_seq_per_launch, int n_kv_heads, int num_sms) {
  return (size_t)(n_seq_per_launch * n_kv_heads + 2 * num_sms + 8) * kPartialFloats;
}

static size_t decode_smem_bytes() { return sizeof(DecodeSmem) + 1024; }

cudaError_t init_decode_kernels() {
  return cudaFuncSetAttribute(st_k_decode, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)decode_smem_bytes());
}

cudaError_t launch_decode(AttnParams &p, int num_sms, cudaStream_t stream, int *n_launches, cudaEvent_t t0,
                          cudaEvent_t t1) {
  *n_launches = 0;
  // tiles per sequence -> prefix
  int total = 0;
  for (int i = 0; i < p.n_seq; ++i) {
    p.seq[i].work_begin = total;
    total += ((p.seq[i].a_len + 63) >> 6) + ((p.seq[i].b_base + 1 + 63) >> 6);
  }
  total *= p.n_kv_heads;
  if (total == 0) return cudaSuccess;
  // one CTA per SM (shared memory allows one resident CTA): a single wave in which every CTA streams the same bytes
  const int max_cta = num_sms;
  const int per = (total + max_cta - 1) / max_cta;
  p.total_work = total;
  p.work_per_cta = per;
  p.n_cta = (total + per - 1) / per;
  if (t0) cudaEventRecord(t0, stream);
  cudaError_t e = launch_dependent(st_k_decode, dim3(p.n_cta), dim3(kThreads), decode_smem_bytes(), stream, p);
  if (e != cudaSuccess) return e;
  if (t1) cudaEventRecord(t1, stream);
  ++*n_launches;
  if (p.n_cta > 1) {
    e = launch_dependent(st_k_decode_merge, dim3(p.n_seq * p.n_q_heads), dim3(128), 0, stream, p);
    if (e != cudaSuccess) return e;
    ++*n_launches;
  }
  return cudaSuccess;
}

}  // namespace st
