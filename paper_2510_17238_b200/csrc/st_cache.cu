// Paged cache kernels: page-table update, RoPE-fused append, debug gather.
//
// The append implements the streaming position encoding of Section 3.2: each cache numbers its own
// tokens from zero, keys are rotated at that position before they are stored, and the query of the
// same token is rotated identically. The rotation runs in fp64 (angle = position * inv_freq, then
// sin/cos, then the 2x2 rotation) and is rounded once to bf16, so the cache holds the correctly
// rounded rotated key even at positions of several 10^4, where an fp32 angle would already be off
// by more than a bf16 ulp.
#include <string.h>

#include <algorithm>

#include "st_internal.h"

namespace st {

__global__ void __launch_bounds__(256) st_k_page_update(const __grid_constant__ PageUpdateParams p) {
  grid_dep_launch();
  grid_dep_wait();
  for (int i = threadIdx.x; i < p.n; i += blockDim.x) {
    const PageUpdate u = p.upd[i];
    const int which = u.slot_which & 1, slot = u.slot_which >> 1;
    p.ptab[which][(size_t)slot * p.stride[which] + u.index] = u.page;
  }
}

cudaError_t launch_page_update(const PageUpdateParams &p, cudaStream_t stream) {
  return launch_dependent(st_k_page_update, dim3(1), dim3(256), 0, stream, p);
}

// One thread block per aligned group of 8 cache positions of one sequence.
__global__ void __launch_bounds__(256) st_k_rope_append(const __grid_constant__ AppendParams p) {
  __shared__ double s_cos[8][64];
  __shared__ double s_sin[8][64];
  grid_dep_launch();

  // sequence of this block: last s with blk_begin <= blockIdx.x
  const int s = last_not_above(p.n_seq, (int)blockIdx.x, [&](int i) { return p.seq[i].blk_begin; });
  const AppendSeq sq = p.seq[s];
  const int g0 = (sq.pos0 >> 3) + ((int)blockIdx.x - sq.blk_begin);  // absolute group of 8 positions
  const int pos_lo = max(sq.pos0, g0 * 8);
  const int pos_hi = min(sq.pos0 + sq.n, g0 * 8 + 8);
  const int nt = pos_hi - pos_lo;
  if (nt <= 0) {
    grid_dep_wait();   // a grid must not finish before the one in front of it: later kernels rely on that order
    return;
  }

  for (int i = threadIdx.x; i < nt * 64; i += blockDim.x) {
    const int t = i >> 6, c = i & 63;
    double sn, cs;
    sincos((double)(pos_lo + t + sq.rope_off) * p.inv_freq[c], &sn, &cs);
    s_cos[t][c] = cs;
    s_sin[t][c] = sn;
  }
  __syncthreads();
  grid_dep_wait();   // the angles above need no memory; everything below reads what earlier kernels wrote

  const int page = p.ptab[(size_t)sq.slot * p.ptab_stride + (pos_lo >> 6)];
  if ((unsigned)page >= (unsigned)p.n_pages) {   // block-uniform: nothing is written through a bad page id
    if (threadIdx.x == 0) atomicExch(p.status, kDevBadPage);
    return;
  }
  const int Hq = p.n_q_heads, Hkv = p.n_kv_heads;
  uint8_t *page_base = p.pool + (size_t)page * Hkv * kBlockBytes;
  const int row0 = sq.q_begin + (pos_lo - sq.pos0);  // packed row of the group's first token

  // keys and queries: one item = (token, head, pair of 16-byte chunks c and c + 64)
  const int items_k = nt * Hkv * 8;
  const int items_q = (p.qhat != nullptr) ? nt * Hq * 8 : 0;
  const bool norm = p.norm_k != nullptr;
  for (int base = 0; base < items_k + items_q; base += blockDim.x) {
    // (the 8 items of one (token, head) row sit in 8 neighbouring lanes: either all of them are in range or none)
    const int it = base + threadIdx.x;
    const bool in_range = it < items_k + items_q;
    const unsigned lanes = __ballot_sync(0xffffffffu, in_range);
    if (!in_range) continue;
    const bool is_q = it >= items_k;
    const int j = is_q ? it - items_k : it;
    const int H = is_q ? Hq : Hkv;
    const int cp = j & 7;
    const int h = (j >> 3) % H;
    const int t = (j >> 3) / H;
    const __nv_bfloat16 *src = (is_q ? p.q : p.k) + ((size_t)(row0 + t) * H + h) * kHeadDim;
    const uint4 lo_raw = *reinterpret_cast<const uint4 *>(src + 8 * cp);
    const uint4 hi_raw = *reinterpret_cast<const uint4 *>(src + 64 + 8 * cp);
    const __nv_bfloat16 *lo = reinterpret_cast<const __nv_bfloat16 *>(&lo_raw);
    const __nv_bfloat16 *hi = reinterpret_cast<const __nv_bfloat16 *>(&hi_raw);
    uint4 lo_out, hi_out;
    __nv_bfloat16 *lo_o = reinterpret_cast<__nv_bfloat16 *>(&lo_out);
    __nv_bfloat16 *hi_o = reinterpret_cast<__nv_bfloat16 *>(&hi_out);
    // optional RMS normalisation of the row over its 128 channels, in fp64 like the rotation: x / sqrt(mean(x^2) + eps) * w
    double rs = 1.0;
    const float *nw = is_q ? p.norm_q : p.norm_k;
    if (norm) {
      double ss = 0.0;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const double x = (double)__bfloat162float(lo[e]), y = (double)__bfloat162float(hi[e]);
        ss += x * x + y * y;
      }
      ss += __shfl_xor_sync(lanes, ss, 1);
      ss += __shfl_xor_sync(lanes, ss, 2);
      ss += __shfl_xor_sync(lanes, ss, 4);
      rs = 1.0 / sqrt(ss * (1.0 / kHeadDim) + (double)p.norm_eps);
    }
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const double cs = s_cos[t][8 * cp + e], sn = s_sin[t][8 * cp + e];
      double x = (double)__bfloat162float(lo[e]), y = (double)__bfloat162float(hi[e]);
      if (norm) {
        x = x * rs * (double)nw[8 * cp + e];
        y = y * rs * (double)nw[64 + 8 * cp + e];
      }
      lo_o[e] = __double2bfloat16(x * cs - y * sn);
      hi_o[e] = __double2bfloat16(y * cs + x * sn);
    }
    if (is_q) {
      __nv_bfloat16 *dst = p.qhat + ((size_t)(row0 + t) * Hq + h) * kHeadDim;
      *reinterpret_cast<uint4 *>(dst + 8 * cp) = lo_out;
      *reinterpret_cast<uint4 *>(dst + 64 + 8 * cp) = hi_out;
    } else {
      const int tok = (pos_lo + t) & 63;
      uint8_t *blk = page_base + (size_t)h * kBlockBytes;
      *reinterpret_cast<uint4 *>(blk + k_byte_offset(tok, 8 * cp)) = lo_out;
      *reinterpret_cast<uint4 *>(blk + k_byte_offset(tok, 64 + 8 * cp)) = hi_out;
    }
  }

  // values, stored transposed: one item = (kv head, channel); a full group of 8 tokens is one
  // 16-byte chunk of the channel's row, a partial group is written element by element.
  const int tok_lo = pos_lo & 63;
  for (int it = threadIdx.x; it < Hkv * kHeadDim; it += blockDim.x) {
    const int c = it & 127, h = it >> 7;
    const __nv_bfloat16 *src = p.v + ((size_t)row0 * Hkv + h) * kHeadDim + c;
    uint8_t *blk = page_base + (size_t)h * kBlockBytes;
    if (nt == 8) {
      uint4 pk;
      __nv_bfloat16 *e = reinterpret_cast<__nv_bfloat16 *>(&pk);
#pragma unroll
      for (int t = 0; t < 8; ++t) e[t] = src[(size_t)t * Hkv * kHeadDim];
      *reinterpret_cast<uint4 *>(blk + vt_byte_offset(tok_lo, c)) = pk;
    } else {
      for (int t = 0; t < nt; ++t)
        *reinterpret_cast<__nv_bfloat16 *>(blk + vt_byte_offset(tok_lo + t, c)) = src[(size_t)t * Hkv * kHeadDim];
    }
  }
}

cudaError_t launch_rope_append(const AppendParams &p, int total_blocks, cudaStream_t stream) {
  if (total_blocks <= 0) return cudaSuccess;
  return launch_dependent(st_k_rope_append, dim3(total_blocks), dim3(256), 0, stream, p);
}

// Rotation tables of the fused decode append: entry [i][c] = (cos, sin) of fl(i * step) * inv_freq[c] in fp64.
// A position p = 1024 a + b then has cos/sin by one angle addition from hi[a] and lo[b]: the difference from
// sincos(fl(p * inv_freq[c])) is a few 1e-12 at the largest positions, far below half a bf16 ulp.
struct RopeTableParams {
  double inv_freq[64];
  double2 *table;
  int n, step;
};
__global__ void st_k_rope_table(const __grid_constant__ RopeTableParams p) {
  const int i = blockIdx.x * 4 + (threadIdx.x >> 6), c = threadIdx.x & 63;
  if (i >= p.n) return;
  double sn, cs;
  sincos((double)((long long)i * p.step) * p.inv_freq[c], &sn, &cs);
  p.table[(size_t)i * 64 + c] = make_double2(cs, sn);
}

cudaError_t launch_rope_table(const double *inv_freq, double2 *table, int n, int step, cudaStream_t stream) {
  RopeTableParams p;
  memcpy(p.inv_freq, inv_freq, sizeof(p.inv_freq));
  p.table = table;
  p.n = n;
  p.step = step;
  st_k_rope_table<<<(n + 3) / 4, 256, 0, stream>>>(p);
  return cudaGetLastError();
}

// Test surface: a kernel whose only work is a bounded wait on a barrier that nothing arrives at. It takes the same
// path as a stalled pipeline in the attention kernels: the wait gives up after `limit_ns`, records the status word
// and returns; the context stays usable.
__global__ void st_k_wait_expiry(int32_t *status, uint64_t limit_ns) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    abort_flag = 0;
    mbar_fence_init();
  }
  __syncthreads();
  mbar_wait(smem_u32(&bar), 0, &abort_flag, status, kDevTimeoutProbe, limit_ns);
}

cudaError_t launch_wait_expiry(int32_t *status, uint64_t limit_ns, cudaStream_t stream) {
  st_k_wait_expiry<<<1, 32, 0, stream>>>(status, limit_ns);
  return cudaGetLastError();
}

__global__ void st_k_fill_u16(uint16_t *dst, size_t n, uint16_t value) {
  // n is even and dst 4-byte aligned for every caller (whole cache blocks): two words per store
  const uint32_t pair = (uint32_t)value | ((uint32_t)value << 16);
  uint32_t *d = reinterpret_cast<uint32_t *>(dst);
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n / 2; i += (size_t)gridDim.x * blockDim.x) d[i] = pair;
}

cudaError_t launch_fill_u16(void *dst, size_t n, uint16_t value, cudaStream_t stream) {
  if (n == 0) return cudaSuccess;
  const size_t blocks = std::min<size_t>((n / 2 + 255) / 256, 148 * 16);
  st_k_fill_u16<<<(unsigned)blocks, 256, 0, stream>>>(reinterpret_cast<uint16_t *>(dst), n, value);
  return cudaGetLastError();
}

__global__ void st_k_cache_gather(const uint8_t *pool, const int32_t *ptab_row, int Hkv, int tok0, int ntok,
                                  __nv_bfloat16 *k_out, __nv_bfloat16 *v_out) {
  const size_t total = (size_t)ntok * Hkv * kHeadDim;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int c = (int)(i & 127);
    const int h = (int)((i >> 7) % Hkv);
    const int t = (int)((i >> 7) / Hkv);
    const int pos = tok0 + t;
    const uint8_t *blk = pool + ((size_t)ptab_row[pos >> 6] * Hkv + h) * kBlockBytes;
    k_out[i] = *reinterpret_cast<const __nv_bfloat16 *>(blk + k_byte_offset(pos & 63, c));
    v_out[i] = *reinterpret_cast<const __nv_bfloat16 *>(blk + vt_byte_offset(pos & 63, c));
  }
}

cudaError_t launch_cache_gather(const uint8_t *pool, const int32_t *ptab_row, int n_kv_heads, int tok0, int ntok,
                                __nv_bfloat16 *k_out, __nv_bfloat16 *v_out, cudaStream_t stream) {
  if (ntok <= 0) return cudaSuccess;
  const size_t total = (size_t)ntok * n_kv_heads * kHeadDim;
  const int blocks = (int)((total + 255) / 256 > 4096 ? 4096 : (total + 255) / 256);
  st_k_cache_gather<<<blocks, 256, 0, stream>>>(pool, ptab_row, n_kv_heads, tok0, ntok, k_out, v_out);
  return cudaGetLastError();
}

}  // namespace st
