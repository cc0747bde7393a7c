// Projection y = x W^T on the 5th-generation tensor cores (tcgen05 + tensor memory, operands fetched by TMA): the
// Q, K, V and output projections of the attention block around the streaming attention path (the Qwen3 backbones
// of Section 4.1; the paper's method itself starts behind them).
//
//   x [M, K] bf16, row-major (leading dimension ldx elements)       activations, one row per token
//   W [N, K] bf16, row-major (leading dimension ldw)                one row per output feature
//   y [M, N] bf16 or fp32, row-major (leading dimension ldy)        fp32 accumulation
//
// Shape of the kernel. One CTA per SM walks the 128 x 256 tiles of y (tile index = CTA index + i * grid size); the
// accumulator is double-buffered in tensor memory (2 x 256 columns), so the epilogue of one tile runs under the MMAs of
// the next, and the operand ring keeps filling across tile boundaries. Both operands are K-major, so a tile of either is a
// box of a 2-D tensor map: 64 elements of K (128 bytes, one swizzle atom) by 128 (x) or 256 (W) rows, landed by TMA in
// the 128-byte-swizzled layout that the MMA's shared-memory descriptors name; rows and K positions past the end of a
// matrix arrive as zeros. Four stages of 48 KiB. Warp 0 lane 0 issues the TMA loads, warp 1 allocates the 512 columns of
// tensor memory and issues, per K block, four MMAs of 128 x 256 x 16 (an elected lane; the loop runs warp-uniform),
// warps 2-5 read the accumulator (one thread per row, 32 columns at a time), convert and store: 64 or 128 contiguous
// bytes per thread and step. No TMA load carries a cluster multicast. Every mbarrier wait is bounded.
#include <cuda.h>
#include <string.h>

#include <algorithm>
#include <mutex>
#include <string>

#include "../../include/streaming_thinker.h"
#include "st_internal.h"

namespace st {

namespace {

constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kStages = 4;
constexpr int kStageA = kBM * kBK * 2;          // 16 KiB
constexpr int kStageB = kBN * kBK * 2;          // 32 KiB
constexpr int kLinThreads = 192;                // producer, issuer, four epilogue warps
constexpr int kLinSmem = kStages * (kStageA + kStageB) + 256;

struct LinBarriers {
  uint64_t full[kStages];
  uint64_t empty[kStages];
  uint64_t acc_full[2];    // the MMAs of a tile into accumulator buffer b are complete
  uint64_t acc_empty[2];   // the four epilogue warps have read buffer b
  uint32_t tmem_base;
  int abort_flag;
};

struct LinParams {
  void *y;
  int32_t *status;
  int64_t M, N, K, ldy;
  int32_t out_fp32;
  int32_t tiles_n, tiles;
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, int x, int y, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
      "l"(map), "r"(x), "r"(y), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void lin_tmem_alloc(uint32_t smem_dst, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
}
__device__ __forceinline__ void lin_tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void lin_tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void lin_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void lin_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ uint32_t lin_elect_one() {
  uint32_t pred;
  asm volatile("{\n.reg .pred P;\nelect.sync _|P, 0xffffffff;\nselp.u32 %0, 1, 0, P;\n}\n" : "=r"(pred));
  return pred;
}
__device__ __forceinline__ void lin_commit(uint32_t bar, uint32_t issue) {
  asm volatile(
      "{\n.reg .pred q;\n"
      "setp.ne.b32 q, %1, 0;\n"
      "@q tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n}\n" ::"r"(bar), "r"(issue)
      : "memory");
}
__device__ __forceinline__ void lin_mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate,
                                           uint32_t issue) {
  asm volatile(
      "{\n.reg .pred p, q;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "setp.ne.b32 q, %5, 0;\n"
      "@q tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
      "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(issue)
      : "memory");
}
__device__ __forceinline__ void lin_tmem_ld32(uint32_t taddr, float *r) {
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
__device__ __forceinline__ void lin_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart (the layout a TMA box of
// 64 bf16 by R rows with SWIZZLE_128B lands in).
__device__ __forceinline__ uint64_t lin_desc(uint32_t smem_addr) {
  return (uint64_t)((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (64ull << 32) | (1ull << 46) | (2ull << 61);
}
// Instruction descriptor: fp32 accumulator, bf16 x bf16, both operands K-major, M = 128, N = 256.
constexpr uint32_t kLinIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);

}  // namespace

__global__ void __launch_bounds__(kLinThreads, 1)
st_k_linear(const __grid_constant__ CUtensorMap map_x, const __grid_constant__ CUtensorMap map_w, const LinParams p) {
  extern __shared__ uint8_t lin_smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(lin_smem_raw) + 1023) & ~(uintptr_t)1023);
  LinBarriers &bar = *reinterpret_cast<LinBarriers *>(smem + kStages * (kStageA + kStageB));
  volatile int *abort_flag = &bar.abort_flag;
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const int k_blocks = (int)((p.K + kBK - 1) / kBK);

  if (threadIdx.x == 0) {
    for (int i = 0; i < kStages; ++i) {
      mbar_init(smem_u32(&bar.full[i]), 1);
      mbar_init(smem_u32(&bar.empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bar.acc_full[i]), 1);
      mbar_init(smem_u32(&bar.acc_empty[i]), 4);
    }
    bar.abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    lin_tmem_alloc(smem_u32(&bar.tmem_base), 2 * kBN);
    lin_tmem_relinquish();
  }
  grid_dep_launch();
  lin_fence_before();
  __syncthreads();
  lin_fence_after();
  const uint32_t tmem = bar.tmem_base;
  grid_dep_wait();   // the activations may come from the kernel in front

  if (warp == 0) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      int it = 0;                                          // K blocks loaded so far, over all tiles of this CTA
      for (int tile = (int)blockIdx.x; tile < p.tiles; tile += (int)gridDim.x) {
        const int tile_m = tile / p.tiles_n, tile_n = tile % p.tiles_n;
        bool ok = true;
        for (int kb = 0; kb < k_blocks; ++kb, ++it) {
          const int st = it % kStages;
          ok = mbar_wait(smem_u32(&bar.empty[st]), ((uint32_t)(it / kStages) & 1u) ^ 1u, abort_flag, p.status, kDevTimeoutLinear);
          if (!ok) break;
          const uint32_t full = smem_u32(&bar.full[st]);
          mbar_arrive_expect_tx(full, kStageA + kStageB);
          tma_load_2d(smem_u32(smem + st * (kStageA + kStageB)), &map_x, kb * kBK, tile_m * kBM, full);
          tma_load_2d(smem_u32(smem + st * (kStageA + kStageB) + kStageA), &map_w, kb * kBK, tile_n * kBN, full);
        }
        if (!ok) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    const uint32_t issue = lin_elect_one();
    bool ok = true;
    int it = 0, n_tile = 0;
    for (int tile = (int)blockIdx.x; tile < p.tiles && ok; tile += (int)gridDim.x, ++n_tile) {
      const int buf = n_tile & 1;
      // the epilogue must have read what the tile before last left in this buffer
      ok = mbar_wait(smem_u32(&bar.acc_empty[buf]), ((uint32_t)(n_tile >> 1) & 1u) ^ 1u, abort_flag, p.status, kDevTimeoutLinear);
      if (!ok) break;
      lin_fence_after();
      const uint32_t d = tmem + (uint32_t)(buf * kBN);
      for (int kb = 0; kb < k_blocks && ok; ++kb, ++it) {
        const int st = it % kStages;
        ok = mbar_wait(smem_u32(&bar.full[st]), (uint32_t)(it / kStages) & 1u, abort_flag, p.status, kDevTimeoutLinear);
        if (!ok) break;
        lin_fence_after();
        const uint64_t ad = lin_desc(smem_u32(smem + st * (kStageA + kStageB)));
        const uint64_t bd = lin_desc(smem_u32(smem + st * (kStageA + kStageB) + kStageA));
#pragma unroll
        for (int ks = 0; ks < kBK / 16; ++ks)
          lin_mma_ss(d, ad + (uint64_t)((ks * 32) >> 4), bd + (uint64_t)((ks * 32) >> 4), kLinIdesc, (kb > 0 || ks > 0) ? 1u : 0u, issue);
        lin_commit(smem_u32(&bar.empty[st]), issue);      // the stage is free once these MMAs have read it
      }
      if (ok) lin_commit(smem_u32(&bar.acc_full[buf]), issue);
    }
  } else {
    // ------------------------------------------------------------------ epilogue: thread = row = TMEM lane
    const int quarter = warp & 3;                        // the TMEM lanes a warp may read: 32 * (warp % 4) ...
    const int r_local = quarter * 32 + lane;
    int n_tile = 0;
    for (int tile = (int)blockIdx.x; tile < p.tiles; tile += (int)gridDim.x, ++n_tile) {
      const int tile_m = tile / p.tiles_n, tile_n = tile % p.tiles_n;
      const int buf = n_tile & 1;
      const int64_t row = (int64_t)tile_m * kBM + r_local;
      if (!mbar_wait(smem_u32(&bar.acc_full[buf]), (uint32_t)(n_tile >> 1) & 1u, abort_flag, p.status, kDevTimeoutLinear)) break;
      lin_fence_after();
      const uint32_t t_addr = tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(buf * kBN);
#pragma unroll 1
      for (int c0 = 0; c0 < kBN; c0 += 32) {
        float acc[32];
        lin_tmem_ld32(t_addr + c0, acc);
        lin_wait_ld();
        if (c0 == kBN - 32) {
          // the last columns are in registers: the buffer may take the tile after next
          lin_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&bar.acc_empty[buf]));
        }
        const int64_t col = (int64_t)tile_n * kBN + c0;
        if (row < p.M && col < p.N) {
          // N is a multiple of 8: a group of 8 columns is inside the matrix or outside it
          if (p.out_fp32) {
            float *dst = reinterpret_cast<float *>(p.y) + row * p.ldy + col;
#pragma unroll
            for (int c = 0; c < 32; c += 4)
              if (col + c < p.N) *reinterpret_cast<float4 *>(dst + c) = make_float4(acc[c], acc[c + 1], acc[c + 2], acc[c + 3]);
          } else {
            __nv_bfloat16 *dst = reinterpret_cast<__nv_bfloat16 *>(p.y) + row * p.ldy + col;
#pragma unroll
            for (int c = 0; c < 32; c += 8)
              if (col + c < p.N)
                *reinterpret_cast<uint4 *>(dst + c) = make_uint4(pack_bf16x2(acc[c], acc[c + 1]), pack_bf16x2(acc[c + 2], acc[c + 3]),
                                                                 pack_bf16x2(acc[c + 4], acc[c + 5]), pack_bf16x2(acc[c + 6], acc[c + 7]));
          }
        }
      }
    }
    lin_fence_before();
  }
  lin_fence_before();
  __syncthreads();
  if (warp == 1) {
    lin_fence_after();
    lin_tmem_dealloc(tmem, 2 * kBN);
  }
}

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct LinearDevice {
  bool ready = false;
  int32_t *status = nullptr;
  int num_sms = 0;
};
constexpr int kLinMaxDevices = 64;
LinearDevice g_lin_device[kLinMaxDevices];
EncodeTiledFn g_encode = nullptr;
std::mutex g_lin_mutex;

int lin_fail(char *err, int32_t cap, int code, const std::string &msg) {
  if (err && cap > 0) {
    strncpy(err, msg.c_str(), (size_t)cap - 1);
    err[cap - 1] = '\0';
  }
  return code;
}

// 2-D map over a row-major bf16 matrix [rows, cols] with leading dimension ld: boxes of 64 columns by box_rows rows,
// 128-byte swizzle, zeros outside the matrix.
CUresult encode_map(CUtensorMap *map, const void *base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return g_encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

}  // namespace

}  // namespace st

extern "C" int st_linear(int32_t device, const void *x, int64_t m, int64_t k, int64_t ldx, const void *w, int64_t n, int64_t ldw,
                         void *y, int64_t ldy, int32_t out_fp32, void *stream, char *err, int32_t err_cap) {
  using namespace st;
  if (err && err_cap > 0) err[0] = '\0';
  if (device < 0 || device >= kLinMaxDevices) return lin_fail(err, err_cap, ST_ERR_INVALID_ARG, "device ordinal out of range");
  if (!x || !w || !y) return lin_fail(err, err_cap, ST_ERR_INVALID_ARG, "NULL argument");
  if (m < 1 || n < 1 || k < 1 || m > INT32_MAX || n > INT32_MAX || k > INT32_MAX)
    return lin_fail(err, err_cap, ST_ERR_INVALID_ARG, "m, n and k must be between 1 and 2^31 - 1");
  if (k % 8 || n % 8) return lin_fail(err, err_cap, ST_ERR_INVALID_ARG, "k and n must be multiples of 8 (16-byte rows and stores)");
  if (ldx < k || ldw < k || ldy < n || ldx % 8 || ldw % 8 || ldy % (out_fp32 ? 4 : 8))
    return lin_fail(err, err_cap, ST_ERR_INVALID_ARG, "leading dimensions must cover a row and keep every row 16-byte aligned");
  if (((uintptr_t)x | (uintptr_t)w | (uintptr_t)y) & 15) return lin_fail(err, err_cap, ST_ERR_INVALID_ARG, "x, w and y must be 16-byte aligned");

  int previous = -1;
  cudaError_t e = cudaGetDevice(&previous);
  if (e == cudaSuccess && previous != device) e = cudaSetDevice(device);
  if (e != cudaSuccess) return lin_fail(err, err_cap, ST_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(e));
  struct Restore {
    int dev, cur;
    ~Restore() { if (dev >= 0 && dev != cur) cudaSetDevice(dev); }
  } restore{previous, device};
  LinearDevice dev;
  {
    std::lock_guard<std::mutex> lock(g_lin_mutex);
    if (!g_encode) {
      void *fn = nullptr;
      cudaDriverEntryPointQueryResult q;
      e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
      if (e != cudaSuccess || !fn || q != cudaDriverEntryPointSuccess)
        return lin_fail(err, err_cap, ST_ERR_CUDA, "the driver does not provide cuTensorMapEncodeTiled");
      g_encode = (EncodeTiledFn)fn;
    }
    LinearDevice &d = g_lin_device[device];
    if (!d.ready) {
      e = cudaFuncSetAttribute(st_k_linear, cudaFuncAttributeMaxDynamicSharedMemorySize, kLinSmem + 1024);
      if (e == cudaSuccess) e = cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, device);
      if (e == cudaSuccess) e = cudaMalloc(&d.status, sizeof(int32_t));
      if (e == cudaSuccess) e = cudaMemset(d.status, 0, sizeof(int32_t));
      if (e != cudaSuccess) return lin_fail(err, err_cap, ST_ERR_CUDA, std::string("kernel set-up: ") + cudaGetErrorString(e));
      d.ready = true;
    }
    dev = d;
  }
  CUtensorMap map_x, map_w;
  if (encode_map(&map_x, x, m, k, ldx, kBM) != CUDA_SUCCESS || encode_map(&map_w, w, n, k, ldw, kBN) != CUDA_SUCCESS)
    return lin_fail(err, err_cap, ST_ERR_CUDA, "cuTensorMapEncodeTiled failed");
  LinParams p;
  p.y = y;
  p.status = dev.status;
  p.M = m;
  p.N = n;
  p.K = k;
  p.ldy = ldy;
  p.out_fp32 = out_fp32 ? 1 : 0;
  p.tiles_n = (int32_t)((n + kBN - 1) / kBN);
  const int64_t tiles = ((m + kBM - 1) / kBM) * p.tiles_n;
  if (tiles > INT32_MAX) return lin_fail(err, err_cap, ST_ERR_INVALID_ARG, "too many output tiles");
  p.tiles = (int32_t)tiles;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)std::min<int64_t>(tiles, dev.num_sms));
  cfg.blockDim = dim3(kLinThreads);
  cfg.dynamicSmemBytes = kLinSmem + 1024;
  cfg.stream = (cudaStream_t)stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  e = cudaLaunchKernelEx(&cfg, st_k_linear, map_x, map_w, p);
  if (e != cudaSuccess) return lin_fail(err, err_cap, ST_ERR_CUDA, std::string("launch: ") + cudaGetErrorString(e));
  return ST_OK;
}

namespace st {
__global__ void st_k_cast_bf16(const float *src, __nv_bfloat16 *dst, int64_t n8) {
  // 8 values per thread: two 16-byte loads, one 16-byte store
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n8; i += (int64_t)gridDim.x * blockDim.x) {
    const float4 a = reinterpret_cast<const float4 *>(src)[2 * i], b = reinterpret_cast<const float4 *>(src)[2 * i + 1];
    reinterpret_cast<uint4 *>(dst)[i] = make_uint4(pack_bf16x2(a.x, a.y), pack_bf16x2(a.z, a.w), pack_bf16x2(b.x, b.y), pack_bf16x2(b.z, b.w));
  }
}
}  // namespace st

extern "C" int st_cast_to_bf16(int32_t device, const void *src, void *dst, int64_t n, void *stream) {
  if (device < 0 || !src || !dst || n < 0 || n % 8 || (((uintptr_t)src | (uintptr_t)dst) & 15)) return ST_ERR_INVALID_ARG;
  if (n == 0) return ST_OK;
  int previous = -1;
  if (cudaGetDevice(&previous) != cudaSuccess) return ST_ERR_CUDA;
  if (previous != device && cudaSetDevice(device) != cudaSuccess) return ST_ERR_CUDA;
  const int64_t n8 = n / 8;
  const unsigned blocks = (unsigned)std::min<int64_t>((n8 + 255) / 256, 148 * 8);
  st::st_k_cast_bf16<<<blocks, 256, 0, (cudaStream_t)stream>>>((const float *)src, (__nv_bfloat16 *)dst, n8);
  const cudaError_t e = cudaGetLastError();
  if (previous != device) cudaSetDevice(previous);
  return e == cudaSuccess ? ST_OK : ST_ERR_CUDA;
}

extern "C" int st_linear_status(int32_t device, void *stream) {
  using namespace st;
  if (device < 0 || device >= kLinMaxDevices) return ST_ERR_INVALID_ARG;
  LinearDevice dev;
  {
    std::lock_guard<std::mutex> lock(g_lin_mutex);
    dev = g_lin_device[device];
  }
  if (!dev.ready) return ST_ERR_INVALID_ARG;
  int previous = -1;
  if (cudaGetDevice(&previous) != cudaSuccess) return ST_ERR_CUDA;
  if (previous != device && cudaSetDevice(device) != cudaSuccess) return ST_ERR_CUDA;
  int32_t h = 0;
  cudaError_t e = cudaMemcpyAsync(&h, dev.status, sizeof(h), cudaMemcpyDeviceToHost, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize((cudaStream_t)stream);
  if (e == cudaSuccess && h != kDevOk) e = cudaMemset(dev.status, 0, sizeof(int32_t));
  if (previous != device) cudaSetDevice(previous);
  if (e != cudaSuccess) return ST_ERR_CUDA;
  return h == kDevOk ? ST_OK : ST_ERR_DEVICE_TIMEOUT;
}
