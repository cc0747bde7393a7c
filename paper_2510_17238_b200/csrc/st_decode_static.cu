// st_decode_attention_static: the dual-cache decode attention for callers that must not allocate.
//
// The regular path keeps the split-K workspace of the decode kernel in memory that st_create obtained
// with cudaMalloc. Some hosts of this library cannot do that: an inference server whose memory manager
// has already claimed the whole GPU (a cudaMalloc from a plug-in then fails, or eats into memory the
// server believes it owns), or a latency-critical serving loop in which the implicit device-wide
// synchronisation of cudaMalloc / cudaFree would stall every stream. For them this file carries the
// workspace inside the library image itself: a file-scope __device__ array of fixed size that every GPU
// which loads the library holds until the process exits. The entry point below runs the same decode and
// merge kernels on it and calls no allocating routine of CUDA, of the C++ runtime's device side, or of
// any other library.
#include <mutex>
#include <string.h>

#include <string>

#include "../../include/streaming_thinker.h"
#include "st_internal.h"

namespace {

// Fixed capacity of the built-in workspace: one partial record per (sequence, kv head) pair plus one per
// CTA of the decode grid. 512 pairs + 304 CTAs = 816 records of 4160 bytes = 3.4 MB per GPU.
constexpr int kStaticMaxPairs = 512;
constexpr int kStaticMaxCtas = 304;
constexpr int kStaticMaxDevices = 64;

static __device__ __align__(256) float g_static_partials[(size_t)(kStaticMaxPairs + kStaticMaxCtas) * st::kPartialFloats];
static __device__ __align__(256) int32_t g_static_status[64];

// In host code the two names above are host-side stand-ins, not device addresses. The real addresses
// are looked up once per device (with that device current) and cached here.
struct StaticDevice {
  bool ready = false;
  float *partials = nullptr;
  int32_t *status = nullptr;
  int num_sms = 0;
};
StaticDevice g_static_device[kStaticMaxDevices];
std::mutex g_static_mutex;

int static_fail(char *err, int32_t cap, int code, const std::string &msg) {
  if (err && cap > 0) {
    strncpy(err, msg.c_str(), (size_t)cap - 1);
    err[cap - 1] = '\0';
  }
  return code;
}

}  // namespace

namespace {

// Makes `device` current for the duration of a call and puts the caller's device back afterwards.
struct DeviceScope {
  int previous = -1;
  cudaError_t enter(int device) {
    cudaError_t e = cudaGetDevice(&previous);
    if (e != cudaSuccess) { previous = -1; return e; }
    return previous == device ? cudaSuccess : cudaSetDevice(device);
  }
  ~DeviceScope() {
    if (previous >= 0) cudaSetDevice(previous);
  }
};

}  // namespace

extern "C" int st_decode_attention_static(int32_t device, const void *pool_source, int64_t n_pages_source,
                                          const void *pool_reason, int64_t n_pages_reason,
                                          const int32_t *page_table_source, int32_t table_stride_source,
                                          const int32_t *page_table_reason, int32_t table_stride_reason,
                                          const int32_t *slots, const int32_t *source_len, const int32_t *reason_len,
                                          int32_t n_seq, const void *q_rotated, void *out, int32_t n_q_heads,
                                          int32_t n_kv_heads, float softmax_scale, void *stream, char *err,
                                          int32_t err_cap) {
  if (err && err_cap > 0) err[0] = '\0';
  if (device < 0 || device >= kStaticMaxDevices) return static_fail(err, err_cap, ST_ERR_INVALID_ARG, "device ordinal out of range");
  if (!pool_source || !pool_reason || !page_table_source || !page_table_reason || !slots || !source_len || !reason_len ||
      !q_rotated || !out)
    return static_fail(err, err_cap, ST_ERR_INVALID_ARG, "NULL argument");
  if (n_pages_source < 1 || n_pages_reason < 1 || n_pages_source > INT32_MAX || n_pages_reason > INT32_MAX)
    return static_fail(err, err_cap, ST_ERR_INVALID_ARG, "n_pages_source and n_pages_reason must be between 1 and 2^31 - 1");
  if (n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads || n_q_heads / n_kv_heads > st::kMaxGroup)
    return static_fail(err, err_cap, ST_ERR_INVALID_ARG, "n_q_heads must be a multiple of n_kv_heads with at most 8 q heads per kv head");
  if (n_seq < 1) return static_fail(err, err_cap, ST_ERR_INVALID_ARG, "n_seq must be >= 1");
  if (n_seq > st::kMaxSeqPerLaunch || (int64_t)n_seq * n_kv_heads > kStaticMaxPairs)
    return static_fail(err, err_cap, ST_ERR_INVALID_ARG,
                       "too many sequences for the built-in workspace: at most " + std::to_string(st::kMaxSeqPerLaunch) +
                           " sequences and " + std::to_string(kStaticMaxPairs) + " (sequence, kv head) pairs per call");
  if (table_stride_source < 1 || table_stride_reason < 1) return static_fail(err, err_cap, ST_ERR_INVALID_ARG, "page table strides must be >= 1");
  for (int i = 0; i < n_seq; ++i) {
    if (slots[i] < 0 || source_len[i] < 0 || reason_len[i] < 1)
      return static_fail(err, err_cap, ST_ERR_INVALID_ARG, "slots and source_len must be >= 0, reason_len >= 1 (it counts the new token)");
    if (((int64_t)source_len[i] + 63) / 64 > table_stride_source || ((int64_t)reason_len[i] + 63) / 64 > table_stride_reason)
      return static_fail(err, err_cap, ST_ERR_INVALID_ARG, "a length exceeds what its page table row can describe");
  }

  DeviceScope scope;
  cudaError_t e = scope.enter(device);
  if (e != cudaSuccess) return static_fail(err, err_cap, ST_ERR_CUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(e));
  StaticDevice dev;
  {
    // first call on this device: resolve the device addresses of the built-in arrays
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDevice &d = g_static_device[device];
    if (!d.ready) {
      e = cudaGetSymbolAddress((void **)&d.partials, g_static_partials);
      if (e != cudaSuccess) return static_fail(err, err_cap, ST_ERR_CUDA, std::string("cudaGetSymbolAddress(partials): ") + cudaGetErrorString(e));
      e = cudaGetSymbolAddress((void **)&d.status, g_static_status);
      if (e != cudaSuccess) return static_fail(err, err_cap, ST_ERR_CUDA, std::string("cudaGetSymbolAddress(status): ") + cudaGetErrorString(e));
      e = cudaDeviceGetAttribute(&d.num_sms, cudaDevAttrMultiProcessorCount, device);
      if (e != cudaSuccess) return static_fail(err, err_cap, ST_ERR_CUDA, std::string("cudaDeviceGetAttribute: ") + cudaGetErrorString(e));
      e = st::init_kernels();
      if (e != cudaSuccess) return static_fail(err, err_cap, ST_ERR_CUDA, std::string("kernel set-up: ") + cudaGetErrorString(e));
      d.ready = true;
    }
    dev = d;
  }

  st::AttnParams p;
  memset(&p, 0, sizeof(p));
  p.pool_a = (const uint8_t *)pool_source;
  p.pool_b = (const uint8_t *)pool_reason;
  p.ptab_a = page_table_source;
  p.ptab_b = page_table_reason;
  p.ptab_stride_a = table_stride_source;
  p.ptab_stride_b = table_stride_reason;
  p.norm_q = p.norm_k = nullptr;
  p.n_pages_a = (int32_t)n_pages_source;
  p.n_pages_b = (int32_t)n_pages_reason;
  p.qhat = (const __nv_bfloat16 *)q_rotated;
  p.out = (float *)out;
  p.partial = dev.partials;
  p.status = dev.status;
  p.n_seq = n_seq;
  p.n_q_heads = n_q_heads;
  p.n_kv_heads = n_kv_heads;
  p.group = n_q_heads / n_kv_heads;
  const double scale = softmax_scale > 0.f ? (double)softmax_scale : 0.08838834764831845;  // 1/sqrt(128)
  p.scale_log2 = (float)(scale * 1.4426950408889634);
  for (int i = 0; i < n_seq; ++i) {
    p.seq[i].slot = slots[i];
    p.seq[i].a_len = source_len[i];
    p.seq[i].b_base = reason_len[i] - 1;
    p.seq[i].n_rows = 1;
    p.seq[i].q_begin = i;
    p.seq[i].work_begin = 0;
    p.seq[i].rope_off = 0;
  }
  cudaStream_t s = (cudaStream_t)stream;
  // the status word is the only part of the workspace that must start at zero; partial records are
  // always written completely before the merge reads them
  e = cudaMemsetAsync(dev.status, 0, sizeof(int32_t), s);
  if (e != cudaSuccess) return static_fail(err, err_cap, ST_ERR_CUDA, std::string("cudaMemsetAsync: ") + cudaGetErrorString(e));
  int n_launches = 0;
  // the decode grid is one CTA per SM; the clamp keeps it within the built-in capacity on any device
  e = st::launch_decode(p, dev.num_sms < kStaticMaxCtas ? dev.num_sms : kStaticMaxCtas, s, &n_launches);
  if (e != cudaSuccess) return static_fail(err, err_cap, ST_ERR_CUDA, std::string("decode launch: ") + cudaGetErrorString(e));
  return ST_OK;
}

extern "C" int st_decode_static_status(int32_t device, void *stream) {
  if (device < 0 || device >= kStaticMaxDevices) return ST_ERR_INVALID_ARG;
  StaticDevice dev;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    dev = g_static_device[device];
  }
  if (!dev.ready) return ST_ERR_INVALID_ARG;
  DeviceScope scope;
  if (scope.enter(device) != cudaSuccess) return ST_ERR_CUDA;
  int32_t h = 0;   // (a stack word: the copy below allocates nothing)
  if (cudaMemcpyAsync(&h, dev.status, sizeof(h), cudaMemcpyDeviceToHost, (cudaStream_t)stream) != cudaSuccess) return ST_ERR_CUDA;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return ST_ERR_CUDA;
  if (h == st::kDevOk) return ST_OK;
  return h == st::kDevBadPage ? ST_ERR_DEVICE_CHECK : ST_ERR_DEVICE_TIMEOUT;
}
