// Host side of the C ABI: context, page allocator, per-sequence streaming state (unit boundaries,
// N_EOS / N_EOT counters of Algorithm 1), call validation, launch planning, cross-stream ordering.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <string>
#include <vector>

#include "../../include/streaming_thinker.h"
#include "st_internal.h"

namespace st {
cudaError_t init_decode_kernels();
cudaError_t init_attn_tc_kernels();
}  // namespace st

namespace {

constexpr int kEventRing = 1024;

struct SeqState {
  int32_t len[2] = {0, 0};            // committed tokens: [0] source cache, [1] reasoning cache
  int32_t n_eos = 0, n_eot = 0;
  std::vector<int32_t> unit_end;      // source prefix P_k of every closed source unit k = 1..n_eos
  std::vector<uint64_t> unit_serial;  // serial of the append call that closed unit k
  uint64_t last_src_serial = 0;       // last append call that touched this sequence
  std::vector<int32_t> pages[2];
  // position ids of reasoning tokens in the modes other than the streaming encoding
  int32_t concat_off = -1;            // ST_POS_CONCATENATED: T, fixed when the first reasoning token is appended
  int32_t unit_tokens = 0;            // ST_POS_UNIT_ALIGNED: reasoning tokens of the current unit (or final stage) so far
  int32_t final_base = -1;            // ST_POS_UNIT_ALIGNED: S, fixed at the first final-depth call
};

struct EventRec {
  cudaEvent_t ev = nullptr;
  cudaStream_t stream = nullptr;
  uint64_t serial = 0;
};

// A step that has been issued for some but not all layers.
struct Pending {
  bool active = false;
  int kind = 0;  // 0 append, 1 decode, 2 extend
  int next_layer = 0;
  uint32_t flags = 0;
  std::vector<int32_t> seq_ids, cu, vis_tokens;
  std::vector<int32_t> rope_off;      // per listed sequence: position id of a new token minus its index in the cache
  std::vector<uint8_t> is_final;      // per listed sequence: the call named ST_VIS_ALL (final depth)
  uint64_t wait_serial = 0;
  bool reverse = false;               // decode step: the kernel walks its tile list backwards (see st_k_decode)
};

thread_local std::string g_create_error;

}  // namespace

struct st_ctx {
  st_config cfg;
  bool host_only = false;
  int group = 1;
  int num_sms = 148;
  float scale_log2 = 0.f;
  double inv_freq[64];

  uint8_t *pool[2] = {nullptr, nullptr};
  bool own_pool = false;
  uint8_t *pool_alloc = nullptr;
  size_t layer_stride[2] = {0, 0};
  int32_t *d_ptab[2] = {nullptr, nullptr};
  int32_t ptab_stride[2] = {0, 0};
  std::vector<int32_t> free_pages[2];
  std::vector<SeqState> seqs;

  __nv_bfloat16 *qhat[2] = {nullptr, nullptr};  // rotated-query scratch per side
  float *partial = nullptr;                     // split-K workspace (reasoning side)
  double2 *rope_hi = nullptr, *rope_lo = nullptr;   // rotation tables of the fused decode append
  float *d_norm = nullptr;                          // q/k normalisation weights [layer][q, k][128], or nullptr
  int32_t *d_status = nullptr;
  // key-split workspace of the tensor-core attention kernel, per side (source appends and reasoning spans may run on
  // two streams at once): un-normalised outputs, (maximum, row sum) pairs, tickets
  float *split_o[2] = {nullptr, nullptr};
  float2 *split_ml[2] = {nullptr, nullptr};
  int32_t *split_ticket[2] = {nullptr, nullptr};
  // staging for ST_IO_HOST, per side
  __nv_bfloat16 *stage_q[2] = {nullptr, nullptr}, *stage_k[2] = {nullptr, nullptr}, *stage_v[2] = {nullptr, nullptr};
  float *stage_out[2] = {nullptr, nullptr};

  std::vector<EventRec> events;
  uint64_t serial = 0;
  // Events per source append are recorded only once a reasoning-side call has come in on another stream than the
  // appends (an event between two kernels serialises them completely, which would keep consecutive appends from
  // overlapping). Until then one catch-all event, recorded when such a call first needs it, covers all appends so far.
  bool cross_stream = false;
  cudaStream_t last_src_stream = nullptr;
  EventRec catch_all;
  Pending pend[2];

  // kernel timing (benchmarks): event pairs in flight and a pool of spare events
  int timing = 0;                // 0 = off, N = every N-th decode launch (and every tensor-core launch) is bracketed
  int64_t timing_seen = 0;       // decode launches since timing was switched on
  struct TimedLaunch { cudaEvent_t t0, t1; int which; };
  std::vector<TimedLaunch> timed;
  std::vector<cudaEvent_t> spare_events;

  std::vector<int32_t> meta_pos, meta_vis_src, meta_vis_rsn;
  std::string err;
  int64_t launches = 0;
  bool precise_p = false;        // ST_CFG_PRECISE_P: two-term probabilities in the tensor-core attention kernel
  bool poison = false;           // ST_CFG_DEBUG_CHECKS: free pages hold a large finite sentinel instead of zeros
  int fail_countdown = 0;        // test hook: the n-th internal device step from now reports ST_ERR_CUDA
  uint64_t decode_steps = 0;     // decode steps issued since the last full reset: odd ones walk the caches backwards
};

namespace {

int fail(st_ctx *ctx, int code, const std::string &msg) {
  if (ctx) ctx->err = msg;
  return code;
}
#define ST_CUDA(ctx, call)                                                                    \
  do {                                                                                        \
    cudaError_t e__ = (call);                                                                 \
    if (e__ != cudaSuccess) return fail(ctx, ST_ERR_CUDA, std::string(#call) + ": " + cudaGetErrorString(e__)); \
  } while (0)

// Test hook (st_debug_fail_after): counts the device steps of a call (stream wait, page-table update, staging copy,
// append launch, attention launch) and makes the chosen one fail on the host, as a CUDA error would.
int injected_failure(st_ctx *ctx, const char *step) {
  if (ctx->fail_countdown > 0 && --ctx->fail_countdown == 0)
    return fail(ctx, ST_ERR_CUDA, std::string(step) + ": failure injected by st_debug_fail_after");
  return ST_OK;
}

bool config_ok(const st_config *c, std::string *why) {
  auto bad = [&](const char *m) { if (why) *why = m; return false; };
  if (!c) return bad("config is NULL");
  if (c->n_layers < 1) return bad("n_layers must be >= 1");
  if (c->head_dim != st::kHeadDim) return bad("head_dim must be 128");
  if (c->page_size != st::kPageTokens) return bad("page_size must be 64");
  if (c->n_kv_heads < 1 || c->n_q_heads < 1 || c->n_q_heads % c->n_kv_heads) return bad("n_q_heads must be a positive multiple of n_kv_heads");
  if (c->n_q_heads / c->n_kv_heads > st::kMaxGroup) return bad("at most 8 q heads per kv head");
  if (c->max_batch < 1) return bad("max_batch must be >= 1");
  if (c->n_pages_source < 0 || c->n_pages_reason < 0) return bad("page counts must be >= 0");
  if (c->n_pages_source > INT32_MAX || c->n_pages_reason > INT32_MAX) return bad("page counts must fit in 31 bits");
  if (c->max_source_len < 0 || c->max_reason_len < 0) return bad("max lengths must be >= 0");
  if (c->max_tokens_per_call < 1) return bad("max_tokens_per_call must be >= 1");
  if (!(c->rope_theta > 0.0)) return bad("rope_theta must be > 0");
  if (c->softmax_scale < 0.f) return bad("softmax_scale must be >= 0");
  if (c->position_mode < ST_POS_STREAMING || c->position_mode > ST_POS_UNIT_ALIGNED) return bad("unknown position_mode");
  if (c->reserved != 0 || c->reserved2 != 0) return bad("reserved fields must be 0");
  if ((c->q_norm_weight == nullptr) != (c->k_norm_weight == nullptr)) return bad("q_norm_weight and k_norm_weight go together");
  if (c->q_norm_weight && !(c->qk_norm_eps >= 0.f)) return bad("qk_norm_eps must be >= 0");
  return true;
}

int32_t table_stride(int64_t n_pages, int32_t max_len) {
  int64_t by_len = max_len > 0 ? ((int64_t)max_len + 63) / 64 : n_pages;
  int64_t s = std::min<int64_t>(n_pages, by_len);
  return (int32_t)std::max<int64_t>(s, 1);
}

void release_device(st_ctx *ctx) {
  if (ctx->host_only) return;
  cudaSetDevice(ctx->cfg.device);
  cudaDeviceSynchronize();
  for (auto &e : ctx->events)
    if (e.ev) cudaEventDestroy(e.ev);
  if (ctx->catch_all.ev) cudaEventDestroy(ctx->catch_all.ev);
  for (auto &t : ctx->timed) { cudaEventDestroy(t.t0); cudaEventDestroy(t.t1); }
  for (auto &e : ctx->spare_events) cudaEventDestroy(e);
  for (int s = 0; s < 2; ++s) {
    cudaFree(ctx->d_ptab[s]);
    cudaFree(ctx->qhat[s]);
    cudaFree(ctx->stage_q[s]);
    cudaFree(ctx->stage_k[s]);
    cudaFree(ctx->stage_v[s]);
    cudaFree(ctx->stage_out[s]);
    cudaFree(ctx->split_o[s]);
    cudaFree(ctx->split_ml[s]);
    cudaFree(ctx->split_ticket[s]);
  }
  cudaFree(ctx->partial);
  cudaFree(ctx->rope_hi);
  cudaFree(ctx->rope_lo);
  cudaFree(ctx->d_norm);
  cudaFree(ctx->d_status);
  if (ctx->own_pool) cudaFree(ctx->pool_alloc);
}

// ---- argument checks shared by the three attention calls --------------------------------------
int check_common(st_ctx *ctx, int32_t layer, const int32_t *seq_ids, int32_t n_seq) {
  if (!ctx) return ST_ERR_INVALID_ARG;
  if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, ST_ERR_INVALID_ARG, "layer out of range");
  if (n_seq < 1 || !seq_ids) return fail(ctx, ST_ERR_INVALID_ARG, "n_seq must be >= 1 and seq_ids non-NULL");
  if (n_seq > ctx->cfg.max_batch) return fail(ctx, ST_ERR_INVALID_ARG, "more sequences than max_batch");
  std::vector<uint8_t> seen(ctx->cfg.max_batch, 0);
  for (int i = 0; i < n_seq; ++i) {
    if (seq_ids[i] < 0 || seq_ids[i] >= ctx->cfg.max_batch) return fail(ctx, ST_ERR_INVALID_ARG, "sequence id out of range");
    if (seen[seq_ids[i]]) return fail(ctx, ST_ERR_INVALID_ARG, "duplicate sequence id");
    seen[seq_ids[i]] = 1;
  }
  return ST_OK;
}

int check_cu(st_ctx *ctx, const int32_t *cu, int32_t n_seq) {
  if (!cu) return fail(ctx, ST_ERR_INVALID_ARG, "cu_tokens is NULL");
  if (cu[0] != 0) return fail(ctx, ST_ERR_INVALID_ARG, "cu_tokens must start at 0");
  for (int i = 0; i < n_seq; ++i)
    if (cu[i + 1] < cu[i]) return fail(ctx, ST_ERR_INVALID_ARG, "cu_tokens must be non-decreasing");
  if (cu[n_seq] > ctx->cfg.max_tokens_per_call) return fail(ctx, ST_ERR_INVALID_ARG, "more tokens than max_tokens_per_call");
  return ST_OK;
}

// Layer protocol: layer 0 opens a step, later layers must repeat it exactly.
int check_layer_order(st_ctx *ctx, int side, int kind, int32_t layer, const int32_t *seq_ids, const int32_t *cu,
                      int32_t n_seq, uint32_t flags) {
  Pending &pd = ctx->pend[side];
  const uint32_t f = flags & ST_END_OF_UNIT;
  if (layer == 0) {
    if (pd.active) return fail(ctx, ST_ERR_STATE, "previous step has not been issued for all layers");
    return ST_OK;
  }
  if (!pd.active || pd.next_layer != layer) return fail(ctx, ST_ERR_STATE, "layer issued out of order");
  if (pd.kind != kind || (pd.flags & ST_END_OF_UNIT) != f || (int)pd.seq_ids.size() != n_seq ||
      !std::equal(pd.seq_ids.begin(), pd.seq_ids.end(), seq_ids) || !std::equal(pd.cu.begin(), pd.cu.end(), cu))
    return fail(ctx, ST_ERR_STATE, "step arguments differ from those given for layer 0");
  return ST_OK;
}

// Page planning for one side: returns ST_ERR_OOM_PAGES without touching state if the pool or a
// page table cannot hold the new tokens; otherwise allocates and lists the table updates.
int plan_pages(st_ctx *ctx, int which, const int32_t *seq_ids, const int32_t *cu, int32_t n_seq,
               std::vector<st::PageUpdate> *updates) {
  int64_t need_total = 0;
  for (int i = 0; i < n_seq; ++i) {
    const SeqState &sq = ctx->seqs[seq_ids[i]];
    const int64_t new_len = (int64_t)sq.len[which] + (cu[i + 1] - cu[i]);
    const int64_t need = (new_len + 63) / 64;
    if (need > ctx->ptab_stride[which]) return fail(ctx, ST_ERR_OOM_PAGES, which ? "reasoning page table of a sequence is full" : "source page table of a sequence is full");
    need_total += std::max<int64_t>(0, need - (int64_t)sq.pages[which].size());
  }
  if (need_total > (int64_t)ctx->free_pages[which].size())
    return fail(ctx, ST_ERR_OOM_PAGES, which ? "reasoning page pool exhausted" : "source page pool exhausted");
  for (int i = 0; i < n_seq; ++i) {
    SeqState &sq = ctx->seqs[seq_ids[i]];
    const int64_t need = ((int64_t)sq.len[which] + (cu[i + 1] - cu[i]) + 63) / 64;
    while ((int64_t)sq.pages[which].size() < need) {
      const int32_t page = ctx->free_pages[which].back();
      ctx->free_pages[which].pop_back();
      updates->push_back({seq_ids[i] * 2 + which, (int32_t)sq.pages[which].size(), page});
      sq.pages[which].push_back(page);
    }
  }
  return ST_OK;
}

// Undo plan_pages: the pages listed in `updates` (in allocation order) go back to the free list, newest first,
// so that the free list is exactly what it was.
void unplan_pages(st_ctx *ctx, const std::vector<st::PageUpdate> &updates) {
  for (auto it = updates.rbegin(); it != updates.rend(); ++it) {
    const int which = it->slot_which & 1, slot = it->slot_which >> 1;
    ctx->seqs[slot].pages[which].pop_back();
    ctx->free_pages[which].push_back(it->page);
  }
}

int push_page_updates(st_ctx *ctx, const std::vector<st::PageUpdate> &updates, cudaStream_t stream) {
  if (int rc = injected_failure(ctx, "page-table update")) return rc;
  if (ctx->host_only) return ST_OK;
  for (size_t off = 0; off < updates.size(); off += st::kMaxPageUpdates) {
    st::PageUpdateParams pp;
    pp.ptab[0] = ctx->d_ptab[0];
    pp.ptab[1] = ctx->d_ptab[1];
    pp.stride[0] = ctx->ptab_stride[0];
    pp.stride[1] = ctx->ptab_stride[1];
    pp.n = (int32_t)std::min<size_t>(st::kMaxPageUpdates, updates.size() - off);
    memcpy(pp.upd, updates.data() + off, sizeof(st::PageUpdate) * pp.n);
    ST_CUDA(ctx, st::launch_page_update(pp, stream));
    ++ctx->launches;
  }
  return ST_OK;
}

// Resolve visible_units to a visible source length per sequence (Algorithm 1's slice I'_cache).
int resolve_visibility(st_ctx *ctx, const int32_t *seq_ids, int32_t n_seq, const int32_t *visible_units,
                       std::vector<int32_t> *vis_tokens, uint64_t *wait_serial) {
  vis_tokens->resize(n_seq);
  *wait_serial = 0;
  for (int i = 0; i < n_seq; ++i) {
    const SeqState &sq = ctx->seqs[seq_ids[i]];
    int32_t k = visible_units ? visible_units[i] : ST_VIS_DEFAULT;
    if (k == ST_VIS_ALL) {
      (*vis_tokens)[i] = sq.len[0];
      *wait_serial = std::max(*wait_serial, sq.last_src_serial);
      continue;
    }
    if (k == ST_VIS_DEFAULT) k = sq.n_eot + 1;
    if (k < 0) return fail(ctx, ST_ERR_INVALID_ARG, "visible_units must be >= 0, ST_VIS_DEFAULT or ST_VIS_ALL");
    if (k > sq.n_eos) return fail(ctx, ST_ERR_NOT_READY, "the requested source unit has not been appended yet");
    if (k == 0) {
      (*vis_tokens)[i] = 0;
    } else {
      (*vis_tokens)[i] = sq.unit_end[k - 1];
      *wait_serial = std::max(*wait_serial, sq.unit_serial[k - 1]);
    }
  }
  return ST_OK;
}

// Position ids of the new reasoning tokens of a call (Section 3.2): offset between a token's position id and its index
// in the reasoning cache, per listed sequence. Zero with the streaming position encoding.
int resolve_positions(st_ctx *ctx, const int32_t *seq_ids, int32_t n_seq, const int32_t *visible_units,
                      std::vector<int32_t> *rope_off, std::vector<uint8_t> *is_final) {
  rope_off->assign(n_seq, 0);
  is_final->assign(n_seq, 0);
  for (int i = 0; i < n_seq; ++i) {
    const SeqState &sq = ctx->seqs[seq_ids[i]];
    (*is_final)[i] = visible_units && visible_units[i] == ST_VIS_ALL;
    if (ctx->cfg.position_mode == ST_POS_CONCATENATED) {
      (*rope_off)[i] = sq.concat_off >= 0 ? sq.concat_off : sq.len[0];            // T + t
    } else if (ctx->cfg.position_mode == ST_POS_UNIT_ALIGNED) {
      int32_t base;
      if ((*is_final)[i]) {
        base = sq.final_base >= 0 ? sq.final_base : sq.len[0];                      // S + i
      } else {
        if (sq.n_eot > sq.n_eos) return fail(ctx, ST_ERR_NOT_READY, "the source unit this reasoning unit aligns to has not been appended yet");
        base = sq.n_eot > 0 ? sq.unit_end[sq.n_eot - 1] : 0;                        // P_{u-1} + i for unit u = N_EOT + 1
      }
      (*rope_off)[i] = base + sq.unit_tokens - sq.len[1];
    }
  }
  return ST_OK;
}

// Make `stream` wait for the source append with the given serial if it ran on another stream.
int wait_for_append(st_ctx *ctx, uint64_t serial, cudaStream_t stream) {
  if (int rc = injected_failure(ctx, "stream wait")) return rc;
  if (ctx->host_only || serial == 0) return ST_OK;
  EventRec &rec = ctx->events[serial % kEventRing];
  if (rec.serial == serial) {
    if (rec.stream != stream) ST_CUDA(ctx, cudaStreamWaitEvent(stream, rec.ev, 0));
    return ST_OK;
  }
  if (rec.serial > serial) {
    // the event slot was recycled by a newer append: source appends are stream-ordered, so the
    // newest recorded event of the ring covers the one we need
    uint64_t best = 0;
    EventRec *newest = nullptr;
    for (auto &e : ctx->events)
      if (e.serial > best) { best = e.serial; newest = &e; }
    if (newest && newest->stream != stream) ST_CUDA(ctx, cudaStreamWaitEvent(stream, newest->ev, 0));
    return ST_OK;
  }
  // no event was recorded for that append (all calls came on one stream so far)
  if (ctx->last_src_stream == stream) return ST_OK;   // same stream: stream order is enough
  ctx->cross_stream = true;                           // from now on every append records its event
  if (ctx->catch_all.serial < serial) {
    if (!ctx->catch_all.ev) ST_CUDA(ctx, cudaEventCreateWithFlags(&ctx->catch_all.ev, cudaEventDisableTiming));
    ST_CUDA(ctx, cudaEventRecord(ctx->catch_all.ev, ctx->last_src_stream));
    ctx->catch_all.stream = ctx->last_src_stream;
    ctx->catch_all.serial = ctx->serial;              // every append submitted so far
  }
  if (ctx->catch_all.stream != stream) ST_CUDA(ctx, cudaStreamWaitEvent(stream, ctx->catch_all.ev, 0));
  return ST_OK;
}

// After the last layer of a source append: the event that later reasoning-side calls on another stream wait for.
int record_append_event(st_ctx *ctx, cudaStream_t stream) {
  if (ctx->host_only) return ST_OK;
  EventRec &rec = ctx->events[(ctx->serial + 1) % kEventRing];
  if (ctx->cross_stream) {
    if (!rec.ev) ST_CUDA(ctx, cudaEventCreateWithFlags(&rec.ev, cudaEventDisableTiming));
    ST_CUDA(ctx, cudaEventRecord(rec.ev, stream));
    rec.stream = stream;
    rec.serial = ctx->serial + 1;
  } else {
    rec.serial = 0;   // none recorded: wait_for_append falls back to the catch-all event
  }
  ctx->last_src_stream = stream;
  return ST_OK;
}

struct IoPtrs {
  const __nv_bfloat16 *q, *k, *v;
  float *out;
  bool in_place = false;   // ST_IO_HOST served by the kernels themselves (no staging copies)
};

// Calls whose q + k + v stay below this size are not staged: the kernels read page-locked host memory in place.
constexpr size_t kInPlaceHostIoBytes = 1u << 20;

// Device-side alias of a page-locked (registered or cudaHostAlloc'ed) host pointer; nullptr for pageable memory.
const void *device_alias_of_host(const void *p) {
  cudaPointerAttributes a;
  if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
    cudaGetLastError();   // not an error of this context: the pointer is simply unknown to the driver
    return nullptr;
  }
  return a.type == cudaMemoryTypeHost ? a.devicePointer : nullptr;
}

// ST_IO_HOST. Large calls (chunk prefill): the packed inputs are copied to device staging on the stream and the rows
// are copied back after the kernels. Small calls (a decode step moves a few hundred KB): four copy-engine
// transfers of that size cost more than the attention itself, so when all buffers are page-locked the append
// kernel reads q/k/v, and the attention kernels write the rows, directly in host memory -- each byte crosses the
// bus once, inside the kernels of the call.
// `may_run_in_place`: small calls on page-locked buffers may be served by the kernels themselves (decode steps only:
// the tensor-core attention kernel writes its rows with bulk stores from shared memory, which are kept to device memory).
int stage_inputs(st_ctx *ctx, int side, uint32_t flags, int32_t total, const void *q, const void *k, const void *v,
                 void *out, cudaStream_t stream, IoPtrs *io, bool may_run_in_place) {
  io->q = (const __nv_bfloat16 *)q;
  io->k = (const __nv_bfloat16 *)k;
  io->v = (const __nv_bfloat16 *)v;
  io->out = (float *)out;
  if (int rc = injected_failure(ctx, "staging copy")) return rc;
  if (!(flags & ST_IO_HOST) || ctx->host_only || total == 0) return ST_OK;
  const size_t qb = (size_t)total * ctx->cfg.n_q_heads * 256, kb = (size_t)total * ctx->cfg.n_kv_heads * 256;
  if (may_run_in_place && qb + 2 * kb <= kInPlaceHostIoBytes) {
    const void *dq = device_alias_of_host(q), *dk = device_alias_of_host(k), *dv = device_alias_of_host(v);
    const void *dout = out ? device_alias_of_host(out) : nullptr;
    if (dq && dk && dv && (dout || !out)) {
      io->q = (const __nv_bfloat16 *)dq;
      io->k = (const __nv_bfloat16 *)dk;
      io->v = (const __nv_bfloat16 *)dv;
      io->out = (float *)const_cast<void *>(dout);
      io->in_place = true;
      return ST_OK;
    }
  }
  if (!ctx->stage_q[side]) {
    // staging buffers exist only for contexts that really stage host calls: allocated on the first such call of a side
    const size_t T = ctx->cfg.max_tokens_per_call;
    ST_CUDA(ctx, cudaMalloc(&ctx->stage_q[side], T * ctx->cfg.n_q_heads * 256));
    ST_CUDA(ctx, cudaMalloc(&ctx->stage_k[side], T * ctx->cfg.n_kv_heads * 256));
    ST_CUDA(ctx, cudaMalloc(&ctx->stage_v[side], T * ctx->cfg.n_kv_heads * 256));
    ST_CUDA(ctx, cudaMalloc(&ctx->stage_out[side], T * ctx->cfg.n_q_heads * 512));
  }
  ST_CUDA(ctx, cudaMemcpyAsync(ctx->stage_q[side], q, qb, cudaMemcpyHostToDevice, stream));
  ST_CUDA(ctx, cudaMemcpyAsync(ctx->stage_k[side], k, kb, cudaMemcpyHostToDevice, stream));
  ST_CUDA(ctx, cudaMemcpyAsync(ctx->stage_v[side], v, kb, cudaMemcpyHostToDevice, stream));
  io->q = ctx->stage_q[side];
  io->k = ctx->stage_k[side];
  io->v = ctx->stage_v[side];
  io->out = out ? ctx->stage_out[side] : nullptr;
  return ST_OK;
}
int unstage_output(st_ctx *ctx, int side, uint32_t flags, int32_t total, void *out, cudaStream_t stream, const IoPtrs &io) {
  if (!(flags & ST_IO_HOST) || ctx->host_only || total == 0 || !out || io.in_place) return ST_OK;
  ST_CUDA(ctx, cudaMemcpyAsync(out, ctx->stage_out[side], (size_t)total * ctx->cfg.n_q_heads * 512,
                               cudaMemcpyDeviceToHost, stream));
  return ST_OK;
}

// Launch the append kernel (K and V into the cache of side `which`, rotated q into scratch).
// Rows of a call per listed sequence: first packed row and row count.
struct RowRanges {
  std::vector<int32_t> begin, count;
  static RowRanges from_cu(const int32_t *cu, int32_t n_seq) {
    RowRanges r;
    r.begin.assign(cu, cu + n_seq);
    r.count.resize(n_seq);
    for (int b = 0; b < n_seq; ++b) r.count[b] = cu[b + 1] - cu[b];
    return r;
  }
};

int run_append(st_ctx *ctx, int which, int32_t layer, const int32_t *seq_ids, const RowRanges &rows, int32_t n_seq,
               const std::vector<int32_t> &rope_off, const IoPtrs &io, bool want_q, cudaStream_t stream) {
  if (int rc = injected_failure(ctx, "append launch")) return rc;
  if (ctx->host_only) return ST_OK;
  for (int s0 = 0; s0 < n_seq; s0 += st::kMaxSeqPerLaunch) {
    const int ns = std::min<int>(st::kMaxSeqPerLaunch, n_seq - s0);
    st::AppendParams ap;
    ap.q = io.q;
    ap.k = io.k;
    ap.v = io.v;
    ap.qhat = want_q ? ctx->qhat[which] : nullptr;
    ap.pool = ctx->pool[which] + (size_t)layer * ctx->layer_stride[which];
    ap.ptab = ctx->d_ptab[which];
    ap.ptab_stride = ctx->ptab_stride[which];
    ap.n_pages = (int32_t)(which ? ctx->cfg.n_pages_reason : ctx->cfg.n_pages_source);
    ap.status = ctx->d_status;
    ap.norm_q = ctx->d_norm ? ctx->d_norm + (size_t)layer * 256 : nullptr;
    ap.norm_k = ctx->d_norm ? ctx->d_norm + (size_t)layer * 256 + 128 : nullptr;
    ap.norm_eps = ctx->cfg.qk_norm_eps;
    ap.n_seq = ns;
    ap.n_q_heads = ctx->cfg.n_q_heads;
    ap.n_kv_heads = ctx->cfg.n_kv_heads;
    memcpy(ap.inv_freq, ctx->inv_freq, sizeof(ap.inv_freq));
    int blocks = 0;
    for (int i = 0; i < ns; ++i) {
      const int b = s0 + i;
      const int32_t pos0 = ctx->seqs[seq_ids[b]].len[which], n = rows.count[b];
      ap.seq[i] = {seq_ids[b], pos0, n, rows.begin[b], blocks, which == 1 ? rope_off[b] : 0};
      if (n > 0) blocks += ((pos0 + n - 1) >> 3) - (pos0 >> 3) + 1;
    }
    if (blocks == 0) continue;
    ST_CUDA(ctx, st::launch_rope_append(ap, blocks, stream));
    ++ctx->launches;
  }
  return ST_OK;
}

void fill_attn_common(st_ctx *ctx, int side, int32_t layer, float *out, st::AttnParams *p) {
  // side 0 (chunk prefill): range A empty, range B = source cache.
  // side 1 (decode / extend): range A = source cache prefix, range B = reasoning cache.
  p->pool_a = ctx->pool[0] + (size_t)layer * ctx->layer_stride[0];
  p->ptab_a = ctx->d_ptab[0];
  p->ptab_stride_a = ctx->ptab_stride[0];
  const int b = side == 0 ? 0 : 1;
  p->pool_b = ctx->pool[b] + (size_t)layer * ctx->layer_stride[b];
  p->ptab_b = ctx->d_ptab[b];
  p->ptab_stride_b = ctx->ptab_stride[b];
  p->n_pages_a = (int32_t)ctx->cfg.n_pages_source;
  p->n_pages_b = (int32_t)(b ? ctx->cfg.n_pages_reason : ctx->cfg.n_pages_source);
  p->qhat = ctx->qhat[side];
  p->q_raw = p->k_raw = p->v_raw = nullptr;
  p->rope_hi = p->rope_lo = nullptr;
  p->out = out;
  p->partial = ctx->partial;
  p->status = ctx->d_status;
  p->n_q_heads = ctx->cfg.n_q_heads;
  p->n_kv_heads = ctx->cfg.n_kv_heads;
  p->group = ctx->group;
  p->scale_log2 = ctx->scale_log2;
  memcpy(p->inv_freq, ctx->inv_freq, sizeof(p->inv_freq));
  p->norm_q = ctx->d_norm ? ctx->d_norm + (size_t)layer * 256 : nullptr;
  p->norm_k = ctx->d_norm ? ctx->d_norm + (size_t)layer * 256 + 128 : nullptr;
  p->norm_eps = ctx->cfg.qk_norm_eps;
  p->total_work = p->work_per_cta = p->n_cta = 0;
  p->reverse = 0;
  p->split_o = ctx->split_o[side];
  p->split_ml = ctx->split_ml[side];
  p->split_ticket = ctx->split_ticket[side];
  p->n_split = 0;
}

// Attention for the rows of a call. kind: 0 chunk prefill, 1 decode, 2 extend.
// `fused`: non-null for a decode step whose append runs inside the decode kernel (the call's un-rotated q/k/v).
// Launches the attention kernels of one call for a list of work entries (one per sequence for the streaming calls,
// one per (sequence, reasoning unit) for the packed forward). kind: 0 chunk prefill, 1 decode, 2 spans.
// `fused`: a decode step whose append runs inside the decode kernel (the call's un-rotated q/k/v).
int launch_attention_entries(st_ctx *ctx, int kind, int32_t layer, const std::vector<st::AttnSeq> &entries_in, int total_rows,
                             float *out, uint32_t flags, cudaStream_t stream, const IoPtrs &io, bool fused) {
  const int side = kind == 0 ? 0 : 1;
  // The tensor-core kernel's CTAs are handed out in entry order and an entry's CTAs all walk about the same number of
  // keys: longest entries first, so that the last, partly filled wave of a ragged call holds the short ones (the
  // decode kernel cuts its tile list into equal slices and needs no such order).
  std::vector<st::AttnSeq> entries(entries_in);
  if (kind != 1)
    std::stable_sort(entries.begin(), entries.end(), [](const st::AttnSeq &a, const st::AttnSeq &b) {
      return (int64_t)a.a_len + a.b_base + a.n_rows > (int64_t)b.a_len + b.b_base + b.n_rows;
    });
  for (size_t s0 = 0; s0 < entries.size(); s0 += st::kMaxSeqPerLaunch) {
    const int ns = (int)std::min<size_t>(st::kMaxSeqPerLaunch, entries.size() - s0);
    st::AttnParams ap;
    fill_attn_common(ctx, side, layer, out, &ap);
    if (fused) {
      ap.q_raw = io.q;
      ap.k_raw = io.k;
      ap.v_raw = io.v;
      ap.rope_hi = ctx->rope_hi;
      ap.rope_lo = ctx->rope_lo;
    } else if (kind != 1 && !(flags & ST_REFERENCE_KERNELS)) {
      ap.q_raw = io.q;   // the tensor-core kernel rotates its query rows itself
    }
    std::copy(entries.begin() + s0, entries.begin() + s0 + ns, ap.seq);
    ap.n_seq = ns;
    int nl = 0;
    cudaEvent_t t0 = nullptr, t1 = nullptr;
    if (ctx->timing && !(flags & ST_REFERENCE_KERNELS) && (kind != 1 || ctx->timing_seen++ % ctx->timing == 0)) {
      for (cudaEvent_t *t : {&t0, &t1}) {
        if (ctx->spare_events.empty()) {
          ST_CUDA(ctx, cudaEventCreate(t));
        } else {
          *t = ctx->spare_events.back();
          ctx->spare_events.pop_back();
        }
      }
      ctx->timed.push_back({t0, t1, kind == 1 ? 0 : 1});
    }
    if (flags & ST_REFERENCE_KERNELS) {
      ST_CUDA(ctx, st::launch_attn_reference(ap, total_rows, stream));
      nl = 1;
    } else if (kind == 1) {
      ap.reverse = ctx->pend[1].reverse ? 1 : 0;
      ST_CUDA(ctx, st::launch_decode(ap, ctx->num_sms, stream, &nl, t0, t1));
    } else {
      ST_CUDA(ctx, st::launch_attn_tc(ap, ctx->precise_p, ctx->num_sms, stream, &nl, t0, t1));
    }
    ctx->launches += nl;
  }
  return ST_OK;
}

// Attention for the rows of a streaming call: one entry per listed sequence with rows.
int run_attention(st_ctx *ctx, int kind, int32_t layer, const int32_t *seq_ids, const int32_t *cu, int32_t n_seq,
                  const std::vector<int32_t> &vis_tokens, const std::vector<int32_t> &rope_off, float *out, uint32_t flags,
                  cudaStream_t stream, const IoPtrs &io, bool fused) {
  if (int rc = injected_failure(ctx, "attention launch")) return rc;
  if (ctx->host_only || !out) return ST_OK;
  const int side = kind == 0 ? 0 : 1;
  if (cu[n_seq] == 0) return ST_OK;
  std::vector<st::AttnSeq> entries;
  for (int b = 0; b < n_seq; ++b) {
    const int32_t n = cu[b + 1] - cu[b];
    if (n == 0) continue;
    st::AttnSeq as;
    as.slot = seq_ids[b];
    as.a_len = kind == 0 ? 0 : vis_tokens[b];
    as.b_base = ctx->seqs[seq_ids[b]].len[side];
    as.n_rows = n;
    as.q_begin = cu[b];
    as.work_begin = 0;
    as.rope_off = kind == 0 ? 0 : rope_off[b];
    entries.push_back(as);
  }
  return launch_attention_entries(ctx, kind, layer, entries, cu[n_seq], out, flags, stream, io, fused);
}

void record_meta(st_ctx *ctx, int kind, const int32_t *seq_ids, const int32_t *cu, int32_t n_seq,
                 const std::vector<int32_t> &vis_tokens, const std::vector<int32_t> &rope_off) {
  const int side = kind == 0 ? 0 : 1;
  const int total = cu[n_seq];
  ctx->meta_pos.assign(total, 0);
  ctx->meta_vis_src.assign(total, 0);
  ctx->meta_vis_rsn.assign(total, 0);
  for (int b = 0; b < n_seq; ++b) {
    const int32_t base = ctx->seqs[seq_ids[b]].len[side];
    for (int r = cu[b]; r < cu[b + 1]; ++r) {
      const int32_t pos = base + (r - cu[b]);
      ctx->meta_pos[r] = pos + (kind == 0 ? 0 : rope_off[b]);
      if (kind == 0) {
        ctx->meta_vis_src[r] = pos + 1;
        ctx->meta_vis_rsn[r] = 0;
      } else {
        ctx->meta_vis_src[r] = vis_tokens[b];
        ctx->meta_vis_rsn[r] = pos + 1;
      }
    }
  }
}

// The body shared by st_append_source_chunk (kind 0), st_reason_decode (1) and st_reason_extend (2).
int attention_call(st_ctx *ctx, int kind, int32_t layer, const int32_t *seq_ids, const int32_t *cu, int32_t n_seq,
                   const int32_t *visible_units, const void *q, const void *k, const void *v, void *out,
                   uint32_t flags, void *stream_v) {
  cudaStream_t stream = (cudaStream_t)stream_v;
  const int side = kind == 0 ? 0 : 1;
  int rc = check_common(ctx, layer, seq_ids, n_seq);
  if (rc) return rc;
  if ((rc = check_cu(ctx, cu, n_seq))) return rc;
  if (flags & ~(ST_END_OF_UNIT | ST_REFERENCE_KERNELS | ST_IO_HOST)) return fail(ctx, ST_ERR_INVALID_ARG, "unknown flag");
  const int32_t total = cu[n_seq];
  if (total > 0 && (!q || !k || !v) && !ctx->host_only) return fail(ctx, ST_ERR_INVALID_ARG, "q, k and v must be non-NULL");
  if ((rc = check_layer_order(ctx, side, kind, layer, seq_ids, cu, n_seq, flags))) return rc;

  Pending &pd = ctx->pend[side];
  std::vector<st::PageUpdate> updates;
  if (layer == 0) {
    std::vector<int32_t> vis;
    uint64_t wait_serial = 0;
    std::vector<int32_t> off(n_seq, 0);
    std::vector<uint8_t> fin(n_seq, 0);
    if (kind != 0) {
      if ((rc = resolve_visibility(ctx, seq_ids, n_seq, visible_units, &vis, &wait_serial))) return rc;
      if ((rc = resolve_positions(ctx, seq_ids, n_seq, visible_units, &off, &fin))) return rc;
    }
    if ((rc = plan_pages(ctx, side, seq_ids, cu, n_seq, &updates))) return rc;
    pd.active = true;
    pd.kind = kind;
    pd.next_layer = 0;
    pd.flags = flags;
    pd.seq_ids.assign(seq_ids, seq_ids + n_seq);
    pd.cu.assign(cu, cu + n_seq + 1);
    pd.vis_tokens = vis;
    pd.rope_off = off;
    pd.is_final = fin;
    pd.wait_serial = wait_serial;
    // consecutive decode steps walk the caches in opposite directions: a step starts on what the last one left in L2
    pd.reverse = kind == 1 && (ctx->decode_steps++ & 1u) != 0;
    record_meta(ctx, kind, seq_ids, cu, n_seq, pd.vis_tokens, pd.rope_off);
  }

  // Device steps. If one of them fails, the host-side plan of this call is taken back (pages to the free list, the
  // step no longer pending), so that the context is what it was before the call; work already queued stays queued.
  uint64_t serial = 0;
  auto device_steps = [&]() -> int {
    int r;
    if (!ctx->host_only) ST_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    if (kind != 0 && (r = wait_for_append(ctx, pd.wait_serial, stream))) return r;
    if ((r = push_page_updates(ctx, updates, stream))) return r;
    IoPtrs io;
    if ((r = stage_inputs(ctx, side, flags, total, q, k, v, out, stream, &io, kind == 1))) return r;
    // A decode step's append (one token per sequence) runs inside the decode kernel: the step is then two kernels
    // instead of three. Cache-only calls and the cross-check kernels keep the separate append.
    const bool fuse_append = kind == 1 && io.out != nullptr && !(flags & ST_REFERENCE_KERNELS) && !ctx->host_only;
    // Rotated queries go to scratch only for the kernels that read them there: the simple cross-check kernels and a
    // decode step whose append is not fused, and the tensor-core kernel's two-term variant (which wants the fp64
    // rotation). The one-term tensor-core kernel rotates its own.
    const bool want_qhat = io.out != nullptr && ((flags & ST_REFERENCE_KERNELS) || kind == 1 || ctx->precise_p);
    if (!fuse_append && (r = run_append(ctx, side, layer, seq_ids, RowRanges::from_cu(cu, n_seq), n_seq, pd.rope_off, io, want_qhat, stream))) return r;
    if ((r = run_attention(ctx, kind, layer, seq_ids, cu, n_seq, pd.vis_tokens, pd.rope_off, io.out, flags, stream, io, fuse_append))) return r;
    if ((r = unstage_output(ctx, side, flags, total, out, stream, io))) return r;
    if (layer == ctx->cfg.n_layers - 1 && kind == 0 && (r = record_append_event(ctx, stream))) return r;
    return ST_OK;
  };
  if ((rc = device_steps())) {
    if (layer == 0) {
      unplan_pages(ctx, updates);
      pd.active = false;
    }
    return rc;
  }

  if (layer == ctx->cfg.n_layers - 1) {
    // commit the step
    if (kind == 0) serial = ++ctx->serial;
    for (int b = 0; b < n_seq; ++b) {
      SeqState &sq = ctx->seqs[seq_ids[b]];
      sq.len[side] += cu[b + 1] - cu[b];
      if (kind == 0) {
        sq.last_src_serial = serial;
        if (flags & ST_END_OF_UNIT) {
          ++sq.n_eos;
          sq.unit_end.push_back(sq.len[0]);
          sq.unit_serial.push_back(serial);
        }
      } else {
        // position-id bookkeeping of the other modes (the streaming encoding needs none)
        if (ctx->cfg.position_mode == ST_POS_CONCATENATED && sq.concat_off < 0 && cu[b + 1] > cu[b]) sq.concat_off = pd.rope_off[b];
        if (pd.is_final[b] && sq.final_base < 0) sq.final_base = sq.len[0];
        sq.unit_tokens += cu[b + 1] - cu[b];
        if (flags & ST_END_OF_UNIT) {
          ++sq.n_eot;
          sq.unit_tokens = 0;
        }
      }
    }
    pd.active = false;
  } else {
    pd.next_layer = layer + 1;
  }
  return ST_OK;
}

// st_forward_packed: one pass over the training layout [source ; reasoning] of every listed sequence.
int forward_packed(st_ctx *ctx, int32_t layer, const int32_t *seq_ids, int32_t n_seq, const int32_t *n_units,
                   const int32_t *src_unit_len, const int32_t *rsn_unit_len, const int32_t *final_len, int32_t lag_units,
                   const void *q, const void *k, const void *v, void *out, uint32_t flags, cudaStream_t stream) {
  int rc = check_common(ctx, layer, seq_ids, n_seq);
  if (rc) return rc;
  if (flags & ~(ST_REFERENCE_KERNELS | ST_IO_HOST)) return fail(ctx, ST_ERR_INVALID_ARG, "unknown flag");
  if (!n_units || !final_len || lag_units < 0) return fail(ctx, ST_ERR_INVALID_ARG, "n_units and final_len must be non-NULL, lag_units >= 0");
  if (ctx->cfg.position_mode == ST_POS_UNIT_ALIGNED)
    return fail(ctx, ST_ERR_INVALID_ARG, "the packed forward supports the streaming and the concatenated position ids");
  // per sequence: S, R, first row in the packed tensors; the schedule signature for the layer protocol
  std::vector<int32_t> S(n_seq), R(n_seq), row0(n_seq), unit0(n_seq), cu_src(n_seq + 1, 0), cu_rsn(n_seq + 1, 0), sig;
  int64_t total = 0, units = 0;
  for (int b = 0; b < n_seq; ++b) {
    if (n_units[b] < 0 || final_len[b] < 0) return fail(ctx, ST_ERR_INVALID_ARG, "unit counts and final lengths must be >= 0");
    if (n_units[b] > 0 && (!src_unit_len || !rsn_unit_len)) return fail(ctx, ST_ERR_INVALID_ARG, "unit length arrays are NULL");
    unit0[b] = (int32_t)units;
    int64_t s_len = 0, r_len = final_len[b];
    for (int u = 0; u < n_units[b]; ++u) {
      const int32_t n = src_unit_len[units + u], m = rsn_unit_len[units + u];
      if (n < 0 || m < 0) return fail(ctx, ST_ERR_INVALID_ARG, "unit lengths must be >= 0");
      s_len += n;
      r_len += m;
      sig.push_back(n);
      sig.push_back(m);
    }
    sig.push_back(final_len[b]);
    units += n_units[b];
    if (total + s_len + r_len > ctx->cfg.max_tokens_per_call) return fail(ctx, ST_ERR_INVALID_ARG, "more tokens than max_tokens_per_call");
    S[b] = (int32_t)s_len;
    R[b] = (int32_t)r_len;
    row0[b] = (int32_t)total;
    total += s_len + r_len;
    cu_src[b + 1] = cu_src[b] + S[b];
    cu_rsn[b + 1] = cu_rsn[b] + R[b];
  }
  sig.push_back(lag_units);
  if (total > 0 && (!q || !k || !v) && !ctx->host_only) return fail(ctx, ST_ERR_INVALID_ARG, "q, k and v must be non-NULL");

  // layer protocol: the step occupies both sides
  Pending &pd = ctx->pend[0];
  if (layer == 0) {
    if (pd.active || ctx->pend[1].active) return fail(ctx, ST_ERR_STATE, "previous step has not been issued for all layers");
    for (int b = 0; b < n_seq; ++b) {
      const SeqState &sq = ctx->seqs[seq_ids[b]];
      if (sq.len[0] || sq.len[1] || sq.n_eos || sq.n_eot) return fail(ctx, ST_ERR_STATE, "the packed forward needs empty sequences (st_reset them first)");
    }
  } else {
    if (!pd.active || pd.kind != 3 || pd.next_layer != layer) return fail(ctx, ST_ERR_STATE, "layer issued out of order");
    if ((int)pd.seq_ids.size() != n_seq || !std::equal(pd.seq_ids.begin(), pd.seq_ids.end(), seq_ids) || pd.cu != sig)
      return fail(ctx, ST_ERR_STATE, "step arguments differ from those given for layer 0");
  }
  std::vector<st::PageUpdate> updates;
  if (layer == 0) {
    if ((rc = plan_pages(ctx, 0, seq_ids, cu_src.data(), n_seq, &updates))) return rc;
    if ((rc = plan_pages(ctx, 1, seq_ids, cu_rsn.data(), n_seq, &updates))) {
      unplan_pages(ctx, updates);
      return rc;
    }
    pd.active = ctx->pend[1].active = true;
    pd.kind = 3;
    pd.next_layer = 0;
    pd.flags = flags;
    pd.seq_ids.assign(seq_ids, seq_ids + n_seq);
    pd.cu = sig;
  }

  // work entries of the reasoning rows: one per (sequence, reasoning unit with tokens), one for the final-depth tokens
  const bool concat = ctx->cfg.position_mode == ST_POS_CONCATENATED;
  std::vector<st::AttnSeq> src_entries, rsn_entries;
  std::vector<int32_t> rsn_off(n_seq, 0);
  ctx->meta_pos.assign((size_t)total, 0);
  ctx->meta_vis_src.assign((size_t)total, 0);
  ctx->meta_vis_rsn.assign((size_t)total, 0);
  for (int b = 0; b < n_seq; ++b) {
    rsn_off[b] = concat ? S[b] : 0;
    if (S[b] > 0) src_entries.push_back({seq_ids[b], 0, 0, S[b], row0[b], 0, 0});
    for (int j = 0; j < S[b]; ++j) {
      ctx->meta_pos[row0[b] + j] = j;
      ctx->meta_vis_src[row0[b] + j] = j + 1;
    }
    std::vector<int32_t> prefix(n_units[b] + 1, 0);
    for (int u = 0; u < n_units[b]; ++u) prefix[u + 1] = prefix[u] + src_unit_len[unit0[b] + u];
    int32_t r = 0;
    for (int u = 0; u <= n_units[b]; ++u) {
      const bool fin = u == n_units[b];
      const int32_t m = fin ? final_len[b] : rsn_unit_len[unit0[b] + u];
      const int32_t vis = fin ? S[b] : prefix[std::min<int64_t>((int64_t)u + 1 + lag_units, n_units[b])];
      if (m > 0) rsn_entries.push_back({seq_ids[b], vis, r, m, row0[b] + S[b] + r, 0, rsn_off[b]});
      for (int i = 0; i < m; ++i) {
        const int32_t row = row0[b] + S[b] + r + i;
        ctx->meta_pos[row] = r + i + rsn_off[b];
        ctx->meta_vis_src[row] = vis;
        ctx->meta_vis_rsn[row] = r + i + 1;
      }
      r += m;
    }
  }

  auto device_steps = [&]() -> int {
    int r;
    if (!ctx->host_only) ST_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    if ((r = push_page_updates(ctx, updates, stream))) return r;
    IoPtrs io;
    if ((r = stage_inputs(ctx, 0, flags, (int32_t)total, q, k, v, out, stream, &io, false))) return r;
    const bool want_qhat = io.out != nullptr && ((flags & ST_REFERENCE_KERNELS) || ctx->precise_p);
    RowRanges src_rows, rsn_rows;
    for (int b = 0; b < n_seq; ++b) {
      src_rows.begin.push_back(row0[b]);
      src_rows.count.push_back(S[b]);
      rsn_rows.begin.push_back(row0[b] + S[b]);
      rsn_rows.count.push_back(R[b]);
    }
    if ((r = run_append(ctx, 0, layer, seq_ids, src_rows, n_seq, rsn_off, io, want_qhat, stream))) return r;
    if ((r = run_append(ctx, 1, layer, seq_ids, rsn_rows, n_seq, rsn_off, io, want_qhat, stream))) return r;
    if ((r = injected_failure(ctx, "attention launch"))) return r;
    if (!ctx->host_only && io.out) {
      if ((r = launch_attention_entries(ctx, 0, layer, src_entries, (int)total, io.out, flags, stream, io, false))) return r;
      if ((r = launch_attention_entries(ctx, 2, layer, rsn_entries, (int)total, io.out, flags, stream, io, false))) return r;
    }
    if ((r = unstage_output(ctx, 0, flags, (int32_t)total, out, stream, io))) return r;
    if (layer == ctx->cfg.n_layers - 1 && (r = record_append_event(ctx, stream))) return r;
    return ST_OK;
  };
  if ((rc = device_steps())) {
    if (layer == 0) {
      unplan_pages(ctx, updates);
      pd.active = ctx->pend[1].active = false;
    }
    return rc;
  }
  if (layer == ctx->cfg.n_layers - 1) {
    const uint64_t serial = ++ctx->serial;
    for (int b = 0; b < n_seq; ++b) {
      SeqState &sq = ctx->seqs[seq_ids[b]];
      sq.len[0] = S[b];
      sq.len[1] = R[b];
      sq.last_src_serial = serial;
      int32_t p = 0;
      for (int u = 0; u < n_units[b]; ++u) {
        p += src_unit_len[unit0[b] + u];
        sq.unit_end.push_back(p);
        sq.unit_serial.push_back(serial);
      }
      sq.n_eos = sq.n_eot = n_units[b];
      if (concat && R[b] > 0) sq.concat_off = S[b];
    }
    pd.active = ctx->pend[1].active = false;
  } else {
    pd.next_layer = layer + 1;
  }
  return ST_OK;
}

int schedule_sizes(const int32_t *n, const int32_t *m, int32_t n_units, int32_t final_len, int64_t *S, int64_t *R) {
  if (n_units < 0 || final_len < 0 || (n_units > 0 && (!n || !m))) return ST_ERR_INVALID_ARG;
  *S = 0;
  *R = final_len;
  for (int u = 0; u < n_units; ++u) {
    if (n[u] < 0 || m[u] < 0) return ST_ERR_INVALID_ARG;
    *S += n[u];
    *R += m[u];
  }
  if (*S + *R > INT32_MAX) return ST_ERR_INVALID_ARG;
  return ST_OK;
}

}  // namespace

// =================================================================================== C ABI

extern "C" {

uint64_t st_pool_bytes(const st_config *cfg) {
  if (!config_ok(cfg, nullptr)) return 0;
  return (uint64_t)cfg->n_layers * (uint64_t)(cfg->n_pages_source + cfg->n_pages_reason) * cfg->n_kv_heads *
         st::kBlockBytes;
}

int st_create(const st_config *cfg, st_ctx **out) {
  std::string why;
  if (!out) { g_create_error = "out is NULL"; return ST_ERR_INVALID_ARG; }
  *out = nullptr;
  if (!config_ok(cfg, &why)) { g_create_error = why; return ST_ERR_INVALID_ARG; }
  if (cfg->flags & ~(ST_CFG_HOST_ONLY | ST_CFG_DEBUG_CHECKS | ST_CFG_PRECISE_P)) { g_create_error = "unknown config flag"; return ST_ERR_INVALID_ARG; }
  const uint64_t pool_bytes = st_pool_bytes(cfg);
  if (cfg->pool_base && (cfg->pool_bytes < pool_bytes || ((uintptr_t)cfg->pool_base & 1023))) {
    g_create_error = "pool_base must be 1024-byte aligned and hold st_pool_bytes() bytes";
    return ST_ERR_INVALID_ARG;
  }
  st_ctx *ctx = new st_ctx();
  ctx->cfg = *cfg;
  ctx->host_only = (cfg->flags & ST_CFG_HOST_ONLY) != 0;
  ctx->poison = (cfg->flags & ST_CFG_DEBUG_CHECKS) != 0;
  ctx->precise_p = (cfg->flags & ST_CFG_PRECISE_P) != 0;
  ctx->group = cfg->n_q_heads / cfg->n_kv_heads;
  const double scale = cfg->softmax_scale > 0.f ? (double)cfg->softmax_scale : 1.0 / sqrt((double)cfg->head_dim);
  ctx->scale_log2 = (float)(scale * 1.4426950408889634);
  for (int c = 0; c < 64; ++c) ctx->inv_freq[c] = pow(cfg->rope_theta, -2.0 * c / 128.0);
  ctx->seqs.resize(cfg->max_batch);
  const int64_t n_pages[2] = {cfg->n_pages_source, cfg->n_pages_reason};
  const int32_t max_len[2] = {cfg->max_source_len, cfg->max_reason_len};
  for (int s = 0; s < 2; ++s) {
    ctx->ptab_stride[s] = table_stride(n_pages[s], max_len[s]);
    ctx->layer_stride[s] = (size_t)n_pages[s] * cfg->n_kv_heads * st::kBlockBytes;
    ctx->free_pages[s].resize(n_pages[s]);
    for (int64_t i = 0; i < n_pages[s]; ++i) ctx->free_pages[s][i] = (int32_t)(n_pages[s] - 1 - i);  // pop lowest first
  }
  ctx->events.resize(kEventRing);

  auto cuda_fail = [&](const char *what, cudaError_t e) {
    g_create_error = std::string(what) + ": " + cudaGetErrorString(e);
    release_device(ctx);
    delete ctx;
    return ST_ERR_CUDA;
  };
#define ST_CREATE_CUDA(call)                              \
  do {                                                    \
    cudaError_t e__ = (call);                             \
    if (e__ != cudaSuccess) return cuda_fail(#call, e__); \
  } while (0)

  if (!ctx->host_only) {
    ST_CREATE_CUDA(cudaSetDevice(cfg->device));
    cudaDeviceProp prop;
    ST_CREATE_CUDA(cudaGetDeviceProperties(&prop, cfg->device));
    if (prop.major != 10) {
      g_create_error = "this library contains sm_100a code only; the device is not a compute capability 10.x GPU";
      delete ctx;
      return ST_ERR_CUDA;
    }
    ctx->num_sms = prop.multiProcessorCount;
    ST_CREATE_CUDA(st::init_kernels());
    if (cfg->pool_base) {
      ctx->pool_alloc = (uint8_t *)cfg->pool_base;
    } else {
      ctx->own_pool = true;
      ST_CREATE_CUDA(cudaMalloc(&ctx->pool_alloc, std::max<uint64_t>(pool_bytes, 1024)));
    }
    ctx->pool[0] = ctx->pool_alloc;
    ctx->pool[1] = ctx->pool_alloc + (size_t)cfg->n_layers * ctx->layer_stride[0];
    // Masked keys multiply whatever the page holds by a weight of (almost) exactly 0, which must not meet NaN or Inf bit
    // patterns: the pools start zero-filled. With ST_CFG_DEBUG_CHECKS they start filled with a large finite bf16 value
    // instead, so that a key or value read from beyond the visible ranges shows in the rows instead of vanishing.
    if (ctx->poison) {
      ST_CREATE_CUDA(st::launch_fill_u16(ctx->pool_alloc, pool_bytes / 2, st::kPoisonBf16, nullptr));
    } else {
      ST_CREATE_CUDA(cudaMemset(ctx->pool_alloc, 0, pool_bytes));
    }
    const size_t T = cfg->max_tokens_per_call;
    for (int s = 0; s < 2; ++s) {
      ST_CREATE_CUDA(cudaMalloc(&ctx->d_ptab[s], sizeof(int32_t) * (size_t)cfg->max_batch * ctx->ptab_stride[s]));
      ST_CREATE_CUDA(cudaMemset(ctx->d_ptab[s], 0, sizeof(int32_t) * (size_t)cfg->max_batch * ctx->ptab_stride[s]));
      ST_CREATE_CUDA(cudaMalloc(&ctx->qhat[s], T * cfg->n_q_heads * 256));
    }
    ST_CREATE_CUDA(cudaMalloc(&ctx->partial, sizeof(float) * st::decode_partial_floats(st::kMaxSeqPerLaunch, cfg->n_kv_heads, ctx->num_sms)));
    {
      // a reasoning position is below the page table's reach: ptab_stride pages of 64 tokens
      // (with the concatenated or unit-aligned position ids a reasoning token's position may also count source tokens)
      const int n_hi = (int)(((int64_t)(ctx->ptab_stride[0] + ctx->ptab_stride[1]) * 64 + st::kRopeLoSteps - 1) / st::kRopeLoSteps) + 1;
      ST_CREATE_CUDA(cudaMalloc(&ctx->rope_hi, sizeof(double2) * 64 * (size_t)n_hi));
      ST_CREATE_CUDA(cudaMalloc(&ctx->rope_lo, sizeof(double2) * 64 * (size_t)st::kRopeLoSteps));
      ST_CREATE_CUDA(st::launch_rope_table(ctx->inv_freq, ctx->rope_hi, n_hi, st::kRopeLoSteps, nullptr));
      ST_CREATE_CUDA(st::launch_rope_table(ctx->inv_freq, ctx->rope_lo, st::kRopeLoSteps, 1, nullptr));
    }
    if (cfg->q_norm_weight) {
      std::vector<float> w((size_t)cfg->n_layers * 256);
      for (int l = 0; l < cfg->n_layers; ++l) {
        std::copy_n(cfg->q_norm_weight + (size_t)l * 128, 128, w.begin() + (size_t)l * 256);
        std::copy_n(cfg->k_norm_weight + (size_t)l * 128, 128, w.begin() + (size_t)l * 256 + 128);
      }
      ST_CREATE_CUDA(cudaMalloc(&ctx->d_norm, sizeof(float) * w.size()));
      ST_CREATE_CUDA(cudaMemcpy(ctx->d_norm, w.data(), sizeof(float) * w.size(), cudaMemcpyHostToDevice));
    }
    ctx->cfg.q_norm_weight = ctx->cfg.k_norm_weight = nullptr;   // (the caller's arrays are not used after this call)
    ST_CREATE_CUDA(cudaMalloc(&ctx->d_status, sizeof(int32_t)));
    ST_CREATE_CUDA(cudaMemset(ctx->d_status, 0, sizeof(int32_t)));
    for (int s = 0; s < 2; ++s) {
      const size_t rows = (size_t)st::kMaxSplitItems * 2 * st::attn_tc_rows_per_cta();
      ST_CREATE_CUDA(cudaMalloc(&ctx->split_o[s], rows * st::kHeadDim * sizeof(float)));
      ST_CREATE_CUDA(cudaMalloc(&ctx->split_ml[s], rows * sizeof(float2)));
      ST_CREATE_CUDA(cudaMalloc(&ctx->split_ticket[s], st::kMaxSplitItems * 2 * sizeof(int32_t)));
      ST_CREATE_CUDA(cudaMemset(ctx->split_ticket[s], 0, st::kMaxSplitItems * 2 * sizeof(int32_t)));
    }
    ST_CREATE_CUDA(cudaDeviceSynchronize());
  }
#undef ST_CREATE_CUDA
  *out = ctx;
  return ST_OK;
}

int st_destroy(st_ctx *ctx) {
  if (!ctx) return ST_ERR_INVALID_ARG;
  release_device(ctx);
  delete ctx;
  return ST_OK;
}

int st_reset(st_ctx *ctx, const int32_t *seq_ids, int32_t n_seq) {
  if (!ctx) return ST_ERR_INVALID_ARG;
  if (n_seq < 0 || (n_seq > 0 && !seq_ids)) return fail(ctx, ST_ERR_INVALID_ARG, "bad sequence list");
  for (int i = 0; i < n_seq; ++i)
    if (seq_ids[i] < 0 || seq_ids[i] >= ctx->cfg.max_batch) return fail(ctx, ST_ERR_INVALID_ARG, "sequence id out of range");
  if (!ctx->host_only) {
    ST_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    ST_CUDA(ctx, cudaDeviceSynchronize());
  }
  cudaError_t fill_err = cudaSuccess;
  auto reset_one = [&](int id) {
    SeqState &sq = ctx->seqs[id];
    for (int s = 0; s < 2; ++s) {
      for (auto it = sq.pages[s].rbegin(); it != sq.pages[s].rend(); ++it) {
        ctx->free_pages[s].push_back(*it);
        if (ctx->poison && !ctx->host_only) {
          // a released page goes back to the sentinel in every layer (debug contexts only)
          const size_t page_bytes = (size_t)ctx->cfg.n_kv_heads * st::kBlockBytes;
          for (int layer = 0; layer < ctx->cfg.n_layers && fill_err == cudaSuccess; ++layer)
            fill_err = st::launch_fill_u16(ctx->pool[s] + (size_t)layer * ctx->layer_stride[s] + (size_t)*it * page_bytes,
                                           page_bytes / 2, st::kPoisonBf16, nullptr);
        }
      }
      sq.pages[s].clear();
    }
    sq = SeqState();
  };
  if (n_seq == 0) {
    for (int id = 0; id < ctx->cfg.max_batch; ++id) reset_one(id);
  } else {
    for (int i = 0; i < n_seq; ++i) reset_one(seq_ids[i]);
  }
  ctx->pend[0].active = ctx->pend[1].active = false;
  if (n_seq == 0) ctx->decode_steps = 0;
  if (n_seq == 0) ctx->cross_stream = false;   // a full reset (which waited for the device) starts in single-stream mode again
  if (fill_err != cudaSuccess) return fail(ctx, ST_ERR_CUDA, std::string("sentinel fill: ") + cudaGetErrorString(fill_err));
  if (ctx->poison && !ctx->host_only) ST_CUDA(ctx, cudaDeviceSynchronize());
  return ST_OK;
}

int st_append_source_chunk(st_ctx *ctx, int32_t layer, const int32_t *seq_ids, const int32_t *cu_tokens, int32_t n_seq,
                           const void *q, const void *k, const void *v, void *out, uint32_t flags, void *stream) {
  return attention_call(ctx, 0, layer, seq_ids, cu_tokens, n_seq, nullptr, q, k, v, out, flags, stream);
}

int st_reason_decode(st_ctx *ctx, int32_t layer, const int32_t *seq_ids, int32_t n_seq, const int32_t *visible_units,
                     const void *q, const void *k, const void *v, void *out, uint32_t flags, void *stream) {
  if (!ctx) return ST_ERR_INVALID_ARG;
  if (n_seq < 1 || n_seq > ctx->cfg.max_batch) return fail(ctx, ST_ERR_INVALID_ARG, "n_seq out of range");
  std::vector<int32_t> cu(n_seq + 1);
  for (int i = 0; i <= n_seq; ++i) cu[i] = i;
  return attention_call(ctx, 1, layer, seq_ids, cu.data(), n_seq, visible_units, q, k, v, out, flags, stream);
}

int st_reason_extend(st_ctx *ctx, int32_t layer, const int32_t *seq_ids, const int32_t *cu_tokens, int32_t n_seq,
                     const int32_t *visible_units, const void *q, const void *k, const void *v, void *out,
                     uint32_t flags, void *stream) {
  return attention_call(ctx, 2, layer, seq_ids, cu_tokens, n_seq, visible_units, q, k, v, out, flags, stream);
}

int st_forward_packed(st_ctx *ctx, int32_t layer, const int32_t *seq_ids, int32_t n_seq, const int32_t *n_units,
                      const int32_t *src_unit_len, const int32_t *rsn_unit_len, const int32_t *final_len, int32_t lag_units,
                      const void *q, const void *k, const void *v, void *out, uint32_t flags, void *stream) {
  return forward_packed(ctx, layer, seq_ids, n_seq, n_units, src_unit_len, rsn_unit_len, final_len, lag_units, q, k, v, out,
                        flags, (cudaStream_t)stream);
}

int st_schedule_build(const int32_t *src_unit_len, const int32_t *rsn_unit_len, int32_t n_units, int32_t final_len,
                      int32_t lag_units, int32_t *pos_ids, int32_t *vis_len, int64_t *S_out, int64_t *R_out) {
  int64_t S, R;
  int rc = schedule_sizes(src_unit_len, rsn_unit_len, n_units, final_len, &S, &R);
  if (rc) return rc;
  if (lag_units < 0) return ST_ERR_INVALID_ARG;
  if (S_out) *S_out = S;
  if (R_out) *R_out = R;
  if (pos_ids) {
    for (int64_t j = 0; j < S; ++j) pos_ids[j] = (int32_t)j;          // source counter from zero
    for (int64_t r = 0; r < R; ++r) pos_ids[S + r] = (int32_t)r;      // reasoning counter from zero
  }
  if (vis_len) {
    std::vector<int64_t> prefix(n_units + 1, 0);
    for (int u = 0; u < n_units; ++u) prefix[u + 1] = prefix[u] + src_unit_len[u];
    int64_t r = 0;
    for (int u = 1; u <= n_units; ++u) {
      const int64_t seen = std::min<int64_t>((int64_t)u + lag_units, n_units);
      for (int i = 0; i < rsn_unit_len[u - 1]; ++i) vis_len[r++] = (int32_t)prefix[seen];
    }
    for (int i = 0; i < final_len; ++i) vis_len[r++] = (int32_t)S;
  }
  return ST_OK;
}

int st_schedule_dense_mask(const int32_t *src_unit_len, const int32_t *rsn_unit_len, int32_t n_units, int32_t final_len,
                           int32_t lag_units, uint8_t *mask) {
  int64_t S, R;
  int rc = schedule_sizes(src_unit_len, rsn_unit_len, n_units, final_len, &S, &R);
  if (rc) return rc;
  if (!mask || lag_units < 0) return ST_ERR_INVALID_ARG;
  std::vector<int32_t> vis(R > 0 ? R : 1);
  rc = st_schedule_build(src_unit_len, rsn_unit_len, n_units, final_len, lag_units, nullptr, vis.data(), nullptr, nullptr);
  if (rc) return rc;
  const int64_t T = S + R;
  memset(mask, 0, (size_t)(T * T));
  for (int64_t i = 0; i < S; ++i) memset(mask + i * T, 1, (size_t)(i + 1));
  for (int64_t r = 0; r < R; ++r) {
    uint8_t *row = mask + (S + r) * T;
    memset(row, 1, (size_t)vis[r]);
    memset(row + S, 1, (size_t)(r + 1));
  }
  return ST_OK;
}

int st_seq_state(const st_ctx *ctx, int32_t seq_id, int32_t *source_len, int32_t *reason_len, int32_t *n_eos,
                 int32_t *n_eot) {
  if (!ctx || seq_id < 0 || seq_id >= ctx->cfg.max_batch) return ST_ERR_INVALID_ARG;
  const SeqState &sq = ctx->seqs[seq_id];
  if (source_len) *source_len = sq.len[0];
  if (reason_len) *reason_len = sq.len[1];
  if (n_eos) *n_eos = sq.n_eos;
  if (n_eot) *n_eot = sq.n_eot;
  return ST_OK;
}

int st_pages_free(const st_ctx *ctx, int64_t *source_pages, int64_t *reason_pages) {
  if (!ctx) return ST_ERR_INVALID_ARG;
  if (source_pages) *source_pages = (int64_t)ctx->free_pages[0].size();
  if (reason_pages) *reason_pages = (int64_t)ctx->free_pages[1].size();
  return ST_OK;
}

int st_debug_last_call_meta(const st_ctx *ctx, int32_t *pos_ids, int32_t *vis_source, int32_t *vis_reason, int32_t cap,
                            int32_t *n_tokens) {
  if (!ctx || cap < 0) return ST_ERR_INVALID_ARG;
  const int32_t n = (int32_t)ctx->meta_pos.size();
  if (n_tokens) *n_tokens = n;
  const int32_t m = std::min(n, cap);
  if (pos_ids) std::copy_n(ctx->meta_pos.begin(), m, pos_ids);
  if (vis_source) std::copy_n(ctx->meta_vis_src.begin(), m, vis_source);
  if (vis_reason) std::copy_n(ctx->meta_vis_rsn.begin(), m, vis_reason);
  return ST_OK;
}

int st_debug_page_table(const st_ctx *ctx, int32_t seq_id, int32_t which, int32_t *pages, int32_t cap,
                        int32_t *n_pages) {
  if (!ctx || seq_id < 0 || seq_id >= ctx->cfg.max_batch || which < 0 || which > 1 || cap < 0) return ST_ERR_INVALID_ARG;
  const std::vector<int32_t> &pg = ctx->seqs[seq_id].pages[which];
  if (n_pages) *n_pages = (int32_t)pg.size();
  if (pages) std::copy_n(pg.begin(), std::min<size_t>(pg.size(), (size_t)cap), pages);
  return ST_OK;
}

int st_debug_read_cache(st_ctx *ctx, int32_t layer, int32_t seq_id, int32_t which, int32_t tok0, int32_t ntok,
                        void *k_out, void *v_out) {
  if (!ctx) return ST_ERR_INVALID_ARG;
  if (ctx->host_only) return fail(ctx, ST_ERR_INVALID_ARG, "host-only context holds no cache");
  if (layer < 0 || layer >= ctx->cfg.n_layers || seq_id < 0 || seq_id >= ctx->cfg.max_batch || which < 0 || which > 1)
    return fail(ctx, ST_ERR_INVALID_ARG, "layer, sequence or cache selector out of range");
  const SeqState &sq = ctx->seqs[seq_id];
  if (tok0 < 0 || ntok < 0 || tok0 + ntok > sq.len[which] || !k_out || !v_out)
    return fail(ctx, ST_ERR_INVALID_ARG, "token range outside the cache, or NULL output");
  if (ntok == 0) return ST_OK;
  ST_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  ST_CUDA(ctx, cudaDeviceSynchronize());
  const size_t bytes = (size_t)ntok * ctx->cfg.n_kv_heads * 256;
  __nv_bfloat16 *dk = nullptr, *dv = nullptr;
  ST_CUDA(ctx, cudaMalloc(&dk, bytes));
  ST_CUDA(ctx, cudaMalloc(&dv, bytes));
  cudaError_t e = st::launch_cache_gather(ctx->pool[which] + (size_t)layer * ctx->layer_stride[which],
                                          ctx->d_ptab[which] + (size_t)seq_id * ctx->ptab_stride[which],
                                          ctx->cfg.n_kv_heads, tok0, ntok, dk, dv, nullptr);
  if (e == cudaSuccess) e = cudaMemcpy(k_out, dk, bytes, cudaMemcpyDeviceToHost);
  if (e == cudaSuccess) e = cudaMemcpy(v_out, dv, bytes, cudaMemcpyDeviceToHost);
  cudaFree(dk);
  cudaFree(dv);
  ++ctx->launches;
  if (e != cudaSuccess) return fail(ctx, ST_ERR_CUDA, cudaGetErrorString(e));
  return ST_OK;
}

int st_device_status(st_ctx *ctx) {
  if (!ctx) return ST_ERR_INVALID_ARG;
  if (ctx->host_only) return ST_OK;
  ST_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  ST_CUDA(ctx, cudaDeviceSynchronize());
  int32_t h = 0;
  ST_CUDA(ctx, cudaMemcpy(&h, ctx->d_status, sizeof(h), cudaMemcpyDeviceToHost));
  if (h != st::kDevOk) {
    ST_CUDA(ctx, cudaMemset(ctx->d_status, 0, sizeof(int32_t)));
    // (a kernel that gave up may have left a key-split ticket odd)
    for (int s = 0; s < 2; ++s) ST_CUDA(ctx, cudaMemset(ctx->split_ticket[s], 0, st::kMaxSplitItems * 2 * sizeof(int32_t)));
    if (h == st::kDevBadPage)
      return fail(ctx, ST_ERR_DEVICE_CHECK, "a page id read from a page table lies outside its pool; the access was skipped");
    return fail(ctx, ST_ERR_DEVICE_TIMEOUT, h == st::kDevTimeoutDecode    ? "a bounded wait expired in the decode kernel"
                                            : h == st::kDevTimeoutPrefill ? "a bounded wait expired in the tensor-core attention kernel"
                                                                          : "a bounded wait expired in the wait-expiry test kernel");
  }
  return ST_OK;
}

int st_debug_wait_expiry(st_ctx *ctx, int32_t limit_ms, void *stream) {
  if (!ctx) return ST_ERR_INVALID_ARG;
  if (limit_ms < 1 || limit_ms > 2000) return fail(ctx, ST_ERR_INVALID_ARG, "limit_ms must be 1..2000");
  if (ctx->host_only) return ST_OK;
  ST_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  ST_CUDA(ctx, st::launch_wait_expiry(ctx->d_status, (uint64_t)limit_ms * 1000000ull, (cudaStream_t)stream));
  return ST_OK;
}

int st_debug_fail_after(st_ctx *ctx, int32_t n_steps) {
  if (!ctx || n_steps < 0) return ST_ERR_INVALID_ARG;
  ctx->fail_countdown = n_steps;
  return ST_OK;
}

int st_debug_corrupt_page_table(st_ctx *ctx, int32_t seq_id, int32_t which, int32_t index, int32_t page, void *stream) {
  if (!ctx || seq_id < 0 || seq_id >= ctx->cfg.max_batch || which < 0 || which > 1) return ST_ERR_INVALID_ARG;
  if (index < 0 || index >= ctx->ptab_stride[which]) return fail(ctx, ST_ERR_INVALID_ARG, "page table index out of range");
  if (ctx->host_only) return ST_OK;
  ST_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
  ST_CUDA(ctx, cudaMemcpyAsync(ctx->d_ptab[which] + (size_t)seq_id * ctx->ptab_stride[which] + index, &page, sizeof(int32_t),
                               cudaMemcpyHostToDevice, (cudaStream_t)stream));
  ST_CUDA(ctx, cudaStreamSynchronize((cudaStream_t)stream));
  return ST_OK;
}

int st_kernel_timing_enable(st_ctx *ctx, int32_t on) {
  if (!ctx) return ST_ERR_INVALID_ARG;
  if (on < 0) return ST_ERR_INVALID_ARG;
  ctx->timing = ctx->host_only ? 0 : on;
  ctx->timing_seen = 0;
  return ST_OK;
}

int st_kernel_timing_read(st_ctx *ctx, int32_t which, int64_t *launches, double *total_ms) {
  if (!ctx || which < 0 || which > 1) return ST_ERR_INVALID_ARG;
  int64_t n = 0;
  double ms = 0.0;
  if (!ctx->host_only) {
    ST_CUDA(ctx, cudaSetDevice(ctx->cfg.device));
    ST_CUDA(ctx, cudaDeviceSynchronize());
    std::vector<st_ctx::TimedLaunch> keep;
    for (auto &t : ctx->timed) {
      if (t.which != which) { keep.push_back(t); continue; }
      float f = 0.f;
      ST_CUDA(ctx, cudaEventElapsedTime(&f, t.t0, t.t1));
      ms += f;
      ++n;
      ctx->spare_events.push_back(t.t0);
      ctx->spare_events.push_back(t.t1);
    }
    ctx->timed.swap(keep);
  }
  if (launches) *launches = n;
  if (total_ms) *total_ms = ms;
  return ST_OK;
}

int64_t st_launch_count(const st_ctx *ctx) { return ctx ? ctx->launches : 0; }

const char *st_last_error_string(const st_ctx *ctx) { return ctx ? ctx->err.c_str() : g_create_error.c_str(); }

}  // extern "C"

namespace st {
cudaError_t init_kernels() {
  cudaError_t e = init_decode_kernels();
  if (e != cudaSuccess) return e;
  return init_attn_tc_kernels();
}
}  // namespace st
