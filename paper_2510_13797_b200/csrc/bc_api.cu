// Host side of the C ABI declared in breadcrumbs.h: argument validation, buffer carving, launch
// sequencing.  No device allocation happens here; the caller owns pool, meta and workspace.
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include <cuda.h>

#include "bc_common.cuh"

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct MetaLayout {
  size_t status, free_top, open, prompt_len, n_beacons, window_len, c, t, window_off, beacon_off, dup_mark, free_stack,
      page_table, total;
};
MetaLayout meta_layout(const bc_config& c) {
  MetaLayout l;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  const size_t seq = (size_t)c.max_seqs * 4;
  l.status = take(16); l.free_top = take(4);
  l.open = take(seq); l.prompt_len = take(seq); l.n_beacons = take(seq); l.window_len = take(seq);
  l.c = take(seq); l.t = take(seq); l.window_off = take(seq); l.beacon_off = take(seq);
  l.dup_mark = take(2 * seq);
  l.free_stack = take((size_t)c.num_pages * 4);
  l.page_table = take((size_t)c.max_seqs * c.max_pages_per_seq * 4);
  l.total = o;
  return l;
}

// Host-buffer steps: input staging buffers and output staging sets, each used in turn.  Eight deep: a buffer is
// refilled (and a set rewritten) eight steps after its use, so the stream operations that wait for its last
// reader are satisfied long before the copy is needed, whatever the latency with which a blocked stream notices.
constexpr int kHostRing = 8;

struct WorkLayout {
  size_t append_row[2], append_pos[2], plan[2], compress_row, compress_pos, restore_ok, restore_bea, tickets, book_flag, part_ml, part_o, part_ml2, part_o2, stage_in[kHostRing],
      stage_out[kHostRing], stage_out2[kHostRing], rope_stage, host_words,
      total;
};
WorkLayout work_layout(const bc_config& c) {
  WorkLayout l;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  const size_t seq = (size_t)c.max_seqs * 4;
  const size_t pieces = BC_MAX_ATTN_CTAS + BC_MAX_ATTN_BATCH;
  // two sets of row destinations of bc_append, used by alternate steps: a fused attention kernel may
  // still read one while the next step's bookkeeping already fills the other
  for (int b = 0; b < 2; ++b) { l.append_row[b] = take(seq); l.append_pos[b] = take(seq); l.plan[b] = take(BC_PLAN_INTS * 4); }
  l.compress_row = take(seq); l.compress_pos = take(seq);
  l.restore_ok = take(seq); l.restore_bea = take(seq + 4);
  // A call with layer = BC_ALL_LAYERS is one launch whose blocks work on several layers at a time: every layer
  // has its own ticket counters and its own partial buffers of BC_MAX_ATTN_CTAS + max_n pieces.
  const size_t max_n = c.max_seqs < BC_MAX_ATTN_BATCH ? c.max_seqs : BC_MAX_ATTN_BATCH;
  const size_t layered = (size_t)c.layers * (BC_MAX_ATTN_CTAS + max_n);
  const size_t pieces1 = layered > pieces ? layered : pieces;
  l.tickets = take((size_t)BC_MAX_ATTN_BATCH * 4 * c.layers);
  l.book_flag = take(4);
  l.part_ml = take(pieces1 * c.q_heads * 2 * 4);
  l.part_o = take(pieces1 * c.q_heads * c.head_dim * 4);
  l.part_ml2 = take(pieces * c.q_heads * 2 * 4);            // the beacons' partials of the paired form
  l.part_o2 = take(pieces * c.q_heads * c.head_dim * 4);
  // host-buffer entry points: a ring of input staging buffers, each k | v | q packed for the largest
  // batch a call can carry (a step that fills a window takes two of them, token and beacon inputs)
  for (int b = 0; b < kHostRing; ++b) l.stage_in[b] = take(max_n * (c.q_heads + 2 * c.kv_heads) * c.head_dim * 2);
  l.host_words = take((kHostRing + 1) * 4);   // one input word per staging buffer, then the "done" word
  for (int b = 0; b < kHostRing; ++b) {   // sets of output staging (a set: token output, beacon output)
    l.stage_out[b] = take(max_n * c.q_heads * c.head_dim * 4);
    l.stage_out2[b] = take(max_n * c.q_heads * c.head_dim * 4);
  }
  l.rope_stage = take(max_n * (c.q_heads + 2 * c.kv_heads) * c.head_dim * 2);   // bc_rope_decode_step: q | k | v
  l.total = o;
  return l;
}

bool config_ok(const bc_config* c, bc_status* why) {
  *why = BC_ERR_INVALID_ARG;
  if (!c) return false;
  if (c->layers < 1 || c->kv_heads < 1 || c->q_heads < 1 || c->page_size < 1 || c->max_seqs < 1 ||
      c->num_pages < 1 || c->max_pages_per_seq < 1 || c->c_default < 1 || c->max_entries_per_seq < 0)
    return false;
  if (c->q_heads % c->kv_heads) return false;
  if ((int64_t)c->num_pages * c->page_size >= (int64_t)1 << 31) return false;
  *why = BC_ERR_UNSUPPORTED;
  if (c->head_dim != 64 && c->head_dim != 128) return false;
  if (c->kv_heads != 1 && c->kv_heads != 2 && c->kv_heads != 4 && c->kv_heads != 8) return false;
  if (c->q_heads / c->kv_heads > 16) return false;
  if (c->q_heads * c->head_dim > BC_MERGE_ELEMS) return false;
  return true;
}

constexpr size_t kFusedBeaconRowBytes = 512u << 10;  // the same for the beacon rows of bc_compress (see there)
constexpr size_t kFusedRowBytes = 32u << 10;  // rows of a batch that the bookkeeping block copies itself (a
                                                // single block moves more than this slower than a second launch)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

}  // namespace

struct bc_cache {
  bc_config cfg;
  BcMeta meta;
  BcGeom geom;
  uint8_t* pool;
  uint8_t* meta_base;
  uint8_t* work;
  MetaLayout ml;
  WorkLayout wl;
  int sm_count;
  int attn_ctas;
  int64_t calls;            // bookkeeping calls issued (1-based index of the next is calls + 1)
  int64_t launches;
  int append_next_layer;    // per-layer ordering of bc_append
  int compress_next_layer;  // per-layer ordering of bc_compress
  int restore_next_layer = 0;   // per-layer ordering of bc_restore
  int append_set = 0;           // which set of append row destinations the current step uses (flips on layer 0)
  int64_t append_call = 0;      // index of the step's append bookkeeping call (its flag's epoch; other calls may lie between the layers)
  // true while the last kernel this handle enqueued that writes metadata (lengths, page table, free stack)
  // has not been followed by an ordinarily launched kernel or an attention launch of this handle: an
  // attention kernel enqueued now could begin before that writer has ended and must not read early
  bool meta_unsettled = true;
  uint32_t wait_limit = 0;      // bc_set_wait_limit: polls of the attention kernel's bounded waits (0: default)
  void* timeline = nullptr;     // bc_attn_timeline: device buffer the attention kernel stamps, or NULL
  int device = -1;              // the CUDA device that was current at bc_cache_create
  bool static_used = false;     // a bc_decode_attn_static launch was issued since the last bc_clear_error
  int last_cuda_error;
  // profiling
  std::vector<cudaEvent_t> ev;
  int prof_cap, prof_used;
  // host-buffer entry points: inputs are copied on a stream of their own into a ring of staging buffers
  static constexpr int kStageRing = kHostRing;
  cudaStream_t copy_stream = nullptr;
  cudaEvent_t ev_in[kStageRing] = {};      // the copies into staging buffer b have been issued up to here
  cudaEvent_t buf_done[kStageRing] = {};   // not owned: the event after which buffer b's last readers have finished
  int stage_next = 0;
  // Host-buffer decode steps of single-layer caches with BC_FLAG_HOST_PIPELINED are tied to their copies by two
  // kinds of words in device memory instead of events on the caller's stream (which then carries nothing but
  // kernels): the copy stream writes a step's number behind its inputs and the step's bookkeeping kernel polls
  // it; every bookkeeping kernel stores the number of the step before it to the "done" word when it ends, and
  // the output stream and the copy stream wait for that word (stream memory operations).
  int32_t host_seq = 0;                       // number of the last such step (0: none yet; 0 is skipped on wrap-around)
  int32_t done_issued = 0;                    // highest step number that an enqueued kernel will store to the done word
  int32_t buf_reader_seq[kStageRing] = {};    // number of the last such step that read staging buffer b (0: none)
  cudaStream_t host_stream = nullptr;         // the caller's stream those steps were enqueued on
  // one event per host-buffer step, recorded on the caller's stream behind the step's kernels
  static constexpr int kDoneRing = 2 * kHostRing;
  cudaEvent_t ev_done[kDoneRing] = {};
  int done_next = 0;
  // BC_FLAG_HOST_PIPELINED: outputs leave on a stream of their own from alternating staging sets
  cudaStream_t out_stream = nullptr;
  static constexpr int kOutSets = kHostRing;
  cudaEvent_t ev_d2h[kOutSets] = {};             // the copies out of set b have been issued up to here
  int out_next = 0;
  // BC_FLAG_HOST_PIPELINED: what the last host-buffer step still owes -- its completion event and the
  // copies of its outputs.  They are issued by the next host-buffer call right behind that call's
  // bookkeeping kernel (which may then start under this step's attention kernel), or by
  // bc_host_outputs_ready / bc_cache_destroy.
  struct Pending {
    bool valid = false;
    int set = 0, bufs[2] = {-1, -1};
    void* out_host = nullptr; void* out2_host = nullptr;
    size_t bytes = 0;
    cudaStream_t stream = nullptr;
    int32_t word_seq = 0;   // a step ordered by words (its number), else 0: ordered by an event
  } pending;
};

namespace {

bc_status cuda_fail(bc_cache* c, cudaError_t e) {
  if (c) c->last_cuda_error = (int)e;
  return BC_ERR_CUDA;
}
#define BC_CUDA(c, expr)                                   \
  do {                                                     \
    cudaError_t e__ = (expr);                              \
    if (e__ != cudaSuccess) return cuda_fail((c), e__);    \
  } while (0)

inline uint8_t* layer_base(bc_cache* c, int layer) { return c->pool + (int64_t)layer * c->geom.layer_bytes; }
template <typename T>
inline T* work_ptr(bc_cache* c, size_t off) { return reinterpret_cast<T*>(c->work + off); }

// layer == BC_ALL_LAYERS: the per-layer tensors carry a leading [layers] dimension and the call runs
// layer 0 .. layers - 1 in order (one launch sequence per layer, the dependency order of a forward pass).
inline const void* layer_slice(const void* p, int layer, size_t bytes_per_layer) {
  return p ? static_cast<const uint8_t*>(p) + (size_t)layer * bytes_per_layer : nullptr;
}
inline void* layer_slice(void* p, int layer, size_t bytes_per_layer) {
  return p ? static_cast<uint8_t*>(p) + (size_t)layer * bytes_per_layer : nullptr;
}

bc_status check_batch(bc_cache* c, int layer, const int32_t* slots, int n) {
  if (!c || !slots || n <= 0 || n > c->cfg.max_seqs) return BC_ERR_INVALID_ARG;
  if (layer < 0 || layer >= c->cfg.layers) return BC_ERR_INVALID_ARG;
  return BC_OK;
}

bc_status attn_impl(bc_cache* c, int layer, const int32_t* slots, int n, const void* q, void* out, float sm_scale,
                    const void* extra_k, const void* extra_v, cudaStream_t s, const BcFusedAppend* fused = nullptr,
                    const void* q2 = nullptr, void* out2 = nullptr, int layers = 1) {
  BcAttnArgs a;
  if (layers > 1) {   // all layers in one launch: q, out, extra (or new) rows are [layers][n][...] arrays
    const size_t max_n = c->cfg.max_seqs < BC_MAX_ATTN_BATCH ? c->cfg.max_seqs : BC_MAX_ATTN_BATCH;
    const size_t pieces = BC_MAX_ATTN_CTAS + max_n;
    a.layers = layers;
    a.ls_pool = c->geom.layer_bytes;
    a.ls_q = (int64_t)n * c->cfg.q_heads * c->cfg.head_dim * 2;
    a.ls_out = (c->cfg.flags & BC_FLAG_OUT_F32) ? a.ls_q * 2 : a.ls_q;
    a.ls_kv = (int64_t)n * c->cfg.kv_heads * c->cfg.head_dim * 2;
    a.ls_part_o = (int64_t)pieces * c->cfg.q_heads * c->cfg.head_dim * 4;
    a.ls_part_ml = (int64_t)pieces * c->cfg.q_heads * 2 * 4;
    a.ls_tickets = BC_MAX_ATTN_BATCH;
  }
  if (q2) {   // the paired form
    a.q2 = q2; a.out2 = out2;
    a.part_o2 = work_ptr<float>(c, c->wl.part_o2);
    a.part_ml2 = work_ptr<float>(c, c->wl.part_ml2);
  }
  a.pool_layer = layer_base(c, layer);
  a.slots = slots; a.n = n; a.q = q; a.out = out;
  a.out_f32 = (c->cfg.flags & BC_FLAG_OUT_F32) ? 1 : 0;
  a.extra_k = extra_k; a.extra_v = extra_v; a.sm_scale = sm_scale;
  a.part_o = work_ptr<float>(c, c->wl.part_o);
  a.part_ml = work_ptr<float>(c, c->wl.part_ml);
  a.tickets = work_ptr<int32_t>(c, c->wl.tickets);
  a.ctas = c->attn_ctas > 0 ? c->attn_ctas : c->sm_count;
  a.timeline = c->timeline;
  a.spin_limit = c->wait_limit;
  a.debug = c->meta.debug;
  a.meta_settled = c->meta_unsettled ? 0 : 1;
  c->meta_unsettled = false;   // whatever follows this launch starts after its blocks have waited for the writer
  if (c->cfg.flags & BC_FLAG_ATTN_REFERENCE) {
    BC_CUDA(c, bc_launch_attn_reference(c->meta, c->geom, a, s));
    c->launches += 1;
    return BC_OK;
  }
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (c->prof_used < c->prof_cap) { e0 = c->ev[2 * c->prof_used]; e1 = c->ev[2 * c->prof_used + 1]; c->prof_used++; }
  int launches = 0;
  BC_CUDA(c, bc_launch_attn(c->meta, c->geom, a, fused, s, e0, e1, &launches));
  c->launches += launches;
  return BC_OK;
}

}  // namespace

namespace {
// The word a fused step's bookkeeping kernel publishes when its results are written: derived from the
// index of the bookkeeping call, never 0 (the word's initial value).
inline int32_t step_epoch(int64_t calls) { return (int32_t)(calls & 0x3fffffff) | 1 << 30; }

// Layer-0 bookkeeping of a step's append, launched on its own (no K/V rows in the same launch).
bc_status append_book_only(bc_cache* c, const int32_t* slots, int n, cudaStream_t s, bool with_plan = false,
                           const BcHostSync* hs = nullptr) {
  c->append_set ^= 1;
  ++c->calls;
  c->append_call = c->calls;
  BC_CUDA(c, bc_launch_append_book(c->meta, slots, n, c->calls, work_ptr<int32_t>(c, c->wl.append_row[c->append_set]),
                                   work_ptr<int32_t>(c, c->wl.append_pos[c->append_set]), c->geom, layer_base(c, 0), nullptr,
                                   nullptr, s, with_plan ? work_ptr<int32_t>(c, c->wl.plan[c->append_set]) : nullptr,
                                   work_ptr<int32_t>(c, c->wl.book_flag), step_epoch(c->calls), hs));
  c->launches += 1;
  c->meta_unsettled = true;
  return BC_OK;
}

// The attention half of bc_decode_step: the step's append bookkeeping (layer 0) has been launched.
// With beacon_q .. out_beacon: the step that fills a window (the paired form of the same kernel).
bc_status decode_step_attn(bc_cache* c, int layer, const int32_t* slots, int n, const void* q, const void* k, const void* v,
                           void* out, float sm_scale, cudaStream_t s, int layers = 1, const void* beacon_q = nullptr,
                           const void* beacon_k = nullptr, const void* beacon_v = nullptr, void* out_beacon = nullptr) {
  BcFusedAppend f;
  f.new_k = k; f.new_v = v;
  f.dst_row = work_ptr<int32_t>(c, c->wl.append_row[c->append_set]);
  f.dst_pos = work_ptr<int32_t>(c, c->wl.append_pos[c->append_set]);
  f.pool_layer = layer_base(c, layer);
  f.flag = work_ptr<int32_t>(c, c->wl.book_flag);
  f.plan = work_ptr<int32_t>(c, c->wl.plan[c->append_set]);   // left by append_book_only(with_plan) of this step
  f.call = c->append_call;
  f.epoch = step_epoch(c->append_call);
  const bc_status st = attn_impl(c, layer, slots, n, q, out, sm_scale, beacon_k, beacon_v, s, &f, beacon_q, out_beacon, layers);
  if (st) return st;
  c->append_next_layer = (layer + layers) % c->cfg.layers;
  return BC_OK;
}
}  // namespace

// ---- bc_decode_attn_static: split-K scratch inside the library image -------------------------------
//
// Layout of the built-in array: partial outputs [pieces][4096] fp32, then (max, sum) pairs
// [pieces][64][2] fp32, then one ticket counter per sequence, [BC_STATIC_MAX_BATCH] int32, with
// pieces = BC_STATIC_MAX_CTAS + BC_STATIC_MAX_BATCH.  The loader zero-fills the array and every
// launch leaves the counters at zero again; the partials need no clearing because a launch reads
// only what it has written.
namespace {
constexpr size_t kStaticPieces = BC_STATIC_MAX_CTAS + BC_STATIC_MAX_BATCH;
constexpr size_t kStaticPartO = kStaticPieces * BC_MERGE_ELEMS * sizeof(float);
constexpr size_t kStaticPartMl = kStaticPieces * 64 * 2 * sizeof(float);
constexpr size_t kStaticIdx = BC_STATIC_MAX_BATCH * sizeof(int32_t);
constexpr size_t kStaticBytes = kStaticPartO + kStaticPartMl + kStaticIdx;
constexpr int kMaxDevices = 64;
}  // namespace

// In host code this name is only a handle for the runtime's symbol lookup, never a device address.
static __device__ __align__(256) unsigned char bc_static_scratch[kStaticBytes];

namespace {
std::mutex g_static_mu;
unsigned char* g_static_ptr[kMaxDevices] = {};

// Device address of bc_static_scratch on the current device; looked up once per device.
cudaError_t static_scratch(unsigned char** out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mu);
  if (!g_static_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, bc_static_scratch);
    if (e != cudaSuccess) return e;
    g_static_ptr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_static_ptr[dev];
  return cudaSuccess;
}

// Zeroes the ticket counters of the built-in array on the current device if a call has already
// looked its address up there (used when a latched error is cleared).
cudaError_t static_scratch_reset_tickets(cudaStream_t s) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  unsigned char* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mu);
    if (dev >= 0 && dev < kMaxDevices) base = g_static_ptr[dev];
  }
  if (!base) return cudaSuccess;
  return cudaMemsetAsync(base + kStaticPartO + kStaticPartMl, 0, kStaticIdx, s);
}
}  // namespace


extern "C" {

namespace {
bc_status flush_pending(bc_cache* c);   // defined with the host-buffer entry points below
}

int32_t bc_version(void) { return 231; }

const char* bc_status_string(bc_status s) {
  switch (s) {
    case BC_OK: return "BC_OK";
    case BC_ERR_INVALID_ARG: return "BC_ERR_INVALID_ARG";
    case BC_ERR_BAD_SLOT: return "BC_ERR_BAD_SLOT";
    case BC_ERR_NO_PAGES: return "BC_ERR_NO_PAGES";
    case BC_ERR_CAPACITY: return "BC_ERR_CAPACITY";
    case BC_ERR_WINDOW_NOT_FULL: return "BC_ERR_WINDOW_NOT_FULL";
    case BC_ERR_WINDOW_FULL: return "BC_ERR_WINDOW_FULL";
    case BC_ERR_ORDER: return "BC_ERR_ORDER";
    case BC_ERR_CUDA: return "BC_ERR_CUDA";
    case BC_ERR_UNSUPPORTED: return "BC_ERR_UNSUPPORTED";
    case BC_ERR_TIMEOUT: return "BC_ERR_TIMEOUT";
    case BC_ERR_TOO_LARGE: return "BC_ERR_TOO_LARGE";
    case BC_ERR_DEBUG_CHECK: return "BC_ERR_DEBUG_CHECK";
    default: return "BC_ERR_UNKNOWN";
  }
}

bc_status bc_cache_query_bytes(const bc_config* cfg, size_t* pool_bytes, size_t* meta_bytes, size_t* workspace_bytes) {
  bc_status why;
  if (!config_ok(cfg, &why)) return why;
  if (!pool_bytes || !meta_bytes || !workspace_bytes) return BC_ERR_INVALID_ARG;
  const size_t E = (size_t)2 * cfg->kv_heads * cfg->head_dim * 2;
  *pool_bytes = (size_t)cfg->layers * cfg->num_pages * cfg->page_size * E;
  *meta_bytes = meta_layout(*cfg).total;
  *workspace_bytes = work_layout(*cfg).total;
  return BC_OK;
}

bc_status bc_cache_create(const bc_config* cfg, void* pool, void* meta, void* workspace, void* stream, bc_cache** out) {
  bc_status why;
  if (!config_ok(cfg, &why)) return why;
  if (!pool || !meta || !workspace || !out) return BC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(pool) | reinterpret_cast<uintptr_t>(meta) | reinterpret_cast<uintptr_t>(workspace)) & 255)
    return BC_ERR_INVALID_ARG;
  bc_cache* c = new (std::nothrow) bc_cache();
  if (!c) return BC_ERR_INVALID_ARG;
  c->cfg = *cfg;
  c->pool = (uint8_t*)pool; c->meta_base = (uint8_t*)meta; c->work = (uint8_t*)workspace;
  c->ml = meta_layout(*cfg); c->wl = work_layout(*cfg);
  c->calls = 0; c->launches = 0; c->append_next_layer = 0; c->compress_next_layer = 0; c->last_cuda_error = 0;
  c->attn_ctas = 0; c->prof_cap = 0; c->prof_used = 0;
  BcMeta& m = c->meta;
  auto at = [&](size_t off) { return reinterpret_cast<int32_t*>(c->meta_base + off); };
  m.status = at(c->ml.status); m.free_top = at(c->ml.free_top); m.free_stack = at(c->ml.free_stack);
  m.open = at(c->ml.open); m.prompt_len = at(c->ml.prompt_len); m.n_beacons = at(c->ml.n_beacons);
  m.window_len = at(c->ml.window_len); m.c = at(c->ml.c); m.t = at(c->ml.t);
  m.window_off = at(c->ml.window_off); m.beacon_off = at(c->ml.beacon_off); m.page_table = at(c->ml.page_table);
  m.dup_mark = reinterpret_cast<unsigned long long*>(c->meta_base + c->ml.dup_mark);
  m.debug = (cfg->flags & BC_FLAG_DEBUG_BOUNDS) ? 1 : 0;
  m.max_seqs = cfg->max_seqs; m.num_pages = cfg->num_pages; m.max_pages_per_seq = cfg->max_pages_per_seq;
  m.max_entries = cfg->max_entries_per_seq; m.page_size = cfg->page_size; m.c_default = cfg->c_default;
  BcGeom& g = c->geom;
  g.kv_heads = cfg->kv_heads; g.q_heads = cfg->q_heads; g.head_dim = cfg->head_dim; g.page_size = cfg->page_size;
  g.head_row_bytes = cfg->head_dim * 2;
  g.entry_bytes = 2 * cfg->kv_heads * g.head_row_bytes;
  g.layer_bytes = (int64_t)cfg->num_pages * cfg->page_size * g.entry_bytes;
  cudaError_t e = cudaGetDevice(&c->device);
  if (e == cudaSuccess) e = bc_attn_setup(&c->sm_count);
  if (e == cudaSuccess) e = bc_launch_init(c->meta, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->work + c->wl.tickets, 0, (size_t)BC_MAX_ATTN_BATCH * 4 * c->cfg.layers, (cudaStream_t)stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->work + c->wl.book_flag, 0, 4, (cudaStream_t)stream);
  if (e != cudaSuccess) { delete c; return BC_ERR_CUDA; }
  c->launches += 1;
  *out = c;
  return BC_OK;
}

bc_status bc_cache_destroy(bc_cache* c) {
  if (!c) return BC_ERR_INVALID_ARG;
  // the cache's own streams touch the caller's workspace: let them drain before the caller may free it
  flush_pending(c);   // what the last host-buffer steps are owed: their event and copies, or the kernel that vouches for them
  if (c->copy_stream) cudaStreamSynchronize(c->copy_stream);
  if (c->out_stream) cudaStreamSynchronize(c->out_stream);
  for (cudaEvent_t e : c->ev) cudaEventDestroy(e);
  for (cudaEvent_t e : c->ev_in) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : c->ev_done) if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : c->ev_d2h) if (e) cudaEventDestroy(e);
  if (c->copy_stream) cudaStreamDestroy(c->copy_stream);
  if (c->out_stream) cudaStreamDestroy(c->out_stream);
  delete c;
  return BC_OK;
}

bc_status bc_seq_open(bc_cache* c, const int32_t* slots, const int32_t* prompt_lens, const int32_t* c_per_seq, int32_t n,
                      void* stream) {
  if (!c || !slots || !prompt_lens || n <= 0 || n > c->cfg.max_seqs) return BC_ERR_INVALID_ARG;
  BC_CUDA(c, bc_launch_open(c->meta, slots, prompt_lens, c_per_seq, n, ++c->calls, (cudaStream_t)stream));
  c->launches += 1;
  c->meta_unsettled = true;
  return BC_OK;
}

bc_status bc_prefill(bc_cache* c, int32_t layer, const int32_t* slots, const int32_t* cu, int32_t n, int32_t total,
                     const void* k, const void* v, void* stream) {
  if (c && layer == BC_ALL_LAYERS) {
    if (total < 0) return BC_ERR_INVALID_ARG;
    const size_t b = (size_t)total * c->cfg.kv_heads * c->cfg.head_dim * 2;
    for (int l = 0; l < c->cfg.layers; ++l) {
      const bc_status st = bc_prefill(c, l, slots, cu, n, total, layer_slice(k, l, b), layer_slice(v, l, b), stream);
      if (st) return st;
    }
    return BC_OK;
  }
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (!cu || total < 0) return BC_ERR_INVALID_ARG;
  if (total == 0) return BC_OK;
  if (!k || !v || !aligned16(k) || !aligned16(v)) return BC_ERR_INVALID_ARG;
  BC_CUDA(c, bc_launch_prefill(c->meta, c->geom, layer_base(c, layer), slots, cu, n, total, k, v, (cudaStream_t)stream));
  c->launches += 1;
  c->meta_unsettled = false;
  return BC_OK;
}

bc_status bc_restore(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const int32_t* cu_tokens,
                     int32_t total_tokens, int32_t total_beacons, const void* tok_k, const void* tok_v,
                     const void* beacon_k, const void* beacon_v, void* stream) {
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (!cu_tokens || total_tokens < 0 || total_beacons < 0) return BC_ERR_INVALID_ARG;
  if (total_tokens && (!tok_k || !tok_v || !aligned16(tok_k) || !aligned16(tok_v))) return BC_ERR_INVALID_ARG;
  if (total_beacons && (!beacon_k || !beacon_v || !aligned16(beacon_k) || !aligned16(beacon_v))) return BC_ERR_INVALID_ARG;
  if (layer != c->restore_next_layer) return BC_ERR_ORDER;
  cudaStream_t s = (cudaStream_t)stream;
  int32_t* ok = work_ptr<int32_t>(c, c->wl.restore_ok);
  int32_t* bea = work_ptr<int32_t>(c, c->wl.restore_bea);
  if (layer == 0) {
    BC_CUDA(c, bc_launch_restore_book(c->meta, slots, cu_tokens, n, ++c->calls, ok, bea, s));
    c->launches += 1;
    c->meta_unsettled = true;
  }
  BC_CUDA(c, bc_launch_restore_rows(c->meta, c->geom, layer_base(c, layer), slots, ok, bea, cu_tokens, n, total_tokens,
                                   total_beacons, tok_k, tok_v, beacon_k, beacon_v, s));
  c->launches += (total_beacons > 0) + (total_tokens > 0);
  if (total_beacons > 0 || total_tokens > 0) c->meta_unsettled = false;
  c->restore_next_layer = (layer + 1) % c->cfg.layers;
  return BC_OK;
}

bc_status bc_append(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* k, const void* v,
                    void* stream) {
  if (c && layer == BC_ALL_LAYERS) {
    // the bookkeeping kernel, then ONE launch that writes the rows of every layer (same row and position in each)
    bc_status st = check_batch(c, 0, slots, n);
    if (st) return st;
    if (!k || !v || !aligned16(k) || !aligned16(v)) return BC_ERR_INVALID_ARG;
    if (c->append_next_layer != 0) return BC_ERR_ORDER;
    cudaStream_t s = (cudaStream_t)stream;
    st = append_book_only(c, slots, n, s);
    if (st) return st;
    BC_CUDA(c, bc_launch_write_rows(c->meta, c->geom, layer_base(c, 0), work_ptr<int32_t>(c, c->wl.append_row[c->append_set]),
                                    work_ptr<int32_t>(c, c->wl.append_pos[c->append_set]), k, v, n, s, c->cfg.layers,
                                    (long long)c->geom.layer_bytes, (long long)n * c->cfg.kv_heads * c->cfg.head_dim * 2));
    c->launches += 1;
    c->meta_unsettled = false;
    return BC_OK;
  }
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (!k || !v || !aligned16(k) || !aligned16(v)) return BC_ERR_INVALID_ARG;
  if (layer != c->append_next_layer) return BC_ERR_ORDER;
  if (layer == 0) c->append_set ^= 1;
  int32_t* row = work_ptr<int32_t>(c, c->wl.append_row[c->append_set]);
  int32_t* pos = work_ptr<int32_t>(c, c->wl.append_pos[c->append_set]);
  cudaStream_t s = (cudaStream_t)stream;
  // Small batches: the bookkeeping block also copies the rows and a launch is saved.
  const bool fused = layer == 0 && (size_t)n * c->geom.entry_bytes <= kFusedRowBytes;
  if (layer == 0) {
    BC_CUDA(c, bc_launch_append_book(c->meta, slots, n, ++c->calls, row, pos, c->geom, layer_base(c, 0),
                                     fused ? k : nullptr, fused ? v : nullptr, s));
    c->launches += 1;
    c->meta_unsettled = true;
  }
  if (!fused) {
    BC_CUDA(c, bc_launch_write_rows(c->meta, c->geom, layer_base(c, layer), row, pos, k, v, n, s));
    c->launches += 1;
    c->meta_unsettled = false;
  }
  c->append_next_layer = (layer + 1) % c->cfg.layers;
  return BC_OK;
}

bc_status bc_decode_attn(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* q, void* out,
                         float sm_scale, const void* extra_k, const void* extra_v, void* stream) {
  if (c && layer == BC_ALL_LAYERS && c->cfg.layers > 1 && !(c->cfg.flags & BC_FLAG_ATTN_REFERENCE)) {
    // one launch: the grid's second dimension walks the layers
    bc_status st = check_batch(c, 0, slots, n);
    if (st) return st;
    if (n > BC_MAX_ATTN_BATCH) return BC_ERR_INVALID_ARG;
    if (!q || !out || !aligned16(q) || !aligned16(out)) return BC_ERR_INVALID_ARG;
    if ((extra_k == nullptr) != (extra_v == nullptr)) return BC_ERR_INVALID_ARG;
    if (extra_k && (!aligned16(extra_k) || !aligned16(extra_v))) return BC_ERR_INVALID_ARG;
    return attn_impl(c, 0, slots, n, q, out, sm_scale, extra_k, extra_v, (cudaStream_t)stream, nullptr, nullptr, nullptr,
                     c->cfg.layers);
  }
  if (c && layer == BC_ALL_LAYERS) {
    if (n <= 0) return BC_ERR_INVALID_ARG;
    const size_t qb = (size_t)n * c->cfg.q_heads * c->cfg.head_dim * 2, kb = (size_t)n * c->cfg.kv_heads * c->cfg.head_dim * 2;
    const size_t ob = (c->cfg.flags & BC_FLAG_OUT_F32) ? qb * 2 : qb;
    for (int l = 0; l < c->cfg.layers; ++l) {
      const bc_status st = bc_decode_attn(c, l, slots, n, layer_slice(q, l, qb), layer_slice(out, l, ob), sm_scale,
                                          layer_slice(extra_k, l, kb), layer_slice(extra_v, l, kb), stream);
      if (st) return st;
    }
    return BC_OK;
  }
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (n > BC_MAX_ATTN_BATCH) return BC_ERR_INVALID_ARG;
  if (!q || !out || !aligned16(q) || !aligned16(out)) return BC_ERR_INVALID_ARG;
  if ((extra_k == nullptr) != (extra_v == nullptr)) return BC_ERR_INVALID_ARG;
  if (extra_k && (!aligned16(extra_k) || !aligned16(extra_v))) return BC_ERR_INVALID_ARG;
  return attn_impl(c, layer, slots, n, q, out, sm_scale, extra_k, extra_v, (cudaStream_t)stream);
}

bc_status bc_decode_attn_pair(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* q, void* out,
                              const void* beacon_q, void* out_beacon, float sm_scale, const void* beacon_k,
                              const void* beacon_v, void* stream) {
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (n > BC_MAX_ATTN_BATCH) return BC_ERR_INVALID_ARG;
  if (!q || !out || !beacon_q || !out_beacon || !beacon_k || !beacon_v) return BC_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(out) || !aligned16(beacon_q) || !aligned16(out_beacon) || !aligned16(beacon_k) ||
      !aligned16(beacon_v))
    return BC_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  if ((c->cfg.flags & BC_FLAG_ATTN_REFERENCE) || c->cfg.q_heads / c->cfg.kv_heads > 8) {
    // no shared pass for the debugging kernel and for groups of more than 8 query heads: two passes
    st = attn_impl(c, layer, slots, n, q, out, sm_scale, nullptr, nullptr, s);
    if (st) return st;
    return attn_impl(c, layer, slots, n, beacon_q, out_beacon, sm_scale, beacon_k, beacon_v, s);
  }
  return attn_impl(c, layer, slots, n, q, out, sm_scale, beacon_k, beacon_v, s, nullptr, beacon_q, out_beacon);
}

bc_status bc_decode_step(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* q, const void* k,
                         const void* v, void* out, float sm_scale, void* stream) {
  const bool all = c && layer == BC_ALL_LAYERS;
  if (all) layer = 0;
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (n > BC_MAX_ATTN_BATCH) return BC_ERR_INVALID_ARG;
  if (!q || !k || !v || !out || !aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out)) return BC_ERR_INVALID_ARG;
  if (layer != c->append_next_layer) return BC_ERR_ORDER;
  cudaStream_t s = (cudaStream_t)stream;
  if (all && c->cfg.layers > 1) {
    const size_t qb = (size_t)n * c->cfg.q_heads * c->cfg.head_dim * 2, kb = (size_t)n * c->cfg.kv_heads * c->cfg.head_dim * 2;
    const size_t ob = (c->cfg.flags & BC_FLAG_OUT_F32) ? qb * 2 : qb;
    if (c->cfg.flags & BC_FLAG_ATTN_REFERENCE) {   // layer by layer
      for (int l = 0; l < c->cfg.layers; ++l) {
        st = bc_decode_step(c, l, slots, n, layer_slice(q, l, qb), layer_slice(k, l, kb), layer_slice(v, l, kb),
                            layer_slice(out, l, ob), sm_scale, stream);
        if (st) return st;
      }
      return BC_OK;
    }
    // the bookkeeping kernel, then ONE attention launch whose grid walks the layers: each layer's blocks take
    // that layer's new entries from the [layers][n] inputs and store them to that layer's pool
    st = append_book_only(c, slots, n, s, true);
    if (st) return st;
    return decode_step_attn(c, 0, slots, n, q, k, v, out, sm_scale, s, c->cfg.layers);
  }
  if (c->cfg.flags & BC_FLAG_ATTN_REFERENCE) {   // the debugging kernel has no fused form
    st = bc_append(c, layer, slots, n, k, v, stream);
    if (st) return st;
    return attn_impl(c, layer, slots, n, q, out, sm_scale, nullptr, nullptr, s);
  }
  // The bookkeeping runs as its own one-block kernel, which may start under the previous attention
  // kernel's last blocks; the rows are written by the attention kernel itself (its service warps),
  // which takes the new entries from the inputs.  So a step costs one full-size launch and no
  // row-writing launch.
  if (layer == 0) {
    st = append_book_only(c, slots, n, s, true);
    if (st) return st;
  }
  return decode_step_attn(c, layer, slots, n, q, k, v, out, sm_scale, s);
}

bc_status bc_rope_split(bc_cache* c, const void* qkv, const int32_t* positions, int32_t n, float theta, void* q_out,
                        void* k_out, void* v_out, void* stream) {
  if (!c || !qkv || !positions || !q_out || !k_out || !v_out || n <= 0 || !(theta > 1.f)) return BC_ERR_INVALID_ARG;
  if (!aligned16(qkv) || !aligned16(q_out) || !aligned16(k_out) || !aligned16(v_out)) return BC_ERR_INVALID_ARG;
  BC_CUDA(c, bc_launch_rope_split(qkv, positions, n, c->cfg.q_heads, c->cfg.kv_heads, c->cfg.head_dim, (double)theta, q_out,
                                  k_out, v_out, (cudaStream_t)stream));
  c->launches += 1;
  c->meta_unsettled = false;   // an ordinarily launched kernel: it starts after everything before it has ended
  return BC_OK;
}

bc_status bc_add_rmsnorm(const void* h, const void* delta, const void* weight, int32_t n, int32_t hidden, float eps, void* h_out,
                         void* normed_out, void* stream) {
  if (!h || !normed_out || n <= 0 || hidden <= 0 || !(eps >= 0.f)) return BC_ERR_INVALID_ARG;
  if (!aligned16(h) || !aligned16(normed_out) || (delta && !aligned16(delta)) || (weight && !aligned16(weight)) ||
      (h_out && !aligned16(h_out)))
    return BC_ERR_INVALID_ARG;
  if (hidden % 8 || hidden > bc_rmsnorm_max_hidden()) return BC_ERR_UNSUPPORTED;
  if (bc_launch_add_rmsnorm(h, delta, weight, n, hidden, eps, h_out, normed_out, (cudaStream_t)stream) != cudaSuccess) return BC_ERR_CUDA;
  return BC_OK;
}

bc_status bc_swiglu(const void* gate_up, int32_t n, int32_t m, void* out, void* stream) {
  if (!gate_up || !out || n <= 0 || m <= 0 || !aligned16(gate_up) || !aligned16(out)) return BC_ERR_INVALID_ARG;
  if (m % 8) return BC_ERR_UNSUPPORTED;
  if (bc_launch_swiglu(gate_up, n, m, out, (cudaStream_t)stream) != cudaSuccess) return BC_ERR_CUDA;
  return BC_OK;
}

bc_status bc_argmax(const void* logits, int32_t n, int32_t vocab, int64_t* out, void* stream) {
  if (!logits || !out || n <= 0 || vocab <= 0 || !aligned16(logits)) return BC_ERR_INVALID_ARG;
  if (vocab % 8) return BC_ERR_UNSUPPORTED;
  if (bc_launch_argmax(logits, n, vocab, reinterpret_cast<long long*>(out), (cudaStream_t)stream) != cudaSuccess) return BC_ERR_CUDA;
  return BC_OK;
}

bc_status bc_rope_decode_step(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* qkv,
                              const int32_t* positions, float theta, void* out, float sm_scale, void* stream) {
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (n > BC_MAX_ATTN_BATCH) return BC_ERR_INVALID_ARG;
  if (layer != c->append_next_layer) return BC_ERR_ORDER;
  uint8_t* q = work_ptr<uint8_t>(c, c->wl.rope_stage);
  uint8_t* k = q + (size_t)n * c->cfg.q_heads * c->cfg.head_dim * 2;
  uint8_t* v = k + (size_t)n * c->cfg.kv_heads * c->cfg.head_dim * 2;
  st = bc_rope_split(c, qkv, positions, n, theta, q, k, v, stream);
  if (st) return st;
  return bc_decode_step(c, layer, slots, n, q, k, v, out, sm_scale, stream);
}

bc_status bc_fill_step(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* q, const void* k,
                       const void* v, const void* beacon_q, const void* beacon_k, const void* beacon_v, void* out,
                       void* out_beacon, float sm_scale, void* stream) {
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (n > BC_MAX_ATTN_BATCH) return BC_ERR_INVALID_ARG;
  if (!q || !k || !v || !beacon_q || !beacon_k || !beacon_v || !out || !out_beacon) return BC_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(beacon_q) || !aligned16(beacon_k) || !aligned16(beacon_v) ||
      !aligned16(out) || !aligned16(out_beacon))
    return BC_ERR_INVALID_ARG;
  if (layer != c->append_next_layer || layer != c->compress_next_layer) return BC_ERR_ORDER;
  cudaStream_t s = (cudaStream_t)stream;
  if ((c->cfg.flags & BC_FLAG_ATTN_REFERENCE) || c->cfg.q_heads / c->cfg.kv_heads > 8) {   // no paired kernel: the three calls
    st = bc_append(c, layer, slots, n, k, v, stream);
    if (st) return st;
    st = bc_decode_attn_pair(c, layer, slots, n, q, out, beacon_q, out_beacon, sm_scale, beacon_k, beacon_v, stream);
    if (st) return st;
    return bc_compress(c, layer, slots, n, beacon_k, beacon_v, stream);
  }
  // the append's bookkeeping kernel (it leaves the plan and its flag), ONE attention launch that takes the token's
  // entry from the inputs and serves both sets of query heads, then the compression
  if (layer == 0) {
    st = append_book_only(c, slots, n, s, true);
    if (st) return st;
  }
  st = decode_step_attn(c, layer, slots, n, q, k, v, out, sm_scale, s, 1, beacon_q, beacon_k, beacon_v, out_beacon);
  if (st) return st;
  return bc_compress(c, layer, slots, n, beacon_k, beacon_v, stream);
}

bc_status bc_compress(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* bk, const void* bv,
                      void* stream) {
  if (c && layer == BC_ALL_LAYERS) {
    // one bookkeeping launch (allocate the beacon slot and evict the window at once: the beacon rows do not
    // depend on the eviction), then ONE launch that writes the beacon rows of every layer
    bc_status st = check_batch(c, 0, slots, n);
    if (st) return st;
    if (!bk || !bv || !aligned16(bk) || !aligned16(bv)) return BC_ERR_INVALID_ARG;
    if (c->compress_next_layer != 0) return BC_ERR_ORDER;
    cudaStream_t s = (cudaStream_t)stream;
    int32_t* row = work_ptr<int32_t>(c, c->wl.compress_row);
    int32_t* pos = work_ptr<int32_t>(c, c->wl.compress_pos);
    ++c->calls;
    BC_CUDA(c, bc_launch_compress_book(c->meta, slots, n, c->calls, row, pos, 3, c->geom, layer_base(c, 0), nullptr, nullptr, s));
    BC_CUDA(c, bc_launch_write_rows(c->meta, c->geom, layer_base(c, 0), row, pos, bk, bv, n, s, c->cfg.layers,
                                    (long long)c->geom.layer_bytes, (long long)n * c->cfg.kv_heads * c->cfg.head_dim * 2));
    c->launches += 2;
    c->meta_unsettled = false;
    return BC_OK;
  }
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (!bk || !bv || !aligned16(bk) || !aligned16(bv)) return BC_ERR_INVALID_ARG;
  if (layer != c->compress_next_layer) return BC_ERR_ORDER;
  int32_t* row = work_ptr<int32_t>(c, c->wl.compress_row);
  int32_t* pos = work_ptr<int32_t>(c, c->wl.compress_pos);
  cudaStream_t s = (cudaStream_t)stream;
  const int L = c->cfg.layers;
  // The beacon rows of layer 0 are written by the bookkeeping block itself when they are few (64 entries of 4 KB take
  // it 3 us): that kernel may run under the last blocks of the attention kernel ahead, which reads neither the
  // beacon slot being filled nor a page taken from the free stack, whereas a row-writing launch of its own waits
  // for that kernel to end.
  const bool fused = layer == 0 && (size_t)n * c->geom.entry_bytes <= kFusedBeaconRowBytes;
  if (layer == 0) {
    ++c->calls;
    // several layers: allocate now, evict on the last layer's call; a single layer: allocate and
    // evict at once (the beacon row does not depend on the eviction)
    BC_CUDA(c, bc_launch_compress_book(c->meta, slots, n, c->calls, row, pos, L > 1 ? 1 : 3, c->geom, layer_base(c, 0),
                                       fused ? bk : nullptr, fused ? bv : nullptr, s));
    c->launches += 1;
    c->meta_unsettled = true;
  }
  if (!fused) {
    BC_CUDA(c, bc_launch_write_rows(c->meta, c->geom, layer_base(c, layer), row, pos, bk, bv, n, s));
    c->launches += 1;
    c->meta_unsettled = false;
  }
  if (L > 1 && layer == L - 1) {
    BC_CUDA(c, bc_launch_compress_book(c->meta, slots, n, c->calls, row, pos, 2, c->geom, nullptr, nullptr, nullptr, s));
    c->launches += 1;
    c->meta_unsettled = true;
  }
  c->compress_next_layer = (layer + 1) % L;
  return BC_OK;
}

bc_status bc_seq_close(bc_cache* c, const int32_t* slots, int32_t n, void* stream) {
  if (!c || !slots || n <= 0 || n > c->cfg.max_seqs) return BC_ERR_INVALID_ARG;
  BC_CUDA(c, bc_launch_close(c->meta, slots, n, ++c->calls, (cudaStream_t)stream));
  c->launches += 1;
  c->meta_unsettled = true;
  return BC_OK;
}

namespace {

bc_status host_setup(bc_cache* c) {   // first host-buffer call on this cache
  if (c->copy_stream) return BC_OK;
  BC_CUDA(c, cudaStreamCreateWithFlags(&c->copy_stream, cudaStreamNonBlocking));
  for (cudaEvent_t& e : c->ev_in) BC_CUDA(c, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  for (cudaEvent_t& e : c->ev_done) BC_CUDA(c, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  if (c->cfg.flags & BC_FLAG_HOST_PIPELINED) {
    BC_CUDA(c, cudaStreamCreateWithFlags(&c->out_stream, cudaStreamNonBlocking));
    for (cudaEvent_t& e : c->ev_d2h) BC_CUDA(c, cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  }
  return BC_OK;
}

// Stream memory operations (driver entry points, looked up once): a 32-bit word in device memory written, or
// waited for, in the order of a stream, without a kernel.
typedef CUresult (*StreamValueFn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
StreamValueFn stream_value_fn(const char* name) {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) return nullptr;
  return reinterpret_cast<StreamValueFn>(p);
}
StreamValueFn stream_wait_value() { static StreamValueFn fn = stream_value_fn("cuStreamWaitValue32"); return fn; }
StreamValueFn stream_write_value() { static StreamValueFn fn = stream_value_fn("cuStreamWriteValue32"); return fn; }
#define BC_DRV(c, expr)                                               \
  do {                                                                \
    if ((expr) != CUDA_SUCCESS) return cuda_fail((c), cudaErrorUnknown); \
  } while (0)

inline int32_t* in_word(bc_cache* c, int buf) { return work_ptr<int32_t>(c, c->wl.host_words) + buf; }
inline int32_t* done_word(bc_cache* c) { return work_ptr<int32_t>(c, c->wl.host_words) + bc_cache::kStageRing; }

// The host-buffer steps whose completion no enqueued kernel vouches for yet get a one-thread kernel that does,
// behind everything enqueued on their stream so far.
bc_status vouch_for_host_steps(bc_cache* c) {
  if (c->done_issued == c->host_seq) return BC_OK;
  BC_CUDA(c, bc_launch_host_steps_done(done_word(c), c->host_seq, c->host_stream));
  c->launches += 1;
  c->done_issued = c->host_seq;
  return BC_OK;
}

// The copy stream waits until staging buffer `buf` has no reader left: the event of its last reader among the
// steps ordered by events, the done word for its last reader among the steps ordered by words.
bc_status wait_buffer_free(bc_cache* c, int buf) {
  if (c->buf_done[buf]) BC_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->buf_done[buf], 0));
  if (c->buf_reader_seq[buf])
    BC_DRV(c, stream_wait_value()((CUstream)c->copy_stream, (CUdeviceptr)done_word(c), (cuuint32_t)c->buf_reader_seq[buf],
                                  CU_STREAM_WAIT_VALUE_GEQ));
  return BC_OK;
}

// Stages k, v, q of a host-buffer step: the copies run on the cache's own copy stream, so the next
// steps' inputs travel while this step's kernels run; `s` waits for them before the kernels that read
// them.  Returns the staging buffer used.
bc_status stage_inputs(bc_cache* c, int32_t n, const void* q_host, const void* k_host, const void* v_host, cudaStream_t s,
                       int* buf_out, void** dq, void** dk, void** dv, int32_t word_seq = 0) {
  const int buf = c->stage_next;
  c->stage_next = (buf + 1) % bc_cache::kStageRing;
  const size_t qb = (size_t)n * c->cfg.q_heads * c->cfg.head_dim * 2, kb = (size_t)n * c->cfg.kv_heads * c->cfg.head_dim * 2;
  uint8_t* base = c->work + c->wl.stage_in[buf];
  *dk = base; *dv = base + kb; *dq = base + 2 * kb;
  // the buffer's previous readers (a whole turn of the ring ago) must be done
  {
    const bc_status st = wait_buffer_free(c, buf);
    if (st) return st;
  }
  // Pipelined outputs: the step that receives these inputs writes the output staging set whose last
  // copies to the host (two steps ago) must be over.  The copy stream waits for them here, so that the
  // one event the caller's stream waits for below covers both and no second wait sits between kernels.
  if (c->out_stream) BC_CUDA(c, cudaStreamWaitEvent(c->copy_stream, c->ev_d2h[c->out_next], 0));
  const uint8_t *kh = static_cast<const uint8_t*>(k_host), *vh = static_cast<const uint8_t*>(v_host),
                *qh = static_cast<const uint8_t*>(q_host);
  if (vh == kh + kb && qh == vh + kb) {   // one packed host buffer k | v | q: one copy
    BC_CUDA(c, cudaMemcpyAsync(base, kh, 2 * kb + qb, cudaMemcpyHostToDevice, c->copy_stream));
  } else {
    BC_CUDA(c, cudaMemcpyAsync(*dk, kh, kb, cudaMemcpyHostToDevice, c->copy_stream));
    BC_CUDA(c, cudaMemcpyAsync(*dv, vh, kb, cudaMemcpyHostToDevice, c->copy_stream));
    BC_CUDA(c, cudaMemcpyAsync(*dq, qh, qb, cudaMemcpyHostToDevice, c->copy_stream));
  }
  if (word_seq != 0) {   // the step's bookkeeping kernel polls the word: no wait on the caller's stream
    BC_DRV(c, stream_write_value()((CUstream)c->copy_stream, (CUdeviceptr)in_word(c, buf), (cuuint32_t)word_seq,
                                   CU_STREAM_WRITE_VALUE_DEFAULT));
    c->buf_reader_seq[buf] = word_seq;
    c->buf_done[buf] = nullptr;
  } else {
    BC_CUDA(c, cudaEventRecord(c->ev_in[buf], c->copy_stream));
    BC_CUDA(c, cudaStreamWaitEvent(s, c->ev_in[buf], 0));
    c->buf_reader_seq[buf] = 0;   // finish_step names the event of this step's readers
  }
  *buf_out = buf;
  return BC_OK;
}

// Output staging of a host-buffer step.  Plain mode: one set, the copies follow the kernels on `s`.
// Pipelined mode (BC_FLAG_HOST_PIPELINED): four sets in turn; the copies of a step run on the cache's
// output stream after its kernels, so the next step's kernels do not wait for them; `s` waits for
// them only in bc_host_outputs_ready.
bc_status begin_outputs(bc_cache* c, cudaStream_t s, int* set, void** dout, void** dout2) {
  *set = 0;
  if (c->cfg.flags & BC_FLAG_HOST_PIPELINED) {
    *set = c->out_next;   // its copies of four steps ago are over: the copy stream waited for them before this step's inputs
    c->out_next = (c->out_next + 1) % bc_cache::kOutSets;
  }
  *dout = c->work + c->wl.stage_out[*set];
  *dout2 = c->work + c->wl.stage_out2[*set];
  return BC_OK;
}

// What follows a host-buffer step's kernels: ONE event on the caller's stream (the input staging
// buffers the step read are free after it, and the output copies may start after it), then the copies
// of the outputs -- on `s` itself in plain mode, on the cache's output stream in pipelined mode.
bc_status finish_step(bc_cache* c, const bc_cache::Pending& p) {
  cudaEvent_t done = c->ev_done[c->done_next];
  c->done_next = (c->done_next + 1) % bc_cache::kDoneRing;
  BC_CUDA(c, cudaEventRecord(done, p.stream));
  for (int b : p.bufs) if (b >= 0) c->buf_done[b] = done;
  cudaStream_t cs = p.stream;
  if (c->cfg.flags & BC_FLAG_HOST_PIPELINED) {
    BC_CUDA(c, cudaStreamWaitEvent(c->out_stream, done, 0));
    cs = c->out_stream;
  }
  BC_CUDA(c, cudaMemcpyAsync(p.out_host, c->work + c->wl.stage_out[p.set], p.bytes, cudaMemcpyDeviceToHost, cs));
  if (p.out2_host) BC_CUDA(c, cudaMemcpyAsync(p.out2_host, c->work + c->wl.stage_out2[p.set], p.bytes, cudaMemcpyDeviceToHost, cs));
  if (c->cfg.flags & BC_FLAG_HOST_PIPELINED) BC_CUDA(c, cudaEventRecord(c->ev_d2h[p.set], cs));
  return BC_OK;
}

bc_status flush_pending(bc_cache* c) {
  {   // steps ordered by words that nothing vouches for yet: what follows is ordered by events
    const bc_status st = vouch_for_host_steps(c);
    if (st) return st;
  }
  if (!c->pending.valid) return BC_OK;
  c->pending.valid = false;
  if (c->pending.word_seq) {
    // A kernel that stores this step's number to the done word is enqueued by now (the next step's bookkeeping
    // kernel, or the one-thread kernel above): the wait below never depends on a call still to be made, so a
    // device-wide synchronisation by the caller cannot block on it.
    const bc_cache::Pending& p = c->pending;
    BC_DRV(c, stream_wait_value()((CUstream)c->out_stream, (CUdeviceptr)done_word(c), (cuuint32_t)p.word_seq, CU_STREAM_WAIT_VALUE_GEQ));
    BC_CUDA(c, cudaMemcpyAsync(p.out_host, c->work + c->wl.stage_out[p.set], p.bytes, cudaMemcpyDeviceToHost, c->out_stream));
    if (p.out2_host)
      BC_CUDA(c, cudaMemcpyAsync(p.out2_host, c->work + c->wl.stage_out2[p.set], p.bytes, cudaMemcpyDeviceToHost, c->out_stream));
    BC_CUDA(c, cudaEventRecord(c->ev_d2h[p.set], c->out_stream));
    return BC_OK;
  }
  return finish_step(c, c->pending);
}

// The end of a host-buffer call: in plain mode the step's event and output copies are issued at once;
// in pipelined mode they are left to the next host-buffer call (see bc_cache::Pending).
bc_status close_step(bc_cache* c, cudaStream_t s, int set, int buf, int buf2, void* out_host, void* out2_host, size_t bytes) {
  bc_cache::Pending p;
  p.valid = true; p.set = set; p.bufs[0] = buf; p.bufs[1] = buf2; p.out_host = out_host; p.out2_host = out2_host;
  p.bytes = bytes; p.stream = s;
  if (c->cfg.flags & BC_FLAG_HOST_PIPELINED) { c->pending = p; return BC_OK; }
  return finish_step(c, p);
}

}  // namespace

bc_status bc_host_outputs_ready(bc_cache* c, void* stream) {
  if (!c) return BC_ERR_INVALID_ARG;
  bc_status st = flush_pending(c);   // also vouches for the steps ordered by words
  if (st) return st;
  if (c->out_stream)
    for (int b = 0; b < bc_cache::kOutSets; ++b) BC_CUDA(c, cudaStreamWaitEvent((cudaStream_t)stream, c->ev_d2h[b], 0));
  return BC_OK;
}

bc_status bc_decode_step_host(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* q_host,
                              const void* k_host, const void* v_host, void* out_host, float sm_scale, void* stream) {
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (n > BC_MAX_ATTN_BATCH || !q_host || !k_host || !v_host || !out_host) return BC_ERR_INVALID_ARG;
  if (layer != c->append_next_layer) return BC_ERR_ORDER;
  cudaStream_t s = (cudaStream_t)stream;
  st = host_setup(c);
  if (st) return st;
  const size_t qb = (size_t)n * c->cfg.q_heads * c->cfg.head_dim * 2;
  const size_t ob = (c->cfg.flags & BC_FLAG_OUT_F32) ? qb * 2 : qb;
  const bool reference = (c->cfg.flags & BC_FLAG_ATTN_REFERENCE) != 0;
  if (c->cfg.layers == 1 && (c->cfg.flags & BC_FLAG_HOST_PIPELINED) && !reference && stream_wait_value() && stream_write_value()) {
    // Ordered by words (see bc_cache::host_seq): the caller's stream gets the bookkeeping kernel and the attention
    // kernel, nothing else, so the step overlaps with its neighbours exactly as a device-resident bc_decode_step.
    if ((c->pending.valid && !c->pending.word_seq) || c->host_stream != s) {
      // a step ordered by events is still owed its event and output copies; or the caller changed streams: the
      // steps so far are vouched for on the stream they were enqueued on
      st = flush_pending(c);
      if (st) return st;
      c->host_stream = s;
    }
    const int32_t prev = c->host_seq;
    int32_t id = prev + 1;
    if (id == 0) id = 1;
    void *dq, *dk, *dv, *dout, *dout2;
    int buf, set;
    st = stage_inputs(c, n, q_host, k_host, v_host, s, &buf, &dq, &dk, &dv, id);   // also waits for the output set's last copies
    if (st) return st;
    st = begin_outputs(c, s, &set, &dout, &dout2);
    if (st) return st;
    BcHostSync hs = {in_word(c, buf), id, prev ? done_word(c) : nullptr, prev, nullptr};
    st = append_book_only(c, slots, n, s, true, &hs);
    if (st) return st;
    c->done_issued = prev;       // that kernel vouches for every step before this one ...
    st = flush_pending(c);       // ... so the last step's output rows may be sent on their way now
    if (st) return st;
    c->host_seq = id;
    st = decode_step_attn(c, layer, slots, n, dq, dk, dv, dout, sm_scale, s);
    if (st) return st;
    // this step's output rows leave with the next host-buffer call, bc_host_outputs_ready or bc_cache_destroy
    bc_cache::Pending p;
    p.valid = true; p.set = set; p.out_host = out_host; p.bytes = ob; p.stream = s; p.word_seq = id;
    c->pending = p;
    return BC_OK;
  }
  // The step's bookkeeping needs nothing from the host, so it goes out first, directly behind the last
  // step's attention kernel (under whose last blocks it may start); only then the events and copies
  // that the last step still owes, and this step's own copies.
  if (layer == 0 && !reference) {
    st = append_book_only(c, slots, n, s, true);
    if (st) return st;
  }
  st = flush_pending(c);
  if (st) return st;
  void *dq, *dk, *dv, *dout, *dout2;
  int buf, set;
  st = stage_inputs(c, n, q_host, k_host, v_host, s, &buf, &dq, &dk, &dv);
  if (st) return st;
  st = begin_outputs(c, s, &set, &dout, &dout2);
  if (st) return st;
  if (reference) {
    st = bc_decode_step(c, layer, slots, n, dq, dk, dv, dout, sm_scale, stream);
  } else {
    st = decode_step_attn(c, layer, slots, n, dq, dk, dv, dout, sm_scale, s);
  }
  if (st) return st;
  return close_step(c, s, set, buf, -1, out_host, nullptr, ob);
}

bc_status bc_fill_step_host(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* q_host,
                            const void* k_host, const void* v_host, const void* bq_host, const void* bk_host,
                            const void* bv_host, void* out_host, void* out_beacon_host, float sm_scale, void* stream) {
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (n > BC_MAX_ATTN_BATCH || !q_host || !k_host || !v_host || !bq_host || !bk_host || !bv_host || !out_host || !out_beacon_host)
    return BC_ERR_INVALID_ARG;
  if (layer != c->append_next_layer || layer != c->compress_next_layer) return BC_ERR_ORDER;
  cudaStream_t s = (cudaStream_t)stream;
  st = host_setup(c);
  if (st) return st;
  const size_t qb = (size_t)n * c->cfg.q_heads * c->cfg.head_dim * 2;
  const size_t ob = (c->cfg.flags & BC_FLAG_OUT_F32) ? qb * 2 : qb;
  void *dq, *dk, *dv, *dbq, *dbk, *dbv, *dout, *dout2;
  int buf, buf2, set;
  const bool paired_kernel = !(c->cfg.flags & BC_FLAG_ATTN_REFERENCE) && c->cfg.q_heads / c->cfg.kv_heads <= 8;
  if (paired_kernel && c->cfg.layers == 1 && (c->cfg.flags & BC_FLAG_HOST_PIPELINED) && stream_wait_value() && stream_write_value()) {
    // Ordered by words, like the regular step (see bc_decode_step_host): the bookkeeping kernel polls the words of
    // both sets of inputs; the caller's stream carries the kernels of bc_fill_step and nothing else.
    if ((c->pending.valid && !c->pending.word_seq) || c->host_stream != s) {
      st = flush_pending(c);
      if (st) return st;
      c->host_stream = s;
    }
    const int32_t prev = c->host_seq;
    int32_t id = prev + 1;
    if (id == 0) id = 1;
    st = stage_inputs(c, n, q_host, k_host, v_host, s, &buf, &dq, &dk, &dv, id);
    if (st) return st;
    st = stage_inputs(c, n, bq_host, bk_host, bv_host, s, &buf2, &dbq, &dbk, &dbv, id);
    if (st) return st;
    st = begin_outputs(c, s, &set, &dout, &dout2);
    if (st) return st;
    BcHostSync hs = {in_word(c, buf), id, prev ? done_word(c) : nullptr, prev, in_word(c, buf2)};
    st = append_book_only(c, slots, n, s, true, &hs);
    if (st) return st;
    c->done_issued = prev;
    st = flush_pending(c);
    if (st) return st;
    c->host_seq = id;
    st = decode_step_attn(c, layer, slots, n, dq, dk, dv, dout, sm_scale, s, 1, dbq, dbk, dbv, dout2);
    if (st) return st;
    st = bc_compress(c, layer, slots, n, dbk, dbv, stream);
    if (st) return st;
    bc_cache::Pending p;
    p.valid = true; p.set = set; p.out_host = out_host; p.out2_host = out_beacon_host; p.bytes = ob; p.stream = s; p.word_seq = id;
    c->pending = p;
    return BC_OK;
  }
  // as in bc_decode_step_host: the append's bookkeeping first (when its rows go out in a launch of their own, or
  // when the attention kernel takes them from the inputs)
  const bool rows_apart = (size_t)n * c->geom.entry_bytes > kFusedRowBytes;
  bool book_done = false;
  if (layer == 0 && (rows_apart || paired_kernel)) {
    st = append_book_only(c, slots, n, s, paired_kernel);
    if (st) return st;
    book_done = true;
  }
  st = flush_pending(c);
  if (st) return st;
  st = stage_inputs(c, n, q_host, k_host, v_host, s, &buf, &dq, &dk, &dv);
  if (st) return st;
  st = stage_inputs(c, n, bq_host, bk_host, bv_host, s, &buf2, &dbq, &dbk, &dbv);
  if (st) return st;
  st = begin_outputs(c, s, &set, &dout, &dout2);
  if (st) return st;
  if (paired_kernel) {   // one attention launch appends the token's entry and serves both sets of rows
    st = decode_step_attn(c, layer, slots, n, dq, dk, dv, dout, sm_scale, s, 1, dbq, dbk, dbv, dout2);
    if (st) return st;
    st = bc_compress(c, layer, slots, n, dbk, dbv, stream);
    if (st) return st;
    return close_step(c, s, set, buf, buf2, out_host, out_beacon_host, ob);
  }
  if (book_done || (layer > 0 && rows_apart)) {   // the rows of this layer (the bookkeeping is done, or was done on layer 0)
    BC_CUDA(c, bc_launch_write_rows(c->meta, c->geom, layer_base(c, layer), work_ptr<int32_t>(c, c->wl.append_row[c->append_set]),
                                    work_ptr<int32_t>(c, c->wl.append_pos[c->append_set]), dk, dv, n, s));
    c->launches += 1;
    c->meta_unsettled = false;
    c->append_next_layer = (layer + 1) % c->cfg.layers;
  } else {
    st = bc_append(c, layer, slots, n, dk, dv, stream);
    if (st) return st;
  }
  st = bc_decode_attn_pair(c, layer, slots, n, dq, dout, dbq, dout2, sm_scale, dbk, dbv, stream);
  if (st) return st;
  st = bc_compress(c, layer, slots, n, dbk, dbv, stream);
  if (st) return st;
  return close_step(c, s, set, buf, buf2, out_host, out_beacon_host, ob);
}

bc_status bc_compress_step_host(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* bq_host,
                                const void* bk_host, const void* bv_host, void* out_host, float sm_scale, void* stream) {
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (n > BC_MAX_ATTN_BATCH || !bq_host || !bk_host || !bv_host || !out_host) return BC_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  st = host_setup(c);
  if (st) return st;
  st = flush_pending(c);
  if (st) return st;
  const size_t qb = (size_t)n * c->cfg.q_heads * c->cfg.head_dim * 2;
  const size_t ob = (c->cfg.flags & BC_FLAG_OUT_F32) ? qb * 2 : qb;
  void *dq, *dk, *dv, *dout, *dout2;
  int buf, set;
  st = stage_inputs(c, n, bq_host, bk_host, bv_host, s, &buf, &dq, &dk, &dv);
  if (st) return st;
  st = begin_outputs(c, s, &set, &dout, &dout2);
  if (st) return st;
  st = attn_impl(c, layer, slots, n, dq, dout, sm_scale, dk, dv, s);
  if (st) return st;
  st = bc_compress(c, layer, slots, n, dk, dv, stream);
  if (st) return st;
  return close_step(c, s, set, buf, -1, out_host, nullptr, ob);
}

bc_status bc_get_state(bc_cache* c, int32_t slot, bc_seq_state* out, int32_t* pages, int32_t pages_cap, void* stream) {
  if (!c || !out || slot < 0 || slot >= c->cfg.max_seqs) return BC_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  BC_CUDA(c, cudaStreamSynchronize(s));
  auto rd = [&](int32_t* arr, int32_t* dst) { return cudaMemcpy(dst, arr + slot, 4, cudaMemcpyDeviceToHost); };
  int32_t woff = 0, boff = 0;
  BC_CUDA(c, rd(c->meta.open, &out->open));
  BC_CUDA(c, rd(c->meta.prompt_len, &out->prompt_len));
  BC_CUDA(c, rd(c->meta.n_beacons, &out->n_beacons));
  BC_CUDA(c, rd(c->meta.window_len, &out->window_len));
  BC_CUDA(c, rd(c->meta.c, &out->c));
  BC_CUDA(c, rd(c->meta.t, &out->t));
  BC_CUDA(c, rd(c->meta.window_off, &woff));
  BC_CUDA(c, rd(c->meta.beacon_off, &boff));
  const int ps = c->cfg.page_size;
  out->n_prompt_pages = (out->prompt_len + ps - 1) / ps;
  out->n_beacon_pages = (out->n_beacons + ps - 1) / ps;
  out->n_window_pages = (out->window_len + ps - 1) / ps;
  if (pages && pages_cap > 0 && out->open) {
    std::vector<int32_t> row(c->cfg.max_pages_per_seq);
    BC_CUDA(c, cudaMemcpy(row.data(), c->meta.page_table + (int64_t)slot * c->cfg.max_pages_per_seq, row.size() * 4,
                          cudaMemcpyDeviceToHost));
    int o = 0;
    for (int k = 0; k < out->n_prompt_pages && o < pages_cap; ++k) pages[o++] = row[k];
    for (int k = 0; k < out->n_beacon_pages && o < pages_cap; ++k) pages[o++] = row[boff + k];
    for (int k = 0; k < out->n_window_pages && o < pages_cap; ++k) pages[o++] = row[woff + k];
  }
  return BC_OK;
}

bc_status bc_get_free_list(bc_cache* c, int32_t* pages, int32_t* count, void* stream) {
  if (!c || !pages || !count) return BC_ERR_INVALID_ARG;
  BC_CUDA(c, cudaStreamSynchronize((cudaStream_t)stream));
  BC_CUDA(c, cudaMemcpy(count, c->meta.free_top, 4, cudaMemcpyDeviceToHost));
  if (*count < 0 || *count > c->cfg.num_pages) return BC_ERR_INVALID_ARG;
  if (*count) BC_CUDA(c, cudaMemcpy(pages, c->meta.free_stack, (size_t)*count * 4, cudaMemcpyDeviceToHost));
  return BC_OK;
}

bc_status bc_poll_error(bc_cache* c, int32_t* code, int32_t* slot, int64_t* call_index, void* stream) {
  if (!c || !code) return BC_ERR_INVALID_ARG;
  BC_CUDA(c, cudaStreamSynchronize((cudaStream_t)stream));
  int32_t rec[4];
  BC_CUDA(c, cudaMemcpy(rec, c->meta.status, 16, cudaMemcpyDeviceToHost));
  *code = rec[0];
  if (slot) *slot = rec[1];
  if (call_index) memcpy(call_index, rec + 2, 8);
  return BC_OK;
}

bc_status bc_clear_error(bc_cache* c, void* stream) {
  if (!c) return BC_ERR_INVALID_ARG;
  BC_CUDA(c, cudaMemsetAsync(c->meta.status, 0, 16, (cudaStream_t)stream));
  // an attention launch that gave up (BC_ERR_TIMEOUT) may have left ticket counters non-zero
  BC_CUDA(c, cudaMemsetAsync(c->work + c->wl.tickets, 0, (size_t)BC_MAX_ATTN_BATCH * 4 * c->cfg.layers, (cudaStream_t)stream));
  // The counters of the built-in array are shared by every cache of the process: they are touched
  // only when THIS cache has used the static entry point since its last clear (a launch of its own
  // may have left them non-zero), never on behalf of a cache that did not.
  if (c->static_used) {
    BC_CUDA(c, static_scratch_reset_tickets((cudaStream_t)stream));
    c->static_used = false;
  }
  return BC_OK;
}

bc_status bc_export_seq(bc_cache* c, int32_t layer, int32_t slot, void* k_out, void* v_out, int32_t capacity,
                        void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.layers || slot < 0 || slot >= c->cfg.max_seqs || !k_out || !v_out ||
      capacity < 0 || !aligned16(k_out) || !aligned16(v_out))
    return BC_ERR_INVALID_ARG;
  BC_CUDA(c, bc_launch_export(c->meta, c->geom, layer_base(c, layer), slot, k_out, v_out, capacity, (cudaStream_t)stream));
  c->launches += 1;
  return BC_OK;
}

bc_status bc_set_attn_ctas(bc_cache* c, int32_t ctas) {
  if (!c || ctas < 0 || ctas > BC_MAX_ATTN_CTAS) return BC_ERR_INVALID_ARG;
  c->attn_ctas = ctas;
  return BC_OK;
}

bc_status bc_set_wait_limit(bc_cache* c, uint32_t polls) {
  if (!c) return BC_ERR_INVALID_ARG;
  if (polls != 0 && (c->cfg.head_dim != 128 || c->cfg.q_heads / c->cfg.kv_heads > 8)) return BC_ERR_UNSUPPORTED;
  c->wait_limit = polls;
  return BC_OK;
}

bc_status bc_attn_timeline(bc_cache* c, void* device_words, int32_t blocks) {
  if (!c) return BC_ERR_INVALID_ARG;
  if (device_words == nullptr) { c->timeline = nullptr; return BC_OK; }
  if ((reinterpret_cast<uintptr_t>(device_words) & 7) || blocks < BC_MAX_ATTN_CTAS) return BC_ERR_INVALID_ARG;
  c->timeline = device_words;
  return BC_OK;
}

bc_status bc_profile_enable(bc_cache* c, int32_t max_launches) {
  if (!c || max_launches < 0) return BC_ERR_INVALID_ARG;
  while ((int)c->ev.size() < 2 * max_launches) {
    cudaEvent_t e;
    BC_CUDA(c, cudaEventCreate(&e));
    c->ev.push_back(e);
  }
  c->prof_cap = max_launches;
  c->prof_used = 0;
  return BC_OK;
}

bc_status bc_profile_read(bc_cache* c, int32_t* launches, float* total_ms) {
  if (!c || !launches || !total_ms) return BC_ERR_INVALID_ARG;
  float sum = 0.f;
  for (int i = 0; i < c->prof_used; ++i) {
    BC_CUDA(c, cudaEventSynchronize(c->ev[2 * i + 1]));
    float ms = 0.f;
    BC_CUDA(c, cudaEventElapsedTime(&ms, c->ev[2 * i], c->ev[2 * i + 1]));
    sum += ms;
  }
  *launches = c->prof_used;
  *total_ms = sum;
  c->prof_cap = 0;
  c->prof_used = 0;
  return BC_OK;
}

bc_status bc_decode_attn_static(bc_cache* c, int32_t layer, const int32_t* slots, int32_t n, const void* q, void* out,
                                float sm_scale, const void* extra_k, const void* extra_v, void* stream) {
  if (c && layer == BC_ALL_LAYERS) {   // as bc_decode_attn: tensors with a leading [layers] dimension, layer by layer
    if (n <= 0) return BC_ERR_INVALID_ARG;
    const size_t qb = (size_t)n * c->cfg.q_heads * c->cfg.head_dim * 2, kb = (size_t)n * c->cfg.kv_heads * c->cfg.head_dim * 2;
    const size_t ob = (c->cfg.flags & BC_FLAG_OUT_F32) ? qb * 2 : qb;
    for (int l = 0; l < c->cfg.layers; ++l) {
      const bc_status st = bc_decode_attn_static(c, l, slots, n, layer_slice(q, l, qb), layer_slice(out, l, ob), sm_scale,
                                                 layer_slice(extra_k, l, kb), layer_slice(extra_v, l, kb), stream);
      if (st) return st;
    }
    return BC_OK;
  }
  bc_status st = check_batch(c, layer, slots, n);
  if (st) return st;
  if (!q || !out || !aligned16(q) || !aligned16(out)) return BC_ERR_INVALID_ARG;
  if ((extra_k == nullptr) != (extra_v == nullptr)) return BC_ERR_INVALID_ARG;
  if (extra_k && (!aligned16(extra_k) || !aligned16(extra_v))) return BC_ERR_INVALID_ARG;
  if (n > BC_STATIC_MAX_BATCH || c->cfg.q_heads * c->cfg.head_dim > BC_MERGE_ELEMS || c->cfg.q_heads > 64)
    return BC_ERR_TOO_LARGE;
  // the built-in array is per device: the one that is looked up must be the one the cache lives on
  int dev = -1;
  BC_CUDA(c, cudaGetDevice(&dev));
  if (dev != c->device) return BC_ERR_INVALID_ARG;
  BcAttnArgs a;
  a.pool_layer = layer_base(c, layer);
  a.slots = slots; a.n = n; a.q = q; a.out = out;
  a.out_f32 = (c->cfg.flags & BC_FLAG_OUT_F32) ? 1 : 0;
  a.extra_k = extra_k; a.extra_v = extra_v; a.sm_scale = sm_scale;
  if (c->cfg.flags & BC_FLAG_ATTN_REFERENCE) {   // the debugging kernel needs no scratch at all
    a.part_o = nullptr; a.part_ml = nullptr; a.tickets = nullptr; a.ctas = 0;
    BC_CUDA(c, bc_launch_attn_reference(c->meta, c->geom, a, (cudaStream_t)stream));
    c->launches += 1;
    return BC_OK;
  }
  unsigned char* base = nullptr;
  BC_CUDA(c, static_scratch(&base));
  a.part_o = reinterpret_cast<float*>(base);
  a.part_ml = reinterpret_cast<float*>(base + kStaticPartO);
  a.tickets = reinterpret_cast<int32_t*>(base + kStaticPartO + kStaticPartMl);
  int ctas = c->attn_ctas > 0 ? c->attn_ctas : c->sm_count;
  a.ctas = ctas < BC_STATIC_MAX_CTAS ? ctas : BC_STATIC_MAX_CTAS;
  int launches = 0;
  a.spin_limit = c->wait_limit;
  a.debug = c->meta.debug;
  a.meta_settled = c->meta_unsettled ? 0 : 1;
  c->meta_unsettled = false;
  c->static_used = true;
  BC_CUDA(c, bc_launch_attn(c->meta, c->geom, a, nullptr, (cudaStream_t)stream, nullptr, nullptr, &launches));
  c->launches += launches;
  return BC_OK;
}

bc_status bc_probe_read_stream(const void* device_buf, size_t bytes, void* stream) {
  if (!device_buf || bytes < (64u << 10) || (reinterpret_cast<uintptr_t>(device_buf) & 15)) return BC_ERR_INVALID_ARG;
  return bc_launch_read_stream(device_buf, bytes, nullptr, (cudaStream_t)stream) == cudaSuccess ? BC_OK : BC_ERR_CUDA;
}

int64_t bc_kernel_launches(const bc_cache* c) { return c ? c->launches : 0; }
int32_t bc_last_cuda_error(const bc_cache* c) { return c ? c->last_cuda_error : 0; }

}  // extern "C"
