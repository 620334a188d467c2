// Shared declarations of the breadcrumbs library: device-side views of the bookkeeping, the
// store layout helpers and the kernel launch wrappers implemented in the .cu files.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "breadcrumbs.h"

// Upper bounds the workspace is sized for.
#define BC_MAX_ATTN_CTAS 304   // thread blocks of the decode-attention kernel
#define BC_MAX_ATTN_BATCH 512  // sequences per bc_decode_attn call
#define BC_MERGE_ELEMS 4096    // q_heads * head_dim that fits the in-block merge buffer
// The attention plan the append bookkeeping can leave for the fused decode step: BC_PLAN_HEADER ints
// {n, total tiles, log2(rows per tile), -}, then seven arrays of BC_MAX_ATTN_BATCH (+1 for the last) ints:
// prompt length, beacons, window length, slot (| BC_PLAN_NEW_ROW if the step appended an entry), first
// beacon column, first window column, and the exclusive prefix sums of the sequences' tile counts.
#define BC_PLAN_HEADER 4
#define BC_PLAN_INTS (BC_PLAN_HEADER + 7 * BC_MAX_ATTN_BATCH + 4)
#define BC_PLAN_NEW_ROW (1 << 30)
#define BC_TIMELINE_SLOTS 16   // 64-bit words per thread block in a bc_attn_timeline buffer

// Device view of the bookkeeping ("meta" buffer).  All arrays are int32.
struct BcMeta {
  int32_t* status;      // [0] code, [1] slot, [2..3] call index (int64)
  int32_t* free_top;    // number of free pages
  int32_t* free_stack;  // [num_pages]; free_stack[top-1] is handed out next
  int32_t* open;        // [max_seqs] 1 = open
  int32_t* prompt_len;  // [max_seqs]
  int32_t* n_beacons;   // [max_seqs]
  int32_t* window_len;  // [max_seqs]
  int32_t* c;           // [max_seqs]
  int32_t* t;           // [max_seqs] generated entries appended so far
  int32_t* window_off;  // [max_seqs] column of the first window page in the page-table row
  int32_t* beacon_off;  // [max_seqs] column of the first beacon page
  int32_t* page_table;  // [max_seqs][max_pages_per_seq]: prompt pages from column 0
  unsigned long long* dup_mark;  // [max_seqs] BC_FLAG_DEBUG_BOUNDS: (call index << 32 | ~first batch index) of the last call naming the slot
  int32_t max_seqs, num_pages, max_pages_per_seq, max_entries, page_size, c_default;
  int32_t debug;        // BC_FLAG_DEBUG_BOUNDS set
};

// Geometry of the K/V pool for one cache.
struct BcGeom {
  int32_t kv_heads, q_heads, head_dim, page_size;
  int32_t entry_bytes;       // E = 2 * kv_heads * head_dim * 2
  int32_t head_row_bytes;    // head_dim * 2
  int64_t layer_bytes;       // num_pages * page_size * E
};

// Byte offset, inside one entry, of 16-byte chunk j of (K|V = which, head h) for an entry whose
// position inside its segment is pos: the chunk index is XOR-permuted with pos & 7.
__host__ __device__ __forceinline__ int bc_chunk_offset(const BcGeom& g, int which, int h, int j, int pos) {
  return (which * g.kv_heads + h) * g.head_row_bytes + ((j ^ (pos & 7)) << 4);
}

// ---- launch wrappers (bc_book.cu) ------------------------------------------------------------
cudaError_t bc_launch_init(const BcMeta& m, cudaStream_t s);
cudaError_t bc_launch_open(const BcMeta& m, const int32_t* slots, const int32_t* plens, const int32_t* cs,
                           int n, int64_t call, cudaStream_t s);
// k, v non-null: the same launch also writes the rows into pool_layer (what bc_launch_write_rows
// does), which saves a launch when the batch is small enough for one thread block to copy.
// plan non-null (k, v null): the launch also leaves the attention plan of the batch (BC_PLAN_INTS ints) and
// then stores `epoch` to *flag with release semantics
// Host-buffer steps whose copies are tied to the kernels by words in device memory instead of events on the
// caller's stream: the bookkeeping kernel waits (bounded) until *in_word == in_seq before it lets the attention
// kernel read the step's inputs, and stores done_seq to *done_word when everything ahead of it has ended.
struct BcHostSync {
  const int32_t* in_word;   // NULL: no wait
  int32_t in_seq;
  int32_t* done_word;       // NULL: no store
  int32_t done_seq;
  const int32_t* in_word2;  // the step that fills a window has two sets of inputs (token, beacon); NULL: one
};
cudaError_t bc_launch_host_steps_done(int32_t* done_word, int32_t seq, cudaStream_t s);
cudaError_t bc_launch_append_book(const BcMeta& m, const int32_t* slots, int n, int64_t call, int32_t* dst_row,
                                  int32_t* dst_pos, const BcGeom& g, uint8_t* pool_layer, const void* k, const void* v,
                                  cudaStream_t s, int32_t* plan = nullptr, int32_t* flag = nullptr, int32_t epoch = 0,
                                  const BcHostSync* hs = nullptr);
// phase bit 1: allocate the beacon slot; phase bit 2: evict the window and bump the counters
cudaError_t bc_launch_compress_book(const BcMeta& m, const int32_t* slots, int n, int64_t call, int32_t* dst_row,
                                    int32_t* dst_pos, int phase, const BcGeom& g, uint8_t* pool_layer, const void* k,
                                    const void* v, cudaStream_t s);
cudaError_t bc_launch_close(const BcMeta& m, const int32_t* slots, int n, int64_t call, cudaStream_t s);
// m is used for the checks of BC_FLAG_DEBUG_BOUNDS only
cudaError_t bc_launch_write_rows(const BcMeta& m, const BcGeom& g, uint8_t* pool_layer, const int32_t* dst_row, const int32_t* dst_pos,
                                 const void* k, const void* v, int n, cudaStream_t s, int layers = 1, long long ls_pool = 0,
                                 long long ls_kv = 0);   // layers > 1: the rows of every layer ([layers][n] inputs) in one launch
cudaError_t bc_launch_restore_book(const BcMeta& m, const int32_t* slots, const int32_t* cu, int n, int64_t call, int32_t* ok,
                                   int32_t* bea, cudaStream_t s);
cudaError_t bc_launch_restore_rows(const BcMeta& m, const BcGeom& g, uint8_t* pool_layer, const int32_t* slots, const int32_t* ok,
                                   const int32_t* bea, const int32_t* cu, int n, int total_tokens, int total_beacons,
                                   const void* tok_k, const void* tok_v, const void* bea_k, const void* bea_v, cudaStream_t s);
cudaError_t bc_launch_prefill(const BcMeta& m, const BcGeom& g, uint8_t* pool_layer, const int32_t* slots,
                              const int32_t* cu, int n, int total, const void* k, const void* v, cudaStream_t s);
cudaError_t bc_launch_export(const BcMeta& m, const BcGeom& g, const uint8_t* pool_layer, int slot, void* k_out,
                             void* v_out, int capacity, cudaStream_t s);

// ---- attention (bc_attn.cu) ----------------------------------------------------------------------
struct BcAttnArgs {
  const uint8_t* pool_layer;
  const int32_t* slots;
  int32_t n;
  const void* q;
  void* out;
  int32_t out_f32;
  const void* extra_k;
  const void* extra_v;
  float sm_scale;
  float* part_o;         // [(ctas + n)][q_heads][head_dim]
  float* part_ml;        // [(ctas + n)][q_heads][2]
  int32_t* tickets;      // [n] pieces of each sequence published so far; zero between launches
  int32_t ctas;
  void* timeline = nullptr;  // NULL, or the device buffer of bc_attn_timeline
  uint32_t spin_limit = 0;   // 0: the default poll limit of the bounded waits
  int32_t debug = 0;         // BC_FLAG_DEBUG_BOUNDS
  int32_t meta_settled = 0;  // 1: the kernel that last wrote this cache's metadata has ended by the time this launch may begin
  // layer == BC_ALL_LAYERS as one launch: the number of layers and the byte strides from one layer to the next of
  // the pool, q, out, the extra (or new) K/V rows and the partial buffers; tickets: counters per layer
  int32_t layers = 1;
  int64_t ls_pool = 0, ls_q = 0, ls_out = 0, ls_kv = 0, ls_part_o = 0, ls_part_ml = 0;
  int32_t ls_tickets = 0;
  // the paired form (NULL otherwise): the beacons' queries, their outputs and their partial buffers
  const void* q2 = nullptr;
  void* out2 = nullptr;
  float* part_o2 = nullptr;
  float* part_ml2 = nullptr;
};
// Configures the kernels once per process/device (shared-memory opt-in).  Returns the SM count.
cudaError_t bc_attn_setup(int* sm_count);
// The append half of a fused decode step (bc_decode_step): the new entries and where they go.
struct BcFusedAppend {
  const void* new_k;     // [n][kv_heads][head_dim] bf16
  const void* new_v;
  int32_t* dst_row;      // [n] workspace: pool row of each item's new entry, -1 if refused (written on layer 0)
  int32_t* dst_pos;      // [n] workspace: its position in the window
  uint8_t* pool_layer;   // the layer's pool (writable)
  const int32_t* plan;   // NULL, or the plan the step's bookkeeping kernel left (BC_PLAN_INTS ints)
  int32_t* flag;         // workspace word: "the bookkeeping of launch `epoch` is done"
  int32_t epoch;
  int64_t call;          // bookkeeping call index (error latch)
};
// Launches the pipelined decode-attention kernel (the split combine is part of it); with `fused`
// the same launch appends the step's new entries first.  *launches gets the number of kernels.
cudaError_t bc_launch_attn(const BcMeta& m, const BcGeom& g, const BcAttnArgs& a, const BcFusedAppend* fused,
                           cudaStream_t s, cudaEvent_t ev_start, cudaEvent_t ev_stop, int* launches);
// Decoder-layer operators around the cache calls (bc_model_ops.cu).
cudaError_t bc_launch_add_rmsnorm(const void* h, const void* delta, const void* weight, int n, int hidden, float eps, void* h_out,
                                  void* normed, cudaStream_t s);
cudaError_t bc_launch_swiglu(const void* gate_up, int n, int m, void* out, cudaStream_t s);
cudaError_t bc_launch_argmax(const void* logits, int n, int vocab, long long* out, cudaStream_t s);
int bc_rmsnorm_max_hidden();
// Rotary embedding of the q and k heads of n packed QKV rows, split into three contiguous arrays.
cudaError_t bc_launch_rope_split(const void* qkv, const int32_t* positions, int n, int q_heads, int kv_heads, int head_dim,
                                 double theta, void* q_out, void* k_out, void* v_out, cudaStream_t s);
// Read-only streaming probe: reads bytes (rounded down to 64 KB) of buf once with the attention kernel's copy pattern.
cudaError_t bc_launch_read_stream(const void* buf, size_t bytes, int* sink, cudaStream_t s);
// Slow device reference (one warp per query head).
cudaError_t bc_launch_attn_reference(const BcMeta& m, const BcGeom& g, const BcAttnArgs& a, cudaStream_t s);
