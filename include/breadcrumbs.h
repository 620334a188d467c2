/*
 * breadcrumbs.h - C ABI of libbreadcrumbs.so
 *
 * Batched decode-step attention over a beacon-compressed, paged bf16 KV cache, and the
 * compress-and-evict step, for NVIDIA B200 (sm_100a).
 *
 * The method (Breadcrumbs Reasoning, Algorithm 1 and Section 3.1 of the paper): a sequence's
 * cache holds the prompt entries, one "beacon" entry per completed window of c generated tokens,
 * and the live entries of the current window.  When the window holds c tokens, a beacon token is
 * run through the model; its query attends to prompt + earlier beacons + the window + itself, its
 * K/V entry is appended and the c window entries are evicted.  Attention itself is ordinary
 * softmax attention over whatever the cache holds (Section 2; Figure 2 caption).  The model
 * forward pass is not part of this library: q, k, v and the beacon's k, v are inputs.
 *
 * Conventions
 *  - Every function returns a bc_status (0 = BC_OK, negative = error).  Nothing throws, aborts or
 *    traps on the device.
 *  - "device pointer" = memory of the current CUDA device, owned by the caller, 16-byte aligned,
 *    contiguous; the library never allocates or frees device memory.  "host pointer" = ordinary
 *    host memory.  `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *  - Hot-path calls only enqueue work on `stream` and return; they never synchronise, so a decode
 *    step can be captured in a CUDA graph.  Argument errors are returned at once.  State errors
 *    found on the device (no free page, window full, ...) make the operation a no-op for that
 *    sequence and are latched in a device status record read by bc_poll_error: the first call
 *    in which an item fails writes the record, and of that call's failing items the one with the
 *    lowest batch index is recorded (whichever check it failed); later failures change nothing
 *    until bc_clear_error.
 *  - Tensors are bf16.  K/V tensors are [n, kv_heads, head_dim]; q and out are
 *    [n, q_heads, head_dim]; query head h reads KV head h / (q_heads / kv_heads).
 *  - Layers: `layer` in [0, layers) addresses one layer.  A sequence's bookkeeping (lengths, page
 *    table) is shared by all layers and changes once per step: bc_append reserves the new slot on
 *    its layer-0 call, bc_compress allocates the beacon slot on its layer-0 call and evicts the
 *    window on its call for the last layer.  For one step, call the layers in ascending order
 *    with the same `slots`; anything else returns BC_ERR_ORDER.  bc_prefill, bc_append,
 *    bc_decode_attn, bc_decode_step and bc_compress also take layer = BC_ALL_LAYERS (-1): every
 *    per-layer tensor of the call (k, v, q, out, extra_k, extra_v, beacon_k, beacon_v) then carries
 *    a leading [layers] dimension and the call covers layer 0 .. layers - 1; results are those of
 *    the per-layer calls in ascending order (a forward pass computes layer l + 1's inputs from
 *    layer l's output, so this form serves replays and measurements, not a model).  The call is
 *    legal where the layer-0 call would be (else BC_ERR_ORDER) and leaves the order at layer 0.
 *    Launches: bc_decode_attn and bc_decode_step run ONE attention kernel whose grid's second
 *    dimension is the layer (the blocks of a layer are dispatched as those of the layer before
 *    retire; every layer has its own split-K counters and partial buffers in the workspace), after
 *    the one bookkeeping kernel in the case of bc_decode_step; bc_append and bc_compress run their
 *    bookkeeping kernel and ONE kernel that writes the rows of every layer (bc_compress allocates
 *    the beacon slot and evicts the window in the same bookkeeping launch).  bc_prefill, the
 *    static entry point and a cache with BC_FLAG_ATTN_REFERENCE run one launch sequence per layer.
 *  - A batch must not name the same slot twice.
 *  - Overlap (programmatic stream serialisation).  Three kinds of kernel of this library may begin
 *    before the kernel enqueued just ahead of them on `stream` has ended, provided that kernel
 *    releases its dependents early; after any other kernel (the caller's own, a copy) they keep
 *    plain stream order.
 *      (1) The bookkeeping kernels of bc_append (when the call's K/V rows go out in a launch of
 *          their own or are taken by the attention kernel: bc_decode_step, bc_fill_step) and of
 *          bc_compress.  They touch only the cache's metadata and `slots`, read nothing an attention
 *          kernel writes, and end only once the kernel they overtook has ended, so everything enqueued
 *          behind them is ordered after both.  The bookkeeping kernel of bc_compress also stores the
 *          beacon rows of layer 0 when they are few (up to 512 KB): it reads beacon_k / beacon_v, and
 *          writes slots and pages that no kernel still running ahead of it reads.
 *      (2) The attention kernels.  Before they wait for the kernel ahead they read `slots`, their
 *          inputs (q, the extra entry, beacon_q) and, of the cache, only what a kernel that has ENDED
 *          wrote: metadata and pool rows other than the newest entries of a beacon or window segment.
 *          The split-K scratch, the ticket counters and every output are touched after the wait.  An
 *          attention kernel that follows its step's bookkeeping kernel directly (bc_decode_step)
 *          reads that kernel's results only after a release/acquire handshake with it.
 *      (3) Kernels that release their dependents early: the attention kernels (once they have read
 *          the lengths they need) and the row-writing kernel of bc_append / bc_compress (at once).
 *    What this asks of the caller: `slots`, the input tensors of an attention call (q, extra_k,
 *    extra_v, beacon_q) and the beacon_k / beacon_v of bc_compress must not be written by a kernel
 *    that releases its dependents early.  Kernels
 *    launched the ordinary way (any GEMM or element-wise kernel that produces q) never do; of this
 *    library's kernels only an attention kernel's OUTPUT could be in that position, so do not pass
 *    the output buffer of one attention call as the query buffer of the next call on the stream.
 *    K/V rows, outputs and the caller's own kernels keep plain stream order.
 *
 * Store layout (owned by the library inside the caller's `pool` buffer)
 *    pool[layer][page][slot_in_page][K|V][kv_head][head_dim] bf16: one token's entry of one layer
 *    is E = 2*kv_heads*head_dim*2 contiguous bytes and a page is page_size*E contiguous bytes, so
 *    any run of tokens inside a page is one contiguous block.  Inside each head row the 16-byte
 *    chunks are stored XOR-permuted by (position of the entry in its segment) & 7, which makes the
 *    shared-memory image of a bulk copy free of bank conflicts; bc_export_seq undoes it.
 *
 * Page allocation discipline (deterministic, so page ownership is reproducible bit for bit)
 *    Free pages form a LIFO stack; a fresh cache hands out pages 0, 1, 2, ...  Within one call,
 *    allocations come first: batch item i needing need[i] pages takes the pages at stack depth
 *    off[i] .. off[i]+need[i]-1, off = exclusive prefix sum of the needs of all items that passed
 *    validation; it is granted iff need[i] == 0 or off[i]+need[i] <= pages free at the start of
 *    the call.  Frees follow, in batch order; a sequence's pages are pushed prompt pages first,
 *    then beacon pages, then window pages, each in ascending order.
 */
#ifndef BREADCRUMBS_H_
#define BREADCRUMBS_H_

#include <stddef.h>
#include <stdint.h>

#if defined(__GNUC__)
#define BC_API __attribute__((visibility("default")))
#else
#define BC_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

#define BC_ALL_LAYERS (-1)   /* `layer` argument: all layers in one call, tensors with a leading [layers] dimension */

typedef int32_t bc_status;
enum {
  BC_OK = 0,
  BC_ERR_INVALID_ARG = -1,     /* null/misaligned pointer, n <= 0, bad layer, bad config, c < 1 */
  BC_ERR_BAD_SLOT = -2,        /* slot out of range, not open, or already open */
  BC_ERR_NO_PAGES = -3,        /* free stack too small for this item */
  BC_ERR_CAPACITY = -4,        /* max_entries_per_seq or max_pages_per_seq would be exceeded */
  BC_ERR_WINDOW_NOT_FULL = -5, /* bc_compress on a window that does not hold exactly c entries */
  BC_ERR_WINDOW_FULL = -6,     /* bc_append on a full window (c > 1): compress first */
  BC_ERR_ORDER = -7,           /* per-layer calls out of order */
  BC_ERR_CUDA = -8,            /* a CUDA runtime call failed; see bc_last_cuda_error */
  BC_ERR_UNSUPPORTED = -9,     /* shape outside what the kernels are built for */
  BC_ERR_TIMEOUT = -10,        /* a bounded device-side wait gave up (kernel returned early) */
  BC_ERR_TOO_LARGE = -11,      /* bc_decode_attn_static: the call does not fit the built-in scratch */
  BC_ERR_DEBUG_CHECK = -12     /* BC_FLAG_DEBUG_BOUNDS: a checked index was out of range, or a batch named a slot twice */
};

enum {
  BC_FLAG_OUT_F32 = 1u,        /* bc_decode_attn writes fp32 instead of bf16 */
  BC_FLAG_ATTN_REFERENCE = 2u, /* use the slow one-warp-per-head device kernel (debugging aid) */
  BC_FLAG_HOST_PIPELINED = 4u, /* host-buffer steps: outputs are copied back on a stream of the cache's own, see bc_host_outputs_ready */
  BC_FLAG_DEBUG_BOUNDS = 8u    /* Checked mode (stands in for a memory checker).  Every kernel that turns a page id, a
                                  page-table column or a pool row into an address checks it first: a column must lie
                                  inside the page-table row, a page id inside the pool, a row inside the pool.  A failed
                                  check latches BC_ERR_DEBUG_CHECK (the offending value in the record's slot field) and
                                  the access is skipped, or, in the attention kernel, redirected to page 0, so that the
                                  kernel still finishes; nothing traps.  The bookkeeping calls also refuse, with the
                                  same code, every batch item whose slot an item with a lower index of the same call
                                  names (that first item goes through).  Costs a few compares per page, no extra pass. */
};

typedef struct bc_cache bc_cache; /* opaque host-side handle */

typedef struct {
  int32_t layers;
  int32_t kv_heads;            /* 1, 2, 4 or 8 */
  int32_t q_heads;             /* multiple of kv_heads, q_heads/kv_heads <= 16, q_heads*head_dim <= 4096 */
  int32_t head_dim;            /* 64 or 128 */
  int32_t c_default;           /* compression ratio used when bc_seq_open gets no per-sequence c;
                                  1 = never compress (in the paper's tables the ratio-1
                                  column is the uncompressed teacher) */
  int32_t page_size;           /* tokens per page, >= 1; need not divide or equal c */
  int32_t max_seqs;            /* number of sequence slots */
  int32_t num_pages;           /* pages in the pool (each page spans all layers) */
  int32_t max_pages_per_seq;   /* width of one page-table row */
  int32_t max_entries_per_seq; /* cap on beacons + live window entries of a sequence, the cache-size
                                  limit of the paper's evaluation, at which generation is cut off
                                  (Evaluation paragraph); 0 = unlimited */
  uint32_t flags;
} bc_config;

typedef struct {
  int32_t open;                /* 1 if the slot is open */
  int32_t prompt_len, n_beacons, window_len, c;
  int32_t t;                   /* generated-token entries appended so far */
  int32_t n_prompt_pages, n_beacon_pages, n_window_pages;
} bc_seq_state;

/* Library version, major*10000 + minor*100 + patch. */
BC_API int32_t bc_version(void);

/* Sizes of the three caller-provided device buffers for this configuration (host pointers out).
 * pool: the K/V pages; meta: lengths, page tables, free stack, status; workspace: split-K
 * partials and per-call scratch. */
BC_API bc_status bc_cache_query_bytes(const bc_config* cfg, size_t* pool_bytes, size_t* meta_bytes,
                               size_t* workspace_bytes);

/* Creates the host handle over caller-owned device buffers of at least the queried sizes
 * (256-byte aligned) and enqueues, on `stream`, the kernel that resets the bookkeeping.  The pool
 * content is not touched.  The five-argument form bc_cache_create(layers, kv_heads, head_dim, c,
 * page_size) of the problem statement is this call with the remaining fields of bc_config filled
 * in by the caller. */
BC_API bc_status bc_cache_create(const bc_config* cfg, void* pool, void* meta, void* workspace,
                          void* stream, bc_cache** out);

/* Frees the host handle (and the streams and events the host-buffer entry points created, after
 * waiting for the copies still running on them).  pool, meta and workspace stay the caller's; work
 * the caller enqueued on its own streams is not waited for. */
BC_API bc_status bc_cache_destroy(bc_cache* cache);

/* Algorithm 1, initialisation: opens n sequence slots with their prompt lengths and compression
 * ratios and allocates ceil(prompt_len/page_size) prompt pages each.  slots, prompt_lens,
 * c_per_seq (may be NULL -> c_default): device pointers to n int32.  c stays fixed for the life
 * of the sequence (Discussion section: a ratio, once chosen, is not changed mid-generation). */
BC_API bc_status bc_seq_open(bc_cache* cache, const int32_t* slots, const int32_t* prompt_lens,
                      const int32_t* c_per_seq, int32_t n, void* stream);

/* Algorithm 1, prompt encoding: stores the prompt K/V of one layer.  k, v: device
 * [total_tokens, kv_heads, head_dim] bf16, sequences packed back to back; cu_prompt_lens: device
 * int32[n+1] exclusive prefix sums (cu[n] == total_tokens, passed again as a host int). */
BC_API bc_status bc_prefill(bc_cache* cache, int32_t layer, const int32_t* slots,
                     const int32_t* cu_prompt_lens, int32_t n, int32_t total_tokens,
                     const void* k, const void* v, void* stream);

/* Algorithm 1 run over a stored trajectory, in one call per layer: each of n sequences that were
 * opened (and whose prompt is, or will be, stored by bc_prefill) but have received no entry yet gets
 * the state the sampling loop is in after its T_i generated tokens -- its floor(T_i / c) beacons and
 * the T_i mod c tokens of its unfinished window (all T_i tokens when c = 1); the evicted tokens are
 * never copied.  This is what lets a trajectory scored in one pass (Section 3.2, the mask form,
 * whose inputs have the same packing) be continued by the decode loop.
 * cu_tokens: device int32[n + 1], prefix sums of T_i.  tok_k, tok_v: device bf16
 * [total_tokens, kv_heads, head_dim], the generated tokens' entries, sequences back to back;
 * beacon_k, beacon_v: device bf16 [total_beacons, kv_heads, head_dim], sequence i's floor(T_i / c)
 * beacons back to back in batch order (an item whose slot is not open has none).  total_tokens and
 * total_beacons (host) bound what is read.  Per-layer ordering as for bc_append: layer 0 first (it
 * does the bookkeeping: beacon pages, then window pages, per item in batch order), then 1 .. layers - 1
 * with the same `slots` and `cu_tokens`.  Device-side failures (latched): BC_ERR_BAD_SLOT (not open),
 * BC_ERR_INVALID_ARG (the sequence has entries already, or T_i < 0), BC_ERR_CAPACITY, BC_ERR_NO_PAGES;
 * a failed item is left untouched. */
BC_API bc_status bc_restore(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n,
                            const int32_t* cu_tokens, int32_t total_tokens, int32_t total_beacons,
                            const void* tok_k, const void* tok_v, const void* beacon_k,
                            const void* beacon_v, void* stream);

/* Algorithm 1, sampling step (the forward pass of a token adds its entry to the cache): appends one generated
 * token's K/V entry to the live window of each of n sequences.  A window page is allocated when
 * the window length is a multiple of page_size.  k, v: device [n, kv_heads, head_dim]. */
BC_API bc_status bc_append(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n,
                    const void* k, const void* v, void* stream);

/* The attention read of a decode step (Section 2, standard attention; Figure 2 caption for what
 * is visible): out[i,h] = softmax_j(sm_scale * <q[i,h], K_j>) V_j over every live entry of
 * sequence slots[i] in `layer`: prompt, beacons, window.  If extra_k/extra_v are non-NULL
 * ([n, kv_heads, head_dim]) one more entry per sequence is attended without being stored: this is
 * the beacon's own K/V when the beacon query is evaluated (Algorithm 1, the beacon-encoding step).  q: device
 * [n, q_heads, head_dim] bf16; out: same shape, bf16 (fp32 with BC_FLAG_OUT_F32), rounded to
 * nearest even from fp32.  Accumulation is fp32.  A sequence with no entry at all gets zeros.
 * n <= 512 per call. */
BC_API bc_status bc_decode_attn(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n,
                         const void* q, void* out, float sm_scale, const void* extra_k,
                         const void* extra_v, void* stream);

/* The step that fills a window, and the encoding of the beacon that follows it, in one pass over the
 * cache (Algorithm 1: the token's forward pass and the beacon's read the same entries; the beacon
 * also sees itself).  out = what bc_decode_attn(q) returns; out_beacon = what
 * bc_decode_attn(beacon_q, extra = beacon_k, beacon_v) returns, both over the cache as it stands (call
 * it after the token's bc_append and before bc_compress).  The K/V entries are read from HBM once
 * for both: at ratio c this saves the 1/c extra attention traffic of the beacon steps.  For groups
 * of more than 8 query heads per KV head (and with BC_FLAG_ATTN_REFERENCE) the two results come from
 * two passes.  Arguments as for bc_decode_attn; beacon_q, out_beacon like q, out. */
BC_API bc_status bc_decode_attn_pair(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n,
                                     const void* q, void* out, const void* beacon_q, void* out_beacon,
                                     float sm_scale, const void* beacon_k, const void* beacon_v,
                                     void* stream);

/* One decode step of one layer: bc_append(k, v) followed by bc_decode_attn(q) (Algorithm 1: the
 * forward pass of a token adds its entry, then its query reads the cache, the new entry included),
 * without the row-writing launch.  Results, bookkeeping, layer-order rule and error behaviour are
 * exactly those of the two calls made one after the other.
 * How: the append bookkeeping runs as its own one-block kernel (on the layer-0 call; it may begin
 * under the last blocks of the attention kernel enqueued before it, see "Overlap" above); the
 * attention kernel takes the new entries from the input tensors where it needs them, and one of
 * its warps stores them to the pool for later steps.
 * q [n, q_heads, head_dim], k, v [n, kv_heads, head_dim], out like q; n <= 512.  With
 * BC_FLAG_ATTN_REFERENCE the call simply issues the two separate calls.  layer = BC_ALL_LAYERS:
 * see the layer convention at the top of this file. */
BC_API bc_status bc_decode_step(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n, const void* q,
                                const void* k, const void* v, void* out, float sm_scale, void* stream);

/* Rotary position embedding and split of a packed QKV projection: what sits between a decoder
 * layer's QKV GEMM and the cache calls.  (The paper leaves the position encoding to the model,
 * Section 2: attention is unchanged; its models use rotary embeddings.)  Row i of qkv is
 * [q heads | k heads | v heads], (q_heads + 2 kv_heads) * head_dim bf16 values, of a token (or beacon)
 * at position positions[i].  Every q and k head is rotated: coordinate j < head_dim/2 is paired
 * with coordinate j + head_dim/2 (the half-split pairing of the paper's models) and the pair is
 * turned by positions[i] * theta^(-2j/head_dim) radians; v is copied.  Angles are evaluated in double
 * precision, the rotation in fp32, results rounded to nearest-even bf16.
 * qkv: device, [n, (q_heads + 2 kv_heads) * head_dim] bf16, 16-byte aligned; positions: device int32[n],
 * >= 0; theta > 1 (10000 in RoFormer, 1e6 in Qwen2.5); q_out [n, q_heads, head_dim], k_out, v_out
 * [n, kv_heads, head_dim]: device bf16, 16-byte aligned, caller-owned, must not overlap qkv.  They are
 * laid out as bc_append / bc_decode_attn / bc_decode_step / bc_compress take them.  The head counts and
 * head_dim are the cache's; the call touches no cache state, records no error and may be issued at any
 * point of the layer order.  One kernel launch; asynchronous on `stream`; it completes before any
 * later kernel of the stream starts (it takes no part in the overlap described above).
 * BC_ERR_INVALID_ARG: a null or misaligned pointer, n <= 0, theta <= 1. */
BC_API bc_status bc_rope_split(bc_cache* cache, const void* qkv, const int32_t* positions, int32_t n, float theta,
                               void* q_out, void* k_out, void* v_out, void* stream);

/* bc_rope_split followed by bc_decode_step on its results: one decode step of one layer straight from
 * the packed QKV projection (two launches: the rotation, then the attention kernel that also appends
 * the new entries; plus the one-block bookkeeping kernel on layer 0).  The rotated q, k and v pass
 * through a staging buffer the cache owns (one per cache: the next call of this entry point on the same
 * stream reuses it, which stream order makes safe).  Arguments as for the two calls; n <= 512 and
 * n <= max_seqs.  Errors: those of bc_decode_step and bc_rope_split. */
BC_API bc_status bc_rope_decode_step(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n, const void* qkv,
                                     const int32_t* positions, float theta, void* out, float sm_scale, void* stream);

/* The step whose token fills the window, in one call: bc_append(k, v), bc_decode_attn_pair(q, beacon_q;
 * extra = beacon_k, beacon_v) and bc_compress(beacon_k, beacon_v) (Algorithm 1: the token's forward
 * pass, the beacon's forward pass, the eviction).  Results, bookkeeping, layer-order rule (the layer
 * must be the next one of both the append and the compress order) and error behaviour are exactly
 * those of the three calls made one after the other.  How: as in bc_decode_step the append's
 * bookkeeping runs as its own one-block kernel and ONE attention launch takes the token's entry from
 * the inputs, serves the token's and the beacon's query heads in one pass over the cache and stores
 * the entry; then the compression (bookkeeping kernel, beacon rows).  Two launches fewer than the
 * three calls, and the attention kernel overlaps with the step before it like a regular step's.
 * q, beacon_q [n, q_heads, head_dim], k, v, beacon_k, beacon_v [n, kv_heads, head_dim], out,
 * out_beacon like q; all device, 16-byte aligned; n <= 512.  For groups of more than 8 query heads
 * per KV head, and with BC_FLAG_ATTN_REFERENCE, the call issues the three calls. */
BC_API bc_status bc_fill_step(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n, const void* q,
                              const void* k, const void* v, const void* beacon_q, const void* beacon_k,
                              const void* beacon_v, void* out, void* out_beacon, float sm_scale, void* stream);

/* ---- the operators of a decoder layer between its GEMMs and the cache calls --------------------
 * (Experimental Setup: the paper's models are pre-norm decoders with RMSNorm, a SiLU-gated MLP and a
 * residual stream in bf16; Algorithm 1 samples the next token, the latency protocol greedily.)
 * Stateless: no cache handle, nothing is latched; errors are the return value.  All pointers device,
 * 16-byte aligned; one kernel launch each, asynchronous on `stream`, ordinary stream order.
 *
 * bc_add_rmsnorm: h' = h + delta rounded to bf16 (delta NULL: h' = h), stored to h_out (NULL: not
 *   stored; h_out may be h itself), and normed_out = h' / sqrt(mean(h'^2) + eps) * weight (weight
 *   NULL: ones), the mean over the hidden dimension of the stored bf16 values, arithmetic in fp32.
 *   h, delta, h_out, normed_out [n, hidden] bf16, weight [hidden] bf16; hidden a multiple of 8 and
 *   <= 8192 (else BC_ERR_UNSUPPORTED); eps >= 0.
 * bc_swiglu: out[r, j] = silu(gate_up[r, j]) * gate_up[r, m + j], silu(x) = x / (1 + exp(-x));
 *   gate_up [n, 2 m] bf16 (gate in the first half of a row), out [n, m] bf16; m a multiple of 8.
 * bc_argmax: out[r] = the lowest index at which row r of logits [n, vocab] bf16 attains its maximum
 *   (int64, the type token ids usually have); vocab a multiple of 8. */
BC_API bc_status bc_add_rmsnorm(const void* h, const void* delta, const void* weight, int32_t n, int32_t hidden,
                                float eps, void* h_out, void* normed_out, void* stream);
BC_API bc_status bc_swiglu(const void* gate_up, int32_t n, int32_t m, void* out, void* stream);
BC_API bc_status bc_argmax(const void* logits, int32_t n, int32_t vocab, int64_t* out, void* stream);

/* Limits of bc_decode_attn_static. */
#define BC_STATIC_MAX_BATCH 128   /* sequences per call */
#define BC_STATIC_MAX_CTAS 160    /* thread blocks it will use at most */

/* bc_decode_attn for callers that cannot hand the library a workspace carved from freshly
 * allocated device memory.  (The paper has no counterpart to this call; it computes exactly what
 * bc_decode_attn computes.)
 *
 * Who needs it: code that runs where device allocation is off limits -- a memory-budgeted serving
 * process whose allocator is frozen once start-up is over, a plug-in that is only handed tensors
 * and a stream by its host application and must not go to the CUDA allocator behind the host's
 * back, or a latency-critical loop in which an allocation (which may synchronise the device) is not
 * acceptable.  Such callers already own the cache buffers, but the split-K
 * scratch (per-piece partial outputs, their running max and sum, and one ticket counter per
 * sequence) has to live somewhere.  Here it lives in a fixed array inside the library image:
 * about 4.9 MB of device memory that every GPU which loads the library keeps until the process
 * exits.  The call itself performs no device or host allocation and calls no allocating routine.
 *
 * Arguments, layouts, results and error behaviour are those of bc_decode_attn (layer =
 * BC_ALL_LAYERS and BC_FLAG_ATTN_REFERENCE included; the debugging kernel of that flag uses no
 * scratch), with these limits: n <= BC_STATIC_MAX_BATCH, at most BC_STATIC_MAX_CTAS thread blocks
 * (fewer SMs are used on a larger part), q_heads * head_dim <= 4096.  A call beyond them returns
 * BC_ERR_TOO_LARGE and enqueues nothing.  The cache's own `workspace` is not touched.  Two
 * differences: the launches are not bracketed by bc_profile_enable, and the device that is current
 * at the call must be the one the cache was created on (else BC_ERR_INVALID_ARG), because the
 * built-in array exists once per device.
 *
 * The first call on each device looks up the device address of the built-in array (once per
 * device, with that device current); make that first call outside any stream capture.  All calls,
 * from all caches and streams of the process, share the one array: it still holds the previous
 * call's partials when the next call starts (every partial a call reads it has written first,
 * and every call returns the ticket counters to zero, so nothing needs clearing), and two calls
 * whose kernels overlap on the GPU race on it.  Issue them
 * on one stream, or order them with events.
 *
 * Errors.  A launch that gives up with BC_ERR_TIMEOUT (latched in the record of the cache that
 * issued it) may leave counters of the shared array non-zero; until they are cleared, static calls
 * of EVERY cache on that device can merge wrongly, and only the issuing cache's record says so.
 * bc_clear_error of a cache that has used this entry point since its last clear zeroes the shared
 * counters on the given stream: that is a write to the one array, so it has to be ordered (same
 * stream, or events) against every static call of the process like a static call itself.  After
 * such a timeout issue no further static call, from any cache, before that bc_clear_error. */
BC_API bc_status bc_decode_attn_static(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n,
                                       const void* q, void* out, float sm_scale, const void* extra_k,
                                       const void* extra_v, void* stream);

/* Algorithm 1, the eviction statement (keep everything but the c entries before the beacon, then
 * the beacon): for each of n sequences whose window holds exactly c entries, stores the beacon's
 * K/V in the beacon segment (a beacon page is allocated when n_beacons is a multiple of
 * page_size), returns the window's pages to the free stack, sets window_len = 0 and n_beacons += 1.
 * beacon_k, beacon_v: device [n, kv_heads, head_dim]. */
BC_API bc_status bc_compress(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n,
                      const void* beacon_k, const void* beacon_v, void* stream);

/* Algorithm 1, stop token / cache cap: closes n sequences and returns all their pages. */
BC_API bc_status bc_seq_close(bc_cache* cache, const int32_t* slots, int32_t n, void* stream);

/* ---- end-to-end helpers with HOST buffers (pinned memory recommended) ------------------------
 * One decode step of one layer: copies q, k, v to device staging inside `workspace`, runs
 * bc_decode_step (the append and the attention of the step; same ordering rule over the layers),
 * copies out back.  n <= 512.  Asynchronous: out_host is valid, and the
 * three input buffers may be reused, once `stream` has passed the call.  The inputs are copied on a
 * stream the cache owns (created by the first such call) into one of eight staging buffers used in
 * turn, so a call's inputs travel while the previous calls' kernels run: they are read from the
 * moment of the call, not in the order of `stream` -- they must be complete in host memory when the
 * call is made.  If the three buffers are one packed block k | v | q (v_host == k_host + bytes(k),
 * q_host == v_host + bytes(v)) a single copy moves them.  The host-buffer calls use streams of the
 * library's own beside `stream` and must not be made inside a stream capture.
 * On a single-layer cache created with BC_FLAG_HOST_PIPELINED the call puts nothing but its two
 * kernels on `stream` (no event, no wait): the copy stream writes the step's number to a word in
 * `workspace` behind the inputs (a stream memory operation) and the step's bookkeeping kernel polls
 * that word (bounded: if the inputs do not arrive within about a second the step is reported as
 * BC_ERR_TIMEOUT by bc_poll_error and its output is undefined) before it lets the attention kernel
 * read them; the output copies of a step are released by a word the next step's bookkeeping kernel
 * (or bc_host_outputs_ready, or bc_cache_destroy) stores once the step's kernels have ended.
 * Consecutive steps then overlap as device-resident bc_decode_step calls do.  Issue such steps on
 * one stream; a change of stream is handled, at the price of one small kernel on the old stream. */
BC_API bc_status bc_decode_step_host(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n,
                              const void* q_host, const void* k_host, const void* v_host,
                              void* out_host, float sm_scale, void* stream);
/* With BC_FLAG_HOST_PIPELINED the host-buffer steps copy their outputs back on a stream the cache owns
 * (from eight staging sets used in turn), so the next step's kernels do not wait behind the copy.  The
 * price: `stream` alone no longer orders the outputs, and the copies of a step's outputs are enqueued
 * by the NEXT host-buffer call (directly behind that call's bookkeeping kernel), by
 * bc_host_outputs_ready or by bc_cache_destroy.  out_host of every step issued so far is complete
 * once bc_host_outputs_ready(cache, stream) has been called and `stream` has passed it; without the
 * flag the call does nothing.  No wait the library enqueues depends on a call still to be made, so
 * the caller may synchronise the device at any point.  At most eight steps' outputs are in flight:
 * the staging set of a step is reused eight host-buffer calls later. */
BC_API bc_status bc_host_outputs_ready(bc_cache* cache, void* stream);

/* The step that fills a window, with host buffers: bc_fill_step (bc_append of the token,
 * bc_decode_attn_pair for the token and its beacon in one pass over the cache, bc_compress).
 * Equivalent to bc_decode_step_host followed by bc_compress_step_host; same conventions, the
 * ordering by words on single-layer caches with BC_FLAG_HOST_PIPELINED included. */
BC_API bc_status bc_fill_step_host(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n,
                                   const void* q_host, const void* k_host, const void* v_host,
                                   const void* beacon_q_host, const void* beacon_k_host,
                                   const void* beacon_v_host, void* out_host, void* out_beacon_host,
                                   float sm_scale, void* stream);
/* The beacon step with host buffers: beacon-query attention (beacon K/V as the extra entry), then
 * bc_compress. */
BC_API bc_status bc_compress_step_host(bc_cache* cache, int32_t layer, const int32_t* slots, int32_t n,
                                const void* beacon_q_host, const void* beacon_k_host,
                                const void* beacon_v_host, void* out_host, float sm_scale,
                                void* stream);

/* ---- the mask form: a whole trajectory in one pass (Section 3.2, Figure 2) ---------------------
 * Training simulates the eviction with an attention mask over the teacher-forced trajectory
 * [prompt, x_0 .. x_{c-1}, b_1, x_c, ...]: a generated token attends to the prompt, to every
 * earlier beacon and to the tokens of its own window up to itself; beacon b_m, placed after the
 * m-th window of c tokens, attends to the prompt, the beacons b_1 .. b_m (itself included) and
 * that window.  The paper states that this computes what the inference loop computes (Section
 * 3.2); here it is one dense pass on the tensor cores, independent of any bc_cache.
 *
 * Sequences are packed back to back.  cu_prompt, cu_tokens: HOST int32[n_seqs + 1] prefix sums of
 * the prompt and generated-token counts.  Sequence i has floor(T_i / c) beacons (none when c = 1),
 * packed in the same order.  Device tensors, bf16: prompt_k, prompt_v [sum P, kv_heads, head_dim];
 * tok_q [sum T, q_heads, head_dim]; tok_k, tok_v [sum T, kv_heads, head_dim]; beacon_q
 * [sum nb, q_heads, head_dim]; beacon_k, beacon_v [sum nb, kv_heads, head_dim]; outputs out_tok
 * [sum T, q_heads, head_dim] and out_beacon [sum nb, q_heads, head_dim] (32-byte aligned), bf16 rounded to nearest
 * even from fp32 (accumulation in fp32, softmax weights rounded to bf16 before the second product).
 * head_dim must be 128 and q_heads / kv_heads <= 16 (else BC_ERR_UNSUPPORTED); sm_scale > 0.  `workspace`: device
 * memory of at least bc_mask_attn_query_bytes bytes, 256-byte aligned (it receives the list of
 * query tiles and the status word).  A sequence's rows depend on that sequence's inputs only: rows of K
 * and V that a tile reads beyond the sequence's own are masked (K) and cleared (V) before they can enter a
 * product, so non-finite values in a neighbouring sequence do not spread.  Asynchronous on `stream`; the two host arrays are read before the
 * call returns (pageable host memory is staged by the copy, so do not call this inside a stream
 * capture).  One call at a time per workspace.  A bounded device-side wait that expires is reported
 * by bc_mask_attn_status as BC_ERR_TIMEOUT (the outputs are then incomplete). */
BC_API bc_status bc_mask_attn_query_bytes(int32_t n_seqs, int32_t q_heads, int32_t kv_heads, int32_t head_dim,
                                          int64_t total_prompt, int64_t total_tokens, int64_t total_beacons,
                                          size_t* workspace_bytes);
BC_API bc_status bc_mask_attn_forward(int32_t n_seqs, int32_t q_heads, int32_t kv_heads, int32_t head_dim, int32_t c,
                                      const int32_t* cu_prompt, const int32_t* cu_tokens, const void* prompt_k,
                                      const void* prompt_v, const void* tok_q, const void* tok_k, const void* tok_v,
                                      const void* beacon_q, const void* beacon_k, const void* beacon_v,
                                      void* out_tok, void* out_beacon, float sm_scale, void* workspace,
                                      size_t workspace_bytes, void* stream);
/* Poll limit of the bounded waits of bc_mask_attn_forward (process-wide; 0 = the default).  A block
 * whose wait runs out waits, with the full default limit, for the tensor copies and products it has in
 * flight, releases its tensor memory and returns; bc_mask_attn_status then reports BC_ERR_TIMEOUT. */
BC_API bc_status bc_mask_attn_set_wait_limit(uint32_t polls);

/* Synchronises `stream` and returns in *code the status the last bc_mask_attn_forward on this
 * workspace left on the device (BC_OK or BC_ERR_TIMEOUT).  The totals are those of that call. */
BC_API bc_status bc_mask_attn_status(const void* workspace, int32_t n_seqs, int32_t q_heads, int32_t kv_heads,
                                     int64_t total_prompt, int64_t total_tokens, int64_t total_beacons,
                                     void* stream, int32_t* code);

/* ---- the distillation loss (Section 3.2, Eq. 1) -------------------------------------------------
 * loss = (1 / n_traj) * sum_b (1 / |x_b|) * sum_{positions r of trajectory b} KL_K(teacher_r || student_r),
 * the mean over the batch of the per-trajectory mean token-level divergence between the frozen
 * uncompressed teacher and the compressed student.  The teacher is given the way the paper stores
 * it (Implementation Details: the top 100 entries per time step, more than 90 % of the mass): for
 * every position top_k vocabulary indices (distinct, in [0, vocab)) and the teacher's
 * log-probabilities of those entries under its full-vocabulary normalisation; -inf marks an unused
 * entry.  KL_K(p || q) = sum over the stored entries of p_k (log p_k - log q_k), q = softmax of the
 * student's logits over the whole vocabulary; with top_k = vocab this is Eq. 1 exactly (the paper
 * does not say how the stored entries are normalised; this is the reading taken).
 *
 * Device pointers: cu_rows int32[n_traj + 1] prefix sums of the trajectories' positions
 * (cu_rows[n_traj] == rows); student_logits bf16 [rows, vocab]; teacher_idx int32 [rows, top_k];
 * teacher_logprob fp32 [rows, top_k]; row_loss fp32 [rows] (KL_K of every position, written);
 * loss fp32 [1] (written).  grad: NULL, or bf16 [rows, vocab] receiving d loss / d student_logits =
 * w_r (q_j sum_k p_k - p_j [j stored]), w_r = 1 / (n_traj |x_b|); it must have the same 16-byte
 * phase as student_logits.  fp32 arithmetic; additions in a fixed order (results are reproducible).
 * Asynchronous on `stream`; nothing is allocated. */
BC_API bc_status bc_distill_loss(int32_t n_traj, const int32_t* cu_rows, int64_t rows, int32_t vocab, int32_t top_k,
                                 const void* student_logits, const int32_t* teacher_idx,
                                 const float* teacher_logprob, float* row_loss, float* loss, void* grad, void* stream);

/* ---- inspection (these synchronise `stream`; for tests and tools) ---------------------------- */

/* Bookkeeping of one slot.  pages (host, may be NULL) receives up to pages_cap page ids: prompt
 * pages, then beacon pages, then window pages. */
BC_API bc_status bc_get_state(bc_cache* cache, int32_t slot, bc_seq_state* out, int32_t* pages,
                       int32_t pages_cap, void* stream);

/* The free stack, bottom first (the last element is handed out next).  pages: host array of at
 * least num_pages int32. */
BC_API bc_status bc_get_free_list(bc_cache* cache, int32_t* pages, int32_t* count, void* stream);

/* First latched device-side error, or BC_OK: its code, slot and the 1-based index of the
 * bookkeeping call (open/append/compress/close, counted per cache) that raised it. */
BC_API bc_status bc_poll_error(bc_cache* cache, int32_t* code, int32_t* slot, int64_t* call_index,
                        void* stream);

/* Clears the latched error record and zeroes the split-K ticket counters in the cache's workspace
 * (a launch that gave up with BC_ERR_TIMEOUT may have left them non-zero).  If this cache has
 * called bc_decode_attn_static since its last clear, the counters of the array built into the
 * library are zeroed as well: see the ordering rule stated there. */
BC_API bc_status bc_clear_error(bc_cache* cache, void* stream);

/* Gathers the live entries of one sequence in logical order (prompt, beacons, window), with the
 * storage permutation undone: k_out, v_out device [capacity, kv_heads, head_dim] bf16; writes
 * min(entries, capacity) rows.  Asynchronous. */
BC_API bc_status bc_export_seq(bc_cache* cache, int32_t layer, int32_t slot, void* k_out, void* v_out,
                        int32_t capacity, void* stream);

/* ---- tuning and measurement ------------------------------------------------------------------ */

/* Number of thread blocks of the decode-attention kernel (0 = one per SM).  The flat tile
 * partition adapts, so this also forces a given number of key splits per sequence in tests. */
BC_API bc_status bc_set_attn_ctas(bc_cache* cache, int32_t ctas);

/* While enabled, every bc_decode_attn brackets its attention kernel with CUDA events on `stream`
 * (up to max_launches per enable).  bc_profile_read synchronises and returns the number of
 * bracketed launches and the sum of their durations in milliseconds. */
BC_API bc_status bc_profile_enable(bc_cache* cache, int32_t max_launches);
BC_API bc_status bc_profile_read(bc_cache* cache, int32_t* launches, float* total_ms);

/* Poll limit of the bounded waits inside the kernels of bc_decode_attn and bc_decode_step this handle
 * launches (0 = the default, about a quarter of a second; the paired form keeps the default).  The
 * settable limit lives in kernel variants of its own, built for head_dim 128 with at most 8 query
 * heads per KV head: other shapes return BC_ERR_UNSUPPORTED.  A wait that runs out makes its thread block stop issuing
 * copies, wait (with the full default limit) for the copies it has in flight, record BC_ERR_TIMEOUT
 * in the status record and return; the call's outputs are then undefined and split-K ticket counters may
 * be left non-zero until bc_clear_error.  A limit of 1 makes practically every launch give up at
 * once: that is how the expiry path is exercised without hanging or faulting anything. */
BC_API bc_status bc_set_wait_limit(bc_cache* cache, uint32_t polls);

/* Where a decode-attention launch spends its time.  While a buffer is set, thread 0 of every thread
 * block of every attention kernel this handle launches (bc_decode_attn, _pair, bc_decode_step; not
 * the static entry point) stores nanosecond stamps of the GPU's global timer, so that the figures a
 * design discussion rests on can be regenerated: device_words is device memory of at least
 * blocks * BC_TIMELINE_WORDS uint64 (blocks >= 304, the largest grid), block b writing words
 * [b * BC_TIMELINE_WORDS ..): 0 block entered the kernel, 1 its plan is built, 2 it has waited for the
 * kernel ahead on the stream, 3 its first tile has landed in shared memory, 4 the last tile of its
 * final piece is consumed, 5 that piece is written / merged / published, 6 the ticket of its first
 * piece is known, 7 it leaves (after the merges it owed); word 8 = tiles << 32 | first sequence;
 * word 9 = how it ended: bit 0 its final piece was a whole sequence, bit 1 it merged that piece's
 * sequence at once, bit 2 it published the piece, bits 3 / 4 it merged the sequence of its first /
 * final piece after taking that sequence's last ticket.
 * A block without tiles writes only 0 and 1.  Each launch overwrites the last one's stamps; zero
 * the buffer before the launch of interest and read it after synchronising.  NULL switches it off
 * (the default; the kernel then executes a few predicated-off stores per block and nothing else). */
#define BC_TIMELINE_WORDS 16
BC_API bc_status bc_attn_timeline(bc_cache* cache, void* device_words, int32_t blocks);

/* A measurement aid, no part of the method: reads `bytes` (rounded down to a multiple of 64 KB) of
 * device memory once, with the decode-attention kernel's own access pattern (one thread block per SM,
 * 64 KB bulk copies into a three-stage shared-memory ring, two in flight, evict-first) and no
 * arithmetic.  Timed by the caller with events, bytes / time is the read bandwidth that pattern can
 * reach on the device at hand: the ceiling for the attention kernel's streaming phase, and a
 * denominator that, unlike a copy benchmark's, keeps roofline fractions below 1.  Asynchronous on
 * `stream`; device_buf 16-byte aligned, bytes >= 64 KB. */
BC_API bc_status bc_probe_read_stream(const void* device_buf, size_t bytes, void* stream);

/* Kernels launched by this handle since creation (for launch accounting). */
BC_API int64_t bc_kernel_launches(const bc_cache* cache);

/* Last CUDA runtime error code seen by this handle (0 if none) and its text. */
BC_API int32_t bc_last_cuda_error(const bc_cache* cache);
BC_API const char* bc_status_string(bc_status s);

#ifdef __cplusplus
}
#endif
#endif /* BREADCRUMBS_H_ */
