// Decode attention over the paged, segmented (prompt | beacons | window) bf16 store.
//
// k_attn_pipe is the product kernel: a persistent, warp-specialised split-K flash-decoding kernel.
//   * One producer warp streams K/V rows from HBM into a ring of shared-memory stages with 1-D bulk
//     asynchronous copies (one per contiguous run of tokens inside a page) that complete on an
//     mbarrier; eight consumer warps run QK^T and PV on the tensor cores (mma.sync m16n8k16, bf16
//     in, fp32 accumulate) with an fp32 online softmax.  The G query heads that share a KV head are
//     packed on the M dimension of the MMA, so each K/V byte is read from HBM once.
//   * A sequence's live entries are laid out in a virtual row space: prompt rows from 0, beacon
//     rows from the next multiple of 8, window rows from the next multiple of 8 after the beacons.
//     Aligning segment starts to 8 keeps (row & 7) equal to the entry's position in its segment,
//     which is the XOR key of the store's chunk permutation, so ldmatrix reads are conflict free.
//   * Work is cut into tiles of T = 16 * (8 / kv_heads) virtual rows; the tiles of all sequences of
//     the batch, in order, are divided evenly over the grid (each block gets a contiguous span), so
//     ragged batches balance to within one tile.  A block's share of one sequence is a "piece"; a
//     piece that covers the whole sequence writes the final output, otherwise it writes an
//     unnormalised partial (m, l, O) and takes a ticket from the sequence's counter; the block
//     that takes the last ticket merges all pieces of the sequence (always in piece order, so the
//     result does not depend on which block came last) and resets the counter.  Nobody waits.
//   * The producer never stalls on the page table: page ids are fetched a few tiles ahead with
//     4-byte asynchronous copies into a small shared-memory ring.
//   * Every wait is bounded: on expiry the block records BC_ERR_TIMEOUT, stops issuing copies,
//     drains the copies already in flight (bounded) and returns.
//
// k_attn_reference is a slow, straightforward kernel (one warp per query head) kept as a
// debugging aid behind BC_FLAG_ATTN_REFERENCE.
#include "bc_common.cuh"

namespace {

#include "bc_book_device.cuh"

constexpr int kConsumerWarps = 8;
constexpr int kPipeThreads = (kConsumerWarps + 2) * 32;  // consumer warps, producer warp, service warp
constexpr int kPlanMax = BC_MAX_ATTN_BATCH;
constexpr uint32_t kSpinLimit = 1u << 21;  // polls of try_wait before giving up
constexpr int kPidAhead = 4;               // tiles of page-id lookahead of the producer
constexpr int kInFlight = 2;               // stages whose copies may be outstanding at once: HBM
                                           // delivers less when every SM keeps more in flight
constexpr int kNewRowBit = 1 << 30;        // in the plan's slot word: the sequence got a new entry in this launch
constexpr int kTimelineSlots = BC_TIMELINE_SLOTS;
static_assert(kNewRowBit == BC_PLAN_NEW_ROW, "the bookkeeping kernel's plan uses the same bit");
constexpr int kPidSlot = 136;              // ints per descriptor slot: 4 header + up to 132 page ids

// ---------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// 1-D bulk asynchronous copy global -> this block's shared memory, completing on an mbarrier.
// `policy` is an L2 cache policy: the K/V stream is read once per launch and is larger than L2,
// so it is marked evict-first and leaves the lengths, page tables, queries and partial results
// of the previous launches resident.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(dst),
      "l"(src), "r"(bytes), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
// 4-byte asynchronous copy global -> shared (page-id prefetch), grouped by commit / wait_group.
__device__ __forceinline__ void cp_async4(uint32_t dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// Waits until at most `pending` (clamped to kPidAhead) of the most recent groups are outstanding.
__device__ __forceinline__ void cp_async_wait_dyn(int pending) {
  switch (pending) {
    case 0: cp_async_wait<0>(); break;
    case 1: cp_async_wait<1>(); break;
    case 2: cp_async_wait<2>(); break;
    case 3: cp_async_wait<3>(); break;
    default: cp_async_wait<kPidAhead>(); break;
  }
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void consumer_bar() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
// D(16x8,f32) += A(16x16,bf16,row) * B(16x8,bf16,col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
// Takes a ticket: release for the piece this block has just stored (the stores of the other threads are
// ordered before it by the block barrier ahead of the call), acquire for the pieces the earlier ticket
// holders stored (the threads that read them come after a block barrier behind the call).
__device__ __forceinline__ int ticket_acq_rel(int* counter) {
  int old;
  asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(counter) : "memory");
  return old;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

// Bounded wait; returns false when it gave up or another warp already aborted.
__device__ __forceinline__ uint32_t mbar_test_wait(uint32_t bar, uint32_t parity) {   // never suspends the thread
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
constexpr uint32_t kShortLimit = 1024;   // limits below this poll without suspending (try_wait may sleep for a while inside)

// Bounded wait; returns false when it gave up or another warp already aborted.  The ordinary
// instantiation has a compile-time limit: with the limit as a run-time value the polling loop compiles
// into something measurably slower (3 us per launch on 64-row tiles), so the settable limit of
// bc_set_wait_limit lives in instantiations of its own (SHORTW), which the host picks only when a
// limit has been set.  Limits below kShortLimit poll with test_wait, which never suspends the thread.
template <bool SHORTW>
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, uint32_t limit) {
  if (SHORTW && limit < kShortLimit) {
    for (uint32_t polls = 0; polls <= limit; ++polls)
      if (mbar_test_wait(bar, parity)) return true;
    *abort_flag = 1;
    return false;
  }
  const uint32_t lim = SHORTW ? limit : kSpinLimit;
  uint32_t polls = 0;
  while (!mbar_try_wait(bar, parity)) {
    if (++polls > 1024) __nanosleep(64);
    if (polls > lim || *abort_flag) {
      *abort_flag = 1;
      return false;
    }
  }
  return true;
}

// ---------------------------------------------------------------- shared-memory plan
// Exact unsigned division by a runtime constant (round-up method of Granlund and Montgomery):
// q = (t + ((n - t) >> sh1)) >> sh2 with t = umulhi(mul, n), for every 32-bit n.
struct FastDiv {
  uint32_t mul, sh1, sh2;
};
__device__ __forceinline__ int fast_div(int n, const FastDiv& d) {
  const uint32_t t = __umulhi(d.mul, (uint32_t)n);
  return (int)((t + (((uint32_t)n - t) >> d.sh1)) >> d.sh2);
}

// The fused decode step (append + attention in one launch): the new token's K/V rows, where the
// bookkeeping puts them, and the hand-shake by which block 0 tells the others that it is done.
struct FusedArgs {
  const uint8_t* new_k;   // [n][kv_heads][head_dim] bf16
  const uint8_t* new_v;
  int32_t* dst_row;       // [n] pool row of every item's new entry (-1: the item was refused)
  int32_t* dst_pos;       // [n] its position in the window
  uint8_t* pool_w;        // the layer's pool, writable
  const int32_t* plan;    // the plan the bookkeeping kernel of the step left (bc_decode_step), or NULL
  int32_t* flag;          // set to `epoch` by block 0 once the bookkeeping of this launch is done
  int32_t epoch;
  int64_t call;           // index of the bookkeeping call (for the error latch)
};

struct PipeParams {
  BcMeta m;
  BcGeom g;
  BcAttnArgs a;
  FusedArgs f;
  float scale_log2;
  int rows_per_tile;  // T = 16 * n_groups, a power of two
  int tile_shift;     // log2(T)
  int n_groups;       // 8 / kv_heads
  int G;              // q_heads / kv_heads
  FastDiv div_ps;     // division by page_size
  uint32_t spin_limit;            // polls after which a wait of a consumer, producer or service warp gives up
                                  // (kSpinLimit unless bc_set_wait_limit lowered it); the final drain of copies
                                  // in flight always uses kSpinLimit
  int debug;                      // BC_FLAG_DEBUG_BOUNDS: every page-table column, page id and pool row is checked
  unsigned long long* timeline;   // NULL, or [gridDim.x][kTimelineSlots] device words: %globaltimer stamps of one thread per block
  // layer == BC_ALL_LAYERS in one launch: blockIdx.y is the layer, and the block moves every per-layer pointer
  // by these strides (bytes; tickets: counters).  The metadata, slots, plan and row destinations are shared.
  long long ls_pool, ls_q, ls_out, ls_kv, ls_part_o, ls_part_ml;
  int ls_tickets;
  int early_meta;     // 1: the cache's metadata was last written by a kernel that has ENDED, so the plan and the
                      // first page-table reads may run before the wait for the kernel ahead; 0: wait first
};

template <int D>
struct PipeSmem {
  static constexpr int kStageBytes = 512 * D;  // T * E, independent of kv_heads
  static constexpr int kStages = D == 128 ? 3 : 6;
  static constexpr int kRingBytes = kStageBytes * kStages;
  static constexpr int kMergeOff = kRingBytes;
  static constexpr int kMergeMlOff = kMergeOff + BC_MERGE_ELEMS * 4;
  static constexpr int kPlanOff = kMergeMlOff + 64 * 2 * 4;  // up to 64 query heads
  // plan arrays: P, nb, w, slot, beacon column, window column [kPlanMax] and cum [kPlanMax + 1]
  static constexpr int kPidOff = kPlanOff + (6 * kPlanMax + kPlanMax + 8) * 4;
  // descriptors of the tiles ahead: (kPidAhead + 1) slots of {rows, first position, first page,
  // unused} followed by the page ids of the tile
  static constexpr int kBarOff = kPidOff + (kPidAhead + 1) * kPidSlot * 4;
  // barriers: full[kStages], empty[kStages], piece published, ticket taken
  static constexpr int kMiscOff = kBarOff + 2 * kStages * 8 + 16;  // abort flag, pending tickets
  static constexpr int kTotal = kMiscOff + 32;
};

// Merges the pieces of sequence i (published by blocks first..last) into the final output.  The
// pieces are folded in block order with a running maximum, so the result does not depend on which
// block does the merging.  Piece `own` is taken from the caller's shared-memory copy (own_o,
// own_ml) instead of global memory; pass own = -1 to read every piece from global memory.  Called
// by the 256 consumer threads; each owns up to four float4 of the [q_heads, head_dim] output.
// The loads of all four vectors of up to three pieces are issued together, so a merge of three
// pieces costs about one trip to L2.
__device__ __forceinline__ void combine_pieces(const float* part_o, const float* part_ml, void* out, int out_f32, int Hq,
                                            int D, int i, int first, int last, int own, const float* own_o,
                                            const float* own_ml, int tid) {
  constexpr int kThreads = kConsumerWarps * 32;
  constexpr int KV = BC_MERGE_ELEMS / 4 / kThreads;  // float4 per thread
  constexpr int PB = 3;                              // pieces per batch
  const int nvec = Hq * D / 4;
  const int64_t obase = (int64_t)i * Hq * D;
  float4 acc[KV];
  float mrun[KV], den[KV];
#pragma unroll
  for (int k = 0; k < KV; ++k) { acc[k] = make_float4(0.f, 0.f, 0.f, 0.f); mrun[k] = -INFINITY; den[k] = 0.f; }
#pragma unroll 1
  for (int c0 = first; c0 <= last; c0 += PB) {
    float mc[KV][PB], lc[KV][PB];
    float4 oc[KV][PB];
#pragma unroll
    for (int j = 0; j < PB; ++j) {
      const int c = c0 + j;
      const int64_t ps = (int64_t)(c + i);
#pragma unroll
      for (int k = 0; k < KV; ++k) {
        const int e = tid + k * kThreads;
        const int h = (e * 4) / D;
        mc[k][j] = -INFINITY; lc[k][j] = 0.f; oc[k][j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (c <= last && e < nvec) {
          if (c == own) {
            mc[k][j] = own_ml[h * 2]; lc[k][j] = own_ml[h * 2 + 1];
            oc[k][j] = reinterpret_cast<const float4*>(own_o)[e];
          } else {
            mc[k][j] = __ldcg(part_ml + (ps * Hq + h) * 2);
            lc[k][j] = __ldcg(part_ml + (ps * Hq + h) * 2 + 1);
            oc[k][j] = __ldcg(reinterpret_cast<const float4*>(part_o + ps * Hq * D) + e);
          }
        }
      }
    }
#pragma unroll
    for (int j = 0; j < PB; ++j)
#pragma unroll
      for (int k = 0; k < KV; ++k) {
        const float mn = fmaxf(mrun[k], mc[k][j]);
        const float msafe = mn == -INFINITY ? 0.f : mn;
        const float sa = exp2f(mrun[k] - msafe), sb = exp2f(mc[k][j] - msafe);
        acc[k].x = acc[k].x * sa + oc[k][j].x * sb; acc[k].y = acc[k].y * sa + oc[k][j].y * sb;
        acc[k].z = acc[k].z * sa + oc[k][j].z * sb; acc[k].w = acc[k].w * sa + oc[k][j].w * sb;
        den[k] = den[k] * sa + lc[k][j] * sb;
        mrun[k] = mn;
      }
  }
#pragma unroll
  for (int k = 0; k < KV; ++k) {
    const int e = tid + k * kThreads;
    if (e < nvec) {
      const float inv = den[k] > 0.f ? 1.f / den[k] : 0.f;
      const float4 r = make_float4(acc[k].x * inv, acc[k].y * inv, acc[k].z * inv, acc[k].w * inv);
      if (out_f32) reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + obase)[e] = r;
      else {
        uint2 pk; pk.x = pack_bf16(r.x, r.y); pk.y = pack_bf16(r.z, r.w);
        reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + obase)[e] = pk;
      }
    }
  }
}

// FUSED: the launch also appends the step's new entries (bc_decode_step).  The step's bookkeeping kernel,
// enqueued just ahead, leaves the plan and publishes a flag; the blocks of this kernel poll it.  The new
// rows are not read back from the pool: the bulk copy of a sequence's last tile leaves the new row
// out, the consumer warps write it into the shared-memory tile straight from the input, and the
// service warp stores it to the pool for the steps to come.  So the step costs no second and third
// launch and no fence.
// PAIR: every sequence has two sets of query heads, the token's (rows 0..G-1 of a warp's 16-row
// fragment) and its beacon's (rows 8..8+G-1), which share one pass over the cache: the step whose token
// fills the window and the encoding of the beacon that follows it (Algorithm 1) read the same entries.
// The beacon's rows also see the extra entry (the beacon's own K/V).  Needs G <= 8; with 2 G <= 8 both
// sets of heads share the first 8 rows (token rows 0..G-1, beacon rows G..2G-1: the instantiation with
// G_LE_8 = true), else it runs on the 16-row path; results go to out (token) and out2 (beacon).  FUSED and PAIR
// together are the step that fills a window as one launch: the token's entry comes from the inputs as in
// a regular fused step, and both sets of rows see it.
// LAYERED: one launch for all layers of a call with layer = BC_ALL_LAYERS.  The grid is (blocks, layers):
// the blocks of layer l + 1 are dispatched as those of layer l retire, so the layers follow one another
// without a kernel boundary; each layer has its own ticket counters and partial buffers, because the last
// blocks of one layer and the first of the next run side by side.
template <int D, bool G_LE_8, bool FUSED, bool PAIR = false, bool SHORTW = false, bool LAYERED = false>
__global__ void __launch_bounds__(kPipeThreads, 1) k_attn_pipe(const PipeParams p_in) {
  // PAIR with G_LE_8: the packed paired form, for 2 G <= 8: the token's heads in rows 0..G-1 and the
  // beacon's in rows G..2G-1 of the same 8-row half, so that a tile costs what it costs the plain kernel
  // (one softmax per 16 keys instead of two).  PAIR without G_LE_8: token rows 0..G-1, beacon rows 8..8+G-1.
  constexpr bool PACK = PAIR && G_LE_8;
  static_assert(!LAYERED || (!PAIR && !SHORTW), "the all-layers launch exists for the plain and the fused step");
  PipeParams p_layer;
  if constexpr (LAYERED) {
    p_layer = p_in;
    const long long l = blockIdx.y;
    p_layer.a.pool_layer = p_in.a.pool_layer + l * p_in.ls_pool;
    p_layer.a.q = static_cast<const uint8_t*>(p_in.a.q) + l * p_in.ls_q;
    p_layer.a.out = static_cast<uint8_t*>(p_in.a.out) + l * p_in.ls_out;
    if (p_in.a.extra_k != nullptr) {
      p_layer.a.extra_k = static_cast<const uint8_t*>(p_in.a.extra_k) + l * p_in.ls_kv;
      p_layer.a.extra_v = static_cast<const uint8_t*>(p_in.a.extra_v) + l * p_in.ls_kv;
    }
    p_layer.a.part_o = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(p_in.a.part_o) + l * p_in.ls_part_o);
    p_layer.a.part_ml = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(p_in.a.part_ml) + l * p_in.ls_part_ml);
    p_layer.a.tickets = p_in.a.tickets + l * p_in.ls_tickets;
    if (FUSED) {
      p_layer.f.new_k = p_in.f.new_k + l * p_in.ls_kv;
      p_layer.f.new_v = p_in.f.new_v + l * p_in.ls_kv;
      p_layer.f.pool_w = p_in.f.pool_w + l * p_in.ls_pool;
    }
  }
  const PipeParams& p = LAYERED ? p_layer : p_in;
  using L = PipeSmem<D>;
  constexpr int NSTAGE = L::kStages;
  constexpr int KSTEPS = D / 16;  // k-steps of QK^T
  constexpr int NT = D / 8;       // n-tiles of PV
  constexpr int RING = kPidAhead + 1;
  extern __shared__ __align__(1024) uint8_t smem[];

  float* merge_o = reinterpret_cast<float*>(smem + L::kMergeOff);
  float* merge_ml = reinterpret_cast<float*>(smem + L::kMergeMlOff);
  int* s_P = reinterpret_cast<int*>(smem + L::kPlanOff);
  int* s_nb = s_P + kPlanMax;
  int* s_w = s_nb + kPlanMax;
  int* s_slot = s_w + kPlanMax;
  int* s_bcol = s_slot + kPlanMax;  // first beacon column of the page-table row
  int* s_wcol = s_bcol + kPlanMax;  // first window column
  int* s_cum = s_wcol + kPlanMax;   // [n + 1] exclusive prefix sums of tiles
  int* s_desc = reinterpret_cast<int*>(smem + L::kPidOff);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::kMiscOff);
  volatile int* s_pend = s_abort + 1;  // {sequence, ticket} of the first and of the final piece; [4]: peeked count
  const uint32_t ring = smem_u32(smem);
  const uint32_t desc_ring = smem_u32(smem + L::kPidOff);
  const uint32_t bar_full = smem_u32(smem + L::kBarOff);
  const uint32_t bar_empty = bar_full + NSTAGE * 8;
  const uint32_t bar_pub = bar_empty + NSTAGE * 8;  // the consumers have stored the block's first piece
  const uint32_t bar_tk = bar_pub + 8;              // the service warp has taken that piece's ticket

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = p.a.n, T = p.rows_per_tile, TS = p.tile_shift, E = p.g.entry_bytes, ps = p.g.page_size;
  const int Hkv = p.g.kv_heads, Hq = p.g.q_heads, G = p.G;

  // Timeline (bc_attn_timeline): thread 0 of every block stamps a few points of its life with the global
  // nanosecond timer; a handful of predicated stores per block, none per tile.
  auto stamp = [&](int k) {
    if (p.timeline != nullptr && tid == 0) p.timeline[(size_t)blockIdx.x * kTimelineSlots + k] = global_timer_ns();
  };
  auto stamp_val = [&](int k, unsigned long long v) {
    if (p.timeline != nullptr && tid == 0) p.timeline[(size_t)blockIdx.x * kTimelineSlots + k] = v;
  };
  stamp(0);
  if (tid == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      mbar_init(bar_full + s * 8, 1);
      mbar_init(bar_empty + s * 8, kConsumerWarps);
    }
    mbar_init(bar_pub, kConsumerWarps);
    mbar_init(bar_tk, 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }

  // Launched with programmatic stream serialisation, this kernel may have begun before the kernel ahead
  // of it on the stream has ended.  What it may read before it waits for that kernel is only what a kernel
  // that has ended wrote.  The host says whether that holds for the cache's metadata (early_meta): it does
  // when an ordinarily launched kernel (the row writes of the step) or another attention launch lies
  // between the last bookkeeping kernel and this one; it does not when this launch follows a bookkeeping
  // kernel directly (the fused step, small batches whose rows the bookkeeping block writes itself, a
  // call right after open / close / restore): then the wait comes first and nothing is read early.
  bool early = !FUSED && p.early_meta;
  if (FUSED && p.f.plan != nullptr) {
    // bc_decode_step: the kernel ahead is this step's bookkeeping kernel.  It is running (it is what let this
    // kernel begin) and stores the step's epoch to a flag word, with release semantics, as soon as its
    // results -- lengths, page-table column, row destinations, the plan -- are written; then it only waits
    // for the kernel ahead of IT, the previous step's attention kernel, to end.  Reading the flag with
    // acquire semantics makes those results visible here, so this kernel, too, can plan and stream settled
    // tiles while the previous step's last blocks finish.  If the flag does not show up in a while the
    // block simply waits for the kernel ahead to end, which makes everything visible the ordinary way.
    volatile int* sh_flag_seen = s_abort + 6;   // a word of the block's own scratch: no static shared memory in this kernel
    if (tid == 0) {
      int seen = 0;
      for (uint32_t polls = 0; polls < 2048; ++polls) {
        if (ld_acquire(p.f.flag) == p.f.epoch) { seen = 1; break; }
        __nanosleep(40);
      }
      *sh_flag_seen = seen;
    }
    __syncthreads();
    early = *sh_flag_seen != 0;
  }
  if (!early) asm volatile("griddepcontrol.wait;" ::: "memory");

  // ---- plan: tiles per sequence, prefix sums, this block's span --------------------------------
  // Each segment (prompt, beacons, window) starts a new tile, so a tile never straddles segments;
  // a partly filled tile costs masked arithmetic but no memory traffic.
  if (FUSED && p.f.plan != nullptr) {
    // bc_decode_step: the step's bookkeeping kernel, whose results are visible (the flag, or the wait,
    // above), left the plan of this very batch: seven coalesced reads instead of slots -> lengths -> prefix sum
    const int32_t* a = p.f.plan + BC_PLAN_HEADER;
    for (int i = tid; i < n; i += kPipeThreads) {
      s_P[i] = a[i]; s_nb[i] = a[BC_MAX_ATTN_BATCH + i]; s_w[i] = a[2 * BC_MAX_ATTN_BATCH + i];
      s_slot[i] = a[3 * BC_MAX_ATTN_BATCH + i]; s_bcol[i] = a[4 * BC_MAX_ATTN_BATCH + i]; s_wcol[i] = a[5 * BC_MAX_ATTN_BATCH + i];
      s_cum[i] = a[6 * BC_MAX_ATTN_BATCH + i];
    }
    if (tid == 0) s_cum[n] = a[6 * BC_MAX_ATTN_BATCH + n];
    __syncthreads();
  } else {
    for (int i = tid; i < n; i += kPipeThreads) {
      const int slot = p.a.slots[i];
      int P = 0, nb = 0, w = 0, bcol = 0, wcol = 0, sl = 0;
      if (slot >= 0 && slot < p.m.max_seqs && p.m.open[slot]) {
        P = p.m.prompt_len[slot]; nb = p.m.n_beacons[slot]; w = p.m.window_len[slot];
        bcol = p.m.beacon_off[slot]; wcol = p.m.window_off[slot]; sl = slot;
      }
      if (FUSED && w > 0 && p.f.dst_row[i] >= 0) sl |= kNewRowBit;  // the window's last entry is this launch's
      s_P[i] = P; s_nb[i] = nb; s_w[i] = w; s_slot[i] = sl; s_bcol[i] = bcol; s_wcol[i] = wcol;
      const int tiles = ((P + T - 1) >> TS) + ((nb + T - 1) >> TS) + ((w + T - 1) >> TS);
      s_cum[i + 1] = tiles > 0 ? tiles : 1;  // an empty sequence still owns one (empty) tile
    }
    __syncthreads();
    if (warp == 0) {  // inclusive scan of s_cum[1..n]
      int carry = 0;
      for (int base = 0; base < n; base += 32) {
        const int i = base + lane;
        int x = i < n ? s_cum[i + 1] : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          int y = __shfl_up_sync(0xffffffffu, x, d);
          if (lane >= d) x += y;
        }
        if (i < n) s_cum[i + 1] = carry + x;
        carry += __shfl_sync(0xffffffffu, x, 31);
      }
      if (lane == 0) s_cum[0] = 0;
    }
    __syncthreads();
  }
  const int total_tiles = s_cum[n];
  stamp(1);
  // Every read of the sequences' lengths is done (the page-table columns the producer reads later are
  // below those lengths and never rewritten while they are): a kernel enqueued behind this one with
  // programmatic stream serialisation -- the next step's bookkeeping -- may start on the first SM
  // that frees up instead of after this kernel's last block.  Kernels launched the ordinary way wait
  // for the whole grid as before.  The fused form goes on reading the rows' destinations (dst_row,
  // dst_pos); the next step's bookkeeping fills the other of two sets, so it may start early as well.
  // A fused step that started early lets its dependents go only once it has waited for the kernel ahead
  // (see wait_for_kernel_ahead): its service warps write pool rows, and at most two row-writing launches
  // may be alive at a time for the "settled" rule below to hold.
  if (FUSED ? !early : true) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // With early_meta the wait for the kernel ahead is still to come: every role below executes it before it
  // touches anything but `slots` and the metadata -- the pool rows of this step, q, the extra entry, the
  // partial buffers and tickets this launch shares with the one before it, and every output.  So the plan
  // above (three dependent trips to memory) and the producer's first page-table reads run under the
  // predecessor instead of after it.
  auto wait_for_kernel_ahead = [&]() {
    if (early) {
      asm volatile("griddepcontrol.wait;" ::: "memory");
      if (FUSED) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
  };
  const int n_ctas = (int)gridDim.x;
  const int per = total_tiles / n_ctas, rem = total_tiles % n_ctas;
  const int cta = (int)blockIdx.x;
  const int g0 = cta * per + min(cta, rem);
  const int g1 = g0 + per + (cta < rem ? 1 : 0);
  if (g0 >= g1) return;
  // block that owns global tile g under the flat partition
  auto cta_of = [&](int g) { return g < rem * (per + 1) ? g / (per + 1) : rem + (g - rem * (per + 1)) / per; };
  int seq0 = 0;
  {  // largest i with cum[i] <= g0
    int lo = 0, hi = n;
    while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (s_cum[mid] <= g0) lo = mid; else hi = mid; }
    seq0 = lo;
  }

  // The block's first piece: if it covers only part of its sequence and more pieces follow, the
  // service warp publishes it (fence, then ticket), because the fence has to wait until the
  // piece's stores have reached L2 -- microseconds while every SM is streaming -- and a consumer
  // warp that waited there would stall the whole pipeline between pieces.
  bool svc_publishes;
  {
    const int tiles0 = s_cum[seq0 + 1] - s_cum[seq0], ta0 = g0 - s_cum[seq0];
    const int tb0 = min(tiles0, ta0 + (g1 - g0));
    svc_publishes = !(ta0 == 0 && tb0 == tiles0) && (g0 + (tb0 - ta0) < g1);
  }
  if (warp == kConsumerWarps + 1) {
    // ================================ service warp =============================================
    wait_for_kernel_ahead();
    if (FUSED) {
      // store the new entries of the sequences whose last tile this block owns (for the steps to come)
      const int chunks = p.g.head_row_bytes >> 4, per_side = Hkv * chunks;
      for (int i = seq0; i < n && s_cum[i + 1] - 1 < g1; ++i) {
        if (s_cum[i + 1] - 1 < g0 || !(s_slot[i] & kNewRowBit)) continue;
        if (p.debug && (unsigned)p.f.dst_row[i] >= (unsigned)(p.m.num_pages * ps)) {   // row outside the pool: not written
          if (lane == 0) debug_note(p.m, p.f.dst_row[i]);
          continue;
        }
        uint8_t* dst = p.f.pool_w + (int64_t)p.f.dst_row[i] * E;
        const int key = p.f.dst_pos[i] & 7;
        for (int idx = lane; idx < 2 * per_side; idx += 32) {
          const int which = idx / per_side, rem = idx - which * per_side, h = rem / chunks, j = rem - h * chunks;
          const uint8_t* src = (which ? p.f.new_v : p.f.new_k) + ((int64_t)i * Hkv + h) * p.g.head_row_bytes + (j << 4);
          *reinterpret_cast<uint4*>(dst + (which * Hkv + h) * p.g.head_row_bytes + ((j ^ key) << 4)) =
              *reinterpret_cast<const uint4*>(src);
        }
      }
    }
    if (svc_publishes) {
      const bool ok = bounded_wait<SHORTW>(bar_pub, 0, s_abort, p.spin_limit);  // every consumer warp has stored its share
      if (lane == 0) {
        if (ok) {
          __threadfence();
          s_pend[1] = atomicAdd(p.a.tickets + seq0, 1);
          s_pend[0] = seq0;
        } else {
          s_pend[0] = -1;
        }
        mbar_arrive(bar_tk);
      }
    }
    return;
  }
  if (warp == kConsumerWarps) {
    // ================================ producer warp ============================================
    // describe(gt) runs kPidAhead tiles ahead of the copies: it works out which rows tile gt holds,
    // writes {rows, first position, first page} to a small descriptor ring and starts 4-byte
    // asynchronous copies of the tile's page-table entries into the same slot.  Issuing the bulk
    // copies of a tile then takes a handful of instructions and never waits on the page table.
    const uint64_t stream_policy = l2_policy_evict_first();
    int fi = seq0;
    int f_P, f_nb, f_w, f_tp, f_tpb, f_bcol, f_wcol;
    bool f_new = false;
    const int32_t* f_tab;
    auto load_seq = [&](int i) {
      f_P = s_P[i]; f_nb = s_nb[i]; f_w = s_w[i]; f_bcol = s_bcol[i]; f_wcol = s_wcol[i];
      f_tp = (f_P + T - 1) >> TS; f_tpb = f_tp + ((f_nb + T - 1) >> TS);
      f_tab = p.m.page_table + (int64_t)(s_slot[i] & ~kNewRowBit) * p.m.max_pages_per_seq;
      f_new = FUSED && (s_slot[i] & kNewRowBit);
    };
    load_seq(fi);
    auto describe = [&](int gt, int it) {
      int nrows = 0, p0 = 0, pg0 = 0, settled = 1;
      const int slot_idx = (it % RING) * kPidSlot;
      if (gt < g1) {
        while (gt >= s_cum[fi + 1]) { ++fi; load_seq(fi); }
        const int t = gt - s_cum[fi];
        int len, tt, col;
        if (t < f_tp) { len = f_P; tt = t; col = 0; }
        else if (t < f_tpb) { len = f_nb; tt = t - f_tp; col = f_bcol; settled = t != f_tpb - 1; }
        else {
          // a fused step may run while the fused step before it still stores ITS new window entry, which
          // can lie in the tile before the last one: there the last two window tiles are left alone
          len = f_w; tt = t - f_tpb; col = f_wcol; settled = gt < s_cum[fi + 1] - (FUSED ? 2 : 1);
        }
        p0 = tt << TS;
        nrows = max(min(T, len - p0), 0);
        if (FUSED && f_new && gt == s_cum[fi + 1] - 1) nrows -= 1;  // the new row comes from the input, not the pool
        if (nrows > 0) {
          pg0 = fast_div(p0, p.div_ps);
          const int pg_last = fast_div(p0 + nrows - 1, p.div_ps);
          for (int pg = pg0 + lane; pg <= pg_last; pg += 32) {
            if (p.debug && (unsigned)(col + pg) >= (unsigned)p.m.max_pages_per_seq) {   // column outside the row
              debug_note(p.m, col + pg);
              s_desc[slot_idx + 4 + pg - pg0] = 0;
            } else {
              cp_async4(desc_ring + (uint32_t)(slot_idx + 4 + pg - pg0) * 4u, f_tab + col + pg);
            }
          }
        }
      }
      // settled: every row of the tile was stored by a kernel that has ended by the time this one may
      // begin -- all but the last tile of a beacon or window segment, where the newest entry lives
      if (lane == 0) { s_desc[slot_idx] = nrows; s_desc[slot_idx + 1] = p0; s_desc[slot_idx + 2] = pg0; s_desc[slot_idx + 3] = settled; }
      cp_async_commit();  // one group per described tile
    };
    // The first tile is described alone so that its copies start as early as possible; the
    // lookahead then grows by up to two tiles per iteration until it is kPidAhead deep.
    int described = 1;
    describe(g0, 0);
    // With early_meta the producer does not wait for the kernel ahead before it starts to stream: page-table
    // entries and "settled" tiles may be fetched while that kernel finishes.  The kernels of this library
    // that can still be running then (they release their dependents early) are the row-writing kernel and
    // another attention kernel, and in the pool those write nothing but the newest entry of a beacon or
    // window segment, which lies in the segment's last tile.  Before the first tile that is not settled
    // the producer waits like everybody else.  (The consumers wait before they touch q or a tile, so the
    // ring fills up to its three stages and stalls there until the kernel ahead has ended.)
    bool waited = !early;
    int it = 0;
    bool aborted = false;
#pragma unroll 1
    for (int gt = g0; gt < g1; ++gt, ++it) {
      cp_async_wait_dyn(described - it - 1);  // the page ids of tile gt have landed
      __syncwarp();
      if (!waited && !s_desc[(it % RING) * kPidSlot + 3]) { wait_for_kernel_ahead(); waited = true; }
      const int stage = it % NSTAGE;
      const uint32_t full = bar_full + stage * 8, empty = bar_empty + stage * 8;
      if (!bounded_wait<SHORTW>(empty, ((it / NSTAGE) & 1) ^ 1, s_abort, p.spin_limit)) aborted = true;
      // at most kInFlight stages in flight: the copies of tile it - kInFlight must have landed
      if (!aborted && it >= kInFlight &&
          !bounded_wait<SHORTW>(bar_full + ((it - kInFlight) % NSTAGE) * 8, ((it - kInFlight) / NSTAGE) & 1, s_abort, p.spin_limit))
        aborted = true;
      if (aborted) break;   // `it` stages have been armed; the consumers see the abort flag in their own waits
      {
        const int* d = s_desc + (it % RING) * kPidSlot;
        const int nrows = d[0], p0 = d[1], pg0 = d[2];
        if (lane == 0) {
          if (nrows > 0) mbar_arrive_expect_tx(full, (uint32_t)nrows * (uint32_t)E);
          else mbar_arrive(full);
        }
        const uint32_t stage_base = ring + stage * L::kStageBytes;
        for (int k = lane;; k += 32) {
          const int pg = pg0 + k;
          const int lo = max(p0, pg * ps), hi = min(p0 + nrows, pg * ps + ps);
          if (lo >= hi) break;
          int page = d[4 + k];
          if (p.debug && (unsigned)page >= (unsigned)p.m.num_pages) { debug_note(p.m, page); page = 0; }   // read a valid page instead
          const uint8_t* src = p.a.pool_layer + ((int64_t)page * ps + (lo - pg * ps)) * E;
          bulk_g2s(stage_base + (uint32_t)(lo - p0) * (uint32_t)E, src, (uint32_t)(hi - lo) * (uint32_t)E, full, stream_policy);
        }
      }
      __syncwarp();  // the slot read above may be rewritten by the describe() calls below
#pragma unroll 1
      for (int r = 0; r < 2 && described < it + 1 + kPidAhead && g0 + described < g1; ++r, ++described)
        describe(g0 + described, described);
    }
    cp_async_wait<0>();
    // Drain: every armed stage whose copies might still be in flight must complete before exit.
    if (aborted || *s_abort) {
      const int armed = it;
      for (int k = max(0, armed - NSTAGE); k < armed; ++k) {
        uint32_t polls = 0;
        while (!mbar_try_wait(bar_full + (k % NSTAGE) * 8, (k / NSTAGE) & 1) && ++polls < kSpinLimit) __nanosleep(64);
      }
      if (lane == 0 && p.m.status[0] == 0) { p.m.status[0] = BC_ERR_TIMEOUT; p.m.status[1] = -1; }
    }
    return;
  }

  // ================================== consumer warps ===========================================
  // The consumers do not wait for the kernel ahead before they start either: they read the queries and
  // the extra entry (inputs, which no kernel that releases its dependents early may write) and whatever
  // settled tiles the producer has brought in, and they write nothing outside the block until a piece
  // ends.  They wait before the first thing they share with the launch before them: the ticket
  // counters, the partial buffers, the outputs.
  bool cons_waited = !early;
  auto consumers_wait = [&]() {
    if (!cons_waited) { wait_for_kernel_ahead(); cons_waited = true; stamp(2); }
  };
  if (!early) stamp(2);
  stamp_val(8, ((unsigned long long)(g1 - g0) << 32) | (unsigned)seq0);
  const int kvh = warp % Hkv, grp = warp / Hkv;
  const int gq = lane >> 2, qd = lane & 3;  // fragment row and column-pair index
  // ldmatrix lane offsets inside this warp's 16 rows of a stage
  const int lm = lane >> 3, lr = lane & 7;
  const uint32_t k_lane_off = (uint32_t)((((lm >> 1) << 3) + lr) * E + kvh * p.g.head_row_bytes);
  const int k_chunk_sel = lm & 1;
  const uint32_t v_lane_off = (uint32_t)((((lm & 1) << 3) + lr) * E + (Hkv + kvh) * p.g.head_row_bytes);
  const int v_chunk_sel = lm >> 1;
  const uint32_t warp_rows_off = (uint32_t)(grp * 16) * (uint32_t)E;

  // query fragments of sequence i: rows = the G query heads of this warp's KV head
  auto load_q = [&](uint32_t (&qr)[KSTEPS][4], int i) {
    const __nv_bfloat16* qb = reinterpret_cast<const __nv_bfloat16*>(p.a.q) + ((int64_t)i * Hq + kvh * G) * D;
#pragma unroll
    for (int kk = 0; kk < KSTEPS; ++kk) {
      const int d0 = kk * 16 + qd * 2;
      if (PACK) {
        const __nv_bfloat16* qb2 = reinterpret_cast<const __nv_bfloat16*>(p.a.q2) + ((int64_t)i * Hq + kvh * G) * D;
        const __nv_bfloat16* src = gq < G ? qb + gq * D : qb2 + (gq - G) * D;
        qr[kk][0] = gq < 2 * G ? *reinterpret_cast<const uint32_t*>(src + d0) : 0u;
        qr[kk][2] = gq < 2 * G ? *reinterpret_cast<const uint32_t*>(src + d0 + 8) : 0u;
        qr[kk][1] = 0u; qr[kk][3] = 0u;
        continue;
      }
      qr[kk][0] = gq < G ? *reinterpret_cast<const uint32_t*>(qb + gq * D + d0) : 0u;
      qr[kk][2] = gq < G ? *reinterpret_cast<const uint32_t*>(qb + gq * D + d0 + 8) : 0u;
      if (G_LE_8) { qr[kk][1] = 0u; qr[kk][3] = 0u; }
      else if (PAIR) {   // rows 8 .. 8 + G - 1: the beacon's query heads of the same KV head
        const __nv_bfloat16* qb2 = reinterpret_cast<const __nv_bfloat16*>(p.a.q2) + ((int64_t)i * Hq + kvh * G) * D;
        qr[kk][1] = gq < G ? *reinterpret_cast<const uint32_t*>(qb2 + gq * D + d0) : 0u;
        qr[kk][3] = gq < G ? *reinterpret_cast<const uint32_t*>(qb2 + gq * D + d0 + 8) : 0u;
      } else {
        qr[kk][1] = gq + 8 < G ? *reinterpret_cast<const uint32_t*>(qb + (gq + 8) * D + d0) : 0u;
        qr[kk][3] = gq + 8 < G ? *reinterpret_cast<const uint32_t*>(qb + (gq + 8) * D + d0 + 8) : 0u;
      }
    }
  };

  int i = seq0;
  int it = 0;
  int gt = g0;
  int pend_seq = -1, pend_tk = 0;  // thread 0: ticket of the block's final piece, if it had to be published
  unsigned tl_path = 0;            // timeline word 9: how the block's final piece left and which merges it owed
  bool published_last = false;
  uint32_t qf[KSTEPS][4];
  load_q(qf, seq0);
  while (gt < g1) {
    while (gt >= s_cum[i + 1]) ++i;
    const int c_P = s_P[i], c_nb = s_nb[i], c_w = s_w[i];
    const int c_tp = (c_P + T - 1) >> TS, c_tpb = c_tp + ((c_nb + T - 1) >> TS);
    const int tiles_i = s_cum[i + 1] - s_cum[i];
    const int ta = gt - s_cum[i];
    const int tb = min(tiles_i, ta + (g1 - gt));
    const bool whole = (ta == 0 && tb == tiles_i);
    // the next piece's query fragments are fetched now, so the switch between pieces does not wait
    const bool has_next = gt + (tb - ta) < g1;
    uint32_t qn[KSTEPS][4];
    if (has_next) load_q(qn, i + 1);

    float o[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    int early_cnt = -1;   // thread 0: the ticket counter as seen at the start of the final piece's last tile

    // ---- the extra (unstored) entry seeds the state of the piece that owns tile 0 ---------------
    if (p.a.extra_k != nullptr && ta == 0 && grp == 0) {
      const __nv_bfloat16* ek = reinterpret_cast<const __nv_bfloat16*>(p.a.extra_k) + ((int64_t)i * Hkv + kvh) * D;
      const __nv_bfloat16* ev = reinterpret_cast<const __nv_bfloat16*>(p.a.extra_v) + ((int64_t)i * Hkv + kvh) * D;
      float d0 = 0.f, d1 = 0.f;
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk) {
        const int dd = kk * 16 + qd * 2;
        const uint32_t ka = *reinterpret_cast<const uint32_t*>(ek + dd);
        const uint32_t kb = *reinterpret_cast<const uint32_t*>(ek + dd + 8);
        d0 += bf16_lo(qf[kk][0]) * bf16_lo(ka) + bf16_hi(qf[kk][0]) * bf16_hi(ka) +
              bf16_lo(qf[kk][2]) * bf16_lo(kb) + bf16_hi(qf[kk][2]) * bf16_hi(kb);
        if (!G_LE_8)
          d1 += bf16_lo(qf[kk][1]) * bf16_lo(ka) + bf16_hi(qf[kk][1]) * bf16_hi(ka) +
                bf16_lo(qf[kk][3]) * bf16_lo(kb) + bf16_hi(qf[kk][3]) * bf16_hi(kb);
      }
      d0 += __shfl_xor_sync(0xffffffffu, d0, 1); d0 += __shfl_xor_sync(0xffffffffu, d0, 2);
      if (!G_LE_8) { d1 += __shfl_xor_sync(0xffffffffu, d1, 1); d1 += __shfl_xor_sync(0xffffffffu, d1, 2); }
      // paired form: only the beacon's rows see the extra entry
      const bool r0 = PACK ? (gq >= G && gq < 2 * G) : (!PAIR && gq < G);
      const bool r1 = PACK ? false : (PAIR ? gq < G : (!G_LE_8 && (gq + 8 < G)));
      if (r0) { m0 = d0 * p.scale_log2; l0 = qd == 0 ? 1.f : 0.f; }
      if (r1) { m1 = d1 * p.scale_log2; l1 = qd == 0 ? 1.f : 0.f; }
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        const uint32_t vv = *reinterpret_cast<const uint32_t*>(ev + nt * 8 + qd * 2);
        if (r0) { o[nt][0] = bf16_lo(vv); o[nt][1] = bf16_hi(vv); }
        if (r1) { o[nt][2] = bf16_lo(vv); o[nt][3] = bf16_hi(vv); }
      }
    }

    // ---- stream the tiles of this piece ----------------------------------------------------------
    for (int t = ta; t < tb; ++t, ++it, ++gt) {
      const int stage = it % NSTAGE;
      // FUSED: the sequence's last tile lacks this launch's new entry (the bulk copy left it out);
      // the warps whose 16-row group holds it fetch their head's K and V chunks of it from the input
      // (lanes 0-15: K, lanes 16-31: V) while the tile is still in flight.
      // The final piece's last tile: look at the sequence's ticket counter now, while the tile is still
      // in flight.  If every other piece is there already, the merge after the tile starts at once (the
      // count cannot go back); if not, the counter is read again after the tile.
      if (!PAIR && !has_next && !whole && t == tb - 1) {
        consumers_wait();   // the counter is shared with the launch before this one
        if (tid == 0) early_cnt = ld_acquire(p.a.tickets + i);
      }
      bool patch = false;
      int patch_row = 0;
      uint4 patch_val = make_uint4(0u, 0u, 0u, 0u);
      if (FUSED && (s_slot[i] & kNewRowBit) && t == tiles_i - 1) {
        patch_row = (c_w - 1) - ((t - c_tpb) << TS);
        if ((patch_row >> 4) == grp) {
          patch = true;
          if ((lane & 15) < (p.g.head_row_bytes >> 4))
            patch_val = *reinterpret_cast<const uint4*>(((lane >> 4) ? p.f.new_v : p.f.new_k) +
                                                        ((int64_t)i * Hkv + kvh) * p.g.head_row_bytes + ((lane & 15) << 4));
        }
      }
      const bool ok = __all_sync(0xffffffffu, bounded_wait<SHORTW>(bar_full + stage * 8, (it / NSTAGE) & 1, s_abort, p.spin_limit));
      if (it == 0) stamp(3);
      if (!ok && lane == 0 && p.m.status[0] == 0) { p.m.status[0] = BC_ERR_TIMEOUT; p.m.status[1] = -1; }
      // rows of this tile that hold entries; my warp looks at rows grp*16 .. grp*16+15 of it
      int seg_left;
      if (t < c_tp) seg_left = c_P - (t << TS);
      else if (t < c_tpb) seg_left = c_nb - ((t - c_tp) << TS);
      else seg_left = c_w - ((t - c_tpb) << TS);
      const int cnt = max(min(seg_left - grp * 16, 16), 0);
      bool wrote_smem = false;
      if (ok && cnt > 0) {
        const uint32_t rows_base = ring + stage * L::kStageBytes + warp_rows_off;
        if (FUSED && patch) {
          if ((lane & 15) < (p.g.head_row_bytes >> 4))
            *reinterpret_cast<uint4*>(smem + stage * L::kStageBytes + warp_rows_off + (patch_row & 15) * E +
                                      ((lane >> 4) * Hkv + kvh) * p.g.head_row_bytes +
                                      (((lane & 15) ^ ((c_w - 1) & 7)) << 4)) = patch_val;
          wrote_smem = true;
          __syncwarp();
        }
        if (cnt < 16) {
          // rows nobody copied may hold anything: zero their V so that 0 * garbage cannot be NaN
          uint8_t* rows_ptr = smem + stage * L::kStageBytes + warp_rows_off;
          for (int r = cnt; r < 16; ++r) {
            if (lane < (p.g.head_row_bytes >> 4))
              *reinterpret_cast<uint4*>(rows_ptr + r * E + (Hkv + kvh) * p.g.head_row_bytes + lane * 16) =
                  make_uint4(0, 0, 0, 0);
          }
          wrote_smem = true;
          __syncwarp();
        }
        // S = Q K^T for 16 keys: two n-tiles of 8 keys
        float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int kk = 0; kk < KSTEPS; ++kk) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4(rows_base + k_lane_off + (uint32_t)(((kk * 2 + k_chunk_sel) ^ lr) << 4), b0, b1, b2, b3);
          mma_bf16(s[0], qf[kk], b0, b1);
          mma_bf16(s[1], qf[kk], b2, b3);
        }
        // scale to the log2 domain and mask
#pragma unroll
        for (int j = 0; j < 2; ++j)
#pragma unroll
          for (int e = 0; e < 4; ++e) s[j][e] *= p.scale_log2;
        if (cnt < 16) {
#pragma unroll
          for (int j = 0; j < 2; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              if (j * 8 + qd * 2 + e >= cnt) { s[j][e] = -INFINITY; s[j][e + 2] = -INFINITY; }
            }
        }
        // online softmax, row gq (and gq + 8)
        float mx0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
        const float mn0 = fmaxf(m0, mx0);
        const float ms0 = mn0 == -INFINITY ? 0.f : mn0;
        const float al0 = exp2f(m0 - ms0);
        m0 = mn0;
        const float p00 = exp2f(s[0][0] - ms0), p01 = exp2f(s[0][1] - ms0);
        const float p10 = exp2f(s[1][0] - ms0), p11 = exp2f(s[1][1] - ms0);
        l0 = l0 * al0 + (p00 + p01 + p10 + p11);
        uint32_t pa[4];
        pa[0] = pack_bf16(p00, p01);
        pa[2] = pack_bf16(p10, p11);
        float al1 = 1.f;
        if (G_LE_8) { pa[1] = 0u; pa[3] = 0u; }
        else {
          float mx1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
          mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
          const float mn1 = fmaxf(m1, mx1);
          const float ms1 = mn1 == -INFINITY ? 0.f : mn1;
          al1 = exp2f(m1 - ms1);
          m1 = mn1;
          const float q00 = exp2f(s[0][2] - ms1), q01 = exp2f(s[0][3] - ms1);
          const float q10 = exp2f(s[1][2] - ms1), q11 = exp2f(s[1][3] - ms1);
          l1 = l1 * al1 + (q00 + q01 + q10 + q11);
          pa[1] = pack_bf16(q00, q01);
          pa[3] = pack_bf16(q10, q11);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
          o[nt][0] *= al0; o[nt][1] *= al0;
          if (!G_LE_8) { o[nt][2] *= al1; o[nt][3] *= al1; }
        }
        // O += P V
#pragma unroll
        for (int jj = 0; jj < NT / 2; ++jj) {
          uint32_t b0, b1, b2, b3;
          ldsm_x4_t(rows_base + v_lane_off + (uint32_t)(((jj * 2 + v_chunk_sel) ^ lr) << 4), b0, b1, b2, b3);
          mma_bf16(o[jj * 2], pa, b0, b1);
          mma_bf16(o[jj * 2 + 1], pa, b2, b3);
        }
      }
      __syncwarp();
      if (lane == 0) {
        if (wrote_smem) fence_proxy_async();
        mbar_arrive(bar_empty + stage * 8);
      }
    }

    // ---- end of piece: merge the groups of each KV head in shared memory, then write -------------
    consumers_wait();
    if (!has_next) stamp(4);
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    if (!G_LE_8) { l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2); }
    if constexpr (PAIR) {
      // How this piece leaves: 0 = the whole sequence is here, 1 = final piece and every other piece is
      // published (merge now), 2 = publish.  The same for the token's and the beacon's heads, which go
      // through the merge buffer one after the other.
      int mode = whole ? 0 : 2;
      int first = 0, last = 0;
      if (!whole) {
        first = cta_of(s_cum[i]); last = cta_of(s_cum[i + 1] - 1);
        if (!has_next) {
          if (tid == 0) s_pend[4] = ld_acquire(p.a.tickets + i);
          consumer_bar();
          if (s_pend[4] == last - first) { mode = 1; __threadfence(); }
        }
      }
      const int64_t pslot = (int64_t)cta + i;
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        for (int gi = 0; gi < p.n_groups; ++gi) {
          const bool takes_part = PACK ? (gq >= half * G && gq < (half + 1) * G) : gq < G;
          if (grp == gi && takes_part) {
            const int h = kvh * G + (PACK ? gq - half * G : gq);
            const bool second = half && !PACK;   // the row's state: rows 8..15 of the fragment, or (packed) rows 0..7
            const float mm = second ? m1 : m0, ll = second ? l1 : l0;
            float sa = 0.f, sb = 1.f, mnew = mm, lnew = ll;
            if (gi > 0) {
              const float mb = merge_ml[h * 2], lb = merge_ml[h * 2 + 1];
              mnew = fmaxf(mb, mm);
              const float msafe = mnew == -INFINITY ? 0.f : mnew;
              sa = exp2f(mb - msafe); sb = exp2f(mm - msafe);
              lnew = lb * sa + ll * sb;
            }
            float* orow = merge_o + h * D;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              const int d = nt * 8 + qd * 2;
              float2 cur = gi > 0 ? *reinterpret_cast<float2*>(orow + d) : make_float2(0.f, 0.f);
              cur.x = cur.x * sa + (second ? o[nt][2] : o[nt][0]) * sb;
              cur.y = cur.y * sa + (second ? o[nt][3] : o[nt][1]) * sb;
              *reinterpret_cast<float2*>(orow + d) = cur;
            }
            __syncwarp(__activemask());
            if (qd == 0) { merge_ml[h * 2] = mnew; merge_ml[h * 2 + 1] = lnew; }
          }
          consumer_bar();
        }
        void* outp = half ? p.a.out2 : p.a.out;
        float* part_o = half ? p.a.part_o2 : p.a.part_o;
        float* part_ml = half ? p.a.part_ml2 : p.a.part_ml;
        if (mode == 0) {
          const int64_t obase = (int64_t)i * Hq * D;
          for (int idx = tid; idx < Hq * D; idx += kConsumerWarps * 32) {
            const int h = idx / D;
            const float l = merge_ml[h * 2 + 1];
            const float val = l > 0.f ? merge_o[idx] / l : 0.f;
            if (p.a.out_f32) reinterpret_cast<float*>(outp)[obase + idx] = val;
            else reinterpret_cast<__nv_bfloat16*>(outp)[obase + idx] = __float2bfloat16_rn(val);
          }
        } else if (mode == 1) {
          combine_pieces(part_o, part_ml, outp, p.a.out_f32, Hq, D, i, first, last, cta, merge_o, merge_ml, tid);
        } else {
          float* po = part_o + pslot * Hq * D;
          for (int idx = tid; idx < Hq * D; idx += kConsumerWarps * 32) po[idx] = merge_o[idx];
          if (tid < Hq * 2) part_ml[pslot * Hq * 2 + tid] = merge_ml[tid];
        }
        consumer_bar();  // the merge buffer is reused by the other half and by the next piece
      }
      if (mode == 1) {
        if (tid == 0) p.a.tickets[i] = 0;  // ready for the next launch
      } else if (mode == 2) {
        if (has_next) {
          // the block's first piece: hand it to the service warp and go on streaming
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_pub);
        } else {
          if (tid == 0) {
            __threadfence();
            pend_tk = atomicAdd(p.a.tickets + i, 1);
            pend_seq = i;
          }
          published_last = true;
        }
      }
    } else {
    for (int gi = 0; gi < p.n_groups; ++gi) {
      if (grp == gi) {
#pragma unroll
        for (int half = 0; half < (G_LE_8 ? 1 : 2); ++half) {
          const int row = gq + half * 8;
          if (row < G) {
            const int h = kvh * G + row;
            const float mm = half ? m1 : m0, ll = half ? l1 : l0;
            float sa = 0.f, sb = 1.f, mnew = mm, lnew = ll;
            if (gi > 0) {
              const float mb = merge_ml[h * 2], lb = merge_ml[h * 2 + 1];
              mnew = fmaxf(mb, mm);
              const float msafe = mnew == -INFINITY ? 0.f : mnew;
              sa = exp2f(mb - msafe); sb = exp2f(mm - msafe);
              lnew = lb * sa + ll * sb;
            }
            float* orow = merge_o + h * D;
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
              const int d = nt * 8 + qd * 2;
              float2 cur = gi > 0 ? *reinterpret_cast<float2*>(orow + d) : make_float2(0.f, 0.f);
              cur.x = cur.x * sa + o[nt][half * 2] * sb;
              cur.y = cur.y * sa + o[nt][half * 2 + 1] * sb;
              *reinterpret_cast<float2*>(orow + d) = cur;
            }
            __syncwarp(__activemask());
            if (qd == 0) { merge_ml[h * 2] = mnew; merge_ml[h * 2 + 1] = lnew; }
          }
        }
      }
      consumer_bar();
    }
    if (whole) {
      const int64_t obase = (int64_t)i * Hq * D;
      for (int idx = tid; idx < Hq * D; idx += kConsumerWarps * 32) {
        const int h = idx / D;
        const float l = merge_ml[h * 2 + 1];
        const float val = l > 0.f ? merge_o[idx] / l : 0.f;
        if (p.a.out_f32) reinterpret_cast<float*>(p.a.out)[obase + idx] = val;
        else reinterpret_cast<__nv_bfloat16*>(p.a.out)[obase + idx] = __float2bfloat16_rn(val);
      }
      consumer_bar();  // the merge buffer is reused by the next piece
      if (!has_next) tl_path |= 1u;
    } else {
      const int first = cta_of(s_cum[i]), last = cta_of(s_cum[i + 1] - 1);
      bool merged = false;
      if (!has_next) {
        // The block's final piece.  If every other piece of this sequence was there already when the last
        // tile began (the counter was read then, under the tile), this block merges right away, taking
        // its own piece from shared memory, and publishes nothing.  Otherwise it publishes and takes a
        // ticket like everybody else -- no second look at the counter: the blocks of a sequence finish
        // within a microsecond or two of each other, so a look now mostly fails and costs a trip to L2.
        if (tid == 0) s_pend[4] = early_cnt;
        consumer_bar();
        if (s_pend[4] == last - first) {
          __threadfence();
          combine_pieces(p.a.part_o, p.a.part_ml, p.a.out, p.a.out_f32, Hq, D, i, first, last, cta, merge_o, merge_ml, tid);
          if (tid == 0) p.a.tickets[i] = 0;  // ready for the next launch
          merged = true;
          tl_path |= 2u;
        }
      }
      if (!merged) {
        // Publish this piece and take a ticket from the sequence's counter.  Nobody looks at the
        // ticket before the block has streamed all its tiles: whoever took a sequence's last
        // ticket merges its pieces then.
        const int64_t pslot = (int64_t)cta + i;
        float* po = p.a.part_o + pslot * Hq * D;
        for (int idx = tid; idx < Hq * D; idx += kConsumerWarps * 32) po[idx] = merge_o[idx];
        if (tid < Hq * 2) p.a.part_ml[pslot * Hq * 2 + tid] = merge_ml[tid];
        if (has_next) {
          // the block's first piece: hand it to the service warp and go on streaming
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_pub);
          consumer_bar();  // frees the merge buffer
        } else {
          consumer_bar();  // orders every thread's stores before thread 0's fence
          if (tid == 0) {
            pend_tk = ticket_acq_rel(p.a.tickets + i);
            pend_seq = i;
          }
          published_last = true;
          tl_path |= 4u;
        }
      }
    }
    }
    if (has_next) {
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk) {
        qf[kk][0] = qn[kk][0]; qf[kk][2] = qn[kk][2];
        if (!G_LE_8) { qf[kk][1] = qn[kk][1]; qf[kk][3] = qn[kk][3]; }
      }
    }
  }

  // ---- all tiles streamed: merge the sequences whose last ticket this block took -----------------
  stamp(5);
  if (svc_publishes) bounded_wait<SHORTW>(bar_tk, 0, s_abort, p.spin_limit);
  stamp(6);
  if (published_last) {
    if (tid == 0) { s_pend[2] = pend_seq; s_pend[3] = pend_tk; }
    consumer_bar();
  }
  for (int k = 0; k < 2; ++k) {
    if (k == 0 ? !svc_publishes : !published_last) continue;
    const int seq = s_pend[2 * k], tk = s_pend[2 * k + 1];
    if (seq < 0) continue;
    const int first = cta_of(s_cum[seq]), last = cta_of(s_cum[seq + 1] - 1);
    if (tk == last - first) {
      tl_path |= 8u << k;
      if (k == 0 || PAIR) __threadfence();   // the service warp's and the paired form's tickets are plain atomics
      // the final piece is still in the merge buffer (nothing followed it); the first piece is not
      const bool own_here = k == 1 && !PAIR;
      combine_pieces(p.a.part_o, p.a.part_ml, p.a.out, p.a.out_f32, Hq, D, seq, first, last, own_here ? cta : -1,
                     own_here ? merge_o : nullptr, own_here ? merge_ml : nullptr, tid);
      if (PAIR) combine_pieces(p.a.part_o2, p.a.part_ml2, p.a.out2, p.a.out_f32, Hq, D, seq, first, last, -1, nullptr, nullptr, tid);
      if (tid == 0) p.a.tickets[seq] = 0;  // ready for the next launch
    }
  }
  stamp(7);
  stamp_val(9, tl_path);
}

// ---------------------------------------------------------------- read-only streaming probe
// What the decode kernel's own access pattern can draw from HBM when nothing is computed: every block
// copies its share of a buffer in 64 KB pieces into a three-stage ring with the same 1-D bulk copies,
// the same evict-first policy and the same limit of two stages in flight; one warp consumes (waits
// for a stage and hands it back).  A measurement aid for the roofline's denominator: the copy
// benchmark that defines the reported peak reads AND writes, a decode step only reads.
__global__ void __launch_bounds__(64, 1) k_read_stream(const uint8_t* __restrict__ buf, long long pieces, int* sink) {
  constexpr int kPiece = 64 << 10, kRing = 3;
  extern __shared__ __align__(1024) uint8_t smem[];
  __shared__ __align__(8) uint64_t bars[2 * kRing];
  __shared__ int s_abort_word;
  volatile int* s_abort = &s_abort_word;
  const uint32_t ring = smem_u32(smem), bar_full = smem_u32(bars), bar_empty = bar_full + kRing * 8;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kRing; ++s) { mbar_init(bar_full + s * 8, 1); mbar_init(bar_empty + s * 8, 1); }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }
  __syncthreads();
  const long long per = pieces / gridDim.x, rem = pieces % gridDim.x;
  const long long p0 = blockIdx.x * per + (blockIdx.x < rem ? blockIdx.x : rem), p1 = p0 + per + (blockIdx.x < rem ? 1 : 0);
  if (warp == 0) {
    const uint64_t policy = l2_policy_evict_first();
    int it = 0;
    bool ok = true;
    for (long long pc = p0; pc < p1 && ok; ++pc, ++it) {
      const int stage = it % kRing;
      ok = bounded_wait<false>(bar_empty + stage * 8, ((it / kRing) & 1) ^ 1, s_abort, kSpinLimit);
      if (ok && it >= kInFlight) ok = bounded_wait<false>(bar_full + ((it - kInFlight) % kRing) * 8, ((it - kInFlight) / kRing) & 1, s_abort, kSpinLimit);
      if (!ok) break;
      if (lane == 0) {
        mbar_arrive_expect_tx(bar_full + stage * 8, kPiece);
        bulk_g2s(ring + stage * kPiece, buf + pc * kPiece, kPiece, bar_full + stage * 8, policy);
      }
      __syncwarp();
    }
    for (int k = max(0, it - kRing); k < it; ++k) {   // nothing may be in flight when the block leaves
      uint32_t polls = 0;
      while (!mbar_try_wait(bar_full + (k % kRing) * 8, (k / kRing) & 1) && ++polls < kSpinLimit) __nanosleep(64);
    }
  } else {
    int it = 0, acc = 0;
    for (long long pc = p0; pc < p1; ++pc, ++it) {
      const int stage = it % kRing;
      if (!bounded_wait<false>(bar_full + stage * 8, (it / kRing) & 1, s_abort, kSpinLimit)) break;
      acc ^= reinterpret_cast<const int*>(smem + stage * kPiece)[lane];
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_empty + stage * 8);
    }
    if (acc == 0x7fffffff && sink) *sink = acc;   // keeps the read alive
  }
}

// ---------------------------------------------------------------- slow device reference
// grid (n, q_heads), one warp per block; lanes split head_dim.
__global__ void k_attn_reference(BcMeta m, BcGeom g, BcAttnArgs a) {
  const int i = blockIdx.x, h = blockIdx.y, lane = threadIdx.x;
  const int D = g.head_dim, G = g.q_heads / g.kv_heads, kvh = h / G;
  const int per = D / 32;  // elements per lane (2 or 4)
  const int slot = a.slots[i];
  int P = 0, nb = 0, w = 0;
  if (slot >= 0 && slot < m.max_seqs && m.open[slot]) { P = m.prompt_len[slot]; nb = m.n_beacons[slot]; w = m.window_len[slot]; }
  const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(a.q) + ((int64_t)i * g.q_heads + h) * D;
  float qv[4], acc[4] = {0.f, 0.f, 0.f, 0.f};
  for (int e = 0; e < per; ++e) qv[e] = __bfloat162float(q[lane * per + e]);
  float mrun = -INFINITY, lrun = 0.f;
  const int total = P + nb + w + (a.extra_k ? 1 : 0);
  for (int e = 0; e < total; ++e) {
    const __nv_bfloat16 *kp, *vp;
    int key = 0;  // XOR key of the chunk permutation (0 for the unstored extra entry)
    if (e < P + nb + w) {
      int pos, col0;
      if (e < P) { pos = e; col0 = 0; }
      else if (e < P + nb) { pos = e - P; col0 = m.beacon_off[slot]; }
      else { pos = e - P - nb; col0 = m.window_off[slot]; }
      const int page = m.page_table[(int64_t)slot * m.max_pages_per_seq + col0 + pos / g.page_size];
      const uint8_t* row = a.pool_layer + ((int64_t)page * g.page_size + pos % g.page_size) * g.entry_bytes;
      kp = reinterpret_cast<const __nv_bfloat16*>(row + kvh * g.head_row_bytes);
      vp = reinterpret_cast<const __nv_bfloat16*>(row + (g.kv_heads + kvh) * g.head_row_bytes);
      key = pos & 7;
    } else {
      kp = reinterpret_cast<const __nv_bfloat16*>(a.extra_k) + ((int64_t)i * g.kv_heads + kvh) * D;
      vp = reinterpret_cast<const __nv_bfloat16*>(a.extra_v) + ((int64_t)i * g.kv_heads + kvh) * D;
    }
    float dot = 0.f, vv[4];
    for (int x = 0; x < per; ++x) {
      const int d = lane * per + x;
      const int idx = (((d >> 3) ^ key) << 3) + (d & 7);
      dot += qv[x] * __bfloat162float(kp[idx]);
      vv[x] = __bfloat162float(vp[idx]);
    }
    for (int sft = 16; sft; sft >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, sft);
    const float sc = dot * a.sm_scale;
    const float mn = fmaxf(mrun, sc);
    const float al = expf(mrun - mn), pe = expf(sc - mn);
    lrun = lrun * al + pe;
    for (int x = 0; x < per; ++x) acc[x] = acc[x] * al + pe * vv[x];
    mrun = mn;
  }
  for (int x = 0; x < per; ++x) {
    const float val = lrun > 0.f ? acc[x] / lrun : 0.f;
    const int64_t o = ((int64_t)i * g.q_heads + h) * D + lane * per + x;
    if (a.out_f32) reinterpret_cast<float*>(a.out)[o] = val;
    else reinterpret_cast<__nv_bfloat16*>(a.out)[o] = __float2bfloat16_rn(val);
  }
}

FastDiv make_fast_div(uint32_t d) {
  FastDiv f;
  if (d <= 1) { f.mul = 0; f.sh1 = 0; f.sh2 = 0; return f; }
  uint32_t l = 0;
  while ((1ull << l) < d) ++l;  // ceil(log2 d)
  f.mul = (uint32_t)(((1ull << 32) * ((1ull << l) - d)) / d + 1);
  f.sh1 = 1;
  f.sh2 = l - 1;
  return f;
}

template <int D, bool G8, bool FUSED, bool PAIR = false, bool SHORTW = false, bool LAYERED = false>
cudaError_t launch_pipe(const PipeParams& p, cudaStream_t s) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.a.ctas, LAYERED ? p.a.layers : 1); cfg.blockDim = dim3(kPipeThreads); cfg.dynamicSmemBytes = PipeSmem<D>::kTotal; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;   // see the kernel: it waits for its predecessor after its plan
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, k_attn_pipe<D, G8, FUSED, PAIR, SHORTW, LAYERED>, p);
}

}  // namespace

namespace {
template <int D, bool G8, bool FUSED, bool PAIR = false, bool SHORTW = false, bool LAYERED = false>
cudaError_t opt_in_smem() {
  return cudaFuncSetAttribute(k_attn_pipe<D, G8, FUSED, PAIR, SHORTW, LAYERED>, cudaFuncAttributeMaxDynamicSharedMemorySize, PipeSmem<D>::kTotal);
}
}  // namespace

cudaError_t bc_attn_setup(int* sm_count) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(sm_count, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  const cudaError_t r[26] = {opt_in_smem<128, true, true, true>(), opt_in_smem<64, true, true, true>(),
                             opt_in_smem<128, true, false, true>(), opt_in_smem<64, true, false, true>(),
                             opt_in_smem<128, false, true, true>(), opt_in_smem<64, false, true, true>(),
                             opt_in_smem<128, true, false, false, false, true>(), opt_in_smem<128, false, false, false, false, true>(),
                             opt_in_smem<64, true, false, false, false, true>(), opt_in_smem<64, false, false, false, false, true>(),
                             opt_in_smem<128, true, true, false, false, true>(), opt_in_smem<128, false, true, false, false, true>(),
                             opt_in_smem<64, true, true, false, false, true>(), opt_in_smem<64, false, true, false, false, true>(),
                             opt_in_smem<128, true, false, false, true>(), opt_in_smem<128, true, true, false, true>(),
                             opt_in_smem<128, true, false>(), opt_in_smem<128, false, false>(), opt_in_smem<64, true, false>(),
                             opt_in_smem<64, false, false>(), opt_in_smem<128, true, true>(), opt_in_smem<128, false, true>(),
                             opt_in_smem<64, true, true>(), opt_in_smem<64, false, true>(),
                             opt_in_smem<128, false, false, true>(), opt_in_smem<64, false, false, true>()};
  for (cudaError_t x : r)
    if (x != cudaSuccess) return x;
  return cudaSuccess;
}

cudaError_t bc_launch_attn(const BcMeta& m, const BcGeom& g, const BcAttnArgs& a, const BcFusedAppend* fused, cudaStream_t s,
                           cudaEvent_t ev_start, cudaEvent_t ev_stop, int* launches) {
  PipeParams p;
  p.m = m; p.g = g; p.a = a;
  p.early_meta = (a.meta_settled && !fused) ? 1 : 0;
  p.timeline = reinterpret_cast<unsigned long long*>(a.timeline);
  p.spin_limit = a.spin_limit ? a.spin_limit : kSpinLimit;
  // a settable limit exists for head_dim 128 with groups of at most 8 query heads, plain and fused step
  const bool shortw = a.spin_limit != 0 && g.head_dim == 128 && g.q_heads / g.kv_heads <= 8 && a.q2 == nullptr;
  p.debug = a.debug;
  p.f = FusedArgs{};
  if (fused) {
    p.f.new_k = static_cast<const uint8_t*>(fused->new_k); p.f.new_v = static_cast<const uint8_t*>(fused->new_v);
    p.f.dst_row = fused->dst_row; p.f.dst_pos = fused->dst_pos; p.f.pool_w = fused->pool_layer;
    p.f.flag = fused->flag; p.f.epoch = fused->epoch; p.f.call = fused->call;
    p.f.plan = fused->plan;
  }
  p.scale_log2 = a.sm_scale * 1.4426950408889634f;
  p.n_groups = kConsumerWarps / g.kv_heads;
  p.rows_per_tile = 16 * p.n_groups;
  p.tile_shift = 0;
  while ((1 << p.tile_shift) < p.rows_per_tile) ++p.tile_shift;
  p.G = g.q_heads / g.kv_heads;
  p.div_ps = make_fast_div((uint32_t)g.page_size);
  cudaError_t e;
  if (ev_start) { e = cudaEventRecord(ev_start, s); if (e != cudaSuccess) return e; }
  const bool g8 = p.G <= 8;
  p.ls_pool = a.ls_pool; p.ls_q = a.ls_q; p.ls_out = a.ls_out; p.ls_kv = a.ls_kv; p.ls_part_o = a.ls_part_o;
  p.ls_part_ml = a.ls_part_ml; p.ls_tickets = a.ls_tickets;
  if (a.layers > 1) {      // every layer in this launch (no paired form, no settable wait limit, no timeline)
    if (a.q2 != nullptr) return cudaErrorInvalidValue;
    p.timeline = nullptr;
    if (fused) {
      if (g.head_dim == 128) e = g8 ? launch_pipe<128, true, true, false, false, true>(p, s) : launch_pipe<128, false, true, false, false, true>(p, s);
      else e = g8 ? launch_pipe<64, true, true, false, false, true>(p, s) : launch_pipe<64, false, true, false, false, true>(p, s);
    } else {
      if (g.head_dim == 128) e = g8 ? launch_pipe<128, true, false, false, false, true>(p, s) : launch_pipe<128, false, false, false, false, true>(p, s);
      else e = g8 ? launch_pipe<64, true, false, false, false, true>(p, s) : launch_pipe<64, false, false, false, false, true>(p, s);
    }
  } else if (a.q2 != nullptr) {   // the paired form (token and beacon queries in one pass); the caller has checked G <= 8
    const bool pack = 2 * p.G <= 8;   // both sets of heads fit the first 8 rows of a fragment
    if (pack) {
      if (fused) e = g.head_dim == 128 ? launch_pipe<128, true, true, true>(p, s) : launch_pipe<64, true, true, true>(p, s);
      else e = g.head_dim == 128 ? launch_pipe<128, true, false, true>(p, s) : launch_pipe<64, true, false, true>(p, s);
    } else if (fused) e = g.head_dim == 128 ? launch_pipe<128, false, true, true>(p, s) : launch_pipe<64, false, true, true>(p, s);
    else e = g.head_dim == 128 ? launch_pipe<128, false, false, true>(p, s) : launch_pipe<64, false, false, true>(p, s);
  } else if (shortw) {
    e = fused ? launch_pipe<128, true, true, false, true>(p, s) : launch_pipe<128, true, false, false, true>(p, s);
  } else if (fused) {
    if (g.head_dim == 128) e = g8 ? launch_pipe<128, true, true>(p, s) : launch_pipe<128, false, true>(p, s);
    else e = g8 ? launch_pipe<64, true, true>(p, s) : launch_pipe<64, false, true>(p, s);
  } else {
    if (g.head_dim == 128) e = g8 ? launch_pipe<128, true, false>(p, s) : launch_pipe<128, false, false>(p, s);
    else e = g8 ? launch_pipe<64, true, false>(p, s) : launch_pipe<64, false, false>(p, s);
  }
  if (e != cudaSuccess) return e;
  if (ev_stop) { e = cudaEventRecord(ev_stop, s); if (e != cudaSuccess) return e; }
  *launches = 1;
  return cudaSuccess;
}

cudaError_t bc_launch_read_stream(const void* buf, size_t bytes, int* sink, cudaStream_t s) {
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e == cudaSuccess) e = cudaFuncSetAttribute(k_read_stream, cudaFuncAttributeMaxDynamicSharedMemorySize, 3 * (64 << 10));
  if (e != cudaSuccess) return e;
  k_read_stream<<<sms, 64, 3 * (64 << 10), s>>>(static_cast<const uint8_t*>(buf), (long long)(bytes >> 16), sink);
  return cudaGetLastError();
}

cudaError_t bc_launch_attn_reference(const BcMeta& m, const BcGeom& g, const BcAttnArgs& a, cudaStream_t s) {
  k_attn_reference<<<dim3(a.n, g.q_heads), 32, 0, s>>>(m, g, a);
  return cudaGetLastError();
}
