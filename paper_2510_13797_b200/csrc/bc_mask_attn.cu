// Mask-form (teacher-forced) attention forward: the dense formulation of Figure 2 / Section 3.2.
//
// During training the eviction is simulated by an attention mask over the whole trajectory: a
// generated token sees the prompt, every earlier beacon, and the tokens of its own window up to
// itself; the beacon that closes a window sees the prompt, the earlier beacons, that window and
// itself.  This file computes those rows for a batch of trajectories in one pass -- the other side
// of the cache that the decode path maintains step by step (same results, Section 3.2).
//
// Unlike decode this is a dense contraction, so it runs on the tcgen05 tensor cores:
//   * one work item per (query tile, KV head): 128 query rows = floor(128/G) tokens (or beacons) times
//     the G query heads that share the KV head, so a K/V tile is reused by G heads;
//   * per key tile of 128 keys:  S = Q K^T  (tcgen05.mma, M = N = K = 128, fp32 in tensor memory)
//     -> tcgen05.ld, mask, online softmax in fp32 registers, P as bf16 back into tensor memory
//     -> O += P V  (second tcgen05.mma, P read from tensor memory, accumulating in tensor memory; the
//        rows are rescaled in place, by tcgen05.ld / tcgen05.st, only when their reference maximum has
//        to be raised);
//   * operands live in shared memory in the 128-byte-swizzled layouts the MMA descriptors describe,
//     written by tiled tensor copies (cp.async.bulk.tensor, 128-byte swizzle, completion on an
//     mbarrier) issued by one thread: Q and K row by row (K-major), V as it is stored, keys by rows
//     (N-major B operand), so nothing is transposed or staged;
//   * key tiles a query tile cannot see are skipped: all prompt tiles, the beacon tiles up to its
//     last visible beacon, and the token tiles that overlap its own windows;
//   * the kernel is persistent: two blocks per SM walk the work items (sequence by sequence, heaviest
//     first, dealt out in alternating direction), keep their tensor memory and barriers, and request the next item's
//     first tiles while the current item's output is still being written.
// K and V rows past the end of a sequence belong to the next sequence (or read as zero past the end
// of the array): their scores are overwritten with -inf, their weights are exactly zero, and their V
// rows are cleared in shared memory before the second product, so whatever a neighbouring sequence
// holds (infinities, NaNs) cannot reach this sequence's rows.  Every wait is bounded; on expiry the block records BC_ERR_TIMEOUT, releases
// its tensor memory and returns.
#include <cuda.h>

#include <algorithm>
#include <vector>

#include "bc_common.cuh"

namespace {

constexpr int kTile = 128;        // query rows and keys per tile
constexpr int kD = 128;           // head_dim
constexpr int kRowThreads = 128;   // one per query row
constexpr int kThreads = kRowThreads + 32;   // plus the control warp
constexpr int kOperandBytes = kTile * kD * 2;  // 32 KB: one bf16 operand tile
constexpr uint32_t kWaitLimit = 1u << 20;  // polls of a bounded wait (about 0.1 s) before a block gives up

struct TileDesc {
  int32_t kind;        // 0: token rows, 1: beacon rows
  int32_t first;       // first token / beacon (0-based, inside the sequence) of the tile
  int32_t count;       // tokens / beacons in the tile
  int32_t P, T, nb;    // lengths of the sequence
  int32_t prompt_row, tok_row, bea_row;  // first row of the sequence in the packed inputs
  int32_t pad[7];
};

// The key tiles one query tile walks: nt0 prompt tiles, nt1 beacon tiles, nt2 token tiles starting at
// token lo2 (a multiple of 128).
struct TilePlan {
  int32_t nt0, nt1, nt2, lo2, N;
};
__host__ __device__ inline TilePlan make_plan(const TileDesc& td, int c) {
  const int last = td.first + td.count - 1;
  const int bmax = td.kind == 0 ? (c > 1 ? last / c : 0) : last + 1;           // beacons [0, bmax)
  const int tlo = td.kind == 0 ? (c > 1 ? (td.first / c) * c : 0) : td.first * c;
  const int thi = td.kind == 0 ? last + 1 : (last + 1) * c;                      // tokens [tlo, thi)
  TilePlan p;
  p.lo2 = (tlo / kTile) * kTile;
  p.nt0 = (td.P + kTile - 1) / kTile;
  p.nt1 = (bmax + kTile - 1) / kTile;
  p.nt2 = thi > p.lo2 ? (thi - p.lo2 + kTile - 1) / kTile : 0;
  p.N = p.nt0 + p.nt1 + p.nt2;
  return p;
}
// tile n -> segment (0 prompt, 1 beacons, 2 tokens) and first key of the tile inside the segment
__device__ __forceinline__ int plan_kind(const TilePlan& p, int n) { return n < p.nt0 ? 0 : (n < p.nt0 + p.nt1 ? 1 : 2); }
__device__ __forceinline__ int plan_k0(const TilePlan& p, int n, int kind) {
  return kind == 0 ? n * kTile : (kind == 1 ? (n - p.nt0) * kTile : p.lo2 + (n - p.nt0 - p.nt1) * kTile);
}

// Tensor maps (bf16, [rows][heads][128] seen as (d, head, row), 128-byte swizzle): q boxes of
// (64, G, tokens per tile); k and v boxes of (64, 1, 128).
struct MaskMaps {
  CUtensorMap q_tok, q_bea, k_prompt, k_tok, k_bea, v_prompt, v_tok, v_bea;
};

struct MaskArgs {
  const TileDesc* tiles;   // sequence by sequence, heaviest query tiles of a sequence first
  int32_t n_items;         // tiles x kv_heads; item i = (tile i / kv_heads, head i % kv_heads)
  __nv_bfloat16 *out_tok, *out_bea;
  int32_t* status;     // device int: first error code
  int32_t Hq, Hkv, G, c, rows_per_tile;  // rows_per_tile = tokens per query tile = 128 / G
  float scale_log2;
  uint32_t wait_limit;   // polls after which a wait gives up (kWaitLimit unless bc_mask_attn_set_wait_limit lowered it)
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Byte offset of 16-byte chunk `ch16` (0..15 = 8 elements each) of row r in a 128 x 128 bf16 operand
// tile stored K-major with 128-byte swizzling: two blocks of 64 elements, each 128 rows of 128 bytes,
// the chunk index inside a row XOR-ed with the row number modulo 8.
__device__ __forceinline__ uint32_t swz(int r, int ch16) {
  return (uint32_t)((ch16 >> 3) * (kTile * 128) + r * 128 + (((ch16 & 7) ^ (r & 7)) << 4));
}

// Tiled tensor copies global -> shared memory, completing on an mbarrier.  The innermost coordinate
// is a multiple of 64 bf16 elements (128 bytes) in every call.
__device__ __forceinline__ void tma_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];" ::"r"(dst),
      "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void st_zero16(uint32_t dst) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(dst), "r"(0) : "memory");
}

// Shared-memory matrix descriptor: K-major, 128-byte swizzle, 8-row groups 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3ffff) >> 4);   // start address
  d |= (uint64_t)0 << 16;                    // leading byte offset: unused for swizzled K-major
  d |= (uint64_t)(1024 >> 4) << 32;          // stride byte offset between 8-row groups
  d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                    // 128-byte swizzle
  return d;
}
// The same for an N-major B operand (V as stored: 128 keys by rows of 128 bytes = 64 head dimensions,
// the other 64 dimensions 16 KB further): 8-key groups 1024 bytes apart along K, the two 64-wide
// halves of N kLeadBytes apart.
__device__ __forceinline__ uint64_t umma_desc_nmajor(uint32_t saddr) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3ffff) >> 4);
  d |= (uint64_t)((kTile * 128) >> 4) << 16;  // leading byte offset: next 64 elements of N
  d |= (uint64_t)(1024 >> 4) << 32;           // stride byte offset: next 8 keys
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = 128.
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTile >> 3) << 17) | ((uint32_t)(kTile >> 4) << 24);

constexpr uint32_t kIdescBN = kIdesc | (1u << 16);   // B operand N-major
__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t a, uint64_t b, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(a), "l"(b), "r"(kIdesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 consecutive columns of this thread's row; the registers are valid after tmem_wait_ld().
__device__ __forceinline__ void tmem_ld32_async(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const float (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};" ::"r"(taddr),
      "r"(__float_as_uint(v[0])), "r"(__float_as_uint(v[1])), "r"(__float_as_uint(v[2])), "r"(__float_as_uint(v[3])),
      "r"(__float_as_uint(v[4])), "r"(__float_as_uint(v[5])), "r"(__float_as_uint(v[6])), "r"(__float_as_uint(v[7])),
      "r"(__float_as_uint(v[8])), "r"(__float_as_uint(v[9])), "r"(__float_as_uint(v[10])), "r"(__float_as_uint(v[11])),
      "r"(__float_as_uint(v[12])), "r"(__float_as_uint(v[13])), "r"(__float_as_uint(v[14])), "r"(__float_as_uint(v[15])),
      "r"(__float_as_uint(v[16])), "r"(__float_as_uint(v[17])), "r"(__float_as_uint(v[18])), "r"(__float_as_uint(v[19])),
      "r"(__float_as_uint(v[20])), "r"(__float_as_uint(v[21])), "r"(__float_as_uint(v[22])), "r"(__float_as_uint(v[23])),
      "r"(__float_as_uint(v[24])), "r"(__float_as_uint(v[25])), "r"(__float_as_uint(v[26])), "r"(__float_as_uint(v[27])),
      "r"(__float_as_uint(v[28])), "r"(__float_as_uint(v[29])), "r"(__float_as_uint(v[30])), "r"(__float_as_uint(v[31]))
      : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// tcgen05.mma with the A operand in tensor memory (the softmax weights) and B in shared memory.
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t b, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(tmem_d),
      "r"(tmem_a), "l"(b), "r"(kIdescBN), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
      "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ bool elect_one() {   // true in exactly one lane of a converged warp
  uint32_t pred;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ void mbar_arrive_cta(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait that also gives up as soon as another thread of the block has reported a failure.  The
// ordinary instantiation has a compile-time limit (with a run-time limit the polling loops cost a
// third of the kernel's throughput); the settable limit of bc_mask_attn_set_wait_limit lives in an
// instantiation of its own (SHORTW), where limits below 1024 poll with the non-suspending test_wait.
template <bool SHORTW>
__device__ __forceinline__ bool mbar_wait_or_fail(uint32_t bar, uint32_t parity, volatile int* fail, uint32_t limit_arg) {
  if (SHORTW && limit_arg < 1024) {
    for (uint32_t polls = 0; polls < limit_arg; ++polls) {
      uint32_t ok;
      asm volatile(
          "{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
          : "=r"(ok)
          : "r"(bar), "r"(parity)
          : "memory");
      if (ok) return true;
    }
    return false;
  }
  const uint32_t limit = SHORTW ? limit_arg : kWaitLimit;
  for (uint32_t polls = 0; polls < limit; ++polls) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if ((polls & 63) == 63 && *fail) return false;
    if (polls > 4096) __nanosleep(128);
  }
  return false;
}

// Roles: warps 0..3 own the 128 query rows (one row per thread: mask, softmax, rescaling, output);
// warp 4 is the control warp, whose first lane issues every tensor copy and every product.
//
// Per key tile n (K_n, V_n):   S = Q K_n^T   ->  [rows] P_n = weights(S), bf16, written over S in
// tensor memory   ->   O += P_n V_n (A operand from tensor memory).  The control thread keeps the copy
// engine one tile ahead: K_{n+1} is requested as soon as S_n exists (the K buffer is free), V_{n+1} as
// soon as O += P_n V_n has completed (the V buffer is free), so their latency hides behind the softmax
// and the products; the products of the block's neighbour on the SM fill the tensor pipe meanwhile.
// Q K_{n+1}^T overwrites P_n; it is issued right behind P_n V_n, and the tensor pipe, which runs one
// block's products in issue order, starts it only when P_n has been read.  The tile stream runs
// on across work items: after an item's last S the next item's Q and first K are requested, and its
// first product into O waits until the rows have read the finished O.
//
// Barriers (single-phase mbarriers; t counts key tiles, e work items, parity = count & 1):
//   bar_k: the block's first Q and K have landed
//   bar_in: V of tile t and K of tile t + 1 (with Q, at the start of an item) have landed: two arrivals per
//           tile, the two requests, or a plain arrival in place of the K request after the block's last tile
//   bar_s: completion t = S of tile t is ready (and every earlier product has finished)
//   bar_p: the 128 row threads have stored P of tile t                bar_o: P V of a tile has completed
//   bar_f: completion e = O of item e is final                       bar_e: the rows have read O of item e
template <bool SHORTW>
__global__ void __launch_bounds__(kThreads, 2) k_mask_attn(const MaskArgs a, const __grid_constant__ MaskMaps maps) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sQ = smem_addr(smem), sK = sQ + kOperandBytes, sV = sK + kOperandBytes;
  __shared__ __align__(8) uint64_t s_bars[8];
  __shared__ uint32_t s_tmem;
  __shared__ int s_fail_word;
  volatile int* s_fail = &s_fail_word;
  const uint32_t bar_k = smem_addr(&s_bars[0]), bar_in = bar_k + 8, bar_s = bar_k + 16, bar_p = bar_k + 24, bar_o = bar_k + 32,
                 bar_f = bar_k + 40, bar_e = bar_k + 48, bar_d = bar_k + 56;   // bar_d: drain of the products on the give-up path
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = a.G, Hq = a.Hq, Hkv = a.Hkv, c = a.c;

  if (tid == 0) {
    const uint32_t counts[8] = {1, 2, 1, (uint32_t)kRowThreads, 1, 1, (uint32_t)kRowThreads, 1};   // bar_in: two arrivals per tile
    for (int i = 0; i < 8; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar_k + i * 8), "r"(counts[i]) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    *s_fail = 0;
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_addr(&s_tmem)), "r"(256) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // Rows of the Q buffer that no tensor copy writes (only when G does not divide 128) stay zero.
  const int box_rows = a.rows_per_tile * G;
  for (int idx = tid; idx < (kTile - box_rows) * 16; idx += kThreads) {
    const int r = box_rows + (idx >> 4), ch = idx & 15;
    st_zero16(sQ + swz(r, ch));
  }
  proxy_fence();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = s_tmem;
  const uint32_t tS = tmem, tO = tmem + kTile;   // columns [0,128): S, then P in its first 64; [128,256): O
  const uint32_t tP = tS;

  // Work items of this block: round r hands out items [r * grid, (r + 1) * grid), forwards in even
  // rounds and backwards in odd ones, so that the heavy and the light end of the sorted list meet.
  const int grid = (int)gridDim.x, bid = (int)blockIdx.x;
  auto item_of = [&](int r) {
    const int it = r * grid + ((r & 1) ? grid - 1 - bid : bid);
    return it < a.n_items ? it : -1;
  };

  if (warp == kRowThreads / 32) {
    // ======================================= control warp ===========================================
    // All 32 lanes walk the loop and the waits together, so that loop state and the matrix descriptors
    // are warp-uniform; one elected lane issues the copies and the products.
    int item = item_of(0);
    if (item >= 0) {
      auto issue_q = [&](const TileDesc& td, int kvh, uint32_t bar) {
        // rows of Q beyond the tile's tokens belong to the next sequence or are zero-filled: they are never
        // visible (their outputs are not written and they contribute to no other row)
        const CUtensorMap* qm = td.kind == 0 ? &maps.q_tok : &maps.q_bea;
        const int qrow = (td.kind == 0 ? td.tok_row : td.bea_row) + td.first;
        tma_3d(sQ, qm, 0, kvh * G, qrow, bar);
        tma_3d(sQ + kTile * 128, qm, 64, kvh * G, qrow, bar);
      };
      auto issue_k = [&](const TileDesc& td, const TilePlan& pl, int kvh, int n, uint32_t bar) {
        const int kind = plan_kind(pl, n), k0 = plan_k0(pl, n, kind);
        const CUtensorMap* km = kind == 0 ? &maps.k_prompt : (kind == 1 ? &maps.k_bea : &maps.k_tok);
        const int row = (kind == 0 ? td.prompt_row : (kind == 1 ? td.bea_row : td.tok_row)) + k0;
        tma_3d(sK, km, 0, kvh, row, bar);
        tma_3d(sK + kTile * 128, km, 64, kvh, row, bar);
      };
      auto issue_v = [&](const TileDesc& td, const TilePlan& pl, int kvh, int n) {
        const int kind = plan_kind(pl, n), k0 = plan_k0(pl, n, kind);
        const CUtensorMap* vm = kind == 0 ? &maps.v_prompt : (kind == 1 ? &maps.v_bea : &maps.v_tok);
        const int row = (kind == 0 ? td.prompt_row : (kind == 1 ? td.bea_row : td.tok_row)) + k0;
        mbar_expect_tx(bar_in, (uint32_t)kOperandBytes);
        tma_3d(sV, vm, 0, kvh, row, bar_in);
        tma_3d(sV + kTile * 128, vm, 64, kvh, row, bar_in);
      };
      const uint64_t dQ = umma_desc(sQ), dK = umma_desc(sK), dV = umma_desc_nmajor(sV);
      auto qk = [&]() {   // descriptor start addresses advance in 16-byte units
#pragma unroll
        for (int kk = 0; kk < kD / 16; ++kk) {
          const uint64_t off = (uint64_t)(((kk >> 2) * (kTile * 128) + (kk & 3) * 32) >> 4);
          umma(tS, dQ + off, dK + off, kk > 0);
        }
      };
      // Every lane polls (one warp-wide instruction on one address) and a vote joins the answers.  Barrier
      // polls and shuffles go through the same queue as the special-function instructions the rows keep it
      // full of, so each costs this warp a couple of hundred cycles: a poll by one lane followed by a
      // shuffle of its answer would be two of them per wait.
      auto wait_all = [&](uint32_t bar, uint32_t parity) {
        const bool ok1 = mbar_wait_or_fail<SHORTW>(bar, parity, s_fail, a.wait_limit);
        return __all_sync(0xffffffffu, ok1);
      };
      const uint32_t q_bytes = (uint32_t)(box_rows * kD * 2);
      TileDesc td = a.tiles[item / Hkv];
      int kvh = item % Hkv;
      TilePlan pl = make_plan(td, c);
      if (elect_one()) {
        mbar_expect_tx(bar_k, q_bytes + (uint32_t)kOperandBytes);   // the first Q and K: a barrier of their own
        issue_q(td, kvh, bar_k);
        issue_k(td, pl, kvh, 0, bar_k);
        issue_v(td, pl, kvh, 0);
      }
      __syncwarp();
      // for the give-up path (what is still in flight): the first copies not seen to land; the number of
      // bar_in completions begun (tile t is completion t: V_t, then K_{t+1} or a plain arrival); whether the
      // last one begun still lacks its second arrival
      bool first_out = true, in_open = true, products_issued = false;
      uint32_t n_in = 1;
      uint32_t ph_o = 0, t = 0, e = 0;
      bool ok = wait_all(bar_k, 0);
      if (ok) first_out = false;
      if (ok) {
        products_issued = true;
        tc_fence_after();
        if (elect_one()) { qk(); umma_commit(bar_s); }
        __syncwarp();
      }
      for (int r = 0; ok; ++r, ++e) {
        const int nitem = item_of(r + 1);
        TileDesc ntd = td;
        TilePlan npl = pl;
        int nkvh = 0;
        if (nitem >= 0) { ntd = a.tiles[nitem / Hkv]; nkvh = nitem % Hkv; npl = make_plan(ntd, c); }
        for (int n = 0; n < pl.N && ok; ++n, ++t) {
          ok = wait_all(bar_s, t & 1u);                                        // S exists: the K buffer is free
          if (!ok) break;
          const bool last = n + 1 == pl.N;
          const bool more = !last || nitem >= 0;                               // another tile follows, here or in the next item
          // the second arrival of this tile's bar_in completion (the first was the request of V_t): the
          // request of the next K, or a plain arrival where no tile follows
          if (elect_one()) {
            if (!more) mbar_arrive_cta(bar_in);
            else if (!last) {
              mbar_expect_tx(bar_in, (uint32_t)kOperandBytes);
              issue_k(td, pl, kvh, n + 1, bar_in);
            } else {                                                           // ... and so is the Q buffer
              mbar_expect_tx(bar_in, q_bytes + (uint32_t)kOperandBytes);
              issue_q(ntd, nkvh, bar_in);
              issue_k(ntd, npl, nkvh, 0, bar_in);
            }
          }
          __syncwarp();
          in_open = false;
          // everything the products below need besides P is waited for while the rows are busy: V_t and
          // K_{t+1} (with its Q) have landed -- one barrier, one wait
          ok = wait_all(bar_in, t & 1u);
          if (ok) {
            // A key tile that reaches past its segment has loaded rows that are not this sequence's (the
            // next sequence's, or zeros past the end of the array).  Their scores are overwritten with -inf
            // and their weights are exactly 0, but 0 * inf would still poison the second product: the V
            // rows past the segment's end are cleared here, by this warp, before the product is issued
            // (partial tiles only; the row threads' code is untouched).
            const int kind = plan_kind(pl, n), k0 = plan_k0(pl, n, kind);
            const int seg_len = kind == 0 ? td.P : (kind == 1 ? td.nb : td.T);
            const int nvalid = min(max(seg_len - k0, 0), kTile);
            if (nvalid < kTile) {
              for (int idx = nvalid * 16 + lane; idx < kTile * 16; idx += 32) st_zero16(sV + swz(idx >> 4, idx & 15));
              proxy_fence();   // the product reads shared memory through the asynchronous proxy
              __syncwarp();
            }
          }
          if (ok && n == 0 && e > 0) ok = wait_all(bar_e, (e - 1) & 1u);       // the rows have read the last O
          ok = ok && wait_all(bar_p, t & 1u);
          if (!ok) break;
          tc_fence_after();
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < kTile / 16; ++kk)                             // O += P V, 16 keys at a time
              umma_ts(tO, tP + (uint32_t)(kk * 8), dV + (uint64_t)((kk * 16 * 128) >> 4), (n > 0 || kk > 0) ? 1u : 0u);
            if (last) umma_commit(bar_f);
            if (more) {
              umma_commit(bar_o);
              // The next S overwrites P: the tensor pipe runs one block's products in the order they were
              // issued, so it starts only after the product above has read P.
              qk();
              umma_commit(bar_s);
            }
          }
          __syncwarp();
          if (more) {
            ok = wait_all(bar_o, ph_o);                                         // the V buffer is free
            ph_o ^= 1;
            if (!ok) break;
            if (elect_one()) { if (!last) issue_v(td, pl, kvh, n + 1); else issue_v(ntd, npl, nkvh, 0); }
            in_open = true; ++n_in;
            __syncwarp();
          }
        }
        if (nitem < 0) break;
        td = ntd; pl = npl; kvh = nkvh;
      }
      if (!ok) {
        // Giving up: nothing may still be on its way into this block's shared or tensor memory when the block
        // leaves.  Wait, with the full limit, for the tensor copies that were requested and not yet seen to
        // land, and for every product issued so far (one more commit arrives when all of them are done).
        *s_fail = 1;
        __syncwarp();
        if (elect_one()) {   // the lane that issued the copies and the products
          int never = 0;
          if (in_open) mbar_arrive_cta(bar_in);   // a completion with only its first arrival gets its second one
          if (first_out) mbar_wait_or_fail<false>(bar_k, 0, &never, kWaitLimit);
          mbar_wait_or_fail<false>(bar_in, (n_in - 1) & 1u, &never, kWaitLimit);
          if (products_issued) {
            umma_commit(bar_d);
            mbar_wait_or_fail<false>(bar_d, 0, &never, kWaitLimit);
          }
        }
      }
    }
    __syncwarp();
  } else {
    // ========================================= row threads ==========================================
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;      // this warp's 32 lanes of tensor memory
    const int my_local = tid / G, my_head = tid % G;              // token / beacon inside the tile, head inside the group
    // The output accumulator stays in tensor memory for a whole item: the second product adds to it,
    // and it is rescaled in place only when the row's reference maximum moves.  The reference follows
    // the true maximum lazily: it is raised only when a tile exceeds it by more than kMaxSlack (in the
    // log2 domain), so the softmax weights relative to it stay below 2^kMaxSlack -- exact in the end,
    // because numerator and denominator share the reference.
    constexpr float kMaxSlack = 8.f;
    bool failed = false;
    uint32_t t = 0, e = 0;
    int item = item_of(0);
    TileDesc td = {};
    if (item >= 0) td = a.tiles[item / Hkv];
    // tcgen05.ld / tcgen05.st are warp-wide instructions: every lane executes them, whatever its row
    // can see, and every branch around them is warp-uniform, so that no transformation of the code
    // can split a warp between two copies of one of them.
    for (int r = 0; item >= 0 && !failed; ++r, ++e) {
      const int kvh = item % Hkv;
      const TilePlan pl = make_plan(td, c);
      const bool row_valid = tid < td.count * G;
      const int my_idx = td.first + my_local;       // token index i, or beacon index (0-based; beacon number my_idx + 1)
      int vis_beacons, tok_lo, tok_hi;              // visible: beacons [0, vis_beacons), tokens [tok_lo, tok_hi)
      if (td.kind == 0) { vis_beacons = c > 1 ? my_idx / c : 0; tok_lo = c > 1 ? (my_idx / c) * c : 0; tok_hi = my_idx + 1; }
      else { vis_beacons = my_idx + 1; tok_lo = my_idx * c; tok_hi = (my_idx + 1) * c; }
      float m_ref = -INFINITY, l_run = 0.f;

      for (int n = 0; n < pl.N; ++n, ++t) {
        const bool ok = mbar_wait_or_fail<SHORTW>(bar_s, t & 1u, s_fail, a.wait_limit);
        if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
        tc_fence_after();
        const int kind = plan_kind(pl, n), k0 = plan_k0(pl, n, kind);
        // The keys of this segment the row may see form one interval [vlo, vhi); j indexes the tile.
        int vlo, vhi;
        if (kind == 0) { vlo = 0; vhi = td.P; }
        else if (kind == 1) { vlo = 0; vhi = min(vis_beacons, td.nb); }
        else { vlo = tok_lo; vhi = min(tok_hi, td.T); }
        if (!row_valid) vhi = vlo;
        const int jlo = max(vlo - k0, 0), jhi = min(vhi - k0, kTile);   // visible columns of the tile
        const bool all_visible = __all_sync(0xffffffffu, jlo == 0 && jhi == kTile);
        float s[kTile];
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) tmem_ld32_async(tS + lane_base + cb * 32, s + cb * 32);
        tmem_wait_ld();
        if (!all_visible) {   // partial tile: hide what the row cannot see (warp-uniform branch, no tensor-memory access inside)
#pragma unroll
          for (int j = 0; j < kTile; ++j)
            if (j < jlo || j >= jhi) s[j] = -INFINITY;
        }
        // four independent chains each for the maximum and the sum: a single chain of 128 dependent
        // operations would cost more than the exponentials
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int j = 0; j < kTile; j += 8) {   // three-input maxima: two elements per instruction
          mx[0] = max3(mx[0], s[j], s[j + 1]); mx[1] = max3(mx[1], s[j + 2], s[j + 3]);
          mx[2] = max3(mx[2], s[j + 4], s[j + 5]); mx[3] = max3(mx[3], s[j + 6], s[j + 7]);
        }
        const float tile_max = fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])) * a.scale_log2;   // the scale is positive
        float alpha = 1.f;
        const bool raise = tile_max > m_ref + kMaxSlack || (m_ref == -INFINITY && tile_max > -INFINITY);
        if (raise) {
          alpha = fast_exp2(m_ref - tile_max);   // 0 when nothing had been seen yet
          m_ref = tile_max;
          l_run *= alpha;
        }
        const float m_safe = m_ref == -INFINITY ? 0.f : m_ref;   // hidden entries: exp2(-inf) = 0
        float sum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int cb = 0; cb < 4; ++cb) {
          uint32_t pk[16];
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const float p0 = fast_exp2(fmaf(s[cb * 32 + j], a.scale_log2, -m_safe));
            const float p1 = fast_exp2(fmaf(s[cb * 32 + j + 1], a.scale_log2, -m_safe));
            sum[(j >> 1) & 3] += p0 + p1;
            const __nv_bfloat162 pb = __floats2bfloat162_rn(p0, p1);   // key 2q in the low half of column q
            pk[j >> 1] = *reinterpret_cast<const uint32_t*>(&pb);
          }
          tmem_st16(tP + lane_base + cb * 16, pk);   // all of S is in registers already
        }
        l_run += (sum[0] + sum[1]) + (sum[2] + sum[3]);
        // ---- rescale the accumulator rows whose reference moved (whole warp, if any lane needs it); every
        //      earlier product has finished, or this tile's S would not exist --------------------------------
        if (n > 0 && __any_sync(0xffffffffu, raise)) {
#pragma unroll 1
          for (int cb = 0; cb < 4; ++cb) {
            float u[32];
            tmem_ld32_async(tO + lane_base + cb * 32, u);
            tmem_wait_ld();
#pragma unroll
            for (int j = 0; j < 32; ++j) u[j] *= alpha;
            tmem_st32(tO + lane_base + cb * 32, u);
          }
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive_cta(bar_p);
      }
      if (failed) break;

      // ---- the item's output: read the accumulator, hand it back, write the rows ----------------------
      const int nitem = item_of(r + 1);
      TileDesc ntd = {};
      if (nitem >= 0) ntd = a.tiles[nitem / Hkv];   // in flight during the wait below
      const bool ok = mbar_wait_or_fail<SHORTW>(bar_f, e & 1u, s_fail, a.wait_limit);
      if (!__all_sync(0xffffffffu, ok)) { failed = true; break; }
      tc_fence_after();
      float o[kD];
#pragma unroll
      for (int cb = 0; cb < 4; ++cb) tmem_ld32_async(tO + lane_base + cb * 32, o + cb * 32);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive_cta(bar_e);
      if (row_valid) {
        const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
        __nv_bfloat16* dst = (td.kind == 0 ? a.out_tok + (int64_t)(td.tok_row + my_idx) * Hq * kD
                                           : a.out_bea + (int64_t)(td.bea_row + my_idx) * Hq * kD) +
                             (int64_t)(kvh * G + my_head) * kD;
        auto pack = [&](int d) {
          const __nv_bfloat162 t = __floats2bfloat162_rn(o[d] * inv, o[d + 1] * inv);
          return *reinterpret_cast<const uint32_t*>(&t);
        };
        // 32-byte stores: whole sectors, half as many store instructions as with 16-byte ones (the rows
        // of a warp lie 256 bytes or more apart, so nothing coalesces across lanes)
#pragma unroll
        for (int d = 0; d < kD; d += 16)
          asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst + d), "r"(pack(d)), "r"(pack(d + 2)),
                       "r"(pack(d + 4)), "r"(pack(d + 6)), "r"(pack(d + 8)), "r"(pack(d + 10)), "r"(pack(d + 12)), "r"(pack(d + 14))
                       : "memory");
      }
      item = nitem;
      td = ntd;
    }
    if (failed) *s_fail = 1;
  }
  tc_fence_before();
  __syncthreads();
  if (*s_fail && tid == 0) atomicCAS(a.status, 0, BC_ERR_TIMEOUT);
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(256) : "memory");
  }
}

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link against the driver library).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}
// [rows][heads][128] bf16 seen as (d, head, row); box (64, box_heads, box_rows); out-of-range elements read as zero
bool map_3d(CUtensorMap* m, const void* base, int heads, int64_t rows, int box_heads, int box_rows) {
  const cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)heads, (cuuint64_t)(rows > 0 ? rows : 1)};
  const cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)heads * kD * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows}, es[3] = {1, 1, 1};
  return encode_tiled()(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, es,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
struct MaskLayout {
  size_t tiles, status, total;
  int64_t n_tiles;
};

// Upper bound from the totals alone (every sequence may add one partial tile of each kind).
MaskLayout mask_layout(int n_seqs, int q_heads, int kv_heads, int64_t total_tokens, int64_t total_beacons) {
  MaskLayout l;
  const int G = q_heads / kv_heads, per = kTile / G;
  l.n_tiles = (total_tokens + per - 1) / per + (total_beacons + per - 1) / per + 2 * (int64_t)n_seqs;
  size_t o = 0;
  auto take = [&](size_t b) { size_t at = o; o = align_up(o + b, 256); return at; };
  l.tiles = take((size_t)l.n_tiles * sizeof(TileDesc));
  l.status = take(256);
  l.total = o;
  return l;
}

uint32_t g_mask_wait_limit = 0;   // bc_mask_attn_set_wait_limit (0: kWaitLimit)

int sm_count() {
  static int n = 0;
  if (!n) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) n = 148;
  }
  return n;
}

}  // namespace

extern "C" {

bc_status bc_mask_attn_query_bytes(int32_t n_seqs, int32_t q_heads, int32_t kv_heads, int32_t head_dim,
                                   int64_t total_prompt, int64_t total_tokens, int64_t total_beacons,
                                   size_t* workspace_bytes) {
  if (!workspace_bytes || n_seqs < 1 || kv_heads < 1 || q_heads < 1 || q_heads % kv_heads || total_prompt < 0 ||
      total_tokens < 0 || total_beacons < 0)
    return BC_ERR_INVALID_ARG;
  if (head_dim != kD || q_heads / kv_heads > 16) return BC_ERR_UNSUPPORTED;
  *workspace_bytes = mask_layout(n_seqs, q_heads, kv_heads, total_tokens, total_beacons).total;
  return BC_OK;
}

bc_status bc_mask_attn_forward(int32_t n_seqs, int32_t q_heads, int32_t kv_heads, int32_t head_dim, int32_t c,
                               const int32_t* cu_prompt, const int32_t* cu_tokens, const void* prompt_k,
                               const void* prompt_v, const void* tok_q, const void* tok_k, const void* tok_v,
                               const void* beacon_q, const void* beacon_k, const void* beacon_v, void* out_tok,
                               void* out_beacon, float sm_scale, void* workspace, size_t workspace_bytes,
                               void* stream) {
  if (n_seqs < 1 || !cu_prompt || !cu_tokens || c < 1 || kv_heads < 1 || q_heads < 1 || q_heads % kv_heads || !workspace)
    return BC_ERR_INVALID_ARG;
  if (head_dim != kD || q_heads / kv_heads > 16) return BC_ERR_UNSUPPORTED;
  if (reinterpret_cast<uintptr_t>(workspace) & 255) return BC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(out_tok) | reinterpret_cast<uintptr_t>(out_beacon)) & 31) return BC_ERR_INVALID_ARG;   // 32-byte stores
  if (!(sm_scale > 0.f)) return BC_ERR_INVALID_ARG;  // the kernel takes row maxima before scaling
  const int G = q_heads / kv_heads, per = kTile / G;
  int64_t total_prompt = cu_prompt[n_seqs], total_tokens = cu_tokens[n_seqs], total_beacons = 0;
  for (int i = 0; i < n_seqs; ++i) {
    if (cu_prompt[i + 1] < cu_prompt[i] || cu_tokens[i + 1] < cu_tokens[i]) return BC_ERR_INVALID_ARG;
    total_beacons += c > 1 ? (cu_tokens[i + 1] - cu_tokens[i]) / c : 0;
  }
  if ((total_prompt && (!prompt_k || !prompt_v)) || (total_tokens && (!tok_q || !tok_k || !tok_v || !out_tok)) ||
      (total_beacons && (!beacon_q || !beacon_k || !beacon_v || !out_beacon)))
    return BC_ERR_INVALID_ARG;
  const MaskLayout l = mask_layout(n_seqs, q_heads, kv_heads, total_tokens, total_beacons);
  if (workspace_bytes < l.total) return BC_ERR_INVALID_ARG;
  cudaStream_t s = (cudaStream_t)stream;
  uint8_t* ws = static_cast<uint8_t*>(workspace);

  // host side: the query tiles, heaviest (most key tiles) first
  std::vector<TileDesc> tiles;
  int64_t bea_row = 0;
  for (int i = 0; i < n_seqs; ++i) {
    const int P = cu_prompt[i + 1] - cu_prompt[i], T = cu_tokens[i + 1] - cu_tokens[i], nb = c > 1 ? T / c : 0;
    TileDesc td = {};
    td.P = P; td.T = T; td.nb = nb;
    td.prompt_row = cu_prompt[i]; td.tok_row = cu_tokens[i]; td.bea_row = (int32_t)bea_row;
    for (int f = 0; f < T; f += per) { td.kind = 0; td.first = f; td.count = T - f < per ? T - f : per; tiles.push_back(td); }
    for (int f = 0; f < nb; f += per) { td.kind = 1; td.first = f; td.count = nb - f < per ? nb - f : per; tiles.push_back(td); }
    bea_row += nb;
  }
  if ((int64_t)tiles.size() > l.n_tiles) return BC_ERR_INVALID_ARG;
  if (tiles.empty()) return BC_OK;
  if ((int64_t)tiles.size() * kv_heads > 0x7fffffff) return BC_ERR_UNSUPPORTED;
  // Long sequences first; inside a sequence the query tiles with the most key tiles first.  The blocks
  // running at any moment then share one or two sequences' K and V in L2, and the last rounds are light.
  std::stable_sort(tiles.begin(), tiles.end(), [c](const TileDesc& x, const TileDesc& y) {
    const int64_t lx = (int64_t)x.P + x.T, ly = (int64_t)y.P + y.T;
    if (lx != ly) return lx > ly;
    if (x.tok_row != y.tok_row) return x.tok_row < y.tok_row;
    return make_plan(x, c).N > make_plan(y, c).N;
  });
  cudaError_t e = cudaMemcpyAsync(ws + l.tiles, tiles.data(), tiles.size() * sizeof(TileDesc), cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemsetAsync(ws + l.status, 0, 4, s);
  // the copy above reads pageable host memory: it has been staged when the call returns
  if (e != cudaSuccess) return BC_ERR_CUDA;

  MaskArgs a;
  a.tiles = reinterpret_cast<const TileDesc*>(ws + l.tiles);
  a.n_items = (int32_t)tiles.size() * kv_heads;
  a.out_tok = (__nv_bfloat16*)out_tok; a.out_bea = (__nv_bfloat16*)out_beacon;
  a.status = reinterpret_cast<int32_t*>(ws + l.status);
  a.Hq = q_heads; a.Hkv = kv_heads; a.G = G; a.c = c; a.rows_per_tile = per;
  a.scale_log2 = sm_scale * 1.4426950408889634f;
  a.wait_limit = g_mask_wait_limit ? g_mask_wait_limit : kWaitLimit;
  const int smem_bytes = 3 * kOperandBytes + 1024;
  const bool shortw = g_mask_wait_limit != 0;
  if (cudaFuncSetAttribute(shortw ? k_mask_attn<true> : k_mask_attn<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes) != cudaSuccess)
    return BC_ERR_CUDA;
  if (!encode_tiled()) return BC_ERR_CUDA;
  MaskMaps maps;
  const void* dummy = ws;   // arrays that do not exist (no prompt, no beacons) get a map that is never used
  bool ok = map_3d(&maps.q_tok, tok_q ? tok_q : dummy, q_heads, total_tokens, G, per) &&
            map_3d(&maps.q_bea, beacon_q ? beacon_q : dummy, q_heads, total_beacons, G, per) &&
            map_3d(&maps.k_prompt, prompt_k ? prompt_k : dummy, kv_heads, total_prompt, 1, kTile) &&
            map_3d(&maps.k_tok, tok_k ? tok_k : dummy, kv_heads, total_tokens, 1, kTile) &&
            map_3d(&maps.k_bea, beacon_k ? beacon_k : dummy, kv_heads, total_beacons, 1, kTile) &&
            map_3d(&maps.v_prompt, prompt_v ? prompt_v : dummy, kv_heads, total_prompt, 1, kTile) &&
            map_3d(&maps.v_tok, tok_v ? tok_v : dummy, kv_heads, total_tokens, 1, kTile) &&
            map_3d(&maps.v_bea, beacon_v ? beacon_v : dummy, kv_heads, total_beacons, 1, kTile);
  if (!ok) return BC_ERR_CUDA;
  const int grid = a.n_items < 2 * sm_count() ? a.n_items : 2 * sm_count();   // two resident blocks per SM
  if (shortw) k_mask_attn<true><<<grid, kThreads, smem_bytes, s>>>(a, maps);
  else k_mask_attn<false><<<grid, kThreads, smem_bytes, s>>>(a, maps);
  return cudaGetLastError() == cudaSuccess ? BC_OK : BC_ERR_CUDA;
}

bc_status bc_mask_attn_set_wait_limit(uint32_t polls) {
  g_mask_wait_limit = polls;
  return BC_OK;
}

bc_status bc_mask_attn_status(const void* workspace, int32_t n_seqs, int32_t q_heads, int32_t kv_heads,
                              int64_t total_prompt, int64_t total_tokens, int64_t total_beacons, void* stream,
                              int32_t* code) {
  if (!workspace || !code) return BC_ERR_INVALID_ARG;
  const MaskLayout l = mask_layout(n_seqs, q_heads, kv_heads, total_tokens, total_beacons);
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return BC_ERR_CUDA;
  if (cudaMemcpy(code, static_cast<const uint8_t*>(workspace) + l.status, 4, cudaMemcpyDeviceToHost) != cudaSuccess) return BC_ERR_CUDA;
  return BC_OK;
}

}  // extern "C"
