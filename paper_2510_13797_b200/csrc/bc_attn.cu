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
//     unnormalised partial (m, l, O) and k_attn_combine merges the pieces.
//   * Every wait is bounded: on expiry the block records BC_ERR_TIMEOUT, stops issuing copies,
//     drains the copies already in flight (bounded) and returns.
//
// k_attn_reference is a slow, straightforward kernel (one warp per query head) kept as a
// debugging aid behind BC_FLAG_ATTN_REFERENCE.
#include "bc_common.cuh"

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kPipeThreads = (kConsumerWarps + 1) * 32;
constexpr int kPlanMax = BC_MAX_ATTN_BATCH;
constexpr uint32_t kSpinLimit = 1u << 21;  // polls of try_wait before giving up

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
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
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
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }

// Bounded wait; returns false when it gave up or another warp already aborted.
__device__ __forceinline__ bool bounded_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
  uint32_t polls = 0;
  while (!mbar_try_wait(bar, parity)) {
    if (++polls > 1024) __nanosleep(64);
    if (polls > kSpinLimit || *abort_flag) {
      *abort_flag = 1;
      return false;
    }
  }
  return true;
}

// ---------------------------------------------------------------- shared-memory plan
struct SeqInfo {
  int P, nb, w, Rb, Rw, slot;
};

struct PipeParams {
  BcMeta m;
  BcGeom g;
  BcAttnArgs a;
  float scale_log2;
  int rows_per_tile;  // T
  int n_groups;       // 8 / kv_heads
  int G;              // q_heads / kv_heads
};

template <int D>
struct PipeSmem {
  static constexpr int kStageBytes = 512 * D;  // T * E, independent of kv_heads
  static constexpr int kStages = D == 128 ? 3 : 6;
  static constexpr int kRingBytes = kStageBytes * kStages;
  static constexpr int kMergeOff = kRingBytes;
  static constexpr int kMergeMlOff = kMergeOff + BC_MERGE_ELEMS * 4;
  static constexpr int kPlanOff = kMergeMlOff + 64 * 2 * 4;  // up to 64 query heads
  // plan arrays: P, nb, w, slot [kPlanMax] and cum [kPlanMax + 1]
  static constexpr int kBarOff = kPlanOff + (4 * kPlanMax + kPlanMax + 8) * 4;
  static constexpr int kAbortOff = kBarOff + 2 * kStages * 8;
  static constexpr int kTotal = kAbortOff + 16;
};

template <int D, bool G_LE_8>
__global__ void __launch_bounds__(kPipeThreads, 1) k_attn_pipe(const PipeParams p) {
  using L = PipeSmem<D>;
  constexpr int NSTAGE = L::kStages;
  constexpr int KSTEPS = D / 16;  // k-steps of QK^T
  constexpr int NT = D / 8;       // n-tiles of PV
  extern __shared__ __align__(1024) uint8_t smem[];

  float* merge_o = reinterpret_cast<float*>(smem + L::kMergeOff);
  float* merge_ml = reinterpret_cast<float*>(smem + L::kMergeMlOff);
  int* s_P = reinterpret_cast<int*>(smem + L::kPlanOff);
  int* s_nb = s_P + kPlanMax;
  int* s_w = s_nb + kPlanMax;
  int* s_slot = s_w + kPlanMax;
  int* s_cum = s_slot + kPlanMax;  // [n + 1] exclusive prefix sums of tiles
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + L::kAbortOff);
  const uint32_t ring = smem_u32(smem);
  const uint32_t bar_full = smem_u32(smem + L::kBarOff);
  const uint32_t bar_empty = bar_full + NSTAGE * 8;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n = p.a.n, T = p.rows_per_tile, E = p.g.entry_bytes, ps = p.g.page_size;
  const int Hkv = p.g.kv_heads, Hq = p.g.q_heads, G = p.G;

  if (tid == 0) {
    for (int s = 0; s < NSTAGE; ++s) {
      mbar_init(bar_full + s * 8, 1);
      mbar_init(bar_empty + s * 8, kConsumerWarps);
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async();
  }

  // ---- plan: tiles per sequence, prefix sums, this block's span --------------------------------
  for (int i = tid; i < n; i += kPipeThreads) {
    const int slot = p.a.slots[i];
    int P = 0, nb = 0, w = 0;
    if (slot >= 0 && slot < p.m.max_seqs && p.m.open[slot]) {
      P = p.m.prompt_len[slot]; nb = p.m.n_beacons[slot]; w = p.m.window_len[slot];
    }
    s_P[i] = P; s_nb[i] = nb; s_w[i] = w; s_slot[i] = slot;
    const int Rb = (P + 7) & ~7, Rw = (Rb + nb + 7) & ~7;
    const int rows = Rw + w;
    s_cum[i + 1] = rows > 0 ? (rows + T - 1) / T : 1;  // an empty sequence still owns one tile
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
  const int total_tiles = s_cum[n];
  const int per = total_tiles / (int)gridDim.x, rem = total_tiles % (int)gridDim.x;
  const int cta = blockIdx.x;
  const int g0 = cta * per + min(cta, rem);
  const int g1 = g0 + per + (cta < rem ? 1 : 0);
  if (g0 >= g1) return;
  int seq0 = 0;
  {  // largest i with cum[i] <= g0
    int lo = 0, hi = n;
    while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (s_cum[mid] <= g0) lo = mid; else hi = mid; }
    seq0 = lo;
  }

  auto seq_info = [&](int i) {
    SeqInfo s;
    s.P = s_P[i]; s.nb = s_nb[i]; s.w = s_w[i]; s.slot = s_slot[i];
    s.Rb = (s.P + 7) & ~7; s.Rw = (s.Rb + s.nb + 7) & ~7;
    return s;
  };

  if (warp == kConsumerWarps) {
    // ================================ producer warp ============================================
    int i = seq0;
    SeqInfo si = seq_info(i);
    int it = 0;
    bool aborted = false;
    for (int gt = g0; gt < g1; ++gt, ++it) {
      while (gt >= s_cum[i + 1]) { ++i; si = seq_info(i); }
      const int t = gt - s_cum[i];
      const int stage = it % NSTAGE;
      const uint32_t full = bar_full + stage * 8, empty = bar_empty + stage * 8;
      if (!aborted && !bounded_wait(empty, ((it / NSTAGE) & 1) ^ 1, s_abort)) aborted = true;
      if (aborted) continue;
      const int v0 = t * T, v1 = v0 + T;
      const int seg_start[3] = {0, si.Rb, si.Rw};
      const int seg_len[3] = {si.P, si.nb, si.w};
      int rows = 0;
#pragma unroll
      for (int sgi = 0; sgi < 3; ++sgi) {
        const int a = max(v0, seg_start[sgi]), b = min(v1, seg_start[sgi] + seg_len[sgi]);
        rows += max(b - a, 0);
      }
      if (lane == 0) {
        if (rows > 0) mbar_arrive_expect_tx(full, (uint32_t)rows * (uint32_t)E);
        else mbar_arrive(full);
      }
      __syncwarp();
      if (rows > 0) {
        const int32_t* row_tab = p.m.page_table + (int64_t)si.slot * p.m.max_pages_per_seq;
        const int seg_col[3] = {0, p.m.beacon_off[si.slot], p.m.window_off[si.slot]};
        const uint32_t stage_base = ring + stage * L::kStageBytes;
#pragma unroll
        for (int sgi = 0; sgi < 3; ++sgi) {
          const int a = max(v0, seg_start[sgi]), b = min(v1, seg_start[sgi] + seg_len[sgi]);
          if (a >= b) continue;
          const int p0 = a - seg_start[sgi], p1 = b - seg_start[sgi];
          const int pg_last = (p1 - 1) / ps;
          for (int pg = p0 / ps + lane; pg <= pg_last; pg += 32) {
            const int lo = max(p0, pg * ps), hi = min(p1, (pg + 1) * ps);
            const int page = row_tab[seg_col[sgi] + pg];
            const uint8_t* src = p.a.pool_layer + ((int64_t)page * ps + (lo - pg * ps)) * E;
            const uint32_t dst = stage_base + (uint32_t)(seg_start[sgi] + lo - v0) * (uint32_t)E;
            bulk_g2s(dst, src, (uint32_t)(hi - lo) * (uint32_t)E, full);
          }
        }
      }
    }
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
  const int kvh = warp % Hkv, grp = warp / Hkv;
  const int gq = lane >> 2, qd = lane & 3;  // fragment row and column-pair index
  // ldmatrix lane offsets inside this warp's 16 rows of a stage
  const int lm = lane >> 3, lr = lane & 7;
  const uint32_t k_lane_off = (uint32_t)((((lm >> 1) << 3) + lr) * E + kvh * p.g.head_row_bytes);
  const int k_chunk_sel = lm & 1;
  const uint32_t v_lane_off = (uint32_t)((((lm & 1) << 3) + lr) * E + (Hkv + kvh) * p.g.head_row_bytes);
  const int v_chunk_sel = lm >> 1;
  const uint32_t warp_rows_off = (uint32_t)(grp * 16) * (uint32_t)E;

  int i = seq0;
  int it = 0;
  int gt = g0;
  while (gt < g1) {
    while (gt >= s_cum[i + 1]) ++i;
    const SeqInfo si = seq_info(i);
    const int tiles_i = s_cum[i + 1] - s_cum[i];
    const int ta = gt - s_cum[i];
    const int tb = min(tiles_i, ta + (g1 - gt));
    const bool whole = (ta == 0 && tb == tiles_i);

    // ---- query fragments: rows = the G query heads of this KV head -----------------------------
    uint32_t qf[KSTEPS][4];
    {
      const __nv_bfloat16* qb = reinterpret_cast<const __nv_bfloat16*>(p.a.q) + ((int64_t)i * Hq + kvh * G) * D;
#pragma unroll
      for (int kk = 0; kk < KSTEPS; ++kk) {
        const int d0 = kk * 16 + qd * 2;
        qf[kk][0] = gq < G ? *reinterpret_cast<const uint32_t*>(qb + gq * D + d0) : 0u;
        qf[kk][2] = gq < G ? *reinterpret_cast<const uint32_t*>(qb + gq * D + d0 + 8) : 0u;
        if (G_LE_8) { qf[kk][1] = 0u; qf[kk][3] = 0u; }
        else {
          qf[kk][1] = gq + 8 < G ? *reinterpret_cast<const uint32_t*>(qb + (gq + 8) * D + d0) : 0u;
          qf[kk][3] = gq + 8 < G ? *reinterpret_cast<const uint32_t*>(qb + (gq + 8) * D + d0 + 8) : 0u;
        }
      }
    }
    float o[NT][4];
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { o[nt][0] = o[nt][1] = o[nt][2] = o[nt][3] = 0.f; }
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;

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
      const bool r0 = gq < G, r1 = !G_LE_8 && (gq + 8 < G);
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
      const bool ok = __all_sync(0xffffffffu, bounded_wait(bar_full + stage * 8, (it / NSTAGE) & 1, s_abort));
      if (!ok && lane == 0 && p.m.status[0] == 0) { p.m.status[0] = BC_ERR_TIMEOUT; p.m.status[1] = -1; }
      const int vrow0 = t * T + grp * 16;  // virtual row of this warp's first row
      // valid rows among my 16
      int cnt = 0;
      {
        const int a0 = max(vrow0, 0), b0 = min(vrow0 + 16, si.P);
        const int a1 = max(vrow0, si.Rb), b1 = min(vrow0 + 16, si.Rb + si.nb);
        const int a2 = max(vrow0, si.Rw), b2 = min(vrow0 + 16, si.Rw + si.w);
        cnt = max(b0 - a0, 0) + max(b1 - a1, 0) + max(b2 - a2, 0);
      }
      bool wrote_smem = false;
      if (ok && cnt > 0) {
        const uint32_t rows_base = ring + stage * L::kStageBytes + warp_rows_off;
        auto row_valid = [&](int v) {
          return (v < si.P) || (v >= si.Rb && v < si.Rb + si.nb) || (v >= si.Rw && v < si.Rw + si.w);
        };
        if (cnt < 16) {
          // rows nobody copied may hold anything: zero their V so that 0 * garbage cannot be NaN
          uint8_t* rows_ptr = smem + stage * L::kStageBytes + warp_rows_off;
          for (int r = 0; r < 16; ++r) {
            if (!row_valid(vrow0 + r) && lane < (p.g.head_row_bytes >> 4))
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
              if (!row_valid(vrow0 + j * 8 + qd * 2 + e)) { s[j][e] = -INFINITY; s[j][e + 2] = -INFINITY; }
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
    l0 += __shfl_xor_sync(0xffffffffu, l0, 1); l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
    if (!G_LE_8) { l1 += __shfl_xor_sync(0xffffffffu, l1, 1); l1 += __shfl_xor_sync(0xffffffffu, l1, 2); }
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
    {
      const int ctid = tid;  // 0..255 among consumers
      if (whole) {
        for (int idx = ctid; idx < Hq * D; idx += kConsumerWarps * 32) {
          const int h = idx / D;
          const float l = merge_ml[h * 2 + 1];
          const float val = l > 0.f ? merge_o[idx] / l : 0.f;
          if (p.a.out_f32) reinterpret_cast<float*>(p.a.out)[(int64_t)i * Hq * D + idx] = val;
          else reinterpret_cast<__nv_bfloat16*>(p.a.out)[(int64_t)i * Hq * D + idx] = __float2bfloat16_rn(val);
        }
      } else {
        const int64_t pslot = (int64_t)cta + i;
        float* po = p.a.part_o + pslot * Hq * D;
        for (int idx = ctid; idx < Hq * D; idx += kConsumerWarps * 32) po[idx] = merge_o[idx];
        if (ctid < Hq * 2) p.a.part_ml[pslot * Hq * 2 + ctid] = merge_ml[ctid];
      }
      if (ctid == 0) {
        if (ta == 0) p.a.first_cta[i] = cta;
        if (tb == tiles_i) p.a.last_cta[i] = cta;
      }
    }
    consumer_bar();  // the merge buffer is reused by the next piece
  }
}

// Merges the pieces of every sequence that was split over several blocks.
__global__ void k_attn_combine(BcAttnArgs a, int Hq, int D) {
  const int i = blockIdx.x;
  const int first = a.first_cta[i], last = a.last_cta[i];
  if (first == last) return;  // written directly by the attention kernel
  for (int idx = threadIdx.x; idx < Hq * D; idx += blockDim.x) {
    const int h = idx / D;
    float mmax = -INFINITY;
    for (int c = first; c <= last; ++c) mmax = fmaxf(mmax, a.part_ml[((int64_t)(c + i) * Hq + h) * 2]);
    const float msafe = mmax == -INFINITY ? 0.f : mmax;
    float num = 0.f, den = 0.f;
    for (int c = first; c <= last; ++c) {
      const int64_t ps = (int64_t)(c + i);
      const float sc = exp2f(a.part_ml[(ps * Hq + h) * 2] - msafe);
      num += sc * a.part_o[ps * Hq * D + idx];
      den += sc * a.part_ml[(ps * Hq + h) * 2 + 1];
    }
    const float val = den > 0.f ? num / den : 0.f;
    if (a.out_f32) reinterpret_cast<float*>(a.out)[(int64_t)i * Hq * D + idx] = val;
    else reinterpret_cast<__nv_bfloat16*>(a.out)[(int64_t)i * Hq * D + idx] = __float2bfloat16_rn(val);
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

template <int D, bool G8>
cudaError_t launch_pipe(const PipeParams& p, cudaStream_t s) {
  k_attn_pipe<D, G8><<<p.a.ctas, kPipeThreads, PipeSmem<D>::kTotal, s>>>(p);
  return cudaGetLastError();
}

}  // namespace

cudaError_t bc_attn_setup(int* sm_count) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(sm_count, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_attn_pipe<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PipeSmem<128>::kTotal);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_attn_pipe<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PipeSmem<128>::kTotal);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(k_attn_pipe<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, PipeSmem<64>::kTotal);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(k_attn_pipe<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, PipeSmem<64>::kTotal);
}

cudaError_t bc_launch_attn(const BcMeta& m, const BcGeom& g, const BcAttnArgs& a, cudaStream_t s, cudaEvent_t ev_start,
                           cudaEvent_t ev_stop, int* launches) {
  PipeParams p;
  p.m = m; p.g = g; p.a = a;
  p.scale_log2 = a.sm_scale * 1.4426950408889634f;
  p.n_groups = kConsumerWarps / g.kv_heads;
  p.rows_per_tile = 16 * p.n_groups;
  p.G = g.q_heads / g.kv_heads;
  cudaError_t e;
  if (ev_start) { e = cudaEventRecord(ev_start, s); if (e != cudaSuccess) return e; }
  const bool g8 = p.G <= 8;
  if (g.head_dim == 128) e = g8 ? launch_pipe<128, true>(p, s) : launch_pipe<128, false>(p, s);
  else e = g8 ? launch_pipe<64, true>(p, s) : launch_pipe<64, false>(p, s);
  if (e != cudaSuccess) return e;
  if (ev_stop) { e = cudaEventRecord(ev_stop, s); if (e != cudaSuccess) return e; }
  k_attn_combine<<<a.n, 256, 0, s>>>(a, g.q_heads, g.head_dim);
  *launches = 2;
  return cudaGetLastError();
}

cudaError_t bc_launch_attn_reference(const BcMeta& m, const BcGeom& g, const BcAttnArgs& a, cudaStream_t s) {
  k_attn_reference<<<dim3(a.n, g.q_heads), 32, 0, s>>>(m, g, a);
  return cudaGetLastError();
}
