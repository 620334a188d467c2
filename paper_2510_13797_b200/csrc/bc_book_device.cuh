// Device-side pieces of the bookkeeping that more than one kernel uses: the block-wide prefix sum,
// the first-error latch and the append step itself (one thread block, any size that is a multiple
// of 32).  Included inside each translation unit's unnamed namespace.
#pragma once

__device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Exclusive prefix sum of one int per thread over the block; *total gets the block sum.
// Must be called by all threads of the block.
__device__ int block_exclusive_scan(int x, int* total) {
  __shared__ int warp_sums[32];
  __shared__ int block_total;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = x;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += y;
  }
  __syncthreads();  // protects warp_sums / block_total of a previous call
  if (lane == 31) warp_sums[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int nw = (blockDim.x + 31) >> 5;
    int w = lane < nw ? warp_sums[lane] : 0;
    int wi = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, wi, d);
      if (lane >= d) wi += y;
    }
    warp_sums[lane] = wi - w;  // exclusive warp offsets
    if (lane == 31) block_total = wi;
  }
  __syncthreads();
  *total = block_total;
  return warp_sums[warp] + incl - x;
}

// The same over ONE warp, without shared memory (the one-warp form of the append bookkeeping).
__device__ __forceinline__ int warp_exclusive_scan(int x, int* total) {
  const int lane = threadIdx.x & 31;
  int incl = x;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int y = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += y;
  }
  *total = __shfl_sync(0xffffffffu, incl, 31);
  return incl - x;
}
template <bool WARP>
__device__ __forceinline__ int group_exclusive_scan(int x, int* total) {
  if constexpr (WARP) return warp_exclusive_scan(x, total);
  else return block_exclusive_scan(x, total);
}
template <bool WARP>
__device__ __forceinline__ void group_sync() {
  if constexpr (WARP) __syncwarp();
  else __syncthreads();
}

// ---- BC_FLAG_DEBUG_BOUNDS -------------------------------------------------------------------------
// Records a failed check (the offending value in the record's slot field) unless an error is latched
// already.  The caller skips or redirects the access; nothing traps.
__device__ __forceinline__ void debug_note(const BcMeta& m, int value) {
  if (atomicCAS(m.status, 0, BC_ERR_DEBUG_CHECK) == 0) m.status[1] = value;
}
// A page id read from the page table or the free stack: true if it lies in the pool.
__device__ __forceinline__ bool debug_page_ok(const BcMeta& m, int page) {
  if (!m.debug || (unsigned)page < (unsigned)m.num_pages) return true;
  debug_note(m, page);
  return false;
}
// A batch must not name a slot twice.  With the flag set every bookkeeping kernel (one thread block)
// first marks, per slot, the lowest batch index that names it in this call; an item that is not that
// one is refused with BC_ERR_DEBUG_CHECK, so the first occurrence goes through alone.
template <bool WARP = false>
__device__ void dup_prepass(const BcMeta& m, const int32_t* __restrict__ slots, int n, int64_t call) {
  if (!m.debug) return;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const int slot = slots[i];
    if (slot >= 0 && slot < m.max_seqs)
      atomicMax(m.dup_mark + slot, ((unsigned long long)call << 32) | (0xffffffffu - (unsigned)i));
  }
  group_sync<WARP>();
}
__device__ __forceinline__ bool is_dup(const BcMeta& m, int slot, int i, int64_t call) {
  return m.debug && m.dup_mark[slot] != (((unsigned long long)call << 32) | (0xffffffffu - (unsigned)i));
}

// Per-call error latch: the failing item with the lowest batch index reports, and only if no
// earlier call has latched an error.
struct ErrLatch {
  int* first_item;  // shared
  __device__ void init(int* sh) {
    first_item = sh;
    if (threadIdx.x == 0) *sh = 0x7fffffff;
    __syncthreads();
  }
  __device__ void note(int item) { atomicMin(first_item, item); }
  // all threads call; `item`/`code`/`slot` are this thread's failure (code == 0: none)
  __device__ void commit(const BcMeta& m, int item, int code, int slot, int64_t call) {
    __syncthreads();
    if (code != 0 && item == *first_item && m.status[0] == 0) {
      m.status[0] = code;
      m.status[1] = slot;
      *reinterpret_cast<int64_t*>(m.status + 2) = call;
    }
  }
};

// The append bookkeeping of one batch (Algorithm 1, sampling step), executed by ONE thread block:
// validates every item, allocates a window page where the window length is a multiple of the page
// size (block-wide prefix sum: deterministic page ids), bumps window_len and t, and writes for
// every item its pool row (dst_row; -1 if the item failed) and its position in the window
// (dst_pos).  The first failing item is latched.  Every thread of the block must call it.
// With `plan` non-NULL the block also leaves the decode-attention kernel's plan for this batch, as the
// lengths stand after the append (see BcPlan in bc_common.cuh): one coalesced read there instead of
// slots -> lengths -> prefix sum.
// WARP: the block is one warp; the same steps with shuffles and warp barriers and no shared memory.
template <bool WARP = false>
__device__ void append_book_block(const BcMeta& m, const int32_t* __restrict__ slots, int n, int64_t call, int32_t* dst_row,
                                  int32_t* dst_pos, int32_t* plan = nullptr, int tile_shift = 0) {
  ErrLatch latch;
  if constexpr (!WARP) {
    __shared__ int sh_first;
    latch.init(&sh_first);
  }
  dup_prepass<WARP>(m, slots, n, call);
  const int top0 = *m.free_top;
  const int ps = m.page_size;
  group_sync<WARP>();
  int base = 0, used = 0, my_code = 0, my_item = -1, my_slot = 0;
  for (int chunk = 0; chunk < n; chunk += blockDim.x) {
    const int i = chunk + threadIdx.x;
    int need = 0, slot = -1, w = 0, code = 0;
    bool valid = false;
    if (i < n) {
      slot = slots[i];
      if (slot < 0 || slot >= m.max_seqs || !m.open[slot]) code = BC_ERR_BAD_SLOT;
      else if (is_dup(m, slot, i, call)) code = BC_ERR_DEBUG_CHECK;
      else {
        const int c = m.c[slot], nb = m.n_beacons[slot];
        w = m.window_len[slot];
        if (c > 1 && w >= c) code = BC_ERR_WINDOW_FULL;
        else if (m.max_entries > 0 && nb + w + 1 > m.max_entries) code = BC_ERR_CAPACITY;
        else {
          need = (w % ps == 0) ? 1 : 0;
          const int pages = ceil_div(m.prompt_len[slot], ps) + ceil_div(nb, ps) + ceil_div(w, ps);
          if (need && pages + 1 > m.max_pages_per_seq) { code = BC_ERR_CAPACITY; need = 0; }
          else valid = true;
        }
      }
    }
    int total;
    const int off = base + group_exclusive_scan<WARP>(need, &total);
    base += total;
    int row_out = -1;
    if (valid) {
      if (need == 0 || off + need <= top0) {
        int32_t* col = m.page_table + (int64_t)slot * m.max_pages_per_seq + m.window_off[slot] + w / ps;
        if (need) { *col = m.free_stack[top0 - 1 - off]; used = max(used, off + 1); }
        if (debug_page_ok(m, *col)) {
          row_out = *col * ps + w % ps;
          m.window_len[slot] = w + 1;
          m.t[slot] += 1;
        }
      } else code = BC_ERR_NO_PAGES;
    }
    if (i < n) { dst_row[i] = row_out; dst_pos[i] = w; }
    if (code && my_code == 0) {
      my_code = code; my_item = i; my_slot = slot;
      if constexpr (!WARP) latch.note(i);
    }
  }
  used = __reduce_max_sync(0xffffffffu, used);
  if constexpr (WARP) {
    // the failing item with the lowest batch index reports, if no earlier call has latched an error
    const int first = __reduce_min_sync(0xffffffffu, my_code ? my_item : 0x7fffffff);
    if (my_code != 0 && my_item == first && m.status[0] == 0) {
      m.status[0] = my_code;
      m.status[1] = my_slot;
      *reinterpret_cast<int64_t*>(m.status + 2) = call;
    }
    __syncwarp();
    if (threadIdx.x == 0) *m.free_top = top0 - used;
  } else {
    __shared__ int sh_used;
    if (threadIdx.x == 0) sh_used = 0;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) atomicMax(&sh_used, used);
    latch.commit(m, my_item, my_code, my_slot, call);
    __syncthreads();
    if (threadIdx.x == 0) *m.free_top = top0 - sh_used;
  }
  if (plan != nullptr && n <= BC_MAX_ATTN_BATCH) {
    // every thread sees the block's own writes to the lengths after the barrier above
    const int T = 1 << tile_shift;
    int32_t* a = plan + BC_PLAN_HEADER;
    int carry = 0;
    for (int chunk = 0; chunk < n; chunk += blockDim.x) {
      const int i = chunk + threadIdx.x;
      int tiles = 0;
      if (i < n) {
        const int slot = slots[i];
        int P = 0, nb = 0, w = 0, bcol = 0, wcol = 0, sl = 0;
        if (slot >= 0 && slot < m.max_seqs && m.open[slot]) {
          P = m.prompt_len[slot]; nb = m.n_beacons[slot]; w = m.window_len[slot];
          bcol = m.beacon_off[slot]; wcol = m.window_off[slot]; sl = slot;
        }
        if (w > 0 && dst_row[i] >= 0) sl |= BC_PLAN_NEW_ROW;
        a[0 * BC_MAX_ATTN_BATCH + i] = P; a[1 * BC_MAX_ATTN_BATCH + i] = nb; a[2 * BC_MAX_ATTN_BATCH + i] = w;
        a[3 * BC_MAX_ATTN_BATCH + i] = sl; a[4 * BC_MAX_ATTN_BATCH + i] = bcol; a[5 * BC_MAX_ATTN_BATCH + i] = wcol;
        tiles = ((P + T - 1) >> tile_shift) + ((nb + T - 1) >> tile_shift) + ((w + T - 1) >> tile_shift);
        if (tiles == 0) tiles = 1;   // an empty sequence still owns one (empty) tile
      }
      int total;
      const int off = carry + group_exclusive_scan<WARP>(tiles, &total);
      if (i < n) a[6 * BC_MAX_ATTN_BATCH + i] = off;
      carry += total;
    }
    if (threadIdx.x == 0) { a[6 * BC_MAX_ATTN_BATCH + n] = carry; plan[0] = n; plan[1] = carry; plan[2] = tile_shift; }
  }
}
