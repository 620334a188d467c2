// Bookkeeping and data-movement kernels of the paged store: reset, open, append, compress/evict,
// close, prefill copy, single-row writes, export.
//
// Every bookkeeping kernel runs as ONE thread block so that page allocation is a prefix sum over
// the batch and page ownership is a pure function of the call sequence (the discipline stated in
// breadcrumbs.h).  The amount of work is a few integers per sequence.
#include "bc_common.cuh"

namespace {

constexpr int kBookThreads = 1024;

#include "bc_book_device.cuh"

// Copies the K and V rows of n batch items into their pool rows with the whole block, 16 bytes
// per thread and step, applying the chunk permutation of the store layout.  Items with
// dst_row < 0 (failed validation) are skipped.  Used by the single-block kernels that have just
// computed dst_row/dst_pos (their global writes are visible to the block after __syncthreads).
__device__ void block_write_rows(const BcMeta& m, const BcGeom& g, uint8_t* __restrict__ pool_layer, const int32_t* dst_row,
                                 const int32_t* dst_pos, const uint8_t* __restrict__ k,
                                 const uint8_t* __restrict__ v, int n) {
  const int chunks_per_head = g.head_row_bytes >> 4;
  const int per_side = g.kv_heads * chunks_per_head;
  const int per_item = 2 * per_side;
  for (int idx = threadIdx.x; idx < n * per_item; idx += blockDim.x) {
    const int i = idx / per_item, r = idx - i * per_item;
    const int row = dst_row[i];
    if (row < 0) continue;
    if (m.debug && row >= m.num_pages * g.page_size) { debug_note(m, row); continue; }
    const int which = r / per_side, rem = r - which * per_side;
    const int h = rem / chunks_per_head, j = rem - h * chunks_per_head;
    const uint8_t* src = (which ? v : k) + ((int64_t)i * g.kv_heads + h) * g.head_row_bytes + (j << 4);
    *reinterpret_cast<uint4*>(pool_layer + (int64_t)row * g.entry_bytes + bc_chunk_offset(g, which, h, j, dst_pos[i])) =
        *reinterpret_cast<const uint4*>(src);
  }
}

__global__ void k_init(BcMeta m) {
  const int tid = blockIdx.x * blockDim.x + threadIdx.x, nth = gridDim.x * blockDim.x;
  for (int i = tid; i < m.num_pages; i += nth) m.free_stack[i] = m.num_pages - 1 - i;
  for (int i = tid; i < m.max_seqs; i += nth) {
    m.open[i] = 0; m.prompt_len[i] = 0; m.n_beacons[i] = 0; m.window_len[i] = 0;
    m.c[i] = 0; m.t[i] = 0; m.window_off[i] = 0; m.beacon_off[i] = 0;
    m.dup_mark[i] = 0ull;
  }
  if (tid == 0) {
    *m.free_top = m.num_pages;
    m.status[0] = 0; m.status[1] = 0; m.status[2] = 0; m.status[3] = 0;
  }
}

__global__ void __launch_bounds__(kBookThreads, 1)
k_open(BcMeta m, const int32_t* __restrict__ slots, const int32_t* __restrict__ plens,
       const int32_t* __restrict__ cs, int n, int64_t call) {
  __shared__ int sh_first;
  ErrLatch latch; latch.init(&sh_first);
  dup_prepass(m, slots, n, call);
  const int top0 = *m.free_top;
  __syncthreads();
  int base = 0, used = 0, my_code = 0, my_item = -1, my_slot = 0;
  for (int chunk = 0; chunk < n; chunk += blockDim.x) {
    const int i = chunk + threadIdx.x;
    int need = 0, slot = -1, P = 0, c = 0, code = 0;
    bool valid = false;
    if (i < n) {
      slot = slots[i]; P = plens[i]; c = cs ? cs[i] : m.c_default;
      if (slot < 0 || slot >= m.max_seqs || m.open[slot]) code = BC_ERR_BAD_SLOT;
      else if (is_dup(m, slot, i, call)) code = BC_ERR_DEBUG_CHECK;
      else if (c < 1 || P < 0) code = BC_ERR_INVALID_ARG;
      else {
        need = ceil_div(P, m.page_size);
        const int nwp = c > 1 ? ceil_div(c, m.page_size) : 0;
        if (need + nwp > m.max_pages_per_seq) { code = BC_ERR_CAPACITY; need = 0; }
        else valid = true;
      }
    }
    int total;
    const int off = base + block_exclusive_scan(need, &total);
    base += total;
    if (valid) {
      if (need == 0 || off + need <= top0) {
        int32_t* row = m.page_table + (int64_t)slot * m.max_pages_per_seq;
        for (int k = 0; k < need; ++k) row[k] = m.free_stack[top0 - 1 - off - k];
        if (need) used = max(used, off + need);
        m.open[slot] = 1; m.prompt_len[slot] = P; m.n_beacons[slot] = 0; m.window_len[slot] = 0;
        m.c[slot] = c; m.t[slot] = 0; m.window_off[slot] = need;
        m.beacon_off[slot] = need + (c > 1 ? ceil_div(c, m.page_size) : 0);
      } else code = BC_ERR_NO_PAGES;
    }
    if (code && my_code == 0) { my_code = code; my_item = i; my_slot = slot; latch.note(i); }
  }
  used = __reduce_max_sync(0xffffffffu, used);
  __shared__ int sh_used;
  if (threadIdx.x == 0) sh_used = 0;
  __syncthreads();
  if ((threadIdx.x & 31) == 0) atomicMax(&sh_used, used);
  latch.commit(m, my_item, my_code, my_slot, call);
  __syncthreads();
  if (threadIdx.x == 0) *m.free_top = top0 - sh_used;
}

// Last statement of a bookkeeping kernel that may have started before the kernel ahead of it in the
// stream had finished (programmatic stream serialisation): it ends only when that kernel has ended,
// so that whatever is enqueued next -- above all the kernels that write K/V rows, possibly into pages
// a compression has just recycled -- comes after BOTH, as plain stream order would have it.  Returns
// at once when nothing was overtaken.
__device__ __forceinline__ void wait_for_overtaken_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// WARP: launched as ONE warp, and then without a byte of shared memory.  The attention kernel's blocks hold an
// SM's shared memory but for the kilobyte every block is charged, and nearly all registers of two of its four
// sub-partitions; a one-warp block without shared memory still finds room beside such a block (measured), a
// block of several warps or with shared memory of its own does not and has to wait for the first SM the
// attention kernel leaves.  So the bookkeeping of a small batch begins as soon as the attention kernel ahead
// has let its dependents go, and the next attention launch finds its plan and its flag waiting.
template <bool WARP>
__global__ void __launch_bounds__(WARP ? 32 : kBookThreads, 1)
k_append_book(BcMeta m, const int32_t* __restrict__ slots, int n, int64_t call,
              int32_t* dst_row, int32_t* dst_pos, BcGeom g, uint8_t* pool_layer, const uint8_t* k, const uint8_t* v,
              int32_t* plan, int32_t* flag, int32_t epoch, BcHostSync hs) {
  // With a plan to leave, this is the bookkeeping of a fused decode step, and the kernel enqueued behind it
  // is that step's attention kernel.  Its blocks may take their places on the SMs now; what they read of
  // this kernel's results they read after the flag below (release here, acquire there), and everything the
  // kernel ahead of this one may still be writing only after this kernel has ended.
  if (plan != nullptr) {
    // The flag word still holds an older epoch -- possibly this very one, when a captured step is replayed.
    // It is cleared, and the clearing made visible device-wide, before any block of the dependent kernel
    // can exist.
    if (threadIdx.x == 0) { *reinterpret_cast<volatile int32_t*>(flag) = 0; __threadfence(); }
    group_sync<WARP>();
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
  int tile_shift = 4;   // rows per tile of the attention kernel: 16 * (8 / kv_heads)
  while ((16 << (tile_shift - 4)) * g.kv_heads < 128) ++tile_shift;
  append_book_block<WARP>(m, slots, n, call, dst_row, dst_pos, plan, tile_shift);
  group_sync<WARP>();
  if (plan != nullptr && threadIdx.x == 0) {   // lengths, page-table column, row destinations and plan are written
    // A host-buffer step: q, k, v travel on the cache's copy stream, which writes the step's number to a word
    // behind the copy (a stream memory operation, not a kernel).  The flag below lets the attention kernel read
    // those inputs, so it is published only once the word shows this step; the caller's stream then needs no
    // wait for the copy between this kernel and the attention kernel.  If the word does not show up within the
    // limit the step is reported (BC_ERR_TIMEOUT) and no flag is published.
    bool inputs_in = true;
    if (hs.in_word != nullptr) {
      inputs_in = false;
      for (uint32_t polls = 0; polls < (1u << 21); ++polls) {
        int seen, seen2 = hs.in_seq;
        asm volatile("ld.acquire.sys.global.s32 %0, [%1];" : "=r"(seen) : "l"(hs.in_word) : "memory");
        if (hs.in_word2 != nullptr) asm volatile("ld.acquire.sys.global.s32 %0, [%1];" : "=r"(seen2) : "l"(hs.in_word2) : "memory");
        if (seen == hs.in_seq && seen2 == hs.in_seq) { inputs_in = true; break; }
        __nanosleep(100);
      }
      if (!inputs_in && m.status[0] == 0) {
        m.status[0] = BC_ERR_TIMEOUT; m.status[1] = -1;
        *reinterpret_cast<int64_t*>(m.status + 2) = call;
      }
    }
    if (inputs_in) {
      __threadfence();
      asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(flag), "r"(epoch) : "memory");
    }
  }
  if (k != nullptr) block_write_rows(m, g, pool_layer, dst_row, dst_pos, k, v, n);  // layer 0's rows, same launch
  wait_for_overtaken_kernel();
  // Everything enqueued ahead of this kernel has ended, the previous host-buffer step's attention kernel
  // included: its output rows may be copied to the host and its input staging buffer refilled.  The word is
  // read by stream memory operations of the cache's other streams, the rows by a copy engine: agents of this
  // GPU, which meet the SMs in L2, so a device-scope fence orders the store behind what this thread has
  // observed (a system-scope fence here cost 11 us per step: the next attention kernel waits for this kernel
  // to end).
  if (hs.done_word != nullptr && threadIdx.x == 0) {
    __threadfence();
    *reinterpret_cast<volatile int32_t*>(hs.done_word) = hs.done_seq;
  }
}

// Writes the number of the last host-buffer step to the "done" word once everything ahead of it on the stream
// has ended (an ordinary launch): for the step that no later bookkeeping kernel vouches for.
__global__ void k_host_steps_done(int32_t* done_word, int32_t seq) {
  __threadfence();
  *reinterpret_cast<volatile int32_t*>(done_word) = seq;
}

// phase & 1: validate, allocate the beacon slot, fill dst_row/dst_pos (dst_row < 0: item failed).
// phase & 2: for items with dst_row >= 0, push the window pages, clear the window, count the beacon.
__global__ void __launch_bounds__(kBookThreads, 1)
k_compress_book(BcMeta m, const int32_t* __restrict__ slots, int n, int64_t call,
                int32_t* dst_row, int32_t* dst_pos, int phase, BcGeom g, uint8_t* pool_layer,
                const uint8_t* k, const uint8_t* v) {
  __shared__ int sh_first;
  __shared__ int sh_used;
  const int ps = m.page_size;
  int top = *m.free_top;
  __syncthreads();
  if (phase & 1) {
    ErrLatch latch; latch.init(&sh_first);
    dup_prepass(m, slots, n, call);
    int base = 0, used = 0, my_code = 0, my_item = -1, my_slot = 0;
    for (int chunk = 0; chunk < n; chunk += blockDim.x) {
      const int i = chunk + threadIdx.x;
      int need = 0, slot = -1, nb = 0, code = 0;
      bool valid = false;
      if (i < n) {
        slot = slots[i];
        if (slot < 0 || slot >= m.max_seqs || !m.open[slot]) code = BC_ERR_BAD_SLOT;
        else if (is_dup(m, slot, i, call)) code = BC_ERR_DEBUG_CHECK;
        else {
          const int c = m.c[slot];
          nb = m.n_beacons[slot];
          if (c <= 1 || m.window_len[slot] != c) code = BC_ERR_WINDOW_NOT_FULL;
          else {
            need = (nb % ps == 0) ? 1 : 0;
            const int pages = ceil_div(m.prompt_len[slot], ps) + ceil_div(nb, ps) + ceil_div(c, ps);
            if (need && pages + 1 > m.max_pages_per_seq) { code = BC_ERR_CAPACITY; need = 0; }
            else valid = true;
          }
        }
      }
      int total;
      const int off = base + block_exclusive_scan(need, &total);
      base += total;
      int row_out = -1;
      if (valid) {
        if (need == 0 || off + need <= top) {
          int32_t* col = m.page_table + (int64_t)slot * m.max_pages_per_seq + m.beacon_off[slot] + nb / ps;
          if (need) { *col = m.free_stack[top - 1 - off]; used = max(used, off + 1); }
          if (debug_page_ok(m, *col)) row_out = *col * ps + nb % ps;
        } else code = BC_ERR_NO_PAGES;
      }
      if (i < n) { dst_row[i] = row_out; dst_pos[i] = nb; }
      if (code && my_code == 0) { my_code = code; my_item = i; my_slot = slot; latch.note(i); }
    }
    used = __reduce_max_sync(0xffffffffu, used);
    if (threadIdx.x == 0) sh_used = 0;
    __syncthreads();
    if ((threadIdx.x & 31) == 0) atomicMax(&sh_used, used);
    latch.commit(m, my_item, my_code, my_slot, call);
    __syncthreads();
    top -= sh_used;
    __syncthreads();
  }
  if (phase & 2) {
    int base = 0;
    for (int chunk = 0; chunk < n; chunk += blockDim.x) {
      const int i = chunk + threadIdx.x;
      int cnt = 0, slot = -1;
      if (i < n && dst_row[i] >= 0) {
        slot = slots[i];
        cnt = ceil_div(m.window_len[slot], ps);
      }
      int total;
      const int off = base + block_exclusive_scan(cnt, &total);
      base += total;
      if (slot >= 0) {
        const int32_t* col = m.page_table + (int64_t)slot * m.max_pages_per_seq + m.window_off[slot];
        for (int k = 0; k < cnt; ++k) m.free_stack[top + off + k] = col[k];
        m.window_len[slot] = 0;
        m.n_beacons[slot] += 1;
      }
    }
    top += base;
  }
  __syncthreads();
  if (threadIdx.x == 0) *m.free_top = top;
  if (k != nullptr) block_write_rows(m, g, pool_layer, dst_row, dst_pos, k, v, n);  // the beacon rows, same launch
  wait_for_overtaken_kernel();
}

__global__ void __launch_bounds__(kBookThreads, 1)
k_close(BcMeta m, const int32_t* __restrict__ slots, int n, int64_t call) {
  __shared__ int sh_first;
  ErrLatch latch; latch.init(&sh_first);
  dup_prepass(m, slots, n, call);
  const int ps = m.page_size;
  const int top = *m.free_top;
  __syncthreads();
  int base = 0, my_code = 0, my_item = -1, my_slot = 0;
  for (int chunk = 0; chunk < n; chunk += blockDim.x) {
    const int i = chunk + threadIdx.x;
    int slot = -1, np = 0, nbp = 0, nwp = 0, code = 0;
    if (i < n) {
      slot = slots[i];
      if (slot < 0 || slot >= m.max_seqs || !m.open[slot]) { code = BC_ERR_BAD_SLOT; slot = -1; }
      else if (is_dup(m, slot, i, call)) { code = BC_ERR_DEBUG_CHECK; slot = -1; }
      else {
        np = ceil_div(m.prompt_len[slot], ps);
        nbp = ceil_div(m.n_beacons[slot], ps);
        nwp = ceil_div(m.window_len[slot], ps);
      }
    }
    int total;
    const int off = base + block_exclusive_scan(np + nbp + nwp, &total);
    base += total;
    if (slot >= 0) {
      const int32_t* row = m.page_table + (int64_t)slot * m.max_pages_per_seq;
      int o = top + off;
      for (int k = 0; k < np; ++k) m.free_stack[o++] = row[k];
      for (int k = 0; k < nbp; ++k) m.free_stack[o++] = row[m.beacon_off[slot] + k];
      for (int k = 0; k < nwp; ++k) m.free_stack[o++] = row[m.window_off[slot] + k];
      m.open[slot] = 0; m.prompt_len[slot] = 0; m.n_beacons[slot] = 0; m.window_len[slot] = 0;
      m.c[slot] = 0; m.t[slot] = 0;
    }
    if (code && my_code == 0) { my_code = code; my_item = i; my_slot = slots[i]; latch.note(i); }
  }
  latch.commit(m, my_item, my_code, my_slot, call);
  __syncthreads();
  if (threadIdx.x == 0) *m.free_top = top + base;
}

// One block per batch item: copies the item's K and V rows (all heads) into its pool row,
// 16 bytes per thread, applying the chunk permutation of the store layout.
__global__ void k_write_rows(BcMeta m, BcGeom g, uint8_t* __restrict__ pool_layer, const int32_t* __restrict__ dst_row,
                             const int32_t* __restrict__ dst_pos, const uint8_t* __restrict__ k,
                             const uint8_t* __restrict__ v, int n, long long ls_pool, long long ls_kv) {
  // the attention kernel of the step may start planning now; it waits for this kernel before it reads a row
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // blockIdx.y: the layer, when one launch writes the rows of all layers (same row and position in every layer)
  pool_layer += blockIdx.y * ls_pool; k += blockIdx.y * ls_kv; v += blockIdx.y * ls_kv;
  const int i = blockIdx.x;
  const int row = dst_row[i];
  if (row < 0) return;
  if (m.debug && row >= m.num_pages * g.page_size) { if (threadIdx.x == 0) debug_note(m, row); return; }
  const int pos = dst_pos[i];
  const int chunks_per_head = g.head_row_bytes >> 4;
  const int per_side = g.kv_heads * chunks_per_head;
  uint8_t* dst = pool_layer + (int64_t)row * g.entry_bytes;
  for (int idx = threadIdx.x; idx < 2 * per_side; idx += blockDim.x) {
    const int which = idx / per_side, rem = idx - which * per_side;
    const int h = rem / chunks_per_head, j = rem - h * chunks_per_head;
    const uint8_t* src = (which ? v : k) + ((int64_t)i * g.kv_heads + h) * g.head_row_bytes + (j << 4);
    *reinterpret_cast<uint4*>(dst + bc_chunk_offset(g, which, h, j, pos)) = *reinterpret_cast<const uint4*>(src);
  }
}

// One block per prompt token of the packed [total, kv_heads, head_dim] input.
__global__ void k_prefill(BcMeta m, BcGeom g, uint8_t* __restrict__ pool_layer, const int32_t* __restrict__ slots,
                          const int32_t* __restrict__ cu, int n, const uint8_t* __restrict__ k,
                          const uint8_t* __restrict__ v) {
  const int tok = blockIdx.x;
  __shared__ int sh_row, sh_pos;
  if (threadIdx.x == 0) {
    int lo = 0, hi = n;  // largest s with cu[s] <= tok
    while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (cu[mid] <= tok) lo = mid; else hi = mid; }
    const int slot = slots[lo], pos = tok - cu[lo];
    int row = -1;
    if (slot >= 0 && slot < m.max_seqs && m.open[slot] && pos < m.prompt_len[slot]) {
      const int col = pos / g.page_size;
      if (m.debug && col >= m.max_pages_per_seq) debug_note(m, col);
      else {
        const int page = m.page_table[(int64_t)slot * m.max_pages_per_seq + col];
        if (debug_page_ok(m, page)) row = page * g.page_size + pos % g.page_size;
      }
    }
    sh_row = row; sh_pos = pos;
  }
  __syncthreads();
  const int row = sh_row, pos = sh_pos;
  if (row < 0) return;
  const int chunks_per_head = g.head_row_bytes >> 4;
  const int per_side = g.kv_heads * chunks_per_head;
  uint8_t* dst = pool_layer + (int64_t)row * g.entry_bytes;
  for (int idx = threadIdx.x; idx < 2 * per_side; idx += blockDim.x) {
    const int which = idx / per_side, rem = idx - which * per_side;
    const int h = rem / chunks_per_head, j = rem - h * chunks_per_head;
    const uint8_t* src = (which ? v : k) + ((int64_t)tok * g.kv_heads + h) * g.head_row_bytes + (j << 4);
    *reinterpret_cast<uint4*>(dst + bc_chunk_offset(g, which, h, j, pos)) = *reinterpret_cast<const uint4*>(src);
  }
}

// Bookkeeping of bc_restore (one thread block): item i is a freshly opened sequence that receives a
// stored trajectory of T_i = cu[i + 1] - cu[i] generated tokens, i.e. the state Algorithm 1 is in
// after T_i sampling steps: floor(T_i / c) beacons and the T_i mod c tokens of the unfinished window
// (all T_i when c = 1).  Allocates the beacon pages, then the window pages, of every item by a
// block-wide prefix sum, and writes for the copy kernels ok[i] (1: granted) and bea[i] = number of
// beacon rows of the items before i in the packed beacon arrays (items whose slot is not open count
// none), bea[n] = their total.
__global__ void __launch_bounds__(kBookThreads, 1)
k_restore_book(BcMeta m, const int32_t* __restrict__ slots, const int32_t* __restrict__ cu, int n, int64_t call,
               int32_t* __restrict__ ok, int32_t* __restrict__ bea) {
  __shared__ int sh_first;
  ErrLatch latch; latch.init(&sh_first);
  dup_prepass(m, slots, n, call);
  const int top0 = *m.free_top;
  const int ps = m.page_size;
  __syncthreads();
  int base = 0, bea_base = 0, used = 0, my_code = 0, my_item = -1, my_slot = 0;
  for (int chunk = 0; chunk < n; chunk += blockDim.x) {
    const int i = chunk + threadIdx.x;
    int need = 0, slot = -1, code = 0, nb = 0, w = 0, nbp = 0, nwp = 0, T = 0, rows = 0;
    bool valid = false;
    if (i < n) {
      slot = slots[i];
      T = cu[i + 1] - cu[i];
      if (slot < 0 || slot >= m.max_seqs || !m.open[slot]) code = BC_ERR_BAD_SLOT;
      else {
        const int c = m.c[slot];
        if (T >= 0) { nb = c > 1 ? T / c : 0; w = T - nb * c; rows = nb; }   // an open slot's item has beacon rows in the packed input
        if (is_dup(m, slot, i, call)) code = BC_ERR_DEBUG_CHECK;
        else if (T < 0 || m.t[slot] != 0 || m.n_beacons[slot] != 0 || m.window_len[slot] != 0) code = BC_ERR_INVALID_ARG;
        else if (m.max_entries > 0 && nb + w > m.max_entries) code = BC_ERR_CAPACITY;
        else {
          nbp = ceil_div(nb, ps); nwp = ceil_div(w, ps);
          const int reserved = c > 1 ? ceil_div(c, ps) : nwp;   // the window's columns of the page-table row
          if (ceil_div(m.prompt_len[slot], ps) + reserved + nbp > m.max_pages_per_seq) code = BC_ERR_CAPACITY;
          else { valid = true; need = nbp + nwp; }
        }
      }
    }
    int total, bea_total;
    const int off = base + block_exclusive_scan(need, &total);
    base += total;
    const int bea_off = bea_base + block_exclusive_scan(rows, &bea_total);
    bea_base += bea_total;
    int granted = 0;
    if (valid) {
      if (need == 0 || off + need <= top0) {
        int32_t* row = m.page_table + (int64_t)slot * m.max_pages_per_seq;
        for (int k = 0; k < nbp; ++k) row[m.beacon_off[slot] + k] = m.free_stack[top0 - 1 - off - k];
        for (int k = 0; k < nwp; ++k) row[m.window_off[slot] + k] = m.free_stack[top0 - 1 - off - nbp - k];
        if (need) used = max(used, off + need);
        m.n_beacons[slot] = nb; m.window_len[slot] = w; m.t[slot] = T;
        granted = 1;
      } else code = BC_ERR_NO_PAGES;
    }
    if (i < n) { ok[i] = granted; bea[i] = bea_off; }
    if (code && my_code == 0) { my_code = code; my_item = i; my_slot = slot; latch.note(i); }
  }
  used = __reduce_max_sync(0xffffffffu, used);
  __shared__ int sh_used;
  if (threadIdx.x == 0) { sh_used = 0; bea[n] = bea_base; }
  __syncthreads();
  if ((threadIdx.x & 31) == 0) atomicMax(&sh_used, used);
  latch.commit(m, my_item, my_code, my_slot, call);
  __syncthreads();
  if (threadIdx.x == 0) *m.free_top = top0 - sh_used;
}

// Copies one K/V entry (all heads) into pool row `row`, 16 bytes per thread, with the store's chunk permutation.
__device__ __forceinline__ void copy_entry(const BcGeom& g, uint8_t* __restrict__ pool_layer, int row, int pos,
                                           const uint8_t* __restrict__ k, const uint8_t* __restrict__ v, int64_t src_row) {
  const int chunks_per_head = g.head_row_bytes >> 4;
  const int per_side = g.kv_heads * chunks_per_head;
  uint8_t* dst = pool_layer + (int64_t)row * g.entry_bytes;
  for (int idx = threadIdx.x; idx < 2 * per_side; idx += blockDim.x) {
    const int which = idx / per_side, rem = idx - which * per_side;
    const int h = rem / chunks_per_head, j = rem - h * chunks_per_head;
    const uint8_t* src = (which ? v : k) + (src_row * g.kv_heads + h) * g.head_row_bytes + (j << 4);
    *reinterpret_cast<uint4*>(dst + bc_chunk_offset(g, which, h, j, pos)) = *reinterpret_cast<const uint4*>(src);
  }
}

// bc_restore, beacons: one block per row of the packed beacon arrays.
__global__ void k_restore_beacons(BcMeta m, BcGeom g, uint8_t* __restrict__ pool_layer, const int32_t* __restrict__ slots,
                                  const int32_t* __restrict__ ok, const int32_t* __restrict__ bea, int n,
                                  const uint8_t* __restrict__ k, const uint8_t* __restrict__ v) {
  const int b = blockIdx.x;
  __shared__ int sh_row, sh_pos;
  if (threadIdx.x == 0) {
    int row = -1, pos = 0;
    if (b < bea[n]) {
      int lo = 0, hi = n;  // largest i with bea[i] <= b (items without beacons share their successor's offset)
      while (hi - lo > 1) { int mid = (lo + hi) >> 1; if (bea[mid] <= b) lo = mid; else hi = mid; }
      if (ok[lo]) {
        const int slot = slots[lo];
        pos = b - bea[lo];
        const int col = m.beacon_off[slot] + pos / g.page_size;
        if (m.debug && (unsigned)col >= (unsigned)m.max_pages_per_seq) debug_note(m, col);
        else {
          const int page = m.page_table[(int64_t)slot * m.max_pages_per_seq + col];
          if (debug_page_ok(m, page)) row = page * g.page_size + pos % g.page_size;
        }
      }
    }
    sh_row = row; sh_pos = pos;
  }
  __syncthreads();
  if (sh_row >= 0) copy_entry(g, pool_layer, sh_row, sh_pos, k, v, b);
}

// bc_restore, unfinished windows: blocks (item, y) copy window entries y, y + gridDim.y, ... of the item,
// which are the last window_len rows of its tokens in the packed token arrays.
__global__ void k_restore_window(BcMeta m, BcGeom g, uint8_t* __restrict__ pool_layer, const int32_t* __restrict__ slots,
                                 const int32_t* __restrict__ ok, const int32_t* __restrict__ cu, int total_tokens,
                                 const uint8_t* __restrict__ k, const uint8_t* __restrict__ v) {
  const int i = blockIdx.x;
  if (!ok[i]) return;
  const int slot = slots[i];
  const int w = m.window_len[slot];
  const int64_t first = (int64_t)cu[i + 1] - w;   // row of the window's first token
  const int32_t* cols = m.page_table + (int64_t)slot * m.max_pages_per_seq + m.window_off[slot];
  for (int j = blockIdx.y; j < w; j += gridDim.y) {
    if (first + j < 0 || first + j >= total_tokens) continue;
    if (m.debug && (unsigned)(m.window_off[slot] + j / g.page_size) >= (unsigned)m.max_pages_per_seq) {
      if (threadIdx.x == 0) debug_note(m, m.window_off[slot] + j / g.page_size);
      continue;
    }
    const int page = cols[j / g.page_size];
    if (m.debug && (unsigned)page >= (unsigned)m.num_pages) { if (threadIdx.x == 0) debug_note(m, page); continue; }
    copy_entry(g, pool_layer, page * g.page_size + j % g.page_size, j, k, v, first + j);
  }
}

// One block per exported entry, logical order prompt | beacons | window.
__global__ void k_export(BcMeta m, BcGeom g, const uint8_t* __restrict__ pool_layer, int slot,
                         uint8_t* __restrict__ k_out, uint8_t* __restrict__ v_out, int capacity) {
  const int e = blockIdx.x;
  if (slot < 0 || slot >= m.max_seqs || !m.open[slot]) return;
  const int P = m.prompt_len[slot], nb = m.n_beacons[slot], w = m.window_len[slot];
  if (e >= capacity || e >= P + nb + w) return;
  int pos, col0;
  if (e < P) { pos = e; col0 = 0; }
  else if (e < P + nb) { pos = e - P; col0 = m.beacon_off[slot]; }
  else { pos = e - P - nb; col0 = m.window_off[slot]; }
  if (m.debug && (unsigned)(col0 + pos / g.page_size) >= (unsigned)m.max_pages_per_seq) {
    if (threadIdx.x == 0) debug_note(m, col0 + pos / g.page_size);
    return;
  }
  const int page = m.page_table[(int64_t)slot * m.max_pages_per_seq + col0 + pos / g.page_size];
  if (m.debug && (unsigned)page >= (unsigned)m.num_pages) { if (threadIdx.x == 0) debug_note(m, page); return; }
  const uint8_t* src = pool_layer + ((int64_t)page * g.page_size + pos % g.page_size) * g.entry_bytes;
  const int chunks_per_head = g.head_row_bytes >> 4;
  const int per_side = g.kv_heads * chunks_per_head;
  for (int idx = threadIdx.x; idx < 2 * per_side; idx += blockDim.x) {
    const int which = idx / per_side, rem = idx - which * per_side;
    const int h = rem / chunks_per_head, j = rem - h * chunks_per_head;
    uint8_t* dst = (which ? v_out : k_out) + ((int64_t)e * g.kv_heads + h) * g.head_row_bytes + (j << 4);
    *reinterpret_cast<uint4*>(dst) = *reinterpret_cast<const uint4*>(src + bc_chunk_offset(g, which, h, j, pos));
  }
}

inline int copy_threads(const BcGeom& g) {
  int t = g.entry_bytes >> 4;
  return t < 32 ? 32 : (t > 256 ? 256 : t);
}

}  // namespace

cudaError_t bc_launch_init(const BcMeta& m, cudaStream_t s) {
  k_init<<<64, 256, 0, s>>>(m);
  return cudaGetLastError();
}
cudaError_t bc_launch_open(const BcMeta& m, const int32_t* slots, const int32_t* plens, const int32_t* cs, int n,
                           int64_t call, cudaStream_t s) {
  k_open<<<1, kBookThreads, 0, s>>>(m, slots, plens, cs, n, call);
  return cudaGetLastError();
}
// Launch of a bookkeeping kernel that touches nothing but the metadata (no K/V rows in the same
// launch): with programmatic stream serialisation, so that it may begin while the attention kernel
// enqueued before it -- which has read all the lengths it needs by the time it lets dependents go --
// is still finishing its last blocks.  It waits for nothing of that kernel: it reads no output of it.
// After any other predecessor the attribute changes nothing (no early trigger, ordinary order).
constexpr int kWarpBookItems = 256;
template <typename... KArgs, typename... Args>
cudaError_t launch_book_overlapped(void (*kernel)(KArgs...), cudaStream_t s, int threads, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(1); cfg.blockDim = dim3(threads); cfg.dynamicSmemBytes = 0; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

cudaError_t bc_launch_append_book(const BcMeta& m, const int32_t* slots, int n, int64_t call, int32_t* dst_row,
                                  int32_t* dst_pos, const BcGeom& g, uint8_t* pool_layer, const void* k, const void* v,
                                  cudaStream_t s, int32_t* plan, int32_t* flag, int32_t epoch, const BcHostSync* hs) {
  const BcHostSync none = {nullptr, 0, nullptr, 0, nullptr};
  if (k == nullptr) {  // the rows follow in a launch of their own (ordinary order: it waits for everything before it)
    if (n <= kWarpBookItems)   // one warp walks them in at most eight rounds of dependent reads
      return launch_book_overlapped(k_append_book<true>, s, 32, m, slots, n, call, dst_row, dst_pos, g, pool_layer,
                                    (const uint8_t*)nullptr, (const uint8_t*)nullptr, plan, flag, epoch, hs ? *hs : none);
    return launch_book_overlapped(k_append_book<false>, s, kBookThreads, m, slots, n, call, dst_row, dst_pos, g, pool_layer,
                                  (const uint8_t*)nullptr, (const uint8_t*)nullptr, plan, flag, epoch, hs ? *hs : none);
  }
  k_append_book<false><<<1, kBookThreads, 0, s>>>(m, slots, n, call, dst_row, dst_pos, g, pool_layer, (const uint8_t*)k,
                                           (const uint8_t*)v, (int32_t*)nullptr, (int32_t*)nullptr, 0, none);
  return cudaGetLastError();
}
cudaError_t bc_launch_host_steps_done(int32_t* done_word, int32_t seq, cudaStream_t s) {
  k_host_steps_done<<<1, 1, 0, s>>>(done_word, seq);
  return cudaGetLastError();
}
cudaError_t bc_launch_compress_book(const BcMeta& m, const int32_t* slots, int n, int64_t call, int32_t* dst_row,
                                    int32_t* dst_pos, int phase, const BcGeom& g, uint8_t* pool_layer, const void* k,
                                    const void* v, cudaStream_t s) {
  // With rows as without: the beacon rows come from the caller's inputs, which no kernel of this library writes,
  // and go to slots and pages that the kernel which may still be running ahead does not read.
  return launch_book_overlapped(k_compress_book, s, kBookThreads, m, slots, n, call, dst_row, dst_pos, phase, g, pool_layer,
                                (const uint8_t*)k, (const uint8_t*)v);
}
cudaError_t bc_launch_close(const BcMeta& m, const int32_t* slots, int n, int64_t call, cudaStream_t s) {
  k_close<<<1, kBookThreads, 0, s>>>(m, slots, n, call);
  return cudaGetLastError();
}
cudaError_t bc_launch_write_rows(const BcMeta& m, const BcGeom& g, uint8_t* pool_layer, const int32_t* dst_row, const int32_t* dst_pos,
                                 const void* k, const void* v, int n, cudaStream_t s, int layers, long long ls_pool,
                                 long long ls_kv) {
  k_write_rows<<<dim3(n, layers), copy_threads(g), 0, s>>>(m, g, pool_layer, dst_row, dst_pos, (const uint8_t*)k, (const uint8_t*)v, n,
                                                           ls_pool, ls_kv);
  return cudaGetLastError();
}
cudaError_t bc_launch_prefill(const BcMeta& m, const BcGeom& g, uint8_t* pool_layer, const int32_t* slots,
                              const int32_t* cu, int n, int total, const void* k, const void* v, cudaStream_t s) {
  if (total == 0) return cudaSuccess;
  k_prefill<<<total, copy_threads(g), 0, s>>>(m, g, pool_layer, slots, cu, n, (const uint8_t*)k, (const uint8_t*)v);
  return cudaGetLastError();
}
cudaError_t bc_launch_restore_book(const BcMeta& m, const int32_t* slots, const int32_t* cu, int n, int64_t call, int32_t* ok,
                                   int32_t* bea, cudaStream_t s) {
  k_restore_book<<<1, kBookThreads, 0, s>>>(m, slots, cu, n, call, ok, bea);
  return cudaGetLastError();
}
cudaError_t bc_launch_restore_rows(const BcMeta& m, const BcGeom& g, uint8_t* pool_layer, const int32_t* slots, const int32_t* ok,
                                   const int32_t* bea, const int32_t* cu, int n, int total_tokens, int total_beacons,
                                   const void* tok_k, const void* tok_v, const void* bea_k, const void* bea_v, cudaStream_t s) {
  if (total_beacons > 0)
    k_restore_beacons<<<total_beacons, copy_threads(g), 0, s>>>(m, g, pool_layer, slots, ok, bea, n, (const uint8_t*)bea_k,
                                                              (const uint8_t*)bea_v);
  if (total_tokens > 0)
    k_restore_window<<<dim3(n, 32), copy_threads(g), 0, s>>>(m, g, pool_layer, slots, ok, cu, total_tokens, (const uint8_t*)tok_k,
                                                          (const uint8_t*)tok_v);
  return cudaGetLastError();
}
cudaError_t bc_launch_export(const BcMeta& m, const BcGeom& g, const uint8_t* pool_layer, int slot, void* k_out,
                             void* v_out, int capacity, cudaStream_t s) {
  if (capacity <= 0) return cudaSuccess;
  k_export<<<capacity, copy_threads(g), 0, s>>>(m, g, pool_layer, slot, (uint8_t*)k_out, (uint8_t*)v_out, capacity);
  return cudaGetLastError();
}
