"""Integer-only model of the paged store's bookkeeping.

TEST INFRASTRUCTURE ONLY (see oracle/__init__.py).  The paper has no paging:
its cache is a Python list (Algorithm 1).  The paged store, its per-sequence
page table and its device free list come from the build's target statement, so
this model follows the allocation discipline the library documents in
include/breadcrumbs.h, written here independently with plain Python lists:

* Free pages form a LIFO stack; ``stack[-1]`` is handed out first.  A fresh
  store hands out pages 0, 1, 2, ... in that order.
* One batch call first allocates, then frees.
  Allocation: walk the batch in order; item i with need[i] pages receives the
  pages at stack depth off[i] .. off[i]+need[i]-1, off = exclusive prefix sum
  of the needs of ALL items that passed validation; an item is granted iff
  need[i] == 0 or off[i] + need[i] <= pages free at the start of the call.
  Frees: walk the batch in order; a sequence's pages are pushed in the order
  prompt pages, beacon pages, window pages, each in ascending index.
* restore (a stored trajectory of T generated tokens put into a freshly
  opened sequence in one call) leaves the lengths that T appends with their
  compressions leave (Algorithm 1: floor(T/c) beacons, T mod c window
  entries); an item needs ceil(beacons/page) + ceil(window/page) pages and
  receives its beacon pages first, then its window pages.
* A failed item is a no-op for its sequence; the first failure of the store's
  lifetime is latched as (code, slot, call index); when several items of one
  call fail, the one with the lowest batch index is reported.
* Checked mode (``debug_bounds=True``, the library's BC_FLAG_DEBUG_BOUNDS): a
  batch must not name a slot twice; every item whose (valid) slot an item with
  a lower index of the same call names is refused with DEBUG_CHECK, after the
  slot check and before every other check, and the first occurrence goes
  through alone.  Without the flag such a batch is outside the contract.

Pinned by tests/test_oracle_pins.py: conservation (owned + free = all pages,
no page twice), per-segment page counts = ceil(len / page_size), lengths equal
to the closed form, exhaustion on tiny pools worked out by hand.
"""
from __future__ import annotations

OK = "OK"
BAD_SLOT = "BAD_SLOT"
NO_PAGES = "NO_PAGES"
CAPACITY = "CAPACITY"
WINDOW_NOT_FULL = "WINDOW_NOT_FULL"
WINDOW_FULL = "WINDOW_FULL"
INVALID_ARG = "INVALID_ARG"
DEBUG_CHECK = "DEBUG_CHECK"


def _ceil_div(a, b):
    return -(-a // b)


class _Seq:
    def __init__(self, P, c):
        self.P, self.c = P, c
        self.n_beacons = 0
        self.window_len = 0
        self.t = 0
        self.prompt_pages = []
        self.beacon_pages = []
        self.window_pages = []


class PagingModel:
    def __init__(self, num_pages, page_size, max_seqs, max_pages_per_seq,
                 max_entries_per_seq=0, c_default=1, debug_bounds=False):
        self.ps = page_size
        self.num_pages = num_pages
        self.max_seqs = max_seqs
        self.max_pages_per_seq = max_pages_per_seq
        self.max_entries = max_entries_per_seq
        self.c_default = c_default
        self.debug_bounds = debug_bounds
        self.stack = list(range(num_pages - 1, -1, -1))   # stack[-1] == page 0
        self.seqs = {}
        self.first_error = None       # (code, slot, call_index)
        self._pending = []
        self.calls = 0

    # ------------------------------------------------------------------ utils
    def _dup(self, slots, i):
        """Checked mode: does an item with a lower batch index name the same slot?"""
        return self.debug_bounds and slots[i] in slots[:i]

    def _fail(self, code, slot, item):
        self._pending.append((item, code, slot))
        return code

    def _latch(self, res):
        """Of the failures of one call, the one with the lowest batch index is the call's
        error; the first failing call of the store's lifetime is the latched one."""
        if self._pending and self.first_error is None:
            _, code, slot = min(self._pending)
            self.first_error = (code, slot, self.calls)
        self._pending = []
        return res

    def _allocate(self, needs):
        """needs: list of (item index, pages needed) for validated items, in
        batch order.  Returns {item index: [pages]} for granted items."""
        free_at_start = len(self.stack)
        granted, off, used = {}, 0, 0
        for i, need in needs:
            if need == 0:
                granted[i] = []
            elif off + need <= free_at_start:
                granted[i] = [self.stack[free_at_start - 1 - off - k] for k in range(need)]
                used = off + need
            off += need
        # granted items form a prefix of the requesters, so `used` pages leave the top
        if used:
            del self.stack[free_at_start - used:]
        return granted

    # ------------------------------------------------------------------- calls
    def open(self, slots, prompt_lens, cs=None):
        self.calls += 1
        res, needs, plan = [None] * len(slots), [], {}
        for i, slot in enumerate(slots):
            c = self.c_default if cs is None else cs[i]
            P = prompt_lens[i]
            if not (0 <= slot < self.max_seqs) or slot in self.seqs:
                res[i] = self._fail(BAD_SLOT, slot, i); continue
            if self._dup(slots, i):
                res[i] = self._fail(DEBUG_CHECK, slot, i); continue
            if c < 1 or P < 0:
                res[i] = self._fail(INVALID_ARG, slot, i); continue
            npp = _ceil_div(P, self.ps)
            nwp = _ceil_div(c, self.ps) if c > 1 else 0
            if npp + nwp > self.max_pages_per_seq:
                res[i] = self._fail(CAPACITY, slot, i); continue
            needs.append((i, npp)); plan[i] = (slot, P, c)
        granted = self._allocate(needs)
        for i, _ in needs:
            slot, P, c = plan[i]
            if i not in granted:
                res[i] = self._fail(NO_PAGES, slot, i); continue
            s = _Seq(P, c); s.prompt_pages = granted[i]
            self.seqs[slot] = s; res[i] = OK
        return self._latch(res)

    def append(self, slots):
        self.calls += 1
        res, needs = [None] * len(slots), []
        for i, slot in enumerate(slots):
            s = self.seqs.get(slot)
            if s is None:
                res[i] = self._fail(BAD_SLOT, slot, i); continue
            if self._dup(slots, i):
                res[i] = self._fail(DEBUG_CHECK, slot, i); continue
            if s.c > 1 and s.window_len >= s.c:
                res[i] = self._fail(WINDOW_FULL, slot, i); continue
            if self.max_entries and s.n_beacons + s.window_len + 1 > self.max_entries:
                res[i] = self._fail(CAPACITY, slot, i); continue
            need = 1 if s.window_len % self.ps == 0 else 0
            if need and (len(s.prompt_pages) + len(s.beacon_pages) + len(s.window_pages) + 1
                         > self.max_pages_per_seq):
                res[i] = self._fail(CAPACITY, slot, i); continue
            needs.append((i, need))
        granted = self._allocate(needs)
        for i, _ in needs:
            slot = slots[i]; s = self.seqs[slot]
            if i not in granted:
                res[i] = self._fail(NO_PAGES, slot, i); continue
            s.window_pages += granted[i]
            s.window_len += 1; s.t += 1; res[i] = OK
        return self._latch(res)

    def compress(self, slots):
        self.calls += 1
        res, needs = [None] * len(slots), []
        for i, slot in enumerate(slots):
            s = self.seqs.get(slot)
            if s is None:
                res[i] = self._fail(BAD_SLOT, slot, i); continue
            if self._dup(slots, i):
                res[i] = self._fail(DEBUG_CHECK, slot, i); continue
            if s.c <= 1 or s.window_len != s.c:
                res[i] = self._fail(WINDOW_NOT_FULL, slot, i); continue
            need = 1 if s.n_beacons % self.ps == 0 else 0
            if need and (len(s.prompt_pages) + len(s.beacon_pages) + _ceil_div(s.c, self.ps) + 1
                         > self.max_pages_per_seq):
                res[i] = self._fail(CAPACITY, slot, i); continue
            needs.append((i, need))
        granted = self._allocate(needs)
        ok_items = []
        for i, _ in needs:
            slot = slots[i]; s = self.seqs[slot]
            if i not in granted:
                res[i] = self._fail(NO_PAGES, slot, i); continue
            s.beacon_pages += granted[i]; ok_items.append(i); res[i] = OK
        # frees come after every allocation of the call
        for i in ok_items:
            s = self.seqs[slots[i]]
            self.stack.extend(s.window_pages)
            s.window_pages = []; s.window_len = 0; s.n_beacons += 1
        return self._latch(res)

    def restore(self, slots, gen_lens):
        """Puts a stored trajectory of gen_lens[i] generated tokens into slot i, which must be open
        and untouched since (no appends): the state Algorithm 1 is in after that many sampling
        steps, i.e. floor(T / c) beacons and the T mod c tokens of the unfinished window (all T
        tokens when c = 1)."""
        self.calls += 1
        res, needs, plan = [None] * len(slots), [], {}
        for i, slot in enumerate(slots):
            s = self.seqs.get(slot)
            T = gen_lens[i]
            if s is None:
                res[i] = self._fail(BAD_SLOT, slot, i); continue
            if self._dup(slots, i):
                res[i] = self._fail(DEBUG_CHECK, slot, i); continue
            if T < 0 or s.t != 0 or s.n_beacons != 0 or s.window_len != 0:
                res[i] = self._fail(INVALID_ARG, slot, i); continue
            nb = T // s.c if s.c > 1 else 0
            w = T - nb * s.c
            if self.max_entries and nb + w > self.max_entries:
                res[i] = self._fail(CAPACITY, slot, i); continue
            nbp, nwp = _ceil_div(nb, self.ps), _ceil_div(w, self.ps)
            reserved = _ceil_div(s.c, self.ps) if s.c > 1 else nwp   # the window's columns of the page table
            if len(s.prompt_pages) + reserved + nbp > self.max_pages_per_seq:
                res[i] = self._fail(CAPACITY, slot, i); continue
            needs.append((i, nbp + nwp)); plan[i] = (nb, w, nbp, T)
        granted = self._allocate(needs)
        for i, _ in needs:
            slot = slots[i]; s = self.seqs[slot]
            nb, w, nbp, T = plan[i]
            if i not in granted:
                res[i] = self._fail(NO_PAGES, slot, i); continue
            s.beacon_pages = granted[i][:nbp]; s.window_pages = granted[i][nbp:]
            s.n_beacons, s.window_len, s.t = nb, w, T
            res[i] = OK
        return self._latch(res)

    def close(self, slots):
        self.calls += 1
        res = [None] * len(slots)
        open_at_start = set(self.seqs)           # every item is validated against the state the call finds
        for i, slot in enumerate(slots):
            if slot not in open_at_start or (not self.debug_bounds and slot not in self.seqs):
                res[i] = self._fail(BAD_SLOT, slot, i); continue
            if self._dup(slots, i):
                res[i] = self._fail(DEBUG_CHECK, slot, i); continue
            s = self.seqs[slot]
            self.stack.extend(s.prompt_pages + s.beacon_pages + s.window_pages)
            del self.seqs[slot]; res[i] = OK
        return self._latch(res)

    # ------------------------------------------------------------------- views
    def state(self, slot):
        s = self.seqs.get(slot)
        if s is None:
            return None
        return dict(prompt_len=s.P, n_beacons=s.n_beacons, window_len=s.window_len, c=s.c, t=s.t,
                    prompt_pages=list(s.prompt_pages), beacon_pages=list(s.beacon_pages),
                    window_pages=list(s.window_pages))

    def free_list(self):
        """Free pages, bottom of the stack first (the last one is handed out next)."""
        return list(self.stack)
