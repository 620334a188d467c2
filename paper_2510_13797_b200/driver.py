"""Drives lock-step decode of one workload through the C ABI (no arithmetic of the method here).

A DecodeDriver owns one cache for a batch of sequences that all use the same prompt length and
ratio c, the seeded input tensors, and the position t in the generation.  Step inputs are drawn
once (a ring of `ring` distinct steps and `beacon_ring` distinct beacons) and reused cyclically:

    generated token n (1-based)      -> q, k, v row (n - 1) % ring
    beacon m (1-based, at t = m * c) -> beacon q, k, v row m % beacon_ring

The window's tokens are always distinct (ring >= c).  The beacons a cache holds are distinct only
up to beacon_ring: the benchmark keeps the default of 4 (the values do not change the traffic),
the parity tests pass a ring as long as the run (every stored beacon unique) or a prime longer
than a page, so that a kernel that read beacon m +- k for m, or beacon page j for page k, fails.

so the cache content at any step is a pure function of the workload's seed, which is what lets a
test rebuild it on the CPU without replaying the run.  Used by bench.py and by the full-size tests.
"""
from __future__ import annotations

import itertools

import torch

from . import binding as B
from .workloads import InputStream


class DecodeDriver:
    def __init__(self, w, device, seed_offset=0, fused=False, paired=True, host_pipelined=True, beacon_ring=4):
        self.w, self.dev = w, torch.device(device)
        self.fused = fused                             # True: regular steps through bc_decode_step (one launch)
        self.paired = paired                           # True: the step that fills a window attends for the token and
                                                       # for its beacon in one pass over the cache (bc_decode_attn_pair)
        c, ps, Bn = w.cs[0], w.page_size, w.batch
        P, T = w.prompt_lens[0], w.steps
        assert all(x == c for x in w.cs) and all(x == P for x in w.prompt_lens), "uniform batches only"
        assert w.layers == 1, "single-layer workloads only"
        self.c, self.P, self.T, self.n = c, P, T, Bn
        cd = lambda a, b: -(-a // b)
        if c > 1:
            pages_per_seq = cd(P, ps) + cd(c, ps) + cd(cd(T, c), ps) + 1
        else:
            pages_per_seq = cd(P + T, ps) + 1
        self.pages_per_seq = pages_per_seq
        self.num_pages = Bn * pages_per_seq
        # host-buffer steps return their outputs on the cache's own stream (bc_host_outputs_ready orders them)
        self.cache = B.Cache(w.layers, w.kv_heads, w.q_heads, w.head_dim, c, ps, max_seqs=Bn,
                             num_pages=self.num_pages, max_pages_per_seq=pages_per_seq,
                             flags=B.BC_FLAG_HOST_PIPELINED if host_pipelined else 0, device=self.dev)
        self.slots = torch.arange(Bn, dtype=torch.int32, device=self.dev)
        self.plens = torch.tensor(w.prompt_lens, dtype=torch.int32, device=self.dev)
        self.cu = torch.tensor([0] + list(itertools.accumulate(w.prompt_lens)), dtype=torch.int32, device=self.dev)
        stream = InputStream(w, self.dev)
        self.pk, self.pv = stream.prompt_kv(0)
        self.ring = max(c, 16)                         # distinct step inputs, reused cyclically
        self.q, self.k, self.v = stream.step_chunk(0, seed_offset, self.ring)
        self.bring = int(beacon_ring)                  # distinct beacons, reused cyclically
        self.bq, self.bk, self.bv = stream.beacon_chunk(0, seed_offset, self.bring)
        self.out = self.cache.new_out(Bn)
        self.out_b = self.cache.new_out(Bn)
        self.t = 0
        self.opened = False
        self.h = None                                  # pinned host copies for the host-buffer calls

    def reset_to(self, t_target):
        """(Re)opens the batch, stores the prompts and replays appends/compressions up to t_target."""
        c = self.cache
        if self.opened:
            c.bc_seq_close(self.slots)
        c.bc_seq_open(self.slots, self.plens)
        c.bc_prefill(0, self.slots, self.cu, int(self.cu[-1]), self.pk, self.pv)
        self.opened, self.t = True, 0
        while self.t < t_target:
            j = self.t % self.ring
            c.bc_append(0, self.slots, self.k[j], self.v[j])
            self.t += 1
            if self.c > 1 and self.t % self.c == 0:
                b = (self.t // self.c) % self.bring
                c.bc_compress(0, self.slots, self.bk[b], self.bv[b])

    def step(self):
        """One decode step of the whole batch through the device-pointer calls.  Returns True if the
        window filled and the beacon step (beacon-query attention into out_b, then compress) ran."""
        c, j = self.cache, self.t % self.ring
        if self.paired and self.c > 1 and (self.t + 1) % self.c == 0:
            b = ((self.t + 1) // self.c) % self.bring
            if self.fused:      # append inside the paired attention launch
                c.bc_fill_step(0, self.slots, self.q[j], self.k[j], self.v[j], self.bq[b], self.bk[b], self.bv[b], self.out, self.out_b,
                               self.w.sm_scale)
                self.t += 1
                return True
            c.bc_append(0, self.slots, self.k[j], self.v[j])
            c.bc_decode_attn_pair(0, self.slots, self.q[j], self.out, self.bq[b], self.out_b, self.w.sm_scale, self.bk[b], self.bv[b])
            self.t += 1
            c.bc_compress(0, self.slots, self.bk[b], self.bv[b])
            return True
        if self.fused:
            c.bc_decode_step(0, self.slots, self.q[j], self.k[j], self.v[j], self.out, self.w.sm_scale)
        else:
            c.bc_append(0, self.slots, self.k[j], self.v[j])
            c.bc_decode_attn(0, self.slots, self.q[j], self.out, self.w.sm_scale)
        self.t += 1
        if self.c > 1 and self.t % self.c == 0:
            b = (self.t // self.c) % self.bring
            c.bc_decode_attn(0, self.slots, self.bq[b], self.out_b, self.w.sm_scale, self.bk[b], self.bv[b])
            c.bc_compress(0, self.slots, self.bk[b], self.bv[b])
            return True
        return False

    def step_host(self):
        """The same step through the host-buffer entry points (H2D of q,k,v and D2H of out inside)."""
        if self.h is None:
            pin = lambda t: t.cpu().pin_memory()

            def packed(k, v, q):
                """Per ring slot one pinned block k | v | q, which the library moves with a single copy."""
                ks, vs, qs = [], [], []
                for j in range(k.shape[0]):
                    nk, nq = k[j].numel(), q[j].numel()
                    flat = torch.empty(2 * nk + nq, dtype=k.dtype).pin_memory()
                    flat[:nk] = k[j].reshape(-1).cpu(); flat[nk:2 * nk] = v[j].reshape(-1).cpu(); flat[2 * nk:] = q[j].reshape(-1).cpu()
                    ks.append(flat[:nk].view(k[j].shape)); vs.append(flat[nk:2 * nk].view(v[j].shape)); qs.append(flat[2 * nk:].view(q[j].shape))
                return ks, vs, qs
            hk, hv, hq = packed(self.k, self.v, self.q)
            hbk, hbv, hbq = packed(self.bk, self.bv, self.bq)
            self.h = dict(q=hq, k=hk, v=hv, bq=hbq, bk=hbk, bv=hbv, out=pin(self.out), out_b=pin(self.out_b))
        c, j, h = self.cache, self.t % self.ring, self.h
        if self.paired and self.c > 1 and (self.t + 1) % self.c == 0:
            b = ((self.t + 1) // self.c) % self.bring
            c.bc_fill_step_host(0, self.slots, h["q"][j], h["k"][j], h["v"][j], h["bq"][b], h["bk"][b], h["bv"][b],
                                h["out"], h["out_b"], self.w.sm_scale)
            self.t += 1
            return
        c.bc_decode_step_host(0, self.slots, h["q"][j], h["k"][j], h["v"][j], h["out"], self.w.sm_scale)
        self.t += 1
        if self.c > 1 and self.t % self.c == 0:
            b = (self.t // self.c) % self.bring
            c.bc_compress_step_host(0, self.slots, h["bq"][b], h["bk"][b], h["bv"][b], h["out_b"], self.w.sm_scale)

    def check_error(self):
        code, slot, call = self.cache.bc_poll_error()
        if code != 0:
            raise RuntimeError(f"device-side error {B.STATUS_NAMES.get(code, code)} slot {slot} call {call}")
