"""Drives the CUDA library and the CPU oracle with the same calls and compares them.

The oracle side is a PagingModel (integer bookkeeping) plus one SeqCache per open slot; the CUDA
side is reached through the C ABI (paper_2510_13797_b200.binding).  Inputs are torch bf16 tensors;
the oracle receives their exact values widened to fp64.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle.breadcrumbs_oracle import SeqCache
from oracle.paging_model import OK, PagingModel
from oracle.rope_oracle import split_and_rope
from paper_2510_13797_b200 import binding as B

ABS_TOL = 2e-2   # max-abs error of a head vector (bf16 in, fp32 accumulate)
REL_TOL = 1e-2   # max-abs error relative to the head vector's largest magnitude


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def assert_close(gpu: torch.Tensor, ref: np.ndarray, what=""):
    """Per (sequence, head) vector: max|gpu-ref| <= 2e-2 and <= 1e-2 * max(|ref|_inf, 1e-6)."""
    g = f64(gpu)
    assert g.shape == ref.shape, (g.shape, ref.shape)
    assert np.all(np.isfinite(g)), f"{what}: non-finite output"
    err = np.abs(g - ref).max(axis=-1)
    scale = np.maximum(np.abs(ref).max(axis=-1), 1e-6)
    worst_abs, worst_rel = err.max(), (err / scale).max()
    assert worst_abs <= ABS_TOL, f"{what}: max abs err {worst_abs:.3e}"
    assert worst_rel <= REL_TOL, f"{what}: max rel err {worst_rel:.3e} (abs {worst_abs:.3e})"
    return worst_abs, worst_rel


class Pair:
    def __init__(self, layers, kv_heads, q_heads, head_dim, page_size, max_seqs, num_pages, max_pages_per_seq,
                 c_default=1, max_entries=0, flags=0, device="cuda"):
        self.dev = torch.device(device)
        self.L, self.Hkv, self.Hq, self.D = layers, kv_heads, q_heads, head_dim
        self.gpu = B.Cache(layers, kv_heads, q_heads, head_dim, c_default, page_size, max_seqs, num_pages,
                           max_pages_per_seq, max_entries, flags, device=device)
        self.model = PagingModel(num_pages, page_size, max_seqs, max_pages_per_seq, max_entries, c_default,
                                 debug_bounds=bool(flags & B.BC_FLAG_DEBUG_BOUNDS))
        self.seqs = {}
        self.max_seqs = max_seqs
        self._append_ok = None
        self._compress_ok = None

    def _i32(self, xs):
        return torch.tensor(list(xs), dtype=torch.int32, device=self.dev)

    # ------------------------------------------------------------------ calls
    def open(self, slots, plens, cs=None):
        self.gpu.bc_seq_open(self._i32(slots), self._i32(plens), None if cs is None else self._i32(cs))
        res = self.model.open(list(slots), list(plens), None if cs is None else list(cs))
        for slot, r in zip(slots, res):
            if r == OK:
                self.seqs[slot] = SeqCache(self.L, self.model.state(slot)["c"])
        return res

    def prefill(self, layer, slots, plens, k, v):
        """k, v: packed [sum(plens), Hkv, D] bf16 device tensors."""
        cu = np.concatenate([[0], np.cumsum(plens)]).astype(np.int32)
        self.gpu.bc_prefill(layer, self._i32(slots), self._i32(cu), int(cu[-1]), k, v)
        kk, vv = f64(k), f64(v)
        for i, slot in enumerate(slots):
            if slot in self.seqs:
                self.seqs[slot].prefill(layer, kk[cu[i]:cu[i + 1]], vv[cu[i]:cu[i + 1]])

    def restore(self, layer, slots, gen_lens, tok_k, tok_v, bea_k, bea_v):
        """tok_*: packed [sum(gen_lens), Hkv, D]; bea_*: packed beacons, floor(T / c) per open sequence."""
        cu = np.concatenate([[0], np.cumsum(gen_lens)]).astype(np.int32)
        nbs = [(gen_lens[i] // self.model.seqs[s].c if s in self.model.seqs and self.model.seqs[s].c > 1 else 0)
               if gen_lens[i] >= 0 else 0 for i, s in enumerate(slots)]
        cb = np.concatenate([[0], np.cumsum(nbs)]).astype(np.int64)
        self.gpu.bc_restore(layer, self._i32(slots), self._i32(cu), int(cu[-1]), int(cb[-1]), tok_k, tok_v, bea_k, bea_v)
        if layer == 0:
            self._restore_ok = self.model.restore(list(slots), list(gen_lens))
        tk, tv = f64(tok_k), f64(tok_v)
        bk, bv = (f64(bea_k), f64(bea_v)) if cb[-1] else (np.zeros((0, self.Hkv, self.D)),) * 2
        for i, slot in enumerate(slots):
            if self._restore_ok[i] == OK:
                self.seqs[slot].replay(layer, tk[cu[i]:cu[i + 1]], tv[cu[i]:cu[i + 1]], bk[cb[i]:cb[i + 1]], bv[cb[i]:cb[i + 1]])
        return self._restore_ok

    def append(self, layer, slots, k, v):
        self.gpu.bc_append(layer, self._i32(slots), k, v)
        if layer == 0:
            self._append_ok = self.model.append(list(slots))
        kk, vv = f64(k), f64(v)
        for i, slot in enumerate(slots):
            if self._append_ok[i] == OK:
                self.seqs[slot].append(layer, kk[i], vv[i])
        return self._append_ok

    def step(self, layer, slots, q, k, v, sm_scale):
        """The fused call: append k, v and attend with q.  Returns (append results, out, reference out)."""
        out = self.gpu.new_out(len(slots))
        self.gpu.bc_decode_step(layer, self._i32(slots), q, k, v, out, sm_scale)
        if layer == 0:
            self._append_ok = self.model.append(list(slots))
        kk, vv, qq = f64(k), f64(v), f64(q)
        ref = np.zeros((len(slots), self.Hq, self.D))
        for i, slot in enumerate(slots):
            if self._append_ok[i] == OK:
                self.seqs[slot].append(layer, kk[i], vv[i])
            seq = self.seqs.get(slot) or SeqCache(self.L, 1)
            ref[i] = seq.attend(layer, qq[i], sm_scale)
        return self._append_ok, out, ref

    def rope_step(self, layer, slots, qkv, positions, theta, sm_scale):
        """bc_rope_decode_step: the step straight from the packed QKV projection.  The oracle rotates in fp64
        and rounds q, k to bf16 (the precision the entries are stored in) before its own append and attend."""
        out = self.gpu.new_out(len(slots))
        self.gpu.bc_rope_decode_step(layer, self._i32(slots), qkv, self._i32(positions), theta, out, sm_scale)
        if layer == 0:
            self._append_ok = self.model.append(list(slots))
        bf = lambda a: torch.from_numpy(a).to(torch.bfloat16).to(torch.float64).numpy()
        qq, kk, vv = split_and_rope(f64(qkv), list(positions), self.Hq, self.Hkv, self.D, theta)
        qq, kk = bf(qq), bf(kk)
        ref = np.zeros((len(slots), self.Hq, self.D))
        for i, slot in enumerate(slots):
            if self._append_ok[i] == OK:
                self.seqs[slot].append(layer, kk[i], vv[i])
            seq = self.seqs.get(slot) or SeqCache(self.L, 1)
            ref[i] = seq.attend(layer, qq[i], sm_scale)
        return self._append_ok, out, ref

    def fill(self, layer, slots, q, k, v, bq, bk, bv, sm_scale):
        """bc_fill_step: the token's append, the token's and the beacon's attention, the compression; items the
        bookkeeping refuses behave as in the three separate calls.  Returns (append results, compress results,
        out, out_beacon, reference out, reference out_beacon)."""
        n = len(slots)
        out, out_b = self.gpu.new_out(n), self.gpu.new_out(n)
        self.gpu.bc_fill_step(layer, self._i32(slots), q, k, v, bq, bk, bv, out, out_b, sm_scale)
        if layer == 0:
            self._append_ok = self.model.append(list(slots))
        qq, kk, vv, bqq, bkk, bvv = (f64(x) for x in (q, k, v, bq, bk, bv))
        ref, ref_b = np.zeros((n, self.Hq, self.D)), np.zeros((n, self.Hq, self.D))
        for i, slot in enumerate(slots):
            if self._append_ok[i] == OK:
                self.seqs[slot].append(layer, kk[i], vv[i])
        for i, slot in enumerate(slots):
            seq = self.seqs.get(slot) or SeqCache(self.L, 1)
            ref[i] = seq.attend(layer, qq[i], sm_scale)
            ref_b[i] = seq.beacon_attend(layer, bqq[i], bkk[i], bvv[i], sm_scale)
        if layer == 0:
            self._compress_ok = self.model.compress(list(slots))
        for i, slot in enumerate(slots):
            if self._compress_ok[i] == OK:
                self.seqs[slot].compress(layer, bkk[i], bvv[i])
        return self._append_ok, self._compress_ok, out, out_b, ref, ref_b

    def attend(self, layer, slots, q, sm_scale, extra_k=None, extra_v=None, static=False):
        """static=True: through bc_decode_attn_static (split-K scratch inside the library image)."""
        out = self.gpu.new_out(len(slots))
        call = self.gpu.bc_decode_attn_static if static else self.gpu.bc_decode_attn
        call(layer, self._i32(slots), q, out, sm_scale, extra_k, extra_v)
        qq = f64(q)
        ref = np.zeros((len(slots), self.Hq, self.D))
        for i, slot in enumerate(slots):
            seq = self.seqs.get(slot)
            if seq is None:
                seq = SeqCache(self.L, 1)       # unknown slot: empty cache
            if extra_k is None:
                ref[i] = seq.attend(layer, qq[i], sm_scale)
            else:
                ref[i] = seq.beacon_attend(layer, qq[i], f64(extra_k)[i], f64(extra_v)[i], sm_scale)
        return out, ref

    def compress(self, layer, slots, bk, bv):
        self.gpu.bc_compress(layer, self._i32(slots), bk, bv)
        if layer == 0:
            # the model applies allocation and eviction at once; per-layer data follows below
            self._compress_ok = self.model.compress(list(slots))
        kk, vv = f64(bk), f64(bv)
        for i, slot in enumerate(slots):
            if self._compress_ok[i] == OK:
                self.seqs[slot].compress(layer, kk[i], vv[i])
        return self._compress_ok

    def close(self, slots):
        self.gpu.bc_seq_close(self._i32(slots))
        res = self.model.close(list(slots))
        for slot, r in zip(slots, res):
            if r == OK:
                del self.seqs[slot]
        return res

    # ------------------------------------------------------------------ checks
    def check_state(self, slots=None):
        """Bit-exact bookkeeping: lengths, page lists, free stack, latched error."""
        for slot in (range(self.max_seqs) if slots is None else slots):
            assert self.gpu.bc_get_state(slot) == self.model.state(slot), f"slot {slot}"
        assert self.gpu.bc_get_free_list() == self.model.free_list()
        code, slot, call = self.gpu.bc_poll_error()
        if self.model.first_error is None:
            assert code == 0, (B.STATUS_NAMES.get(code), slot, call)
        else:
            assert (B.STATUS_NAMES[code], slot, call) == self.model.first_error

    def check_content(self, layer, slot):
        """Bit-exact stored content: export (prompt, beacons, window order) vs the oracle's list."""
        K, V = self.seqs[slot].entries(layer)
        k, v = self.gpu.bc_export_seq(layer, slot, max(K.shape[0], 1))
        if K.shape[0]:
            assert np.array_equal(f64(k), K) and np.array_equal(f64(v), V), f"content of slot {slot}"
        ids = self.seqs[slot].live_ids(layer)
        kinds = [k_ for k_, _ in ids]
        assert kinds == sorted(kinds, key=["prompt", "beacon", "token"].index)


def randn_bf16(gen, shape, device, scale=1.0):
    x = torch.randn(shape, generator=gen, device=device, dtype=torch.float32) * scale
    return x.to(torch.bfloat16)
