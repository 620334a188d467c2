"""ctypes binding of libbreadcrumbs.so: argument marshalling only.

Function names and argument order mirror include/breadcrumbs.h.  Tensors are
torch CUDA tensors used purely as device buffers; every step of the hot path
runs inside the library's kernels.  If the shared library is missing the import
of `lib()` raises: there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

from . import build as _build

# status codes and flags of breadcrumbs.h
BC_OK = 0
BC_ERR_INVALID_ARG, BC_ERR_BAD_SLOT, BC_ERR_NO_PAGES, BC_ERR_CAPACITY = -1, -2, -3, -4
BC_ERR_WINDOW_NOT_FULL, BC_ERR_WINDOW_FULL, BC_ERR_ORDER, BC_ERR_CUDA = -5, -6, -7, -8
BC_ERR_UNSUPPORTED, BC_ERR_TIMEOUT, BC_ERR_TOO_LARGE, BC_ERR_DEBUG_CHECK = -9, -10, -11, -12
BC_FLAG_OUT_F32, BC_FLAG_ATTN_REFERENCE, BC_FLAG_HOST_PIPELINED, BC_FLAG_DEBUG_BOUNDS = 1, 2, 4, 8
STATUS_NAMES = {0: "OK", -1: "INVALID_ARG", -2: "BAD_SLOT", -3: "NO_PAGES", -4: "CAPACITY",
                -5: "WINDOW_NOT_FULL", -6: "WINDOW_FULL", -7: "ORDER", -8: "CUDA",
                -9: "UNSUPPORTED", -10: "TIMEOUT", -11: "TOO_LARGE", -12: "DEBUG_CHECK"}


class BcConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("layers", "kv_heads", "q_heads", "head_dim", "c_default", "page_size", "max_seqs",
                 "num_pages", "max_pages_per_seq", "max_entries_per_seq")] + [("flags", C.c_uint32)]


class BcSeqState(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("open", "prompt_len", "n_beacons", "window_len", "c", "t",
                 "n_prompt_pages", "n_beacon_pages", "n_window_pages")]


class BreadcrumbsError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        super().__init__(f"{where}: BC_ERR_{STATUS_NAMES.get(status, status)}")


_LIB = None

# every symbol breadcrumbs.h declares: name -> (restype, argtypes)
_P, _I32, _I64, _F = C.c_void_p, C.c_int32, C.c_int64, C.c_float
SYMBOLS = {
    "bc_version": (_I32, []),
    "bc_cache_query_bytes": (_I32, [C.POINTER(BcConfig), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]),
    "bc_cache_create": (_I32, [C.POINTER(BcConfig), _P, _P, _P, _P, C.POINTER(_P)]),
    "bc_cache_destroy": (_I32, [_P]),
    "bc_seq_open": (_I32, [_P, _P, _P, _P, _I32, _P]),
    "bc_prefill": (_I32, [_P, _I32, _P, _P, _I32, _I32, _P, _P, _P]),
    "bc_restore": (_I32, [_P, _I32, _P, _I32, _P, _I32, _I32, _P, _P, _P, _P, _P]),
    "bc_append": (_I32, [_P, _I32, _P, _I32, _P, _P, _P]),
    "bc_decode_attn": (_I32, [_P, _I32, _P, _I32, _P, _P, _F, _P, _P, _P]),
    "bc_decode_step": (_I32, [_P, _I32, _P, _I32, _P, _P, _P, _P, _F, _P]),
    "bc_host_outputs_ready": (_I32, [_P, _P]),
    "bc_fill_step_host": (_I32, [_P, _I32, _P, _I32, _P, _P, _P, _P, _P, _P, _P, _P, _F, _P]),
    "bc_decode_attn_pair": (_I32, [_P, _I32, _P, _I32, _P, _P, _P, _P, _F, _P, _P, _P]),
    "bc_decode_attn_static": (_I32, [_P, _I32, _P, _I32, _P, _P, _F, _P, _P, _P]),
    "bc_mask_attn_query_bytes": (_I32, [_I32, _I32, _I32, _I32, _I64, _I64, _I64, C.POINTER(C.c_size_t)]),
    "bc_mask_attn_forward": (_I32, [_I32, _I32, _I32, _I32, _I32, C.POINTER(_I32), C.POINTER(_I32)] + [_P] * 10
                             + [_F, _P, C.c_size_t, _P]),
    "bc_mask_attn_status": (_I32, [_P, _I32, _I32, _I32, _I64, _I64, _I64, _P, C.POINTER(_I32)]),
    "bc_distill_loss": (_I32, [_I32, _P, _I64, _I32, _I32, _P, _P, _P, _P, _P, _P, _P]),
    "bc_compress": (_I32, [_P, _I32, _P, _I32, _P, _P, _P]),
    "bc_seq_close": (_I32, [_P, _P, _I32, _P]),
    "bc_decode_step_host": (_I32, [_P, _I32, _P, _I32, _P, _P, _P, _P, _F, _P]),
    "bc_compress_step_host": (_I32, [_P, _I32, _P, _I32, _P, _P, _P, _P, _F, _P]),
    "bc_get_state": (_I32, [_P, _I32, C.POINTER(BcSeqState), C.POINTER(_I32), _I32, _P]),
    "bc_get_free_list": (_I32, [_P, C.POINTER(_I32), C.POINTER(_I32), _P]),
    "bc_poll_error": (_I32, [_P, C.POINTER(_I32), C.POINTER(_I32), C.POINTER(_I64), _P]),
    "bc_clear_error": (_I32, [_P, _P]),
    "bc_export_seq": (_I32, [_P, _I32, _I32, _P, _P, _I32, _P]),
    "bc_set_attn_ctas": (_I32, [_P, _I32]),
    "bc_attn_timeline": (_I32, [_P, _P, _I32]),
    "bc_set_wait_limit": (_I32, [_P, C.c_uint32]),
    "bc_mask_attn_set_wait_limit": (_I32, [C.c_uint32]),
    "bc_profile_enable": (_I32, [_P, _I32]),
    "bc_profile_read": (_I32, [_P, C.POINTER(_I32), C.POINTER(_F)]),
    "bc_probe_read_stream": (_I32, [_P, C.c_size_t, _P]),
    "bc_fill_step": (_I32, [_P, _I32, _P, _I32, _P, _P, _P, _P, _P, _P, _P, _P, _F, _P]),
    "bc_add_rmsnorm": (_I32, [_P, _P, _P, _I32, _I32, _F, _P, _P, _P]),
    "bc_swiglu": (_I32, [_P, _I32, _I32, _P, _P]),
    "bc_argmax": (_I32, [_P, _I32, _I32, _P, _P]),
    "bc_rope_split": (_I32, [_P, _P, _P, _I32, _F, _P, _P, _P, _P]),
    "bc_rope_decode_step": (_I32, [_P, _I32, _P, _I32, _P, _P, _F, _P, _F, _P]),
    "bc_kernel_launches": (_I64, [_P]),
    "bc_last_cuda_error": (_I32, [_P]),
    "bc_status_string": (C.c_char_p, [_I32]),
}


def lib() -> C.CDLL:
    """Loads libbreadcrumbs.so (building it first if sources are newer).  Raises if unavailable."""
    global _LIB
    if _LIB is None:
        path = _build.LIB_PATH
        if not os.path.exists(path) or os.environ.get("BC_REBUILD"):
            path = _build.build_library()
        if not os.path.exists(path):
            raise RuntimeError("libbreadcrumbs.so is missing and could not be built; there is no fallback path")
        handle = C.CDLL(path)
        for name, (res, args) in SYMBOLS.items():
            fn = getattr(handle, name)
            fn.restype, fn.argtypes = res, args
        _LIB = handle
    return _LIB


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream) -> C.c_void_p:
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _check(status, where):
    if status != BC_OK:
        raise BreadcrumbsError(status, where)


class Cache:
    """Owns the three device buffers (as torch tensors) and the library handle."""

    def __init__(self, layers, kv_heads, q_heads, head_dim, c_default, page_size, max_seqs, num_pages,
                 max_pages_per_seq, max_entries_per_seq=0, flags=0, device="cuda", stream=None):
        self.cfg = BcConfig(layers, kv_heads, q_heads, head_dim, c_default, page_size, max_seqs, num_pages,
                            max_pages_per_seq, max_entries_per_seq, flags)
        self.device = torch.device(device)
        sizes = [C.c_size_t() for _ in range(3)]
        _check(lib().bc_cache_query_bytes(C.byref(self.cfg), *[C.byref(s) for s in sizes]), "bc_cache_query_bytes")
        self.pool_bytes, self.meta_bytes, self.workspace_bytes = [s.value for s in sizes]
        self.pool = torch.empty(self.pool_bytes, dtype=torch.uint8, device=self.device)
        self.meta = torch.empty(self.meta_bytes, dtype=torch.uint8, device=self.device)
        self.workspace = torch.empty(self.workspace_bytes, dtype=torch.uint8, device=self.device)
        h = C.c_void_p()
        _check(lib().bc_cache_create(C.byref(self.cfg), _ptr(self.pool), _ptr(self.meta), _ptr(self.workspace),
                                     _stream(stream), C.byref(h)), "bc_cache_create")
        self.handle = h
        self.out_dtype = torch.float32 if flags & BC_FLAG_OUT_F32 else torch.bfloat16

    def close(self):
        if getattr(self, "handle", None) and lib is not None:   # at interpreter exit the module may be gone already
            lib().bc_cache_destroy(self.handle)
            self.handle = None

    __del__ = close

    # ---- the calls of breadcrumbs.h, same names -------------------------------------------------
    def bc_seq_open(self, slots, prompt_lens, c_per_seq=None, stream=None):
        _check(lib().bc_seq_open(self.handle, _ptr(slots), _ptr(prompt_lens), _ptr(c_per_seq), slots.numel(),
                                 _stream(stream)), "bc_seq_open")

    def bc_prefill(self, layer, slots, cu_prompt_lens, total_tokens, k, v, stream=None):
        _check(lib().bc_prefill(self.handle, layer, _ptr(slots), _ptr(cu_prompt_lens), slots.numel(), total_tokens,
                                _ptr(k), _ptr(v), _stream(stream)), "bc_prefill")

    def bc_restore(self, layer, slots, cu_tokens, total_tokens, total_beacons, tok_k, tok_v, beacon_k, beacon_v, stream=None):
        _check(lib().bc_restore(self.handle, layer, _ptr(slots), slots.numel(), _ptr(cu_tokens), total_tokens, total_beacons,
                                _ptr(tok_k), _ptr(tok_v), _ptr(beacon_k), _ptr(beacon_v), _stream(stream)), "bc_restore")

    def bc_append(self, layer, slots, k, v, stream=None):
        _check(lib().bc_append(self.handle, layer, _ptr(slots), slots.numel(), _ptr(k), _ptr(v), _stream(stream)),
               "bc_append")

    def bc_decode_attn(self, layer, slots, q, out, sm_scale, extra_k=None, extra_v=None, stream=None):
        _check(lib().bc_decode_attn(self.handle, layer, _ptr(slots), slots.numel(), _ptr(q), _ptr(out), sm_scale,
                                    _ptr(extra_k), _ptr(extra_v), _stream(stream)), "bc_decode_attn")

    def bc_host_outputs_ready(self, stream=None):
        _check(lib().bc_host_outputs_ready(self.handle, _stream(stream)), "bc_host_outputs_ready")

    def bc_fill_step_host(self, layer, slots, q, k, v, beacon_q, beacon_k, beacon_v, out, out_beacon, sm_scale, stream=None):
        _check(lib().bc_fill_step_host(self.handle, layer, _ptr(slots), slots.numel(), _ptr(q), _ptr(k), _ptr(v), _ptr(beacon_q),
                                       _ptr(beacon_k), _ptr(beacon_v), _ptr(out), _ptr(out_beacon), sm_scale, _stream(stream)),
               "bc_fill_step_host")

    def bc_decode_attn_pair(self, layer, slots, q, out, beacon_q, out_beacon, sm_scale, beacon_k, beacon_v, stream=None):
        _check(lib().bc_decode_attn_pair(self.handle, layer, _ptr(slots), slots.numel(), _ptr(q), _ptr(out), _ptr(beacon_q),
                                         _ptr(out_beacon), sm_scale, _ptr(beacon_k), _ptr(beacon_v), _stream(stream)),
               "bc_decode_attn_pair")

    def bc_decode_step(self, layer, slots, q, k, v, out, sm_scale, stream=None):
        """bc_append(k, v) + bc_decode_attn(q) in one launch."""
        _check(lib().bc_decode_step(self.handle, layer, _ptr(slots), slots.numel(), _ptr(q), _ptr(k), _ptr(v), _ptr(out),
                                    sm_scale, _stream(stream)), "bc_decode_step")

    def bc_fill_step(self, layer, slots, q, k, v, beacon_q, beacon_k, beacon_v, out, out_beacon, sm_scale, stream=None):
        """The step that fills a window: bc_append + bc_decode_attn_pair + bc_compress, the append inside the attention launch."""
        _check(lib().bc_fill_step(self.handle, layer, _ptr(slots), slots.numel(), _ptr(q), _ptr(k), _ptr(v), _ptr(beacon_q),
                                  _ptr(beacon_k), _ptr(beacon_v), _ptr(out), _ptr(out_beacon), sm_scale, _stream(stream)),
               "bc_fill_step")

    def bc_rope_split(self, qkv, positions, theta, q_out, k_out, v_out, stream=None):
        """Rotary embedding of the q and k heads of a packed QKV projection, split into the three arrays the cache calls take."""
        _check(lib().bc_rope_split(self.handle, _ptr(qkv), _ptr(positions), positions.numel(), theta, _ptr(q_out), _ptr(k_out),
                                   _ptr(v_out), _stream(stream)), "bc_rope_split")

    def bc_rope_decode_step(self, layer, slots, qkv, positions, theta, out, sm_scale, stream=None):
        """bc_rope_split + bc_decode_step: a layer's decode step straight from the packed QKV projection."""
        _check(lib().bc_rope_decode_step(self.handle, layer, _ptr(slots), slots.numel(), _ptr(qkv), _ptr(positions), theta,
                                         _ptr(out), sm_scale, _stream(stream)), "bc_rope_decode_step")

    def bc_decode_attn_static(self, layer, slots, q, out, sm_scale, extra_k=None, extra_v=None, stream=None):
        """bc_decode_attn with the split-K scratch taken from the array built into the library, for callers
        that may not allocate device memory.  At most 128 sequences per call; calls share the scratch."""
        _check(lib().bc_decode_attn_static(self.handle, layer, _ptr(slots), slots.numel(), _ptr(q), _ptr(out),
                                           sm_scale, _ptr(extra_k), _ptr(extra_v), _stream(stream)),
               "bc_decode_attn_static")

    def bc_compress(self, layer, slots, beacon_k, beacon_v, stream=None):
        _check(lib().bc_compress(self.handle, layer, _ptr(slots), slots.numel(), _ptr(beacon_k), _ptr(beacon_v),
                                 _stream(stream)), "bc_compress")

    def bc_seq_close(self, slots, stream=None):
        _check(lib().bc_seq_close(self.handle, _ptr(slots), slots.numel(), _stream(stream)), "bc_seq_close")

    def bc_decode_step_host(self, layer, slots, q_host, k_host, v_host, out_host, sm_scale, stream=None):
        _check(lib().bc_decode_step_host(self.handle, layer, _ptr(slots), slots.numel(), _ptr(q_host), _ptr(k_host),
                                         _ptr(v_host), _ptr(out_host), sm_scale, _stream(stream)),
               "bc_decode_step_host")

    def bc_compress_step_host(self, layer, slots, bq_host, bk_host, bv_host, out_host, sm_scale, stream=None):
        _check(lib().bc_compress_step_host(self.handle, layer, _ptr(slots), slots.numel(), _ptr(bq_host),
                                           _ptr(bk_host), _ptr(bv_host), _ptr(out_host), sm_scale, _stream(stream)),
               "bc_compress_step_host")

    def bc_get_state(self, slot, stream=None):
        st = BcSeqState()
        cap = self.cfg.max_pages_per_seq
        pages = (C.c_int32 * cap)()
        _check(lib().bc_get_state(self.handle, slot, C.byref(st), pages, cap, _stream(stream)), "bc_get_state")
        if not st.open:
            return None
        p = list(pages)
        a, b, w = st.n_prompt_pages, st.n_beacon_pages, st.n_window_pages
        return dict(prompt_len=st.prompt_len, n_beacons=st.n_beacons, window_len=st.window_len, c=st.c, t=st.t,
                    prompt_pages=p[:a], beacon_pages=p[a:a + b], window_pages=p[a + b:a + b + w])

    def bc_get_free_list(self, stream=None):
        pages = (C.c_int32 * self.cfg.num_pages)()
        count = C.c_int32()
        _check(lib().bc_get_free_list(self.handle, pages, C.byref(count), _stream(stream)), "bc_get_free_list")
        return list(pages[:count.value])

    def bc_poll_error(self, stream=None):
        code, slot, call = C.c_int32(), C.c_int32(), C.c_int64()
        _check(lib().bc_poll_error(self.handle, C.byref(code), C.byref(slot), C.byref(call), _stream(stream)),
               "bc_poll_error")
        return code.value, slot.value, call.value

    def bc_clear_error(self, stream=None):
        _check(lib().bc_clear_error(self.handle, _stream(stream)), "bc_clear_error")

    def bc_export_seq(self, layer, slot, capacity, stream=None):
        shape = (capacity, self.cfg.kv_heads, self.cfg.head_dim)
        k = torch.zeros(shape, dtype=torch.bfloat16, device=self.device)
        v = torch.zeros(shape, dtype=torch.bfloat16, device=self.device)
        _check(lib().bc_export_seq(self.handle, layer, slot, _ptr(k), _ptr(v), capacity, _stream(stream)),
               "bc_export_seq")
        return k, v

    def bc_set_attn_ctas(self, ctas):
        _check(lib().bc_set_attn_ctas(self.handle, ctas), "bc_set_attn_ctas")

    def bc_set_wait_limit(self, polls):
        _check(lib().bc_set_wait_limit(self.handle, polls), "bc_set_wait_limit")

    def bc_attn_timeline(self, words, blocks=0):
        """words: uint64/int64 CUDA tensor of at least blocks * 16 elements, or None to switch it off."""
        _check(lib().bc_attn_timeline(self.handle, _ptr(words), blocks), "bc_attn_timeline")

    def bc_profile_enable(self, max_launches):
        _check(lib().bc_profile_enable(self.handle, max_launches), "bc_profile_enable")

    def bc_profile_read(self):
        n, ms = C.c_int32(), C.c_float()
        _check(lib().bc_profile_read(self.handle, C.byref(n), C.byref(ms)), "bc_profile_read")
        return n.value, ms.value

    def bc_kernel_launches(self):
        return lib().bc_kernel_launches(self.handle)

    # ---- convenience ------------------------------------------------------------------------------
    def new_out(self, n):
        return torch.empty((n, self.cfg.q_heads, self.cfg.head_dim), dtype=self.out_dtype, device=self.device)


def bc_mask_attn_forward(prompt_lens, token_lens, c, prompt_k, prompt_v, tok_q, tok_k, tok_v, beacon_q, beacon_k,
                         beacon_v, sm_scale, stream=None, check=True):
    """The mask form of a batch of trajectories (breadcrumbs.h): returns (out_tok, out_beacon).

    prompt_lens, token_lens: Python lists, one entry per sequence.  Tensors are packed bf16 CUDA
    tensors as the header describes; beacon tensors may be None when no sequence has a beacon."""
    n = len(prompt_lens)
    q_heads, kv_heads, head_dim = tok_q.shape[1], tok_k.shape[1], tok_q.shape[2]
    cu_p = (C.c_int32 * (n + 1))(0, *list(__import__("itertools").accumulate(prompt_lens)))
    cu_t = (C.c_int32 * (n + 1))(0, *list(__import__("itertools").accumulate(token_lens)))
    total_b = sum(t // c for t in token_lens) if c > 1 else 0
    size = C.c_size_t()
    _check(lib().bc_mask_attn_query_bytes(n, q_heads, kv_heads, head_dim, cu_p[n], cu_t[n], total_b, C.byref(size)),
           "bc_mask_attn_query_bytes")
    ws = torch.empty(size.value, dtype=torch.uint8, device=tok_q.device)
    out_tok = torch.empty_like(tok_q)
    out_bea = torch.empty((total_b, q_heads, head_dim), dtype=tok_q.dtype, device=tok_q.device)
    _check(lib().bc_mask_attn_forward(n, q_heads, kv_heads, head_dim, c, cu_p, cu_t, _ptr(prompt_k), _ptr(prompt_v),
                                      _ptr(tok_q), _ptr(tok_k), _ptr(tok_v), _ptr(beacon_q), _ptr(beacon_k),
                                      _ptr(beacon_v), _ptr(out_tok), _ptr(out_bea), sm_scale, _ptr(ws), size.value,
                                      _stream(stream)), "bc_mask_attn_forward")
    if check:
        code = C.c_int32()
        _check(lib().bc_mask_attn_status(_ptr(ws), n, q_heads, kv_heads, cu_p[n], cu_t[n], total_b, _stream(stream),
                                         C.byref(code)), "bc_mask_attn_status")
        _check(code.value, "bc_mask_attn_forward (device)")
    return out_tok, out_bea


def bc_probe_read_stream(buf, stream=None):
    """Reads the CUDA tensor `buf` once with the attention kernel's copy pattern (breadcrumbs.h)."""
    _check(lib().bc_probe_read_stream(_ptr(buf), buf.numel() * buf.element_size(), _stream(stream)), "bc_probe_read_stream")


def bc_add_rmsnorm(h, delta, weight, eps, h_out, normed_out, stream=None):
    """h' = h + delta (bf16), normed_out = rmsnorm(h') * weight (breadcrumbs.h); delta, weight, h_out may be None."""
    n, hidden = h.shape[0], h.shape[-1]
    _check(lib().bc_add_rmsnorm(_ptr(h), _ptr(delta), _ptr(weight), n, hidden, eps, _ptr(h_out), _ptr(normed_out), _stream(stream)),
           "bc_add_rmsnorm")


def bc_swiglu(gate_up, out, stream=None):
    """out = silu(gate) * up for packed rows [gate | up] (breadcrumbs.h)."""
    _check(lib().bc_swiglu(_ptr(gate_up), gate_up.shape[0], gate_up.shape[-1] // 2, _ptr(out), _stream(stream)), "bc_swiglu")


def bc_argmax(logits, out, stream=None):
    """out[r] (int64) = lowest index of the maximum of row r of bf16 logits (breadcrumbs.h)."""
    _check(lib().bc_argmax(_ptr(logits), logits.shape[0], logits.shape[-1], _ptr(out), _stream(stream)), "bc_argmax")


def bc_distill_loss(cu_rows, student_logits, teacher_idx, teacher_logprob, with_grad=False, stream=None):
    """Eq. 1 (breadcrumbs.h): returns (loss [1] fp32, row_loss [rows] fp32, grad or None).

    cu_rows: int32 CUDA tensor [n_traj + 1]; student_logits bf16 [rows, vocab]; teacher_idx int32 and
    teacher_logprob fp32 [rows, top_k]."""
    rows, vocab = student_logits.shape
    top_k = teacher_idx.shape[1]
    dev = student_logits.device
    row_loss = torch.empty(rows, dtype=torch.float32, device=dev)
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    grad = torch.empty_like(student_logits) if with_grad else None
    _check(lib().bc_distill_loss(cu_rows.numel() - 1, _ptr(cu_rows), rows, vocab, top_k, _ptr(student_logits),
                                 _ptr(teacher_idx), _ptr(teacher_logprob), _ptr(row_loss), _ptr(loss), _ptr(grad),
                                 _stream(stream)), "bc_distill_loss")
    return loss, row_loss, grad
