"""bc_decode_attn_static: decode attention whose split-K scratch is the array built into the
library, for callers that are not allowed to allocate device memory (a serving process with a
frozen allocator, a plug-in that only receives tensors and a stream).  The paper has no
counterpart; the call must return what bc_decode_attn returns.

This file is named so that pytest collects it last: if it fails under `-x`, every other test has
already run.  It creates its own cache and depends on nothing the other tests leave behind, so it
passes alone in a fresh process as well as after them.
"""
import math

import numpy as np
import pytest
import torch

from paper_2510_13797_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda"
ABS_TOL, REL_TOL = 2e-2, 1e-2      # the tolerance of the parity tests


def _close(a, b, what):
    a = a.float().cpu().numpy().astype(np.float64)
    b = b.float().cpu().numpy().astype(np.float64)
    err = np.abs(a - b).max(axis=-1)
    scale = np.maximum(np.abs(b).max(axis=-1), 1e-6)
    assert np.all(np.isfinite(a)), what
    assert err.max() <= ABS_TOL and (err / scale).max() <= REL_TOL, f"{what}: abs {err.max():.3e}"


def test_static_scratch_entry_point_matches_workspace_entry_point():
    Hkv, G, D, ps, c = 8, 4, 128, 16, 16
    plens = [700, 333, 1030, 48]           # long enough that sequences are split over many blocks
    n = len(plens)
    g = torch.Generator(device=DEV); g.manual_seed(99)
    rnd = lambda *shape: torch.randn(shape, generator=g, device=DEV).to(torch.bfloat16)
    cache = B.Cache(1, Hkv, Hkv * G, D, c, ps, max_seqs=n, num_pages=200, max_pages_per_seq=80)
    slots = torch.arange(n, dtype=torch.int32, device=DEV)
    cache.bc_seq_open(slots, torch.tensor(plens, dtype=torch.int32, device=DEV))
    cu = torch.tensor(np.concatenate([[0], np.cumsum(plens)]), dtype=torch.int32, device=DEV)
    cache.bc_prefill(0, slots, cu, sum(plens), rnd(sum(plens), Hkv, D), rnd(sum(plens), Hkv, D))
    scale = 1.0 / math.sqrt(D)
    # two calls in a row (the second one finds the first one's partials in the shared scratch),
    # then a beacon-query call with the extra entry, then a call after the cache has changed
    for call in range(4):
        if call == 3:
            for _ in range(c):
                cache.bc_append(0, slots, rnd(n, Hkv, D), rnd(n, Hkv, D))
            cache.bc_compress(0, slots, rnd(n, Hkv, D), rnd(n, Hkv, D))
        q = rnd(n, Hkv * G, D)
        ek, ev = (rnd(n, Hkv, D), rnd(n, Hkv, D)) if call == 2 else (None, None)
        want, got = cache.new_out(n), cache.new_out(n)
        cache.bc_decode_attn(0, slots, q, want, scale, ek, ev)
        cache.bc_decode_attn_static(0, slots, q, got, scale, ek, ev)
        torch.cuda.synchronize()
        _close(got, want, f"call {call}")
    assert cache.bc_poll_error()[0] == 0


def test_static_scratch_entry_point_rejects_oversized_calls():
    cache = B.Cache(1, 1, 2, 64, 1, 16, max_seqs=200, num_pages=8, max_pages_per_seq=4)
    n = 129                                  # one more than BC_STATIC_MAX_BATCH
    slots = torch.arange(n, dtype=torch.int32, device=DEV)
    q = torch.zeros((n, 2, 64), dtype=torch.bfloat16, device=DEV)
    out = torch.full((n, 2, 64), 7.0, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(B.BreadcrumbsError) as e:
        cache.bc_decode_attn_static(0, slots, q, out, 1.0)
    assert e.value.status == B.BC_ERR_TOO_LARGE
    torch.cuda.synchronize()
    assert float(out.min()) == 7.0           # nothing was enqueued
    # the largest allowed batch is accepted (closed slots: zeros)
    cache.bc_decode_attn_static(0, slots[:128], q[:128], out[:128], 1.0)
    torch.cuda.synchronize()
    assert float(out[:128].abs().max()) == 0.0 and float(out[128:].min()) == 7.0
