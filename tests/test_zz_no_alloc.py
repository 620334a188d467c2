"""bc_decode_attn_static: decode attention whose split-K scratch is the array built into the
library, for callers that are not allowed to allocate device memory (a serving process with a
frozen allocator, a plug-in that only receives tensors and a stream).  The paper has no
counterpart; the call must return what bc_decode_attn returns, which is what the CPU oracle's
plain softmax attention over the cache content gives.

This file is named so that pytest collects it last: if it fails under `-x`, every other test has
already run.  It creates its own caches and depends on nothing the other tests leave behind, so it
passes alone in a fresh process as well as after them.
"""
import math

import numpy as np
import pytest
import torch

from paper_2510_13797_b200 import binding as B
from tests.harness import Pair, assert_close, randn_bf16

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _filled_pair(Hkv, G, D, ps, c, plens, seed):
    """A cache (CUDA side and oracle side) with prompts stored: sequences long enough to be split
    over many thread blocks."""
    n = len(plens)
    g = torch.Generator(device=DEV); g.manual_seed(seed)
    pages = sum(-(-p // ps) for p in plens) + n * (-(-c // ps) + 4)
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=n, num_pages=pages, max_pages_per_seq=max(-(-p // ps) for p in plens) + -(-c // ps) + 4,
                c_default=c, device=DEV)
    slots = list(range(n))
    pair.open(slots, plens)
    pair.prefill(0, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    return pair, slots, g


@pytest.mark.parametrize("Hkv,G,D,ctas", [(8, 4, 128, 0), (2, 2, 64, 0), (2, 16, 128, 0), (8, 4, 128, 200), (1, 6, 128, 7)])
def test_static_scratch_entry_point_against_the_oracle(Hkv, G, D, ctas):
    """Outputs of the static entry point against the CPU oracle (and against bc_decode_attn), on
    calls in a row that find the previous call's partials in the shared array: a plain call, the
    same again, a beacon-query call with the extra entry, and a call after the cache has changed.
    ctas = 200 asks for more thread blocks than the built-in array is sized for: the call must
    clamp to its limit; ctas = 7 splits every sequence over few, large pieces."""
    ps, c = 16, 16
    plens = [700, 333, 1030, 48, 1, 257]
    pair, slots, g = _filled_pair(Hkv, G, D, ps, c, plens, seed=99)
    n, Hq = len(plens), Hkv * G
    scale = 1.0 / math.sqrt(D)
    if ctas:
        pair.gpu.bc_set_attn_ctas(ctas)
    for call in range(4):
        if call == 3:
            for _ in range(c):
                pair.append(0, slots, randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV))
            pair.compress(0, slots, randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV))
            pair.append(0, slots, randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV))
        q = randn_bf16(g, (n, Hq, D), DEV)
        ek, ev = (randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV)) if call == 2 else (None, None)
        got, ref = pair.attend(0, slots, q, scale, ek, ev, static=True)
        plain, _ = pair.attend(0, slots, q, scale, ek, ev)
        torch.cuda.synchronize()
        assert_close(got, ref, f"static call {call} vs oracle")
        assert_close(got, plain.to(torch.float64).cpu().numpy(), f"static call {call} vs bc_decode_attn")
    pair.check_state()


def test_static_scratch_calls_allocate_nothing():
    """After a first call (which looks the array's address up), further calls leave the device's free
    memory and torch's allocator untouched."""
    pair, slots, g = _filled_pair(8, 4, 128, 16, 16, [900, 400, 77], seed=5)
    q = randn_bf16(g, (3, 32, 128), DEV)
    out = pair.gpu.new_out(3)
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    pair.gpu.bc_decode_attn_static(0, sl, q, out, 0.1)
    torch.cuda.synchronize()
    free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(5):
        pair.gpu.bc_decode_attn_static(0, sl, q, out, 0.1)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0


def test_static_scratch_shared_by_two_caches_with_a_clear_between():
    """Two caches use the one built-in array in turn on one stream.  bc_clear_error of the cache
    that has used it zeroes the shared ticket counters (a write to the array, ordered by the stream);
    bc_clear_error of a cache that has not used it since its last clear leaves the array alone.
    Every result must still be the oracle's."""
    a, slots_a, g = _filled_pair(8, 4, 128, 16, 16, [640, 1200, 35], seed=11)
    b, slots_b, _ = _filled_pair(2, 6, 128, 8, 8, [300, 2000], seed=12)
    for rnd in range(3):
        qa, qb = randn_bf16(g, (3, 32, 128), DEV), randn_bf16(g, (2, 12, 128), DEV)
        got_a, ref_a = a.attend(0, slots_a, qa, 0.09, static=True)
        if rnd == 1:
            a.gpu.bc_clear_error()          # a has used the array: its counters are zeroed (they are zero anyway)
        got_b, ref_b = b.attend(0, slots_b, qb, 0.09, static=True)
        if rnd == 2:
            a.gpu.bc_clear_error()          # b's launch is enqueued before the reset on the same stream: ordered
            b.gpu.bc_clear_error()
        got_a2, ref_a2 = a.attend(0, slots_a, qa, 0.09, static=True)
        torch.cuda.synchronize()
        assert_close(got_a, ref_a, f"round {rnd}: cache a"); assert_close(got_b, ref_b, f"round {rnd}: cache b")
        assert_close(got_a2, ref_a2, f"round {rnd}: cache a again")
    assert a.gpu.bc_poll_error()[0] == 0 and b.gpu.bc_poll_error()[0] == 0


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
