"""GPU parity: the CUDA path (through the C ABI) against the fp64 CPU oracle.

Attention outputs: per head vector, max-abs error <= 2e-2 and <= 1e-2 of the vector's largest
magnitude.  Bookkeeping (lengths, page lists, free stack, latched error) and stored content:
bit-exact.
"""
import math

import numpy as np
import pytest
import torch

from oracle.breadcrumbs_oracle import closed_form_length
from paper_2510_13797_b200 import binding as B
from paper_2510_13797_b200.workloads import InputStream, make_workload
from oracle.paging_model import OK
from tests.harness import Pair, assert_close, f64, randn_bf16

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _gen(seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return g


def run_decode(pair: Pair, slots, plens, cs, steps, seed, sm_scale, check_state_every=1, compare_every=1,
               k_scale=1.0, beacon_k_scale=1.0, content_every=0):
    """Lock-step decode of `slots`: append, attend, and for every sequence whose window is full the
    beacon-query attention followed by compress.  Returns the worst errors seen."""
    g = _gen(seed)
    L, Hkv, Hq, D = pair.L, pair.Hkv, pair.Hq, pair.D
    n = len(slots)
    assert pair.open(slots, plens, cs) == ["OK"] * n
    for l in range(L):
        pair.prefill(l, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV, k_scale),
                     randn_bf16(g, (sum(plens), Hkv, D), DEV))
    pair.check_state()
    worst = [0.0, 0.0]
    for step in range(1, steps + 1):
        for l in range(L):
            assert pair.append(l, slots, randn_bf16(g, (n, Hkv, D), DEV, k_scale),
                               randn_bf16(g, (n, Hkv, D), DEV)) == ["OK"] * n
            q = randn_bf16(g, (n, Hq, D), DEV)
            if step % compare_every == 0 or step == steps:
                out, ref = pair.attend(l, slots, q, sm_scale)
                a, r = assert_close(out, ref, f"step {step} layer {l}")
                worst = [max(worst[0], a), max(worst[1], r)]
        full = [i for i, s in enumerate(slots) if cs[i] > 1 and step % cs[i] == 0]
        if full:
            fs = [slots[i] for i in full]
            for l in range(L):
                qb = randn_bf16(g, (len(fs), Hq, D), DEV)
                bk = randn_bf16(g, (len(fs), Hkv, D), DEV, beacon_k_scale)
                bv = randn_bf16(g, (len(fs), Hkv, D), DEV)
                out, ref = pair.attend(l, fs, qb, sm_scale, bk, bv)
                a, r = assert_close(out, ref, f"beacon query, step {step} layer {l}")
                worst = [max(worst[0], a), max(worst[1], r)]
                assert pair.compress(l, fs, bk, bv) == ["OK"] * len(fs)
        if step % check_state_every == 0 or step == steps:
            pair.check_state()
            for i, s in enumerate(slots):
                st = pair.gpu.bc_get_state(s)
                assert st["prompt_len"] + st["n_beacons"] + st["window_len"] == closed_form_length(plens[i], step, cs[i])
        if content_every and (step % content_every == 0 or step == steps):
            for s in slots:
                for l in range(L):
                    pair.check_content(l, s)
    return worst


def test_tiny_config_every_step():
    """Benchmark configuration 'tiny': every step's output, lengths, page lists and content."""
    w = make_workload("tiny")
    pair = Pair(1, w.kv_heads, w.q_heads, w.head_dim, w.page_size, max_seqs=2, num_pages=64, max_pages_per_seq=16)
    worst = run_decode(pair, [0], w.prompt_lens, w.cs, w.steps, seed=1, sm_scale=w.sm_scale, content_every=37)
    st = pair.gpu.bc_get_state(0)
    assert (st["prompt_len"], st["n_beacons"], st["window_len"], st["t"]) == (64, 32, 0, 512)
    assert pair.close([0]) == ["OK"]
    pair.check_state()
    assert sorted(pair.gpu.bc_get_free_list()) == list(range(64))
    print("tiny worst abs/rel", worst)


@pytest.mark.parametrize("Hkv,G,D,ps,c,plens,steps", [
    (1, 1, 64, 16, 16, [5], 40),
    (1, 2, 128, 4, 6, [0, 1], 30),          # empty prompt, c not a multiple of the page size
    (2, 6, 128, 16, 16, [70, 33, 129], 50),  # the 12/2 head shape of the 1.5B model
    (2, 6, 128, 16, 4, [70, 9], 40),         # c smaller than a page
    (4, 3, 128, 3, 7, [20, 21, 22, 23], 30), # odd page size, odd c
    (8, 4, 128, 2, 2, [40, 17], 24),         # the sweep shape at c = 2
    (8, 4, 128, 32, 32, [64], 70),
    (8, 1, 64, 1, 5, [10, 3], 20),           # one token per page
    (2, 12, 128, 8, 8, [50], 20),            # G > 8: both row halves of the MMA
    (1, 16, 64, 16, 1, [30, 8], 40),         # ratio 1: never compresses, window grows by pages
    (4, 8, 128, 16, 3, [130], 20),
])
def test_shapes_every_step(Hkv, G, D, ps, c, plens, steps):
    n = len(plens)
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=n + 1, num_pages=400, max_pages_per_seq=200)
    run_decode(pair, list(range(n)), plens, [c] * n, steps, seed=7, sm_scale=1.0 / math.sqrt(D), content_every=9)


def test_splits_give_the_same_answer():
    """Any number of thread blocks (hence key splits per sequence) gives the oracle's answer."""
    Hkv, G, D, ps = 8, 4, 128, 16
    plens = [700, 333, 1030]
    n = len(plens)
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=n, num_pages=200, max_pages_per_seq=80, c_default=16)
    g = _gen(3)
    slots = list(range(n))
    assert pair.open(slots, plens) == ["OK"] * n
    pair.prefill(0, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    for _ in range(5):
        pair.append(0, slots, randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV))
    q = randn_bf16(g, (n, Hkv * G, D), DEV)
    ek, ev = randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV)
    outs = []
    for ctas in (1, 2, 3, 7, 64, 148, 304, 0):
        pair.gpu.bc_set_attn_ctas(ctas)
        out, ref = pair.attend(0, slots, q, 1.0 / math.sqrt(D))
        assert_close(out, ref, f"ctas {ctas}")
        outb, refb = pair.attend(0, slots, q, 1.0 / math.sqrt(D), ek, ev)
        assert_close(outb, refb, f"ctas {ctas} with extra entry")
        outs.append(f64(out))
    for o in outs[1:]:
        assert np.abs(o - outs[0]).max() < 4e-3
    pair.check_state()


def test_sharp_and_diffuse_logits():
    """Keys pre-scaled by 1/sqrt(D) with sm_scale 1, beacon keys left N(0,1): logits of the beacons have
    standard deviation sqrt(D), so the softmax mixes a diffuse part and sharp peaks (config 2's recipe)."""
    Hkv, G, D, ps, c = 2, 6, 128, 16, 16
    plens = [256, 100]
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=2, num_pages=200, max_pages_per_seq=100)
    run_decode(pair, [0, 1], plens, [c, c], 100, seed=11, sm_scale=1.0, k_scale=1.0 / math.sqrt(D),
               check_state_every=10, compare_every=1)


def test_multi_layer_order_and_eviction_timing():
    L, Hkv, G, D, ps, c = 3, 2, 2, 64, 4, 4
    pair = Pair(L, Hkv, Hkv * G, D, ps, max_seqs=3, num_pages=64, max_pages_per_seq=32)
    run_decode(pair, [2, 0], [9, 4], [c, c], 21, seed=5, sm_scale=0.125, content_every=4)
    # out-of-order layer calls are refused on the host, before anything is enqueued
    g = _gen(1)
    k = randn_bf16(g, (2, Hkv, D), DEV)
    slots = torch.tensor([2, 0], dtype=torch.int32, device=DEV)
    with pytest.raises(B.BreadcrumbsError) as e:
        pair.gpu.bc_append(1, slots, k, k)
    assert e.value.status == B.BC_ERR_ORDER
    with pytest.raises(B.BreadcrumbsError) as e:
        pair.gpu.bc_compress(2, slots, k, k)
    assert e.value.status == B.BC_ERR_ORDER
    pair.check_state()


def test_ragged_batch_open_close_reuse():
    """Sequences with their own prompt length and ratio finish at different steps; their pages go
    back to the device free list and are reused by sequences opened later."""
    Hkv, G, D, ps = 2, 6, 128, 16
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=6, num_pages=120, max_pages_per_seq=40)
    g = _gen(21)
    rng = np.random.RandomState(21)
    live = {}          # slot -> [P, c, T, t]
    next_open = list(range(6))

    def open_some(slots):
        plens = [int(rng.randint(1, 200)) for _ in slots]
        cs = [int(rng.choice([4, 8, 16])) for _ in slots]
        assert pair.open(slots, plens, cs) == ["OK"] * len(slots)
        pair.prefill(0, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
        for s, p, c in zip(slots, plens, cs):
            live[s] = [p, c, int(rng.randint(5, 60)), 0]

    open_some(next_open[:4])
    for step in range(90):
        slots = sorted(live)
        if not slots:
            break
        n = len(slots)
        pair.append(0, slots, randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV))
        out, ref = pair.attend(0, slots, randn_bf16(g, (n, Hkv * G, D), DEV), 1.0 / math.sqrt(D))
        assert_close(out, ref, f"ragged step {step}")
        for s in slots:
            live[s][3] += 1
        full = [s for s in slots if live[s][3] % live[s][1] == 0]
        if full:
            bk, bv = randn_bf16(g, (len(full), Hkv, D), DEV), randn_bf16(g, (len(full), Hkv, D), DEV)
            out, ref = pair.attend(0, full, randn_bf16(g, (len(full), Hkv * G, D), DEV), 1.0 / math.sqrt(D), bk, bv)
            assert_close(out, ref, f"ragged beacon step {step}")
            pair.compress(0, full, bk, bv)
        done = [s for s in slots if live[s][3] >= live[s][2]]
        if done:
            assert pair.close(done) == ["OK"] * len(done)
            for s in done:
                del live[s]
        if step in (10, 30) :
            free_slots = [s for s in range(6) if s not in live][:2]
            if free_slots:
                open_some(free_slots)
        pair.check_state()
    rest = sorted(live)
    if rest:
        pair.close(rest)
    pair.check_state()
    assert sorted(pair.gpu.bc_get_free_list()) == list(range(120))      # conservation: everything came back


def test_device_side_errors_match_the_model():
    Hkv, G, D, ps = 1, 2, 64, 2
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=4, num_pages=6, max_pages_per_seq=5, max_entries=0)
    g = _gen(2)
    kv = lambda n: (randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV))
    # 3 + 2 pages granted, the third sequence (2 pages) does not fit, the empty one always fits
    assert pair.open([0, 1, 2, 3], [5, 3, 4, 0], [2, 2, 2, 2]) == ["OK", "OK", "NO_PAGES", "OK"]
    pair.prefill(0, [0, 1, 3], [5, 3, 0], *kv(8))
    pair.check_state()
    pair.gpu.bc_clear_error()
    pair.model.first_error = None
    assert pair.append(0, [0, 1, 3], *kv(3)) == ["OK", "NO_PAGES", "NO_PAGES"]   # one page left
    pair.check_state()
    pair.gpu.bc_clear_error(); pair.model.first_error = None
    assert pair.compress(0, [0], *kv(1)) == ["WINDOW_NOT_FULL"]
    pair.check_state()
    pair.gpu.bc_clear_error(); pair.model.first_error = None
    assert pair.append(0, [0], *kv(1)) == ["OK"]
    assert pair.append(0, [0], *kv(1)) == ["WINDOW_FULL"]
    pair.check_state()
    pair.gpu.bc_clear_error(); pair.model.first_error = None
    assert pair.close([2, 1]) == ["BAD_SLOT", "OK"]                              # slot 2 never opened
    pair.check_state()
    pair.gpu.bc_clear_error(); pair.model.first_error = None
    assert pair.compress(0, [0], *kv(1)) == ["OK"]                                # beacon page from the freed ones
    pair.check_state()
    # attention over a slot that is not open reads nothing and returns zeros
    q = randn_bf16(g, (2, Hkv * G, D), DEV)
    out, ref = pair.attend(0, [2, 0], q, 0.125)
    assert_close(out, ref, "closed slot")
    assert float(out[0].abs().max()) == 0.0
    # the evaluation's cache cap: generation-side entries are limited
    pair2 = Pair(1, 1, 2, 64, 4, max_seqs=1, num_pages=16, max_pages_per_seq=8, max_entries=3)
    assert pair2.open([0], [6], [1]) == ["OK"]
    for expect in ("OK", "OK", "OK", "CAPACITY"):
        assert pair2.append(0, [0], *kv(1)) == [expect]
    pair2.check_state()


def test_several_failures_in_one_call_latch_the_lowest_item():
    """The status record after calls with two and three failing items of different kinds, against
    records written out by hand from the rule in breadcrumbs.h (first failing call; within it the
    failing item with the lowest batch index), not against the model."""
    i32 = lambda xs: torch.tensor(xs, dtype=torch.int32, device=DEV)
    z = lambda n: torch.zeros((n, 1, 64), dtype=torch.bfloat16, device=DEV)
    name = lambda cache: (lambda c, s, k: (B.STATUS_NAMES[c], s, k))(*cache.bc_poll_error())
    # open (call 1): item 0 fails at allocation (3 pages of 1, 2 free), item 1 at validation (slot 9), item 2 too (c = 0)
    a = B.Cache(1, 1, 2, 64, 1, 1, max_seqs=4, num_pages=2, max_pages_per_seq=8)
    a.bc_seq_open(i32([3, 9, 1]), i32([3, 1, 1]), i32([1, 1, 0]))
    assert name(a) == ("NO_PAGES", 3, 1)
    assert a.bc_get_free_list() == [1, 0] and all(a.bc_get_state(s) is None for s in range(4))
    # append (call 4): [WINDOW_FULL, OK, BAD_SLOT]; a later call (5) with other failures changes nothing
    b = B.Cache(1, 1, 2, 64, 2, 2, max_seqs=8, num_pages=16, max_pages_per_seq=8)
    b.bc_seq_open(i32([5, 2]), i32([1, 1]))
    b.bc_append(0, i32([5]), z(1), z(1)); b.bc_append(0, i32([5]), z(1), z(1))
    assert name(b) == ("OK", 0, 0)
    b.bc_append(0, i32([5, 2, 7]), z(3), z(3))
    assert name(b) == ("WINDOW_FULL", 5, 4)
    assert b.bc_get_state(2)["window_len"] == 1 and b.bc_get_state(5)["window_len"] == 2
    b.bc_append(0, i32([7, 5]), z(2), z(2))
    assert name(b) == ("WINDOW_FULL", 5, 4)
    # compress (call 3): lowest index, not lowest slot id, not the last failure
    c3 = B.Cache(1, 1, 2, 64, 2, 2, max_seqs=8, num_pages=16, max_pages_per_seq=8)
    c3.bc_seq_open(i32([2]), i32([1])); c3.bc_append(0, i32([2]), z(1), z(1))
    c3.bc_compress(0, i32([6, 2, 0]), z(3), z(3))
    assert name(c3) == ("BAD_SLOT", 6, 3)
    # compress (call 4): allocation failures at items 0 and 1 (no page left), validation failure at item 2
    d = B.Cache(1, 1, 2, 64, 2, 1, max_seqs=4, num_pages=4, max_pages_per_seq=8)
    d.bc_seq_open(i32([0, 1]), i32([0, 0]))
    d.bc_append(0, i32([0, 1]), z(2), z(2)); d.bc_append(0, i32([0, 1]), z(2), z(2))
    assert d.bc_get_free_list() == []
    d.bc_compress(0, i32([1, 0, 3]), z(3), z(3))
    assert name(d) == ("NO_PAGES", 1, 4)
    assert d.bc_get_state(1)["window_len"] == 2 and d.bc_get_state(0)["n_beacons"] == 0
    # close (call 2)
    e = B.Cache(1, 1, 2, 64, 4, 4, max_seqs=4, num_pages=8, max_pages_per_seq=16)
    e.bc_seq_open(i32([0]), i32([0]))
    e.bc_seq_close(i32([3, 0, 2]))
    assert name(e) == ("BAD_SLOT", 3, 2)


def test_host_argument_errors():
    pair = Pair(1, 1, 2, 64, 4, max_seqs=2, num_pages=8, max_pages_per_seq=8)
    slots = torch.tensor([0], dtype=torch.int32, device=DEV)
    k = torch.zeros((1, 1, 64), dtype=torch.bfloat16, device=DEV)
    lib = B.lib()
    assert lib.bc_append(pair.gpu.handle, 0, None, 1, k.data_ptr(), k.data_ptr(), None) == B.BC_ERR_INVALID_ARG
    assert lib.bc_append(pair.gpu.handle, 3, slots.data_ptr(), 1, k.data_ptr(), k.data_ptr(), None) == B.BC_ERR_INVALID_ARG
    assert lib.bc_append(pair.gpu.handle, 0, slots.data_ptr(), 0, k.data_ptr(), k.data_ptr(), None) == B.BC_ERR_INVALID_ARG
    assert lib.bc_append(pair.gpu.handle, 0, slots.data_ptr(), 1, k.data_ptr() + 2, k.data_ptr(), None) == B.BC_ERR_INVALID_ARG
    q = torch.zeros((1, 2, 64), dtype=torch.bfloat16, device=DEV)
    assert lib.bc_decode_attn(pair.gpu.handle, 0, slots.data_ptr(), 1, q.data_ptr(), q.data_ptr(), 1.0,
                              k.data_ptr(), None, None) == B.BC_ERR_INVALID_ARG
    bad = B.BcConfig(1, 3, 6, 128, 1, 16, 4, 16, 8, 0, 0)
    sz = [B.C.c_size_t() for _ in range(3)]
    assert lib.bc_cache_query_bytes(B.C.byref(bad), *[B.C.byref(s) for s in sz]) == B.BC_ERR_UNSUPPORTED
    pair.check_state()


def test_reference_kernel_and_f32_output_agree():
    """The slow device kernel and the fp32 output flag agree with the oracle too."""
    Hkv, G, D, ps, c = 2, 6, 128, 16, 8
    for flags in (B.BC_FLAG_ATTN_REFERENCE, B.BC_FLAG_OUT_F32, B.BC_FLAG_OUT_F32 | B.BC_FLAG_ATTN_REFERENCE):
        pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=2, num_pages=64, max_pages_per_seq=32, flags=flags)
        run_decode(pair, [0, 1], [100, 37], [c, c], 24, seed=13, sm_scale=1.0 / math.sqrt(D), check_state_every=8)


def test_host_buffer_steps_over_two_layers(host_route):
    """Host-buffer steps of a two-layer cache, layer after layer without synchronising in between:
    regular steps (bc_decode_step_host) and window-filling steps (bc_fill_step_host)."""
    L, Hkv, G, D, ps, c = 2, 2, 4, 128, 4, 3
    n, plens = 5, [33, 0, 18, 7, 64]
    pair = Pair(L, Hkv, Hkv * G, D, ps, max_seqs=n, num_pages=160, max_pages_per_seq=32)
    g = _gen(23)
    slots = list(range(n))
    pair.open(slots, plens, [c] * n)
    for l in range(L):
        pair.prefill(l, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    pin = lambda t: t.cpu().pin_memory()
    kv = lambda: (randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV))
    for step in range(1, 11):
        fill = step % c == 0
        ins = [kv() for _ in range(L)]
        bea = [kv() for _ in range(L)] if fill else None
        outs = [torch.empty((n, Hkv * G, D), dtype=torch.bfloat16).pin_memory() for _ in range(L)]
        outs_b = [torch.empty((n, Hkv * G, D), dtype=torch.bfloat16).pin_memory() for _ in range(L)]
        host = [[pin(x) for x in ins[l]] for l in range(L)]
        host_b = [[pin(x) for x in bea[l]] for l in range(L)] if fill else None
        for l in range(L):
            k, v, q = host[l]
            if fill:
                bk, bv, bq = host_b[l]
                pair.gpu.bc_fill_step_host(l, sl, q, k, v, bq, bk, bv, outs[l], outs_b[l], 0.1)
            else:
                pair.gpu.bc_decode_step_host(l, sl, q, k, v, outs[l], 0.1)
        torch.cuda.synchronize()
        pair._append_ok = pair.model.append(slots)
        for l in range(L):
            k, v, q = ins[l]
            for i, s in enumerate(slots):
                pair.seqs[s].append(l, f64(k)[i], f64(v)[i])
            ref = np.stack([pair.seqs[s].attend(l, f64(q)[i], 0.1) for i, s in enumerate(slots)])
            assert_close(outs[l], ref, f"step {step} layer {l}")
        if fill:
            for l in range(L):
                bk, bv, bq = bea[l]
                ref = np.stack([pair.seqs[s].beacon_attend(l, f64(bq)[i], f64(bk)[i], f64(bv)[i], 0.1) for i, s in enumerate(slots)])
                assert_close(outs_b[l], ref, f"beacon of step {step} layer {l}")
            pair.model.compress(slots)
            for l in range(L):
                bk, bv, _ = bea[l]
                for i, s in enumerate(slots):
                    pair.seqs[s].compress(l, f64(bk)[i], f64(bv)[i])
        pair.check_state()
    for l in range(L):
        for s in slots:
            pair.check_content(l, s)


def test_host_buffer_entry_points(host_route):
    """bc_decode_step_host / bc_compress_step_host: same results as the device-pointer calls."""
    Hkv, G, D, ps, c = 2, 6, 128, 16, 4
    n, plens = 3, [40, 7, 90]
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=n, num_pages=64, max_pages_per_seq=32)
    g = _gen(17)
    slots = list(range(n))
    pair.open(slots, plens, [c] * n)
    pair.prefill(0, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    pin = lambda t: t.cpu().pin_memory()
    for step in range(1, 10):
        k, v, q = randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)
        out_h = torch.empty((n, Hkv * G, D), dtype=torch.bfloat16).pin_memory()
        pair.gpu.bc_decode_step_host(0, sl, pin(q), pin(k), pin(v), out_h, 0.1)
        torch.cuda.synchronize()
        # mirror on the oracle
        pair._append_ok = pair.model.append(slots)
        for i, s in enumerate(slots):
            pair.seqs[s].append(0, f64(k)[i], f64(v)[i])
        ref = np.stack([pair.seqs[s].attend(0, f64(q)[i], 0.1) for i, s in enumerate(slots)])
        assert_close(out_h, ref, f"host step {step}")
        if step % c == 0:
            bk, bv, bq = randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)
            pair.gpu.bc_compress_step_host(0, sl, pin(bq), pin(bk), pin(bv), out_h, 0.1)
            torch.cuda.synchronize()
            ref = np.stack([pair.seqs[s].beacon_attend(0, f64(bq)[i], f64(bk)[i], f64(bv)[i], 0.1)
                            for i, s in enumerate(slots)])
            assert_close(out_h, ref, f"host beacon step {step}")
            pair.model.compress(slots)
            for i, s in enumerate(slots):
                pair.seqs[s].compress(0, f64(bk)[i], f64(bv)[i])
        pair.check_state()
    for s in slots:
        pair.check_content(0, s)


def run_decode_fused(pair: Pair, slots, plens, cs, steps, seed, sm_scale, content_every=0):
    """Like run_decode, but every regular step goes through the fused bc_decode_step call."""
    g = _gen(seed)
    L, Hkv, Hq, D = pair.L, pair.Hkv, pair.Hq, pair.D
    n = len(slots)
    assert pair.open(slots, plens, cs) == ["OK"] * n
    for l in range(L):
        pair.prefill(l, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    for step in range(1, steps + 1):
        for l in range(L):
            res, out, ref = pair.step(l, slots, randn_bf16(g, (n, Hq, D), DEV), randn_bf16(g, (n, Hkv, D), DEV),
                                      randn_bf16(g, (n, Hkv, D), DEV), sm_scale)
            assert res == ["OK"] * n
            assert_close(out, ref, f"fused step {step} layer {l}")
        full = [i for i, s in enumerate(slots) if cs[i] > 1 and step % cs[i] == 0]
        if full:
            fs = [slots[i] for i in full]
            for l in range(L):
                qb, bk, bv = randn_bf16(g, (len(fs), Hq, D), DEV), randn_bf16(g, (len(fs), Hkv, D), DEV), randn_bf16(g, (len(fs), Hkv, D), DEV)
                out, ref = pair.attend(l, fs, qb, sm_scale, bk, bv)
                assert_close(out, ref, f"beacon query after fused step {step} layer {l}")
                assert pair.compress(l, fs, bk, bv) == ["OK"] * len(fs)
        pair.check_state()
        if content_every and (step % content_every == 0 or step == steps):
            for s in slots:
                for l in range(L):
                    pair.check_content(l, s)


@pytest.mark.parametrize("L,Hkv,G,D,ps,c,plens,steps", [
    (1, 1, 2, 64, 16, 16, [64], 40),
    (1, 8, 4, 128, 2, 2, [40, 17, 300], 20),       # the sweep shape at c = 2: a window page every other step
    (1, 8, 4, 128, 16, 16, [700, 333, 1030], 36),  # sequences split over several blocks
    (1, 2, 6, 128, 16, 4, [70, 9, 0], 30),         # empty prompt: the first entry of the cache comes from the fused step
    (1, 4, 3, 128, 3, 7, [20, 21, 22, 23], 30),
    (1, 2, 12, 128, 8, 8, [50], 20),               # G > 8
    (1, 1, 16, 64, 16, 1, [30, 8], 40),            # ratio 1: the window grows by pages
    (3, 2, 2, 64, 4, 4, [9, 4], 21),               # three layers: bookkeeping on layer 0, rows on every layer
])
def test_fused_decode_step_every_step(L, Hkv, G, D, ps, c, plens, steps):
    n = len(plens)
    pair = Pair(L, Hkv, Hkv * G, D, ps, max_seqs=n + 1, num_pages=600, max_pages_per_seq=200)
    run_decode_fused(pair, list(range(n)), plens, [c] * n, steps, seed=23, sm_scale=1.0 / math.sqrt(D), content_every=5)


def test_fused_decode_step_refusals_and_block_counts():
    """A refused append inside the fused call leaves that sequence as it was (and attends to it as it
    was); any number of thread blocks gives the same answer."""
    Hkv, G, D, ps = 2, 2, 64, 2
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=3, num_pages=8, max_pages_per_seq=6)
    g = _gen(4)
    assert pair.open([0, 1, 2], [3, 2, 4], [2, 2, 2]) == ["OK"] * 3     # 2 + 1 + 2 pages, 3 left
    pair.prefill(0, [0, 1, 2], [3, 2, 4], randn_bf16(g, (9, Hkv, D), DEV), randn_bf16(g, (9, Hkv, D), DEV))
    mk = lambda n: (randn_bf16(g, (n, Hkv * G, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV))
    for ctas in (1, 3, 148):
        pair.gpu.bc_set_attn_ctas(ctas)
        res, out, ref = pair.step(0, [0, 1, 2], *mk(3), 0.125)
        assert_close(out, ref, f"fused, {ctas} blocks")
        pair.check_state()
        pair.gpu.bc_clear_error(); pair.model.first_error = None
    # by now some windows are full and the pool is nearly empty: refusals must match the model
    res, out, ref = pair.step(0, [0, 1, 2, ][:3], *mk(3), 0.125)
    assert any(r != "OK" for r in res)
    assert_close(out, ref, "fused with refused items")
    pair.check_state()
    for s in (0, 1, 2):
        pair.check_content(0, s)


def test_host_buffer_steps_back_to_back_packed(host_route):
    """Host-buffer steps issued without a synchronisation in between, each with its inputs in one
    packed pinned block k | v | q (moved by a single copy): the copies of a step run on the cache's
    copy stream while the previous step's kernels run, in alternating staging buffers.  Every step's
    output, read after one synchronisation at the end, must match the oracle."""
    Hkv, G, D, ps, c = 2, 4, 128, 16, 4
    n, plens = 4, [300, 7, 90, 513]
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=n, num_pages=128, max_pages_per_seq=48)
    g = _gen(23)
    slots = list(range(n))
    pair.open(slots, plens, [c] * n)
    pair.prefill(0, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)

    def packed(k, v, q):
        nk, nq = k.numel(), q.numel()
        flat = torch.empty(2 * nk + nq, dtype=torch.bfloat16).pin_memory()
        flat[:nk], flat[nk:2 * nk], flat[2 * nk:] = k.reshape(-1).cpu(), v.reshape(-1).cpu(), q.reshape(-1).cpu()
        return flat[:nk].view(k.shape), flat[nk:2 * nk].view(v.shape), flat[2 * nk:].view(q.shape)

    steps, outs, refs = 11, [], []
    inputs = []
    for step in range(1, steps + 1):
        k, v, q = randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)
        beacon = None
        if step % c == 0:
            beacon = (randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV))
        inputs.append((k, v, q, beacon))
    torch.cuda.synchronize()
    for k, v, q, beacon in inputs:                 # the GPU side: nothing waits between the calls
        hk, hv, hq = packed(k, v, q)
        out_h = torch.empty((n, Hkv * G, D), dtype=torch.bfloat16).pin_memory()
        pair.gpu.bc_decode_step_host(0, sl, hq, hk, hv, out_h, 0.1)
        outs.append(out_h)
        if beacon is not None:
            hbk, hbv, hbq = packed(*beacon)
            out_b = torch.empty((n, Hkv * G, D), dtype=torch.bfloat16).pin_memory()
            pair.gpu.bc_compress_step_host(0, sl, hbq, hbk, hbv, out_b, 0.1)
            outs.append(out_b)
    torch.cuda.synchronize()
    for k, v, q, beacon in inputs:                 # the oracle, step by step
        pair._append_ok = pair.model.append(slots)
        for i, s in enumerate(slots):
            pair.seqs[s].append(0, f64(k)[i], f64(v)[i])
        refs.append(np.stack([pair.seqs[s].attend(0, f64(q)[i], 0.1) for i, s in enumerate(slots)]))
        if beacon is not None:
            bk, bv, bq = beacon
            refs.append(np.stack([pair.seqs[s].beacon_attend(0, f64(bq)[i], f64(bk)[i], f64(bv)[i], 0.1)
                                  for i, s in enumerate(slots)]))
            pair.model.compress(slots)
            for i, s in enumerate(slots):
                pair.seqs[s].compress(0, f64(bk)[i], f64(bv)[i])
    assert len(outs) == len(refs)
    for j, (o, r) in enumerate(zip(outs, refs)):
        assert_close(o, r, f"back-to-back host call {j}")
    pair.check_state()
    for s in slots:
        pair.check_content(0, s)



def test_all_layers_in_one_call():
    """layer = -1: the per-layer tensors carry a leading [layers] dimension and one call walks the
    layers in order.  Compared per layer with the oracle (and, for the bookkeeping, with the model)."""
    L, Hkv, G, D, ps, c = 3, 2, 4, 128, 8, 4
    n, plens = 3, [20, 0, 65]
    pair = Pair(L, Hkv, Hkv * G, D, ps, max_seqs=n, num_pages=64, max_pages_per_seq=24)
    g = _gen(29)
    slots = list(range(n))
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    pair.open(slots, plens, [c] * n)
    P = sum(plens)
    pk, pv = randn_bf16(g, (L, P, Hkv, D), DEV), randn_bf16(g, (L, P, Hkv, D), DEV)
    cu = torch.tensor([0] + list(np.cumsum(plens)), dtype=torch.int32, device=DEV)
    pair.gpu.bc_prefill(-1, sl, cu, P, pk, pv)
    for l in range(L):
        for i, s in enumerate(slots):
            a, b = int(cu[i]), int(cu[i + 1])
            pair.seqs[s].prefill(l, f64(pk[l, a:b]), f64(pv[l, a:b]))
    for step in range(1, 2 * c + 2):
        k, v, q = randn_bf16(g, (L, n, Hkv, D), DEV), randn_bf16(g, (L, n, Hkv, D), DEV), randn_bf16(g, (L, n, Hkv * G, D), DEV)
        out = torch.empty((L, n, Hkv * G, D), dtype=torch.bfloat16, device=DEV)
        pair.gpu.bc_append(-1, sl, k, v)
        pair.gpu.bc_decode_attn(-1, sl, q, out, 0.11)
        assert pair.model.append(slots) == [OK] * n
        for l in range(L):
            for i, s in enumerate(slots):
                pair.seqs[s].append(l, f64(k[l, i]), f64(v[l, i]))
            ref = np.stack([pair.seqs[s].attend(l, f64(q[l, i]), 0.11) for i, s in enumerate(slots)])
            assert_close(out[l], ref, f"step {step} layer {l}")
        if step % c == 0:
            bk, bv, bq = randn_bf16(g, (L, n, Hkv, D), DEV), randn_bf16(g, (L, n, Hkv, D), DEV), randn_bf16(g, (L, n, Hkv * G, D), DEV)
            pair.gpu.bc_decode_attn(-1, sl, bq, out, 0.11, bk, bv)
            pair.gpu.bc_compress(-1, sl, bk, bv)
            assert pair.model.compress(slots) == [OK] * n
            for l in range(L):
                ref = np.stack([pair.seqs[s].beacon_attend(l, f64(bq[l, i]), f64(bk[l, i]), f64(bv[l, i]), 0.11)
                                for i, s in enumerate(slots)])
                assert_close(out[l], ref, f"beacon step {step} layer {l}")
                for i, s in enumerate(slots):
                    pair.seqs[s].compress(l, f64(bk[l, i]), f64(bv[l, i]))
        pair.check_state()
    for l in range(L):
        for s in slots:
            pair.check_content(l, s)


@pytest.mark.parametrize("L,Hkv,G,D,ps,c,ctas", [(4, 2, 6, 128, 16, 8, 0), (3, 8, 4, 128, 4, 4, 7), (5, 1, 12, 64, 16, 16, 0),
                                                  (2, 4, 2, 64, 8, 2, 3)])
def test_all_layers_one_launch_per_call(L, Hkv, G, D, ps, c, ctas):
    """layer = -1 is ONE attention launch whose grid walks the layers (and one row-writing launch for an
    append or a compression): long ragged sequences cut into pieces across blocks, every layer with its own
    counters and partial buffers; the fused step (bc_decode_step) and the separate calls alternate.  Outputs
    per layer against the oracle, bookkeeping against the model, launch counts as documented."""
    Hq = Hkv * G
    n, plens = 4, [900, 0, 77, 2100]
    pair = Pair(L, Hkv, Hq, D, ps, max_seqs=n, num_pages=4 * (3200 // ps + 8), max_pages_per_seq=3200 // ps + 8)
    if ctas:
        pair.gpu.bc_set_attn_ctas(ctas)
    g = _gen(31)
    slots = list(range(n))
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    pair.open(slots, plens, [c] * n)
    P = sum(plens)
    pk, pv = randn_bf16(g, (L, P, Hkv, D), DEV), randn_bf16(g, (L, P, Hkv, D), DEV)
    cu = torch.tensor([0] + list(np.cumsum(plens)), dtype=torch.int32, device=DEV)
    pair.gpu.bc_prefill(-1, sl, cu, P, pk, pv)
    for l in range(L):
        for i, s in enumerate(slots):
            a, b = int(cu[i]), int(cu[i + 1])
            pair.seqs[s].prefill(l, f64(pk[l, a:b]), f64(pv[l, a:b]))
    for step in range(1, 2 * c + 2):
        k, v, q = randn_bf16(g, (L, n, Hkv, D), DEV), randn_bf16(g, (L, n, Hkv, D), DEV), randn_bf16(g, (L, n, Hq, D), DEV)
        out = torch.full((L, n, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
        before = pair.gpu.bc_kernel_launches()
        if step % 2:
            pair.gpu.bc_decode_step(-1, sl, q, k, v, out, 0.09)
            assert pair.gpu.bc_kernel_launches() - before == 2          # bookkeeping, attention
        else:
            pair.gpu.bc_append(-1, sl, k, v)
            pair.gpu.bc_decode_attn(-1, sl, q, out, 0.09)
            assert pair.gpu.bc_kernel_launches() - before == 3          # bookkeeping, rows, attention
        assert pair.model.append(slots) == [OK] * n
        for l in range(L):
            for i, s in enumerate(slots):
                pair.seqs[s].append(l, f64(k[l, i]), f64(v[l, i]))
            ref = np.stack([pair.seqs[s].attend(l, f64(q[l, i]), 0.09) for i, s in enumerate(slots)])
            assert_close(out[l], ref, f"step {step} layer {l}")
        if step % c == 0:
            bk, bv, bq = randn_bf16(g, (L, n, Hkv, D), DEV), randn_bf16(g, (L, n, Hkv, D), DEV), randn_bf16(g, (L, n, Hq, D), DEV)
            before = pair.gpu.bc_kernel_launches()
            pair.gpu.bc_decode_attn(-1, sl, bq, out, 0.09, bk, bv)
            pair.gpu.bc_compress(-1, sl, bk, bv)
            assert pair.gpu.bc_kernel_launches() - before == 3          # attention; bookkeeping, rows
            assert pair.model.compress(slots) == [OK] * n
            for l in range(L):
                ref = np.stack([pair.seqs[s].beacon_attend(l, f64(bq[l, i]), f64(bk[l, i]), f64(bv[l, i]), 0.09)
                                for i, s in enumerate(slots)])
                assert_close(out[l], ref, f"beacon step {step} layer {l}")
                for i, s in enumerate(slots):
                    pair.seqs[s].compress(l, f64(bk[l, i]), f64(bv[l, i]))
        pair.check_state()
    for l in range(L):
        for s in slots:
            pair.check_content(l, s)
