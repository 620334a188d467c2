"""bc_decode_attn_pair against the oracle: the token's and its beacon's queries in one pass over the
cache must give what two separate bc_decode_attn calls (and the oracle's attend / beacon_attend) give."""
import math

import numpy as np
import pytest
import torch

from oracle.paging_model import OK
from paper_2510_13797_b200 import binding as B
from tests.harness import Pair, assert_close, f64, randn_bf16

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _gen(seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return g


def _build(pair, g, slots, plens, cs, steps):
    """Opens the sequences, stores the prompts and decodes `steps` tokens with compressions where due,
    stopping right after an append (so windows may be full: the state a paired call is made in)."""
    assert pair.open(slots, plens, cs) == [OK] * len(slots)
    for l in range(pair.L):
        pair.prefill(l, slots, plens, randn_bf16(g, (sum(plens), pair.Hkv, pair.D), DEV), randn_bf16(g, (sum(plens), pair.Hkv, pair.D), DEV))
    n = len(slots)
    for t in range(1, steps + 1):
        for l in range(pair.L):
            assert pair.append(l, slots, randn_bf16(g, (n, pair.Hkv, pair.D), DEV), randn_bf16(g, (n, pair.Hkv, pair.D), DEV)) == [OK] * n
        if t == steps:
            break
        full = [s for s in slots if pair.model.state(s)["c"] > 1 and pair.model.state(s)["window_len"] == pair.model.state(s)["c"]]
        for l in range(pair.L):
            if full:
                pair.compress(l, full, randn_bf16(g, (len(full), pair.Hkv, pair.D), DEV), randn_bf16(g, (len(full), pair.Hkv, pair.D), DEV))


def _check_pair(pair, g, slots, sm_scale, layer=0, what=""):
    n = len(slots)
    q, bq = randn_bf16(g, (n, pair.Hq, pair.D), DEV), randn_bf16(g, (n, pair.Hq, pair.D), DEV)
    bk, bv = randn_bf16(g, (n, pair.Hkv, pair.D), DEV), randn_bf16(g, (n, pair.Hkv, pair.D), DEV)
    out, out_b = pair.gpu.new_out(n), pair.gpu.new_out(n)
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    pair.gpu.bc_decode_attn_pair(layer, sl, q, out, bq, out_b, sm_scale, bk, bv)
    torch.cuda.synchronize()
    ref = np.stack([pair.seqs[s].attend(layer, f64(q)[i], sm_scale) for i, s in enumerate(slots)])
    ref_b = np.stack([pair.seqs[s].beacon_attend(layer, f64(bq)[i], f64(bk)[i], f64(bv)[i], sm_scale) for i, s in enumerate(slots)])
    assert_close(out, ref, what + " token rows")
    assert_close(out_b, ref_b, what + " beacon rows")
    assert pair.gpu.bc_poll_error()[0] == 0
    return out, out_b


@pytest.mark.parametrize("Hkv,G,D,ps,c", [(2, 4, 128, 16, 8), (8, 4, 128, 4, 4), (1, 1, 64, 16, 16), (2, 6, 128, 8, 8),
                                          (4, 8, 64, 16, 2), (1, 12, 128, 16, 8)])
def test_pair_matches_oracle_small(Hkv, G, D, ps, c):
    """Short sequences (one block holds a whole sequence), ragged lengths, an empty prompt; G = 12 takes
    the two-pass route."""
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=4, num_pages=256, max_pages_per_seq=64)
    g = _gen(3)
    slots, plens = [0, 1, 2, 3], [33, 0, 100, 7]
    _build(pair, g, slots, plens, [c] * 4, 2 * c)
    assert all(pair.model.state(s)["window_len"] == c for s in slots)
    _check_pair(pair, g, slots, 1.0 / math.sqrt(D), what=f"G={G}")
    _check_pair(pair, g, [2, 0], 0.07, what="subset")


@pytest.mark.parametrize("ctas", [0, 1, 2, 5, 37])
def test_pair_split_over_blocks(ctas):
    """Long sequences cut into pieces by several blocks: pieces published through global memory, the
    last arriver or the final piece's block merging, for both sets of rows.  Repeated launches check
    that the ticket counters return to zero."""
    Hkv, G, D, ps, c = 8, 4, 128, 16, 16
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=5, num_pages=700, max_pages_per_seq=160)
    g = _gen(5)
    slots, plens = [0, 1, 2, 3, 4], [1500, 40, 900, 2047, 3]
    _build(pair, g, slots, plens, [c] * 5, 3 * c)
    if ctas:
        pair.gpu.bc_set_attn_ctas(ctas)
    for rep in range(3):
        _check_pair(pair, g, slots, 1.0 / math.sqrt(D), what=f"ctas={ctas} rep={rep}")
    # a plain call afterwards still works on the same counters
    q = randn_bf16(g, (5, Hkv * G, D), DEV)
    out, ref = pair.attend(0, slots, q, 0.09)
    assert_close(out, ref, "plain call after paired calls")


def test_pair_empty_cache_and_f32_output():
    """No entries at all: the token's rows are zero, the beacon's rows are exactly the beacon's V;
    fp32 outputs."""
    Hkv, G, D = 2, 4, 128
    pair = Pair(1, Hkv, Hkv * G, D, 16, max_seqs=2, num_pages=16, max_pages_per_seq=8, flags=B.BC_FLAG_OUT_F32)
    g = _gen(7)
    assert pair.open([0, 1], [0, 5], [4, 4]) == [OK, OK]
    pair.prefill(0, [0, 1], [0, 5], randn_bf16(g, (5, Hkv, D), DEV), randn_bf16(g, (5, Hkv, D), DEV))
    out, out_b = _check_pair(pair, g, [0, 1], 0.1, what="empty")
    assert out.dtype == torch.float32 and float(out[0].abs().max()) == 0.0


def test_pair_equals_two_separate_calls_bitwise_on_whole_sequences():
    """Where one block holds a whole sequence the paired kernel does the same arithmetic in the same
    order as the plain one: identical bits."""
    Hkv, G, D, ps, c = 2, 4, 128, 16, 8
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=3, num_pages=64, max_pages_per_seq=16)
    g = _gen(9)
    slots = [0, 1, 2]
    _build(pair, g, slots, [60, 10, 90], [c] * 3, c)
    n = 3
    q, bq = randn_bf16(g, (n, Hkv * G, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)
    bk, bv = randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV)
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    o1, o2, p1, p2 = (pair.gpu.new_out(n) for _ in range(4))
    pair.gpu.bc_decode_attn_pair(0, sl, q, p1, bq, p2, 0.1, bk, bv)
    pair.gpu.bc_decode_attn(0, sl, q, o1, 0.1)
    pair.gpu.bc_decode_attn(0, sl, bq, o2, 0.1, bk, bv)
    torch.cuda.synchronize()
    assert torch.equal(o1, p1) and torch.equal(o2, p2)


def test_fill_step_host_matches_oracle(host_route):
    """bc_fill_step_host: append + paired attention + compress with host buffers, issued back to back
    with ordinary host steps; outputs and bookkeeping against the oracle."""
    Hkv, G, D, ps, c = 2, 4, 128, 16, 4
    n, plens = 3, [70, 9, 300]
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=n, num_pages=96, max_pages_per_seq=32)
    g = _gen(13)
    slots = list(range(n))
    assert pair.open(slots, plens, [c] * n) == [OK] * n
    pair.prefill(0, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    pin = lambda t: t.cpu().pin_memory()
    pending = []
    for step in range(1, 2 * c + 1):
        k, v, q = randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)
        out_h = torch.empty((n, Hkv * G, D), dtype=torch.bfloat16).pin_memory()
        assert pair.model.append(slots) == [OK] * n
        for i, s in enumerate(slots):
            pair.seqs[s].append(0, f64(k)[i], f64(v)[i])
        ref = np.stack([pair.seqs[s].attend(0, f64(q)[i], 0.1) for i, s in enumerate(slots)])
        if step % c:
            pair.gpu.bc_decode_step_host(0, sl, pin(q), pin(k), pin(v), out_h, 0.1)
            pending.append((out_h, ref, f"host step {step}"))
        else:
            bk, bv, bq = randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)
            out_b = torch.empty((n, Hkv * G, D), dtype=torch.bfloat16).pin_memory()
            pair.gpu.bc_fill_step_host(0, sl, pin(q), pin(k), pin(v), pin(bq), pin(bk), pin(bv), out_h, out_b, 0.1)
            ref_b = np.stack([pair.seqs[s].beacon_attend(0, f64(bq)[i], f64(bk)[i], f64(bv)[i], 0.1) for i, s in enumerate(slots)])
            pending.append((out_h, ref, f"fill step {step}: token"))
            pending.append((out_b, ref_b, f"fill step {step}: beacon"))
            assert pair.model.compress(slots) == [OK] * n
            for i, s in enumerate(slots):
                pair.seqs[s].compress(0, f64(bk)[i], f64(bv)[i])
    torch.cuda.synchronize()
    for o, r, what in pending:
        assert_close(o, r, what)
    pair.check_state()
    for s in slots:
        pair.check_content(0, s)


def test_host_steps_with_pipelined_outputs(host_route):
    """BC_FLAG_HOST_PIPELINED: the outputs come back on the cache's own stream from two staging sets in
    turn.  Many steps are issued with nothing in between; the caller's stream is made to wait with
    bc_host_outputs_ready and is then the only thing synchronised before the outputs are compared."""
    Hkv, G, D, ps, c = 2, 4, 128, 16, 4
    n, plens = 3, [200, 9, 64]
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=n, num_pages=96, max_pages_per_seq=32, flags=B.BC_FLAG_HOST_PIPELINED)
    g = _gen(17)
    slots = list(range(n))
    assert pair.open(slots, plens, [c] * n) == [OK] * n
    pair.prefill(0, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    pin = lambda t: t.cpu().pin_memory()
    stream = torch.cuda.Stream()
    steps = []
    for step in range(1, 3 * c + 1):
        k, v, q = randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)
        bea = (randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)) if step % c == 0 else None
        steps.append((pin(k), pin(v), pin(q), None if bea is None else tuple(pin(x) for x in bea)))
    torch.cuda.synchronize()
    outs = []
    with torch.cuda.stream(stream):
        for k, v, q, bea in steps:
            out_h = torch.empty((n, Hkv * G, D), dtype=torch.bfloat16).pin_memory()
            if bea is None:
                pair.gpu.bc_decode_step_host(0, sl, q, k, v, out_h, 0.1)
                outs.append((out_h, None))
            else:
                out_b = torch.empty((n, Hkv * G, D), dtype=torch.bfloat16).pin_memory()
                pair.gpu.bc_fill_step_host(0, sl, q, k, v, bea[2], bea[0], bea[1], out_h, out_b, 0.1)
                outs.append((out_h, out_b))
        pair.gpu.bc_host_outputs_ready()
    stream.synchronize()                      # only the caller's stream
    for (k, v, q, bea), (out_h, out_b) in zip(steps, outs):
        assert pair.model.append(slots) == [OK] * n
        for i, s in enumerate(slots):
            pair.seqs[s].append(0, f64(k)[i], f64(v)[i])
        assert_close(out_h, np.stack([pair.seqs[s].attend(0, f64(q)[i], 0.1) for i, s in enumerate(slots)]), "pipelined token rows")
        if bea is not None:
            bk, bv, bq = bea
            assert_close(out_b, np.stack([pair.seqs[s].beacon_attend(0, f64(bq)[i], f64(bk)[i], f64(bv)[i], 0.1)
                                          for i, s in enumerate(slots)]), "pipelined beacon rows")
            assert pair.model.compress(slots) == [OK] * n
            for i, s in enumerate(slots):
                pair.seqs[s].compress(0, f64(bk)[i], f64(bv)[i])
    pair.check_state()


def test_pipelined_host_steps_with_device_synchronisations_in_between():
    """Single-layer cache, pipelined outputs: a regular host-buffer step leaves nothing on the caller's stream but
    its kernels, and the copies are released through words in device memory.  None of the library's waits may
    depend on a call still to be made: the device is synchronised after every call (and pinned memory is
    allocated, which synchronises implicitly), a stream switch sits in the middle, and only
    bc_host_outputs_ready is called before the outputs are read."""
    Hkv, G, D, ps, c = 2, 4, 128, 16, 5
    n, plens = 3, [90, 0, 300]
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=n, num_pages=96, max_pages_per_seq=32, flags=B.BC_FLAG_HOST_PIPELINED)
    g = _gen(41)
    slots = list(range(n))
    assert pair.open(slots, plens, [c] * n) == [OK] * n
    pair.prefill(0, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    pending = []
    for step in range(1, 2 * c + 3):
        k, v, q = randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)
        assert pair.model.append(slots) == [OK] * n
        for i, s in enumerate(slots):
            pair.seqs[s].append(0, f64(k)[i], f64(v)[i])
        ref = np.stack([pair.seqs[s].attend(0, f64(q)[i], 0.1) for i, s in enumerate(slots)])
        hk, hv, hq = k.cpu().pin_memory(), v.cpu().pin_memory(), q.cpu().pin_memory()
        out_h = torch.full((n, Hkv * G, D), float("nan"), dtype=torch.bfloat16).pin_memory()
        stream = s1 if step <= c + 1 else s2
        torch.cuda.synchronize()                       # everything enqueued so far, the library's own streams included
        with torch.cuda.stream(stream):
            if step % c:
                pair.gpu.bc_decode_step_host(0, sl, hq, hk, hv, out_h, 0.1)
                pending.append((out_h, ref, f"host step {step}", (hk, hv, hq)))
            else:
                bk, bv, bq = randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)
                out_b = torch.full((n, Hkv * G, D), float("nan"), dtype=torch.bfloat16).pin_memory()
                hb = (bq.cpu().pin_memory(), bk.cpu().pin_memory(), bv.cpu().pin_memory())
                pair.gpu.bc_fill_step_host(0, sl, hq, hk, hv, hb[0], hb[1], hb[2], out_h, out_b, 0.1)
                ref_b = np.stack([pair.seqs[s].beacon_attend(0, f64(bq)[i], f64(bk)[i], f64(bv)[i], 0.1) for i, s in enumerate(slots)])
                pending.append((out_h, ref, f"fill step {step}: token", (hk, hv, hq, hb)))
                pending.append((out_b, ref_b, f"fill step {step}: beacon", None))
                assert pair.model.compress(slots) == [OK] * n
                for i, s in enumerate(slots):
                    pair.seqs[s].compress(0, f64(bk)[i], f64(bv)[i])
    with torch.cuda.stream(s2):
        pair.gpu.bc_host_outputs_ready()
    s2.synchronize()
    for o, r, what, _ in pending:
        assert_close(o, r, what)
    pair.check_state()


def _run_fill_steps(pair, g, slots, c, steps, sm_scale, what):
    """Regular steps through bc_decode_step, window-filling steps through bc_fill_step; every output against the
    oracle, the bookkeeping against the model."""
    n = len(slots)
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    L = pair.L
    for step in range(1, steps + 1):
        fill = step % c == 0
        for l in range(L):
            q, k, v = randn_bf16(g, (n, pair.Hq, pair.D), DEV), randn_bf16(g, (n, pair.Hkv, pair.D), DEV), randn_bf16(g, (n, pair.Hkv, pair.D), DEV)
            out = torch.full((n, pair.Hq, pair.D), float("nan"), dtype=torch.bfloat16, device=DEV)
            if fill:
                bq, bk, bv = randn_bf16(g, (n, pair.Hq, pair.D), DEV), randn_bf16(g, (n, pair.Hkv, pair.D), DEV), randn_bf16(g, (n, pair.Hkv, pair.D), DEV)
                out_b = torch.full_like(out, float("nan"))
                pair.gpu.bc_fill_step(l, sl, q, k, v, bq, bk, bv, out, out_b, sm_scale)
            else:
                pair.gpu.bc_decode_step(l, sl, q, k, v, out, sm_scale)
            torch.cuda.synchronize()
            if l == 0:
                assert pair.model.append(slots) == [OK] * n
            for i, s in enumerate(slots):
                pair.seqs[s].append(l, f64(k)[i], f64(v)[i])
            ref = np.stack([pair.seqs[s].attend(l, f64(q)[i], sm_scale) for i, s in enumerate(slots)])
            assert_close(out, ref, f"{what}: step {step} layer {l} token rows")
            if fill:
                ref_b = np.stack([pair.seqs[s].beacon_attend(l, f64(bq)[i], f64(bk)[i], f64(bv)[i], sm_scale) for i, s in enumerate(slots)])
                assert_close(out_b, ref_b, f"{what}: step {step} layer {l} beacon rows")
                if l == L - 1:
                    assert pair.model.compress(slots) == [OK] * n
                for i, s in enumerate(slots):
                    pair.seqs[s].compress(l, f64(bk)[i], f64(bv)[i])
        pair.check_state()
    for l in range(L):
        for s in slots:
            pair.check_content(l, s)


@pytest.mark.parametrize("L,Hkv,G,D,ps,c", [(1, 2, 4, 128, 16, 8), (2, 8, 4, 128, 4, 4), (1, 1, 1, 64, 16, 16), (1, 2, 6, 128, 8, 2),
                                            (1, 4, 8, 64, 16, 3), (1, 1, 12, 128, 16, 4)])
def test_fill_step_matches_oracle_small(L, Hkv, G, D, ps, c):
    """bc_fill_step on short ragged sequences (an empty prompt among them), two layers, G = 12 (the three-call
    route) and the reference-free paired kernel with the append inside."""
    pair = Pair(L, Hkv, Hkv * G, D, ps, max_seqs=4, num_pages=4 * (200 // ps + 12), max_pages_per_seq=200 // ps + 12)
    g = _gen(51)
    slots, plens = [0, 1, 2, 3], [33, 0, 100, 7]
    assert pair.open(slots, plens, [c] * 4) == [OK] * 4
    for l in range(L):
        pair.prefill(l, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    _run_fill_steps(pair, g, slots, c, 3 * c + 1, 1.0 / math.sqrt(D), f"G={G}")


@pytest.mark.parametrize("ctas", [0, 1, 2, 5, 37])
def test_fill_step_split_over_blocks(ctas):
    """Long sequences cut into pieces by several blocks, the window's last tile (with the entry that comes from
    the inputs) owned by one block and the pieces merged by another; repeated launches."""
    Hkv, G, D, ps, c = 8, 4, 128, 16, 16
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=5, num_pages=700, max_pages_per_seq=160)
    if ctas:
        pair.gpu.bc_set_attn_ctas(ctas)
    g = _gen(53)
    slots, plens = [0, 1, 2, 3, 4], [1500, 40, 900, 2047, 3]
    assert pair.open(slots, plens, [c] * 5) == [OK] * 5
    pair.prefill(0, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    _run_fill_steps(pair, g, slots, c, 2 * c + 2, 0.09, f"ctas={ctas}")
