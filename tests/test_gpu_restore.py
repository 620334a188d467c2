"""bc_restore against the oracle: a stored trajectory put into the cache in one call per layer must
leave what Algorithm 1, stepped token by token over the same trajectory, leaves (content bit for
bit, bookkeeping as the paging model's restore defines it), and decoding must go on from there."""
import math

import numpy as np
import pytest
import torch

from harness import Pair, assert_close, f64, randn_bf16
from oracle.paging_model import OK

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _gen(seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return g


def _trajectories(g, pair, slots, gen_lens, cs):
    nbs = [T // c if c > 1 else 0 for T, c in zip(gen_lens, cs)]
    per_layer = []
    for _ in range(pair.L):
        per_layer.append((randn_bf16(g, (max(sum(gen_lens), 1), pair.Hkv, pair.D), DEV)[:sum(gen_lens)],
                          randn_bf16(g, (max(sum(gen_lens), 1), pair.Hkv, pair.D), DEV)[:sum(gen_lens)],
                          randn_bf16(g, (max(sum(nbs), 1), pair.Hkv, pair.D), DEV)[:sum(nbs)],
                          randn_bf16(g, (max(sum(nbs), 1), pair.Hkv, pair.D), DEV)[:sum(nbs)]))
    return per_layer


def _decode_on(pair, g, slots, steps, sm_scale):
    """Lock-step decode of open sequences with mixed ratios: append + attend, beacon step where a window filled."""
    for _ in range(steps):
        n = len(slots)
        for l in range(pair.L):
            k, v, q = (randn_bf16(g, (n, pair.Hkv, pair.D), DEV), randn_bf16(g, (n, pair.Hkv, pair.D), DEV),
                       randn_bf16(g, (n, pair.Hq, pair.D), DEV))
            assert pair.append(l, slots, k, v) == [OK] * n
            out, ref = pair.attend(l, slots, q, sm_scale)
            assert_close(out, ref, "decode after restore")
        full = [s for s in slots if pair.model.state(s)["c"] > 1 and pair.model.state(s)["window_len"] == pair.model.state(s)["c"]]
        if full:
            m = len(full)
            for l in range(pair.L):
                bk, bv, bq = (randn_bf16(g, (m, pair.Hkv, pair.D), DEV), randn_bf16(g, (m, pair.Hkv, pair.D), DEV),
                              randn_bf16(g, (m, pair.Hq, pair.D), DEV))
                out, ref = pair.attend(l, full, bq, sm_scale, bk, bv)
                assert_close(out, ref, "beacon step after restore")
                assert pair.compress(l, full, bk, bv) == [OK] * m
        pair.check_state()


@pytest.mark.parametrize("ps", [1, 8, 16])
def test_restore_equals_stepwise_replay_and_decoding_goes_on(ps):
    L, Hkv, G, D = 2, 2, 4, 128
    slots, plens = [0, 1, 2, 3, 4, 5], [40, 0, 17, 100, 5, 33]
    cs, gen_lens = [4, 8, 1, 16, 4, 2], [11, 64, 9, 7, 0, 129]
    pair = Pair(L, Hkv, Hkv * G, D, ps, max_seqs=8, num_pages=2048 // ps + 64, max_pages_per_seq=512 // ps + 16)
    g = _gen(31)
    assert pair.open(slots, plens, cs) == [OK] * len(slots)
    for l in range(L):
        pair.prefill(l, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    traj = _trajectories(g, pair, slots, gen_lens, cs)
    for l in range(L):
        assert pair.restore(l, slots, gen_lens, *traj[l]) == [OK] * len(slots)
    pair.check_state()
    for l in range(L):
        for s in slots:
            pair.check_content(l, s)
    st = pair.gpu.bc_get_state(5)
    assert (st["n_beacons"], st["window_len"], st["t"]) == (64, 1, 129)
    _decode_on(pair, g, slots, 9, 1.0 / math.sqrt(D))
    for l in range(L):
        for s in slots:
            pair.check_content(l, s)
    assert pair.close(slots) == [OK] * len(slots)
    pair.check_state()


def test_restore_refusals_leave_the_sequence_untouched():
    """A sequence that already holds entries, a slot that is not open, and a pool too small for the
    last items: the failing items change nothing, the first failure is latched, the others go through."""
    L, Hkv, G, D, ps = 1, 1, 2, 64, 4
    pair = Pair(L, Hkv, Hkv * G, D, ps, max_seqs=6, num_pages=12, max_pages_per_seq=8)
    g = _gen(37)
    slots, plens, cs = [0, 1, 2, 3], [4, 3, 0, 8], [4, 4, 2, 4]
    assert pair.open(slots, plens, cs) == [OK] * 4            # pages: 1 + 1 + 0 + 2 = 4 of 12
    pair.prefill(0, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    k, v = randn_bf16(g, (1, Hkv, D), DEV), randn_bf16(g, (1, Hkv, D), DEV)
    assert pair.append(0, [1], k, v) == [OK]                  # slot 1 is no longer fresh (5 pages used)
    # slot 0: T = 21 -> 5 beacons (2 pages) + 1 window entry (1 page); slot 1: refused; slot 5: not open;
    # slot 2: T = 17, c = 2 -> 8 beacons (2 pages) + 1 entry (1 page): 6 of the 7 free pages are gone after it;
    # slot 3: T = 9 -> 2 beacons (1 page) + 1 entry (1 page): needs 2, 1 is left -> NO_PAGES
    batch, gen_lens = [0, 1, 5, 2, 3], [21, 6, 4, 17, 9]
    traj = _trajectories(g, pair, batch, gen_lens, [4, 4, 1, 2, 4])
    # the packed beacon array has rows for every OPEN slot of the batch, also the refused ones
    res = pair.restore(0, batch, gen_lens, *_pack_for_open(pair, batch, gen_lens, traj[0]))
    assert res == [OK, "INVALID_ARG", "BAD_SLOT", OK, "NO_PAGES"]
    pair.check_state()
    for s in (0, 1, 2, 3):
        pair.check_content(0, s)
    _decode_on(pair, g, [0, 2], 3, 0.125)


def _pack_for_open(pair, batch, gen_lens, traj):
    """The beacon arrays as bc_restore expects them: floor(T / c) rows for every open slot of the
    batch (with the slot's own c), none for a slot that is not open."""
    tok_k, tok_v, _, _ = traj
    nb = sum((T // pair.model.seqs[s].c if pair.model.seqs[s].c > 1 else 0) for s, T in zip(batch, gen_lens) if s in pair.model.seqs)
    g = _gen(41)
    return tok_k, tok_v, randn_bf16(g, (max(nb, 1), pair.Hkv, pair.D), DEV)[:nb], randn_bf16(g, (max(nb, 1), pair.Hkv, pair.D), DEV)[:nb]


def test_restore_large_uncompressed_and_compressed_side_by_side():
    """Long trajectories: c = 1 keeps all 3000 tokens (the window copy kernel strides over them),
    c = 32 keeps 93 beacons and 24 tokens."""
    L, Hkv, G, D, ps = 1, 2, 4, 128, 16
    pair = Pair(L, Hkv, Hkv * G, D, ps, max_seqs=2, num_pages=256, max_pages_per_seq=200)
    g = _gen(43)
    assert pair.open([0, 1], [64, 64], [1, 32]) == [OK, OK]
    pair.prefill(0, [0, 1], [64, 64], randn_bf16(g, (128, Hkv, D), DEV), randn_bf16(g, (128, Hkv, D), DEV))
    traj = _trajectories(g, pair, [0, 1], [3000, 3000], [1, 32])
    assert pair.restore(0, [0, 1], [3000, 3000], *traj[0]) == [OK, OK]
    pair.check_state()
    pair.check_content(0, 0)
    pair.check_content(0, 1)
    q = randn_bf16(g, (2, Hkv * G, D), DEV)
    out, ref = pair.attend(0, [0, 1], q, 1.0 / math.sqrt(D))
    assert_close(out, ref, "attention over restored caches")


@pytest.mark.parametrize("c,T", [(4, 37), (8, 64), (1, 20)])
def test_mask_form_row_equals_restore_then_decode(c, T):
    """Section 3.2 on the GPU alone: the mask-form output of a trajectory's last token (one dense pass)
    against the decode path (the trajectory minus that token restored into the cache, the token
    appended and attended).  Two different kernels of this library, the same quantity."""
    from paper_2510_13797_b200 import binding as B
    Hkv, G, D, ps, P = 2, 4, 128, 16, 50
    g = _gen(47)
    nb = T // c if c > 1 else 0
    pk, pv = randn_bf16(g, (P, Hkv, D), DEV), randn_bf16(g, (P, Hkv, D), DEV)
    tq, tk, tv = randn_bf16(g, (T, Hkv * G, D), DEV), randn_bf16(g, (T, Hkv, D), DEV), randn_bf16(g, (T, Hkv, D), DEV)
    bq, bk, bv = (randn_bf16(g, (max(nb, 1), Hkv * G, D), DEV)[:nb], randn_bf16(g, (max(nb, 1), Hkv, D), DEV)[:nb],
                  randn_bf16(g, (max(nb, 1), Hkv, D), DEV)[:nb])
    scale = 1.0 / math.sqrt(D)
    out_tok, _ = B.bc_mask_attn_forward([P], [T], c, pk, pv, tq, tk, tv, bq if nb else None, bk if nb else None,
                                        bv if nb else None, scale)
    cache = B.Cache(1, Hkv, Hkv * G, D, c, ps, max_seqs=1, num_pages=32, max_pages_per_seq=32, device=DEV)
    slot = torch.zeros(1, dtype=torch.int32, device=DEV)
    i32 = lambda xs: torch.tensor(xs, dtype=torch.int32, device=DEV)
    cache.bc_seq_open(slot, i32([P]))
    cache.bc_prefill(0, slot, i32([0, P]), P, pk, pv)
    nb_before = (T - 1) // c if c > 1 else 0                  # beacons that exist before the last token
    cache.bc_restore(0, slot, i32([0, T - 1]), T - 1, nb_before, tk, tv, bk if nb_before else None, bv if nb_before else None)
    out = cache.new_out(1)
    cache.bc_decode_step(0, slot, tq[T - 1:T], tk[T - 1:T], tv[T - 1:T], out, scale)
    torch.cuda.synchronize()
    assert cache.bc_poll_error()[0] == 0
    assert_close(out, f64(out_tok[T - 1:T]), "mask-form row vs restore + decode")
