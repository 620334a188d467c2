"""Pins for the CPU oracle: what the paper and the mathematics fix.

None of these re-types the oracle's formula; each one is a closed form, an
invariant, a special case or a second formulation, chosen so that a plausible
mistake in the oracle (dropped scale, wrong head mapping, transposed operand,
off-by-one in the eviction slice, beacon not attending itself, ...) fails.
"""
import math
import os

import numpy as np
import pytest

from oracle.breadcrumbs_oracle import (SeqCache, attention, closed_form_length,
                                       closed_form_live_ids, mask_form_outputs)
from oracle.paging_model import (BAD_SLOT, CAPACITY, NO_PAGES, OK, WINDOW_FULL,
                                 WINDOW_NOT_FULL, PagingModel)

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append([float(x) for x in line.split()])
    return out


# ----------------------------------------------------------------- attention
def test_two_key_closed_form_and_scale():
    """logits ln a, ln b -> weights a/(a+b), b/(a+b); the logit is scale * <q,k>."""
    D = 8
    for a, b, w1, w2 in _rows("softmax_two_keys.txt"):
        for scale in (1.0, 0.5, 1.0 / math.sqrt(D)):
            q = np.zeros((1, D)); q[0, 2] = 2.0          # asymmetric: only coordinate 2 counts
            K = np.zeros((2, 1, D)); V = np.zeros((2, 1, D))
            K[0, 0, 2] = math.log(a) / (2.0 * scale)
            K[1, 0, 2] = math.log(b) / (2.0 * scale)
            K[:, 0, 5] = [9.0, -9.0]                      # must be ignored (q[5] == 0)
            V[0, 0] = np.arange(D); V[1, 0] = -2.0 * np.arange(D) + 1
            o = attention(q, K, V, scale)
            np.testing.assert_allclose(o[0], w1 * V[0, 0] + w2 * V[1, 0], rtol=0, atol=1e-13)


def test_identical_keys_give_mean_of_values():
    rng = np.random.RandomState(0)
    n, Hkv, G, D = 37, 2, 3, 16
    k = rng.randn(Hkv, D)
    K = np.broadcast_to(k, (n, Hkv, D)).copy()
    V = rng.randn(n, Hkv, D)
    q = rng.randn(Hkv * G, D)
    o = attention(q, K, V, 0.3)
    for h in range(Hkv * G):
        np.testing.assert_allclose(o[h], V[:, h // G].mean(axis=0), atol=1e-13)


def test_single_key_and_empty_cache():
    rng = np.random.RandomState(1)
    q = rng.randn(4, 8); K = rng.randn(1, 2, 8); V = rng.randn(1, 2, 8)
    o = attention(q, K, V, 0.7)
    for h in range(4):
        np.testing.assert_array_equal(o[h], V[0, h // 2])
    assert np.all(attention(q, np.zeros((0, 2, 8)), np.zeros((0, 2, 8)), 1.0) == 0.0)


def test_gqa_head_mapping():
    """Query head h must read KV head h // G (not h % Hkv)."""
    Hkv, G, D, n = 3, 4, 8, 5
    rng = np.random.RandomState(2)
    K = rng.randn(n, Hkv, D)
    V = np.zeros((n, Hkv, D))
    for j in range(Hkv):
        V[:, j, :] = j + 1
    o = attention(rng.randn(Hkv * G, D), K, V, 1.0)
    for h in range(Hkv * G):
        np.testing.assert_allclose(o[h], (h // G) + 1, atol=1e-13)


def test_permutation_invariance_and_far_key():
    rng = np.random.RandomState(3)
    n, Hkv, G, D = 50, 2, 2, 16
    q = rng.randn(Hkv * G, D); K = rng.randn(n, Hkv, D); V = rng.randn(n, Hkv, D)
    o = attention(q, K, V, 0.25)
    perm = rng.permutation(n)
    np.testing.assert_allclose(attention(q, K[perm], V[perm], 0.25), o, atol=1e-13)
    # a key whose logit is hugely negative changes nothing
    far_k = np.zeros((1, Hkv, D)); far_v = 1e6 * np.ones((1, Hkv, D))
    for j in range(Hkv):
        qsum = q[j * G:(j + 1) * G].sum(axis=0)
        far_k[0, j] = -1e4 * qsum / np.dot(qsum, qsum)
    # make sure every head of the group sees a very negative logit
    logits = [0.25 * q[h] @ far_k[0, h // G] for h in range(Hkv * G)]
    if max(logits) < -500:
        o2 = attention(q, np.concatenate([K, far_k]), np.concatenate([V, far_v]), 0.25)
        np.testing.assert_allclose(o2, o, atol=1e-12)


def test_dominant_key_selects_its_value():
    """One key with an overwhelming logit -> output is that key's value (argmax limit)."""
    rng = np.random.RandomState(4)
    n, D = 20, 8
    q = rng.randn(1, D); K = 0.01 * rng.randn(n, 1, D); V = rng.randn(n, 1, D)
    K[7, 0] = 100.0 * q[0] / np.dot(q[0], q[0]) * 10
    o = attention(q, K, V, 1.0)
    np.testing.assert_allclose(o[0], V[7, 0], atol=1e-10)


# ------------------------------------------------- eviction: lengths and sets
def _run_sequence(P, T, c, Hq=2, Hkv=1, D=8, layers=1, seed=0, scale=0.35):
    rng = np.random.RandomState(seed)
    data = dict(
        pk=rng.randn(layers, P, Hkv, D), pv=rng.randn(layers, P, Hkv, D),
        k=rng.randn(layers, T, Hkv, D), v=rng.randn(layers, T, Hkv, D), q=rng.randn(layers, T, Hq, D),
        bk=rng.randn(layers, T, Hkv, D), bv=rng.randn(layers, T, Hkv, D), bq=rng.randn(layers, T, Hq, D))
    seq = SeqCache(layers, c)
    for l in range(layers):
        seq.prefill(l, data["pk"][l], data["pv"][l])
    outs, bouts, lens_pre, lens_post, ids_post = [], [], [], [], []
    for n in range(1, T + 1):
        step_out = []
        for l in range(layers):
            seq.append(l, data["k"][l, n - 1], data["v"][l, n - 1])
            step_out.append(seq.attend(l, data["q"][l, n - 1], scale))
        outs.append(step_out)
        lens_pre.append(len(seq.live_ids()))
        if c > 1 and seq.window_len() == c:
            m = n // c
            bo = []
            for l in range(layers):
                bo.append(seq.beacon_attend(l, data["bq"][l, m - 1], data["bk"][l, m - 1],
                                            data["bv"][l, m - 1], scale))
                seq.compress(l, data["bk"][l, m - 1], data["bv"][l, m - 1])
            bouts.append(bo)
        lens_post.append(len(seq.live_ids()))
        ids_post.append(seq.live_ids())
    return data, np.array(outs), np.array(bouts), lens_pre, lens_post, ids_post, seq


@pytest.mark.parametrize("P,T,c", [(5, 40, 4), (3, 33, 16), (0, 20, 2), (7, 64, 32), (4, 30, 1), (6, 25, 5)])
def test_closed_form_lengths_and_live_sets(P, T, c):
    _, _, _, lens_pre, lens_post, ids_post, seq = _run_sequence(P, T, c)
    for t in range(1, T + 1):
        assert lens_post[t - 1] == closed_form_length(P, t, c)
        assert lens_post[t - 1] == (P + t // c + t % c if c > 1 else P + t)
        # just before a compression the window is full: P + (t/c - 1) + c
        if c > 1 and t % c == 0:
            assert lens_pre[t - 1] == P + (t // c - 1) + c
        assert ids_post[t - 1] == closed_form_live_ids(P, t, c)
        # after any step at most c-1 live window tokens remain
        if c > 1:
            assert sum(1 for k, _ in ids_post[t - 1] if k == "token") <= c - 1
    p, b, w = seq.lengths()
    assert (p, b, w) == (P, T // c if c > 1 else 0, T % c if c > 1 else T)


def test_paper_cache_growth_fixture():
    for c, t, nb, w, entries in _rows("cache_growth.txt"):
        c, t = int(c), int(t)
        assert closed_form_length(0, t, c) == entries
        ids = closed_form_live_ids(0, t, c)
        assert sum(1 for k, _ in ids if k == "beacon") == nb
        assert sum(1 for k, _ in ids if k == "token") == w
    # "2-32x fewer entries": generated / kept tends to c
    for c in (2, 4, 8, 16, 32):
        t = 1000 * c
        assert closed_form_length(0, t, c) == 1000
    # literal simulation agrees with the closed form at the fixture points
    _, _, _, _, lens_post, _, _ = _run_sequence(0, 48, 16, D=4)
    assert lens_post[15 - 1] == 15 and lens_post[16 - 1] == 1 and lens_post[17 - 1] == 2


def test_algorithm1_index_form():
    """Re-run Algorithm 1 on token ids only, with the paper's loop index i (compress when
    i > 0 and i mod c == 0, slice [:-c-1] + [-1]) and compare the surviving ids."""
    P, T, c = 3, 29, 4
    _, _, _, _, _, ids_post, _ = _run_sequence(P, T, c)
    kv = [("prompt", j) for j in range(P)]
    nb = 0
    for i in range(0, T + 1):
        # sampling x_i ran the forward pass of x_{i-1}: its entry is in the cache now
        if i > 0:
            kv.append(("token", i - 1))
        if i > 0 and i % c == 0:
            nb += 1
            kv.append(("beacon", nb))
            kv = kv[:-c - 1] + kv[-1:]
        if i > 0:
            assert kv == ids_post[i - 1]


# ------------------------------------------- eviction form == mask form (Fig. 2)
@pytest.mark.parametrize("P,T,c,Hq,Hkv,layers", [(5, 23, 4, 4, 2, 1), (2, 16, 16, 2, 1, 1),
                                                  (0, 9, 2, 2, 2, 1), (6, 20, 1, 2, 1, 1),
                                                  (3, 14, 3, 6, 2, 2)])
def test_mask_form_equals_eviction_form(P, T, c, Hq, Hkv, layers):
    scale = 0.35
    data, outs, bouts, *_ = _run_sequence(P, T, c, Hq=Hq, Hkv=Hkv, layers=layers, seed=5, scale=scale)
    nb = T // c if c > 1 else 0
    for l in range(layers):
        tok, bea = mask_form_outputs(data["pk"][l], data["pv"][l], data["k"][l], data["v"][l], data["q"][l],
                                     data["bk"][l, :nb], data["bv"][l, :nb], data["bq"][l, :nb], c, scale)
        np.testing.assert_allclose(outs[:, l], tok, atol=1e-12)
        if nb:
            np.testing.assert_allclose(bouts[:, l], bea, atol=1e-12)


def test_large_c_equals_uncompressed_full_attention():
    """c larger than the generation length: every step is plain causal attention over
    prompt + all generated tokens, computed here by brute force with dense matrices."""
    P, T, Hq, Hkv, D, scale = 4, 12, 4, 2, 8, 0.4
    data, outs, bouts, *_ = _run_sequence(P, T, 100, Hq=Hq, Hkv=Hkv, D=D, seed=6, scale=scale)
    assert bouts.size == 0
    K = np.concatenate([data["pk"][0], data["k"][0]]); V = np.concatenate([data["pv"][0], data["v"][0]])
    for n in range(1, T + 1):
        Kn, Vn, q = K[:P + n], V[:P + n], data["q"][0, n - 1]
        for h in range(Hq):
            logits = np.einsum("d,nd->n", q[h], Kn[:, h // 2]) * scale
            w = np.exp(logits - np.logaddexp.reduce(logits))
            np.testing.assert_allclose(outs[n - 1, 0, h], np.einsum("n,nd->d", w, Vn[:, h // 2]), atol=1e-12)
    # ratio 1 is the same thing
    _, outs1, _, *_ = _run_sequence(P, T, 1, Hq=Hq, Hkv=Hkv, D=D, seed=6, scale=scale)
    np.testing.assert_array_equal(outs1, outs)


def test_beacon_attends_itself_and_window():
    """With a beacon key that dominates, the beacon query's output is the beacon value; with a
    beacon key that is negligible, it equals the attention over the cache with the full window."""
    P, c, D = 2, 3, 4
    seq = SeqCache(1, c)
    rng = np.random.RandomState(7)
    seq.prefill(0, rng.randn(P, 1, D), rng.randn(P, 1, D))
    for _ in range(c):
        seq.append(0, rng.randn(1, D), rng.randn(1, D))
    qb = rng.randn(1, D)
    bv = rng.randn(1, D)
    strong = 1e3 * qb / np.dot(qb[0], qb[0])
    np.testing.assert_allclose(seq.beacon_attend(0, qb, strong, bv, 1.0), bv, atol=1e-10)
    weak = -1e3 * qb / np.dot(qb[0], qb[0])
    np.testing.assert_allclose(seq.beacon_attend(0, qb, weak, bv, 1.0), seq.attend(0, qb, 1.0), atol=1e-10)
    assert len(seq.live_ids()) == P + c           # beacon_attend mutates nothing
    with pytest.raises(RuntimeError):
        seq.append(0, rng.randn(1, D), rng.randn(1, D))     # window full: compress first
    seq.compress(0, strong, bv)
    assert seq.live_ids() == [("prompt", 0), ("prompt", 1), ("beacon", 1)]
    with pytest.raises(RuntimeError):
        seq.compress(0, strong, bv)                          # window not full


# ------------------------------------------------------------- paging model
def _check_invariants(m: PagingModel):
    owned = []
    for slot in list(m.seqs):
        st = m.state(slot)
        ps = m.ps
        assert len(st["prompt_pages"]) == -(-st["prompt_len"] // ps)
        assert len(st["beacon_pages"]) == -(-st["n_beacons"] // ps)
        assert len(st["window_pages"]) == -(-st["window_len"] // ps)
        if st["c"] > 1:
            assert st["n_beacons"] * st["c"] + st["window_len"] == st["t"] and st["window_len"] <= st["c"]
        owned += st["prompt_pages"] + st["beacon_pages"] + st["window_pages"]
    free = m.free_list()
    assert len(set(owned)) == len(owned), "a page is owned twice"
    assert sorted(owned + free) == list(range(m.num_pages)), "conservation broken"


@pytest.mark.parametrize("ps,c", [(16, 16), (2, 2), (4, 16), (16, 4), (3, 7), (8, 1), (1, 5)])
def test_paging_invariants_and_closed_form(ps, c):
    m = PagingModel(num_pages=400, page_size=ps, max_seqs=4, max_pages_per_seq=200)
    P = [5, 0, 17]
    assert m.open([0, 1, 3], P, [c, c, c]) == [OK, OK, OK]
    _check_invariants(m)
    for t in range(1, 60):
        assert m.append([0, 1, 3]) == [OK, OK, OK]
        _check_invariants(m)
        if c > 1 and t % c == 0:
            assert m.compress([3, 0, 1]) == [OK, OK, OK]
            _check_invariants(m)
        else:
            assert m.compress([0]) == [WINDOW_NOT_FULL]
        for slot, p in zip([0, 1, 3], P):
            st = m.state(slot)
            assert p + st["n_beacons"] + st["window_len"] == closed_form_length(p, t, c)
    assert m.close([1, 0, 3]) == [OK, OK, OK]
    assert sorted(m.free_list()) == list(range(400)) and not m.seqs


def test_paging_order_worked_by_hand():
    """Fresh store hands out 0,1,2,...; frees are pushed in batch order and reused LIFO."""
    m = PagingModel(num_pages=8, page_size=2, max_seqs=3, max_pages_per_seq=8)
    assert m.open([0, 1], [3, 1], [2, 2]) == [OK, OK]          # needs 2 and 1 pages
    assert m.state(0)["prompt_pages"] == [0, 1] and m.state(1)["prompt_pages"] == [2]
    assert m.free_list() == [7, 6, 5, 4, 3]
    assert m.append([1, 0]) == [OK, OK]                         # batch order 1 then 0
    assert m.state(1)["window_pages"] == [3] and m.state(0)["window_pages"] == [4]
    assert m.append([0, 1]) == [OK, OK]                         # second slot of the same page
    assert m.free_list() == [7, 6, 5]
    assert m.append([0]) == [WINDOW_FULL]
    assert m.compress([0, 1]) == [OK, OK]                       # beacon pages 5, 6; then free 4, 3
    assert m.state(0)["beacon_pages"] == [5] and m.state(1)["beacon_pages"] == [6]
    assert m.free_list() == [7, 4, 3]
    assert m.append([0]) == [OK] and m.state(0)["window_pages"] == [3]
    assert m.close([0]) == [OK]                                 # prompt 0,1 then beacon 5 then window 3
    assert m.free_list() == [7, 4, 0, 1, 5, 3]
    assert m.close([0]) == [BAD_SLOT]
    assert m.first_error == (WINDOW_FULL, 0, 4)


def test_paging_exhaustion_and_capacity():
    m = PagingModel(num_pages=3, page_size=1, max_seqs=4, max_pages_per_seq=10, max_entries_per_seq=2)
    assert m.open([0, 1, 2], [1, 3, 0], [1, 1, 1]) == [OK, NO_PAGES, OK]   # 1 granted, 3 refused, 0 needs none
    assert m.free_list() == [2, 1]
    assert m.append([0, 2]) == [OK, OK]
    assert m.append([0, 2]) == [NO_PAGES, NO_PAGES]
    m2 = PagingModel(num_pages=30, page_size=1, max_seqs=1, max_pages_per_seq=30, max_entries_per_seq=2)
    m2.open([0], [5], [1])
    assert m2.append([0]) == [OK] and m2.append([0]) == [OK] and m2.append([0]) == [CAPACITY]
    m3 = PagingModel(num_pages=30, page_size=1, max_seqs=1, max_pages_per_seq=6)
    m3.open([0], [5], [1])
    assert m3.append([0]) == [OK] and m3.append([0]) == [CAPACITY]


def test_latched_error_is_the_lowest_failing_item_of_the_first_failing_call():
    """The rule breadcrumbs.h states for the status record: the first call with a failing item
    latches, and of that call's failing items the one with the lowest batch index is recorded
    (code, slot, 1-based call index); later failures change nothing.  Every expected record below
    is worked out by hand from that sentence.  The cases are chosen so that other plausible rules
    give a different record: "first failure met while processing" (validation failures are met
    before allocation failures, whatever their batch position), "last failure", "lowest slot id",
    "highest severity / lowest code"."""
    # open: item 0 passes validation and fails at ALLOCATION (needs 3 pages, 2 free); item 1 fails
    # VALIDATION (slot out of range); item 2 fails validation (c = 0).  Lowest index: item 0.
    m = PagingModel(num_pages=2, page_size=1, max_seqs=4, max_pages_per_seq=8)
    assert m.open([3, 9, 1], [3, 1, 1], [1, 1, 0]) == [NO_PAGES, BAD_SLOT, "INVALID_ARG"]
    assert m.first_error == (NO_PAGES, 3, 1)
    assert m.free_list() == [1, 0] and not m.seqs            # a failed item changes nothing
    # append: [WINDOW_FULL, OK, BAD_SLOT] in one call, on a store that has no error yet
    m = PagingModel(num_pages=16, page_size=2, max_seqs=8, max_pages_per_seq=8)
    assert m.open([5, 2], [1, 1], [2, 2]) == [OK, OK]                        # call 1
    assert m.append([5]) == [OK] and m.append([5]) == [OK]                   # calls 2, 3: slot 5's window is full
    assert m.first_error is None
    assert m.append([5, 2, 7]) == [WINDOW_FULL, OK, BAD_SLOT]                # call 4
    assert m.first_error == (WINDOW_FULL, 5, 4)
    assert m.state(2)["window_len"] == 1 and m.state(5)["window_len"] == 2   # the good item went through
    # a later failing call does not replace the record, even one with a "worse" or lower-indexed failure
    assert m.append([7, 5]) == [BAD_SLOT, WINDOW_FULL]                       # call 5
    assert m.first_error == (WINDOW_FULL, 5, 4)
    # the failing item with the lowest INDEX, not the lowest slot id and not the last one:
    # items [slot 6 (not open), slot 2 (window of 1: not full), slot 0 (not open)]
    m2 = PagingModel(num_pages=16, page_size=2, max_seqs=8, max_pages_per_seq=8)
    assert m2.open([2], [1], [2]) == [OK] and m2.append([2]) == [OK]         # calls 1, 2
    assert m2.compress([6, 2, 0]) == [BAD_SLOT, WINDOW_NOT_FULL, BAD_SLOT]   # call 3
    assert m2.first_error == (BAD_SLOT, 6, 3)
    # compress: allocation failure at a lower index than a validation failure.  Page size 1, pool of
    # 4: slots 0 and 1 (P = 0, c = 2) take 2 window pages each, so no page is free when both
    # windows are full; compress needs a beacon page for each -> NO_PAGES for item 0 and item 1;
    # item 2 names a closed slot.  Lowest index: item 0, an allocation failure.
    m3 = PagingModel(num_pages=4, page_size=1, max_seqs=4, max_pages_per_seq=8)
    assert m3.open([0, 1], [0, 0], [2, 2]) == [OK, OK]                       # call 1
    assert m3.append([0, 1]) == [OK, OK] and m3.append([0, 1]) == [OK, OK]   # calls 2, 3
    assert m3.free_list() == []
    assert m3.compress([1, 0, 3]) == [NO_PAGES, NO_PAGES, BAD_SLOT]          # call 4
    assert m3.first_error == (NO_PAGES, 1, 4)
    assert m3.state(1)["window_len"] == 2 and m3.state(0)["n_beacons"] == 0
    # close and restore report the same way
    # restore: T = 132 at c = 4 is 33 beacons = 9 pages of 4, the pool has 8 -> allocation failure
    # at item 0; item 1 names a closed slot; item 2 has a negative length
    m4 = PagingModel(num_pages=8, page_size=4, max_seqs=4, max_pages_per_seq=16)
    assert m4.open([0, 1], [0, 0], [4, 4]) == [OK, OK]                       # call 1
    assert m4.restore([1, 2, 0], [132, 1, -1]) == [NO_PAGES, BAD_SLOT, "INVALID_ARG"]   # call 2
    assert m4.first_error == (NO_PAGES, 1, 2)
    m5 = PagingModel(num_pages=8, page_size=4, max_seqs=4, max_pages_per_seq=16)
    assert m5.open([0], [0], [4]) == [OK]                                    # call 1
    assert m5.close([3, 0, 2]) == [BAD_SLOT, OK, BAD_SLOT]                   # call 2
    assert m5.first_error == (BAD_SLOT, 3, 2)



@pytest.mark.parametrize("ps,c", [(1, 2), (4, 4), (16, 8), (8, 32), (16, 1)])
def test_paging_restore_equals_replay_counts_and_conserves_pages(ps, c):
    """restore(T) must leave the lengths that T appends with their compressions leave (and the closed
    form gives), hold exactly ceil(len / page) pages per segment, and conserve pages; the page ids
    differ from a replay's (a replay recycles window pages), which is why only counts are compared."""
    P = 37
    for T in (0, 1, c - 1, c, c + 1, 5 * c + 3, 97):
        a = PagingModel(num_pages=64, page_size=ps, max_seqs=2, max_pages_per_seq=64) if ps > 1 else \
            PagingModel(num_pages=256, page_size=ps, max_seqs=2, max_pages_per_seq=256)
        b = PagingModel(num_pages=a.num_pages, page_size=ps, max_seqs=2, max_pages_per_seq=a.max_pages_per_seq)
        assert a.open([0], [P], [c]) == [OK] and b.open([0], [P], [c]) == [OK]
        assert a.restore([0], [T]) == [OK]
        for n in range(1, T + 1):
            assert b.append([0]) == [OK]
            if c > 1 and n % c == 0:
                assert b.compress([0]) == [OK]
        sa, sb = a.state(0), b.state(0)
        for key in ("prompt_len", "n_beacons", "window_len", "c", "t"):
            assert sa[key] == sb[key], (key, T)
        assert sa["n_beacons"] + sa["window_len"] + P == closed_form_length(P, T, c)
        assert len(sa["beacon_pages"]) == -(-sa["n_beacons"] // ps) and len(sa["window_pages"]) == -(-sa["window_len"] // ps)
        owned = sa["prompt_pages"] + sa["beacon_pages"] + sa["window_pages"]
        assert sorted(owned + a.free_list()) == list(range(a.num_pages))
        # the restored sequence goes on like any other
        assert a.append([0]) == [OK] and a.state(0)["window_len"] == sa["window_len"] + 1


def test_paging_restore_order_and_failures_by_hand():
    """Page 4, pool of 8: slot 0 (P = 4, c = 4) holds page 0, slot 1 (P = 0, c = 4) none.  restore of
    T = 9 for slot 0 needs 1 beacon page (2 beacons) + 1 window page (1 token): pages 1 and 2, beacon
    page first.  A second restore of the same slot is refused; T = 40 for slot 1 needs 3 + 0 pages
    and gets 3, 4, 5; a further item that needs more than what is left is refused with NO_PAGES and
    changes nothing."""
    m = PagingModel(num_pages=8, page_size=4, max_seqs=3, max_pages_per_seq=8)
    assert m.open([0, 1, 2], [4, 0, 0], [4, 4, 4]) == [OK, OK, OK]
    assert m.restore([0], [9]) == [OK]
    s = m.state(0)
    assert (s["beacon_pages"], s["window_pages"], s["n_beacons"], s["window_len"], s["t"]) == ([1], [2], 2, 1, 9)
    assert m.restore([0], [3]) == ["INVALID_ARG"]
    assert m.first_error == ("INVALID_ARG", 0, 3)
    assert m.restore([1, 2], [40, 100]) == [OK, "NO_PAGES"]
    assert m.state(1)["beacon_pages"] == [3, 4, 5] and m.state(1)["window_pages"] == []
    assert m.state(2)["t"] == 0 and m.free_list() == [7, 6]


def test_replay_is_algorithm1_stepwise():
    """SeqCache.replay against the closed form of the live set (which entries survive T steps)."""
    rng = np.random.RandomState(5)
    for c, T in ((4, 11), (8, 8), (1, 6), (16, 5)):
        s = SeqCache(1, c)
        s.prefill(0, rng.standard_normal((3, 1, 4)), rng.standard_normal((3, 1, 4)))
        tk, tv = rng.standard_normal((T, 1, 4)), rng.standard_normal((T, 1, 4))
        nb = T // c if c > 1 else 0
        bk, bv = rng.standard_normal((nb, 1, 4)), rng.standard_normal((nb, 1, 4))
        s.replay(0, tk, tv, bk, bv)
        assert s.live_ids(0) == closed_form_live_ids(3, T, c)
        K, _ = s.entries(0)
        w = T - nb * c
        assert np.array_equal(K[3:3 + nb], bk) and np.array_equal(K[3 + nb:], tk[T - w:])



def test_checked_mode_refuses_the_later_items_of_a_repeated_slot():
    """Checked mode (the library's BC_FLAG_DEBUG_BOUNDS), worked by hand: of the items of one call
    that name the same slot the first goes through and the others get DEBUG_CHECK; an invalid
    slot stays BAD_SLOT however often it is named; pages are allocated for the first item only."""
    m = PagingModel(num_pages=16, page_size=2, max_seqs=4, max_pages_per_seq=8, debug_bounds=True)
    assert m.open([1, 1, 2, 7, 7], [3, 5, 1, 1, 1], [2, 2, 2, 2, 2]) == [OK, "DEBUG_CHECK", OK, BAD_SLOT, BAD_SLOT]
    assert m.state(1)["prompt_pages"] == [0, 1] and m.state(2)["prompt_pages"] == [2]     # P = 3, not 5
    assert m.first_error == ("DEBUG_CHECK", 1, 1)
    m.first_error = None
    assert m.append([2, 1, 2, 2]) == [OK, OK, "DEBUG_CHECK", "DEBUG_CHECK"]
    assert m.state(2)["window_len"] == 1 and m.state(2)["t"] == 1                        # appended once
    assert m.first_error == ("DEBUG_CHECK", 2, 2)
    assert m.append([1, 2]) == [OK, OK]
    m.first_error = None
    assert m.compress([1, 1]) == [OK, "DEBUG_CHECK"]
    assert m.state(1)["n_beacons"] == 1 and m.state(1)["window_len"] == 0
    assert m.close([2, 2, 3]) == [OK, "DEBUG_CHECK", BAD_SLOT]
    assert m.first_error == ("DEBUG_CHECK", 1, 4)
    # without the flag the model does not look for repeats (such a batch is outside the contract)
    assert PagingModel(4, 2, 4, 4).open([0, 1], [1, 1]) == [OK, OK]
