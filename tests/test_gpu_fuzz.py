"""Random programs of open / restore / append / decode step / fill step / compress / close against the oracle.

Small pools and odd page sizes make the programs hit every refusal (no pages, window full, window
not full, bad slot, capacity); after every call the lengths, page lists, free stack and the latched
first error must be those of the integer-only model, bit for bit, and at the end of a program every
sequence is closed and every page is back."""
import numpy as np
import pytest
import torch

from paper_2510_13797_b200 import binding as B
from tests.harness import Pair, assert_close, randn_bf16

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("seed,ps,num_pages,max_pps,max_entries,checked", [
    (0, 1, 40, 12, 0, False), (1, 2, 24, 8, 0, False), (2, 3, 30, 9, 7, False), (3, 4, 64, 16, 0, False),
    (4, 16, 12, 4, 0, False), (5, 5, 50, 6, 11, False),
    # checked mode (BC_FLAG_DEBUG_BOUNDS): the same programs, every index checked on the device, and
    # batches that name a slot more than once (the later items are refused)
    (6, 2, 24, 8, 0, True), (7, 3, 30, 9, 7, True), (8, 16, 12, 4, 0, True), (9, 1, 40, 12, 0, True),
])
def test_random_programs(seed, ps, num_pages, max_pps, max_entries, checked):
    rng = np.random.RandomState(seed)
    S, Hkv, G, D = 8, 1, 2, 64
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=S, num_pages=num_pages, max_pages_per_seq=max_pps,
                max_entries=max_entries, c_default=int(rng.choice([1, 2, 3, 5])),
                flags=B.BC_FLAG_DEBUG_BOUNDS if checked else 0)
    g = torch.Generator(device=DEV); g.manual_seed(seed)
    kv = lambda n: (randn_bf16(g, (n, Hkv, D), DEV), randn_bf16(g, (n, Hkv, D), DEV))
    for step in range(160):
        op = rng.choice(["open", "restore", "append", "append", "step", "step", "fill", "compress", "close"])
        n = int(rng.randint(1, S + 1))
        slots = [int(x) for x in rng.choice(S + 2, size=n, replace=False) - 1]      # -1 and S are invalid slots
        if checked and op not in ("step", "fill") and rng.rand() < 0.3:              # name some slots again
            slots = [int(x) for x in rng.choice(slots, size=min(S, n + int(rng.randint(1, 4))))]
            n = len(slots)
        if op == "open":
            plens = [int(rng.randint(0, 3 * ps + 2)) for _ in slots]
            cs = None if rng.rand() < 0.3 else [int(rng.choice([1, 2, 3, 4, 7])) for _ in slots]
            res = pair.open(slots, plens, cs)
            opened = [(s_, p_) for s_, p_, r_ in zip(slots, plens, res) if r_ == "OK"]
            if opened and sum(p_ for _, p_ in opened):     # the prompts' K/V, so that the attention outputs below mean something
                pair.prefill(0, [s_ for s_, _ in opened], [p_ for _, p_ in opened], *kv(sum(p_ for _, p_ in opened)))
        elif op == "restore":
            # mostly onto sequences that are still fresh, so that restores succeed too
            fresh = [s for s in range(S) if (st := pair.model.state(s)) and st["t"] == 0]
            if fresh and rng.rand() < 0.7:
                slots = fresh[:n]
                n = len(slots)
            gen_lens = [int(rng.randint(0, 4 * ps + 6)) for _ in slots]
            nb = sum(T // st["c"] for s, T in zip(slots, gen_lens) if (st := pair.model.state(s)) and st["c"] > 1)
            tk, tv = kv(max(sum(gen_lens), 1))
            bk, bv = kv(max(nb, 1))
            pair.restore(0, slots, gen_lens, tk[:sum(gen_lens)], tv[:sum(gen_lens)], bk[:nb], bv[:nb])
        elif op == "append":
            pair.append(0, slots, *kv(n))
        elif op == "step":      # bc_decode_step: refused items (bad slot, full window, no page) still get their attention
            q = randn_bf16(g, (n, Hkv * G, D), DEV)
            _, out, ref = pair.step(0, slots, q, *kv(n), 0.2)
            torch.cuda.synchronize()
            assert_close(out, ref, f"program step {step}: bc_decode_step")
        elif op == "fill":      # bc_fill_step, mostly on sequences one entry short of a full window
            ready = [s for s in range(S) if (st := pair.model.state(s)) and st["c"] > 1 and st["window_len"] == st["c"] - 1]
            if ready and rng.rand() < 0.7:
                slots = ready[:n]
                n = len(slots)
            q, bq = randn_bf16(g, (n, Hkv * G, D), DEV), randn_bf16(g, (n, Hkv * G, D), DEV)
            k, v = kv(n)
            bk, bv = kv(n)
            _, _, out, out_b, ref, ref_b = pair.fill(0, slots, q, k, v, bq, bk, bv, 0.2)
            torch.cuda.synchronize()
            assert_close(out, ref, f"program step {step}: bc_fill_step token rows")
            assert_close(out_b, ref_b, f"program step {step}: bc_fill_step beacon rows")
        elif op == "compress":
            # favour the sequences whose window is full, so that compressions succeed too
            full = [s for s in range(S) if (st := pair.model.state(s)) and st["c"] > 1 and st["window_len"] == st["c"]]
            if full and rng.rand() < 0.7:
                slots = full[:n]
            pair.compress(0, slots, *kv(len(slots)))
        else:
            pair.close(slots)
        pair.check_state()
        if pair.model.first_error is not None and rng.rand() < 0.5:
            pair.gpu.bc_clear_error(); pair.model.first_error = None
    open_slots = [s for s in range(S) if pair.model.state(s) is not None]
    if open_slots:
        pair.close(open_slots)
    pair.gpu.bc_clear_error(); pair.model.first_error = None
    pair.check_state()
    assert sorted(pair.gpu.bc_get_free_list()) == list(range(num_pages))
