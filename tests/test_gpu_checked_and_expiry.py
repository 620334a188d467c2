"""Checked mode (BC_FLAG_DEBUG_BOUNDS) and the give-up paths of the bounded waits, on the GPU.

Nothing here faults, traps or hangs: checked mode turns a bad index into a status code and a skipped
or redirected access; a wait whose poll limit is set to 1 runs out at once, the kernel waits (with
the full limit) for what it has in flight and returns with BC_ERR_TIMEOUT in the status record."""
import math

import numpy as np
import pytest
import torch

from oracle.breadcrumbs_oracle import mask_form_outputs
from paper_2510_13797_b200 import binding as B
from tests.harness import Pair, assert_close, f64, randn_bf16
from tests.test_gpu_parity import run_decode

pytestmark = pytest.mark.gpu
DEV = "cuda"


@pytest.mark.parametrize("Hkv,G,D,ps,c,plens,steps", [
    (2, 6, 128, 16, 4, [70, 9], 30),
    (8, 4, 128, 2, 2, [40, 17], 16),
    (1, 16, 64, 16, 1, [30, 8], 24),
    (4, 3, 128, 3, 7, [20, 21, 22, 23], 20),
])
def test_checked_mode_changes_no_result(Hkv, G, D, ps, c, plens, steps):
    """Every step of a decode run with every index checked: same outputs, bookkeeping and content as
    the oracle, and no check fires."""
    n = len(plens)
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=n + 1, num_pages=300, max_pages_per_seq=150, flags=B.BC_FLAG_DEBUG_BOUNDS)
    run_decode(pair, list(range(n)), plens, [c] * n, steps, seed=3, sm_scale=1.0 / math.sqrt(D), content_every=7)
    assert pair.gpu.bc_poll_error()[0] == 0


def _find_page_table_entry(cache, pages):
    """Index, in the metadata buffer seen as int32, of the first of `pages` consecutive page-table
    entries (the test plants a bad page id there; the layout of the buffer is the library's own)."""
    meta = cache.meta.view(torch.int32).cpu().numpy()
    want = np.asarray(pages, dtype=np.int32)
    hits = [i for i in range(len(meta) - len(want) + 1) if np.array_equal(meta[i:i + len(want)], want)]
    assert len(hits) == 1, hits
    return hits[0]


def test_checked_mode_turns_a_corrupt_page_id_into_a_status_code():
    """A page id far outside the pool is planted in a sequence's page-table row (the metadata buffer
    is the caller's memory).  With the flag set the attention kernel, the export kernel and the
    prefill kernel report BC_ERR_DEBUG_CHECK with the bad value and finish; the other sequence's
    results stay the oracle's."""
    Hkv, G, D, ps = 2, 2, 128, 4
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=2, num_pages=64, max_pages_per_seq=24, flags=B.BC_FLAG_DEBUG_BOUNDS)
    g = torch.Generator(device=DEV); g.manual_seed(4)
    plens = [37, 50]
    pair.open([0, 1], plens)
    pair.prefill(0, [0, 1], plens, randn_bf16(g, (87, Hkv, D), DEV), randn_bf16(g, (87, Hkv, D), DEV))
    st = pair.gpu.bc_get_state(0)
    assert len(st["prompt_pages"]) == 10
    at = _find_page_table_entry(pair.gpu, st["prompt_pages"])
    BAD = 10 ** 9
    meta = pair.gpu.meta.view(torch.int32)
    good = int(meta[at + 3])
    meta[at + 3] = BAD
    q = randn_bf16(g, (2, Hkv * G, D), DEV)
    out, ref = pair.attend(0, [0, 1], q, 0.1)
    torch.cuda.synchronize()
    code, value, _ = pair.gpu.bc_poll_error()
    assert (B.STATUS_NAMES[code], value) == ("DEBUG_CHECK", BAD)
    assert bool(torch.isfinite(out.float()).all())
    assert_close(out[1:], ref[1:], "the sequence whose row is intact")
    pair.gpu.bc_clear_error()
    pair.gpu.bc_export_seq(0, 0, 37)
    assert B.STATUS_NAMES[pair.gpu.bc_poll_error()[0]] == "DEBUG_CHECK"
    pair.gpu.bc_clear_error()
    cu = torch.tensor([0, 37], dtype=torch.int32, device=DEV)
    pair.gpu.bc_prefill(0, torch.tensor([0], dtype=torch.int32, device=DEV), cu, 37, randn_bf16(g, (37, Hkv, D), DEV),
                        randn_bf16(g, (37, Hkv, D), DEV))
    assert B.STATUS_NAMES[pair.gpu.bc_poll_error()[0]] == "DEBUG_CHECK"
    # repaired, the cache works again
    meta[at + 3] = good
    pair.gpu.bc_clear_error()
    pair.gpu.bc_seq_close(torch.tensor([0, 1], dtype=torch.int32, device=DEV))
    assert pair.gpu.bc_poll_error()[0] == 0
    assert sorted(pair.gpu.bc_get_free_list()) == list(range(64))


def test_attention_wait_that_runs_out_reports_timeout_and_the_cache_stays_usable():
    """One thread block walks 800 tiles with a poll limit of 1 (two looks at a barrier that do not suspend
    the thread): the producer's wait for a free stage (or a consumer's wait for a tile) runs out at once, the block stops issuing copies,
    waits for those in flight and returns.  The status record says BC_ERR_TIMEOUT; after
    bc_clear_error (which also zeroes the split-K tickets the launch may have left) and with the
    default limit back, the same call gives the oracle's result.  The same with many blocks, where
    tickets of split sequences are left behind."""
    Hkv, G, D, ps = 8, 4, 128, 16
    plens = [9000, 4000]      # 813 tiles of 16 entries: five or six per block even with one block per SM
    pair = Pair(1, Hkv, Hkv * G, D, ps, max_seqs=2, num_pages=830, max_pages_per_seq=570)
    g = torch.Generator(device=DEV); g.manual_seed(8)
    pair.open([0, 1], plens)
    pair.prefill(0, [0, 1], plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    q = randn_bf16(g, (2, Hkv * G, D), DEV)
    for ctas in (1, 0):
        pair.gpu.bc_set_attn_ctas(ctas)
        pair.gpu.bc_set_wait_limit(1)
        pair.attend(0, [0, 1], q, 0.09)
        code, slot, _ = pair.gpu.bc_poll_error()
        assert B.STATUS_NAMES[code] == "TIMEOUT" and slot == -1
        pair.gpu.bc_set_wait_limit(0)
        pair.gpu.bc_clear_error()
        for _ in range(2):
            out, ref = pair.attend(0, [0, 1], q, 0.09)
            assert_close(out, ref, f"after the timeout, ctas={ctas}")
        assert pair.gpu.bc_poll_error()[0] == 0
    # the fused step gives up the same way and appends nothing twice
    pair.gpu.bc_set_wait_limit(1)
    k, v = randn_bf16(g, (2, Hkv, D), DEV), randn_bf16(g, (2, Hkv, D), DEV)
    pair.step(0, [0, 1], q, k, v, 0.09)
    assert B.STATUS_NAMES[pair.gpu.bc_poll_error()[0]] == "TIMEOUT"
    pair.gpu.bc_set_wait_limit(0)
    pair.gpu.bc_clear_error()
    pair.model.first_error = None
    st = pair.gpu.bc_get_state(0)
    assert st["window_len"] == 1 and st["t"] == 1          # the bookkeeping ran once


def test_mask_form_wait_that_runs_out_reports_timeout():
    """The same for the mask-form kernel: with a poll limit of 1 the first wait of every block runs out,
    the blocks wait for the tensor copies (and products) they have in flight, release their tensor
    memory and return; bc_mask_attn_status says BC_ERR_TIMEOUT.  With the default limit back the
    call gives the oracle's rows."""
    Hq, Hkv, D, c = 8, 2, 128, 8
    plens, tlens = [100], [300]
    g = torch.Generator(device=DEV); g.manual_seed(2)
    nb = tlens[0] // c
    pk, pv = randn_bf16(g, (100, Hkv, D), DEV), randn_bf16(g, (100, Hkv, D), DEV)
    tq, tk, tv = randn_bf16(g, (300, Hq, D), DEV), randn_bf16(g, (300, Hkv, D), DEV), randn_bf16(g, (300, Hkv, D), DEV)
    bq, bk, bv = randn_bf16(g, (nb, Hq, D), DEV), randn_bf16(g, (nb, Hkv, D), DEV), randn_bf16(g, (nb, Hkv, D), DEV)
    scale = 1.0 / math.sqrt(D)
    lib = B.lib()
    try:
        assert lib.bc_mask_attn_set_wait_limit(1) == 0
        with pytest.raises(B.BreadcrumbsError) as e:
            B.bc_mask_attn_forward(plens, tlens, c, pk, pv, tq, tk, tv, bq, bk, bv, scale)
        assert e.value.status == B.BC_ERR_TIMEOUT
    finally:
        lib.bc_mask_attn_set_wait_limit(0)
    torch.cuda.synchronize()
    out_t, out_b = B.bc_mask_attn_forward(plens, tlens, c, pk, pv, tq, tk, tv, bq, bk, bv, scale)
    ref_t, ref_b = mask_form_outputs(f64(pk), f64(pv), f64(tk), f64(tv), f64(tq), f64(bk), f64(bv), f64(bq), c, scale)
    assert_close(out_t, ref_t, "tokens after the timeout")
    assert_close(out_b, ref_b, "beacons after the timeout")
