"""The random-weight decoder harness around the cache calls: the generation loop keeps the cache's
bookkeeping where Algorithm 1 puts it, with the beacon encoded in a pass of its own and with the
beacon riding along with the token that fills the window (one 2-token pass)."""
import numpy as np
import pytest
import torch

from oracle.breadcrumbs_oracle import SeqCache, closed_form_length
from oracle.rope_oracle import split_and_rope
from bench_model import ToyDecoder
from tests.harness import assert_close, f64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("paired", [True, False])
@pytest.mark.parametrize("c", [1, 4])
def test_harness_generation_keeps_algorithm1_state(paired, c):
    P, n_tokens = 40, 12
    m = ToyDecoder(batch=3, c=c, gen_len=64, prompt_len=P, layers=2, hidden=256, q_heads=4, kv_heads=2, head_dim=64,
                   mlp=512, vocab=1000, device="cuda", paired=paired)
    warm = m.capture()                      # advances the generation by 2 * warm tokens (eager, then one replayed window)
    m.generate(n_tokens)
    torch.cuda.synchronize()
    st = m.check()                          # raises on a latched device error
    t = warm + n_tokens
    assert st["t"] == t
    assert st["prompt_len"] + st["n_beacons"] + st["window_len"] == closed_form_length(P, t, c)
    assert st["n_beacons"] == (t // c if c > 1 else 0)
    assert int(m.pos) == P + t + st["n_beacons"]          # tokens and beacons both take a position
    assert bool(torch.isfinite(m.tok.float()).all()) and int(m.tok.max()) < 1000


@pytest.mark.parametrize("paired", [True, False])
@pytest.mark.parametrize("c", [1, 3])
def test_harness_cache_calls_against_the_oracles(paired, c):
    """Every cache call the decoder makes during eager generation, replayed on the CPU oracles from the packed
    QKV rows the model produced: fp64 rotation at the recorded positions, bf16 storage, Algorithm 1's append /
    beacon pass / eviction on explicit lists, fp64 attention.  The model's own operators (projections, norms,
    MLP) are PyTorch's and are not under test: the oracle starts from their outputs."""
    P, Bn, L, Hq, Hkv, D = 37, 3, 2, 4, 2, 64
    m = ToyDecoder(batch=Bn, c=c, gen_len=64, prompt_len=P, layers=L, hidden=256, q_heads=Hq, kv_heads=Hkv, head_dim=D,
                   mlp=512, vocab=1000, device="cuda", paired=paired, theta=1e4)
    seqs = [SeqCache(L, c) for _ in range(Bn)]
    for l in range(L):
        for i in range(Bn):
            k, v = m.cache.bc_export_seq(l, i, P)
            seqs[i].prefill(l, f64(k), f64(v))
    m.trace = []
    for i in range(1, 3 * max(c, 2) + 2):
        m._step_eager(i)
    torch.cuda.synchronize()
    m.check()
    bf = lambda a: torch.from_numpy(a).to(torch.bfloat16).to(torch.float64).numpy()
    kinds = set()
    for kind, l, qkv, pos, out in m.trace:
        kinds.add(kind)
        q, k, v = split_and_rope(f64(qkv), f64(pos), Hq, Hkv, D, 1e4)
        q, k = bf(q), bf(k)
        if kind in ("token", "pair"):
            for i in range(Bn):
                seqs[i].append(l, k[i], v[i])
            ref = np.stack([seqs[i].attend(l, q[i], m.scale) for i in range(Bn)])
            assert_close(out[:Bn], ref, f"{kind} rows, layer {l}")
        if kind in ("beacon", "pair"):
            o = Bn if kind == "pair" else 0
            assert np.array_equal(f64(pos)[o:o + Bn], f64(pos)[:Bn] + (1 if kind == "pair" else 0))
            ref = np.stack([seqs[i].beacon_attend(l, q[o + i], k[o + i], v[o + i], m.scale) for i in range(Bn)])
            assert_close(out[o:o + Bn], ref, f"beacon rows, layer {l}")
            for i in range(Bn):
                seqs[i].compress(l, k[o + i], v[o + i])
    assert kinds == ({"token"} if c == 1 else ({"token", "pair"} if paired else {"token", "beacon"}))
    st = m.check()
    for i in range(Bn):     # what the cache holds in the end is what the oracle's lists hold
        K, V = seqs[i].entries(L - 1)
        k, v = m.cache.bc_export_seq(L - 1, i, K.shape[0])
        # V is stored as given; K went through the fp32 rotation before its rounding to bf16, the oracle's through fp64
        assert np.array_equal(f64(v), V) and np.all(np.abs(f64(k) - K) <= 2.0 ** -7 * np.abs(K) + 1e-6)
    assert st["prompt_len"] + st["n_beacons"] + st["window_len"] == seqs[0].entries(0)[0].shape[0]
