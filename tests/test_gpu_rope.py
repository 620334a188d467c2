"""bc_rope_split and bc_rope_decode_step against the fp64 oracle of the rotation (oracle/rope_oracle.py)
and, for the step, the oracle of the cache."""
import math

import numpy as np
import pytest
import torch

from oracle.paging_model import OK
from oracle.rope_oracle import split_and_rope
from paper_2510_13797_b200 import binding as B
from tests.harness import Pair, assert_close, f64, randn_bf16

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _gen(seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return g


def _assert_rotation(gpu, ref, pair_mag, what):
    """A correctly rounded bf16 of the exact value is within half a unit in the last place, 2^-8 |ref| at most;
    the fp32 rotation adds a few 2^-24 of the pair's magnitude before the rounding."""
    g = f64(gpu)
    err = np.abs(g - ref)
    bound = 2.0 ** -8 * np.abs(ref) + 1e-6 * pair_mag
    worst = (err - bound).max()
    assert worst <= 0, f"{what}: {worst:.3e} over the rounding bound at {np.unravel_index((err - bound).argmax(), err.shape)}"


@pytest.mark.parametrize("Hq,Hkv,D,n,theta", [(12, 2, 128, 64, 1e6), (32, 8, 128, 77, 1e4), (4, 4, 64, 1, 1e4),
                                              (16, 1, 64, 130, 5e5), (8, 8, 128, 3, 1e6)])
def test_rope_split_matches_oracle(Hq, Hkv, D, n, theta):
    cache = B.Cache(1, Hkv, Hq, D, 1, 16, max_seqs=4, num_pages=8, max_pages_per_seq=2, device=DEV)
    g = _gen(11)
    qkv = randn_bf16(g, (n, (Hq + 2 * Hkv) * D), DEV)
    rng = np.random.RandomState(5)
    pos = rng.randint(0, 40000, size=n)
    pos[:4] = [0, 1, 131071, 99999][: min(4, n)]      # identity, one step, and angles of 10^5 radians
    positions = torch.tensor(pos, dtype=torch.int32, device=DEV)
    q = torch.full((n, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    k = torch.full((n, Hkv, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    v = torch.full((n, Hkv, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    cache.bc_rope_split(qkv, positions, theta, q, k, v)
    torch.cuda.synchronize()
    rq, rk, rv = split_and_rope(f64(qkv), pos, Hq, Hkv, D, theta)
    x = f64(qkv)
    mag = lambda a: np.tile(np.abs(a[..., : D // 2]) + np.abs(a[..., D // 2:]), 2)
    _assert_rotation(q, rq, mag(x[:, : Hq * D].reshape(n, Hq, D)), "q")
    _assert_rotation(k, rk, mag(x[:, Hq * D:(Hq + Hkv) * D].reshape(n, Hkv, D)), "k")
    assert np.array_equal(f64(v), rv), "v is a copy"
    if n >= 1:                                          # position 0: bit-exact identity
        assert np.array_equal(f64(q[0]), x[0, : Hq * D].reshape(Hq, D))
    assert cache.bc_poll_error()[0] == 0


def test_rope_split_rejects_bad_arguments():
    cache = B.Cache(1, 2, 4, 128, 1, 16, max_seqs=2, num_pages=4, max_pages_per_seq=2, device=DEV)
    qkv = torch.zeros((2, 8 * 128), dtype=torch.bfloat16, device=DEV)
    pos = torch.zeros(2, dtype=torch.int32, device=DEV)
    q, k, v = cache.new_out(2), torch.zeros((2, 2, 128), dtype=torch.bfloat16, device=DEV), torch.zeros((2, 2, 128), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(B.BreadcrumbsError):
        cache.bc_rope_split(qkv, pos, 1.0, q, k, v)                       # theta must exceed 1
    with pytest.raises(B.BreadcrumbsError):
        cache.bc_rope_split(qkv.view(-1)[1:1 + 8 * 128], pos[:1], 1e4, q, k, v)     # misaligned input


@pytest.mark.parametrize("L,Hkv,G,D,ps,c", [(2, 2, 6, 128, 16, 8), (1, 8, 4, 128, 4, 4), (1, 1, 4, 64, 16, 1)])
def test_rope_decode_step_matches_oracles(L, Hkv, G, D, ps, c):
    """Decode steps fed by packed QKV rows: outputs against the oracle chain (fp64 rotation, bf16 storage,
    fp64 attention), stored entries bit-exact against the library's own bc_rope_split, which the test above
    ties to the oracle."""
    Hq = Hkv * G
    pair = Pair(L, Hkv, Hq, D, ps, max_seqs=4, num_pages=4 * (1400 // ps + 8), max_pages_per_seq=1400 // ps + 8)
    g = _gen(23)
    slots, plens = [0, 1, 2, 3], [700, 0, 37, 1200]
    assert pair.open(slots, plens, [c] * 4) == [OK] * 4
    for l in range(L):
        pair.prefill(l, slots, plens, randn_bf16(g, (sum(plens), Hkv, D), DEV), randn_bf16(g, (sum(plens), Hkv, D), DEV))
    theta, scale = 1e6, 1.0 / math.sqrt(D)
    pos = list(plens)
    sl = torch.tensor(slots, dtype=torch.int32, device=DEV)
    for t in range(1, 2 * max(c, 2) + 2):
        for l in range(L):
            qkv = randn_bf16(g, (4, (Hq + 2 * Hkv) * D), DEV)
            ok, out, ref = pair.rope_step(l, slots, qkv, pos, theta, scale)
            torch.cuda.synchronize()
            assert ok == [OK] * 4
            assert_close(out, ref, f"step {t} layer {l}")
            if t == 1:      # what was stored is what bc_rope_split writes
                k = torch.empty((4, Hkv, D), dtype=torch.bfloat16, device=DEV)
                v = torch.empty_like(k)
                pair.gpu.bc_rope_split(qkv, torch.tensor(pos, dtype=torch.int32, device=DEV), theta, pair.gpu.new_out(4), k, v)
                for i, s in enumerate(slots):
                    ek, ev = pair.gpu.bc_export_seq(l, s, plens[i] + 1)
                    assert torch.equal(ek[-1], k[i]) and torch.equal(ev[-1], v[i])
        pos = [p + 1 for p in pos]
        full = [s for s in slots if c > 1 and pair.model.state(s)["window_len"] == c]
        if full:
            for l in range(L):
                pair.compress(l, full, randn_bf16(g, (len(full), Hkv, D), DEV), randn_bf16(g, (len(full), Hkv, D), DEV))
            pos = [p + 1 for p in pos]
    pair.check_state()
