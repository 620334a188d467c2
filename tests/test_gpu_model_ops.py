"""bc_add_rmsnorm, bc_swiglu and bc_argmax against their fp64 oracle (oracle/model_ops_oracle.py)."""
import numpy as np
import pytest
import torch

from oracle.model_ops_oracle import add_rmsnorm, argmax_rows, swiglu
from paper_2510_13797_b200 import binding as B
from tests.harness import f64, randn_bf16

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _gen(seed):
    g = torch.Generator(device=DEV)
    g.manual_seed(seed)
    return g


def _bf16_of(a):
    return torch.from_numpy(np.asarray(a)).to(torch.bfloat16).to(torch.float64).numpy()


@pytest.mark.parametrize("n,H,with_delta,with_weight,in_place", [(64, 1536, True, False, True), (3, 8, True, True, False),
                                                                 (130, 8192, True, True, True), (1, 3072, False, True, False),
                                                                 (7, 2048, False, False, False)])
def test_add_rmsnorm_matches_oracle(n, H, with_delta, with_weight, in_place):
    g = _gen(3)
    h = randn_bf16(g, (n, H), DEV, scale=3.0)
    delta = randn_bf16(g, (n, H), DEV, scale=0.7) if with_delta else None
    w = randn_bf16(g, (H,), DEV) if with_weight else None
    eps = 1e-6
    h0 = f64(h)
    h_out = h if in_place else torch.full_like(h, float("nan"))
    normed = torch.full_like(h, float("nan"))
    B.bc_add_rmsnorm(h, delta, w, eps, h_out, normed)
    torch.cuda.synchronize()
    s_ref, _ = add_rmsnorm(h0, None if delta is None else f64(delta), eps=eps)
    # the residual stream: the exact sum rounded to bf16 (the kernel adds in fp32 first: one unit in the last place at most)
    s_gpu = f64(h_out)
    assert np.all(np.abs(s_gpu - s_ref) <= 2.0 ** -7 * np.abs(s_ref) + 1e-30)
    if delta is None:
        assert np.array_equal(s_gpu, h0)
    exact = np.abs(s_gpu - _bf16_of(s_ref)) == 0
    assert exact.mean() > 0.999
    # the norm, from the residual stream as the kernel stored it
    _, y_ref = add_rmsnorm(s_gpu, None, None if w is None else f64(w), eps=eps)
    y = f64(normed)
    assert np.all(np.isfinite(y))
    assert np.all(np.abs(y - y_ref) <= 2.0 ** -8 * np.abs(y_ref) * (1 + 1e-3) + 1e-6 * np.abs(y_ref).max())


def test_add_rmsnorm_without_residual_output_and_bad_arguments():
    g = _gen(4)
    h = randn_bf16(g, (5, 64), DEV)
    keep = h.clone()
    normed = torch.empty_like(h)
    B.bc_add_rmsnorm(h, None, None, 1e-5, None, normed)
    torch.cuda.synchronize()
    assert torch.equal(h, keep)
    _, y_ref = add_rmsnorm(f64(h), None, eps=1e-5)
    assert np.all(np.abs(f64(normed) - y_ref) <= 2.0 ** -8 * np.abs(y_ref) + 1e-6)
    with pytest.raises(B.BreadcrumbsError):
        B.bc_add_rmsnorm(randn_bf16(g, (2, 12), DEV), None, None, 1e-5, None, torch.empty((2, 12), dtype=torch.bfloat16, device=DEV))   # hidden % 8
    with pytest.raises(B.BreadcrumbsError):
        B.bc_add_rmsnorm(randn_bf16(g, (1, 16384), DEV), None, None, 1e-5, None, torch.empty((1, 16384), dtype=torch.bfloat16, device=DEV))


@pytest.mark.parametrize("n,M", [(64, 8960), (3, 8), (129, 4096)])
def test_swiglu_matches_oracle(n, M):
    g = _gen(5)
    gu = randn_bf16(g, (n, 2 * M), DEV, scale=4.0)
    gu[0, :8] = torch.tensor([0.0, 40.0, -40.0, 88.0, -88.0, 1.0, -1.0, 0.5], dtype=torch.bfloat16, device=DEV)   # saturating gates
    out = torch.full((n, M), float("nan"), dtype=torch.bfloat16, device=DEV)
    B.bc_swiglu(gu, out)
    torch.cuda.synchronize()
    ref = swiglu(f64(gu))
    o = f64(out)
    assert np.all(np.isfinite(o))
    # fp32 arithmetic with the fast exponential (relative error of the order of 1e-6), then one rounding to bf16
    assert np.all(np.abs(o - ref) <= (2.0 ** -8 + 1e-5) * np.abs(ref) + 1e-30)


@pytest.mark.parametrize("n,V", [(64, 151936), (5, 8), (3, 1000)])
def test_argmax_matches_oracle(n, V):
    g = _gen(6)
    z = randn_bf16(g, (n, V), DEV, scale=5.0)     # bf16 logits: ties for the maximum are common at large V
    z[0, V - 1] = 1000.0
    z[1, 0] = 1000.0
    if V >= 1000:
        z[2, 17] = 999.0; z[2, 600] = 999.0; z[2, 999] = 999.0          # the lowest index of equal maxima
    if V > 100000:
        z[3, 150000] = 998.0; z[3, 100] = 998.0; z[3, 100000] = 998.0   # equal maxima in slices of different blocks of the row's cluster
        z[4, :] = float("-inf")                                          # nothing exceeds the start value: index 0
    out = torch.full((n,), -1, dtype=torch.int64, device=DEV)
    B.bc_argmax(z, out)
    torch.cuda.synchronize()
    ref = argmax_rows(f64(z))
    assert np.array_equal(out.cpu().numpy(), ref)
    assert int(out[0]) == V - 1 and int(out[1]) == 0
    if V > 100000:
        assert int(out[3]) == 100 and int(out[4]) == 0
