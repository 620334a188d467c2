"""GPU parity of the distillation-loss kernel (Eq. 1) against the fp64 oracle.

Row losses and the batch loss: |gpu - ref| <= 2e-4 * max(1, |ref|) (fp32 arithmetic on bf16 logits
that both sides read exactly).  Gradient (bf16 output): per row, max |gpu - ref| <= 1e-2 of the
row's largest reference magnitude."""
import numpy as np
import pytest
import torch

from oracle.distill_oracle import batch_loss, loss_gradient, row_losses
from paper_2510_13797_b200 import binding as B

pytestmark = pytest.mark.gpu
DEV = "cuda"


def make_case(seed, traj_lens, vocab, top_k, logit_scale=3.0, unused=0):
    g = torch.Generator(device=DEV); g.manual_seed(seed)
    rows = sum(traj_lens)
    z = (torch.randn((rows, vocab), generator=g, device=DEV) * logit_scale).to(torch.bfloat16)
    zt = torch.randn((rows, vocab), generator=g, device=DEV, dtype=torch.float64) * logit_scale
    lpt = torch.log_softmax(zt, dim=1)
    lp, idx = torch.topk(lpt, top_k, dim=1)
    lp = lp.to(torch.float32)
    if unused:
        lp[:, top_k - unused:] = float("-inf")          # unused storage slots carry no mass
    cu = torch.tensor(np.concatenate([[0], np.cumsum(traj_lens)]), dtype=torch.int32, device=DEV)
    return z, idx.to(torch.int32).contiguous(), lp.contiguous(), cu


def check(z, idx, lp, cu, with_grad):
    loss, rl, grad = B.bc_distill_loss(cu, z, idx, lp, with_grad=with_grad)
    torch.cuda.synchronize()
    zz = z.cpu().to(torch.float64).numpy()
    ii, ll, cc = idx.cpu().numpy(), lp.cpu().to(torch.float64).numpy(), cu.cpu().numpy()
    ref_rows = row_losses(zz, ii, ll)
    got = rl.cpu().to(torch.float64).numpy()
    assert np.all(np.isfinite(got))
    assert np.all(np.abs(got - ref_rows) <= 2e-4 * np.maximum(1.0, np.abs(ref_rows))), np.abs(got - ref_rows).max()
    ref = batch_loss(ref_rows, cc)
    assert abs(float(loss) - ref) <= 2e-4 * max(1.0, abs(ref))
    if with_grad:
        ref_g = loss_gradient(zz, ii, ll, cc)
        gg = grad.cpu().to(torch.float64).numpy()
        err = np.abs(gg - ref_g).max(axis=1)
        assert np.all(err <= 1e-2 * np.abs(ref_g).max(axis=1)), (err / np.abs(ref_g).max(axis=1)).max()


@pytest.mark.parametrize("traj_lens,vocab,top_k", [
    ([3], 64, 5),                  # one vector chunk per thread at most
    ([2, 5, 1], 1000, 100),        # the paper's K
    ([4, 4], 4099, 100),           # vocabulary not a multiple of 8: odd rows start off a 16-byte boundary
    ([3, 1], 8200, 17),            # several chunks per thread, ragged
    ([2], 151936, 100),            # the vocabulary size of the 1.5B model the paper trains
])
def test_loss_and_gradient_match_oracle(traj_lens, vocab, top_k):
    z, idx, lp, cu = make_case(1, traj_lens, vocab, top_k)
    check(z, idx, lp, cu, with_grad=True)
    check(z, idx, lp, cu, with_grad=False)


def test_unused_entries_and_empty_trajectory():
    z, idx, lp, cu = make_case(2, [3, 0, 2], 512, 100, unused=30)
    check(z, idx, lp, cu, with_grad=True)


def test_full_vocabulary_is_the_untruncated_divergence():
    z, idx, lp, cu = make_case(3, [2, 2], 256, 256, logit_scale=1.0)
    check(z, idx, lp, cu, with_grad=True)
    # teacher == student: zero loss, zero gradient
    zs = z.to(torch.float64)
    lps, idxs = torch.topk(torch.log_softmax(zs, dim=1), 256, dim=1)
    loss, rl, grad = B.bc_distill_loss(cu, z, idxs.to(torch.int32).contiguous(), lps.to(torch.float32).contiguous(), with_grad=True)
    assert abs(float(loss)) < 1e-5 and float(grad.abs().max()) < 1e-3
