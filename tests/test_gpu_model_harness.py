"""The random-weight decoder harness around the cache calls: the generation loop keeps the cache's
bookkeeping where Algorithm 1 puts it, with the beacon encoded in a pass of its own and with the
beacon riding along with the token that fills the window (one 2-token pass)."""
import pytest
import torch

from oracle.breadcrumbs_oracle import closed_form_length
from bench_model import ToyDecoder

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
