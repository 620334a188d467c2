"""The element-wise and row-wise operators of a decoder layer around the cache, fp64 (TEST INFRASTRUCTURE ONLY).

The paper's models (Experimental Setup: Qwen2.5-1.5B-Instruct, Phi-4-mini-instruct) are standard pre-norm
decoders: residual stream, RMSNorm before the attention and the MLP blocks, a gated MLP with the SiLU
activation, greedy decoding (Algorithm 1 samples the next token from the model's distribution; the latency
protocol decodes greedily).  These are the textbook definitions:

    rmsnorm(x)_i  = x_i / sqrt(mean_j x_j^2 + eps) * w_i
    swiglu(g, u)  = g * sigmoid(g) * u
    argmax(z)     = the lowest index at which z attains its maximum

Pinned by tests/test_model_ops_oracle_pins.py.
"""
import numpy as np


def add_rmsnorm(h, delta, weight=None, eps=1e-6):
    """Residual add followed by RMSNorm: returns (h + delta, rmsnorm(h + delta)).  h, delta: [..., H]."""
    s = np.asarray(h, dtype=np.float64) + (0.0 if delta is None else np.asarray(delta, dtype=np.float64))
    y = s / np.sqrt(np.mean(s * s, axis=-1, keepdims=True) + eps)
    if weight is not None:
        y = y * np.asarray(weight, dtype=np.float64)
    return s, y


def swiglu(gate_up):
    """gate_up: [..., 2 M], the gate in the first half of the last dimension, the up projection in the second."""
    gu = np.asarray(gate_up, dtype=np.float64)
    m = gu.shape[-1] // 2
    g, u = gu[..., :m], gu[..., m:]
    return g / (1.0 + np.exp(-g)) * u


def argmax_rows(z):
    """z: [n, V]; the lowest index of each row's maximum (NaNs are not expected)."""
    return np.argmax(np.asarray(z, dtype=np.float64), axis=-1)
