"""Seeded synthetic inputs for the decode hot path.

This module only draws random tensors and describes workload shapes.  It holds
none of the method's arithmetic (no attention, no eviction, no paging), so both
the CUDA path and the CPU oracle can be fed from it: a tensor is generated
once, on whatever device is asked for, and the same bits are handed to both
sides (the oracle gets a host copy).

The paper decodes three reasoning datasets with trained 1.5B / 3.8B models;
neither is available or needed here, because the cost and the results of the
hot path depend only on shapes, lengths and values.  The shapes below are the
benchmark configurations: seeded i.i.d. N(0,1) values rounded to bf16, keys
optionally pre-scaled, one beacon K/V per completed window of c tokens.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import List

import numpy as np
import torch

_KINDS = {"prompt_k": 1, "prompt_v": 2, "k": 3, "v": 4, "q": 5,
          "beacon_k": 6, "beacon_v": 7, "beacon_q": 8}


@dataclass
class Workload:
    name: str
    layers: int
    batch: int
    q_heads: int
    kv_heads: int
    head_dim: int
    page_size: int
    prompt_lens: List[int]
    gen_lens: List[int]
    cs: List[int]
    sm_scale: float
    k_prescale: float = 1.0          # applied to prompt and token keys before bf16 rounding
    beacon_k_prescale: float = 1.0
    seed: int = 0
    notes: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def group(self):
        return self.q_heads // self.kv_heads

    @property
    def entry_bytes(self):
        """Bytes of one cache entry in one layer: K and V of every KV head, bf16."""
        return 2 * self.kv_heads * self.head_dim * 2

    @property
    def steps(self):
        return max(self.gen_lens)


def _uniform(batch, value):
    return [int(value)] * batch


def make_workload(name: str, c: int | None = None, seed: int = 0, **over) -> Workload:
    """The benchmark configurations, by name.

    tiny   : 1 layer, batch 1, 2/1 heads, D 64, prompt 64, 512 steps, c 16
    cfg2   : 1 layer, batch 32, 12/2 heads, D 128, prompt 256, 4096 steps, c 16, page 16,
             prompt/token keys pre-scaled by 1/sqrt(128) (softmax scale 1)
    sweep  : 1 layer, batch 64, 32/8 heads, D 128, prompt 512, 16384 steps,
             c in {2,4,8,16,32} with page_size = c, or c = 1 (uncompressed, page 16)
    ragged : 1 layer, batch 128, 12/2 heads, D 128, page 16, per-sequence prompt
             U[64,1024], generation U[1024,32768], c from {4,8,16}
    depth  : 28 layers, batch 256, 12/2 heads, D 128, prompt 512, 8192 steps, c 8, page 8
    """
    if name == "tiny":
        w = Workload(name, 1, 1, 2, 1, 64, 16, [64], [512], [16 if c is None else c],
                     1.0 / math.sqrt(64), seed=seed)
    elif name == "cfg2":
        cc = 16 if c is None else c
        w = Workload(name, 1, 32, 12, 2, 128, 16, _uniform(32, 256), _uniform(32, 4096),
                     _uniform(32, cc), 1.0, k_prescale=1.0 / math.sqrt(128), seed=seed,
                     notes="keys pre-scaled by 1/sqrt(128), beacon keys left N(0,1), sm_scale 1")
    elif name == "sweep":
        cc = 16 if c is None else c
        ps = cc if cc > 1 else 16
        w = Workload(f"sweep_c{cc}", 1, 64, 32, 8, 128, ps, _uniform(64, 512),
                     _uniform(64, 16384), _uniform(64, cc), 1.0 / math.sqrt(128), seed=seed)
    elif name == "ragged":
        rng = np.random.RandomState(seed + 4)
        B = 128
        w = Workload(name, 1, B, 12, 2, 128, 16,
                     [int(x) for x in rng.randint(64, 1025, size=B)],
                     [int(x) for x in rng.randint(1024, 32769, size=B)],
                     [int(x) for x in rng.choice([4, 8, 16], size=B)],
                     1.0 / math.sqrt(128), seed=seed)
    elif name == "depth":
        cc = 8 if c is None else c
        ps = cc if cc > 1 else 16
        w = Workload(name, 28, 256, 12, 2, 128, ps, _uniform(256, 512), _uniform(256, 8192),
                     _uniform(256, cc), 1.0 / math.sqrt(128), seed=seed)
    else:
        raise ValueError(f"unknown workload {name!r}")
    if over:
        batch = over.get("batch", w.batch)
        if batch != w.batch:
            over.setdefault("prompt_lens", (w.prompt_lens * batch)[:batch])
            over.setdefault("gen_lens", (w.gen_lens * batch)[:batch])
            over.setdefault("cs", (w.cs * batch)[:batch])
        w = replace(w, **over)
    return w


def _mix(seed: int, kind: str, layer: int, chunk: int) -> int:
    """Deterministic 63-bit seed from (seed, tensor kind, layer, chunk index)."""
    x = (seed * 0x9E3779B97F4A7C15 + _KINDS[kind] * 0xBF58476D1CE4E5B9
         + (layer + 1) * 0x94D049BB133111EB + (chunk + 1) * 0xD6E8FEB86659FD93) & (2**64 - 1)
    x ^= x >> 31
    x = (x * 0x7FB5D329728EA185) & (2**64 - 1)
    x ^= x >> 27
    return x & (2**63 - 1)


class InputStream:
    """Draws the tensors of one workload, chunk by chunk, on one device.

    All tensors are bf16.  A chunk of steps holds, for `steps` consecutive
    decode steps: q [steps, B, Hq, D], k and v [steps, B, Hkv, D].  A chunk of
    beacons holds beacon_q [n, B, Hq, D], beacon_k/v [n, B, Hkv, D]; row j of
    beacon chunk 0 belongs to the j-th compression event of each sequence.
    """

    def __init__(self, w: Workload, device="cpu"):
        self.w = w
        self.device = torch.device(device)

    def _randn(self, kind, layer, chunk, shape, scale=1.0):
        g = torch.Generator(device=self.device)
        g.manual_seed(_mix(self.w.seed, kind, layer, chunk))
        x = torch.randn(shape, generator=g, device=self.device, dtype=torch.float32)
        if scale != 1.0:
            x = x * scale
        return x.to(torch.bfloat16)

    def prompt_kv(self, layer=0):
        """Packed prompt K, V: [sum(prompt_lens), Hkv, D] each."""
        w = self.w
        n = int(sum(w.prompt_lens))
        shape = (n, w.kv_heads, w.head_dim)
        return (self._randn("prompt_k", layer, 0, shape, w.k_prescale),
                self._randn("prompt_v", layer, 0, shape))

    def step_chunk(self, layer, chunk, steps, batch=None):
        w = self.w
        B = w.batch if batch is None else batch
        q = self._randn("q", layer, chunk, (steps, B, w.q_heads, w.head_dim))
        k = self._randn("k", layer, chunk, (steps, B, w.kv_heads, w.head_dim), w.k_prescale)
        v = self._randn("v", layer, chunk, (steps, B, w.kv_heads, w.head_dim))
        return q, k, v

    def beacon_chunk(self, layer, chunk, n, batch=None):
        w = self.w
        B = w.batch if batch is None else batch
        q = self._randn("beacon_q", layer, chunk, (n, B, w.q_heads, w.head_dim))
        k = self._randn("beacon_k", layer, chunk, (n, B, w.kv_heads, w.head_dim), w.beacon_k_prescale)
        v = self._randn("beacon_v", layer, chunk, (n, B, w.kv_heads, w.head_dim))
        return q, k, v
