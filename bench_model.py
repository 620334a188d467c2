"""A decoder of the 1.5B shape with random weights around the cache library, for end-to-end timing.

What is measured with it: the time to generate N tokens per sequence with the uncompressed cache
(ratio 1) and with Breadcrumbs compression at ratio c -- the protocol behind the paper's only
timing figure (its latency table: generation latency relative to the uncompressed teacher).

Only the cache side (bc_append, bc_decode_attn, bc_compress) is this repository's product.  The
rest of the forward pass -- the embedding lookup and the QKV / output / MLP / LM-head projections (GEMMs) --
are plain PyTorch operators standing in for a model; the rotary embedding and the split of the packed QKV
rows (bc_rope_split, bc_rope_decode_step), the residual add with RMSNorm (bc_add_rmsnorm), the gated MLP
activation (bc_swiglu) and the greedy choice (bc_argmax) are the library's kernels unless lib_rope=False,
which puts the PyTorch operators back for comparison
(random weights: the token stream is meaningless, the shapes and the data flow are real).  Every
sampled token is fed back, and when a window fills, the beacon token's forward pass runs through
the same layers: its query attends with its own K/V as the extra entry, then the window is evicted
(Algorithm 1).  By default the beacon does not get a pass of its own: it is fed together with the
token that fills the window, as a 2-token forward pass (the beacon's input is a fixed special token,
so nothing it needs depends on that token's output), and per layer the two query sets share one pass
over the cache (bc_decode_attn_pair).  One decode step (and one fill or beacon step) is captured in a
CUDA graph and replayed.
"""
from __future__ import annotations

import math

import torch

from paper_2510_13797_b200 import binding as B


class ToyDecoder:
    def __init__(self, batch, c, gen_len, prompt_len=512, layers=28, hidden=1536, q_heads=12, kv_heads=2, head_dim=128,
                 mlp=8960, vocab=151936, device="cuda", seed=0, weights=None, paired=True, lib_rope=True, theta=1e6):
        self.B, self.c, self.L, self.H = batch, c, layers, hidden
        self.lib_rope, self.theta = lib_rope, theta
        self.paired = paired    # True: the beacon is encoded together with the token that fills the window
                                # (one 2-token forward pass, bc_decode_attn_pair), False: in a forward pass of its own
        self.Hq, self.Hkv, self.D, self.V = q_heads, kv_heads, head_dim, vocab
        self.dev = torch.device(device)
        g = torch.Generator(device=self.dev); g.manual_seed(seed)
        rnd = lambda *s, scale=1.0: (torch.randn(s, generator=g, device=self.dev) * scale).to(torch.bfloat16)
        if weights is None:
            sc = 1.0 / math.sqrt(hidden)
            weights = dict(
                emb=rnd(vocab + 1, hidden),                    # last row: the beacon token
                wqkv=[rnd(hidden, (q_heads + 2 * kv_heads) * head_dim, scale=sc) for _ in range(layers)],
                wo=[rnd(q_heads * head_dim, hidden, scale=sc) for _ in range(layers)],
                wgu=[rnd(hidden, 2 * mlp, scale=sc) for _ in range(layers)],
                wdown=[rnd(mlp, hidden, scale=1.0 / math.sqrt(mlp)) for _ in range(layers)],
                head=rnd(hidden, vocab, scale=sc))
        self.weights = weights                                 # may be handed to another instance
        self.emb, self.wqkv, self.wo = weights["emb"], weights["wqkv"], weights["wo"]
        self.wgu, self.wdown, self.head = weights["wgu"], weights["wdown"], weights["head"]
        ps = 16
        cd = lambda a, b: -(-a // b)
        pps = cd(prompt_len, ps) + (cd(c, ps) + cd(cd(gen_len, c), ps) if c > 1 else cd(gen_len, ps)) + 2
        self.cache = B.Cache(layers, kv_heads, q_heads, head_dim, c, ps, max_seqs=batch, num_pages=batch * pps,
                             max_pages_per_seq=pps, device=self.dev)
        self.slots = torch.arange(batch, dtype=torch.int32, device=self.dev)
        self.cache.bc_seq_open(self.slots, torch.full((batch,), prompt_len, dtype=torch.int32, device=self.dev))
        cu = torch.arange(0, (batch + 1) * prompt_len, prompt_len, dtype=torch.int32, device=self.dev)
        for l in range(layers):                               # the prompt's K/V: random stand-ins for a prefill pass
            self.cache.bc_prefill(l, self.slots, cu, batch * prompt_len, rnd(batch * prompt_len, kv_heads, head_dim),
                                  rnd(batch * prompt_len, kv_heads, head_dim))
        self.tok = torch.zeros(batch, dtype=torch.int64, device=self.dev)      # last sampled token
        self.pos = torch.full((1,), prompt_len, dtype=torch.int64, device=self.dev)
        self.attn_out = self.cache.new_out(batch)
        self.attn_out2 = self.cache.new_out(2 * batch)         # the paired step: token rows, then beacon rows
        self.inv_freq = 1.0 / (theta ** (torch.arange(0, head_dim, 2, device=self.dev, dtype=torch.float32) / head_dim))
        # the library's rotation takes one position per row: rows [0, B) at pos, rows [B, 2B) (the beacons of a paired step) at pos + 1
        self.posv = torch.cat((torch.full((batch,), prompt_len, dtype=torch.int32, device=self.dev),
                               torch.full((batch,), prompt_len + 1, dtype=torch.int32, device=self.dev)))
        self.xbuf = torch.empty((2 * batch, hidden), dtype=torch.bfloat16, device=self.dev)    # norm output
        self.actbuf = torch.empty((2 * batch, mlp), dtype=torch.bfloat16, device=self.dev)     # gated MLP activation
        self.q2 = self.cache.new_out(2 * batch)
        self.k2 = torch.empty((2 * batch, kv_heads, head_dim), dtype=torch.bfloat16, device=self.dev)
        self.v2 = torch.empty_like(self.k2)
        self.scale = 1.0 / math.sqrt(head_dim)
        self.graph_tok = self.graph_bea = None
        self.trace = None       # a list: every cache call of an eager step appends (kind, layer, packed QKV rows, positions, outputs)

    # -- stand-ins for the rest of the model -------------------------------------------------------
    @staticmethod
    def _norm(x):
        return (x.float() * torch.rsqrt(x.float().pow(2).mean(-1, keepdim=True) + 1e-6)).to(torch.bfloat16)

    def _rope(self, x, offset=None):
        pos = self.pos.float() if offset is None else (self.pos.float() + offset).view(-1, 1, 1)
        ang = pos * self.inv_freq
        cos, sin = ang.cos(), ang.sin()
        x1, x2 = x.float()[..., 0::2], x.float()[..., 1::2]
        return torch.stack((x1 * cos - x2 * sin, x1 * sin + x2 * cos), dim=-1).flatten(-2).to(torch.bfloat16)

    def _split(self, qkv, offset=None):
        """Rotated q and k and v of the packed rows: the library's kernel, or the PyTorch operators."""
        Hq, Hkv, D = self.Hq, self.Hkv, self.D
        n = qkv.shape[0]
        if self.lib_rope:
            q, k, v = self.q2[:n], self.k2[:n], self.v2[:n]
            self.cache.bc_rope_split(qkv, self.posv[:n], self.theta, q, k, v)
            return q, k, v
        q = self._rope(qkv[:, :Hq * D].view(-1, Hq, D), offset).contiguous()
        k = self._rope(qkv[:, Hq * D:(Hq + Hkv) * D].view(-1, Hkv, D), offset).contiguous()
        v = qkv[:, (Hq + Hkv) * D:].view(-1, Hkv, D).contiguous()
        return q, k, v

    def _record(self, kind, layer, qkv, n, out):
        if self.trace is not None:
            self.trace.append((kind, layer, qkv.clone(), self.posv[:n].clone(), out.clone()))

    def _pre(self, h, delta):
        """Residual add and the norm in front of a block: returns (h + delta, norm(h + delta))."""
        if self.lib_rope:
            x = self.xbuf[:h.shape[0]]
            B.bc_add_rmsnorm(h, delta, None, 1e-6, h, x)          # in place on the residual stream
            return h, x
        if delta is not None:
            h = h + delta
        return h, self._norm(h)

    def _mlp_act(self, gu):
        if self.lib_rope:
            act = self.actbuf[:gu.shape[0]]
            B.bc_swiglu(gu, act)
            return act
        gate, up = gu.chunk(2, dim=-1)
        return torch.nn.functional.silu(gate) * up

    def _sample(self, h, delta):
        """Final norm, LM head, greedy choice into self.tok."""
        _, x = self._pre(h, delta)
        logits = x @ self.head
        if self.lib_rope:
            B.bc_argmax(logits, self.tok)
        else:
            self.tok.copy_(torch.argmax(logits, dim=-1))

    def _forward(self, ids, beacon):
        h, delta = self.emb[ids], None
        Hq, Hkv, D = self.Hq, self.Hkv, self.D
        for l in range(self.L):
            h, x = self._pre(h, delta)
            qkv = x @ self.wqkv[l]
            if self.lib_rope and not beacon:    # rotation, then the append and the attention in one kernel
                self.cache.bc_rope_decode_step(l, self.slots, qkv, self.posv[:self.B], self.theta, self.attn_out, self.scale)
                self._record("token", l, qkv, self.B, self.attn_out)
            else:
                q, k, v = self._split(qkv)
                if beacon:      # the beacon's query sees the cache plus its own entry; then the window goes
                    self.cache.bc_decode_attn(l, self.slots, q, self.attn_out, self.scale, k, v)
                    self.cache.bc_compress(l, self.slots, k, v)
                    self._record("beacon", l, qkv, self.B, self.attn_out)
                else:
                    self.cache.bc_append(l, self.slots, k, v)
                    self.cache.bc_decode_attn(l, self.slots, q, self.attn_out, self.scale)
            h, x = self._pre(h, self.attn_out.view(-1, Hq * D) @ self.wo[l])
            delta = self._mlp_act(x @ self.wgu[l]) @ self.wdown[l]
        return h, delta

    def _forward_pair(self):
        """The token that fills the window and the beacon as one 2-token pass: rows [0, B) are the
        tokens (position pos), rows [B, 2B) the beacons (position pos + 1).  Per layer the token's entry
        is appended, both query sets attend in one pass over the cache (the beacon also sees its own
        entry), and the window is evicted (bc_fill_step; with lib_rope=False the three separate calls)."""
        Bn, Hq, Hkv, D = self.B, self.Hq, self.Hkv, self.D
        h, delta = self.emb[torch.cat((self.tok, torch.full_like(self.tok, self.V)))], None
        offset = torch.cat((torch.zeros(Bn, device=self.dev), torch.ones(Bn, device=self.dev)))
        for l in range(self.L):
            h, x = self._pre(h, delta)
            qkv = x @ self.wqkv[l]
            q, k, v = self._split(qkv, offset)
            if self.lib_rope:
                self.cache.bc_fill_step(l, self.slots, q[:Bn], k[:Bn], v[:Bn], q[Bn:], k[Bn:], v[Bn:], self.attn_out2[:Bn],
                                        self.attn_out2[Bn:], self.scale)
            else:
                self.cache.bc_append(l, self.slots, k[:Bn], v[:Bn])
                self.cache.bc_decode_attn_pair(l, self.slots, q[:Bn], self.attn_out2[:Bn], q[Bn:], self.attn_out2[Bn:], self.scale,
                                               k[Bn:], v[Bn:])
                self.cache.bc_compress(l, self.slots, k[Bn:], v[Bn:])
            self._record("pair", l, qkv, 2 * Bn, self.attn_out2)
            h, x = self._pre(h, self.attn_out2.view(-1, Hq * D) @ self.wo[l])
            delta = self._mlp_act(x @ self.wgu[l]) @ self.wdown[l]
        return h[:Bn], delta[:Bn]

    def _fill_step(self):
        self._sample(*self._forward_pair())
        self.pos.add_(2); self.posv.add_(2)

    def _token_step(self):
        self._sample(*self._forward(self.tok, beacon=False))
        self.pos.add_(1); self.posv.add_(1)

    def _beacon_step(self):
        self._forward(torch.full_like(self.tok, self.V), beacon=True)   # its logits are not needed
        self.pos.add_(1); self.posv.add_(1)

    # -- generation ---------------------------------------------------------------------------------
    def capture(self):
        """Warm up and capture one token step (and one beacon step) as CUDA graphs.  The warm-up
        advances the generation by a whole number of windows, so the state stays consistent."""
        warm = self.c if self.c > 1 else 1
        for i in range(1, warm + 1):
            self._step_eager(i)
        torch.cuda.synchronize()
        s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
        self.graph_tok = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph_tok, stream=s, capture_error_mode="thread_local"):
            self._token_step()
        if self.c > 1:      # the captures enqueue nothing: the cache state is untouched by them
            self.graph_bea = torch.cuda.CUDAGraph()
            with torch.cuda.graph(self.graph_bea, stream=s, capture_error_mode="thread_local"):
                if self.paired:
                    self._fill_step()
                else:
                    self._beacon_step()
        torch.cuda.current_stream().wait_stream(s)
        self.generate(warm)          # first replays upload the graphs: keep that out of any timing
        torch.cuda.synchronize()
        return 2 * warm

    def generate(self, n_tokens):
        """Replays n_tokens token steps (n_tokens a multiple of c), with a beacon step after every c."""
        for i in range(1, n_tokens + 1):
            fill = self.c > 1 and i % self.c == 0
            if fill and self.paired:
                self.graph_bea.replay()          # the token that fills the window and its beacon, one pass
            else:
                self.graph_tok.replay()
                if fill:
                    self.graph_bea.replay()

    def _step_eager(self, i):
        fill = self.c > 1 and i % self.c == 0
        if fill and self.paired:
            self._fill_step()
        else:
            self._token_step()
            if fill:
                self._beacon_step()

    def check(self):
        code, slot, call = self.cache.bc_poll_error()
        if code != 0:
            raise RuntimeError(f"device-side error {B.STATUS_NAMES.get(code, code)} slot {slot} call {call}")
        return self.cache.bc_get_state(0)
