"""Plain fp64 CPU oracle for Breadcrumbs Reasoning inference (cache side).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the
benchmark's CPU-baseline leg.  It shares no code with the CUDA path and the
product never falls back to it.

What it follows
---------------
* Algorithm 1 (the inference loop): after every c generated tokens a beacon
  token is encoded (its K/V entry is appended to the cache), then the cache is
  re-sliced so that the c entries before the beacon disappear and the beacon
  stays.  ``SeqCache.compress`` performs that slice literally on one flat
  Python list.
* Section 3.1: the token sampled right before the beacon is fed again after
  it, so the evicted window is the c tokens whose entries are already cached
  and the re-fed token opens the next window.
* Section 2 (the method keeps the ordinary Transformer attention) and the caption of
  Figure 2: a query attends, with ordinary softmax attention, to whatever the
  cache holds: question tokens, all earlier beacons, the tokens of the current
  window, and itself.  ``attention`` is that definition written out.
* Figure 2 / Section 3.2: at training time the same computation is obtained
  with an attention mask instead of eviction.  ``mask_form_outputs`` builds the
  interleaved sequence and the mask densely; it is an independent second
  formulation used to pin the eviction-form results.

Parity status: every function here is pinned by tests/test_oracle_pins.py
(closed forms, invariants, special cases, mask-form vs eviction-form, brute
force on tiny inputs).  Nothing is "parity unpinned".

Readings taken where the paper is silent (also listed in the design notes):
compression ratio 1 means "never compress" (the tables put the uncompressed
teacher in column 1); the beacon query attends to its own entry; a generated
token attends to itself (append, then attend); an empty cache gives a zero
output vector.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "attention",
    "SeqCache",
    "mask_form_outputs",
    "closed_form_length",
    "closed_form_live_ids",
]


# --------------------------------------------------------------------------
# Attention: the plain definition (Section 2: ordinary Transformer attention)
# --------------------------------------------------------------------------
def attention(q, K, V, sm_scale):
    """Softmax attention of Hq query heads over n cached entries, in fp64.

    q : [Hq, D]      K, V : [n, Hkv, D]      returns [Hq, D]

    Grouped-query attention: query head h reads KV head h // (Hq // Hkv).
    o_h = sum_j softmax_j(sm_scale * <q_h, k_j>) * v_j.
    With n == 0 the sum is empty and the output is zero.
    """
    q = np.asarray(q, dtype=np.float64)
    K = np.asarray(K, dtype=np.float64)
    V = np.asarray(V, dtype=np.float64)
    Hq, D = q.shape
    out = np.zeros((Hq, D), dtype=np.float64)
    n = K.shape[0]
    if n == 0:
        return out
    Hkv = K.shape[1]
    assert Hq % Hkv == 0
    G = Hq // Hkv
    for h in range(Hq):
        kv = h // G
        s = sm_scale * (K[:, kv, :] @ q[h])          # [n] logits
        p = np.exp(s - np.max(s))
        p = p / np.sum(p)
        out[h] = p @ V[:, kv, :]
    return out


# --------------------------------------------------------------------------
# One sequence's cache: explicit flat list, literal eviction (Algorithm 1)
# --------------------------------------------------------------------------
class SeqCache:
    """KV cache of one sequence, one flat Python list per layer.

    Every element is ``(kind, ident, k, v)`` with kind in {"prompt", "token",
    "beacon"}, ident the index of that prompt token / generated token / beacon
    (beacons count from 1), and k, v fp64 arrays [Hkv, D].
    """

    def __init__(self, layers, c):
        if c < 1:
            raise ValueError("compression ratio must be >= 1")
        self.c = int(c)
        self.cache = [[] for _ in range(layers)]
        self.t = 0           # generated-token entries appended so far (layer 0)
        self.n_beacons = 0   # beacons kept so far (counted when the last layer compresses)

    # -- Algorithm 1, initialisation: the prompt is encoded first --------------
    def prefill(self, layer, k, v):
        k = np.asarray(k, dtype=np.float64)
        v = np.asarray(v, dtype=np.float64)
        assert not self.cache[layer], "prefill goes first"
        for j in range(k.shape[0]):
            self.cache[layer].append(("prompt", j, k[j], v[j]))

    # -- Algorithm 1, sampling step: the forward pass of a token appends its entry
    def append(self, layer, k, v):
        if self.c > 1 and self.window_len(layer) >= self.c:
            raise RuntimeError("window full: compress before appending")
        ident = sum(1 for e in self.cache[layer] if e[0] == "token") + self.c * self._beacons_in(layer)
        self.cache[layer].append(("token", ident, np.asarray(k, np.float64), np.asarray(v, np.float64)))
        if layer == 0:
            self.t += 1

    # -- the attention read of a decode step ---------------------------------
    def attend(self, layer, q, sm_scale):
        K, V = self._stack(self.cache[layer])
        return attention(q, K, V, sm_scale)

    # -- Algorithm 1, beacon encoding: its query sees the cache plus itself
    def beacon_attend(self, layer, q_b, beacon_k, beacon_v, sm_scale):
        tail = ("beacon", self._beacons_in(layer) + 1,
                np.asarray(beacon_k, np.float64), np.asarray(beacon_v, np.float64))
        K, V = self._stack(self.cache[layer] + [tail])
        return attention(q_b, K, V, sm_scale)

    # -- Algorithm 1, the eviction statement ---------------------------------
    def compress(self, layer, beacon_k, beacon_v):
        c = self.c
        if c <= 1:
            raise RuntimeError("ratio 1 never compresses")
        if self.window_len(layer) != c:
            raise RuntimeError("compress fires only when the window holds c tokens")
        cache = self.cache[layer]
        before = self._three_lists(layer)
        cache.append(("beacon", self._beacons_in(layer) + 1,
                      np.asarray(beacon_k, np.float64), np.asarray(beacon_v, np.float64)))
        # literal slice: drop the c entries before the beacon, keep the beacon
        cache = cache[: -c - 1] + cache[-1:]
        self.cache[layer] = cache
        # the same thing said with three lists: prompt kept, beacon pushed, window cleared
        prompt, beacons, window = before
        expect = prompt + beacons + [cache[-1]]
        assert len(window) == c
        assert [(e[0], e[1]) for e in cache] == [(e[0], e[1]) for e in expect]
        if layer == len(self.cache) - 1:
            self.n_beacons += 1

    # -- Algorithm 1 run over a stored trajectory -------------------------------
    def replay(self, layer, tok_k, tok_v, beacon_k, beacon_v):
        """The sampling loop of Algorithm 1 with the tokens given instead of sampled: every token's
        entry is appended, and each time the window holds c of them the next stored beacon is
        encoded and the window evicted.  tok_k, tok_v: [T, Hkv, D]; beacon_k, beacon_v:
        [floor(T / c), Hkv, D] (ignored when c = 1).  This is the definition a one-call restore of
        the cache has to reproduce."""
        T = np.asarray(tok_k).shape[0]
        m = 0
        for i in range(T):
            self.append(layer, tok_k[i], tok_v[i])
            if self.c > 1 and self.window_len(layer) == self.c:
                self.compress(layer, beacon_k[m], beacon_v[m])
                m += 1
        assert m == (T // self.c if self.c > 1 else 0)

    # -- views ----------------------------------------------------------------
    def window_len(self, layer=0):
        n = 0
        for e in reversed(self.cache[layer]):
            if e[0] != "token":
                break
            n += 1
        return n

    def lengths(self, layer=0):
        """(prompt entries, beacon entries, live window entries)."""
        kinds = [e[0] for e in self.cache[layer]]
        return kinds.count("prompt"), kinds.count("beacon"), kinds.count("token")

    def live_ids(self, layer=0):
        return [(e[0], e[1]) for e in self.cache[layer]]

    def entries(self, layer=0):
        """Stacked K, V of the live entries in cache order, [n, Hkv, D] each."""
        return self._stack(self.cache[layer])

    # -- helpers ----------------------------------------------------------------
    def _beacons_in(self, layer):
        return sum(1 for e in self.cache[layer] if e[0] == "beacon")

    def _three_lists(self, layer):
        cache = self.cache[layer]
        return ([e for e in cache if e[0] == "prompt"],
                [e for e in cache if e[0] == "beacon"],
                [e for e in cache if e[0] == "token"])

    @staticmethod
    def _stack(entries):
        if not entries:
            return np.zeros((0, 1, 1)), np.zeros((0, 1, 1))
        K = np.stack([e[2] for e in entries])
        V = np.stack([e[3] for e in entries])
        return K, V


# --------------------------------------------------------------------------
# Closed forms (cache growth: +1 entry per c generated tokens)
# --------------------------------------------------------------------------
def closed_form_length(P, t, c):
    """Entries held after the step that appended the t-th generated token and
    applied any compression due at that step."""
    if c <= 1:
        return P + t
    return P + t // c + t % c


def closed_form_live_ids(P, t, c):
    """Live (kind, ident) set after t generated tokens (post-compress)."""
    ids = [("prompt", j) for j in range(P)]
    if c <= 1:
        return ids + [("token", i) for i in range(t)]
    nb = t // c
    ids += [("beacon", m) for m in range(1, nb + 1)]
    ids += [("token", i) for i in range(c * nb, t)]
    return ids


# --------------------------------------------------------------------------
# Mask form (Figure 2): the same computation as one dense masked attention
# --------------------------------------------------------------------------
def mask_form_outputs(prompt_k, prompt_v, tok_k, tok_v, tok_q,
                      beacon_k, beacon_v, beacon_q, c, sm_scale):
    """Teacher-forced formulation of one sequence, one layer.

    The full sequence is laid out as [prompt, x_0 .. x_{c-1}, b_1, x_c, ...]: a
    beacon follows every complete window of c generated tokens.  Row r may
    attend column s iff s <= r and (s is a prompt position, or s is a beacon,
    or s is a generated token with no beacon strictly between s and r).  That
    is the mask of Figure 2: question tokens, all previous beacons, earlier
    tokens of the same window, and the position itself.

    Shapes: prompt_* [P,Hkv,D]; tok_k/v [T,Hkv,D]; tok_q [T,Hq,D];
    beacon_k/v [nb,Hkv,D]; beacon_q [nb,Hq,D] with nb = T // c (0 if c <= 1).
    Returns (token outputs [T,Hq,D], beacon outputs [nb,Hq,D]).
    """
    f = lambda a: np.asarray(a, dtype=np.float64)
    prompt_k, prompt_v, tok_k, tok_v, tok_q = map(f, (prompt_k, prompt_v, tok_k, tok_v, tok_q))
    P, Hkv, D = prompt_k.shape
    T, Hq, _ = tok_q.shape
    G = Hq // Hkv
    nb = T // c if c > 1 else 0
    kinds, K, V, Q = [], [], [], []
    for j in range(P):
        kinds.append(("prompt", j)); K.append(prompt_k[j]); V.append(prompt_v[j]); Q.append(np.zeros((Hq, D)))
    for i in range(T):
        kinds.append(("token", i)); K.append(tok_k[i]); V.append(tok_v[i]); Q.append(tok_q[i])
        if c > 1 and (i + 1) % c == 0:
            m = (i + 1) // c
            kinds.append(("beacon", m)); K.append(f(beacon_k[m - 1])); V.append(f(beacon_v[m - 1]))
            Q.append(f(beacon_q[m - 1]))
    N = len(kinds)
    K = np.stack(K) if N else np.zeros((0, Hkv, D))
    V = np.stack(V) if N else np.zeros((0, Hkv, D))
    Q = np.stack(Q) if N else np.zeros((0, Hq, D))
    # number of beacons at positions <= r, used for the "same window" test
    is_beacon = np.array([k[0] == "beacon" for k in kinds])
    is_token = np.array([k[0] == "token" for k in kinds])
    beacons_upto = np.cumsum(is_beacon)
    mask = np.zeros((N, N), dtype=bool)
    for r in range(N):
        for s in range(r + 1):
            if not is_token[s]:
                mask[r, s] = True                      # prompt or beacon: always visible
            else:
                # generated token: visible iff no beacon lies in (s, r)
                before_r = beacons_upto[r] - (1 if is_beacon[r] else 0)
                mask[r, s] = before_r == beacons_upto[s]
    out = np.zeros((N, Hq, D))
    for h in range(Hq):
        S = sm_scale * (Q[:, h, :] @ K[:, h // G, :].T)      # [N, N]
        S = np.where(mask, S, -np.inf)
        S = S - S.max(axis=1, keepdims=True)
        Pm = np.exp(S)
        Pm = Pm / Pm.sum(axis=1, keepdims=True)
        out[:, h, :] = Pm @ V[:, h // G, :]
    tok_rows = [r for r, k in enumerate(kinds) if k[0] == "token"]
    bea_rows = [r for r, k in enumerate(kinds) if k[0] == "beacon"]
    return out[tok_rows], out[bea_rows].reshape(nb, Hq, D)
