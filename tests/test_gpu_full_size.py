"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times.

The caches are brought to the sampled generation step through the library itself (real bc_append /
bc_compress calls); the expected values never come from the CUDA path: the oracle rebuilds the
content of a sampled sequence from the seeded inputs alone (beacon K/V are inputs, so the cache at
step t is a pure function of the seed: prompt entries, beacons 1..floor((t-1)/c), and the window
tokens since the last beacon -- the oracle's closed-form live set) and applies the plain softmax
definition.  Bookkeeping is compared with the oracle's closed forms and its integer paging model.
"""
import math

import numpy as np
import pytest
import torch

from oracle.breadcrumbs_oracle import attention, closed_form_length, closed_form_live_ids
from oracle.paging_model import OK, PagingModel
from paper_2510_13797_b200 import binding as B
from paper_2510_13797_b200.driver import DecodeDriver
from paper_2510_13797_b200.workloads import InputStream, make_workload
from tests.harness import assert_close, f64

pytestmark = pytest.mark.gpu
DEV = "cuda"


def live_kv(drv: DecodeDriver, s: int, t: int):
    """K, V [entries, Hkv, D] fp64 that the attention of decode step t reads for sequence s: the
    oracle's closed-form live set after t - 1 tokens, plus token t (0-based id t - 1), which was
    appended just before the read; a compression due at t comes after it."""
    P, c = drv.P, drv.c
    ids = closed_form_live_ids(P, t - 1, c) + [("token", t - 1)]
    pk, pv = f64(drv.pk[s * P:(s + 1) * P]), f64(drv.pv[s * P:(s + 1) * P])
    bk, bv = f64(drv.bk[:, s]), f64(drv.bv[:, s])          # this sequence's beacon and token inputs, one copy each
    tk, tv = f64(drv.k[:, s]), f64(drv.v[:, s])
    ks, vs = [], []
    for kind, ident in ids:
        if kind == "prompt":
            ks.append(pk[ident]); vs.append(pv[ident])
        elif kind == "beacon":
            ks.append(bk[ident % drv.bring]); vs.append(bv[ident % drv.bring])
        else:
            ks.append(tk[ident % drv.ring]); vs.append(tv[ident % drv.ring])
    return np.stack(ks), np.stack(vs)


def check_step(drv: DecodeDriver, seqs, what):
    """Runs one driver step and compares the sampled sequences' outputs (all heads)."""
    t = drv.t + 1
    fired = drv.step()
    torch.cuda.synchronize()
    scale = drv.w.sm_scale
    for s in seqs:
        K, V = live_kv(drv, s, t)
        ref = attention(f64(drv.q[(t - 1) % drv.ring, s]), K, V, scale)
        assert_close(drv.out[s], ref, f"{what}: step {t} seq {s}")
        if fired:
            b = (t // drv.c) % drv.bring
            Kb = np.concatenate([K, f64(drv.bk[b, s])[None]]); Vb = np.concatenate([V, f64(drv.bv[b, s])[None]])
            refb = attention(f64(drv.bq[b, s]), Kb, Vb, scale)
            assert_close(drv.out_b[s], refb, f"{what}: beacon query at step {t} seq {s}")
    return fired


def check_lengths_and_conservation(drv: DecodeDriver):
    owned = []
    for s in range(drv.n):
        st = drv.cache.bc_get_state(s)
        assert st["prompt_len"] + st["n_beacons"] + st["window_len"] == closed_form_length(drv.P, drv.t, drv.c)
        assert st["t"] == drv.t and st["c"] == drv.c
        owned += st["prompt_pages"] + st["beacon_pages"] + st["window_pages"]
    free = drv.cache.bc_get_free_list()
    assert len(set(owned)) == len(owned), "a page is owned twice"
    assert not (set(owned) & set(free))
    assert len(owned) + len(free) == drv.num_pages


@pytest.mark.parametrize("c", [2, 4, 8, 16, 32])
def test_sweep_mid_generation(c):
    """The ratio sweep (batch 64, 32/8 heads, D 128, prompt 512, page_size = c) around the middle of
    the 16384-step generation: a whole window of steps including the beacon query and the eviction."""
    w = make_workload("sweep", c=c)
    drv = DecodeDriver(w, DEV, beacon_ring=w.steps // 2 // c + 8)      # every beacon the cache holds is unique
    t0 = (w.steps // 2 // c) * c - 2
    drv.reset_to(t0)
    seqs = [0, 17, 63]
    fired = 0
    for _ in range(min(c, 4) + 2):
        fired += check_step(drv, seqs, f"sweep c={c}")
    assert fired >= 1
    check_lengths_and_conservation(drv)
    drv.check_error()


def test_sweep_mid_generation_fused_step():
    """The same window at c = 16 with the regular steps issued as bc_decode_step (one launch)."""
    w = make_workload("sweep", c=16)
    drv = DecodeDriver(w, DEV, fused=True, beacon_ring=w.steps // 2 // 16 + 8)
    drv.reset_to((w.steps // 2 // 16) * 16 - 2)
    fired = sum(check_step(drv, [3, 31, 60], "sweep c=16 fused") for _ in range(6))
    assert fired >= 1
    check_lengths_and_conservation(drv)
    drv.check_error()


@pytest.mark.parametrize("c,paired,fused", [(2, True, True), (16, True, True), (16, False, False), (32, True, True), (32, True, False),
                                            (4, False, True)])
def test_sweep_window_replayed_as_cuda_graph(c, paired, fused):
    """The launch configuration the benchmark times: whole windows of steps captured once as a CUDA
    graph and replayed.  A replay feeds the inputs of the captured steps again, so the captured span
    is a whole number of input periods (the step inputs repeat every `ring` steps, the beacons every
    37 windows -- a prime longer than a page of beacons, so neighbouring beacons and neighbouring
    beacon pages differ): then the replayed generation is the one the oracle rebuilds from the seeds.  After
    three replays the outputs left by the last step (it fills a window: token rows and beacon rows,
    paired or as two passes) and the bookkeeping must be those of the oracle for that step."""
    w = make_workload("sweep", c=c)
    drv = DecodeDriver(w, DEV, paired=paired, fused=fused, beacon_ring=37)   # fused: regular steps through bc_decode_step, as bench.py times them
    span = math.lcm(drv.ring, drv.bring * c)
    t0 = (w.steps // 2 // span) * span
    drv.reset_to(t0)
    for _ in range(span):                                # one eager span: warms every kernel
        drv.step()
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    t_save = drv.t
    with torch.cuda.graph(graph, stream=side, capture_error_mode="thread_local"):
        for _ in range(span):
            drv.step()
    drv.t = t_save                                       # the capture enqueued nothing
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        graph.replay()
        drv.t += span
    torch.cuda.synchronize()
    drv.check_error()
    t = drv.t                                            # the last replayed step; it filled the window
    assert t % c == 0
    scale, b = w.sm_scale, (t // c) % drv.bring
    for s in (0, 29, 63):
        K, V = live_kv(drv, s, t)
        assert_close(drv.out[s], attention(f64(drv.q[(t - 1) % drv.ring, s]), K, V, scale), f"graph c={c}: step {t} seq {s}")
        Kb = np.concatenate([K, f64(drv.bk[b, s])[None]]); Vb = np.concatenate([V, f64(drv.bv[b, s])[None]])
        assert_close(drv.out_b[s], attention(f64(drv.bq[b, s]), Kb, Vb, scale), f"graph c={c}: beacon rows at step {t} seq {s}")
    check_lengths_and_conservation(drv)


def test_sweep_host_buffer_steps_full_size(host_route):
    """The end-to-end leg of the benchmark: host-buffer steps (packed inputs on the cache's copy stream,
    pipelined outputs; page-locked and pageable buffers) at the sweep's size, c = 4, seven steps back to
    back across two window-fill steps."""
    w = make_workload("sweep", c=4)
    drv = DecodeDriver(w, DEV, beacon_ring=37)
    t0 = (w.steps // 2 // 16) * 16 + 1
    drv.reset_to(t0)
    for _ in range(7):                                   # steps t0+1 .. t0+7; the third and the last fill the window (paired)
        drv.step_host()
    drv.cache.bc_host_outputs_ready()
    torch.cuda.synchronize()
    drv.check_error()
    t = drv.t
    assert t % 4 == 0
    scale, b = w.sm_scale, (t // 4) % drv.bring
    for s in (1, 33, 62):
        K, V = live_kv(drv, s, t)
        assert_close(drv.h["out"][s], attention(f64(drv.q[(t - 1) % drv.ring, s]), K, V, scale), f"host step {t} seq {s}")
        Kb = np.concatenate([K, f64(drv.bk[b, s])[None]]); Vb = np.concatenate([V, f64(drv.bv[b, s])[None]])
        assert_close(drv.h["out_b"][s], attention(f64(drv.bq[b, s]), Kb, Vb, scale), f"host step {t} seq {s}: beacon rows")
    check_lengths_and_conservation(drv)


@pytest.mark.parametrize("fused", [False, True])
def test_sweep_c2_long_run_content_bit_exact(fused):
    """400 steps back to back at c = 2 with pages of 2 entries: a window page is recycled at every
    second step while the next step's bookkeeping already runs beside (one warp) or under the last
    blocks of the attention kernel, and with fused=True (bc_decode_step, bc_fill_step: the calls the
    benchmark times) the compression's kernel stores its beacon rows under that kernel as well.
    Nothing may be overwritten early: the last outputs and the stored content of sampled
    sequences (every prompt entry, beacon and window token, bit for bit) must be the oracle's."""
    w = make_workload("sweep", c=2)
    t0 = (w.steps // 2 // 16) * 16
    drv = DecodeDriver(w, DEV, fused=fused, beacon_ring=(t0 + 400) // 2 + 8)         # every stored beacon is unique
    drv.reset_to(t0)
    for _ in range(399):
        drv.step()
    seqs = [0, 31, 63]
    check_step(drv, seqs, "c=2 long run")               # step t0 + 400: fills a window (paired attention, then compress)
    drv.check_error()
    t = drv.t
    for s in seqs:
        K, V = live_kv(drv, s, t + 1)                   # what step t + 1 would read, minus its own new token
        k, v = drv.cache.bc_export_seq(0, s, K.shape[0])
        n_live = closed_form_length(drv.P, t, 2)
        assert np.array_equal(f64(k)[:n_live], K[:n_live]) and np.array_equal(f64(v)[:n_live], V[:n_live]), f"content of sequence {s}"
    check_lengths_and_conservation(drv)


def test_sweep_uncompressed_mid_generation():
    w = make_workload("sweep", c=1)
    drv = DecodeDriver(w, DEV)
    drv.reset_to(w.steps // 2 - 1)
    for _ in range(2):
        check_step(drv, [5, 40], "sweep uncompressed")
    check_lengths_and_conservation(drv)
    drv.check_error()


def test_sweep_c16_end_of_run_pages_bit_exact():
    """c = 16 to the last step of the generation: page lists and the free stack equal the paging
    model replayed over the same 16384 appends and 1024 compressions."""
    w = make_workload("sweep", c=16)
    drv = DecodeDriver(w, DEV, beacon_ring=w.steps // 16 + 7)           # 1031 > 1024 beacons: all unique
    model = PagingModel(drv.num_pages, w.page_size, w.batch, drv.pages_per_seq, 0, 16)
    slots = list(range(w.batch))
    assert model.open(slots, w.prompt_lens) == [OK] * w.batch
    drv.reset_to(w.steps - 3)
    for t in range(1, w.steps - 2):
        model.append(slots)
        if t % 16 == 0:
            model.compress(slots)
    for _ in range(3):
        check_step(drv, [1, 62], "sweep c=16 end of run")
        model.append(slots)
        if drv.t % 16 == 0:
            model.compress(slots)
    assert drv.t == w.steps
    for s in slots:
        assert drv.cache.bc_get_state(s) == model.state(s), f"slot {s}"
    assert drv.cache.bc_get_free_list() == model.free_list()
    assert model.first_error is None
    drv.check_error()


@pytest.mark.parametrize("fused", [False, True])
def test_cfg2_sampled_steps(fused):
    """Batch 32, 12/2 heads, prompt 256, 4096 steps, c = 16: keys pre-scaled by 1/sqrt(128), beacon
    keys left N(0,1), softmax scale 1 (diffuse logits plus sharp beacon peaks).  fused: through
    bc_decode_step / bc_fill_step, all 4096 steps back to back (the small batch's bookkeeping is one warp
    that runs beside the attention kernel of the step before)."""
    w = make_workload("cfg2")
    drv = DecodeDriver(w, DEV, fused=fused, beacon_ring=w.steps // 16 + 1)           # 257 > 256 beacons: all unique
    model = PagingModel(drv.num_pages, w.page_size, w.batch, drv.pages_per_seq, 0, 16)
    slots = list(range(w.batch))
    model.open(slots, w.prompt_lens)
    drv.reset_to(0)
    sampled = {1, 15, 16, 17, 2048, 4095, 4096, 777, 3000}
    while drv.t < w.steps:
        if drv.t + 1 in sampled:
            check_step(drv, [0, 13, 31], "cfg2")
        else:
            drv.step()
        model.append(slots)
        if drv.t % 16 == 0:
            model.compress(slots)
        if drv.t in sampled or drv.t % 512 == 0:
            for s in (0, 13, 31):
                assert drv.cache.bc_get_state(s) == model.state(s), f"slot {s} at step {drv.t}"
            assert drv.cache.bc_get_free_list() == model.free_list()
    check_lengths_and_conservation(drv)
    drv.check_error()


@pytest.mark.parametrize("fused", [False, True])
def test_ragged_batch_full_size(fused):
    """Batch 128, 12/2 heads, page 16; per-sequence prompt U[64,1024], generation U[1024,32768], c from
    {4,8,16}.  Sequences finish at their own step and free their pages on the device; bookkeeping is
    compared with the paging model at every close and at sampled steps, outputs at sampled
    (step, sequence) pairs, and at the end every page is back on the free stack."""
    w = make_workload("ragged")
    Bn, ps, Hkv, Hq, D = w.batch, w.page_size, w.kv_heads, w.q_heads, w.head_dim
    cd = lambda a, b: -(-a // b)
    max_pps = max(cd(P, ps) + cd(c, ps) + cd(cd(T, c), ps) + 1 for P, T, c in zip(w.prompt_lens, w.gen_lens, w.cs))
    num_pages = sum(cd(P, ps) + cd(c, ps) + cd(cd(T, c), ps) + 1 for P, T, c in zip(w.prompt_lens, w.gen_lens, w.cs))
    cache = B.Cache(1, Hkv, Hq, D, 1, ps, max_seqs=Bn, num_pages=num_pages, max_pages_per_seq=max_pps, device=DEV)
    model = PagingModel(num_pages, ps, Bn, max_pps, 0, 1)
    stream = InputStream(w, DEV)
    pk, pv = stream.prompt_kv(0)
    ring = 16
    q, k, v = stream.step_chunk(0, 0, ring)
    BR = 37                                              # distinct beacons per sequence: a prime longer than a page
    bq, bk, bv = stream.beacon_chunk(0, 0, BR)
    i32 = lambda xs: torch.tensor(list(xs), dtype=torch.int32, device=DEV)
    i64 = lambda xs: torch.tensor(list(xs), dtype=torch.int64, device=DEV)
    all_slots = list(range(Bn))
    cu = np.concatenate([[0], np.cumsum(w.prompt_lens)])
    cache.bc_seq_open(i32(all_slots), i32(w.prompt_lens), i32(w.cs))
    cache.bc_prefill(0, i32(all_slots), i32(cu), int(cu[-1]), pk, pv)
    assert model.open(all_slots, w.prompt_lens, w.cs) == [OK] * Bn
    rng = np.random.RandomState(5)
    T_max = max(w.gen_lens)
    check_steps = set(int(x) for x in rng.randint(1, T_max, size=10)) | {1, 16, 1024, min(w.gen_lens), T_max}
    live = list(all_slots)

    def content(s, t):
        P, c = w.prompt_lens[s], w.cs[s]
        t_done = t - 1 if t % c == 0 else t
        nb = t_done // c
        ks = [f64(pk[cu[s]:cu[s + 1]])] + [f64(bk[m % BR, s])[None] for m in range(1, nb + 1)]
        vs = [f64(pv[cu[s]:cu[s + 1]])] + [f64(bv[m % BR, s])[None] for m in range(1, nb + 1)]
        for i in range(nb * c, t):
            ks.append(f64(k[i % ring, s])[None]); vs.append(f64(v[i % ring, s])[None])
        return np.concatenate(ks), np.concatenate(vs)

    for t in range(1, T_max + 1):
        j = (t - 1) % ring
        idx, sl = i64(live), i32(live)
        out = cache.new_out(len(live))
        qs = q[j].index_select(0, idx)
        if fused:       # as bench.py --workload ragged issues the regular steps
            cache.bc_decode_step(0, sl, qs, k[j].index_select(0, idx), v[j].index_select(0, idx), out, w.sm_scale)
        else:
            cache.bc_append(0, sl, k[j].index_select(0, idx), v[j].index_select(0, idx))
            cache.bc_decode_attn(0, sl, qs, out, w.sm_scale)
        model.append(live)
        if t in check_steps:
            for pos in sorted(set(int(x) for x in rng.randint(0, len(live), size=3))):
                s = live[pos]
                K, V = content(s, t)
                assert_close(out[pos], attention(f64(q[j, s]), K, V, w.sm_scale), f"ragged step {t} seq {s}")
        full = [s for s in live if t % w.cs[s] == 0]
        if full:
            fidx, fsl = i64(full), i32(full)
            b = None
            # beacon number m = t / c differs per sequence: group by m % BR
            for r in sorted(set((t // w.cs[s]) % BR for s in full)):
                grp = [s for s in full if (t // w.cs[s]) % BR == r]
                gidx, gsl = i64(grp), i32(grp)
                gbk, gbv = bk[r].index_select(0, gidx), bv[r].index_select(0, gidx)
                outb = cache.new_out(len(grp))
                cache.bc_decode_attn(0, gsl, bq[r].index_select(0, gidx), outb, w.sm_scale, gbk, gbv)
                if t in check_steps:
                    s = grp[0]
                    K, V = content(s, t)
                    ref = attention(f64(bq[r, s]), np.concatenate([K, f64(bk[r, s])[None]]),
                                    np.concatenate([V, f64(bv[r, s])[None]]), w.sm_scale)
                    assert_close(outb[0], ref, f"ragged beacon step {t} seq {s}")
                cache.bc_compress(0, gsl, gbk, gbv)
                assert model.compress(grp) == [OK] * len(grp)
        done = [s for s in live if t >= w.gen_lens[s]]
        if done:
            cache.bc_seq_close(i32(done))
            assert model.close(done) == [OK] * len(done)
            live = [s for s in live if s not in set(done)]
            assert cache.bc_get_free_list() == model.free_list(), f"free stack after closes at step {t}"
        if t in check_steps:
            for s in live[:4] + live[-4:]:
                assert cache.bc_get_state(s) == model.state(s), f"slot {s} at step {t}"
            assert cache.bc_get_free_list() == model.free_list()
        if not live:
            break
    assert not live
    assert sorted(cache.bc_get_free_list()) == list(range(num_pages))      # conservation: everything came back
    code, slot, call = cache.bc_poll_error()
    assert code == 0 and model.first_error is None


@pytest.mark.parametrize("fused", [False, True])
def test_depth_config_first_windows(fused):
    """28 layers, batch 256, 12/2 heads, prompt 512, c = 8, page 8: three windows of per-layer calls
    in dependency order; sampled (layer, sequence) outputs, and the shared bookkeeping.  fused: the calls
    the benchmark issues (bc_decode_step per layer, bc_fill_step per layer at the step that fills the window)."""
    w = make_workload("depth")
    L, Bn, ps, Hkv, Hq, D, c, P = w.layers, w.batch, w.page_size, w.kv_heads, w.q_heads, w.head_dim, w.cs[0], w.prompt_lens[0]
    steps = 3 * c + 1
    pps = -(-P // ps) + 1 + 2
    cache = B.Cache(L, Hkv, Hq, D, c, ps, max_seqs=Bn, num_pages=Bn * pps, max_pages_per_seq=pps, device=DEV)
    model = PagingModel(Bn * pps, ps, Bn, pps, 0, c)
    slots_l = list(range(Bn))
    slots = torch.arange(Bn, dtype=torch.int32, device=DEV)
    cu = torch.arange(0, (Bn + 1) * P, P, dtype=torch.int32, device=DEV)
    cache.bc_seq_open(slots, torch.full((Bn,), P, dtype=torch.int32, device=DEV))
    model.open(slots_l, w.prompt_lens)
    stream = InputStream(w, DEV)
    sample_layers, sample_seqs = [0, 13, 27], [0, 101, 255]
    kept = {}
    for l in range(L):
        pk, pv = stream.prompt_kv(l)
        cache.bc_prefill(l, slots, cu, Bn * P, pk, pv)
        if l in sample_layers:
            kept[l] = dict(pk=pk, pv=pv, step=stream.step_chunk(l, 0, steps), beacon=stream.beacon_chunk(l, 0, 4))
    out, out_b = cache.new_out(Bn), cache.new_out(Bn)

    def content(l, s, t):
        d = kept[l]
        t_done = t - 1 if t % c == 0 else t
        nb = t_done // c
        ks = [f64(d["pk"][s * P:(s + 1) * P])] + [f64(d["beacon"][1][m, s])[None] for m in range(1, nb + 1)]
        vs = [f64(d["pv"][s * P:(s + 1) * P])] + [f64(d["beacon"][2][m, s])[None] for m in range(1, nb + 1)]
        for i in range(nb * c, t):
            ks.append(f64(d["step"][1][i, s])[None]); vs.append(f64(d["step"][2][i, s])[None])
        return np.concatenate(ks), np.concatenate(vs)

    for t in range(1, steps + 1):
        fill_now = fused and t % c == 0
        for l in range(L):
            q, k, v = kept[l]["step"] if l in kept else stream.step_chunk(l, 0, steps)
            if fill_now:      # append, token and beacon rows in one pass, eviction: one call per layer
                m = t // c
                bq, bk, bv = kept[l]["beacon"] if l in kept else stream.beacon_chunk(l, 0, 4)
                cache.bc_fill_step(l, slots, q[t - 1], k[t - 1], v[t - 1], bq[m], bk[m], bv[m], out, out_b, w.sm_scale)
                if l in kept:
                    s = sample_seqs[1]
                    K, V = content(l, s, t)
                    ref = attention(f64(bq[m, s]), np.concatenate([K, f64(bk[m, s])[None]]),
                                    np.concatenate([V, f64(bv[m, s])[None]]), w.sm_scale)
                    assert_close(out_b[s], ref, f"depth beacon rows, step {t} layer {l}")
            elif fused:
                cache.bc_decode_step(l, slots, q[t - 1], k[t - 1], v[t - 1], out, w.sm_scale)
            else:
                cache.bc_append(l, slots, k[t - 1], v[t - 1])
                cache.bc_decode_attn(l, slots, q[t - 1], out, w.sm_scale)
            if l in kept:
                for s in sample_seqs:
                    K, V = content(l, s, t)
                    assert_close(out[s], attention(f64(q[t - 1, s]), K, V, w.sm_scale), f"depth step {t} layer {l} seq {s}")
        model.append(slots_l)
        if fill_now:
            model.compress(slots_l)
        elif t % c == 0:
            m = t // c
            for l in range(L):
                bq, bk, bv = kept[l]["beacon"] if l in kept else stream.beacon_chunk(l, 0, 4)
                cache.bc_decode_attn(l, slots, bq[m], out, w.sm_scale, bk[m], bv[m])
                if l in kept:
                    s = sample_seqs[1]
                    K, V = content(l, s, t)
                    ref = attention(f64(bq[m, s]), np.concatenate([K, f64(bk[m, s])[None]]),
                                    np.concatenate([V, f64(bv[m, s])[None]]), w.sm_scale)
                    assert_close(out[s], ref, f"depth beacon step {t} layer {l}")
                cache.bc_compress(l, slots, bk[m], bv[m])
            model.compress(slots_l)
        for s in (0, 255):
            assert cache.bc_get_state(s) == model.state(s), f"slot {s} at step {t}"
    assert cache.bc_get_free_list() == model.free_list()
    code, _, _ = cache.bc_poll_error()
    assert code == 0
