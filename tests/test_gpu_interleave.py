"""Two batches served side by side: calls on two streams with two workspaces, issued alternately from one host
thread, with other kernels of the library in between.

Every workspace carries a small table of streaming rates that the next call on it reads while the previous one
may still be running (programmatic launch), rotated by the number of attention launches on THAT workspace.  All
CTAs of a launch must read the same table, or they cut the tile stream differently and tiles are dropped or
doubled.  These runs interleave everything that could disturb the rotation and compare every output of every
round with the oracle; the workloads are large enough (a few hundred MB of KV) that launches queue up and the
preamble of one call really overlaps the tail of the one before.
"""
import numpy as np
import pytest
import torch

from oracle import spd_oracle as orc
from paper_2409_19134_b200 import binding as spd
from paper_2409_19134_b200 import workloads as wl
from tests.test_gpu_parity import assert_close, oracle_inputs

pytestmark = pytest.mark.gpu

ROUNDS = 60
A_CFG = dict(name="batch_a", batch=4, hq=32, hkv=8, d=128, dtype="bf16", lin=("uniform", 12000, 20000), lout=("uniform", 1, 300), seed=201)
B_CFG = dict(name="batch_b", batch=24, hq=16, hkv=16, d=128, dtype="bf16", lin=("uniform", 100, 3000), lout=("uniform", 0, 200), seed=202)


def _batch(cfg):
    w = wl.make_workload(cfg)
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    wg = w.to("cuda")
    outs = [torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda") for _ in range(ROUNDS)]
    return w, wg, ref, shape, spd.alloc_workspace(shape), outs


def _check(w, ref, outs, ws, stream, what):
    assert spd.spd_query_device_status(ws, stream=stream) == (spd.SPD_OK, -1)
    for r, o in enumerate(outs):
        assert_close(o.cpu().numpy(), ref, w.dtype, f"{what}, round {r}")


def test_two_batches_on_two_streams_alternating():
    wa, ga, ref_a, shape_a, ws_a, outs_a = _batch(A_CFG)
    wb, gb, ref_b, shape_b, ws_b, outs_b = _batch(B_CFG)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for r in range(ROUNDS):                                     # host order A1 B1 A2 B2 ...
        spd.spd_decode_step(shape_a, ga.q, ga.priv, ga.pub, outs_a[r], ws_a, fused=True, stream=sa)
        spd.spd_decode_step(shape_b, gb.q, gb.priv, gb.pub, outs_b[r], ws_b, fused=(r % 3 != 0), stream=sb)
    torch.cuda.synchronize()
    _check(wa, ref_a, outs_a, ws_a, sa, "batch A beside batch B")
    _check(wb, ref_b, outs_b, ws_b, sb, "batch B beside batch A")
    # both workspaces kept adapting: each has seen its own launches, one after the other
    la, _ = spd.spd_debug_sm_moves(ws_a, stream=sa)
    lb, _ = spd.spd_debug_sm_moves(ws_b, stream=sb)
    assert la >= ROUNDS - 2 and lb >= ROUNDS - 2


def test_attention_on_one_stream_small_kernels_on_the_other():
    """Between two back-to-back steps on stream A the host enqueues an append and a stand-alone merge on stream B:
    other kernels of the library, which must not move workspace A's rotation."""
    wa, ga, ref_a, shape_a, ws_a, outs_a = _batch(A_CFG)
    wb, gb, ref_b, shape_b, ws_b, _ = _batch(B_CFG)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    pa, pb = spd.alloc_partial(shape_b), spd.alloc_partial(shape_b)
    merged = torch.full((wb.batch, wb.num_q_heads, wb.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    gen = torch.Generator(device="cuda").manual_seed(5)
    k_new = torch.randn((wb.batch, wb.num_kv_heads, wb.head_dim), generator=gen, device="cuda").to(torch.bfloat16)
    # a scratch copy of B's public cache takes the appends (one spare page per user, lengths moved back)
    scratch = wl.make_workload(dict(B_CFG, lout=("const", 16 * 8)), device="cuda").pub
    scratch.seq_lens.fill_(0)
    spd.spd_partial_attn(shape_b, gb.q, gb.priv, pa, ws_b, stream=sb)
    spd.spd_partial_attn(shape_b, gb.q, gb.pub, pb, ws_b, stream=sb)
    torch.cuda.synchronize()
    for r in range(ROUNDS):
        spd.spd_decode_step(shape_a, ga.q, ga.priv, ga.pub, outs_a[r], ws_a, fused=True, stream=sa)
        spd.spd_append_kv(shape_b, k_new, k_new, scratch, ws_b, stream=sb)
        spd.spd_merge_partials(shape_b, [pa, pb], merged, stream=sb)
    torch.cuda.synchronize()
    _check(wa, ref_a, outs_a, ws_a, sa, "batch A beside appends and merges")
    assert spd.spd_query_device_status(ws_b, stream=sb) == (spd.SPD_OK, -1)
    assert int(scratch.seq_lens.min()) == ROUNDS and int(scratch.seq_lens.max()) == ROUNDS
    assert_close(merged.cpu().numpy(), ref_b, wb.dtype, "stand-alone merge beside batch A")


def test_per_layer_calls_without_a_kernel_in_between():
    """The per-user / service split issued layer by layer on one stream and one workspace: private partial, then
    public partial + merge, again and again, nothing else in between (so each launch's preamble overlaps the
    launch before it), plus the same on a second stream for another batch."""
    wa, ga, ref_a, shape_a, ws_a, outs_a = _batch(A_CFG)
    wb, gb, ref_b, shape_b, ws_b, outs_b = _batch(B_CFG)
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    part_a, part_b = spd.alloc_partial(shape_a), spd.alloc_partial(shape_b)
    torch.cuda.synchronize()
    for r in range(ROUNDS):
        spd.spd_partial_attn(shape_a, ga.q, ga.priv, part_a, ws_a, stream=sa)
        spd.spd_partial_attn(shape_b, gb.q, gb.priv, part_b, ws_b, stream=sb)
        spd.spd_service_attn_merge(shape_a, ga.q, ga.pub, part_a, outs_a[r], ws_a, stream=sa)
        spd.spd_service_attn_merge(shape_b, gb.q, gb.pub, part_b, outs_b[r], ws_b, stream=sb)
    torch.cuda.synchronize()
    _check(wa, ref_a, outs_a, ws_a, sa, "layer-by-layer calls, batch A")
    _check(wb, ref_b, outs_b, ws_b, sb, "layer-by-layer calls, batch B")


def test_two_host_threads_two_workspaces():
    """Calls may come from several host threads as long as each workspace is driven by one of them: two threads, each
    with its own batch, workspace and stream, issue their steps at the same time (ctypes releases the interpreter
    lock during a call, so the launches really interleave in the library)."""
    import threading
    batches = [_batch(A_CFG), _batch(B_CFG)]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    errors = []

    def serve(k):
        try:
            w, g, ref, shape, ws, outs = batches[k]
            for r in range(ROUNDS):
                spd.spd_decode_step(shape, g.q, g.priv, g.pub, outs[r], ws, fused=(k == 0 or r % 2 == 0), stream=streams[k])
        except Exception as e:          # noqa: BLE001  (reported by the main thread)
            errors.append(e)
    threads = [threading.Thread(target=serve, args=(k,)) for k in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for k, what in enumerate(("thread 0, batch A", "thread 1, batch B")):
        w, g, ref, shape, ws, outs = batches[k]
        _check(w, ref, outs, ws, streams[k], what)
