"""The allocation-free entry point, spd_decode_step_static.

Some callers cannot allocate device memory (code running under stream capture, plug-ins of an engine
that owns the whole pool, sandboxed per-user workers with a fixed footprint), so this entry point keeps
its workspace in an array inside the library.  It must give what spd_decode_step gives with a
caller-provided workspace -- also on a second call, when the shared array still holds the first call's
plan, scratch and flags -- and must refuse shapes that need more than the array holds.

This file is collected last on purpose: a run that stops at the first failure has then already run
every other test.  It does not depend on them.
"""
import numpy as np
import pytest
import torch

from paper_2409_19134_b200 import binding as spd
from paper_2409_19134_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_MAX_ABS, TOL_REL_L2 = 2e-3, 1e-3   # the bf16 tolerances of the parity tests


def _regular(w):
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws, fused=True)
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    return shape, out


def _close(a, b):
    a, b = a.double().cpu().numpy(), b.double().cpu().numpy()
    assert np.all(np.isfinite(a))
    assert np.max(np.abs(a - b)) <= TOL_MAX_ABS
    assert np.linalg.norm(a - b) / np.linalg.norm(b) <= TOL_REL_L2


def test_static_workspace_matches_regular_entry_point_twice_in_a_row():
    cfgs = [dict(batch=9, hq=32, hkv=8, d=128, dtype="bf16", lin=("uniform", 1, 2500), lout=("uniform", 0, 300), seed=31),
            # second call: fewer users and long prompts, cut into many pieces that leave their floats in the scratch
            dict(batch=4, hq=32, hkv=8, d=128, dtype="bf16", lin=("uniform", 20000, 30000), lout=("uniform", 1, 60), seed=32)]
    for cfg in cfgs:
        w = wl.make_workload(cfg, device="cuda", slack=True)
        shape, ref = _regular(w)
        assert spd.spd_workspace_size(shape) <= spd.STATIC_WS_BYTES
        out = torch.full_like(ref, float("nan"))
        torch.cuda.synchronize()
        before = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        code, bad = spd.spd_decode_step_static(shape, w.q, w.priv, w.pub, out)
        assert (code, bad) == (spd.SPD_OK, -1)
        assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == before
        _close(out, ref)


def test_static_workspace_survives_a_change_of_shape_between_calls():
    """The array is laid out per call.  When the batch grows, the new call's merge tickets lie where the previous
    call kept scratch floats; when the dtype or the number of KV heads changes, pitch and offsets move.  Whatever
    the previous call left there, every row of the output must be written and right."""
    seq = [dict(batch=4, hq=32, hkv=8, d=128, dtype="bf16", lin=("uniform", 20000, 30000), lout=("uniform", 1, 60), seed=34),
           dict(batch=128, hq=32, hkv=8, d=128, dtype="bf16", lin=("uniform", 600, 5000), lout=("uniform", 0, 100), seed=35),   # batch grows
           dict(batch=3, hq=8, hkv=2, d=128, dtype="f32", lin=("uniform", 9000, 12000), lout=("uniform", 1, 50), seed=36),      # fp32: 4 warps per CTA
           dict(batch=70, hq=32, hkv=32, d=128, dtype="bf16", lin=("uniform", 900, 4000), lout=("uniform", 1, 100), seed=37),   # bf16 again, four times the KV heads
           dict(batch=9, hq=16, hkv=1, d=64, dtype="bf16", lin=("uniform", 3000, 9000), lout=("uniform", 0, 40), seed=38)]      # one KV head, groups of 8, head_dim 64
    for k, cfg in enumerate(seq):
        w = wl.make_workload(cfg, device="cuda")
        shape, ref = _regular(w)
        assert spd.spd_workspace_size(shape) <= spd.STATIC_WS_BYTES
        for wait in (False, True):
            out = torch.full_like(ref, float("nan"))
            code, bad = spd.spd_decode_step_static(shape, w.q, w.priv, w.pub, out, wait_and_check=wait)
            torch.cuda.synchronize()
            assert (code, bad) == (spd.SPD_OK, -1), f"call {k}"
            assert bool(torch.isfinite(out).all()), f"call {k}: rows left unwritten"
            if w.dtype == torch.float32:
                assert float((out - ref).abs().max()) <= 1e-5
            else:
                _close(out, ref)


def test_static_workspace_clears_stale_flags_and_rejects_big_shapes():
    cfg = dict(batch=5, hq=8, hkv=2, d=128, dtype="bf16", lin=("uniform", 1, 400), lout=("uniform", 1, 50), seed=33)
    w = wl.make_workload(cfg, device="cuda")
    shape, ref = _regular(w)
    out = torch.full_like(ref, float("nan"))
    # a call with a page index outside the pool raises the sticky flag inside the shared array ...
    good = w.priv.page_indices.clone()
    w.priv.page_indices[int(w.priv.page_indptr[2])] = w.priv.num_pages + 7
    code, bad = spd.spd_decode_step_static(shape, w.q, w.priv, w.pub, out)
    assert (code, bad) == (4, 2) and bool((out[2] == 0).all())
    _close(out[[0, 1, 3, 4]], ref[[0, 1, 3, 4]])
    # ... and the next call, without waiting this time, starts clean
    w.priv.page_indices.copy_(good)
    out.fill_(float("nan"))
    assert spd.spd_decode_step_static(shape, w.q, w.priv, w.pub, out, wait_and_check=False) == (spd.SPD_OK, -1)
    torch.cuda.synchronize()
    _close(out, ref)
    # beyond the built-in array: refused on the host, nothing launched
    big = spd.make_shape(512, 64, 8, 128, torch.bfloat16, 0.1)
    assert spd.spd_workspace_size(big) > spd.STATIC_WS_BYTES
    n0 = spd.spd_kernel_launch_count()
    with pytest.raises(spd.SpdError) as e:
        spd.spd_decode_step_static(big, w.q, w.priv, w.pub, out)
    assert e.value.code == 3 and spd.spd_kernel_launch_count() == n0
