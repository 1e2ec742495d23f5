"""Randomised parity runs of the CUDA path against the oracle.

The kernel cuts the tile stream into rate-proportional shares, reorders each share, and merges split
sequences by tickets; the cut points move from call to call as the per-CTA rate table adapts.  These
tests throw many small random shapes with awkward lengths at it, call each several times on one
workspace, and also cover batches larger than the kernel's in-shared-memory user cache.
"""
import numpy as np
import pytest
import torch

from oracle import spd_oracle as orc
from paper_2409_19134_b200 import binding as spd
from paper_2409_19134_b200 import workloads as wl
from tests.test_gpu_parity import assert_close, oracle_inputs

pytestmark = pytest.mark.gpu

EDGE = [0, 1, 15, 16, 17, 31, 32, 33, 47, 48, 49]
HEADS = [(1, 1), (2, 1), (4, 4), (4, 1), (8, 2), (8, 1), (16, 2), (16, 1), (32, 8), (12, 6)]


def _lengths(rng, B, hi):
    out = np.empty(B, dtype=np.int64)
    for u in range(B):
        r = rng.random()
        out[u] = rng.choice(EDGE) if r < 0.4 else (rng.integers(0, hi + 1) if r < 0.9 else rng.integers(hi, 8 * hi + 1))
    return out


def _run(w, calls=3, fused_modes=(True, False)):
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    wg = w.to("cuda")
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device="cuda")
    for fused in fused_modes:
        for k in range(calls):
            out.fill_(float("nan"))
            spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=fused)
            assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
            assert_close(out.cpu().numpy(), ref, w.dtype, f"{w.name} fused={fused} call {k}")


@pytest.mark.parametrize("seed", range(24))
def test_random_small_shapes(seed):
    rng = np.random.default_rng(1000 + seed)
    hq, hkv = HEADS[rng.integers(0, len(HEADS))]
    d = int(rng.choice([64, 128]))
    dtype = "bf16" if rng.random() < 0.6 else "f32"
    B = int(rng.integers(1, 13))
    hi = int(rng.choice([40, 300, 2500]))
    lin, lout = _lengths(rng, B, hi), _lengths(rng, B, max(8, hi // 8))
    cfg = dict(name=f"rand{seed}", batch=B, hq=hq, hkv=hkv, d=d, dtype=dtype, lin=("const", 0), lout=("const", 0), seed=seed)
    w = wl.make_workload(cfg, lengths=(lin, lout), slack=bool(rng.integers(0, 2)))
    _run(w)


@pytest.mark.parametrize("dtype,B", [("bf16", 1500), ("f32", 1100)])
def test_batches_beyond_the_user_cache(dtype, B):
    """More users than the kernel caches in shared memory (and than a CTA has threads)."""
    rng = np.random.default_rng(77)
    lin, lout = _lengths(rng, B, 60), _lengths(rng, B, 20)
    lin[-1], lout[-1] = 700, 33          # the last user is the longest: its pieces sit beyond the cache
    cfg = dict(name=f"wide_{dtype}", batch=B, hq=2, hkv=1, d=64, dtype=dtype, lin=("const", 0), lout=("const", 0), seed=5)
    w = wl.make_workload(cfg, lengths=(lin, lout))
    _run(w, calls=2, fused_modes=(True,))


def test_one_user_one_head_long():
    """A single sequence cut across the whole grid: every warp delivers a piece of the same sequence."""
    cfg = dict(name="solo", batch=1, hq=1, hkv=1, d=128, dtype="bf16", lin=("const", 60000), lout=("const", 17), seed=9)
    _run(wl.make_workload(cfg), calls=3)


MID = [("bf16", 64, 16, 4), ("bf16", 64, 8, 8), ("bf16", 128, 32, 2), ("bf16", 128, 64, 2), ("f32", 64, 16, 2), ("f32", 128, 8, 8),
       ("f32", 128, 32, 4), ("bf16", 128, 6, 6)]


@pytest.mark.parametrize("dtype,d,hq,hkv", MID)
def test_mid_size_batches_every_head_grouping(dtype, d, hq, hkv):
    """Forty users with prompts up to 6000 tokens (hundreds of tiles per sequence, so shares cut sequences and pieces
    are merged), for head_dim 64 and 128, both dtypes, groups of 1, 4, 8, 16 and 32 query heads per KV head: every row
    of the fused step, the chained step, and the step with the append inside, against the oracle."""
    rng = np.random.default_rng(hq * 131 + hkv * 7 + d)
    B = 40
    lin = rng.integers(1, 6001, size=B)
    lout = rng.integers(0, 300, size=B)
    lout[lout % 16 == 0] += 1                      # room for one more token in every user's last public page
    cfg = dict(name=f"mid_{dtype}_{d}_{hq}_{hkv}", batch=B, hq=hq, hkv=hkv, d=d, dtype=dtype, lin=("const", 0), lout=("const", 0), seed=hq + hkv)
    w = wl.make_workload(cfg, lengths=(lin, lout))
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    wg = w.to("cuda")
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device="cuda")
    for fused in (True, False):
        for k in range(2):
            out.fill_(float("nan"))
            spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=fused)
            assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
            assert_close(out.cpu().numpy(), ref, w.dtype, f"{w.name} fused={fused} call {k}")
    gen = torch.Generator().manual_seed(hq)
    k_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
    v_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
    assert orc.append(kout, orc.q_from_torch(k_new), orc.q_from_torch(v_new)).all()
    out.fill_(float("nan"))
    spd.spd_decode_step_append(shape, wg.q, k_new.cuda(), v_new.cuda(), wg.priv, wg.pub, out, ws)
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    assert np.array_equal(wg.pub.seq_lens.cpu().numpy(), kout.seq_lens)
    assert_close(out.cpu().numpy(), orc.full(q, kin, kout, w.sm_scale), w.dtype, f"{w.name} append inside the launch")
