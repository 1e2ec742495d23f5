"""The plan of the attention kernel, made observable and controllable.

Split-K is not in the paper: any way of cutting a partition into pieces must give the same attention (Theorem 1
applied n-ways).  These tests force the cut granularity (every page a piece of its own, one share and no merge at
all, and values in between), compare the share boundaries that the device derived with a re-derivation in NumPy,
integer for integer, check that with the measured rates ignored a repeated call is bit-identical, and cover the
plan's reuse by later calls over the same lengths (the *_planned entry points and the token step).
"""
import numpy as np
import pytest
import torch

from oracle import spd_oracle as orc
from paper_2409_19134_b200 import binding as spd
from paper_2409_19134_b200 import workloads as wl
from tests.test_gpu_parity import SMALL, assert_close, oracle_inputs

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True)
def default_split():
    yield
    spd.spd_set_split(0, False)


def _setup(cfg, **kw):
    w = wl.make_workload(cfg, slack=True, **kw)
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    return w, ref, shape


def _tiles(w):
    """Page tiles in the stream of a fused call: per user (private + public pages in use) x sequences per user."""
    g = w.num_q_heads // w.num_kv_heads
    S = w.num_kv_heads * max(1, g // 8)
    per_user = (w.priv.seq_lens.numpy().astype(np.int64) + 15) // 16 + (w.pub.seq_lens.numpy().astype(np.int64) + 15) // 16
    return int(per_user.sum()) * S


@pytest.mark.parametrize("name", ["bf16_gqa4_d128", "bf16_mha_d128", "f32_gqa4_d128", "f32_long_split"])
@pytest.mark.parametrize("min_tiles", [1, 2, 7, 64, 1 << 30])
def test_forced_cut_granularities_match_the_oracle(name, min_tiles):
    """min_tiles = 1: as many shares as there are tiles (or warps); 2^30: a single share, so nothing is merged."""
    w, ref, shape = _setup(dict(SMALL[name], name=name))
    wg = w.to("cuda")
    ws = spd.alloc_workspace(shape)
    spd.spd_set_split(min_tiles, True)
    for fused in (True, False):
        out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
        spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=fused)
        assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
        assert_close(out.cpu().numpy(), ref, w.dtype, f"{name} min_tiles={min_tiles} fused={fused}")
    T, A, bnd = spd.spd_debug_read_plan(ws, which=2)
    assert T == _tiles(w)
    warps = torch.cuda.get_device_properties(0).multi_processor_count * (8 if w.dtype == torch.bfloat16 else 4)
    assert A == min(warps, -(-T // min_tiles))
    if min_tiles == 1 << 30:
        assert A == 1 and bnd == [0, T]
    if min_tiles == 1 and T <= warps:
        assert bnd == list(range(T + 1))         # every page tile a share, hence a piece, of its own


@pytest.mark.parametrize("name,min_tiles", [("bf16_gqa8_d128", 4), ("bf16_long_split", 4), ("bf16_long_split", 3), ("f32_mha_d64", 1)])
def test_share_boundaries_equal_a_numpy_rederivation(name, min_tiles):
    """With equal weights, share w of A starts at tile floor(T * w / A), evaluated as the kernel does: the exact
    integer product in double, one correctly rounded division, truncation."""
    w, ref, shape = _setup(dict(SMALL[name], name=name))
    wg = w.to("cuda")
    ws = spd.alloc_workspace(shape)
    spd.spd_set_split(min_tiles, True)
    out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device="cuda")
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True)
    T, A, bnd = spd.spd_debug_read_plan(ws, which=2)
    warps = torch.cuda.get_device_properties(0).multi_processor_count * (8 if w.dtype == torch.bfloat16 else 4)
    assert T == _tiles(w) and A == min(warps, -(-T // min_tiles))
    ws_ = np.arange(A + 1, dtype=np.int64) * 1024                     # every CTA weighs 1024, every warp its CTA's weight
    want = (np.float64(T) * ws_.astype(np.float64) / np.float64(A * 1024)).astype(np.int64)
    assert bnd == want.tolist()
    assert np.array_equal(want, np.arange(A + 1, dtype=np.int64) * T // A)   # and that is the exact floor here
    # the two halves of a chained step keep plans of their own
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=False)
    g = w.num_q_heads // w.num_kv_heads
    S = w.num_kv_heads * max(1, g // 8)
    T0, _, b0 = spd.spd_debug_read_plan(ws, which=0)
    T1, _, b1 = spd.spd_debug_read_plan(ws, which=1)
    assert T0 == int(((w.priv.seq_lens.numpy().astype(np.int64) + 15) // 16).sum()) * S and b0[-1] == T0
    assert T1 == int(((w.pub.seq_lens.numpy().astype(np.int64) + 15) // 16).sum()) * S and b1[-1] == T1


@pytest.mark.parametrize("name", ["bf16_long_split", "bf16_gqa8_d128", "f32_long_split"])
def test_rates_ignored_means_bit_identical_calls(name):
    w, ref, shape = _setup(dict(SMALL[name], name=name))
    wg = w.to("cuda")
    ws = spd.alloc_workspace(shape)
    spd.spd_set_split(0, True)
    outs = []
    for _ in range(4):
        out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
        spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True)
        outs.append(out)
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    for o in outs[1:]:
        assert torch.equal(o, outs[0])
    assert_close(outs[0].cpu().numpy(), ref, w.dtype, name)


@pytest.mark.parametrize("name", ["bf16_gqa4_d128", "bf16_long_split", "f32_gqa8_d64", "bf16_gqa16_d128"])
@pytest.mark.parametrize("fused", [True, False])
def test_stored_plan_is_reused_by_later_calls(name, fused):
    """SPD_PLAN_STORE then SPD_PLAN_REUSE: same cut, hence the same bits; new q values and reshuffled pages (same
    lengths) are followed, since the plan depends on the lengths only."""
    w, ref, shape = _setup(dict(SMALL[name], name=name))
    wg = w.to("cuda")
    ws = spd.alloc_workspace(shape)

    def run(plan, wl_gpu):
        out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
        spd.spd_decode_step(shape, wl_gpu.q, wl_gpu.priv, wl_gpu.pub, out, ws, fused=fused, plan=plan)
        assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
        return out
    first = run(spd.SPD_PLAN_STORE, wg)
    assert_close(first.cpu().numpy(), ref, w.dtype, f"{name} store")
    for k in range(3):
        again = run(spd.SPD_PLAN_REUSE, wg)
        assert torch.equal(again, first), f"reuse {k} differs from the storing call"
    # a plain call in between derives its own plan and invalidates nothing that the next STORE does not redo
    run(None, wg)
    # same lengths, other values: a fresh workload with the same length arrays, another seed for values and pages
    w2 = wl.make_workload(dict(SMALL[name], name=name), seed=SMALL[name]["seed"] + 100, slack=False,
                          lengths=(w.priv.seq_lens.numpy().astype(np.int64), w.pub.seq_lens.numpy().astype(np.int64)))
    q2, kin2, kout2 = oracle_inputs(w2)
    ref2 = orc.full(q2, kin2, kout2, w2.sm_scale)
    run(spd.SPD_PLAN_STORE, wg)
    got2 = run(spd.SPD_PLAN_REUSE, w2.to("cuda"))
    assert_close(got2.cpu().numpy(), ref2, w2.dtype, f"{name} reuse on other values and page tables")


def test_reuse_without_a_stored_plan_is_reported():
    name = "bf16_gqa4_d128"
    w, ref, shape = _setup(dict(SMALL[name], name=name))
    wg = w.to("cuda")
    ws = spd.alloc_workspace(shape)
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True, plan=spd.SPD_PLAN_REUSE)
    assert spd.spd_query_device_status(ws) == (7, -1)              # SPD_ERR_PLAN; nothing was streamed
    # a plan stored for another shape does not fit either
    other = dict(SMALL["bf16_mha_d128"], name="other")
    w2, ref2, shape2 = _setup(other)
    ws2 = spd.alloc_workspace(shape2)
    big = ws if ws.numel() >= ws2.numel() else ws2
    out2 = torch.empty((w2.batch, w2.num_q_heads, w2.head_dim), dtype=torch.float32, device="cuda")
    w2g = w2.to("cuda")
    spd.spd_decode_step(shape2, w2g.q, w2g.priv, w2g.pub, out2, big, fused=True, plan=spd.SPD_PLAN_STORE)
    assert spd.spd_query_device_status(big) == (spd.SPD_OK, -1)
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, big, fused=True, plan=spd.SPD_PLAN_REUSE)
    assert spd.spd_query_device_status(big) == (7, -1)
    # and the workspace is usable right away
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, big, fused=True)
    assert spd.spd_query_device_status(big) == (spd.SPD_OK, -1)
    assert_close(out.cpu().numpy(), ref, w.dtype, "after a refused reuse")


def test_reuse_over_changed_lengths_never_faults():
    """The caller's promise broken on purpose, on the host: lengths shrink (and one grows) after the plan was stored.
    Results of the users concerned are then undefined, but every index is still checked: the call ends, bystanders
    whose tiles did not move may be anything too, and the next planning call is right again."""
    name = "bf16_gqa4_d128"
    w, ref, shape = _setup(dict(SMALL[name], name=name))
    wg = w.to("cuda")
    ws = spd.alloc_workspace(shape)
    out = torch.empty((w.batch, w.num_q_heads, w.head_dim), dtype=torch.float32, device="cuda")
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True, plan=spd.SPD_PLAN_STORE)
    keep = wg.priv.seq_lens.clone()
    wg.priv.seq_lens.copy_(torch.clamp(keep // 3, min=0))
    wg.priv.seq_lens[-1] = 0
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True, plan=spd.SPD_PLAN_REUSE)
    code, _ = spd.spd_query_device_status(ws)          # waits: the kernel has ended
    assert code in (spd.SPD_OK, 4, 7)                  # a stale cursor may also meet a page slot that is no longer listed
    wg.priv.seq_lens.copy_(keep)
    out.fill_(float("nan"))
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True)
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    assert_close(out.cpu().numpy(), ref, w.dtype, "planning call after a stale reuse")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_token_step_with_one_plan_for_all_layers(dtype):
    """Every layer caches the same tokens, so all layers have the same lengths: layer 0 derives the plan, the others
    load it.  Values, page tables and the new rows differ per layer; outputs, caches and lengths must be what the
    oracle gets, eagerly and from a replayed graph."""
    n_layers, B, hq, hkv, d = 4, 6, 16, 4, 128
    rng = np.random.default_rng(91)
    lin, lout = rng.integers(1, 900, size=B), rng.integers(0, 120, size=B)
    layers_gpu, checks = [], []
    shape = None
    for i in range(n_layers):
        cfg = dict(name=f"layer{i}", batch=B, hq=hq, hkv=hkv, d=d, dtype=dtype, lin=("const", 0), lout=("const", 0), seed=92 + i)
        w = wl.make_workload(cfg, lengths=(lin, lout + 3))
        w.pub.seq_lens = torch.clamp(w.pub.seq_lens - 3, min=0)        # room for three more tokens in the listed pages
        gen = torch.Generator().manual_seed(100 + i)
        k_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
        v_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
        wg = w.to("cuda")
        out = torch.full((B, hq, d), float("nan"), dtype=torch.float32, device="cuda")
        layers_gpu.append((wg.q, k_new.cuda(), v_new.cuda(), wg.priv, wg.pub, out))
        checks.append((w, k_new, v_new, oracle_inputs(w)))
        shape = spd.make_shape(B, hq, hkv, d, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)

    def check(what):
        torch.cuda.synchronize()
        assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
        for i, ((w, k_new, v_new, (q, kin, kout)), lg) in enumerate(zip(checks, layers_gpu)):
            assert orc.append(kout, orc.q_from_torch(k_new), orc.q_from_torch(v_new)).all()
            assert np.array_equal(lg[4].seq_lens.cpu().numpy(), kout.seq_lens), f"{what}: lengths of layer {i}"
            assert_close(lg[5].cpu().numpy(), orc.full(q, kin, kout, w.sm_scale), w.dtype, f"{what}: layer {i}")
            lg[5].fill_(float("nan"))

    spd.spd_token_step(shape, layers_gpu, ws, same_lengths=True)
    check("eager")
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        spd.spd_token_step(shape, layers_gpu, ws, same_lengths=True)
    for r in range(2):
        graph.replay()
        check(f"graph replay {r}")
