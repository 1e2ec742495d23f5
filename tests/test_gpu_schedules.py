"""Other ways to schedule the same decode step: a stand-alone merge of partials, the private and public
halves on two streams, and a captured CUDA graph.  Each must give what the oracle gives."""
import numpy as np
import pytest
import torch

from oracle import spd_oracle as orc
from paper_2409_19134_b200 import binding as spd
from paper_2409_19134_b200 import workloads as wl
from tests.test_gpu_parity import SMALL, assert_close, oracle_inputs

pytestmark = pytest.mark.gpu


def _setup(name):
    w = wl.make_workload(dict(SMALL[name], name=name), slack=True)
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    return w, (q, kin, kout), ref, shape


@pytest.mark.parametrize("name", ["bf16_gqa4_d128", "f32_mha_d64"])
def test_merge_partials_of_oracle_pieces(name):
    """Partials computed elsewhere (here by the oracle over three token ranges plus the public partition,
    rounded to fp32) merge into the full attention."""
    w, (q, kin, kout), ref, shape = _setup(name)
    cuts = [(0, 37), (37, 400), (400, 1 << 40)]
    pieces = [orc.partial(q, kin, w.sm_scale, a, b) for a, b in cuts] + [orc.partial(q, kout, w.sm_scale)]
    parts = [tuple(torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda() for x in p) for p in pieces]
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    spd.spd_merge_partials(shape, parts, out)
    torch.cuda.synchronize()
    got = out.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got)) and np.max(np.abs(got - ref)) <= 1e-5   # fp32 inputs, fp32 merge
    outb = torch.empty_like(out, dtype=torch.bfloat16)
    spd.spd_merge_partials(shape, parts, outb)
    assert np.max(np.abs(outb.float().cpu().numpy() - ref)) <= 2.0 ** -8 * np.max(np.abs(ref)) + 1e-5
    with pytest.raises(spd.SpdError):
        spd.spd_merge_partials(shape, parts * 3, out)       # more than eight partials


@pytest.mark.parametrize("name", ["bf16_gqa8_d128", "bf16_long_split", "f32_gqa4_d128"])
def test_two_stream_schedule(name):
    """Private half on one stream, public half on another (each with its own workspace), then the merge."""
    w, _, ref, shape = _setup(name)
    wg = w.to("cuda")
    ws_a, ws_b = spd.alloc_workspace(shape), spd.alloc_workspace(shape)
    pa, pb = spd.alloc_partial(shape), spd.alloc_partial(shape)
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(3):
        done_b = torch.cuda.Event()
        spd.spd_partial_attn(shape, wg.q, wg.priv, pa, ws_a, stream=sa)
        spd.spd_partial_attn(shape, wg.q, wg.pub, pb, ws_b, stream=sb)     # the public partition, same kernel
        done_b.record(sb)
        sa.wait_event(done_b)
        spd.spd_merge_partials(shape, [pa, pb], out, stream=sa)
        sa.synchronize()
        assert spd.spd_query_device_status(ws_a, stream=sa) == (spd.SPD_OK, -1)
        assert spd.spd_query_device_status(ws_b, stream=sb) == (spd.SPD_OK, -1)
        assert_close(out.cpu().numpy(), ref, w.dtype, f"{name} two streams")


@pytest.mark.parametrize("name", ["bf16_gqa4_d128", "bf16_long_split"])
def test_cuda_graph_replay(name):
    """The fused step captured once and replayed: same result every time, and it follows new q values."""
    w, (q, kin, kout), ref, shape = _setup(name)
    wg = w.to("cuda")
    ws = spd.alloc_workspace(shape)
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    for _ in range(4):                                                        # warm up outside the capture
        spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True)
        spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True)  # two in a row: the second overlaps the first's tail
    for _ in range(3):
        out.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert_close(out.cpu().numpy(), ref, w.dtype, f"{name} graph replay")
    wg.q.copy_((wg.q.float() * 0.5).to(wg.q.dtype))                          # new query values, same buffers
    w.q = wg.q.cpu()
    ref2 = orc.full(orc.q_from_torch(w.q), kin, kout, w.sm_scale)
    graph.replay()
    torch.cuda.synchronize()
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    assert_close(out.cpu().numpy(), ref2, w.dtype, f"{name} graph replay with new q")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_token_step_over_layers_eager_and_as_one_graph(dtype):
    """Step 3 for every layer of a model in one call: per layer the append and the fused decode step.  Run once
    eagerly, then captured in a CUDA graph and replayed twice; after every run each layer's output, cache and
    lengths must be what the oracle gets from the same number of appends."""
    n_layers, B, hq, hkv, d = 3, 5, 8, 2, 128
    rng = np.random.default_rng(61)
    layers_cpu, layers_gpu, oracles = [], [], []
    shape = None
    for i in range(n_layers):
        lin, lout = rng.integers(1, 400, size=B), rng.integers(1, 90, size=B)
        cfg = dict(name=f"layer{i}", batch=B, hq=hq, hkv=hkv, d=d, dtype=dtype, lin=("const", 0), lout=("const", 0), seed=62 + i)
        w = wl.make_workload(cfg, lengths=(lin, lout))
        w.pub.seq_lens = torch.clamp(w.pub.seq_lens - 3, min=0)          # room for three more tokens in the listed pages
        gen = torch.Generator().manual_seed(70 + i)
        k_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
        v_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
        wg = w.to("cuda")
        out = torch.full((B, hq, d), float("nan"), dtype=torch.float32, device="cuda")
        layers_cpu.append((w, k_new, v_new))
        layers_gpu.append((wg.q, k_new.cuda(), v_new.cuda(), wg.priv, wg.pub, out))
        oracles.append(oracle_inputs(w))
        shape = spd.make_shape(B, hq, hkv, d, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)

    def bits(t):
        return t.cpu().view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32).numpy()

    def check(what):
        torch.cuda.synchronize()
        assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
        for i, ((w, k_new, v_new), (q, kin, kout), lg) in enumerate(zip(layers_cpu, oracles, layers_gpu)):
            assert orc.append(kout, orc.q_from_torch(k_new), orc.q_from_torch(v_new)).all()
            pub, out = lg[4], lg[5]
            assert np.array_equal(pub.seq_lens.cpu().numpy(), kout.seq_lens), f"{what}: lengths of layer {i}"
            assert np.array_equal(bits(pub.k_pool), kout.k_pool.view(bits(pub.k_pool).dtype)), f"{what}: K cache of layer {i}"
            assert np.array_equal(bits(pub.v_pool), kout.v_pool.view(bits(pub.v_pool).dtype)), f"{what}: V cache of layer {i}"
            assert_close(out.cpu().numpy(), orc.full(q, kin, kout, w.sm_scale), w.dtype, f"{what}: layer {i}")
            out.fill_(float("nan"))

    launches = spd.spd_kernel_launch_count()
    spd.spd_token_step(shape, layers_gpu, ws)
    assert spd.spd_kernel_launch_count() - launches == n_layers      # append and attention share a launch
    check("eager")
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        spd.spd_token_step(shape, layers_gpu, ws)
    for r in range(2):
        graph.replay()
        check(f"graph replay {r}")
