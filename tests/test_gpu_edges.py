"""Edge cases of the CUDA path through the C ABI.

  - bit-exact page-table / length handling (indexing probe with integer-coded values)
  - empty partitions, users with nothing cached, slack pages, NaN-poisoned unused slots
  - device-detected mistakes (page index outside the pool, length beyond the pages listed): no
    fault, zeros for that user, sticky status, everyone else untouched
"""
import numpy as np
import pytest
import torch

from oracle import spd_oracle as orc
from paper_2409_19134_b200 import binding as spd
from paper_2409_19134_b200 import workloads as wl
from tests.test_gpu_parity import SMALL, TOL, assert_close, oracle_inputs, run_decode

pytestmark = pytest.mark.gpu


def _decode(w, fused=True):
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws, fused=fused)
    status = spd.spd_query_device_status(ws)
    return out, status, (shape, ws)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("fused", [True, False])
def test_indexing_probe_is_bit_exact(dtype, fused):
    """V rows carry (user, kv head, token // 64, token % 64, ...) as small integers; each query head
    puts an overwhelming score on one token, so the output must be that token's V exactly."""
    cfg = dict(batch=6, hq=8, hkv=4, d=64, dtype=dtype, lin=("uniform", 1, 900), lout=("uniform", 0, 200), seed=41)
    w = wl.make_workload(cfg, slack=True)
    rng = np.random.default_rng(42)
    g, D, P = 2, 64, 16
    expect = np.zeros((w.batch, w.num_q_heads, D), np.float64)
    w.q.zero_()
    for part in (w.priv, w.pub):
        valid = ~torch.isnan(part.k_pool.float())
        part.k_pool[valid] = 0      # scores come only from the planted components
    for u in range(w.batch):
        lin, lout = int(w.priv.seq_lens[u]), int(w.pub.seq_lens[u])
        for part, n, tag in ((w.priv, lin, 1), (w.pub, lout, 2)):
            lo = int(part.page_indptr[u])
            for t in range(n):
                pg = int(part.page_indices[lo + t // P])
                for kvh in range(w.num_kv_heads):
                    code = torch.tensor([u, kvh, t // 64, t % 64, tag] + [3] * (D - 5), dtype=torch.float32)
                    part.v_pool[pg, kvh, t % P] = code.to(part.v_pool.dtype)
        for h in range(w.num_q_heads):
            t = int(rng.integers(0, lin + lout))
            part, tt, tag = (w.priv, t, 1) if t < lin else (w.pub, t - lin, 2)
            pg = int(part.page_indices[int(part.page_indptr[u]) + tt // P])
            axis = h            # 8 heads, 64 channels: every head has its own axis
            w.q[u, h, axis] = 16.0
            part.k_pool[pg, h // g, tt % P, axis] = 64.0     # score 1024 * scale vs 0 elsewhere
            expect[u, h] = [u, h // g, tt // 64, tt % 64, tag] + [3] * (D - 5)
    out, status, _ = _decode(w.to("cuda"), fused)
    assert status == (spd.SPD_OK, -1)
    assert np.array_equal(out.cpu().numpy().astype(np.float64), expect)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_empty_partitions_and_idle_users(dtype):
    lin = np.array([0, 40, 0, 17, 16, 0, 300])
    lout = np.array([0, 0, 25, 0, 16, 1, 0])
    cfg = dict(batch=7, hq=8, hkv=2, d=128, dtype=dtype, lin=("const", 0), lout=("const", 0), seed=43)
    w = wl.make_workload(cfg, lengths=(lin, lout), slack=True)
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    assert np.all(ref[0] == 0)
    for fused in (True, False):
        out, status, _ = _decode(w.to("cuda"), fused)
        assert status == (spd.SPD_OK, -1)
        assert bool((out[0] == 0).all())                      # nothing cached at all: zeros, not NaN
        assert_close(out.cpu().numpy(), ref, w.dtype, f"empty partitions fused={fused}")
    # a batch whose public partition is empty for everyone (no public pages exist)
    w2 = wl.make_workload(dict(cfg, batch=3), lengths=(np.array([5, 64, 33]), np.zeros(3, dtype=np.int64)))
    q, kin, kout = oracle_inputs(w2)
    out, status, _ = _decode(w2.to("cuda"))
    assert status == (spd.SPD_OK, -1)
    assert_close(out.cpu().numpy(), orc.full(q, kin, kout, w2.sm_scale), w2.dtype, "no public tokens")


def test_bad_page_index_and_bad_length_are_contained():
    name = "bf16_gqa4_d128"
    w = wl.make_workload(dict(SMALL[name], name=name), slack=False)
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    wg = w.to("cuda")
    others = [u for u in range(w.batch) if u not in (3, 5)]
    # user 3: a private page index beyond the pool; user 5: a public length beyond its listed pages
    wg.priv.page_indices[int(wg.priv.page_indptr[3]) + 1] = wg.priv.num_pages
    wg.pub.seq_lens[5] = 16 * int(wg.pub.page_indptr[6] - wg.pub.page_indptr[5]) + 1
    for fused in (True, False):
        out, status, (shape, ws) = _decode(wg, fused)
        assert status == (4, 3)                               # SPD_ERR_BAD_PAGE, lowest flagged user
        assert bool((out[3] == 0).all()) and bool((out[5] == 0).all())
        assert_close(out[others].cpu().numpy(), ref[others], w.dtype, f"bystanders fused={fused}")
        assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)   # the query cleared the flag
    # chained step, flag raised by the private half on users whose public partition is one to four tiles: the
    # second half must keep them zeroed whether it finishes their sequences in one piece or not
    lin = np.array([300, 200, 150, 400, 90, 60])
    lout = np.array([5, 16, 33, 64, 40, 0])
    w3 = wl.make_workload(dict(SMALL[name], name="short_public", batch=6), lengths=(lin, lout))
    q3, kin3, kout3 = oracle_inputs(w3)
    ref3 = orc.full(q3, kin3, kout3, w3.sm_scale)
    g3 = w3.to("cuda")
    for u in range(4):
        g3.priv.page_indices[int(g3.priv.page_indptr[u]) + u] = g3.priv.num_pages + u
    for fused in (False, True):
        out, status, _ = _decode(g3, fused)
        assert status == (4, 0)
        assert bool((out[:4] == 0).all()), f"fused={fused}: flagged users must get zeros"
        assert_close(out[4:].cpu().numpy(), ref3[4:], w3.dtype, f"bystanders of the private half's flags, fused={fused}")
    # negative index, negative length
    wg = w.to("cuda")
    wg.priv.page_indices[int(wg.priv.page_indptr[0])] = -1
    wg.priv.seq_lens[1] = -4
    out, status, _ = _decode(wg)
    assert status == (4, 0) and bool((out[:2] == 0).all())
    assert_close(out[2:].cpu().numpy(), ref[2:], w.dtype, "bystanders of negative inputs")


@pytest.mark.parametrize("name", ["bf16_gqa4_d128", "f32_mha_d64"])
def test_host_blob_step_matches_oracle(name):
    """The end-to-end entry point: per-step inputs in one host buffer, output read back from it."""
    w = wl.make_workload(dict(SMALL[name], name=name), slack=True)
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    lay = spd.spd_step_blob_layout(shape, int(w.priv.page_indices.numel()), int(w.pub.page_indices.numel()), torch.float32)
    host = torch.zeros(lay.total_bytes, dtype=torch.uint8).pin_memory()
    spd.fill_step_blob(lay, host, w.q, w.priv, w.pub)
    devb = torch.empty(lay.total_bytes, dtype=torch.uint8, device="cuda")
    pools = [(p.k_pool.cuda(), p.v_pool.cuda()) for p in (w.priv, w.pub)]
    n = w.batch * w.num_q_heads * w.head_dim
    for _ in range(2):
        host[lay.out:] = 0xFF
        assert spd.spd_decode_step_host(shape, lay, host, devb, pools[0], pools[1], torch.float32, ws) == (spd.SPD_OK, -1)
        out = host[lay.out:lay.out + 4 * n].view(torch.float32).reshape(w.batch, w.num_q_heads, w.head_dim)
        assert_close(out.numpy(), ref, w.dtype, f"{name} host blob")
    step = spd.HostStep(shape, lay, host, devb, pools[0], pools[1], torch.float32, ws)   # marshalled once
    host[lay.out:] = 0xFF
    assert step() == (spd.SPD_OK, -1)
    assert_close(host[lay.out:lay.out + 4 * n].view(torch.float32).reshape(w.batch, w.num_q_heads, w.head_dim).numpy(),
                 ref, w.dtype, f"{name} prepared host step")
    # a page index outside the pool, planted in the host blob: reported, contained, cleared
    idx = host[lay.priv_indices:lay.priv_indices + 4 * w.priv.page_indices.numel()].view(torch.int32)
    keep = int(idx[int(w.priv.page_indptr[1])])
    idx[int(w.priv.page_indptr[1])] = w.priv.num_pages + 3
    assert spd.spd_decode_step_host(shape, lay, host, devb, pools[0], pools[1], torch.float32, ws) == (4, 1)
    out = host[lay.out:lay.out + 4 * n].view(torch.float32).reshape(w.batch, w.num_q_heads, w.head_dim)
    assert bool((out[1] == 0).all())
    idx[int(w.priv.page_indptr[1])] = keep
    assert spd.spd_decode_step_host(shape, lay, host, devb, pools[0], pools[1], torch.float32, ws) == (spd.SPD_OK, -1)
    # a table that claims more pages than the blob holds is refused on the host
    ip = host[lay.priv_indptr:lay.priv_indptr + 4 * (w.batch + 1)].view(torch.int32)
    ip[w.batch] += 1
    with pytest.raises(spd.SpdError):
        spd.spd_decode_step_host(shape, lay, host, devb, pools[0], pools[1], torch.float32, ws)


@pytest.mark.parametrize("batch,out_dtype", [(161, torch.float32), (300, torch.bfloat16), (601, torch.float32)])
def test_host_blob_step_in_parts(batch, out_dtype):
    """A batch whose q and output are megabytes is served in two parts inside the call (the second part's q goes up
    and the first part's output comes down on a copy stream, under the other part's kernel).  Every row against
    the oracle, three steps in a row on the same buffers, odd batches (unequal parts), and a page index outside the
    pool planted in the last part: reported with the user's index in the whole batch."""
    cfg = dict(name="halves", batch=batch, hq=32, hkv=8, d=128, dtype="bf16", lin=("uniform", 1, 400), lout=("uniform", 0, 60), seed=71)
    w = wl.make_workload(cfg)
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    lay = spd.spd_step_blob_layout(shape, int(w.priv.page_indices.numel()), int(w.pub.page_indices.numel()), out_dtype)
    host = torch.zeros(lay.total_bytes, dtype=torch.uint8).pin_memory()
    spd.fill_step_blob(lay, host, w.q, w.priv, w.pub)
    devb = torch.empty(lay.total_bytes, dtype=torch.uint8, device="cuda")
    pools = [(p.k_pool.cuda(), p.v_pool.cuda()) for p in (w.priv, w.pub)]
    n = w.batch * w.num_q_heads * w.head_dim
    es = 4 if out_dtype == torch.float32 else 2
    tol = 2e-3 if out_dtype == torch.float32 else 2e-3 + 2.0 ** -8 * float(np.max(np.abs(ref)))

    def result():
        return host[lay.out:lay.out + es * n].view(out_dtype).reshape(w.batch, w.num_q_heads, w.head_dim).float().numpy()
    for _ in range(3):
        host[lay.out:] = 0xFF
        assert spd.spd_decode_step_host(shape, lay, host, devb, pools[0], pools[1], out_dtype, ws) == (spd.SPD_OK, -1)
        got = result()
        assert np.all(np.isfinite(got)) and np.max(np.abs(got - ref)) <= tol
    victim = batch - 7                                   # in the last part
    idx = host[lay.priv_indices:lay.priv_indices + 4 * w.priv.page_indices.numel()].view(torch.int32)
    at = int(w.priv.page_indptr[victim])
    keep = int(idx[at])
    idx[at] = w.priv.num_pages + 11
    assert spd.spd_decode_step_host(shape, lay, host, devb, pools[0], pools[1], out_dtype, ws) == (4, victim)
    got = result()
    others = [u for u in range(batch) if u != victim]
    assert np.all(got[victim] == 0) and np.max(np.abs(got[others] - ref[others])) <= tol
    idx[at] = keep
    assert spd.spd_decode_step_host(shape, lay, host, devb, pools[0], pools[1], out_dtype, ws) == (spd.SPD_OK, -1)
    assert np.max(np.abs(result() - ref)) <= tol
    # the plain entry point on the same workspace afterwards: the halves left it clean
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    wg = w.to("cuda")
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True)
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    assert_close(out.cpu().numpy(), ref, w.dtype, "plain step after steps in parts")


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_append_kv_is_bit_exact_and_feeds_the_next_step(dtype):
    """Step 3a: the new token's K/V rows go into the public cache, then attention sees them."""
    rng = np.random.default_rng(51)
    B, hq, hkv, d = 6, 8, 4, 128
    lout = np.array([0, 15, 16, 31, 5, 32])           # page boundaries on both sides
    lin = rng.integers(1, 200, size=B)
    cfg = dict(name="append", batch=B, hq=hq, hkv=hkv, d=d, dtype=dtype, lin=("const", 0), lout=("const", 0), seed=52)
    w = wl.make_workload(cfg, lengths=(lin, lout), slack=False, over_alloc=2.0)   # leaves free pages in the pools
    # one spare page for everybody except the last user, whose pages are exactly full
    need = (lout + 15) // 16
    cap = need + 1
    cap[-1] = need[-1]
    used = set(w.pub.page_indices.tolist())
    free = iter(sorted(set(range(w.pub.num_pages)) - used))
    indices, indptr = [], [0]
    for u in range(B):
        own = w.pub.page_indices[int(w.pub.page_indptr[u]):int(w.pub.page_indptr[u + 1])].tolist()
        while len(own) < cap[u]:
            own.append(next(free))
        indices += own
        indptr.append(len(indices))
    w.pub.page_indptr = torch.tensor(indptr, dtype=torch.int32)
    w.pub.page_indices = torch.tensor(indices, dtype=torch.int32)
    gen = torch.Generator().manual_seed(53)
    k_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
    v_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)

    wg = w.to("cuda")
    shape = spd.make_shape(B, hq, hkv, d, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    spd.spd_append_kv(shape, k_new.cuda(), v_new.cuda(), wg.pub, ws)
    status = spd.spd_query_device_status(ws)
    assert status == (4, B - 1)                        # the full user is reported, everybody else appended

    q, kin, kout = oracle_inputs(w)
    done = orc.append(kout, orc.q_from_torch(k_new), orc.q_from_torch(v_new))
    assert done.tolist() == [True] * (B - 1) + [False]
    assert np.array_equal(wg.pub.seq_lens.cpu().numpy(), kout.seq_lens)

    def bits(t):
        return t.cpu().view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32).numpy()
    assert np.array_equal(bits(wg.pub.k_pool), kout.k_pool.view(bits(wg.pub.k_pool).dtype))
    assert np.array_equal(bits(wg.pub.v_pool), kout.v_pool.view(bits(wg.pub.v_pool).dtype))

    out = torch.full((B, hq, d), float("nan"), dtype=torch.float32, device="cuda")
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=True)
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    assert_close(out.cpu().numpy(), orc.full(q, kin, kout, w.sm_scale), w.dtype, "decode after append")


@pytest.mark.parametrize("dtype,hq,hkv,d", [("bf16", 8, 4, 128), ("f32", 8, 4, 128), ("bf16", 32, 2, 128), ("bf16", 4, 4, 64), ("f32", 16, 2, 64)])
def test_append_inside_the_decode_launch(dtype, hq, hkv, d):
    """Steps 3a to 3c in one launch: the new rows reach the cache bit for bit, the lengths grow by one, and the
    output is the attention over the grown cache -- on page boundaries, for an empty public partition, with group
    sizes that split a KV head over several warps (16 query heads per KV head), twice in a row on a stored plan.
    A user whose listed pages are full gets zeros, no append and an unchanged length."""
    rng = np.random.default_rng(151)
    B = 7
    lout = np.array([0, 15, 16, 31, 5, 47, 32])        # the append lands at slot 0, 15, 0 (new page), 15, 5, 15, 0 (no room)
    lin = rng.integers(1, 260, size=B)
    lin[2] = 2900                                       # one long prompt: its sequence is cut into pieces
    cfg = dict(name="append_fused", batch=B, hq=hq, hkv=hkv, d=d, dtype=dtype, lin=("const", 0), lout=("const", 0), seed=152)
    w = wl.make_workload(cfg, lengths=(lin, lout), slack=False, over_alloc=2.0)
    need = (lout + 15) // 16
    cap = need + 1
    cap[-1] = need[-1]                                  # the last user's pages are exactly full
    used = set(w.pub.page_indices.tolist())
    free = iter(sorted(set(range(w.pub.num_pages)) - used))
    indices, indptr = [], [0]
    for u in range(B):
        own = w.pub.page_indices[int(w.pub.page_indptr[u]):int(w.pub.page_indptr[u + 1])].tolist()
        while len(own) < cap[u]:
            own.append(next(free))
        indices += own
        indptr.append(len(indices))
    w.pub.page_indptr = torch.tensor(indptr, dtype=torch.int32)
    w.pub.page_indices = torch.tensor(indices, dtype=torch.int32)
    q, kin, kout = oracle_inputs(w)
    wg = w.to("cuda")
    shape = spd.make_shape(B, hq, hkv, d, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    gen = torch.Generator().manual_seed(153)

    def bits(t):
        return t.cpu().view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32).numpy()

    for step, plan in enumerate((spd.SPD_PLAN_PER_CALL, spd.SPD_PLAN_STORE)):
        k_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
        v_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
        done = orc.append(kout, orc.q_from_torch(k_new), orc.q_from_torch(v_new))
        ref = orc.full(q, kin, kout, w.sm_scale)
        out = torch.full((B, hq, d), float("nan"), dtype=torch.float32, device="cuda")
        spd.spd_decode_step_append(shape, wg.q, k_new.cuda(), v_new.cuda(), wg.priv, wg.pub, out, ws, plan=plan)
        full = [u for u in range(B) if not done[u]]
        status = spd.spd_query_device_status(ws)
        assert status == ((4, full[0]) if full else (spd.SPD_OK, -1)), (step, status)
        assert np.array_equal(wg.pub.seq_lens.cpu().numpy(), kout.seq_lens), f"lengths after append {step}"
        assert np.array_equal(bits(wg.pub.k_pool), kout.k_pool.view(bits(wg.pub.k_pool).dtype)), f"K cache after append {step}"
        assert np.array_equal(bits(wg.pub.v_pool), kout.v_pool.view(bits(wg.pub.v_pool).dtype)), f"V cache after append {step}"
        ok = [u for u in range(B) if done[u]]
        assert bool((out[full] == 0).all())
        assert_close(out[ok].cpu().numpy(), ref[ok], w.dtype, f"attention over the grown cache, step {step}")
    # the paper's split with the append at the head of the service call: the per-user process computes the private
    # partial (it never sees the public cache), the service appends, computes the public partial and merges
    k_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
    v_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
    done = orc.append(kout, orc.q_from_torch(k_new), orc.q_from_torch(v_new))
    ref = orc.full(q, kin, kout, w.sm_scale)
    part = spd.alloc_partial(shape)
    spd.spd_partial_attn(shape, wg.q, wg.priv, part, ws)
    out = torch.full((B, hq, d), float("nan"), dtype=torch.float32, device="cuda")
    spd.spd_service_attn_merge_append(shape, wg.q, k_new.cuda(), v_new.cuda(), wg.pub, part, out, ws)
    assert spd.spd_query_device_status(ws)[0] == 4
    ok = [u for u in range(B) if done[u]]
    assert np.array_equal(wg.pub.seq_lens.cpu().numpy(), kout.seq_lens)
    assert np.array_equal(bits(wg.pub.k_pool), kout.k_pool.view(bits(wg.pub.k_pool).dtype))
    assert np.array_equal(bits(wg.pub.v_pool), kout.v_pool.view(bits(wg.pub.v_pool).dtype))
    assert bool((out[[u for u in range(B) if not done[u]]] == 0).all())
    assert_close(out[ok].cpu().numpy(), ref[ok], w.dtype, "service call with the append at its head")
    wg.pub.seq_lens.copy_(torch.clamp(wg.pub.seq_lens - 1, min=0))            # back to the storing call's lengths + 1
    kout.seq_lens[:] = np.maximum(kout.seq_lens - 1, 0)
    wg.pub.seq_lens[-1] = int(lout[-1]); kout.seq_lens[-1] = int(lout[-1])
    # the stored plan serves another cache with the lengths this one had before the storing call's append
    # (same arrays moved back by one), values of the rows that are appended again differ
    wg.pub.seq_lens.copy_(torch.clamp(wg.pub.seq_lens - 1, min=0))
    kout.seq_lens[:] = np.maximum(kout.seq_lens - 1, 0)
    wg.pub.seq_lens[-1] = int(lout[-1]); kout.seq_lens[-1] = int(lout[-1])     # the full user never moved
    k_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
    v_new = torch.randn((B, hkv, d), generator=gen).to(w.dtype)
    done = orc.append(kout, orc.q_from_torch(k_new), orc.q_from_torch(v_new))
    ref = orc.full(q, kin, kout, w.sm_scale)
    out = torch.full((B, hq, d), float("nan"), dtype=torch.float32, device="cuda")
    spd.spd_decode_step_append(shape, wg.q, k_new.cuda(), v_new.cuda(), wg.priv, wg.pub, out, ws, plan=spd.SPD_PLAN_REUSE)
    assert spd.spd_query_device_status(ws)[0] == 4
    ok = [u for u in range(B) if done[u]]
    assert np.array_equal(wg.pub.seq_lens.cpu().numpy(), kout.seq_lens)
    assert np.array_equal(bits(wg.pub.k_pool), kout.k_pool.view(bits(wg.pub.k_pool).dtype))
    assert_close(out[ok].cpu().numpy(), ref[ok], w.dtype, "append on a reused plan")


@pytest.mark.parametrize("name", ["bf16_gqa4_d128", "bf16_gqa8_d128", "bf16_long_split", "f32_mha_d64", "f32_long_split"])
def test_watched_attention_mass(name):
    """The input-attention monitor: softmax mass on a watched range of the private partition."""
    w = wl.make_workload(dict(SMALL[name], name=name), slack=True)
    rng = np.random.default_rng(61)
    lin = w.priv.seq_lens.numpy()
    lo = np.array([rng.integers(0, max(1, n)) for n in lin])
    hi = np.array([rng.integers(l, n + 40) for l, n in zip(lo, lin)])       # some reach past the partition
    if w.batch > 2:
        hi[0], lo[1], hi[1] = lo[0], 5, 2                                    # an empty and an inverted interval
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    full_ref, own_ref = orc.watched_mass(q, kin, kout, w.sm_scale, lo, hi)
    wg = w.to("cuda")
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    tlo = torch.tensor(lo, dtype=torch.int32, device="cuda")
    thi = torch.tensor(hi, dtype=torch.int32, device="cuda")
    mass = torch.full((w.batch, w.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    tol = TOL[w.dtype][0]
    for _ in range(2):
        spd.spd_decode_step_watch(shape, wg.q, wg.priv, wg.pub, out, tlo, thi, mass, ws)
        assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
        assert_close(out.cpu().numpy(), ref, w.dtype, f"{name} output with the monitor on")
        got = mass.cpu().numpy().astype(np.float64)
        assert np.all(np.isfinite(got)) and np.max(np.abs(got - full_ref)) <= tol, np.max(np.abs(got - full_ref))
    part = spd.alloc_partial(shape)
    lw = torch.full((w.batch, w.num_q_heads), float("nan"), dtype=torch.float32, device="cuda")
    spd.spd_partial_attn_watch(shape, wg.q, wg.priv, part, tlo, thi, lw, ws)
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    l = part[2].cpu().numpy().astype(np.float64)
    share = np.divide(lw.cpu().numpy().astype(np.float64), l, out=np.zeros_like(l), where=l > 0)
    assert np.max(np.abs(share - own_ref)) <= tol
    # the unwatched calls give the same attention output
    out2 = torch.empty_like(out)
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out2, ws, fused=True)
    assert float((out2 - out).abs().max()) <= 2 * tol
