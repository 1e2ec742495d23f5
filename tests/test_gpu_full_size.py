"""The benchmark's workloads at full size, in the benchmark's launch configuration, every row of every output.

For each of the four bf16 configurations the pools are generated on the GPU, copied to the host once, and the
oracle computes the full attention and the private partial for ALL users and query heads.  Against those, element
by element at the bf16 tolerances (max-abs 2e-3, relative L2 1e-3):
  - spd_decode_step, fused (what the benchmark times) and chained (the paper's two calls through a partial);
  - spd_partial_attn: gauge-free A = O / l and lse = m + ln l, and m itself against the true maximum;
  - spd_service_attn_merge fed with the oracle's private partial rounded to fp32 (a message produced elsewhere).
  - spd_decode_step_append (append and attention in one launch) deriving and storing its plan, then once more on the
    stored plan: every row, the lengths, and the appended rows in the cache bit for bit.
The measured errors are appended to full_size_errors.jsonl in the folder that SPD_TEST_RECORD_DIR names, if it is set.
"""
import json
import os

import numpy as np
import pytest
import torch

from oracle import spd_oracle as orc
from paper_2409_19134_b200 import binding as spd
from paper_2409_19134_b200 import workloads as wl
from tests.test_gpu_parity import TOL, assert_close, errors

pytestmark = pytest.mark.gpu

FULL = ["c2_llama2_7b", "c3_llama3_8b_gqa", "c4_long_prompt", "c5_many_user"]


def _record(entry):
    folder = os.environ.get("SPD_TEST_RECORD_DIR")
    if not folder:
        return
    try:
        os.makedirs(folder, exist_ok=True)
        with open(os.path.join(folder, "full_size_errors.jsonl"), "a") as f:
            f.write(json.dumps(entry) + "\n")
    except OSError:
        pass


@pytest.mark.parametrize("name", FULL)
def test_full_size_every_row_of_every_entry_point(name):
    w = wl.make_workload(name, device="cuda")
    B, Hq, D = w.batch, w.num_q_heads, w.head_dim
    # the same bytes for the oracle: one copy of the pools to the host
    wc = w.to("cpu")
    q, kin, kout = orc.q_from_torch(wc.q), orc.kv_from_torch(wc.priv), orc.kv_from_torch(wc.pub)
    ref = orc.full(q, kin, kout, w.sm_scale)
    o_ref, m_ref, l_ref = orc.partial(q, kin, w.sm_scale)
    assert np.all(l_ref > 0)                       # every config has prompts of at least 16 tokens

    shape = spd.make_shape(B, Hq, w.num_kv_heads, D, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    out = torch.empty((B, Hq, D), dtype=torch.float32, device="cuda")
    report = {"config": name, "rows": B * Hq}

    def check_out(what):
        assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
        got = out.cpu().numpy()
        report[what] = dict(zip(("max_abs", "rel_l2"), errors(got, ref)))
        assert_close(got, ref, w.dtype, f"{name} {what}")

    for warm in range(3):                          # the third call runs on shares sized by measured rates, like the benchmark's
        out.fill_(float("nan"))
        spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws, fused=True)
    check_out("decode_step_fused")
    out.fill_(float("nan"))
    spd.spd_decode_step(shape, w.q, w.priv, w.pub, out, ws, fused=False)
    check_out("decode_step_chained")

    part = spd.alloc_partial(shape)
    for t in part:
        t.fill_(float("nan"))
    spd.spd_partial_attn(shape, w.q, w.priv, part, ws)
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    o, m, l = (t.cpu().numpy().astype(np.float64) for t in part)
    assert np.all(np.isfinite(o)) and np.all(l > 0)
    a_got, a_ref = o / l[..., None], o_ref / l_ref[..., None]
    report["partial_attn_A"] = dict(zip(("max_abs", "rel_l2"), errors(a_got, a_ref)))
    assert_close(a_got, a_ref, w.dtype, f"{name} A_in of spd_partial_attn")
    lse_err = float(np.max(np.abs((m + np.log(l)) - (m_ref + np.log(l_ref)))))
    m_err = float(np.max(np.abs(m - m_ref)))
    report["partial_attn_lse_max_abs"], report["partial_attn_m_max_abs"] = lse_err, m_err
    assert lse_err < 1e-3 and m_err < 1e-4

    ext = tuple(torch.from_numpy(x.astype(np.float32)).cuda() for x in (o_ref, m_ref, l_ref))
    out.fill_(float("nan"))
    spd.spd_service_attn_merge(shape, w.q, w.pub, ext, out, ws)
    check_out("service_attn_merge")

    # the append inside the launch, twice: once deriving and storing the plan, once more on the stored plan after the
    # lengths have been moved back (what the layers of a token step do).  The listed pages have room for one more
    # token for every user whose public length is not a multiple of 16; the others are full: zeros, no append, flagged.
    gen = torch.Generator(device="cuda").manual_seed(77)
    k_new = torch.randn((B, w.num_kv_heads, D), generator=gen, device="cuda").to(w.dtype)
    v_new = torch.randn((B, w.num_kv_heads, D), generator=gen, device="cuda").to(w.dtype)
    lens_before = w.pub.seq_lens.clone()
    done = orc.append(kout, orc.q_from_torch(k_new.cpu()), orc.q_from_torch(v_new.cpu()))
    ref = orc.full(q, kin, kout, w.sm_scale)
    ok = torch.from_numpy(np.flatnonzero(done)).cuda()
    full = torch.from_numpy(np.flatnonzero(~done)).cuda()
    assert len(ok) > B // 2
    for plan in (spd.SPD_PLAN_STORE, spd.SPD_PLAN_REUSE):
        w.pub.seq_lens.copy_(lens_before)
        out.fill_(float("nan"))
        spd.spd_decode_step_append(shape, w.q, k_new, v_new, w.priv, w.pub, out, ws, plan=plan)
        code, first_bad = spd.spd_query_device_status(ws)
        assert (code, first_bad) == ((4, int(full.min())) if len(full) else (spd.SPD_OK, -1))
        assert np.array_equal(w.pub.seq_lens.cpu().numpy(), kout.seq_lens)
        assert bool((out[full] == 0).all())
        got = out[ok].cpu().numpy()
        report[f"decode_step_append_plan{plan}"] = dict(zip(("max_abs", "rel_l2"), errors(got, ref[ok.cpu().numpy()])))
        assert_close(got, ref[ok.cpu().numpy()], w.dtype, f"{name} append inside the launch, plan mode {plan}")
    # the appended rows sit in the cache bit for bit: position lens_before of every user that had room
    pos = lens_before[ok].long()
    pages = w.pub.page_indices[(w.pub.page_indptr[ok].long() + pos // 16)].long()
    assert torch.equal(w.pub.k_pool[pages, :, pos % 16], k_new[ok]) and torch.equal(w.pub.v_pool[pages, :, pos % 16], v_new[ok])
    _record(report)
