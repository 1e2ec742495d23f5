"""Parity of the CUDA path (through the C ABI) with the float64 CPU oracle, element by element.

Tolerances (max-abs and relative-L2 of the final output):
  bf16 KV, fp32 accumulation : 2e-3 and 1e-3
  fp32 KV                    : 1e-5 and 1e-5
Partials are compared gauge-free (A = O / l and lse = m + ln l), because fp32 and fp64 may settle on
maxima that differ in the last bits; m itself must equal the true maximum within fp32 rounding.
"""
import math

import numpy as np
import pytest
import torch

from oracle import spd_oracle as orc
from paper_2409_19134_b200 import binding as spd
from paper_2409_19134_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL = {torch.float32: (1e-5, 1e-5), torch.bfloat16: (2e-3, 1e-3)}


def errors(got: np.ndarray, ref: np.ndarray):
    diff = got.astype(np.float64) - ref
    return float(np.max(np.abs(diff))) if diff.size else 0.0, float(np.linalg.norm(diff) / max(np.linalg.norm(ref), 1e-30))


def assert_close(got, ref, dtype, what=""):
    ma, rl = errors(got, ref)
    ta, tr = TOL[dtype]
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    assert ma <= ta and rl <= tr, f"{what}: max-abs {ma:.3e} (tol {ta}), rel-L2 {rl:.3e} (tol {tr})"


def oracle_inputs(w):
    return orc.q_from_torch(w.q), orc.kv_from_torch(w.priv), orc.kv_from_torch(w.pub)


def run_decode(wg, fused, out_dtype=torch.float32):
    shape = spd.make_shape(wg.batch, wg.num_q_heads, wg.num_kv_heads, wg.head_dim, wg.dtype, wg.sm_scale)
    ws = spd.alloc_workspace(shape)
    out = torch.full((wg.batch, wg.num_q_heads, wg.head_dim), float("nan"), dtype=out_dtype, device="cuda")
    spd.spd_decode_step(shape, wg.q, wg.priv, wg.pub, out, ws, fused=fused)
    code, bad = spd.spd_query_device_status(ws)
    assert code == spd.SPD_OK and bad == -1
    return out.float().cpu().numpy()


SMALL = {
    "f32_mha_d64": dict(batch=4, hq=8, hkv=8, d=64, dtype="f32", lin=("uniform", 1, 300), lout=("uniform", 0, 70), seed=11),
    "f32_gqa4_d128": dict(batch=5, hq=8, hkv=2, d=128, dtype="f32", lin=("uniform", 1, 500), lout=("uniform", 0, 90), seed=12),
    "f32_gqa8_d64": dict(batch=3, hq=16, hkv=2, d=64, dtype="f32", lin=("uniform", 1, 200), lout=("uniform", 1, 50), seed=13),
    "f32_gqa2_d128": dict(batch=3, hq=4, hkv=2, d=128, dtype="f32", lin=("uniform", 1, 200), lout=("uniform", 1, 50), seed=14),
    "bf16_mha_d128": dict(batch=6, hq=8, hkv=8, d=128, dtype="bf16", lin=("uniform", 1, 700), lout=("uniform", 0, 100), seed=15),
    "bf16_gqa4_d128": dict(batch=9, hq=32, hkv=8, d=128, dtype="bf16", lin=("uniform", 1, 2500), lout=("uniform", 0, 300), seed=16),
    "bf16_gqa8_d128": dict(batch=7, hq=64, hkv=8, d=128, dtype="bf16", lin=("lognormal", 300, 0.8, 16, 4000), lout=("uniform", 0, 500), seed=17),
    "bf16_gqa16_d128": dict(batch=3, hq=32, hkv=2, d=128, dtype="bf16", lin=("uniform", 1, 600), lout=("uniform", 0, 100), seed=18),
    "bf16_gqa2_d64": dict(batch=5, hq=8, hkv=4, d=64, dtype="bf16", lin=("uniform", 1, 900), lout=("uniform", 0, 100), seed=19),
    # few long sequences: every sequence is cut across many warps (second-level merge everywhere)
    "bf16_long_split": dict(batch=2, hq=8, hkv=2, d=128, dtype="bf16", lin=("uniform", 30000, 40000), lout=("uniform", 1, 40), seed=20),
    "f32_long_split": dict(batch=1, hq=2, hkv=2, d=64, dtype="f32", lin=("const", 20000), lout=("const", 33), seed=21),
}


@pytest.mark.parametrize("name", list(SMALL))
@pytest.mark.parametrize("fused", [True, False])
def test_decode_step_matches_oracle(name, fused):
    w = wl.make_workload(dict(SMALL[name], name=name), slack=True)
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    got = run_decode(w.to("cuda"), fused)
    assert_close(got, ref, w.dtype, f"{name} fused={fused}")


def test_config1_tiny_mha_fp32():
    w = wl.make_workload("c1_tiny_mha")
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    for fused in (True, False):
        assert_close(run_decode(w.to("cuda"), fused), ref, w.dtype, f"config 1 fused={fused}")
    # the paper's Eq. 1 carries no 1/sqrt(d): same check with scale 1 on smaller values
    w1 = wl.make_workload("c1_tiny_mha", sm_scale=1.0)
    w1.q.mul_(0.2)
    q, kin, kout = oracle_inputs(w1)
    assert_close(run_decode(w1.to("cuda"), True), orc.full(q, kin, kout, 1.0), w1.dtype, "config 1 scale 1")


@pytest.mark.parametrize("name", ["f32_gqa4_d128", "bf16_gqa4_d128", "bf16_gqa8_d128", "bf16_long_split", "f32_long_split"])
def test_partial_and_service_calls(name):
    """The two halves separately: the private partial as a message, then public partial + merge."""
    w = wl.make_workload(dict(SMALL[name], name=name), slack=True)
    q, kin, kout = oracle_inputs(w)
    o_ref, m_ref, l_ref = orc.partial(q, kin, w.sm_scale)
    ref = orc.full(q, kin, kout, w.sm_scale)
    wg = w.to("cuda")
    shape = spd.make_shape(w.batch, w.num_q_heads, w.num_kv_heads, w.head_dim, w.dtype, w.sm_scale)
    ws = spd.alloc_workspace(shape)
    part = spd.alloc_partial(shape)
    for t in part:
        t.fill_(float("nan"))
    spd.spd_partial_attn(shape, wg.q, wg.priv, part, ws)
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    o, m, l = (t.cpu().numpy().astype(np.float64) for t in part)
    nonempty = l_ref > 0
    assert np.array_equal(l > 0, nonempty)
    assert np.all(np.isneginf(m[~nonempty])) and np.all(o[~nonempty] == 0) and np.all(l[~nonempty] == 0)
    a_ref = o_ref[nonempty] / l_ref[nonempty][:, None]
    assert_close(o[nonempty] / l[nonempty][:, None], a_ref, w.dtype, f"{name} A_in")
    lse_tol = 1e-5 if w.dtype == torch.float32 else 1e-3
    assert np.max(np.abs((m + np.log(l))[nonempty] - (m_ref + np.log(l_ref))[nonempty])) < lse_tol
    # m is the running maximum itself (bf16 products are exact in fp32, so only summation order differs)
    assert np.max(np.abs(m[nonempty] - m_ref[nonempty])) < 1e-4
    out = torch.full((w.batch, w.num_q_heads, w.head_dim), float("nan"), dtype=torch.float32, device="cuda")
    spd.spd_service_attn_merge(shape, wg.q, wg.pub, part, out, ws)
    assert spd.spd_query_device_status(ws) == (spd.SPD_OK, -1)
    assert_close(out.cpu().numpy(), ref, w.dtype, f"{name} service merge")
    # a partial produced elsewhere (here: by the oracle, rounded to fp32) merges just as well
    ext = tuple(torch.from_numpy(x.astype(np.float32)).cuda() for x in (o_ref, m_ref, l_ref))
    out.fill_(float("nan"))
    spd.spd_service_attn_merge(shape, wg.q, wg.pub, ext, out, ws)
    assert_close(out.cpu().numpy(), ref, w.dtype, f"{name} service merge of an external partial")


def test_bf16_output_dtype():
    w = wl.make_workload(dict(SMALL["bf16_gqa4_d128"], name="bf16out"))
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    got = run_decode(w.to("cuda"), True, out_dtype=torch.bfloat16)
    # output rounded to bf16: half an ulp of values up to ~4 on top of the compute error
    assert np.max(np.abs(got - ref)) <= 2e-3 + 2.0 ** -8 * np.max(np.abs(ref))


@pytest.mark.parametrize("name", ["bf16_mha_d128", "bf16_gqa4_d128", "bf16_gqa8_d128", "bf16_gqa16_d128", "bf16_gqa2_d64", "bf16_long_split"])
def test_bf16_fma_pipe_arm_matches_oracle(name):
    """The comparison arm (bf16 tiles on the FMA pipes instead of the tensor cores) computes the same thing."""
    w = wl.make_workload(dict(SMALL[name], name=name), slack=True)
    q, kin, kout = oracle_inputs(w)
    ref = orc.full(q, kin, kout, w.sm_scale)
    spd.spd_set_bf16_math(1)
    try:
        for fused in (True, False):
            assert_close(run_decode(w.to("cuda"), fused), ref, w.dtype, f"{name} FMA arm fused={fused}")
    finally:
        spd.spd_set_bf16_math(0)
