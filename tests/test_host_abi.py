"""CPU-side checks: the library loads, exports what include/spd.h declares, and rejects bad arguments
before touching a device.  No kernel runs here."""
import ctypes as C
import os
import re

import pytest
import torch

from paper_2409_19134_b200 import binding as spd
from paper_2409_19134_b200 import build as spd_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    spd_build.build()
    return spd.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "spd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(spd_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 9
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(spd.EXPORTS) == names


def test_status_strings(lib):
    seen = {spd.status_string(c) for c in range(8)}
    assert len(seen) == 8 and "unknown status" not in seen
    assert spd.status_string(99) == "unknown status"


def test_struct_layouts_match_header(lib):
    assert C.sizeof(spd.Shape) == 28
    assert C.sizeof(spd.PagedKV) == 48 and spd.PagedKV.page_indptr.offset == 24
    assert C.sizeof(spd.Partial) == 24
    assert C.sizeof(spd.StepBlob) == 104


def test_bad_arguments_are_rejected_on_the_host(lib):
    n = C.c_size_t(0)
    ok = spd.make_shape(4, 8, 8, 64, torch.float32, 0.125)
    assert lib.spd_workspace_size(None, C.byref(n)) == 1
    for bad, code in ((spd.make_shape(4, 8, 8, 96, torch.float32, 1.0), 2),          # head_dim
                      (spd.make_shape(4, 8, 3, 64, torch.float32, 1.0), 2),          # heads not divisible
                      (spd.make_shape(4, 24, 8, 64, torch.float32, 1.0), 2),         # group of 3
                      (spd.make_shape(4, 8, 8, 64, torch.float32, 1.0, page_size=32), 2),
                      (spd.make_shape(0, 8, 8, 64, torch.float32, 1.0), 1),
                      (spd.make_shape(4, 8, 8, 64, torch.float32, float("nan")), 1)):
        assert lib.spd_workspace_size(C.byref(bad), C.byref(n)) == code
    part = spd.Partial(None, None, None)
    kv = spd.PagedKV(None, None, 0, None, None, None)
    assert lib.spd_partial_attn(C.byref(ok), None, None, part, None, 0, None) == 1
    assert lib.spd_partial_attn(C.byref(ok), None, C.byref(kv), part, None, 0, None) == 1   # null tables
    assert lib.spd_decode_step(C.byref(ok), None, None, None, None, 0, 1, None, 0, None) == 1
    assert lib.spd_query_device_status(None, None, None) == 1
    assert lib.spd_profile_begin(0) == 1
    lay = spd.StepBlob()
    assert lib.spd_step_blob_layout(C.byref(ok), -1, 0, 0, C.byref(lay)) == 1
    assert lib.spd_step_blob_layout(C.byref(ok), 10, 10, 0, C.byref(lay)) == 0
    assert lay.in_bytes >= 4 * 8 * 64 * 4 + 2 * (5 + 4 + 10) * 4 and lay.total_bytes >= lay.out + 4 * 8 * 64 * 4
    assert lay.q == 0 and lay.out == lay.in_bytes and lay.status + 256 == lay.in_bytes and lay.priv_indices % 256 == 0
    assert lib.spd_decode_step_host(C.byref(ok), C.byref(lay), None, None, None, None, 0, None, None, 0, None) == 1
    # prefill: positive scale only, null offsets refused; the token step and the knobs check their arguments
    pf_args = (C.c_int64(0), None, None, None, None, None, None, 0, None, None, None, None, 1, None, 0, None)
    assert lib.spd_prefill_attn(C.byref(ok), *pf_args) == 1
    assert lib.spd_prefill_attn(C.byref(spd.make_shape(2, 8, 8, 128, torch.bfloat16, -1.0)), *pf_args) == 2
    assert lib.spd_prefill_attn(C.byref(spd.make_shape(2, 8, 8, 128, torch.bfloat16, 0.1)), *pf_args) == 1   # null offsets
    assert lib.spd_token_step(C.byref(ok), 0, None, 0, 0, None, 0, None) == 1
    assert lib.spd_token_step(C.byref(ok), 2, None, 0, 1, None, 0, None) == 1
    # the planned calls check the plan mode first; the knobs and the debugging aids check their arguments
    assert lib.spd_decode_step_planned(C.byref(ok), None, None, None, None, 0, 1, 3, None, 0, None) == 1
    assert lib.spd_partial_attn_planned(C.byref(ok), None, None, part, -1, None, 0, None) == 1
    assert lib.spd_service_attn_merge_planned(C.byref(ok), None, None, part, None, 0, 5, None, 0, None) == 1
    assert lib.spd_set_split(-1, 0) == 1 and lib.spd_set_split(4, 2) == 1 and lib.spd_set_split(0, 0) == 0
    assert lib.spd_set_programmatic_launch(2) == 1
    assert lib.spd_debug_read_plan(None, 0, None, None, None, None, 0) == 1
    assert lib.spd_debug_sm_moves(None, None, None, None) == 1
    assert lib.spd_set_prefill_rows(64) == 1 and lib.spd_set_prefill_rows(256) == 0 and lib.spd_set_prefill_rows(8) == 0
    assert lib.spd_set_prefill_rows(0) == 0
    assert lib.spd_set_bf16_math(2) == 1


def test_watch_alarm_thresholds_the_mean_over_the_watched_heads(lib):
    """Sec. 2.4.4: an attack is detected whenever the monitored attention score falls below a threshold."""
    mass = torch.tensor([[0.50, 0.10, 0.30, 0.10],      # mean 0.25 over all heads, 0.40 over heads 0 and 2
                         [0.05, 0.90, 0.01, 0.90],      # mean 0.465 over all, 0.03 over heads 0 and 2
                         [0.20, 0.20, 0.20, 0.20],
                         [float("nan"), 0.9, 0.9, 0.9]], dtype=torch.float32)
    alarm, score = spd.spd_watch_alarm(mass, 0.25)
    assert alarm.tolist() == [0, 0, 1, 1]                # 0.25 is not below 0.25; NaN raises the alarm
    assert torch.allclose(score[:3], torch.tensor([0.25, 0.465, 0.20]), atol=1e-7)
    alarm, score = spd.spd_watch_alarm(mass, 0.25, head_mask=torch.tensor([1, 0, 1, 0]))
    assert alarm.tolist() == [0, 1, 1, 1]
    assert torch.allclose(score[:3], torch.tensor([0.40, 0.03, 0.20]), atol=1e-7)
    alarm, _ = spd.spd_watch_alarm(mass, 0.0, head_mask=torch.zeros(4))
    assert alarm.tolist() == [1, 1, 1, 1]                # nothing watched: nothing vouches for the user
    a = (C.c_int32 * 4)()
    assert lib.spd_watch_alarm(None, 4, 4, None, 0.1, a, None) == 1
    assert lib.spd_watch_alarm(mass.data_ptr(), 0, 4, None, 0.1, a, None) == 1
    assert lib.spd_watch_alarm(mass.data_ptr(), 4, 4, None, float("nan"), a, None) == 1


def test_binding_fails_loudly_without_the_library(monkeypatch):
    monkeypatch.setattr(spd, "_lib", None)
    monkeypatch.setattr(spd, "LIB_PATH", "/nonexistent/libspd.so")
    with pytest.raises(FileNotFoundError):
        spd.lib()
