"""Host-side checks that need no GPU: the library loads, exports what the header declares, and
rejects bad arguments before touching the device."""
import ctypes as C
import math
import os
import re

import pytest
import torch

from paper_2510_03515_b200 import binding as rb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = 0x10000  # a non-NULL, 256-byte aligned "device pointer" that is never dereferenced on the host


def _declared_symbols():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if fn.endswith(".h"):
            text = open(os.path.join(inc, fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(rapid_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    L = rb.lib()
    declared = _declared_symbols()
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(L, name), f"{name} declared in include/ but not exported"
    assert set(rb.EXPORTS) <= declared


def test_struct_layout_matches_header():
    assert C.sizeof(rb.RapidDesc) == 48
    assert C.sizeof(rb.RapidStats) == 48
    assert rb.RapidDesc.ld.offset == 16 and rb.RapidDesc.eta.offset == 32 and rb.RapidDesc.norm_z.offset == 40
    assert rb.RapidStats.mean_log_cw.offset == 24


def test_status_strings_and_version():
    assert rb.status_string(0) == "RAPID_OK"
    assert rb.status_string(rb.RAPID_ERR_WORKSPACE) == "RAPID_ERR_WORKSPACE"
    assert rb.status_string(99) == "RAPID_ERR_UNKNOWN"
    assert rb.rapid_version() >= 100


def test_workspace_bytes():
    d = rb.make_desc(64, 1024, 151936, 8, torch.bfloat16)
    n = rb.rapid_workspace_bytes(d)
    T = 64 * 1024
    assert 21 * T <= n <= 21 * T + 64 * 1024
    with pytest.raises(rb.RapidError) as e:
        rb.rapid_workspace_bytes(rb.make_desc(0, 4, 8, 1, torch.float32))
    assert e.value.code == rb.RAPID_ERR_INVALID_ARG


def _call_fwd_bwd(desc, logits=FAKE, dlogits=FAKE + (1 << 30), ws=FAKE, ws_bytes=1 << 40, **kw):
    L = rb.lib()
    args = dict(targets=FAKE, mask=None, behav=FAKE, rewards=FAKE, go=FAKE, loss=FAKE)
    args.update(kw)
    return L.rapid_pg_loss_fwd_bwd(C.byref(desc), logits, args["targets"], args["mask"], args["behav"],
                                   args["rewards"], args["go"], dlogits, args["loss"], None, None, None,
                                   ws, ws_bytes, None)


def test_argument_validation_happens_before_any_launch():
    good = rb.make_desc(4, 8, 64, 2, torch.bfloat16)
    assert _call_fwd_bwd(good, logits=None) == rb.RAPID_ERR_INVALID_ARG
    assert _call_fwd_bwd(good, targets=None) == rb.RAPID_ERR_INVALID_ARG
    assert _call_fwd_bwd(good, loss=None) == rb.RAPID_ERR_INVALID_ARG
    assert _call_fwd_bwd(good, logits=FAKE + 8) == rb.RAPID_ERR_ALIGNMENT
    assert _call_fwd_bwd(good, ws=None) == rb.RAPID_ERR_WORKSPACE
    assert _call_fwd_bwd(good, ws=FAKE + 16) == rb.RAPID_ERR_WORKSPACE
    assert _call_fwd_bwd(good, ws_bytes=100) == rb.RAPID_ERR_WORKSPACE
    # partial overlap of logits and dlogits
    assert _call_fwd_bwd(good, dlogits=FAKE + 64) == rb.RAPID_ERR_INVALID_ARG
    for bad in (rb.make_desc(4, 8, 64, 2, torch.bfloat16, ld=60),          # ld < vocab
                rb.make_desc(4, 0, 64, 2, torch.bfloat16),                 # empty grid
                rb.make_desc(4, 8, 64, 0, torch.bfloat16),                 # no groups
                rb.make_desc(4, 8, 64, 2, torch.bfloat16, eta=0.0),
                rb.make_desc(4, 8, 64, 2, torch.bfloat16, eta=math.nan),
                rb.make_desc(4, 8, 64, 2, torch.bfloat16, flags=rb.FLAG_NORM_GIVEN, norm_z=0.0),
                rb.make_desc(4, 8, 64, 2, torch.bfloat16, flags=rb.FLAG_NORM_GIVEN, norm_z=math.inf),
                rb.make_desc(4, 8, 64, 2, torch.bfloat16, flags=rb.FLAG_ADV_INPUT_IS_WEIGHT)):
        assert _call_fwd_bwd(bad) == rb.RAPID_ERR_INVALID_ARG
    odd = rb.make_desc(4, 8, 60, 2, torch.bfloat16, ld=60)                 # 120-byte pitch
    assert _call_fwd_bwd(odd) == rb.RAPID_ERR_ALIGNMENT
    bad_dtype = rb.make_desc(4, 8, 64, 2, torch.bfloat16)
    bad_dtype.dtype = 5
    assert _call_fwd_bwd(bad_dtype) == rb.RAPID_ERR_INVALID_ARG
    assert rb.lib().rapid_pg_loss_fwd_bwd(None, FAKE, FAKE, None, FAKE, FAKE, FAKE, FAKE, FAKE, None,
                                          None, None, FAKE, 1 << 40, None) == rb.RAPID_ERR_INVALID_ARG


def test_chunk_range_validation():
    L = rb.lib()
    d = rb.make_desc(4, 8, 64, 2, torch.float32)
    big = 1 << 40
    assert L.rapid_pg_stats_chunk(C.byref(d), FAKE, 30, 3, FAKE, None, FAKE, big, None) == rb.RAPID_ERR_INVALID_ARG
    assert L.rapid_pg_stats_chunk(C.byref(d), FAKE, -1, 3, FAKE, None, FAKE, big, None) == rb.RAPID_ERR_INVALID_ARG
    assert L.rapid_pg_dlogits_chunk(C.byref(d), FAKE, FAKE + 256, 0, 8, FAKE, None, FAKE, big, None) == rb.RAPID_ERR_INVALID_ARG
    assert L.rapid_group_advantage(C.byref(d), None, None, FAKE, FAKE, None, None, None) == rb.RAPID_ERR_INVALID_ARG


@pytest.mark.skipif(torch.cuda.is_available(), reason="only meaningful on a machine without a GPU")
def test_no_gpu_means_an_error_not_a_fallback():
    """With valid arguments but no CUDA device the call must fail loudly (there is no CPU path)."""
    d = rb.make_desc(4, 8, 64, 2, torch.float32)
    code = _call_fwd_bwd(d)
    assert code in (rb.RAPID_ERR_CUDA, rb.RAPID_ERR_UNSUPPORTED)


def test_missing_library_raises(monkeypatch):
    monkeypatch.setattr(rb, "_lib", None)
    monkeypatch.setattr(rb, "LIB_PATH", "/nonexistent/librapid_pg.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        rb.lib()


def test_onpolicy_argument_validation():
    L = rb.lib()
    good = rb.make_desc(4, 8, 64, 2, torch.bfloat16)
    big = 1 << 40

    def call(desc, logits=FAKE, dlogits=FAKE + (1 << 30), targets=FAKE, rewards=FAKE, go=FAKE, loss=FAKE,
             ws=FAKE, ws_bytes=big):
        return L.rapid_pg_loss_onpolicy_fwd_bwd(C.byref(desc), logits, targets, None, rewards, go, dlogits, loss,
                                                None, None, None, ws, ws_bytes, None)

    assert call(good, logits=None) == rb.RAPID_ERR_INVALID_ARG
    assert call(good, rewards=None) == rb.RAPID_ERR_INVALID_ARG
    assert call(good, loss=None) == rb.RAPID_ERR_INVALID_ARG
    assert call(good, logits=FAKE + 4) == rb.RAPID_ERR_ALIGNMENT
    assert call(good, dlogits=FAKE + 64) == rb.RAPID_ERR_INVALID_ARG       # partial overlap
    assert call(good, ws=None) == rb.RAPID_ERR_WORKSPACE
    assert call(good, ws_bytes=64) == rb.RAPID_ERR_WORKSPACE
    assert call(rb.make_desc(4, 8, 64, 2, torch.bfloat16, ld=60)) == rb.RAPID_ERR_INVALID_ARG
    assert call(rb.make_desc(4, 8, 60, 2, torch.bfloat16, ld=60)) == rb.RAPID_ERR_ALIGNMENT


def test_fused_head_argument_validation():
    L = rb.lib()
    good = rb.make_desc(4, 8, 64, 2, torch.bfloat16)
    big = 1 << 40
    WS = 0x100000   # 1024-byte aligned

    def call(desc, D=64, hidden=FAKE, w=FAKE, dh=FAKE, dW=FAKE, loss=FAKE, ws=WS, ws_bytes=big):
        return L.rapid_pg_loss_fused_head(C.byref(desc), D, hidden, w, FAKE, None, FAKE, FAKE, FAKE, loss, dh, dW,
                                          None, None, None, ws, ws_bytes, None)

    assert call(good, hidden=None) == rb.RAPID_ERR_INVALID_ARG
    assert call(good, dW=None) == rb.RAPID_ERR_INVALID_ARG
    assert call(good, D=0) == rb.RAPID_ERR_INVALID_ARG
    assert call(good, D=60) == rb.RAPID_ERR_ALIGNMENT                      # hidden pitch not 16-byte
    assert call(good, w=FAKE + 8) == rb.RAPID_ERR_ALIGNMENT
    assert call(good, ws=WS + 256) == rb.RAPID_ERR_WORKSPACE               # needs 1024-byte alignment
    assert call(good, ws_bytes=1000) == rb.RAPID_ERR_WORKSPACE
    assert call(rb.make_desc(4, 8, 64, 2, torch.float32)) == rb.RAPID_ERR_INVALID_ARG      # bf16 only
    assert call(rb.make_desc(4, 8, 60, 2, torch.bfloat16, ld=60)) == rb.RAPID_ERR_ALIGNMENT
    n = rb.rapid_fused_head_workspace_bytes(rb.make_desc(64, 256, 151936, 8, torch.bfloat16), 1536)
    T, V = 64 * 256, 151936
    assert T * ((V + 63) // 64 * 64) * 2 <= n <= T * ((V + 63) // 64 * 64) * 2 + 2 * 594 * T * 4 + 64 * T
    with pytest.raises(rb.RapidError):
        rb.rapid_fused_head_workspace_bytes(rb.make_desc(64, 256, 151936, 8, torch.float32), 1536)


def test_bounded_wait_selftest_refuses_bad_limits_on_the_host():
    """NULL statistics, a zero limit and a limit above one second are refused before anything is launched."""
    L = rb.lib()
    assert L.rapid_selftest_bounded_wait(1000, None, None) == rb.RAPID_ERR_INVALID_ARG
    assert L.rapid_selftest_bounded_wait(0, FAKE, None) == rb.RAPID_ERR_INVALID_ARG
    assert L.rapid_selftest_bounded_wait(1_000_000_001, FAKE, None) == rb.RAPID_ERR_UNSUPPORTED
