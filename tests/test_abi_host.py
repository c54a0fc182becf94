"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header
declares, sizes its buffers as documented, and rejects bad arguments before anything is launched."""
import ctypes as C
import os
import re

import pytest

from paper_2603_22943_b200 import binding as tb
from paper_2603_22943_b200 import build as tbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    tbuild.build_library()
    return tb.lib()


def _declared_functions():
    src = open(os.path.join(ROOT, "include", "taq.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(taq_[a-z0-9_]+)\s*\(", src)))


def test_every_declared_symbol_is_exported(L):
    names = _declared_functions()
    assert len(names) >= 17
    for n in names:
        assert hasattr(L, n), n
    assert sorted(tb.EXPORTS) == names


def test_status_strings(L):
    assert L.taq_status_string(0) == b"ok"
    seen = {L.taq_status_string(i) for i in range(8)}
    assert len(seen) == 8 and L.taq_status_string(99) == b"unknown status"
    assert L.taq_version() == 1


def test_packed_weight_bytes(L):
    # header 128 + codes + fp32 scales + fp32 bias, each section rounded up to 128 bytes
    d = tb.weight_desc(320, 320, 4, 128)
    assert tb.taq_packed_weight_bytes(d) == 128 + 320 * 160 + 320 * 3 * 4 + 320 * 4
    d8 = tb.weight_desc(1280, 768, 8, 0)
    assert tb.taq_packed_weight_bytes(d8) == 128 + 1280 * 768 + 1280 * 4 + 1280 * 4
    for bad in (tb.weight_desc(320, 320, 3, 0), tb.weight_desc(0, 320, 4, 0), tb.weight_desc(8, 12, 4, 0),
                tb.weight_desc(8, 64, 4, 48), tb.weight_desc(8, 64, 8, 32)):
        assert tb.taq_packed_weight_bytes(bad) == 0
    # the 4-8x memory claim: 32-bit weights over the packed size
    full = 320 * 768 * 4
    assert 7.3 < full / tb.taq_packed_weight_bytes(tb.weight_desc(320, 768, 4, 128)) < 7.6
    assert 3.9 < full / tb.taq_packed_weight_bytes(tb.weight_desc(320, 768, 8, 0)) < 4.0


def test_kv_layout(L):
    d = tb.layer_desc(2, 4096, 320, 8, 77, 768, 4, 128, max_trigger=4)
    lay = tb.taq_kv_layout_of(d)
    codes = -(-8 * 77 * 40 // 128) * 128
    scales = -(-8 * 77 * 4 // 128) * 128
    trig = -(-4 * 8 * 40 * 2 // 128) * 128
    assert lay.off_k_codes == 0 and lay.off_v_codes == codes
    assert lay.off_k_scales == 2 * codes and lay.off_v_scales == 2 * codes + scales
    assert lay.off_k_trigger == 2 * codes + 2 * scales and lay.off_v_trigger == lay.off_k_trigger + trig
    assert lay.off_trig_slot == lay.off_v_trigger + trig and lay.off_operands == lay.off_trig_slot + 512 and lay.block_bytes == lay.off_operands + 8 * lay.operand_head_bytes
    assert lay.operand_head_bytes == 80 * 128 + 2 * 48 * 128 + 1024          # K~ tile, V~^T tile, constants (d = 40)
    assert tb.taq_kv_bytes(d) == 2 * lay.block_bytes
    assert tb.taq_workspace_bytes(d, 1) == 8192 * 320 + 8192 * 8 * 4 + 8192 * 320 * 2
    d0 = tb.layer_desc(2, 4096, 320, 8, 77, 768, 4, 128, q_bits=0)
    assert tb.taq_workspace_bytes(d0, 1) == 8192 * 320 * 2 + 8192 * 8 * 4 + 8192 * 320 * 2


@pytest.mark.parametrize("kwargs,status", [
    (dict(heads=7), tb.TAQ_ERR_SHAPE),                 # 320 % 7 != 0
    (dict(n_ctx=129), tb.TAQ_ERR_SHAPE),
    (dict(n_ctx=0), tb.TAQ_ERR_SHAPE),
    (dict(w_bits=5), tb.TAQ_ERR_INVALID_ARG),
    (dict(q_bits=4), tb.TAQ_ERR_INVALID_ARG),
    (dict(kv_bits=3), tb.TAQ_ERR_UNSUPPORTED),
    (dict(p_bits=2), tb.TAQ_ERR_UNSUPPORTED),
    (dict(max_trigger=78), tb.TAQ_ERR_SHAPE),
    (dict(ctx_dim=100), tb.TAQ_ERR_SHAPE),
    (dict(channels=324, heads=81), tb.TAQ_ERR_SHAPE),  # head width 4
])
def test_bad_layer_descriptors(L, kwargs, status):
    base = dict(batch=2, n_query=64, channels=320, heads=8, n_ctx=77, ctx_dim=768, w_bits=4, w_group=128)
    base.update(kwargs)
    d = tb.layer_desc(**base)
    out = tb.KvLayout()
    assert L.taq_kv_layout_of(C.byref(d), C.byref(out)) == status
    assert L.taq_last_error()
    assert tb.taq_kv_bytes(d) == 0 and tb.taq_workspace_bytes(d, 1) == 0


def test_null_misaligned_and_small_buffers_are_rejected_on_the_host(L):
    d = tb.layer_desc(1, 64, 320, 8, 77, 768, 4, 128)
    wd = tb.weight_desc(320, 320, 4, 128)
    ok = 0x10000            # never dereferenced: every check below fails before a launch
    assert L.taq_pack_weights(C.byref(wd), None, None, ok, 1 << 20, None) == tb.TAQ_ERR_INVALID_ARG
    assert L.taq_pack_weights(C.byref(wd), ok, None, ok + 4, 1 << 20, None) == tb.TAQ_ERR_ALIGNMENT
    assert L.taq_pack_weights(C.byref(wd), ok, None, ok, 100, None) == tb.TAQ_ERR_BUFFER_TOO_SMALL
    assert b"needed" in L.taq_last_error()
    assert L.taq_quantize_rows(ok, 4, 8, 128, ok, ok, None) == tb.TAQ_ERR_INVALID_ARG
    assert L.taq_quantize_rows(ok, -1, 8, 127, ok, ok, None) == tb.TAQ_ERR_SHAPE
    assert L.taq_quantize_rows(None, 0, 8, 127, None, None, None) == tb.TAQ_OK          # empty input: nothing to do
    assert L.taq_kv_project(C.byref(d), ok, ok, ok, ok, ok, 16, None) == tb.TAQ_ERR_BUFFER_TOO_SMALL
    assert L.taq_kv_project(C.byref(d), ok, ok, ok, None, ok, 1 << 30, None) == tb.TAQ_ERR_INVALID_ARG
    assert L.taq_quantized_linear(C.byref(wd), ok, 4, ok, ok, 7, 1, None, None) == tb.TAQ_ERR_INVALID_ARG
    assert L.taq_quantized_linear(C.byref(wd), ok, 4, ok, ok, tb.TAQ_OUT_INT8_HEAD_ROWS, 7, ok, None) == tb.TAQ_ERR_SHAPE
    assert L.taq_quantized_linear(C.byref(wd), ok, 4, ok, ok, tb.TAQ_OUT_INT8_HEAD_ROWS, 8, None, None) == tb.TAQ_ERR_INVALID_ARG
    assert L.taq_cross_attention(C.byref(d), ok, None, ok, ok, ok, None) == tb.TAQ_ERR_INVALID_ARG   # q_bits=8 needs scales
    assert L.taq_layer_forward(C.byref(d), ok, ok, ok, ok, ok, ok, ok + 16, 1 << 30, None) == tb.TAQ_ERR_ALIGNMENT
    assert L.taq_layer_forward(C.byref(d), ok, ok, ok, ok, ok, ok, 0x10000 + 128, 64, None) == tb.TAQ_ERR_BUFFER_TOO_SMALL
    d2 = tb.layer_desc(2, 64, 320, 8, 77, 768, 4, 128)
    assert L.taq_layer_forward_batched(C.byref(d2), ok, 4, ok, ok, 0x20000, 1 << 30, None) == tb.TAQ_ERR_SHAPE   # batch must be 1
    assert L.taq_layer_forward_batched(C.byref(d), ok, 70000, ok, ok, 0x20000, 1 << 30, None) == tb.TAQ_ERR_SHAPE
    # empty problems succeed without touching any pointer
    d_empty = tb.layer_desc(2, 0, 320, 8, 77, 768, 4, 128)
    assert L.taq_layer_forward(C.byref(d_empty), None, None, None, None, None, None, None, 0, None) == tb.TAQ_OK


def test_binding_fails_loudly_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(tb, "_lib", None)
    monkeypatch.setattr(tb, "LIB_PATH", str(tmp_path / "libtaq.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        tb.lib()


def test_linear_plan_keeps_every_region_inside_shared_memory(L):
    """The dequant-GEMM's epilogue stages a tile's output in the ring of operand stages.  For every problem the
    tensor-core kernel accepts, the ring must hold that staging area and every fixed section must lie inside the
    shared memory the launch asks for (a two-stage ring at a short fan-in once was too small for a 160-wide fp32 tile)."""
    seen = 0
    for n_out in (64, 80, 160, 320, 640, 1280):
        for k_in in (64, 128, 192, 256, 320, 640, 768, 1280, 1536, 2048):
            for bits, group in ((4, 128), (4, 0), (4, 64), (8, 0)):
                for rows in (77, 128, 8192, 65536):
                    for kind, heads in ((tb.TAQ_OUT_F16, 1), (tb.TAQ_OUT_F32, 1), (tb.TAQ_OUT_INT8_HEAD_ROWS, max(1, n_out // 40)),
                                        (tb.TAQ_OUT_INT8_HEAD_ROWS, max(1, n_out // 160))):
                        for i8 in (False, True):
                            for batched in (False, True):
                                if kind == tb.TAQ_OUT_INT8_HEAD_ROWS and n_out % heads:
                                    continue
                                plan = tb.taq_linear_plan(tb.weight_desc(n_out, k_in, bits, group), rows, kind, heads, i8, batched)
                                if plan["bn"] == 0:
                                    continue
                                seen += 1
                                what = (n_out, k_in, bits, group, rows, kind, heads, i8, batched, plan)
                                assert plan["nstage"] >= 2, what
                                assert plan["staging_bytes"] <= plan["ring_bytes"], what
                                assert plan["ring_bytes"] <= plan["off_raw"] <= plan["off_bias"] < plan["off_bars"] < plan["total"], what
                                assert plan["total"] <= plan["limit"], what
    assert seen > 1000
    # the case that used to overflow: a 160-wide fp32 tile over a fan-in of 128 (two K blocks)
    plan = tb.taq_linear_plan(tb.weight_desc(320, 128, 4, 128), 8192, tb.TAQ_OUT_F32)
    assert plan["bn"] == 160 and plan["staging_bytes"] == 128 * 160 * 4 and plan["ring_bytes"] >= plan["staging_bytes"]


def test_linear_plan_of_heads_of_160_channels(L):
    """Per-head Q_a over heads of 160 channels: up to one wave of split tiles the projection runs on 80-wide tiles (two
    per head, resident weight tiles); beyond that on one 160-wide tile per head."""
    wd = tb.weight_desc(1280, 1280, 4, 128)
    assert tb.taq_linear_plan(wd, 512, tb.TAQ_OUT_INT8_HEAD_ROWS, heads=8)["bn"] == 80
    assert tb.taq_linear_plan(wd, 64, tb.TAQ_OUT_INT8_HEAD_ROWS, heads=8)["bn"] == 80
    assert tb.taq_linear_plan(wd, 1300, tb.TAQ_OUT_INT8_HEAD_ROWS, heads=8)["bn"] == 160
    assert tb.taq_linear_plan(tb.weight_desc(1280, 1280, 8, 0), 64, tb.TAQ_OUT_INT8_HEAD_ROWS, heads=8)["bn"] == 160   # W8: codes too large to stage


def test_dispatch_counters_start_at_zero_and_reset(L):
    tb.taq_dispatch_reset()
    assert set(tb.taq_dispatch_counts().values()) == {0}
    assert len(tb.taq_dispatch_counts()) == 7


def test_wait_expiry_selftest_rejects_bad_limits(L):
    for bad in (0, -5, (1 << 31) + 1):                 # (refused on the host: nothing is launched)
        assert L.taq_selftest_wait_expiry(bad, None) == tb.TAQ_ERR_INVALID_ARG
