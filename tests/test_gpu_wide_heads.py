"""The stand-alone attention kernel when a CTA walks a group of several heads (launches large enough that one head per
CTA would oversubscribe the GPU): heads of 80 and 160 channels reload K~ and V~^T separately into a single image buffer
and move Q~ / O by TMA through staging buffers that are reused from head to head, heads of 40 and 64 rotate two image
buffers.  Fed with the oracle's own Q~, K~, V~ and compared element by element on every row."""
from dataclasses import replace

import numpy as np
import pytest

from oracle import taq_oracle as orc
from paper_2603_22943_b200 import binding as tb
from paper_2603_22943_b200 import synth

import taq_testlib as tl
from taq_testlib import dev

pytestmark = pytest.mark.gpu


def _cases():
    c3 = synth.config3_layers()
    return [
        (replace(c3[10], batch=64, n_query=256, seed=51), 8),                 # d = 160: 128 row tiles, eight heads per CTA
        (replace(c3[10], batch=40, n_query=200, seed=52, q_bits=0), 8),       # fp16 Q: one shared staging buffer; ragged tiles
        (replace(c3[5], batch=16, n_query=1024, seed=53), 8),                 # d = 80
        (replace(c3[5], batch=9, n_query=1000, seed=54, p_bits=4, kv_bits=4), 8),
        (replace(synth.config4_layers()[0], batch=8, n_query=2048, seed=55), 8),   # d = 64, ten heads: two image buffers
        (replace(synth.config2(), batch=32, n_query=1024, seed=56), 8),       # d = 40 beyond one wave: the per-head kernel
    ]


@pytest.mark.parametrize("shape,q_bits", _cases(), ids=lambda v: getattr(v, "name", str(v)))
def test_attention_over_head_groups(shape, q_bits):
    shape = replace(shape, q_bits=shape.q_bits if shape.q_bits == 0 else q_bits)
    data = synth.make_layer(shape)
    cfg = tl.oracle_cfg(shape)
    kv = orc.taq_kv(data["ctx"], data["Wk"], data["Wv"], data["mask"], cfg)
    q = orc.taq_q(data["X"], data["Wq"], cfg)
    want = orc.taq_attention(q["Q_tilde"], kv["K_tilde"], kv["V_tilde"], data["mask"], cfg)
    desc = tl.gpu_desc(shape)
    blk = tl.build_kv_block(desc, kv["K_codes"], kv["K_scales"], kv["V_codes"], kv["V_scales"], kv["K_tilde"], kv["V_tilde"], data["mask"])
    tb.taq_dispatch_reset()
    if shape.q_bits == 8:
        qc = orc.merge_heads(q["Q_codes"]).astype(np.int8)
        qs = np.ascontiguousarray(q["Q_scales"].transpose(0, 2, 1)).astype(np.float32)
        o = tb.taq_cross_attention(desc, dev(qc), dev(qs), tb.taq_kv_finalize(desc, dev(blk)), dev(data["mask"]))
    else:
        q16 = orc.merge_heads(q["Q_tilde"]).astype(np.float16)
        o = tb.taq_cross_attention(desc, dev(q16), None, tb.taq_kv_finalize(desc, dev(blk)), dev(data["mask"]))
    tb.taq_poll_device_status()
    counts = tb.taq_dispatch_counts()
    assert counts["attention_tensor"] == 1 and counts["attention_generic"] == 0
    max_abs, rel = tl.assert_layer_close(o.cpu().numpy(), want, "O")
    assert rel < 5e-4
