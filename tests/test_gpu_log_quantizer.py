"""The logarithmic probability quantizer (Table 4's "Logarithmic" rows; the paper does not define it, the reading is
power-of-two codes: code = clamp(rint(-log2 p), 0, 2^bits - 1), p^ = 2^-code) on the GPU against the oracle.

A code is decided by which side of 2^-(k + 1/2) a probability falls on.  The two sides compute the probability with
different exponentials, so a probability within a few float32 ulps of a boundary may take the neighbouring code on
the GPU, which halves or doubles that one p^.  The comparison therefore is: wherever no probability of a (row, head)
is near a boundary the outputs agree to the arithmetic tolerance; where one is, the output may differ by at most what
flipping those codes changes (2^-(k+1) |V~ row|), and such (row, head) pairs stay a small minority."""
from dataclasses import replace

import numpy as np
import pytest

from oracle import taq_oracle as orc
from paper_2603_22943_b200 import binding as tb
from paper_2603_22943_b200 import synth

import taq_testlib as tl
from taq_testlib import dev

pytestmark = pytest.mark.gpu

NEAR = 2e-4            # distance of -log2 p from k + 1/2 below which the code may differ between the two sides
ATOL, RTOL = 4e-3, 2e-3


def _cases():
    c3 = synth.config3_layers()
    return [
        replace(synth.shrink(synth.config2(), 300), seed=41, p_log=1),                                  # d = 40
        replace(synth.shrink(synth.config2(), 200), seed=42, p_log=1, p_bits=4, q_bits=0),
        replace(synth.shrink(c3[5], 200), seed=43, p_log=1),                                            # d = 80: TMA data path
        replace(synth.shrink(c3[5], 130), seed=44, p_log=1, p_bits=4),
        replace(synth.config1(), p_log=1),                                                              # d = 160, W8
        replace(synth.shrink(synth.config4_layers()[0], 130), seed=45, p_log=1),                        # d = 64
        replace(synth.shrink(synth.config2(), 100), seed=46, n_ctx=100, ctx_dim=768, p_log=1),          # T > 80: generic kernel
    ]


@pytest.mark.parametrize("shape", _cases(), ids=lambda s: f"{s.name}_p{s.p_bits}_q{s.q_bits}_T{s.n_ctx}")
def test_attention_with_logarithmic_probabilities(shape):
    data = synth.make_layer(shape)
    cfg = tl.oracle_cfg(shape)
    kv = orc.taq_kv(data["ctx"], data["Wk"], data["Wv"], data["mask"], cfg)
    q = orc.taq_q(data["X"], data["Wq"], cfg)
    want, A, A_hat = orc.taq_attention(q["Q_tilde"], kv["K_tilde"], kv["V_tilde"], data["mask"], cfg, return_probs=True)
    desc = tl.gpu_desc(shape)
    blk = tl.build_kv_block(desc, kv["K_codes"], kv["K_scales"], kv["V_codes"], kv["V_scales"], kv["K_tilde"], kv["V_tilde"], data["mask"])
    if shape.q_bits == 8:
        qc = orc.merge_heads(q["Q_codes"]).astype(np.int8)
        qs = np.ascontiguousarray(q["Q_scales"].transpose(0, 2, 1)).astype(np.float32)
        o = tb.taq_cross_attention(desc, dev(qc), dev(qs), tb.taq_kv_finalize(desc, dev(blk)), dev(data["mask"]))
    else:
        q16 = orc.merge_heads(q["Q_tilde"]).astype(np.float16)
        o = tb.taq_cross_attention(desc, dev(q16), None, tb.taq_kv_finalize(desc, dev(blk)), dev(data["mask"]))
    tb.taq_poll_device_status()
    got = o.cpu().numpy().astype(np.float64)

    cmax = 2 ** shape.p_bits - 1
    with np.errstate(divide="ignore"):
        x = -np.log2(A)                                                     # [B,H,N,T]
    k = np.floor(x)
    near = (np.abs(x - (k + 0.5)) < NEAR) & (x < cmax + 0.5) & ~(np.asarray(data["mask"]) != 0)[:, None, None, :]
    flip = np.where(near, np.exp2(-(k + 1)), 0.0)                           # what the neighbouring code changes p^ by
    extra = orc.merge_heads(np.einsum("bhnt,bhtd->bhnd", flip, np.abs(orc.f16_round(kv["V_tilde"]))))
    diff = np.abs(got - want)
    bound = ATOL + RTOL * np.abs(want) + 1.01 * extra
    bad = diff > bound
    assert not bad.any(), f"{int(bad.sum())} outputs off, worst {diff[bad].max():.3e} at {np.argwhere(bad)[0]}"
    frac_near = float(near.any(axis=-1).mean())
    assert frac_near < 0.05, frac_near                                      # the widened bound is the exception
    # the ordinary columns really are powers of two on the oracle side, and the result is not the linear quantizer's
    lin = orc.taq_attention(q["Q_tilde"], kv["K_tilde"], kv["V_tilde"], data["mask"], replace(cfg, p_log=False))
    assert np.linalg.norm(want - lin) > 20 * np.linalg.norm(got - want)


def test_layer_with_logarithmic_probabilities_runs_as_three_tensor_core_launches():
    shape = replace(synth.shrink(synth.config2(), 400), seed=47, p_log=1)
    data = synth.make_layer(shape)
    tb.taq_dispatch_reset()
    y, parts = tl.gpu_layer(shape, data, return_parts=True)
    counts = tb.taq_dispatch_counts()
    assert counts["layer_fused"] == 0 and counts["query_attention_fused"] == 0
    assert counts["attention_tensor"] == 1 and counts["attention_generic"] == 0 and counts["linear_generic"] == 0
    want = tl.oracle_layer(shape, data)["Y"]
    rel = np.linalg.norm(y.astype(np.float64) - want) / np.linalg.norm(want)
    assert rel < 2e-2, rel                                                  # Q~/K~/V~ code ties and boundary flips included
    y_lin, _ = tl.gpu_layer(replace(shape, p_log=0), data, return_parts=True)
    assert np.linalg.norm(y.astype(np.float64) - y_lin) > 5 * np.linalg.norm(y.astype(np.float64) - want)
