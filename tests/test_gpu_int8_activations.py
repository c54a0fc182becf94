"""Integer-activation projections (a_bits = 8: the W/A reading of Table 1) on the GPU against the oracle.

The per-token quantizer is a stand-alone quantizer: its codes and scales are compared bit for bit.  The integer GEMM is
exact up to the fp32 combination of its per-group sums, so its fp32 output is compared with a tolerance of a few fp32
roundings of the sum of the absolute terms.  The layer pass takes the three-part comparison of the fp16-activation
layer (`taq_testlib.check_layer`) with the oracle switched to a_bits = 8.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from oracle import taq_oracle as orc
from paper_2603_22943_b200 import binding as tb
from paper_2603_22943_b200 import synth

import taq_testlib as tl
from taq_testlib import dev

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,cols", [(1, 8), (77, 768), (300, 320), (130, 1280), (154, 2048), (33, 2056), (5, 4096)])
def test_quantize_rows_f16_is_bit_exact(rows, cols):
    r = np.random.default_rng(rows * 131 + cols)
    x = (r.standard_normal((rows, cols)) * r.uniform(1e-2, 30.0, (rows, 1))).astype(np.float16)
    x[rows // 2] = 0                                      # an all-zero token: scale 0, codes 0
    if rows > 2:
        x[1, :] = np.float16(0.5) * np.sign(x[1, :])      # every element at the row maximum: codes +-127
    if rows > 4 and cols >= 16:                           # exact ties: absmax 127 gives scale 1, half-integers round to even
        x[3, :] = (r.integers(-126, 126, cols) + 0.5).astype(np.float16)
        x[3, 0] = 127
        x[4, :] = (r.integers(-252, 252, cols) * 0.25).astype(np.float16)       # scale 1/2 (absmax 63.5): quarter steps
        x[4, 0] = 63.5
    if rows > 6:
        x[5, :] = (r.integers(-40, 41, cols) * 2.0 ** -24).astype(np.float16)   # subnormal fp16 values: the scale is tiny, not zero
        x[6, :] = np.clip(r.standard_normal(cols) * 3e4, -65504, 65504).astype(np.float16)   # near the top of the fp16 range
    codes, scales = tb.taq_quantize_rows_f16(dev(x))
    want_c, want_s = orc.quantize_rows(x.astype(np.float32), 127)
    assert np.array_equal(scales.cpu().numpy(), want_s)
    assert np.array_equal(codes.cpu().numpy().astype(np.int32), want_c)


LINEAR_CASES = [
    # rows, k_in, n_out, bits, group
    (300, 320, 320, 4, 128),      # ragged last K block (320 = 128 + 128 + 64), five row tiles with a ragged tail
    (154, 768, 320, 4, 128),      # the K/V projection's fan-in
    (64, 1280, 1280, 8, 0),       # W8, one scale per output channel: ten K blocks into one accumulator
    (200, 2048, 640, 4, 128),     # sixteen scale groups: the two TMEM accumulators alternate eight times
    (129, 640, 640, 4, 128),
]


@pytest.mark.parametrize("rows,k_in,n_out,bits,group", LINEAR_CASES)
def test_integer_gemm_equals_the_integer_definition(rows, k_in, n_out, bits, group):
    r = np.random.default_rng(k_in + n_out + rows)
    x = r.standard_normal((rows, k_in)).astype(np.float16)
    x[:, 3] *= 20                                         # an outlier channel, as in the layer inputs
    W = (r.standard_normal((n_out, k_in)) / np.sqrt(k_in)).astype(np.float32)
    b = (0.1 * r.standard_normal(n_out)).astype(np.float32)
    wd = tb.weight_desc(n_out, k_in, bits, group)
    Wp = tb.taq_pack_weights(wd, dev(W), dev(b))
    xc, xs = tb.taq_quantize_rows_f16(dev(x))
    y = tb.taq_quantized_linear_i8(wd, xc, xs, Wp, tb.TAQ_OUT_F32).cpu().numpy().astype(np.float64)
    tb.taq_poll_device_status()
    # the definition, in integers: y = s_x * sum_g s_w[g] * (sum_{k in g} xq wq) + b
    xq, sx = orc.quantize_rows(x.astype(np.float32), 127)
    wq, sw = orc.quantize_weights(W, bits, group)
    g = k_in if group == 0 else group
    want = np.zeros((rows, n_out))
    mag = np.zeros((rows, n_out))
    for gi in range(sw.shape[1]):
        part = xq[:, gi * g:(gi + 1) * g].astype(np.int64) @ wq[:, gi * g:(gi + 1) * g].astype(np.int64).T
        want += part * sw[:, gi].astype(np.float64)[None, :]
        mag += np.abs(part) * sw[:, gi].astype(np.float64)[None, :]
    want = want * sx.astype(np.float64)[:, None] + b
    mag = mag * sx.astype(np.float64)[:, None] + np.abs(b)
    assert np.all(np.abs(y - want) <= 4e-7 * (sw.shape[1] + 3) * mag + 1e-30)
    # and it is what the oracle's a_bits = 8 projection computes
    cfg = orc.TaqConfig(heads=1, w_bits=bits, w_group=group, a_bits=8, contract=False)
    np.testing.assert_allclose(want, orc.taq_out(x[None], W, b, cfg)[0], rtol=1e-12, atol=1e-12)


def test_integer_gemm_rejects_what_the_kernel_does_not_cover():
    wd = tb.weight_desc(320, 320, 4, 64)                  # scale groups of 64: not one K block of the int8 kernel
    z = torch.zeros(320 * 320, dtype=torch.uint8, device="cuda")
    with pytest.raises(tb.TaqError) as e:
        tb.taq_quantized_linear_i8(wd, z.view(torch.int8)[: 16 * 320], z.view(torch.float32)[:16], z, tb.TAQ_OUT_F16)
    assert e.value.status == tb.TAQ_ERR_UNSUPPORTED


def _layer_cases():
    c3 = synth.config3_layers()
    return [
        replace(synth.shrink(synth.config2(), 700), seed=21),           # C = 320, d = 40, W4: ragged K blocks
        replace(synth.shrink(c3[5], 300), seed=22),                     # C = 640, d = 80
        replace(synth.shrink(c3[10], 200), seed=23),                    # C = 1280, d = 160
        synth.config1(),                                                # W8, one sequence of 64 tokens
        replace(synth.shrink(synth.config4_layers()[0], 260), seed=24), # SDXL: d = 64, Dc = 2048, three trigger tokens
    ]


@pytest.mark.parametrize("shape", _layer_cases(), ids=lambda s: s.name)
def test_layer_forward_a8_matches_the_oracle(shape):
    data = synth.make_layer(shape)
    desc = tl.gpu_desc(shape)
    P = tl.pack_layer_weights(shape, data)
    mask = dev(data["mask"])
    kv = tb.taq_kv_project_a8(desc, dev(data["ctx"]), P["Wk"], P["Wv"], mask)
    y = tb.taq_layer_forward_a8(desc, dev(data["X"]), P["Wq"], P["Wout"], kv, mask)
    tb.taq_poll_device_status()
    torch.cuda.synchronize()
    y = y.cpu().numpy()
    assert np.isfinite(y).all()
    res = tl.check_layer(shape, data, y, {"desc": desc, "packed": P, "kv": kv, "mask": mask}, a_bits=8)
    assert res["rows_with_q_flip"] <= 0.05 * res["rows"] + 1, res   # (measured: at most 2.8 % of the rows)
    # the integer path is a different quantized network from the fp16-activation one, not a copy of it
    y16 = tl.gpu_layer(shape, data)
    assert tl.errors(y, y16)[1] > 1e-3, res


def test_a8_pass_is_deterministic_and_stays_inside_its_buffers():
    shape = replace(synth.shrink(synth.config2(), 333), seed=25)          # 2.6 row tiles per sequence
    data = synth.make_layer(shape)
    desc = tl.gpu_desc(shape)
    P = tl.pack_layer_weights(shape, data)
    mask = dev(data["mask"])
    guard = 1024
    kvn = tb.taq_kv_bytes(desc)
    kvbuf = torch.full((kvn + 2 * guard,), 0x5A, dtype=torch.uint8, device="cuda")
    wkn = tb.lib().taq_kv_project_a8_workspace_bytes(tb.C.byref(desc))
    wkbuf = torch.full((wkn + 2 * guard,), 0x5A, dtype=torch.uint8, device="cuda")
    tb.taq_kv_project_a8(desc, dev(data["ctx"]), P["Wk"], P["Wv"], mask, kvbuf[guard: guard + kvn], wkbuf[guard: guard + wkn])
    n = shape.rows * shape.channels
    ybuf = torch.full((n + 2 * guard,), -7.0, dtype=torch.float16, device="cuda")
    wsn = tb.taq_workspace_bytes_a8(desc)
    wsbuf = torch.full((wsn + 2 * guard,), 0x5A, dtype=torch.uint8, device="cuda")
    x = dev(data["X"])
    outs = []
    for _ in range(2):
        tb.taq_layer_forward_a8(desc, x, P["Wq"], P["Wout"], kvbuf[guard: guard + kvn], mask, ybuf[guard: guard + n], wsbuf[guard: guard + wsn])
        torch.cuda.synchronize()
        outs.append(ybuf.cpu().numpy().copy())
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))
    assert np.all(outs[0][:guard] == -7.0) and np.all(outs[0][-guard:] == -7.0)
    for buf in (kvbuf, wkbuf, wsbuf):
        b = buf.cpu().numpy()
        assert np.all(b[:guard] == 0x5A) and np.all(b[-guard:] == 0x5A)
    tb.taq_poll_device_status()


def test_a8_empty_inputs_and_bad_arguments():
    shape = synth.shrink(synth.config2(), 64)
    desc0 = tl.gpu_desc(shape, n_query=0)
    z = torch.zeros(256, dtype=torch.uint8, device="cuda")
    assert tb.taq_layer_forward_a8(desc0, z, z, z, z, z, y=z, workspace=z) is z          # nothing to do, nothing launched
    desc = tl.gpu_desc(shape)
    with pytest.raises(tb.TaqError) as e:                                                 # workspace too small
        tb.taq_layer_forward_a8(desc, z, z, z, z, z, y=z, workspace=z)
    assert e.value.status == tb.TAQ_ERR_BUFFER_TOO_SMALL
    with pytest.raises(tb.TaqError) as e:                                                 # columns not a multiple of 8
        tb.lib().taq_quantize_rows_f16.restype = tb.C.c_int
        tb._check(tb.lib().taq_quantize_rows_f16(z.data_ptr(), 4, 12, z.data_ptr(), z.data_ptr(), None))
    assert e.value.status == tb.TAQ_ERR_SHAPE


@pytest.mark.parametrize("n,q_bits", [(4096, 8), (333, 8), (130, 0)])
def test_one_kernel_a8_layer_equals_the_step_by_step_composition(n, q_bits):
    """At C = 320 / 8 heads / W4 g128 the integer-activation pass is one kernel (Q_a of X and O inside the CTA).  The same
    pass composed from the stand-alone entry points - quantize, integer to_q, attention, quantize, integer to_out - gives
    the same Y up to probability codes on a rounding tie: the per-token codes are the stand-alone quantizer's and the
    integer products are exact, but the two attention kernels add a row's exponentials in different orders, so a
    probability on a rounding boundary may take the neighbouring code (1/255 of one value row, then the O quantizer's
    step)."""
    shape = replace(synth.shrink(synth.config2(), n), seed=26, q_bits=q_bits)
    data = synth.make_layer(shape)
    desc = tl.gpu_desc(shape)
    P = tl.pack_layer_weights(shape, data)
    mask = dev(data["mask"])
    kv = tb.taq_kv_project_a8(desc, dev(data["ctx"]), P["Wk"], P["Wv"], mask)
    x = dev(data["X"])
    y = tb.taq_layer_forward_a8(desc, x, P["Wq"], P["Wout"], kv, mask)
    M, C_, H = shape.rows, shape.channels, shape.heads
    xc, xs = tb.taq_quantize_rows_f16(x.view(M, C_))
    if q_bits == 8:
        qc, qs = tb.taq_quantized_linear_i8(P["wd_cc"], xc, xs, P["Wq"], tb.TAQ_OUT_INT8_HEAD_ROWS, heads=H)
    else:
        qc, qs = tb.taq_quantized_linear_i8(P["wd_cc"], xc, xs, P["Wq"], tb.TAQ_OUT_F16), None
    o = tb.taq_cross_attention(desc, qc, qs, kv, mask)
    oc, os_ = tb.taq_quantize_rows_f16(o.view(M, C_))
    want = tb.taq_quantized_linear_i8(P["wd_cc"], oc, os_, P["Wout"], tb.TAQ_OUT_F16)
    tb.taq_poll_device_status()
    tl.assert_same_up_to_code_ties(y.view(M, C_), want, "Y")
