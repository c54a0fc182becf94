"""Bit-exact parity of the stand-alone quantizers (activation rows, weight packing) with the CPU oracle."""
import numpy as np
import pytest
import torch

from oracle import taq_oracle as orc
from paper_2603_22943_b200 import binding as tb
from paper_2603_22943_b200 import synth
from taq_testlib import dev

pytestmark = pytest.mark.gpu


def _check_rows(x: np.ndarray, qmax=127):
    codes, scales = tb.taq_quantize_rows(dev(x), qmax)
    torch.cuda.synchronize()
    want_c, want_s = orc.quantize_rows(x, qmax)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), want_s.view(np.uint32)), "scales differ in some bit"
    assert np.array_equal(codes.cpu().numpy().astype(np.int32), want_c), "integer codes differ"


@pytest.mark.parametrize("cfg", ["config1", "config2"])
def test_quantize_rows_on_config_tensors(cfg):
    """The un-rounded fp32 hidden states (with x20 outlier channels) and context of configs 1 and 2, quantized
    per (token, head) row exactly as Q_a does inside the layer."""
    shape = synth.config1() if cfg == "config1" else synth.config2()
    data = synth.make_layer(shape, keep_f32=True)
    d = shape.d_head
    _check_rows(data["X_f32"].reshape(-1, d))
    _check_rows(data["ctx_f32"].reshape(-1, shape.ctx_dim))
    _check_rows(data["X_f32"].reshape(-1, shape.channels))


@pytest.mark.parametrize("cols", [1, 3, 8, 40, 77, 160, 1001])
def test_quantize_rows_shapes_and_adversarial_values(cols):
    r = np.random.default_rng(cols)
    rows = 257                                              # not a multiple of the 8 rows a CTA takes
    x = (r.standard_normal((rows, cols)) * np.exp(r.uniform(-30, 30, (rows, 1)))).astype(np.float32)
    x[0] = 0                                                # all-zero row: scale 0, codes 0
    x[1] = np.float32(1e-41)                                # subnormal row
    x[2, :] = np.float32(3.0e38)                            # near the top of the range
    if cols >= 8:
        x[3, :8] = [127, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 63.5]     # exact ties (scale 1)
        x[3, 8:] = 0
        # values that sit on a rounding boundary after division by the scale
        x[4] = (np.arange(cols) % 255 - 127).astype(np.float32) * np.float32(0.37) + np.float32(0.185)
    _check_rows(x)
    _check_rows(x, qmax=7)


def test_quantize_rows_many_random_values():
    r = np.random.default_rng(123)
    x = r.standard_normal((1 << 16, 160)).astype(np.float32)          # 1e7 values
    _check_rows(x)
    x = (r.standard_normal((1 << 14, 40)) * 20).astype(np.float32)
    _check_rows(x)


@pytest.mark.parametrize("part", range(10))
def test_quantize_rows_1e8_values(part):
    """The kernel multiplies by a reciprocal and falls back to the division of the definition only where the two could
    round differently; that shortcut is allowed only if the codes stay bit-exact on a large sample.  Ten parts of 1.05e7
    fp32 values each (1.05e8 in all): Gaussian rows of the widths the layers use, heavy tails, and rows built to sit on
    rounding boundaries (values (k + 1/2) s +- one ulp for the row's own scale s)."""
    r = np.random.default_rng(1000 + part)
    rows, cols = 1 << 16, 160
    if part < 4:
        x = (r.standard_normal((rows, cols)) * r.uniform(1e-3, 50.0, (rows, 1))).astype(np.float32)
    elif part < 6:
        x = r.standard_cauchy((rows, cols)).astype(np.float32)
    elif part < 8:                                           # values at and next to the rounding boundaries of the row's own grid
        amax = r.uniform(0.5, 200.0, (rows, 1)).astype(np.float32)
        s = (amax / np.float32(127.0)).astype(np.float32)
        k = r.integers(-126, 126, (rows, cols)).astype(np.float32)
        x = ((k + np.float32(0.5)) * s).astype(np.float32)
        x = np.nextafter(x, np.where(r.integers(0, 3, x.shape) == 0, -np.inf, np.where(r.integers(0, 2, x.shape) == 0, np.inf, x)).astype(np.float32))
        x[:, 0] = amax[:, 0]
    else:                                                    # fp16-valued data (as the layer inputs are), where exact ties are common
        x = (r.standard_normal((rows, cols)) * r.uniform(0.1, 30.0, (rows, 1))).astype(np.float16).astype(np.float32)
    _check_rows(x)


@pytest.mark.parametrize("part", range(4))
def test_quantize_rows_f16_every_finite_value_for_1024_row_maxima(part):
    """The per-token quantizer of fp16 data, exhaustively: every finite fp16 value as an element of a row, for 1024
    different row maxima (random ones, powers of two, the largest and smallest fp16 numbers).  Elements larger than the
    row's maximum are replaced by it, so that the maximum is what it is meant to be."""
    allv = np.arange(0, 1 << 16, dtype=np.uint16).view(np.float16)
    allv = allv[np.isfinite(allv)]                           # 63488 values (both zeros, subnormals included)
    assert allv.size == 63488 and allv.size % 8 == 0
    r = np.random.default_rng(77 + part)
    rows = 256
    m = np.abs((r.standard_normal(rows) * r.uniform(1e-3, 1e3, rows)).astype(np.float16))
    m[:8] = np.array([65504, 6.1e-5, 5.96e-8, 1.0, 127.0, 63.5, 0.5, 2.0 ** -14], dtype=np.float16)[:8] if part == 0 else m[:8]
    m = np.where(m == 0, np.float16(1.0), m)
    x = np.where(np.abs(allv)[None, :] <= m[:, None], allv[None, :], m[:, None]).astype(np.float16)
    codes, scales = tb.taq_quantize_rows_f16(dev(x))
    want_c, want_s = orc.quantize_rows(x.astype(np.float32), 127)
    assert np.array_equal(scales.cpu().numpy(), want_s)
    got = codes.cpu().numpy()
    assert np.array_equal(got, want_c.astype(np.int8)), f"{int((got != want_c).sum())} codes differ"


@pytest.mark.parametrize("n_out,k_in,bits,group", [
    (320, 320, 4, 128),      # config 2 to_q / to_out: ragged last group of 64
    (320, 768, 4, 128),      # config 2 to_k / to_v
    (1280, 1280, 8, 0),      # config 1 to_q
    (1280, 768, 8, 0),
    (640, 2048, 4, 128),     # SDXL to_k
    (16, 64, 4, 0), (16, 64, 4, 32), (8, 8, 4, 0), (3, 40, 8, 0),
])
def test_pack_weights_codes_bit_exact(n_out, k_in, bits, group):
    r = np.random.default_rng(n_out * 7 + k_in)
    W = (r.standard_normal((n_out, k_in)) / np.sqrt(k_in)).astype(np.float32)
    W[0, : min(8, k_in)] = 0                                # part of a group all zero
    if n_out > 2:
        W[2] = 0                                            # a whole channel zero
    bias = r.standard_normal(n_out).astype(np.float32)
    d = tb.weight_desc(n_out, k_in, bits, group)
    blob = tb.taq_pack_weights(d, dev(W), dev(bias))
    codes, scales = tb.taq_unpack_weights(d, blob)
    torch.cuda.synchronize()
    want_c, want_s = orc.quantize_weights(W, bits, group)
    assert np.array_equal(codes.cpu().numpy().astype(np.int32), want_c)
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), want_s.view(np.uint32))
    # blob header and bias section, as documented in the header file
    raw = blob.cpu().numpy()
    hdr = raw[:32].view(np.uint32)
    assert hdr[0] == 0x57514154 and list(hdr[1:7]) == [1, n_out, k_in, bits, group, want_s.shape[1]] and hdr[7] == 1
    offs = raw[32:64].view(np.uint64)
    assert offs[3] == raw.size == tb.taq_packed_weight_bytes(d)
    assert np.array_equal(raw[int(offs[2]): int(offs[2]) + 4 * n_out].view(np.float32), bias)
    if bits == 4:   # eight codes per little-endian word: even fan-in indices in nibbles 0..3, odd ones in nibbles 4..7, code + 8
        words = raw[int(offs[0]): int(offs[0]) + k_in // 2].view(np.uint32).astype(np.int64)
        for e in range(8):
            pos = (e >> 1) + ((e & 1) << 2)
            assert np.array_equal(((words >> (4 * pos)) & 0xF).astype(np.int32) - 8, want_c[0, e::8])


def test_pack_is_deterministic_and_respects_buffer_bounds():
    r = np.random.default_rng(5)
    W = r.standard_normal((64, 256)).astype(np.float32)
    d = tb.weight_desc(64, 256, 4, 128)
    n = tb.taq_packed_weight_bytes(d)
    guard = 256
    buf = torch.full((n + 2 * guard,), 0xAB, dtype=torch.uint8, device="cuda")
    tb.taq_pack_weights(d, dev(W), None, buf[guard: guard + n])
    a = buf.cpu().numpy().copy()
    tb.taq_pack_weights(d, dev(W), None, buf[guard: guard + n])
    torch.cuda.synchronize()
    assert np.array_equal(a, buf.cpu().numpy())
    assert np.all(a[:guard] == 0xAB) and np.all(a[-guard:] == 0xAB)
