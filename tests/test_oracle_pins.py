"""Pins for the CPU oracle: everything here runs without a GPU and compares the oracle with something
other than itself - values worked out by hand, exact rational arithmetic, closed forms, a textbook
attention from another library (torch, float64), a separately written uniform-quantized attention,
and a brute-force evaluation of Eq. 2-3 with the 0/1 masks multiplied in as the paper writes them.
The last test plants mistakes in a copy of the oracle and checks that the pins notice each one.
"""
import math
import os
import types
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import taq_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed=0):
    return np.random.default_rng(seed)


def _tiny_layer(seed, B=2, N=5, H=2, d=8, T=7, Dc=16):
    r = _rng(seed)
    C = H * d
    X = r.standard_normal((B, N, C)).astype(np.float16)
    ctx = r.standard_normal((B, T, Dc)).astype(np.float16)
    Wq = (r.standard_normal((C, C)) / math.sqrt(C)).astype(np.float32)
    Wk = (r.standard_normal((C, Dc)) / math.sqrt(Dc)).astype(np.float32)
    Wv = (r.standard_normal((C, Dc)) / math.sqrt(Dc)).astype(np.float32)
    Wo = (r.standard_normal((C, C)) / math.sqrt(C)).astype(np.float32)
    bo = (0.1 * r.standard_normal(C)).astype(np.float32)
    return X, ctx, Wq, Wk, Wv, Wo, bo


# ---------------------------------------------------------------------------------------------
# Quantizer
# ---------------------------------------------------------------------------------------------

def check_quantizer_hand_values(o):
    # absmax 127 -> scale exactly 1; ties go to the even integer; clamp is symmetric.
    x = np.array([[127.0, 0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 3.49, -126.5, 0.0]], dtype=np.float32)
    q, s = o.quantize_rows(x, 127)
    assert s[0] == np.float32(1.0)
    assert q[0].tolist() == [127, 0, 2, 2, 0, -2, -2, 3, -126, 0]
    # 4-bit: absmax 7 -> scale 1.
    x4 = np.array([[7.0, -3.5, 1.0, 0.0, 2.5, -7.0]], dtype=np.float32)
    q4, s4 = o.quantize_rows(x4, 7)
    assert s4[0] == np.float32(1.0) and q4[0].tolist() == [7, -4, 1, 0, 2, -7]
    # all-zero row
    qz, sz = o.quantize_rows(np.zeros((1, 6), np.float32), 127)
    assert sz[0] == 0 and not qz.any()
    assert not o.dequantize_rows(qz, sz).any()


def check_quantizer_exact_rational(o):
    """code must be the integer nearest to fl32(x / s), s = fl32(absmax/127), checked with exact
    rational arithmetic: fl32(x/s) is within half an ulp of the true quotient."""
    r = _rng(1)
    x = (r.standard_normal((64, 40)) * r.uniform(1e-3, 1e3, (64, 1))).astype(np.float32)
    q, s = o.quantize_rows(x, 127)
    for i in range(x.shape[0]):
        a = Fraction(float(np.max(np.abs(x[i]))))
        s_true = a / 127
        assert abs(Fraction(float(s[i])) - s_true) <= s_true * Fraction(1, 2 ** 24)     # one fp32 rounding
        for j in range(x.shape[1]):
            quo = Fraction(float(x[i, j])) / Fraction(float(s[i]))
            assert abs(Fraction(int(q[i, j])) - quo) <= Fraction(1, 2) + abs(quo) * Fraction(1, 2 ** 23)
    assert np.all(np.max(np.abs(q), axis=-1) == 127)
    xh = o.dequantize_rows(q, s)
    assert np.all(np.abs(x - xh) <= s[:, None] * np.float32(0.5000001))


def check_quantizer_idempotent_and_pow2(o):
    r = _rng(2)
    x = r.standard_normal((128, 160)).astype(np.float32)
    for qmax in (127, 7):
        q, s = o.quantize_rows(x, qmax)
        xh = o.dequantize_rows(q, s)
        q2, s2 = o.quantize_rows(xh, qmax)                 # scale recomputed from x^
        assert np.array_equal(q, q2)
        assert np.array_equal(s, s2)                       # max|code| = qmax, so absmax(x^) = qmax*s
        for k in (-9, 5):
            qk, sk = o.quantize_rows(x * np.float32(2.0 ** k), qmax)
            assert np.array_equal(q, qk) and np.array_equal(sk, s * np.float32(2.0 ** k))


def check_weight_quantizer(o):
    r = _rng(3)
    W = r.standard_normal((6, 320)).astype(np.float32)
    q, s = o.quantize_weights(W, 4, 128)
    assert s.shape == (6, 3) and q.min() >= -7 and q.max() <= 7
    for g, (lo, hi) in enumerate([(0, 128), (128, 256), (256, 320)]):      # ragged last group of 64
        np.testing.assert_array_equal(s[:, g], (np.max(np.abs(W[:, lo:hi]), axis=1) / np.float32(7)).astype(np.float32))
        assert np.all(np.max(np.abs(q[:, lo:hi]), axis=1) == 7)
    q8, s8 = o.quantize_weights(W, 8, 0)
    assert s8.shape == (6, 1) and np.all(np.max(np.abs(q8), axis=1) == 127)
    # hand example, scale exactly 1 in both groups
    Wh = np.zeros((1, 256), np.float32)
    Wh[0, :4] = [7, -3.5, 2.5, 1.49]
    Wh[0, 128:131] = [-7, 6.5, 0.5]
    qh, sh = o.quantize_weights(Wh, 4, 128)
    assert sh.tolist() == [[1.0, 1.0]]
    assert qh[0, :4].tolist() == [7, -4, 2, 1] and qh[0, 128:131].tolist() == [-7, 6, 0]
    # dequantization: the exact product in both modes
    wi = o.dequantize_weights(q, s, 128, contract=False)
    wc = o.dequantize_weights(q, s, 128, contract=True)
    np.testing.assert_array_equal(wi[:, 130], q[:, 130].astype(np.float64) * s[:, 1].astype(np.float64))
    np.testing.assert_array_equal(wc, wi)
    assert np.all(np.abs(W - wi) <= np.repeat(s, 128, axis=1)[:, :320] * 0.5000001)
    with pytest.raises(ValueError):
        o.quantize_weights(W, 3, 0)


def check_prob_quantizer(o):
    p = np.array([0.0, 1.0, 0.5 / 255, 1.5 / 255, 2.5 / 255, 1 / 77, 0.999, 100.4 / 255, 100.6 / 255])
    code, ph = o.quantize_prob(p)
    # (2k+1)/510 ties: 0.5/255 and 2.5/255 are not exactly representable, so only the sure ones are pinned
    assert code[[0, 1, 5, 7, 8]].tolist() == [0, 255, 3, 100, 101]
    r = _rng(4)
    A = r.dirichlet(np.ones(77), size=200)
    code, Ah = o.quantize_prob(A)
    assert code.min() >= 0 and code.max() <= 255
    assert np.all(np.abs(Ah - A) <= 1 / 510 + 1e-7)
    assert np.all(np.abs(Ah.sum(-1) - 1) <= 77 / 510 + 1e-6)
    np.testing.assert_allclose(Ah, code / 255.0, rtol=0, atol=1e-7)


def check_log_prob_quantizer(o):
    """The logarithmic reading (power-of-two codes; the paper does not define it, so these are closed forms of the
    reading, not of the paper): exact powers of two are fixed points, the decision boundary between codes k and k + 1
    is 2^-(k + 1/2), the last code absorbs everything below, and inside a layer the trigger columns bypass it."""
    p = np.array([1.0, 0.5, 0.25, 2.0 ** -7, 2.0 ** -15, 2.0 ** -40, 0.0])
    c8, h8 = o.quantize_prob_log(p, 8)
    assert c8.tolist() == [0, 1, 2, 7, 15, 40, 255] and h8[:6].tolist() == p[:6].tolist()
    c4, h4 = o.quantize_prob_log(p, 4)
    assert c4.tolist() == [0, 1, 2, 7, 15, 15, 15] and h4[-1] == 2.0 ** -15
    for k in range(6):                                            # just above / below the boundary 2^-(k + 1/2)
        b = 2.0 ** -(k + 0.5)
        c, _ = o.quantize_prob_log(np.array([b * 1.001, b * 0.999]), 8)
        assert c.tolist() == [k, k + 1]
    A = _rng(9).dirichlet(np.ones(77), size=300)
    c, Ah = o.quantize_prob_log(A, 8)
    assert np.all(Ah / A <= 2 ** 0.5 * (1 + 1e-6)) and np.all(Ah / A >= 2 ** -0.5 * (1 - 1e-6))   # within half an octave
    assert np.all(np.log2(Ah) == -c)
    # inside the layer: ordinary columns take the power-of-two value, trigger columns the fp16 probability
    X, ctx, Wq, Wk, Wv, Wo, bo = _tiny_layer(12)
    mask = np.zeros((2, 7), np.uint8)
    mask[:, 2] = 1
    cfg = o.TaqConfig(heads=2, w_bits=0, q_bits=0, kv_bits=0, p_bits=8, p_log=True, contract=False)
    q = o.taq_q(X, Wq, cfg)
    kv = o.taq_kv(ctx, Wk, Wv, mask, cfg)
    _, A0, Ahat = o.taq_attention(q["Q_tilde"], kv["K_tilde"], kv["V_tilde"], mask, cfg, return_probs=True)
    np.testing.assert_array_equal(Ahat[..., 2], A0[..., 2])
    rest = np.delete(Ahat, 2, axis=-1)
    assert np.all(np.log2(rest) == np.rint(np.log2(rest)))
    want = np.exp2(-np.clip(np.rint(-np.log2(np.delete(A0, 2, axis=-1).astype(np.float32))), 0, 255))
    np.testing.assert_array_equal(rest, want)


@pytest.mark.parametrize("check", [check_quantizer_hand_values, check_quantizer_exact_rational,
                                   check_quantizer_idempotent_and_pow2, check_weight_quantizer, check_prob_quantizer,
                                   check_log_prob_quantizer])
def test_quantizers(check):
    check(orc)


# ---------------------------------------------------------------------------------------------
# Whole-layer pins
# ---------------------------------------------------------------------------------------------

def _torch_attention(X, ctx, Wq, Wk, Wv, Wo, bo, H):
    """Textbook multi-head cross-attention in float64 with torch (another library, other code)."""
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    X, ctx, Wq, Wk, Wv, Wo, bo = map(t, (X, ctx, Wq, Wk, Wv, Wo, bo))
    B, N, C = X.shape
    d = C // H
    q = torch.nn.functional.linear(X, Wq).view(B, N, H, d).transpose(1, 2)
    k = torch.nn.functional.linear(ctx, Wk).view(B, -1, H, d).transpose(1, 2)
    v = torch.nn.functional.linear(ctx, Wv).view(B, -1, H, d).transpose(1, 2)
    o = torch.nn.functional.scaled_dot_product_attention(q, k, v)
    o = o.transpose(1, 2).reshape(B, N, C)
    return torch.nn.functional.linear(o, Wo, bo).numpy()


def check_all_trigger_is_textbook_attention(o):
    X, ctx, Wq, Wk, Wv, Wo, bo = _tiny_layer(10, B=2, N=9, H=3, d=8, T=11, Dc=24)
    cfg = o.TaqConfig(heads=3, w_bits=0, q_bits=0, contract=False)
    mask = np.ones((2, 11), np.uint8)
    got = o.taq_layer(X, ctx, Wq, Wk, Wv, Wo, bo, mask, cfg)["Y"]
    want = _torch_attention(X, ctx, Wq, Wk, Wv, Wo, bo, 3)
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)


def _uniform_quantized_attention(X, ctx, Wq_hat, Wk_hat, Wv_hat, Wo_hat, bo, H):
    """Uniformly quantized cross-attention (no token is special), written on its own with torch:
    every K/V/Q row int8, every probability uint8.  Takes already-dequantized weights."""
    t = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))

    def q8(z):                                                # z: [..., d] float64 tensor
        z32 = z.to(torch.float32)
        s = z32.abs().amax(dim=-1, keepdim=True) / torch.tensor(127.0, dtype=torch.float32)
        code = torch.round(z32 / torch.where(s == 0, torch.ones_like(s), s)).clamp(-127, 127)
        return (code * s).to(torch.float64)

    X, ctx, bo = t(X), t(ctx), t(bo)
    B, N, C = X.shape
    d = C // H
    Y = torch.zeros(B, N, C, dtype=torch.float64)
    O = torch.zeros(B, N, C, dtype=torch.float64)
    for b in range(B):
        Q = X[b] @ t(Wq_hat).T
        K = ctx[b] @ t(Wk_hat).T
        V = ctx[b] @ t(Wv_hat).T
        for h in range(H):
            sl = slice(h * d, (h + 1) * d)
            Qh, Kh, Vh = q8(Q[:, sl]), q8(K[:, sl]), q8(V[:, sl])
            A = torch.softmax(Qh @ Kh.T / math.sqrt(d), dim=-1)
            code = torch.round(A.to(torch.float32) * torch.tensor(255.0, dtype=torch.float32))
            Ah = (code / torch.tensor(255.0, dtype=torch.float32)).to(torch.float64)
            O[b, :, sl] = Ah @ Vh
        Y[b] = O[b] @ t(Wo_hat).T + bo
    return Y.numpy(), O.numpy()


def check_empty_mask_is_uniform_quantization(o):
    X, ctx, Wq, Wk, Wv, Wo, bo = _tiny_layer(11, B=2, N=17, H=2, d=8, T=13, Dc=32)
    for bits, group in ((8, 0), (4, 8)):
        cfg = o.TaqConfig(heads=2, w_bits=bits, w_group=group, q_bits=8, contract=False)
        deq = lambda W: o.dequantize_weights(*o.quantize_weights(W, bits, group), group, contract=False)
        got = o.taq_layer(X, ctx, Wq, Wk, Wv, Wo, bo, np.zeros((2, 13), np.uint8), cfg)
        wantY, wantO = _uniform_quantized_attention(X, ctx, deq(Wq), deq(Wk), deq(Wv), deq(Wo), bo, 2)
        np.testing.assert_allclose(got["O"], wantO, rtol=0, atol=1e-9)
        np.testing.assert_allclose(got["Y"], wantY, rtol=0, atol=1e-9)


def check_trigger_rows_pass_through(o):
    X, ctx, Wq, Wk, Wv, Wo, bo = _tiny_layer(12, B=2, N=4, H=2, d=8, T=9, Dc=16)
    mask = np.zeros((2, 9), np.uint8)
    mask[0, [2, 3]] = 1
    mask[1, [5]] = 1
    for contract in (False, True):
        cfg = o.TaqConfig(heads=2, w_bits=8, contract=contract)
        kv = o.taq_kv(ctx, Wk, Wv, mask, cfg)
        for nm in ("K", "V"):
            Z, Zt = kv[nm], kv[nm + "_tilde"]
            ref = Z.astype(np.float16).astype(np.float64) if contract else Z
            for b in range(2):
                for j in range(9):
                    if mask[b, j]:
                        assert np.array_equal(Zt[b, :, j], ref[b, :, j])          # bit-unchanged
                    else:
                        deq = kv[nm + "_codes"][b, :, j].astype(np.float32) * kv[nm + "_scales"][b, :, j, None]
                        assert np.array_equal(Zt[b, :, j], deq.astype(np.float64))
                        assert not np.array_equal(Zt[b, :, j], Z[b, :, j])
    # probability columns: trigger columns equal A, others are multiples of 1/255
    cfg = o.TaqConfig(heads=2, w_bits=8, contract=False)
    kv = o.taq_kv(ctx, Wk, Wv, mask, cfg)
    q = o.taq_q(X, Wq, cfg)
    _, A, Ah = o.taq_attention(q["Q_tilde"], kv["K_tilde"], kv["V_tilde"], mask, cfg, return_probs=True)
    for b in range(2):
        for j in range(9):
            if mask[b, j]:
                assert np.array_equal(Ah[b, :, :, j], A[b, :, :, j])
            else:
                codes = Ah[b, :, :, j] * 255.0
                assert np.all(np.abs(codes - np.rint(codes)) < 1e-4)
                assert np.all(np.abs(Ah[b, :, :, j] - A[b, :, :, j]) <= 1 / 510 + 1e-7)
    np.testing.assert_allclose(A.sum(-1), 1.0, atol=1e-12)


def check_closed_forms(o):
    r = _rng(13)
    H, d = 2, 8
    C = H * d
    cfg = o.TaqConfig(heads=H, contract=False)
    # (i) zero queries -> uniform attention 1/T.  T = 77: rint(255/77) = 3.
    T = 77
    Kt = r.standard_normal((1, H, T, d))
    Vt = r.standard_normal((1, H, T, d))
    Q0 = np.zeros((1, H, 3, d))
    mask = np.zeros((1, T), np.uint8)
    mask[0, [4, 5]] = 1
    O = o.taq_attention(Q0, Kt, Vt, mask, cfg)
    nt = np.ones(T, bool)
    nt[[4, 5]] = False
    want = (Vt[0][:, ~nt].sum(1) / 77.0 + Vt[0][:, nt].sum(1) * (3.0 / 255.0))      # [H, d]
    np.testing.assert_allclose(O[0, 0].reshape(H, d), want, rtol=0, atol=1e-7)
    # T divides 255 -> the uniform row is represented exactly; empty mask gives the mean of the V rows
    for T in (3, 5, 15, 17):
        Vt = r.standard_normal((1, H, T, d))
        O = o.taq_attention(np.zeros((1, H, 2, d)), r.standard_normal((1, H, T, d)), Vt, np.zeros((1, T), np.uint8), cfg)
        np.testing.assert_allclose(O[0, 1].reshape(H, d), Vt[0].mean(1), rtol=0, atol=1e-7)
    # (ii) a single key: A = 1, O is that V row whatever Q is
    Vt = r.standard_normal((1, H, 1, d))
    O = o.taq_attention(r.standard_normal((1, H, 4, d)), r.standard_normal((1, H, 1, d)), Vt, np.zeros((1, 1), np.uint8), cfg)
    np.testing.assert_allclose(O[0, 2].reshape(H, d), Vt[0, :, 0], rtol=0, atol=1e-7)
    # (iii) one key far above the rest (logit gap >= 40): O is that key's V row, masked or not
    T = 6
    Kt = np.zeros((1, H, T, d))
    Kt[0, :, 2, 0] = 200.0
    Qd = np.zeros((1, H, 2, d))
    Qd[..., 0] = 1.0                                                # logit of key 2 = 200/sqrt(8) = 70.7
    Vt = r.standard_normal((1, H, T, d))
    for trig in ([], [2], [0]):
        m = np.zeros((1, T), np.uint8)
        m[0, trig] = 1
        O = o.taq_attention(Qd, Kt, Vt, m, cfg)
        np.testing.assert_allclose(O[0, 0].reshape(H, d), Vt[0, :, 2], rtol=0, atol=1e-9)
    # (iv) all V rows equal to v, empty mask -> O = (sum of codes / 255) v
    T = 9
    v = r.standard_normal((H, d))
    Vt = np.broadcast_to(v[None, :, None, :], (1, H, T, d)).copy()
    Qr, Kr = r.standard_normal((1, H, 3, d)), r.standard_normal((1, H, T, d))
    O, A, Ah = o.taq_attention(Qr, Kr, Vt, np.zeros((1, T), np.uint8), cfg, return_probs=True)
    codes = np.rint(A.astype(np.float32) * np.float32(255))
    np.testing.assert_allclose(O[0].reshape(3, H, d), (codes.sum(-1)[0].T / 255.0)[:, :, None] * v[None], atol=1e-7, rtol=0)
    # softmax scale is sqrt(d), d = head width: two keys, logits (x, 0) -> p = sigmoid(x)
    d1 = 16
    cfg1 = o.TaqConfig(heads=1, contract=False, p_bits=0)
    Qs = np.zeros((1, 1, 1, d1))
    Qs[..., 0] = 4.0
    Ks = np.zeros((1, 1, 2, d1))
    Ks[0, 0, 0, 0] = 2.0                                            # logit 8/sqrt(16) = 2
    Vs = np.zeros((1, 1, 2, d1))
    Vs[0, 0, 0, :] = 1.0
    O = o.taq_attention(Qs, Ks, Vs, np.zeros((1, 2), np.uint8), cfg1)
    np.testing.assert_allclose(O[0, 0], 1.0 / (1.0 + math.exp(-2.0)), atol=1e-12, rtol=0)


def check_structure(o):
    X, ctx, Wq, Wk, Wv, Wo, bo = _tiny_layer(14, B=2, N=6, H=2, d=8, T=10, Dc=16)
    mask = np.zeros((2, 10), np.uint8)
    mask[:, [3, 4]] = 1
    cfg = o.TaqConfig(heads=2, w_bits=4, w_group=8, contract=True)
    base = o.taq_layer(X, ctx, Wq, Wk, Wv, Wo, bo, mask, cfg)
    r = _rng(15)
    perm = r.permutation(6)                                        # query rows are independent
    got = o.taq_layer(X[:, perm], ctx, Wq, Wk, Wv, Wo, bo, mask, cfg)["Y"]
    assert np.array_equal(got, base["Y"][:, perm])
    # permuting text tokens together with the mask changes nothing but the summation order
    cfg_i = o.TaqConfig(heads=2, w_bits=4, w_group=8, contract=False)
    base_i = o.taq_layer(X, ctx, Wq, Wk, Wv, Wo, bo, mask, cfg_i)["Y"]
    pt = r.permutation(10)
    got = o.taq_layer(X, ctx[:, pt], Wq, Wk, Wv, Wo, bo, mask[:, pt], cfg_i)["Y"]
    np.testing.assert_allclose(got, base_i, rtol=0, atol=1e-12)
    # batch entries are independent, each with its own mask
    m2 = mask.copy()
    m2[1] = 0
    m2[1, 7] = 1
    both = o.taq_layer(X, ctx, Wq, Wk, Wv, Wo, bo, m2, cfg)["Y"]
    one = o.taq_layer(X[1:], ctx[1:], Wq, Wk, Wv, Wo, bo, m2[1:], cfg)["Y"]
    assert np.array_equal(both[1], one[0]) and np.array_equal(both[0], base["Y"][0])
    assert not np.array_equal(both[1], base["Y"][1])                # the mask matters
    # head h of O depends only on head h's slice of Wq (rows h*d..)
    Wq2 = Wq.copy()
    Wq2[8:] *= 1.5
    O2 = o.taq_layer(X, ctx, Wq2, Wk, Wv, Wo, bo, mask, cfg)["O"]
    assert np.array_equal(O2[..., :8], base["O"][..., :8]) and not np.array_equal(O2[..., 8:], base["O"][..., 8:])
    # protecting a whole span: every index of the span passes through
    kv = o.taq_kv(ctx, Wk, Wv, mask, cfg_i)
    assert np.array_equal(kv["K_tilde"][:, :, 3:5], kv["K"][:, :, 3:5])


def _brute_force_layer(X, ctx, Wq_hat, Wk_hat, Wv_hat, Wo_hat, bo, mkv, ma, H):
    """Eq. 2 and Eq. 3 evaluated element by element with the 0/1 masks multiplied in, as the paper
    writes them; scalar float32 quantizers; pure Python loops.  Ideal arithmetic (no fp16)."""
    f32 = np.float32

    def q_row(row, qmax):                                   # list of python floats -> dequantized list
        r32 = [f32(v) for v in row]
        a = max(abs(v) for v in r32)
        if a == 0:
            return [0.0] * len(row)
        s = f32(a / f32(qmax))
        out = []
        for v in r32:
            c = float(np.rint(f32(v / s)))
            c = max(-qmax, min(qmax, c))
            out.append(float(f32(f32(c) * s)))
        return out

    B, N, C = X.shape
    T, Dc = ctx.shape[1], ctx.shape[2]
    d = C // H
    Y = np.zeros((B, N, C))
    for b in range(B):
        proj = lambda x, W: [[sum(float(x[i][k]) * float(W[n][k]) for k in range(len(W[0]))) for n in range(len(W))] for i in range(len(x))]
        Q, K, V = proj(X[b], Wq_hat), proj(ctx[b], Wk_hat), proj(ctx[b], Wv_hat)
        O = [[0.0] * C for _ in range(N)]
        for h in range(H):
            lo = h * d
            Kt, Vt = [], []
            for j in range(T):
                kq, vq = q_row(K[j][lo:lo + d], 127), q_row(V[j][lo:lo + d], 127)
                m = float(mkv[b][j])
                Kt.append([m * K[j][lo + c] + (1 - m) * kq[c] for c in range(d)])       # Eq. 2
                Vt.append([m * V[j][lo + c] + (1 - m) * vq[c] for c in range(d)])
            for n in range(N):
                qt = q_row(Q[n][lo:lo + d], 127)                                           # Q~ = Q_a(Q)
                logits = [sum(qt[c] * Kt[j][c] for c in range(d)) / math.sqrt(d) for j in range(T)]
                mx = max(logits)
                e = [math.exp(l - mx) for l in logits]
                z = sum(e)
                for j in range(T):
                    a = e[j] / z
                    aq = float(f32(f32(np.rint(f32(f32(a) * f32(255)))) / f32(255)))
                    m = float(ma[b][j])
                    ah = m * a + (1 - m) * aq                                              # Eq. 3
                    for c in range(d):
                        O[n][lo + c] += ah * Vt[j][c]
        for n in range(N):
            for co in range(C):
                Y[b, n, co] = sum(O[n][k] * float(Wo_hat[co][k]) for k in range(C)) + float(bo[co])
    return Y


def check_brute_force(o):
    for seed, (B, N, H, d, T, Dc) in enumerate([(1, 3, 2, 8, 5, 8), (2, 2, 1, 4, 3, 8), (1, 1, 2, 2, 1, 4)]):
        X, ctx, Wq, Wk, Wv, Wo, bo = _tiny_layer(20 + seed, B=B, N=N, H=H, d=d, T=T, Dc=Dc)
        r = _rng(30 + seed)
        mask = (r.random((B, T)) < 0.4).astype(np.uint8)
        cfg = o.TaqConfig(heads=H, w_bits=4, w_group=0, contract=False)
        deq = lambda W: o.dequantize_weights(*o.quantize_weights(W, 4, 0), 0, contract=False)
        got = o.taq_layer(X, ctx, Wq, Wk, Wv, Wo, bo, mask, cfg)["Y"]
        want = _brute_force_layer(X.astype(np.float64), ctx.astype(np.float64), deq(Wq), deq(Wk), deq(Wv), deq(Wo), bo, mask, mask, H)
        np.testing.assert_allclose(got, want, rtol=0, atol=1e-9)


def check_contract_close_to_ideal(o):
    """The fp16 storage roundings of contract mode are small next to the quantization itself."""
    X, ctx, Wq, Wk, Wv, Wo, bo = _tiny_layer(16, B=1, N=32, H=2, d=16, T=12, Dc=32)
    mask = np.zeros((1, 12), np.uint8)
    mask[0, 4] = 1
    yi = o.taq_layer(X, ctx, Wq, Wk, Wv, Wo, bo, mask, o.TaqConfig(heads=2, w_bits=0, q_bits=0, kv_bits=0, p_bits=0, contract=False))["Y"]
    yc = o.taq_layer(X, ctx, Wq, Wk, Wv, Wo, bo, mask, o.TaqConfig(heads=2, w_bits=0, q_bits=0, kv_bits=0, p_bits=0, contract=True))["Y"]
    rel = np.linalg.norm(yc - yi) / np.linalg.norm(yi)
    assert 0 < rel < 2e-3
    assert np.array_equal(yc, yc.astype(np.float16).astype(np.float64))      # Y is fp16 data


def check_contract_roundings(o):
    """Every fp16 rounding point of contract mode on a hand-built case whose expected value is typed in as a literal
    (worked out by hand from the fp16 grid: spacing 2^-4 in [64,128), 2^-9 in [2,4), 2^-10 in [1,2), 2^-14 in [1/16,1/8))."""
    cfg = o.TaqConfig(heads=1, w_bits=0, q_bits=0, kv_bits=8, p_bits=8, contract=True)
    one = np.ones((1, 1, 1, 1))
    # (1) a trigger probability column is stored in the unit of the uint8 codes, 1/255, as fp16(255 A) / 255.
    #     Two keys with logits (0, ln(154.7 / 100.3)): A = (100.3, 154.7) / 255.  255 A_0 = 100.3 lies between the fp16
    #     numbers 100.25 and 100.3125 and is nearer the second; A_0 itself (0.39333...) would round to 0.393310546875.
    K = np.array([0.0, np.log(154.7 / 100.3)]).reshape(1, 1, 2, 1)
    V = np.array([1.0, 0.0]).reshape(1, 1, 2, 1)
    _, A, A_hat = o.taq_attention(one, K, V, np.array([[1, 0]], np.uint8), cfg, return_probs=True)
    assert abs(A[0, 0, 0, 0] - 100.3 / 255) < 1e-12
    assert A_hat[0, 0, 0, 0] == 100.3125 / 255                           # not A, not fp16(A) = 0.393310546875
    assert abs(A_hat[0, 0, 0, 1] - 155.0 / 255) < 1e-7                   # the ordinary column: rint(154.7) = 155, dequantized in binary32
    # (2), (3) the value operand of an ordinary row is fp16(code * scale), and O is fp16.  Logits (0, ln 2): A = (1/3, 2/3),
    #     codes (85, 170), so A^ = (1/3, 2/3) exactly.  V~ = (3.001, 0): fp16(3.001) = 3.001953125 (3.001 is 0.00095 from it
    #     and 0.001 from 3.0); a third of that, 1.00065..., rounds to 1.0009765625.  With V~ left unrounded the product is
    #     1.00033..., which rounds to 1.0; with O left unrounded it stays 1.00065104....
    K = np.array([0.0, np.log(2.0)]).reshape(1, 1, 2, 1)
    V = np.array([3.001, 0.0]).reshape(1, 1, 2, 1)
    O = o.taq_attention(one, K, V, np.zeros((1, 2), np.uint8), cfg)
    assert O.shape == (1, 1, 1) and O[0, 0, 0] == 1.0009765625
    O_ideal = o.taq_attention(one, K, V, np.zeros((1, 2), np.uint8), o.TaqConfig(heads=1, w_bits=0, q_bits=0, contract=False))
    assert abs(O_ideal[0, 0, 0] - 3.001 / 3) < 1e-7                      # (the code 85 is dequantized in binary32)
    # (4) an unquantized Q (q_bits = 0) is an fp16 tensor: 1.0 * fp32(0.1) -> 0.0999755859375 (spacing 2^-14 there)
    q = o.taq_q(np.ones((1, 1, 1), np.float16), np.array([[0.1]], np.float32), cfg)
    assert q["Q_tilde"].shape == (1, 1, 1, 1) and q["Q_tilde"][0, 0, 0, 0] == 0.0999755859375
    assert abs(q["Q"][0, 0, 0, 0] - np.float64(np.float32(0.1))) < 1e-15
    # (5) a trigger K/V row is fp16 of the projected row: ctx 1.0, weights 0.1 and 0.3 -> 0.0999755859375, 0.300048828125
    kv = o.taq_kv(np.ones((1, 1, 1), np.float16), np.array([[0.1]], np.float32), np.array([[0.3]], np.float32), np.ones((1, 1), np.uint8), cfg)
    assert kv["K_tilde"][0, 0, 0, 0] == 0.0999755859375 and kv["V_tilde"][0, 0, 0, 0] == 0.300048828125
    # (6) Y is fp16: O = 1 (fp16 data), weight 0.1, bias 0.2 -> fp64 0.3000000014901161 -> 0.300048828125
    Y = o.taq_out(np.ones((1, 1, 1)), np.array([[0.1]], np.float32), np.array([0.2], np.float32), cfg)
    assert Y[0, 0, 0] == 0.300048828125


def check_integer_activations(o):
    """a_bits = 8 (the W/A reading of Table 1: the inputs of the projections are int8 per token).
    (i) the projection is an integer product: Q[b,n,c] = s_x[b,n] * sum_g s_w[c,g] * sum_{k in g} xq[b,n,k] wq[c,k],
    checked in exact rational arithmetic; (ii) inputs that already lie on an int8 grid whose largest code is 127 pass
    through unchanged, so the layer equals the a_bits = 0 layer; (iii) |x - x~| <= s/2, one scale per token."""
    B, N, H, d, T, Dc = 1, 3, 2, 8, 4, 16
    X, ctx, Wq, Wk, Wv, Wo, bo = _tiny_layer(41, B=B, N=N, H=H, d=d, T=T, Dc=Dc)
    C = H * d
    cfg = o.TaqConfig(heads=H, w_bits=4, w_group=8, q_bits=0, a_bits=8, contract=False)
    Q = o.merge_heads(o.taq_q(X, Wq, cfg)["Q"])
    xq, sx = o.quantize_rows(X.astype(np.float32), 127)
    wq, sw = o.quantize_weights(Wq, 4, 8)
    assert sx.shape == (B, N) and np.all(np.max(np.abs(xq), axis=-1) == 127)
    for n in range(N):
        for c in range(C):
            acc = Fraction(0)
            for g in range(C // 8):
                part = sum(int(xq[0, n, k]) * int(wq[c, k]) for k in range(8 * g, 8 * g + 8))
                acc += Fraction(float(sw[c, g])) * part
            want = float(Fraction(float(sx[0, n])) * acc)
            assert abs(Q[0, n, c] - want) <= 1e-12 * max(1.0, abs(want))
    # the same for to_out (with its bias) and for the K projection of the text context
    Oin = X
    Y = o.taq_out(Oin, Wo, bo, cfg)
    wo, swo = o.quantize_weights(Wo, 4, 8)
    for n in range(N):
        for c in range(0, C, 5):
            acc = sum(Fraction(float(swo[c, g])) * sum(int(xq[0, n, k]) * int(wo[c, k]) for k in range(8 * g, 8 * g + 8)) for g in range(C // 8))
            want = float(Fraction(float(sx[0, n])) * acc + Fraction(float(bo[c])))
            assert abs(Y[0, n, c] - want) <= 1e-12 * max(1.0, abs(want))
    cq, sc = o.quantize_rows(ctx.astype(np.float32), 127)
    wk, swk = o.quantize_weights(Wk, 4, 8)
    K = o.merge_heads(o.taq_kv(ctx, Wk, Wv, np.zeros((B, T), np.uint8), cfg)["K"])
    for t in range(T):
        for c in range(0, C, 3):
            acc = sum(Fraction(float(swk[c, g])) * sum(int(cq[0, t, k]) * int(wk[c, k]) for k in range(8 * g, 8 * g + 8)) for g in range(Dc // 8))
            want = float(Fraction(float(sc[0, t])) * acc)
            assert abs(K[0, t, c] - want) <= 1e-12 * max(1.0, abs(want))
    xt = o.quantize_activations(X, cfg)
    assert np.all(np.abs(xt - X.astype(np.float64)) <= sx[..., None].astype(np.float64) * 0.5000001)
    # (ii) grid inputs: codes with absmax 127 times a power of two are fixed points of the quantizer
    r = _rng(42)
    def grid(shape):
        c = r.integers(-127, 128, size=shape)
        c[..., 0] = 127
        return (c * 2.0 ** -6).astype(np.float16)
    Xg, ctxg = grid((B, N, C)), grid((B, T, Dc))
    mask = np.zeros((B, T), np.uint8); mask[0, 1] = 1
    base = dict(heads=H, w_bits=4, w_group=8, contract=False)
    q0 = o.taq_q(Xg, Wq, o.TaqConfig(a_bits=0, **base))
    q8 = o.taq_q(Xg, Wq, o.TaqConfig(a_bits=8, **base))
    np.testing.assert_allclose(q8["Q"], q0["Q"], rtol=1e-13, atol=0)
    k0 = o.taq_kv(ctxg, Wk, Wv, mask, o.TaqConfig(a_bits=0, **base))
    k8 = o.taq_kv(ctxg, Wk, Wv, mask, o.TaqConfig(a_bits=8, **base))
    np.testing.assert_allclose(k8["K"], k0["K"], rtol=1e-13, atol=0)
    np.testing.assert_allclose(k8["V"], k0["V"], rtol=1e-13, atol=0)
    Og = grid((B, N, C))
    np.testing.assert_allclose(o.taq_out(Og, Wo, bo, o.TaqConfig(a_bits=8, **base)), o.taq_out(Og, Wo, bo, o.TaqConfig(a_bits=0, **base)), rtol=1e-13, atol=1e-15)
    # and on ordinary inputs the integer-activation layer stays close to the fp16-activation layer
    X2, ctx2, Wq2, Wk2, Wv2, Wo2, bo2 = _tiny_layer(43, B=1, N=16, H=2, d=16, T=9, Dc=32)
    m2 = np.zeros((1, 9), np.uint8); m2[0, 3] = 1
    y0 = o.taq_layer(X2, ctx2, Wq2, Wk2, Wv2, Wo2, bo2, m2, o.TaqConfig(heads=2, w_bits=8, a_bits=0))["Y"]
    y8 = o.taq_layer(X2, ctx2, Wq2, Wk2, Wv2, Wo2, bo2, m2, o.TaqConfig(heads=2, w_bits=8, a_bits=8))["Y"]
    rel = np.linalg.norm(y8 - y0) / np.linalg.norm(y0)
    assert 0 < rel < 0.05
    with pytest.raises(ValueError):
        o.quantize_activations(X, o.TaqConfig(heads=H, a_bits=4))


def check_four_bit_rows_and_probabilities(o):
    """The 4-bit rows of Table 1 ("8/4"): K/V rows with qmax 7 and probabilities with 15 levels."""
    code, ph = o.quantize_prob(np.array([0.0, 1.0, 1 / 15, 7.4 / 15, 7.6 / 15, 0.5]), 4)
    assert code.tolist() == [0, 15, 1, 7, 8, 8] and abs(ph[2] - 1 / 15) < 1e-7       # 7.5 is a tie: to even
    r = _rng(50)
    A = r.dirichlet(np.ones(9), size=50)
    c4, a4 = o.quantize_prob(A, 4)
    assert c4.max() <= 15 and np.all(np.abs(a4 - A) <= 1 / 30 + 1e-7)
    X, ctx, Wq, Wk, Wv, Wo, bo = _tiny_layer(51, B=1, N=4, H=2, d=8, T=6, Dc=16)
    mask = np.zeros((1, 6), np.uint8); mask[0, 2] = 1
    kv4 = o.taq_kv(ctx, Wk, Wv, mask, o.TaqConfig(heads=2, w_bits=0, kv_bits=4, contract=False))
    assert np.abs(kv4["K_codes"]).max() == 7 and np.abs(kv4["V_codes"]).max() == 7
    nt = [0, 1, 3, 4, 5]
    assert np.all(np.max(np.abs(kv4["K_codes"][:, :, nt]), axis=-1) == 7)
    np.testing.assert_array_equal(kv4["K_tilde"][:, :, 2], kv4["K"][:, :, 2])                 # the trigger row is untouched
    err4 = np.abs(kv4["K_tilde"] - kv4["K"])[:, :, nt]
    assert np.all(err4 <= kv4["K_scales"][:, :, nt, None] * 0.5000001)
    kv8 = o.taq_kv(ctx, Wk, Wv, mask, o.TaqConfig(heads=2, w_bits=0, kv_bits=8, contract=False))
    assert err4.mean() > 8 * np.abs(kv8["K_tilde"] - kv8["K"])[:, :, nt].mean()              # 127/7 = 18 times coarser
    # empty mask, 4-bit everything == separately written uniform 4-bit attention
    Q = o.split_heads(X.astype(np.float64) @ Wq.astype(np.float64).T, 2)
    K, V = kv4["K"], kv4["V"]
    def q4(Z):
        cc, ss = o.quantize_rows(Z.astype(np.float32), 7)
        return (cc.astype(np.float32) * ss[..., None]).astype(np.float64)
    S = np.einsum("bhnd,bhtd->bhnt", Q, q4(K)) / np.sqrt(8.0)
    E = np.exp(S - S.max(-1, keepdims=True)); Af = E / E.sum(-1, keepdims=True)
    Ah = np.rint((Af.astype(np.float32) * np.float32(15)).astype(np.float32)).astype(np.float32) / np.float32(15)
    want = o.merge_heads(np.einsum("bhnt,bhtd->bhnd", Ah.astype(np.float64), q4(V)))
    got = o.taq_attention(Q, q4(K), q4(V), np.zeros((1, 6), np.uint8), o.TaqConfig(heads=2, p_bits=4, contract=False))
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-12)
    with pytest.raises(ValueError):
        o.taq_kv(ctx, Wk, Wv, mask, o.TaqConfig(heads=2, kv_bits=3))


def check_token_sensitivity(o):
    """Eq. 1 at layer level.  (i) one text token: the attention weight is 1, so y - y* = (V^ - V) Wout^T whatever the
    queries are: Delta has a closed form; (ii) K/V rows that already lie on the b-bit grid give Delta = 0; (iii) 4 bits
    hurt more than 8, and a row three times larger (the trigger rows of the workload) is more sensitive in absolute
    terms than the others."""
    full = dict(w_bits=0, q_bits=0, p_bits=0, contract=False)
    X, ctx, Wq, Wk, Wv, Wo, bo = _tiny_layer(60, B=1, N=3, H=2, d=4, T=1, Dc=8)
    for bits, qmax in ((8, 127), (4, 7)):
        d = o.token_sensitivity(X, ctx, Wq, Wk, Wv, Wo, bo, o.TaqConfig(heads=2, **full), bits)
        V = o.split_heads(ctx.astype(np.float64) @ Wv.astype(np.float64).T, 2)                 # [1,H,1,d]
        c, s = o.quantize_rows(V.astype(np.float32), qmax)
        dv = o.merge_heads((c.astype(np.float32) * s[..., None]).astype(np.float64) - V)[0, 0]  # [C]
        want = np.mean((dv @ Wo.astype(np.float64).T) ** 2)
        assert d.shape == (1,) and abs(d[0] - want) <= 1e-12 * want
    # (ii): weights and context built so that K = V = integer codes with absmax 7 per (head, token) row
    H, dd, T, Dc = 2, 4, 5, 8
    C = H * dd
    r = _rng(61)
    ctxg = np.zeros((1, T, Dc), np.float16); ctxg[0, np.arange(T), np.arange(T)] = 1           # one-hot tokens
    rows = r.integers(-7, 8, size=(T, C)).astype(np.float32)
    rows[:, 0] = 7; rows[:, dd] = -7                                                            # absmax 7 in both heads
    Wg = np.zeros((C, Dc), np.float32); Wg[:, :T] = rows.T
    Xg = r.standard_normal((1, 3, C)).astype(np.float16)
    Wqg = (r.standard_normal((C, C)) * 0.3).astype(np.float32)
    dz = o.token_sensitivity(Xg, ctxg, Wqg, Wg, Wg, Wo[:C, :C] if Wo.shape[0] >= C else Wo, None, o.TaqConfig(heads=H, **full), 4)
    assert np.all(dz == 0)
    # (iii)
    X3, ctx3, Wq3, Wk3, Wv3, Wo3, bo3 = _tiny_layer(62, B=2, N=24, H=2, d=8, T=8, Dc=32)
    ctx3 = ctx3.astype(np.float32); ctx3[:, 3] *= 3; ctx3 = ctx3.astype(np.float16)
    d8 = o.token_sensitivity(X3, ctx3, Wq3, Wk3, Wv3, Wo3, bo3, o.TaqConfig(heads=2, **full), 8)
    d4 = o.token_sensitivity(X3, ctx3, Wq3, Wk3, Wv3, Wo3, bo3, o.TaqConfig(heads=2, **full), 4)
    assert np.all(d8 > 0) and np.all(d4 > 20 * d8)
    assert np.argmax(d4) == 3 and np.argmax(d8) == 3


LAYER_CHECKS = [check_all_trigger_is_textbook_attention, check_empty_mask_is_uniform_quantization,
                check_trigger_rows_pass_through, check_closed_forms, check_structure, check_brute_force,
                check_contract_close_to_ideal, check_contract_roundings, check_integer_activations, check_four_bit_rows_and_probabilities,
                check_token_sensitivity]


@pytest.mark.parametrize("check", LAYER_CHECKS)
def test_layer_pins(check):
    check(orc)


# ---------------------------------------------------------------------------------------------
# Cost accounting
# ---------------------------------------------------------------------------------------------

def test_bops_table1_ratios():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "table1_bops.txt")) if l.strip() and not l.startswith("#")]
    by_model = {}
    for model, bw, ba, t in rows:
        by_model.setdefault(model, []).append((int(bw), int(ba), float(t)))
    for model, entries in by_model.items():
        bw0, ba0, t0 = entries[0]
        flops = t0 / orc.bops(1.0, bw0, ba0)                 # FLOPs implied by the full-precision row
        for bw, ba, t in entries[1:]:
            # the table prints integers (6930/32 = 216.56 appears as 216), so allow one unit
            assert abs(orc.bops(flops, bw, ba) - t) < 1.0, (model, bw, ba)
            assert abs(t0 / t - (bw0 * ba0) / (bw * ba)) / ((bw0 * ba0) / (bw * ba)) < 0.01
    assert orc.bops(2.0, 8, 4) == 64.0


def test_memory_reduction_4_to_8x():
    """The paper quotes a 4-8x inference-memory reduction: 32-bit -> 8-bit is 4x, -> 4-bit with one
    fp32 scale per 128 weights is 32/4.25 = 7.5x."""
    n, k = 320, 768
    full = n * k * 32
    assert abs(full / orc.packed_weight_bits(n, k, 8, 0) - 4.0) < 0.03
    assert abs(full / orc.packed_weight_bits(n, k, 4, 128) - 32 / 4.25) < 1e-9


# ---------------------------------------------------------------------------------------------
# Planted mistakes: each must be caught by at least one pin
# ---------------------------------------------------------------------------------------------

def _mutant(**patches):
    m = types.ModuleType("taq_oracle_mutant")
    src = open(orc.__file__).read()
    for old, new in patches.get("text", []):
        assert old in src, old
        src = src.replace(old, new)
    import sys
    sys.modules["taq_oracle_mutant"] = m                        # dataclasses look the module up by name
    exec(compile(src, "taq_oracle_mutant", "exec"), m.__dict__)
    return m


MUTATIONS = {
    "floor_instead_of_rint": [("q = np.rint((x / safe).astype(F32))", "q = np.floor((x / safe).astype(F32))")],
    "mask_inverted_kv": [("Zt = np.where(M, kept, Zq)", "Zt = np.where(M, Zq, kept)")],
    "mask_inverted_a": [("A_hat = np.where(M, kept, Aq)", "A_hat = np.where(M, Aq, kept)")],
    "scale_d_not_sqrt_d": [("/ np.sqrt(F64(d))", "/ F64(d)")],
    "k_v_swapped": [("taq_attention(q[\"Q_tilde\"], kv[\"K_tilde\"], kv[\"V_tilde\"]", "taq_attention(q[\"Q_tilde\"], kv[\"V_tilde\"], kv[\"K_tilde\"]")],
    "transposed_weight": [("ctx @ effective_weight(Wk, cfg).T", "ctx @ effective_weight(Wk, cfg)")],
    "q_not_quantized": [("if cfg.q_bits == 0:", "if True:")],
    "prob_scale_256": [("pmax = F32(2 ** bits - 1)", "pmax = F32(2 ** bits)")],
    "clamp_asymmetric": [("q = np.clip(q, -qmax, qmax)", "q = np.clip(q, -qmax - 1, qmax - 1)")],
    "bias_dropped": [("Y = Y + np.asarray(bout, dtype=F64)", "Y = Y")],
    "renormalised_probs": [("A_hat = np.where(M, kept, Aq)                             # Eq. 3",
                            "A_hat = np.where(M, kept, Aq); A_hat = A_hat / A_hat.sum(-1, keepdims=True)")],
    "group_ignored": [("g = k_in if group == 0 else group\n    n_groups", "g = k_in\n    n_groups")],
    "activation_scale_dropped": [("return codes.astype(F64) * scales.astype(F64)[..., None]", "return codes.astype(F64)")],
    "activations_not_quantized": [("    if cfg.a_bits == 0:\n        return x\n", "    if True:\n        return x\n")],
    "out_input_not_quantized": [("Y = quantize_activations(O, cfg) @ effective_weight(Wout, cfg).T", "Y = np.asarray(O, dtype=F64) @ effective_weight(Wout, cfg).T")],
    "activation_scale_per_tensor": [("    codes, scales = quantize_rows(x.astype(F32), 127)\n    return codes.astype(F64) * scales",
                                     "    codes, scales = quantize_rows(x.astype(F32).reshape(1, -1), 127)\n    codes = codes.reshape(x.shape); scales = np.broadcast_to(scales, x.shape[:-1])\n    return codes.astype(F64) * scales")],
    "four_bit_rows_use_qmax_8": [("127 if cfg.kv_bits == 8 else 7", "127 if cfg.kv_bits == 8 else 8")],
    "four_bit_probs_use_8_bit_levels": [("_, Aq = quantize_prob(A, cfg.p_bits)", "_, Aq = quantize_prob(A, 8)")],
    "sensitivity_quantizes_all_but_i": [("        m = ones.copy()\n        m[:, i] = 0", "        m = 1 - ones\n        m[:, i] = 1")],
    "sensitivity_reference_quantized": [("y_star = taq_layer(X, ctx, Wq, Wk, Wv, Wout, bout, ones, c, mask_a=ones)", "y_star = taq_layer(X, ctx, Wq, Wk, Wv, Wout, bout, 1 - ones, c, mask_a=ones)")],
    "contract_v_not_rounded": [("        V_tilde = f16_round(V_tilde)\n", "        V_tilde = V_tilde\n")],
    "contract_kept_prob_rounded_in_unit_1": [("kept = f16_round(A * pmax) / pmax if cfg.contract else A", "kept = f16_round(A) if cfg.contract else A")],
    "contract_kept_prob_not_rounded": [("kept = f16_round(A * pmax) / pmax if cfg.contract else A", "kept = A")],
    "contract_o_not_rounded": [("    if cfg.contract:\n        O = f16_round(O)\n", "")],
    "contract_q16_not_rounded": [("Qt = f16_round(Q) if cfg.contract else Q", "Qt = Q")],
    "contract_trigger_rows_not_rounded": [("kept = f16_round(Z) if cfg.contract else Z", "kept = Z")],
    "contract_y_not_rounded": [("    return f16_round(Y) if cfg.contract else Y", "    return Y")],
    "log_code_floor_instead_of_rint": [("code = np.where(p > 0, np.clip(np.rint(x), 0, cmax), cmax)", "code = np.where(p > 0, np.clip(np.floor(x), 0, cmax), cmax)")],
    "log_code_not_clamped": [("code = np.where(p > 0, np.clip(np.rint(x), 0, cmax), cmax)", "code = np.where(p > 0, np.rint(x), cmax)")],
    "log_base_e": [("x = (-np.log2(p)).astype(F32)", "x = (-np.log(p)).astype(F32)")],
    "log_mask_ignored": [("        A_hat = np.where(M, kept, Aq)\n    else:", "        A_hat = Aq\n    else:")],
    "heads_interleaved": [("return x.reshape(B, L, heads, d).transpose(0, 2, 1, 3)", "return x.reshape(B, L, d, heads).transpose(0, 3, 1, 2)")],
}


ALL_CHECKS = None


def test_unmutated_copy_passes_every_pin():
    m = _mutant(text=[])
    for c in [check_quantizer_hand_values, check_quantizer_exact_rational, check_quantizer_idempotent_and_pow2,
              check_weight_quantizer, check_prob_quantizer, check_log_prob_quantizer] + LAYER_CHECKS:
        c(m)


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(name):
    m = _mutant(text=MUTATIONS[name])
    checks = [check_quantizer_hand_values, check_quantizer_exact_rational, check_quantizer_idempotent_and_pow2,
              check_weight_quantizer, check_prob_quantizer, check_log_prob_quantizer] + LAYER_CHECKS
    caught = []
    for c in checks:
        try:
            c(m)
        except (AssertionError, ValueError):                     # a failed pin, or a shape mismatch
            caught.append(c.__name__)
    assert caught, f"mutation {name} passed every pin"
