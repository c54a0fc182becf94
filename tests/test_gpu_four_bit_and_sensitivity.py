"""4-bit K/V rows and attention probabilities (the "8/4" rows of Table 1), a probability mask chosen independently of
the K/V mask, and the token-sensitivity sweep of Eq. 1, on the GPU against the oracle."""
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


def _cases():
    c3 = synth.config3_layers()
    return [
        replace(synth.shrink(synth.config2(), 500), seed=31, kv_bits=4, p_bits=4),      # the one-kernel layer pass
        replace(synth.shrink(synth.config2(), 300), seed=32, kv_bits=4, p_bits=8),
        replace(synth.shrink(synth.config2(), 300), seed=33, kv_bits=8, p_bits=4, q_bits=0),
        replace(synth.shrink(c3[5], 200), seed=34, kv_bits=4, p_bits=4),                # three kernels, d = 80
        replace(synth.config1(), kv_bits=4, p_bits=4),                                  # W8, d = 160
        replace(synth.shrink(synth.config2(), 100), seed=35, n_ctx=100, ctx_dim=768, kv_bits=4, p_bits=4),   # T > 80: generic attention kernel
    ]


@pytest.mark.parametrize("shape", _cases(), ids=lambda s: f"{s.name}_kv{s.kv_bits}_p{s.p_bits}_q{s.q_bits}")
def test_layer_with_four_bit_rows_and_probabilities(shape):
    data = synth.make_layer(shape)
    y, parts = tl.gpu_layer(shape, data, return_parts=True)
    assert np.isfinite(y).all()
    kvg = tl.parse_kv_block(parts["desc"], parts["kv"])
    if shape.kv_bits == 4:
        assert np.abs(kvg["K_codes"]).max() == 7 and np.abs(kvg["V_codes"]).max() == 7
    tl.check_layer(shape, data, y, parts)
    # coarser codes move the output: this is not the 8-bit layer again
    y8 = tl.gpu_layer(replace(shape, kv_bits=8, p_bits=8), data)
    assert tl.errors(y, y8)[1] > 3e-3


def test_probability_mask_independent_of_the_row_mask():
    """M_A (Eq. 3) need not equal M_KV (Eq. 2): K/V rows of tokens 4, 5 in fp16, probability columns 5, 9, 20 in fp16."""
    shape = replace(synth.shrink(synth.config2(), 260), seed=36)
    data = synth.make_layer(shape)
    desc = tl.gpu_desc(shape)
    P = tl.pack_layer_weights(shape, data)
    mask_a = np.zeros_like(data["mask"]); mask_a[:, [5, 9, 20]] = 1
    kv = tb.taq_kv_project(desc, dev(data["ctx"]), P["Wk"], P["Wv"], dev(data["mask"]))
    tb.taq_kv_set_prob_mask(desc, kv, dev(mask_a))
    y = tb.taq_layer_forward(desc, dev(data["X"]), P["Wq"], P["Wout"], kv, dev(mask_a)).cpu().numpy()
    tb.taq_poll_device_status()
    cfg = tl.oracle_cfg(shape)
    want = orc.taq_layer(data["X"], data["ctx"], data["Wq"], data["Wk"], data["Wv"], data["Wout"], data["bout"], data["mask"], cfg, mask_a=mask_a)["Y"]
    same = orc.taq_layer(data["X"], data["ctx"], data["Wq"], data["Wk"], data["Wv"], data["Wout"], data["bout"], data["mask"], cfg)["Y"]
    max_abs, rel = tl.errors(y, want)
    assert rel <= tl.TOL_REL_L2, (max_abs, rel)
    assert tl.errors(y, same)[1] > rel * 1.5          # and it is the independent mask that was applied


@pytest.mark.parametrize("bits", [4, 8])
def test_token_sensitivity_sweep(bits):
    """Eq. 1 at layer level on a config-2-shaped layer (77 text tokens, trigger rows of the context three times larger):
    the GPU sweep reproduces the oracle's Delta_i, and the trigger tokens come out as the most sensitive ones."""
    shape = replace(synth.shrink(synth.config2(), 256), seed=37, q_bits=0, kv_bits=bits, w_bits=8, w_group=0)
    data = synth.make_layer(shape)
    T = shape.n_ctx
    desc = tl.gpu_desc(shape, max_trigger=T)
    P = tl.pack_layer_weights(shape, data)
    delta = tb.taq_token_sensitivity(desc, dev(data["X"]), dev(data["ctx"]), P["Wq"], P["Wk"], P["Wv"], P["Wout"])
    tb.taq_poll_device_status()
    delta = delta.cpu().numpy()
    want = orc.token_sensitivity(data["X"], data["ctx"], data["Wq"], data["Wk"], data["Wv"], data["Wout"], data["bout"], tl.oracle_cfg(shape), bits)
    assert delta.shape == (T,) and np.all(delta >= 0)
    # Delta is a mean square of differences of fp16 outputs: tokens whose effect is below the fp16 spacing of Y are noise
    # on both sides, so the comparison weighs tokens by their size
    assert abs(delta.sum() - want.sum()) <= 0.05 * want.sum()
    big = want >= 0.02 * want.max()
    assert big.sum() >= 2
    assert np.all(np.abs(delta[big] - want[big]) <= 0.15 * want[big])
    top = set(np.argsort(want)[-2:].tolist())
    assert top == set(shape.trigger) and set(np.argsort(delta)[-2:].tolist()) == top
