"""`taq_layer_forward_static`: the layer pass that runs on the scratch array built into the library.

It serves callers that have no way to obtain a workspace: a server whose memory pool already owns the whole
GPU (a fresh device allocation would fail or stall every stream), or a plug-in interface that hands over
nothing but input and output pointers.  Its result must equal `taq_layer_forward`'s, which runs the same
kernels on a caller-owned workspace.  The shared array keeps whatever the last call left in it, so the check
is made on two calls in a row with different inputs, both on shapes whose pass really goes through the scratch
(three kernels with Q~ and O in between; the one-kernel shape never touches it): the second call's sections lie
over other bytes of what the first one left, so a stale intermediate result would show up there.
The file name sorts last on purpose, so that a run stopping at the first failure has already run the rest.
"""
import numpy as np
import pytest
import torch

from paper_2603_22943_b200 import binding as tb
from paper_2603_22943_b200 import synth

import taq_testlib as tl
from taq_testlib import dev

pytestmark = pytest.mark.gpu


def _inputs(shape):
    data = synth.make_layer(shape)
    desc = tl.gpu_desc(shape)
    P = tl.pack_layer_weights(shape, data)
    mask = dev(data["mask"])
    kv = tb.taq_kv_project(desc, dev(data["ctx"]), P["Wk"], P["Wv"], mask)
    return data, desc, P, mask, kv, dev(data["X"])


def test_static_workspace_matches_caller_workspace_on_two_calls_in_a_row():
    from dataclasses import replace
    first = replace(synth.shrink(synth.config3_layers()[10], 700), seed=11)   # C = 1280, 5.5 row tiles per sequence, Q~ int8
    second = replace(synth.shrink(synth.config3_layers()[5], 300), seed=12, q_bits=0)   # C = 640, fewer rows, Q stays fp16
    for shape in (first, second):
        data, desc, P, mask, kv, x = _inputs(shape)
        assert 0 < tb.taq_workspace_bytes(desc, 1) <= tb.taq_static_workspace_capacity()
        want = tb.taq_layer_forward(desc, x, P["Wq"], P["Wout"], kv, mask)
        got = torch.full_like(want, float("nan"))
        tb.taq_dispatch_reset()
        tb.taq_layer_forward_static(desc, x, P["Wq"], P["Wout"], kv, mask, got)
        tb.taq_poll_device_status()
        ran = tb.taq_dispatch_counts()
        # the pass went through the scratch: two dequant-GEMMs and the attention as separate kernels, none of them generic
        assert ran["layer_fused"] == 0 and ran["linear_tensor"] == 2 and ran["attention_tensor"] == 1, ran
        assert ran["linear_generic"] == 0 and ran["attention_generic"] == 0, ran
        # same kernels, same inputs, other scratch address: the outputs agree bit for bit, hence within the
        # layer tolerance used throughout (2e-2 max-abs, 1e-3 relative L2)
        tl.assert_layer_close(got.cpu().numpy(), want.cpu().numpy(), shape.name)
        assert torch.equal(got.view(torch.int16), want.view(torch.int16))
        # and the result passes the same three-part comparison with the oracle as the ordinary entry point's
        rows = np.arange(0, shape.n_query, 7)
        tl.check_layer(shape, data, got.cpu().numpy(), {"desc": desc, "packed": P, "kv": kv, "mask": mask}, rows)


def test_static_workspace_rejects_layers_beyond_its_capacity():
    shape = synth.config2()
    big = tl.gpu_desc(shape, n_query=3 * shape.n_query)                        # 24 MB of scratch > 16 MiB
    assert tb.taq_workspace_bytes(big, 1) > tb.taq_static_workspace_capacity()
    z = torch.zeros(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(tb.TaqError) as e:
        tb.taq_layer_forward_static(big, z, z, z, z, z, z)
    assert e.value.status == tb.TAQ_ERR_BUFFER_TOO_SMALL
    assert "built-in workspace" in str(e.value)
