"""Failure detection and dispatch diagnostics on the GPU, without faulting, trapping or hanging anything.

Every wait inside the kernels is bounded; when one runs out the block records TAQ_ERR_TIMEOUT in the device status word
and returns.  `taq_selftest_wait_expiry` launches one block whose only work is such a wait, on a barrier towards which
nothing was ever issued, with a short limit: the wait runs out, the status is read and cleared, and the library keeps
working.  The dispatch counters say which kernel family served a call, so that the parity tests of the benchmark
configurations can also assert that no generic CUDA-core kernel ran.
"""
import numpy as np
import pytest
import torch

from paper_2603_22943_b200 import binding as tb
from paper_2603_22943_b200 import synth

import taq_testlib as tl
from taq_testlib import dev

pytestmark = pytest.mark.gpu


def test_bounded_wait_runs_out_is_reported_and_cleared():
    tb.taq_poll_device_status()                              # clean slate
    tb.taq_selftest_wait_expiry(2_000_000)                   # about a millisecond of SM clock
    with pytest.raises(tb.TaqError) as e:
        tb.taq_poll_device_status()
    assert e.value.status == tb.TAQ_ERR_TIMEOUT
    assert "block 0" in str(e.value)
    assert tb.taq_poll_device_status() == tb.TAQ_OK          # reading cleared it
    # the context is intact: an ordinary call right after works and matches the oracle
    shape = synth.shrink(synth.config2(), 200)
    data = synth.make_layer(shape)
    y, parts = tl.gpu_layer(shape, data, return_parts=True)
    tl.check_layer(shape, data, y, parts)


@pytest.mark.parametrize("shape", [synth.config1(), synth.shrink(synth.config2(), 512)] + [synth.shrink(s, 256) for s in synth.config3_layers()[5:11:5]] +
                         [synth.shrink(s, 256) for s in synth.config4_layers()], ids=lambda s: s.name)
def test_benchmark_shapes_run_on_the_tensor_core_kernels_only(shape):
    """Every shape of the five benchmark configurations: pack, K/V projection and the layer pass launch tensor-core
    kernels only (a shape that silently fell to the generic kernels would still pass parity, 10-40x slower)."""
    data = synth.make_layer(shape)
    tb.taq_dispatch_reset()
    tl.gpu_layer(shape, data)
    ran = tb.taq_dispatch_counts()
    assert ran["linear_generic"] == 0 and ran["attention_generic"] == 0, ran
    if shape.channels == 320:
        assert ran["layer_fused"] == 1 and ran["linear_tensor"] == 2, ran          # K and V projection + the one-kernel pass
    else:
        assert ran["linear_tensor"] == 4 and ran["attention_tensor"] == 1, ran     # K, V, to_q, to_out + attention
