"""Admission through the K~/V~ cache: a request whose (checkpoint, prompt) pair is cached runs its layer pass on the
cached entry without a new K/V projection, and gets bit for bit what a fresh projection gives."""
from dataclasses import replace

import numpy as np
import pytest
import torch

from paper_2603_22943_b200 import binding as tb
from paper_2603_22943_b200 import synth

import taq_testlib as tl
from taq_testlib import dev

pytestmark = pytest.mark.gpu


def test_cached_entries_serve_repeated_checkpoint_prompt_pairs():
    base = replace(synth.shrink(synth.config2(), 200), batch=1)
    desc = tl.gpu_desc(base, max_trigger=3)
    entry = (tb.taq_kv_bytes(desc) + 127) // 128 * 128
    arena = torch.zeros(2 * entry, dtype=torch.uint8, device="cuda")          # room for two pairs
    cache = tb.KvCache(arena.data_ptr(), arena.numel(), entry)
    ckpts, prompts = {}, {}
    for c in (0, 1):                                                          # two checkpoints: their own weights and trigger span
        shape = replace(base, seed=100 + c, trigger=(3 + c, 4 + c))
        data = synth.make_layer(shape)
        ckpts[c] = (shape, data, tl.pack_layer_weights(shape, data))
    for p in (0, 1):                                                          # two prompts: their own text context
        prompts[p] = (list(range(5 + p, 15 + p)), synth.make_layer(replace(base, seed=200 + p))["ctx"])
    x = dev(ckpts[0][1]["X"])
    projections = 0
    outputs = {}
    for c, p in [(0, 0), (1, 0), (0, 0), (0, 1), (1, 0), (0, 0)]:
        shape, data, P = ckpts[c]
        tokens, ctx = prompts[p]
        key = (c, tb.taq_hash_prompt(tokens))
        addr, hit = cache.acquire(*key)
        off = addr - arena.data_ptr()
        kv = arena[off: off + entry]
        mask = dev(data["mask"])
        if not hit:
            tb.taq_kv_project(desc, dev(ctx), P["Wk"], P["Wv"], mask, kv=kv)
            projections += 1
        y = tb.taq_layer_forward(desc, x, P["Wq"], P["Wout"], kv, mask)
        fresh = tb.taq_kv_project(desc, dev(ctx), P["Wk"], P["Wv"], mask)
        want = tb.taq_layer_forward(desc, x, P["Wq"], P["Wout"], fresh, mask)
        tb.taq_poll_device_status()
        assert torch.equal(y.view(torch.int16), want.view(torch.int16)), (c, p, hit)
        outputs.setdefault((c, p), y.clone())
        assert torch.equal(outputs[(c, p)], y)
        cache.release(*key)
    st = cache.stats()
    # (0,0) miss, (1,0) miss, (0,0) hit, (0,1) miss evicting (1,0), (1,0) miss evicting (0,0), (0,0) miss evicting (0,1)
    assert projections == 5 and st["hits"] == 1 and st["misses"] == 5 and st["evictions"] == 3, st
    assert not torch.equal(outputs[(0, 0)], outputs[(1, 0)]) and not torch.equal(outputs[(0, 0)], outputs[(0, 1)])
    cache.close()
