"""Parity of the CUDA path with the CPU oracle, through the C ABI: K/V projection with Eq. 2, the dequant-GEMM
with its epilogues, the fused attention of Eq. 3, the whole layer on the benchmark configurations, the batched
serving entry points, and the edge cases."""
import numpy as np
import pytest
import torch

from oracle import taq_oracle as orc
from paper_2603_22943_b200 import binding as tb
from paper_2603_22943_b200 import synth
import taq_testlib as tl
from taq_testlib import dev

pytestmark = pytest.mark.gpu


def _small(shape, n):
    return synth.shrink(shape, n)


def _code_agreement(got, want, what):
    """Integer codes computed after an fp32 (GPU) or fp64 (oracle) accumulation may differ by one step where the
    pre-rounding value sits within ~1e-6 of a rounding boundary; nothing else is allowed."""
    diff = np.abs(got.astype(np.int32) - want.astype(np.int32))
    assert diff.max() <= 1, f"{what}: a code differs by {diff.max()}"
    frac = float((diff != 0).mean())
    assert frac <= 2e-3, f"{what}: {frac:.2e} of the codes differ"
    return frac


# ---------------------------------------------------------------------------------------------------------
# K/V projection + Eq. 2
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape", [synth.config1(), synth.config2(), synth.config4_layers()[0]], ids=lambda s: s.name)
def test_kv_project(shape):
    shape = _small(shape, 8)
    data = synth.make_layer(shape)
    desc = tl.gpu_desc(shape)
    P = tl.pack_layer_weights(shape, data)
    kv = tb.taq_kv_project(desc, dev(data["ctx"]), P["Wk"], P["Wv"], dev(data["mask"]))
    tb.taq_poll_device_status()
    got = tl.parse_kv_block(desc, kv)
    want = orc.taq_kv(data["ctx"], data["Wk"], data["Wv"], data["mask"], tl.oracle_cfg(shape))
    trig = list(shape.trigger)
    nt = [j for j in range(shape.n_ctx) if j not in trig]
    for nm in ("K", "V"):
        _code_agreement(got[nm + "_codes"][:, :, nt], want[nm + "_codes"][:, :, nt], nm)
        # fp32 accumulation over up to 2048 products against fp64: a few 1e-6 relative
        np.testing.assert_allclose(got[nm + "_scales"][:, :, nt], want[nm + "_scales"][:, :, nt], rtol=2e-5)
        assert not got[nm + "_codes"][:, :, trig].any() and not got[nm + "_scales"][:, :, trig].any()
        for s, j in enumerate(trig):                         # trigger rows: fp16 of the unquantized row
            g = got[nm + "_trigger"][:, s].astype(np.float64)               # [B,H,d]
            w = want[nm + "_tilde"][:, :, j]
            assert np.max(np.abs(g - w)) <= np.max(np.abs(w)) * 2.0 ** -10
            assert (g != w).mean() < 0.03          # an fp16 rounding that lands on the other side is rare (~1 % with tensor-core accumulation)
        deq = got[nm + "_codes"].astype(np.float64) * got[nm + "_scales"][..., None]
        assert tl.errors(deq[:, :, nt], want[nm + "_tilde"][:, :, nt])[1] < 1e-3
    for b in range(shape.batch):
        slot = got["slot"][b]
        assert [int(slot[j]) for j in trig] == list(range(len(trig)))
        assert np.all(slot[nt] == -1) and np.all(slot[shape.n_ctx:] == -1)


def test_kv_project_trigger_capacity_overflow_raises_device_status():
    shape = _small(synth.config2(), 8)
    data = synth.make_layer(shape)
    desc = tl.gpu_desc(shape, max_trigger=1)               # two trigger tokens, room for one
    P = tl.pack_layer_weights(shape, data)
    tb.taq_kv_project(desc, dev(data["ctx"]), P["Wk"], P["Wv"], dev(data["mask"]))
    with pytest.raises(tb.TaqError) as e:
        tb.taq_poll_device_status()
    assert e.value.status == tb.TAQ_ERR_SHAPE
    tb.taq_poll_device_status()                              # cleared by the first poll


# ---------------------------------------------------------------------------------------------------------
# Dequant-GEMM
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("rows,n_out,k_in,bits,group,heads", [
    (8192, 320, 320, 4, 128, 8),      # config 2 to_q
    (300, 320, 320, 4, 128, 8),       # ragged row tile
    (64, 1280, 1280, 8, 0, 8),        # config 1
    (1000, 640, 640, 4, 128, 10),     # SDXL d=64
    (513, 1280, 1280, 4, 128, 20),
    (130, 640, 640, 4, 128, 8),       # d=80
    (512, 1280, 1280, 4, 128, 8),     # d=160: a head over two 80-wide tiles, absmax exchanged through the cluster
    (130, 1280, 1280, 4, 128, 8),     # the same, ragged row tile
    (1300, 1280, 1280, 4, 128, 8),    # d=160 beyond one wave: one 160-wide tile per head
    (5, 16, 8, 4, 0, 2), (1, 64, 64, 8, 0, 1), (77, 96, 72, 4, 0, 4),
])
def test_quantized_linear(rows, n_out, k_in, bits, group, heads):
    r = np.random.default_rng(rows + n_out)
    x = r.standard_normal((rows, k_in)).astype(np.float16)
    x[:, r.integers(0, k_in)] *= 20
    W = (r.standard_normal((n_out, k_in)) / np.sqrt(k_in)).astype(np.float32)
    bias = (0.1 * r.standard_normal(n_out)).astype(np.float32)
    d = tb.weight_desc(n_out, k_in, bits, group)
    blob = tb.taq_pack_weights(d, dev(W), dev(bias))
    cfg = orc.TaqConfig(heads=heads, w_bits=bits, w_group=group)
    What = orc.effective_weight(W, cfg)
    y64 = x.astype(np.float64) @ What.T
    y32 = tb.taq_quantized_linear(d, dev(x), blob, tb.TAQ_OUT_F32).cpu().numpy()
    np.testing.assert_allclose(y32, y64 + bias, rtol=0, atol=2e-5 * np.abs(y64).max() + 1e-6)
    y16 = tb.taq_quantized_linear(d, dev(x), blob, tb.TAQ_OUT_F16).cpu().numpy()
    want16 = (y64 + bias).astype(np.float16)
    # one fp16 step where the fp32 sum lands on the other side of a rounding boundary, plus the accumulation error
    ulp = np.maximum(np.abs(want16.astype(np.float64)), 2.0 ** -14) * 2.0 ** -10
    assert np.all(np.abs(y16.astype(np.float64) - want16.astype(np.float64)) <= ulp + 2e-5 * np.abs(y64).max())
    assert (y16 != want16).mean() < 2e-2       # tensor-core fp32 accumulation: ~1.5e-6 relative, so ~0.6 % of fp16 roundings flip
    yq, sq = tb.taq_quantized_linear(d, dev(x), blob, tb.TAQ_OUT_INT8_HEAD_ROWS, heads=heads)
    dh = n_out // heads
    want_c, want_s = orc.quantize_rows(y64.reshape(rows, heads, dh).astype(np.float32), 127)
    _code_agreement(yq.cpu().numpy().reshape(rows, heads, dh), want_c, "Q codes")
    np.testing.assert_allclose(sq.cpu().numpy(), want_s, rtol=2e-5)
    tb.taq_poll_device_status()


# ---------------------------------------------------------------------------------------------------------
# Attention core in isolation: fed with the oracle's own Q~, K~, V~
# ---------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("shape,n", [(synth.config1(), 64), (synth.config2(), 300), (synth.config3_layers()[5], 200),
                                     (synth.config4_layers()[0], 130)], ids=lambda v: getattr(v, "name", str(v)))
@pytest.mark.parametrize("q_bits", [8, 0])
def test_cross_attention_isolated(shape, n, q_bits):
    from dataclasses import replace
    shape = replace(_small(shape, n), q_bits=q_bits)
    data = synth.make_layer(shape)
    cfg = tl.oracle_cfg(shape)
    kv = orc.taq_kv(data["ctx"], data["Wk"], data["Wv"], data["mask"], cfg)
    q = orc.taq_q(data["X"], data["Wq"], cfg)
    want = orc.taq_attention(q["Q_tilde"], kv["K_tilde"], kv["V_tilde"], data["mask"], cfg)
    desc = tl.gpu_desc(shape)
    blk = tl.build_kv_block(desc, kv["K_codes"], kv["K_scales"], kv["V_codes"], kv["V_scales"], kv["K_tilde"], kv["V_tilde"], data["mask"])
    B, N, C, H = shape.batch, shape.n_query, shape.channels, shape.heads
    if q_bits == 8:
        qc = orc.merge_heads(q["Q_codes"]).astype(np.int8)
        qs = np.ascontiguousarray(q["Q_scales"].transpose(0, 2, 1)).astype(np.float32)        # [B,N,H]
        o = tb.taq_cross_attention(desc, dev(qc), dev(qs), tb.taq_kv_finalize(desc, dev(blk)), dev(data["mask"]))
    else:
        q16 = orc.merge_heads(q["Q_tilde"]).astype(np.float16)
        o = tb.taq_cross_attention(desc, dev(q16), None, tb.taq_kv_finalize(desc, dev(blk)), dev(data["mask"]))
    tb.taq_poll_device_status()
    max_abs, rel = tl.assert_layer_close(o.cpu().numpy(), want, "O")
    assert rel < 5e-4                                         # fp16 output rounding is the only modelled difference


# ---------------------------------------------------------------------------------------------------------
# Whole layer on the benchmark configurations
# ---------------------------------------------------------------------------------------------------------
def _layer_case(shape, sample_rows=None, max_trigger=None):
    data = synth.make_layer(shape)
    y, parts = tl.gpu_layer(shape, data, max_trigger=max_trigger, return_parts=True)
    rows = None
    if sample_rows is not None and sample_rows < shape.n_query:
        rows = np.sort(np.random.default_rng(99).choice(shape.n_query, sample_rows, replace=False))
    return tl.check_layer(shape, data, y, parts, rows)


@pytest.mark.parametrize("shape_fn,n", [(synth.config2, 4096), (synth.config2, 333), (lambda: synth.config3_layers()[5], 200)],
                         ids=["config2_full", "config2_ragged", "C640_unfused"])
@pytest.mark.parametrize("q_bits", [8, 0])
def test_query_attention_equals_the_two_step_path(shape_fn, n, q_bits):
    """taq_query_attention (one fused kernel at C = 320) against taq_quantized_linear + taq_cross_attention on the same
    inputs: the same Q~ codes and scores; the fused kernel sums a row's 80 exponentials in one thread, the stand-alone
    kernel in two, so a probability that sits on a rounding boundary may take the neighbouring code (1/255 of one value
    row): O agrees to that, and both are checked against the oracle's O on sampled rows."""
    from dataclasses import replace
    shape = replace(_small(shape_fn(), n), q_bits=q_bits)
    data = synth.make_layer(shape)
    desc = tl.gpu_desc(shape)
    P = tl.pack_layer_weights(shape, data)
    mask = dev(data["mask"])
    kv = tb.taq_kv_project(desc, dev(data["ctx"]), P["Wk"], P["Wv"], mask)
    x = dev(data["X"])
    o_fused = tb.taq_query_attention(desc, x, P["Wq"], kv, mask)
    x2 = x.reshape(-1, shape.channels)
    if q_bits == 8:
        qc, qs = tb.taq_quantized_linear(P["wd_cc"], x2, P["Wq"], tb.TAQ_OUT_INT8_HEAD_ROWS, heads=shape.heads)
        o_two = tb.taq_cross_attention(desc, qc, qs, kv, mask)
    else:
        q16 = tb.taq_quantized_linear(P["wd_cc"], x2, P["Wq"], tb.TAQ_OUT_F16)
        o_two = tb.taq_cross_attention(desc, q16, None, kv, mask)
    tb.taq_poll_device_status()
    tl.assert_same_up_to_code_ties(o_fused, o_two, "O")
    rows = np.arange(0, shape.n_query, max(1, shape.n_query // 64))
    cfg = tl.oracle_cfg(shape)
    g = tl.gpu_decisions(shape, data, {"desc": desc, "packed": P, "kv": kv, "mask": mask}, rows)
    want = orc.taq_attention(g["Q_tilde"], g["K_tilde"], g["V_tilde"], data["mask"], cfg)
    tl.assert_layer_close(o_fused.cpu().numpy()[:, rows], want, shape.name + " O (same decisions)")


@pytest.mark.parametrize("n,q_bits", [(4096, 8), (333, 8), (130, 0)])
def test_one_kernel_layer_equals_the_step_by_step_path(n, q_bits):
    """At C = 320 taq_layer_forward is a single kernel (pairs of CTAs exchange O through distributed shared memory and
    run to_out themselves).  Its Y must equal taq_query_attention followed by taq_quantized_linear up to the order in
    which the scale groups' partial sums are added (the second CTA of a pair walks the K blocks downwards) and to the
    fp16 rounding of Y that this moves; the oracle comparison at the full tolerance is test_layer_config2_full."""
    from dataclasses import replace
    shape = replace(_small(synth.config2(), n), q_bits=q_bits)
    data = synth.make_layer(shape)
    desc = tl.gpu_desc(shape)
    P = tl.pack_layer_weights(shape, data)
    mask = dev(data["mask"])
    kv = tb.taq_kv_project(desc, dev(data["ctx"]), P["Wk"], P["Wv"], mask)
    x = dev(data["X"])
    y_one = tb.taq_layer_forward(desc, x, P["Wq"], P["Wout"], kv, mask)
    o = tb.taq_query_attention(desc, x, P["Wq"], kv, mask)
    y_two = tb.taq_quantized_linear(P["wd_cc"], o.reshape(-1, shape.channels), P["Wout"], tb.TAQ_OUT_F16).reshape(y_one.shape)
    tb.taq_poll_device_status()
    tl.assert_same_up_to_code_ties(y_one, y_two, "Y")


def test_layer_config1_full():
    _layer_case(synth.config1())


def test_layer_config2_full():
    """Config 2 at its full size (B=2, N=4096, C=320, W4 group 128), the shape the benchmark times."""
    _layer_case(synth.config2())


def test_layer_config2_q_unquantized():
    from dataclasses import replace
    _layer_case(replace(synth.config2(), q_bits=0, name="config2_q16"), sample_rows=512)


@pytest.mark.parametrize("i", range(16))
def test_layer_config3_each_layer_full_size_sampled_rows(i):
    """All 16 SD-1.5 layer shapes at full size on the GPU; the oracle recomputes 256 sampled query rows per
    sequence (query rows are independent), or all rows of the 64-row layer."""
    _layer_case(synth.config3_layers()[i], sample_rows=256)


@pytest.mark.parametrize("i", range(2))
def test_layer_config4_sdxl_full_size_sampled_rows(i):
    _layer_case(synth.config4_layers()[i], sample_rows=256)


@pytest.mark.parametrize("n", [1, 7, 63, 65, 129, 200])
def test_layer_ragged_row_counts(n):
    _layer_case(_small(synth.config2(), n))
    _layer_case(_small(synth.config3_layers()[10], n))


def test_layer_empty_mask_all_trigger_mask_and_single_token_context():
    from dataclasses import replace
    base = _small(synth.config2(), 96)
    _layer_case(replace(base, trigger=(), name="empty_mask"))
    # every token a trigger: nothing in K/V/A is quantized, only Q and the weights are
    _layer_case(replace(base, trigger=tuple(range(77)), name="all_trigger"), max_trigger=77)
    for T in (1, 2, 33):
        _layer_case(replace(base, n_ctx=T, trigger=(0,), name=f"T{T}"))


def test_layer_is_deterministic_and_stays_inside_its_buffers():
    shape = _small(synth.config2(), 200)
    data = synth.make_layer(shape)
    desc = tl.gpu_desc(shape)
    P = tl.pack_layer_weights(shape, data)
    mask = dev(data["mask"])
    kvn = tb.taq_kv_bytes(desc)
    guard = 1024
    kvbuf = torch.full((kvn + 2 * guard,), 0x5A, dtype=torch.uint8, device="cuda")
    tb.taq_kv_project(desc, dev(data["ctx"]), P["Wk"], P["Wv"], mask, kvbuf[guard: guard + kvn])
    n = shape.rows * shape.channels
    ybuf = torch.full((n + 2 * guard,), -7.0, dtype=torch.float16, device="cuda")
    wsn = tb.taq_workspace_bytes(desc, 1)
    wsbuf = torch.full((wsn + 2 * guard,), 0x5A, dtype=torch.uint8, device="cuda")
    x = dev(data["X"])
    outs = []
    for _ in range(2):
        tb.taq_layer_forward(desc, x, P["Wq"], P["Wout"], kvbuf[guard: guard + kvn], mask, ybuf[guard: guard + n], wsbuf[guard: guard + wsn])
        torch.cuda.synchronize()
        outs.append(ybuf.cpu().numpy().copy())
    assert np.array_equal(outs[0].view(np.uint16), outs[1].view(np.uint16))
    assert np.all(outs[0][:guard] == -7.0) and np.all(outs[0][-guard:] == -7.0)
    k = kvbuf.cpu().numpy()
    w = wsbuf.cpu().numpy()
    assert np.all(k[:guard] == 0x5A) and np.all(k[-guard:] == 0x5A) and np.all(w[:guard] == 0x5A) and np.all(w[-guard:] == 0x5A)
    tb.taq_poll_device_status()


def test_empty_inputs():
    shape = _small(synth.config2(), 0)
    desc = tl.gpu_desc(shape)
    z = torch.zeros(16, dtype=torch.uint8, device="cuda")
    y = tb.taq_layer_forward(desc, z, z, z, z, z, y=torch.zeros(16, dtype=torch.float16, device="cuda"), workspace=torch.zeros(128, dtype=torch.uint8, device="cuda"))
    tb.taq_poll_device_status()


# ---------------------------------------------------------------------------------------------------------
# Batched serving: every request carries its own checkpoint (weights, trigger mask) and its own K~/V~
# ---------------------------------------------------------------------------------------------------------
def _serving_case(n_ckpt, n_req, n_query, C_, Dc, T=77, seed=0):
    ckpts = [synth.make_checkpoint(c, C_, Dc, T) for c in range(n_ckpt)]
    route = synth.make_request_batch(n_req, n_ckpt, seed)
    shape = synth.LayerShape(1, n_query, C_, 8, T, Dc, 4, 128, (), seed=0)
    desc = tl.gpu_desc(shape, max_trigger=3)
    packed = []
    for ck in ckpts:
        d = dict(ck.weights)
        packed.append(tl.pack_layer_weights(shape, d))
    lay = tb.taq_kv_layout_of(desc)
    kv_arena = torch.zeros(n_req * lay.block_bytes, dtype=torch.uint8, device="cuda")
    reqs_data = [synth.make_request_activations(ckpts[int(c)], n_query, C_, Dc, T, seed=1000 * seed + r) for r, c in enumerate(route)]
    X = dev(np.concatenate([rd["X"] for rd in reqs_data], axis=0))
    ctx = dev(np.concatenate([rd["ctx"] for rd in reqs_data], axis=0))
    masks = [dev(rd["mask"][0]) for rd in reqs_data]
    kv_blocks = [kv_arena[r * lay.block_bytes: (r + 1) * lay.block_bytes] for r in range(n_req)]
    # admission: K/V with each request's own to_k / to_v
    t_kv = tb.make_request_table([(packed[int(c)]["Wk"], packed[int(c)]["Wv"], kv_blocks[r], masks[r]) for r, c in enumerate(route)], "cuda")
    tb.taq_kv_project_batched(desc, t_kv, n_req, ctx)
    # per-step layer
    t_fw = tb.make_request_table([(packed[int(c)]["Wq"], packed[int(c)]["Wout"], kv_blocks[r], masks[r]) for r, c in enumerate(route)], "cuda")
    y = tb.taq_layer_forward_batched(desc, t_fw, n_req, X)
    tb.taq_poll_device_status()
    y = y.cpu().numpy()
    return shape, desc, ckpts, route, reqs_data, packed, y, kv_blocks


def _check_request(shape, desc, ck, rd, P, kv_block, y_r, rows=None):
    from dataclasses import replace
    shape_r = replace(shape, trigger=ck.trigger, name=f"checkpoint{ck.ckpt_id}")
    data_r = dict(ck.weights)
    data_r.update(rd)
    tl.check_layer(shape_r, data_r, y_r, {"desc": desc, "packed": P, "kv": kv_block}, rows)


def test_batched_serving_matches_oracle_and_single_calls():
    shape, desc, ckpts, route, reqs_data, packed, y, kv_blocks = _serving_case(n_ckpt=5, n_req=8, n_query=160, C_=320, Dc=768)
    assert len(set(route.tolist())) > 1 and len({ck.trigger for ck in ckpts}) > 1
    for r, c in enumerate(route):
        ck, rd, P = ckpts[int(c)], reqs_data[r], packed[int(c)]
        _check_request(shape, desc, ck, rd, P, kv_blocks[r], y[r: r + 1])
        # the same request through the single-sequence entry points gives the same bits
        m = dev(rd["mask"])
        kv1 = tb.taq_kv_project(desc, dev(rd["ctx"]), P["Wk"], P["Wv"], m)
        y1 = tb.taq_layer_forward(desc, dev(rd["X"]), P["Wq"], P["Wout"], kv1, m).cpu().numpy()
        assert np.array_equal(y1.view(np.uint16), y[r: r + 1].view(np.uint16))


def test_batched_serving_full_size_layer_sampled():
    """Config 5's layer shape (N=4096, C=320) with 8 requests over 6 checkpoints; the oracle recomputes 128
    sampled rows of each request."""
    shape, desc, ckpts, route, reqs_data, packed, y, kv_blocks = _serving_case(n_ckpt=6, n_req=8, n_query=4096, C_=320, Dc=768, seed=1)
    rows = np.sort(np.random.default_rng(3).choice(4096, 128, replace=False))
    for r, c in enumerate(route):
        _check_request(shape, desc, ckpts[int(c)], reqs_data[r], packed[int(c)], kv_blocks[r], y[r: r + 1], rows)
