"""Shared helpers of the GPU parity tests: run the CUDA path through the C-ABI binding on the seeded
synthetic inputs, run the CPU oracle on the same arrays, and compare."""
import numpy as np
import torch

from oracle import taq_oracle as orc
from paper_2603_22943_b200 import binding as tb
from paper_2603_22943_b200 import synth

import json
import os

# Layer-output tolerances of the parity contract (fp16 outputs against the fp64 contract-mode oracle).
TOL_MAX_ABS = 2e-2
TOL_REL_L2 = 1e-3
# A query row in which the fp32 accumulation of the GPU and the fp64 one of the oracle round one Q (or, with integer
# activations, O) code to different sides of a tie is compared end to end as well, but it is not the same computation any
# more: one code step of a row of d values moves that row's logits, and the softmax amplifies it.  Such rows must be few,
# and their error stays under a bound of its own.
TOL_MAX_ABS_TIE_ROWS = 6e-2
MAX_TIE_ROW_FRACTION = {0: 0.02, 8: 0.05}          # by a_bits (measured: at most 0.8 % and 2.8 %)


def _log_parity(record):
    """Appends one line per layer comparison to the file named by TAQ_PARITY_LOG (the figures quoted in the design notes)."""
    path = os.environ.get("TAQ_PARITY_LOG")
    if path:
        with open(path, "a") as f:
            f.write(json.dumps(record) + "\n")


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def errors(got: np.ndarray, want: np.ndarray):
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    den = np.linalg.norm(want)
    return float(np.max(np.abs(got - want))) if got.size else 0.0, float(np.linalg.norm(got - want) / den) if den > 0 else 0.0


def assert_layer_close(got, want, what=""):
    max_abs, rel = errors(got, want)
    assert max_abs <= TOL_MAX_ABS and rel <= TOL_REL_L2, f"{what}: max-abs {max_abs:.3e} (<= {TOL_MAX_ABS}), rel-L2 {rel:.3e} (<= {TOL_REL_L2})"
    return max_abs, rel


def oracle_cfg(shape: synth.LayerShape, contract=True, a_bits=0) -> orc.TaqConfig:
    return orc.TaqConfig(heads=shape.heads, w_bits=shape.w_bits, w_group=shape.w_group, q_bits=shape.q_bits, kv_bits=shape.kv_bits,
                         p_bits=shape.p_bits, contract=contract, a_bits=a_bits, p_log=bool(shape.p_log))


def oracle_layer(shape: synth.LayerShape, data, contract=True, rows=None):
    """Oracle on the whole layer, or on a subset of query rows (rows are independent)."""
    X = data["X"] if rows is None else data["X"][:, rows]
    return orc.taq_layer(X, data["ctx"], data["Wq"], data["Wk"], data["Wv"], data["Wout"], data["bout"], data["mask"],
                         oracle_cfg(shape, contract))


def gpu_desc(shape: synth.LayerShape, max_trigger=None, batch=None, n_query=None) -> tb.LayerDesc:
    mt = max(1, len(shape.trigger)) if max_trigger is None else max_trigger
    return tb.layer_desc(shape.batch if batch is None else batch, shape.n_query if n_query is None else n_query,
                         shape.channels, shape.heads, shape.n_ctx, shape.ctx_dim, shape.w_bits, shape.w_group,
                         q_bits=shape.q_bits, kv_bits=shape.kv_bits, p_bits=shape.p_bits, max_trigger=mt, p_log=shape.p_log)


def pack_layer_weights(shape: synth.LayerShape, data):
    C_, Dc = shape.channels, shape.ctx_dim
    wd_cc = tb.weight_desc(C_, C_, shape.w_bits, shape.w_group)
    wd_cd = tb.weight_desc(C_, Dc, shape.w_bits, shape.w_group)
    return {
        "Wq": tb.taq_pack_weights(wd_cc, dev(data["Wq"])),
        "Wk": tb.taq_pack_weights(wd_cd, dev(data["Wk"])),
        "Wv": tb.taq_pack_weights(wd_cd, dev(data["Wv"])),
        "Wout": tb.taq_pack_weights(wd_cc, dev(data["Wout"]), dev(data["bout"])),
        "wd_cc": wd_cc, "wd_cd": wd_cd,
    }


def gpu_layer(shape: synth.LayerShape, data, max_trigger=None, return_parts=False):
    """The whole CUDA path: pack, K/V projection with Eq. 2, then the per-step layer."""
    desc = gpu_desc(shape, max_trigger)
    P = pack_layer_weights(shape, data)
    mask = dev(data["mask"])
    kv = tb.taq_kv_project(desc, dev(data["ctx"]), P["Wk"], P["Wv"], mask)
    y = tb.taq_layer_forward(desc, dev(data["X"]), P["Wq"], P["Wout"], kv, mask)
    tb.taq_poll_device_status()
    torch.cuda.synchronize()
    if return_parts:
        return y.cpu().numpy(), {"desc": desc, "packed": P, "kv": kv, "mask": mask}
    return y.cpu().numpy()


def parse_kv_block(desc: tb.LayerDesc, kv: torch.Tensor):
    """Splits the K~/V~ blocks (layout documented in taq.h) into numpy arrays."""
    lay = tb.taq_kv_layout_of(desc)
    B, H, T, d, R = desc.batch, desc.heads, desc.n_ctx, desc.d_head, desc.max_trigger
    raw = kv.cpu().numpy().reshape(-1)[: B * lay.block_bytes].reshape(B, lay.block_bytes)
    out = {}
    for nm, oc, osc, otr in (("K", lay.off_k_codes, lay.off_k_scales, lay.off_k_trigger), ("V", lay.off_v_codes, lay.off_v_scales, lay.off_v_trigger)):
        out[nm + "_codes"] = np.stack([raw[b, oc: oc + H * T * d].view(np.int8).reshape(H, T, d) for b in range(B)])
        out[nm + "_scales"] = np.stack([raw[b, osc: osc + H * T * 4].view(np.float32).reshape(H, T) for b in range(B)])
        out[nm + "_trigger"] = np.stack([raw[b, otr: otr + R * H * d * 2].view(np.float16).reshape(R, H, d) for b in range(B)])
    out["slot"] = np.stack([raw[b, lay.off_trig_slot: lay.off_trig_slot + 512].view(np.int32) for b in range(B)])
    return out


def build_kv_block(desc: tb.LayerDesc, K_codes, K_scales, V_codes, V_scales, K_rows, V_rows, mask) -> np.ndarray:
    """Host-side packer used to feed the attention kernel with the oracle's own K~/V~ (test isolation)."""
    lay = tb.taq_kv_layout_of(desc)
    B, H, T, d, R = desc.batch, desc.heads, desc.n_ctx, desc.d_head, desc.max_trigger
    raw = np.zeros((B, lay.block_bytes), dtype=np.uint8)
    for b in range(B):
        slot = np.full(128, -1, dtype=np.int32)
        trig = [j for j in range(T) if mask[b, j]]
        assert len(trig) <= R
        kt = np.zeros((R, H, d), np.float16)
        vt = np.zeros((R, H, d), np.float16)
        kc, vc = K_codes[b].astype(np.int8).copy(), V_codes[b].astype(np.int8).copy()
        ks, vs = K_scales[b].astype(np.float32).copy(), V_scales[b].astype(np.float32).copy()
        for s, j in enumerate(trig):
            slot[j] = s
            kt[s] = K_rows[b, :, j].astype(np.float16)
            vt[s] = V_rows[b, :, j].astype(np.float16)
            kc[:, j] = 0; vc[:, j] = 0; ks[:, j] = 0; vs[:, j] = 0
        raw[b, lay.off_k_codes: lay.off_k_codes + H * T * d] = kc.reshape(-1).view(np.uint8)
        raw[b, lay.off_v_codes: lay.off_v_codes + H * T * d] = vc.reshape(-1).view(np.uint8)
        raw[b, lay.off_k_scales: lay.off_k_scales + H * T * 4] = ks.reshape(-1).view(np.uint8)
        raw[b, lay.off_v_scales: lay.off_v_scales + H * T * 4] = vs.reshape(-1).view(np.uint8)
        raw[b, lay.off_k_trigger: lay.off_k_trigger + R * H * d * 2] = kt.reshape(-1).view(np.uint8)
        raw[b, lay.off_v_trigger: lay.off_v_trigger + R * H * d * 2] = vt.reshape(-1).view(np.uint8)
        raw[b, lay.off_trig_slot: lay.off_trig_slot + 512] = slot.view(np.uint8)
    return raw.reshape(-1)


def gpu_decisions(shape: synth.LayerShape, data, parts, rows=None, a_bits=0):
    """The rounding decisions the CUDA path took upstream of the attention: K~/V~ as stored in its block and Q~
    as produced by the same dequant-GEMM kernel the layer call runs (bit-identical by determinism)."""
    desc, P = parts["desc"], parts["packed"]
    B, H, T, d = shape.batch, shape.heads, shape.n_ctx, shape.d_head
    kvg = parse_kv_block(desc, parts["kv"])
    out = {}
    for nm in ("K", "V"):
        Z = (kvg[nm + "_codes"].astype(np.float32) * kvg[nm + "_scales"][..., None]).astype(np.float64)     # [B,H,T,d]
        for b in range(B):
            for j in range(T):
                s = int(kvg["slot"][b, j])
                if s >= 0:
                    Z[b, :, j] = kvg[nm + "_trigger"][b, s].astype(np.float64)
        out[nm + "_tilde"] = Z
        out[nm + "_codes"], out[nm + "_scales"] = kvg[nm + "_codes"], kvg[nm + "_scales"]
    X = data["X"] if rows is None else data["X"][:, rows]
    n = X.shape[1]
    x2 = dev(X.reshape(B * n, shape.channels))
    if a_bits == 8:                      # the integer-activation projection, as taq_layer_forward_a8 runs it
        xc, xs = tb.taq_quantize_rows_f16(x2)
        out["X_codes"], out["X_scales"] = xc.cpu().numpy().reshape(B, n, -1), xs.cpu().numpy().reshape(B, n)
        linear = lambda kind, **kw: tb.taq_quantized_linear_i8(P["wd_cc"], xc, xs, P["Wq"], kind, **kw)
    else:
        linear = lambda kind, **kw: tb.taq_quantized_linear(P["wd_cc"], x2, P["Wq"], kind, **kw)
    if shape.q_bits == 8:
        qc, qs = linear(tb.TAQ_OUT_INT8_HEAD_ROWS, heads=H)
        qc = qc.cpu().numpy().reshape(B, n, H, d).transpose(0, 2, 1, 3)                                   # [B,H,n,d]
        qs = qs.cpu().numpy().reshape(B, n, H).transpose(0, 2, 1)                                          # [B,H,n]
        out["Q_codes"], out["Q_scales"] = qc, qs
        out["Q_tilde"] = (qc.astype(np.float32) * qs[..., None]).astype(np.float64)
    else:
        q16 = linear(tb.TAQ_OUT_F16).cpu().numpy()
        out["Q_tilde"] = q16.reshape(B, n, H, d).transpose(0, 2, 1, 3).astype(np.float64)
    return out


def assert_codes_agree(got, want, pre, scales, what, max_frac=2e-3):
    """Integer codes taken after an fp32 accumulation (GPU) and after an fp64 one (oracle) may differ by one step,
    and only where the value being rounded sits on a rounding boundary to within the accumulation error."""
    got, want = got.astype(np.int32), want.astype(np.int32)
    diff = got != want
    if not diff.any():
        return 0.0
    assert np.abs(got - want).max() <= 1, f"{what}: a code differs by more than one step"
    frac = float(diff.mean())
    assert frac <= max_frac, f"{what}: {frac:.2e} of the codes differ"
    s = np.broadcast_to(scales[..., None], pre.shape)[diff].astype(np.float64)
    boundary = (got[diff] + want[diff]) / 2.0
    dist = np.abs(pre[diff] / s - boundary)                     # in code units
    assert dist.max() < 2e-3, f"{what}: a differing code is {dist.max():.2e} steps away from its rounding boundary"
    return frac


def check_layer(shape: synth.LayerShape, data, y_gpu, parts, rows=None, a_bits=0):
    """Three-part parity of one layer call.
    (1) the integer decisions (Q, K, V codes) of the CUDA path equal the oracle's, up to near-ties;
    (2) given the same decisions, the layer output matches the oracle within the contract tolerances everywhere;
    (3) end to end against the untouched oracle: relative L2 within tolerance over everything, and max-abs within
        tolerance on every query row whose Q codes agree (a one-step flip of a near-tie is amplified by the softmax,
        which is why both sides must take that decision from the same value, as (2) does)."""
    cfg = oracle_cfg(shape, a_bits=a_bits)
    X = data["X"] if rows is None else data["X"][:, rows]
    y = y_gpu if rows is None else y_gpu[:, rows]
    kv_o = orc.taq_kv(data["ctx"], data["Wk"], data["Wv"], data["mask"], cfg)
    q_o = orc.taq_q(X, data["Wq"], cfg)
    Y_o = orc.taq_out(orc.taq_attention(q_o["Q_tilde"], kv_o["K_tilde"], kv_o["V_tilde"], data["mask"], cfg), data["Wout"], data["bout"], cfg)
    g = gpu_decisions(shape, data, parts, rows, a_bits)
    if a_bits == 8:                      # the per-token codes of X are a stand-alone quantizer's: bit-exact
        xc, xs = orc.quantize_rows(X.astype(np.float32), 127)
        assert np.array_equal(g["X_codes"], xc) and np.array_equal(g["X_scales"], xs), "X codes / scales"
    # (1)
    for b in range(data["mask"].shape[0]):                   # per sequence: every request may have its own mask
        nt = np.array([j for j in range(shape.n_ctx) if not data["mask"][b, j]], dtype=np.int64)
        if len(nt):
            for nm in ("K", "V"):
                assert_codes_agree(g[nm + "_codes"][b:b + 1][:, :, nt], kv_o[nm + "_codes"][b:b + 1][:, :, nt], kv_o[nm][b:b + 1][:, :, nt],
                                   kv_o[nm + "_scales"][b:b + 1][:, :, nt], f"{nm} codes of sequence {b}")
    flipped_rows = np.zeros(X.shape[:2], dtype=bool)
    if shape.q_bits == 8:
        assert_codes_agree(g["Q_codes"], q_o["Q_codes"], q_o["Q"], q_o["Q_scales"], "Q codes")
        np.testing.assert_allclose(g["Q_scales"], q_o["Q_scales"], rtol=2e-5)
        flipped_rows = (g["Q_codes"] != q_o["Q_codes"]).any(axis=(1, 3))               # [B,n]
    # (2)
    O_d = orc.taq_attention(g["Q_tilde"], g["K_tilde"], g["V_tilde"], data["mask"], cfg)
    Y_d = orc.taq_out(O_d, data["Wout"], data["bout"], cfg)
    if a_bits == 8:
        # one more integer decision sits downstream of the attention: the per-token codes of O.  Rows in which the K/V
        # near-ties of (1) move one of them are set aside in (3) like rows with a Q flip.
        O_o = orc.taq_attention(q_o["Q_tilde"], kv_o["K_tilde"], kv_o["V_tilde"], data["mask"], cfg)
        oc_d, _ = orc.quantize_rows(O_d.astype(np.float32), 127)
        oc_o, _ = orc.quantize_rows(O_o.astype(np.float32), 127)
        flipped_rows = flipped_rows | (oc_d != oc_o).any(axis=-1)
    same = assert_layer_close(y, Y_d, shape.name + " (same decisions)")
    # (3)
    max_abs, rel = errors(y, Y_o)
    assert rel <= TOL_REL_L2, f"{shape.name}: end-to-end rel-L2 {rel:.3e}"
    err = np.abs(y.astype(np.float64) - Y_o).max(axis=-1)                            # [B,n]: per query row
    ma_same = float(err[~flipped_rows].max()) if (~flipped_rows).any() else 0.0
    ma_tie = float(err[flipped_rows].max()) if flipped_rows.any() else 0.0
    n_tie, n_rows = int(flipped_rows.sum()), int(flipped_rows.size)
    rec = {"shape": shape.name, "a_bits": a_bits, "rows": n_rows, "rows_set_aside": n_tie, "max_abs_all_rows": max_abs, "max_abs_rows_with_equal_codes": ma_same,
           "max_abs_rows_with_a_tie": ma_tie, "rel_l2": rel, "rel_l2_same_decisions": same[1], "max_abs_same_decisions": same[0]}
    _log_parity(rec)
    print(f"parity {shape.name}: max-abs over all {n_rows} rows {max_abs:.3e}, rel-L2 {rel:.3e}; {n_tie} rows set aside (max-abs there {ma_tie:.3e})")
    assert ma_same <= TOL_MAX_ABS, f"{shape.name}: end-to-end max-abs {ma_same:.3e} on rows whose codes agree"
    assert n_tie <= MAX_TIE_ROW_FRACTION[a_bits] * n_rows + 1, f"{shape.name}: {n_tie} of {n_rows} rows have a code on the other side of a tie"
    assert ma_tie <= TOL_MAX_ABS_TIE_ROWS, f"{shape.name}: end-to-end max-abs {ma_tie:.3e} on rows with a code on the other side of a tie"
    return {"same_decisions": same, "end_to_end": (max_abs, rel), "rows_with_q_flip": n_tie, "rows": n_rows, "max_abs_all_rows": max_abs,
            "max_abs_tie_rows": ma_tie}


def assert_same_up_to_code_ties(a, b, what):
    """Two GPU routes through the same arithmetic: equal except where a sum taken in another order moved an fp16
    rounding (one ulp) or a probability code on a tie (1/255 of a value row)."""
    a = a.float().cpu().numpy().astype(np.float64)
    b = b.float().cpu().numpy().astype(np.float64)
    diff = np.abs(a - b)
    ulp = 2.0 ** -10 * np.maximum(np.abs(a), np.abs(b)) + 1e-6
    assert diff.max() <= TOL_MAX_ABS, f"{what}: max difference {diff.max():.3e} at {np.unravel_index(diff.argmax(), diff.shape)}"
    frac = float(np.mean(diff > 2 * ulp))
    assert frac <= 2e-3, f"{what}: {frac:.2e} of the values differ by more than two fp16 ulps"
    rel = np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-30)
    assert rel <= 2e-4, f"{what}: relative L2 difference {rel:.3e}"
