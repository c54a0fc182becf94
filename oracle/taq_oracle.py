"""CPU oracle for Trigger-Aware Quantization (TAQ) cross-attention.  TEST INFRASTRUCTURE ONLY.

This file defines the result that the CUDA path is checked against.  It is plain numpy, slow and
written to be compared with the paper by eye.  It shares no code with the CUDA path and imports
nothing from it; only tests, the smoke check and the benchmark's CPU-baseline leg may call it.  The
product never routes through it.

What it follows (paper Sec. III-B, "Trigger-Aware Quantization"):

* cross-attention per head, A = softmax(Q K^T / sqrt(d)), one K/V row per text token;
* masks M_KV and M_A that are 1 at the trigger-token positions;
* Eq. 2:  K~ = M_KV*K + (1-M_KV)*Q_a(K),  V~ likewise,  Q~ = Q_a(Q);
* Eq. 3:  A^ = M_A*A + (1-M_A)*Q_a(A);
* output O = A^ V~ (heads concatenated), then the to_out projection.

The paper leaves the quantizer Q_a ("a standard affine quantizer") open.  The reading used here,
fixed by the benchmark configuration: symmetric, dynamic, round-to-nearest-even;
  - weights: per output channel, W8 one scale per row (qmax 127), W4 one scale per group of 128
    consecutive fan-in elements (qmax 7, last group may be shorter);
  - Q, K, V: int8, one scale per row, where a row is the d elements of one token in one head;
  - attention probabilities: uint8 over the fixed range [0,1] (code = rint(255 p)), rows are not
    renormalised afterwards.
The quantizer itself is evaluated in IEEE binary32 (numpy float32, no fused multiply-add), because
integer codes are compared bit for bit; everything else is float64.

Logarithmic quantizer (``p_log``): Table 4 of the paper has "Logarithmic" rows and the text never defines that
quantizer.  ``quantize_prob_log`` is this reading's definition (power-of-two codes, see its docstring): PARITY
UNPINNED - its tests check it against closed forms of that definition, not against anything the paper fixes.

Integer activations (``a_bits = 8``): the paper's W/A bit-widths (Table 1, "W/A" column) and its BOPs
accounting count activation bits for every layer, which read literally means that the inputs of the four
projections - the hidden states X, the text context and the attention output O - are quantized too.  With
``a_bits = 8`` each token's row of all C (or Dc) channels passes through the same symmetric int8 quantizer
before its projection, so that a projection is an integer product scaled by (row scale) x (weight scale).
``a_bits = 0`` (the default, and the configuration the benchmark names) leaves these inputs in fp16.

Two modes.  ``ideal``: the equations in real (float64) arithmetic, quantizers as above, no other
rounding.  ``contract``: the same, plus a round-to-nearest-even to fp16 wherever the layer stores an
fp16 value ("full precision" of the trigger pathway is fp16 storage; dequantized V rows are fp16
matrix operands; O and Y are fp16 tensors).  Dequantized weights are exact in both modes (w^ = q * s).  The CUDA path is graded
against ``contract``.

Pins (tests/test_oracle_*.py, no GPU): empty mask == separately written uniform quantized
attention; all-trigger mask + unquantized weights + unquantized Q == textbook float64 attention;
quantizer idempotence, error bound and power-of-two equivariance; trigger rows unchanged; closed
forms (zero queries, one key, dominant key, equal value rows); permutation structure; brute force
over the masked formulas on tiny shapes; BOPs ratios of Table 1.
Parity unpinned: image-level quality (FID / CLIP of Tables 1, 4, 5) - needs data that is not here.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, Optional, Tuple

import numpy as np

F32 = np.float32
F64 = np.float64


# ----------------------------------------------------------------------------------------------
# Quantizers (binary32 arithmetic on purpose)
# ----------------------------------------------------------------------------------------------

def quantize_rows(x: np.ndarray, qmax: int) -> Tuple[np.ndarray, np.ndarray]:
    """Symmetric per-row quantizer Q_a over the last axis.

    a = max|x_i|;  s = a / qmax;  q_i = clamp(rint(x_i / s), -qmax, qmax);  an all-zero row has
    s = 0 and all codes 0.  All in float32; rint rounds half to even.
    Returns (codes int32, scales float32 with the last axis removed).
    """
    x = np.asarray(x, dtype=F32)
    a = np.max(np.abs(x), axis=-1)
    s = (a / F32(qmax)).astype(F32)
    safe = np.where(s == 0, F32(1), s)[..., None]
    q = np.rint((x / safe).astype(F32))
    q = np.clip(q, -qmax, qmax).astype(np.int32)
    q = np.where(s[..., None] == 0, 0, q).astype(np.int32)
    return q, s


def dequantize_rows(codes: np.ndarray, scales: np.ndarray) -> np.ndarray:
    """x^_i = float32(q_i) * s in float32."""
    return (codes.astype(F32) * np.asarray(scales, dtype=F32)[..., None]).astype(F32)


def quantize_weights(W: np.ndarray, bits: int, group: int) -> Tuple[np.ndarray, np.ndarray]:
    """Per-output-channel symmetric round-to-nearest weight quantizer.

    W is [n_out, k_in] float32.  ``group`` == 0: one scale per output channel; otherwise one scale
    per ``group`` consecutive fan-in elements of a channel (the last group may be ragged).
    Returns (codes int32 [n_out, k_in], scales float32 [n_out, n_groups]).
    """
    if bits == 8:
        qmax = 127
    elif bits == 4:
        qmax = 7
    else:
        raise ValueError("bits must be 4 or 8")
    W = np.asarray(W, dtype=F32)
    n_out, k_in = W.shape
    g = k_in if group == 0 else group
    n_groups = (k_in + g - 1) // g
    codes = np.zeros((n_out, k_in), dtype=np.int32)
    scales = np.zeros((n_out, n_groups), dtype=F32)
    for gi in range(n_groups):
        lo, hi = gi * g, min(k_in, (gi + 1) * g)
        q, s = quantize_rows(W[:, lo:hi], qmax)
        codes[:, lo:hi] = q
        scales[:, gi] = s
    return codes, scales


def dequantize_weights(codes: np.ndarray, scales: np.ndarray, group: int, contract: bool) -> np.ndarray:
    """w^ = q * s per group: the exact product, in both modes.  The layer multiplies by the integer codes
    and applies the scale of each group to that group's partial sum, so no rounding sits between the
    code and the product (``contract`` is kept in the signature for symmetry with the other steps)."""
    n_out, k_in = codes.shape
    g = k_in if group == 0 else group
    s_full = np.repeat(scales, g, axis=1)[:, :k_in]
    return codes.astype(F64) * s_full.astype(F64)


def quantize_prob(A: np.ndarray, bits: int = 8) -> Tuple[np.ndarray, np.ndarray]:
    """Unsigned quantizer of attention probabilities over [0,1] with 2^bits levels: code = rint(pmax p) in
    float32 with pmax = 2^bits - 1 (255 for uint8, 15 for the 4-bit rows of Table 1), p^ = float32(code) / pmax.
    Returns (codes int32, p^ float64)."""
    pmax = F32(2 ** bits - 1)
    p = np.asarray(A, dtype=F32)
    code = np.rint((p * pmax).astype(F32))
    code = np.clip(code, 0, int(pmax)).astype(np.int32)
    p_hat = (code.astype(F32) / pmax).astype(F32)
    return code, p_hat.astype(F64)


def quantize_prob_log(A: np.ndarray, bits: int = 8) -> Tuple[np.ndarray, np.ndarray]:
    """Logarithmic quantizer of attention probabilities (the "Logarithmic" rows of Table 4).  The paper names it and
    never defines it; the reading taken here is the usual power-of-two code for softmax outputs:
    code = clamp(rint(-log2 p), 0, 2^bits - 1) taken in float32, p^ = 2^-code (p = 0 takes the last code).
    PARITY UNPINNED: the definition is this reading's, not the paper's.  Returns (codes int32, p^ float64)."""
    cmax = 2 ** bits - 1
    p = np.asarray(A, dtype=F32)
    with np.errstate(divide="ignore"):
        x = (-np.log2(p)).astype(F32)
    code = np.where(p > 0, np.clip(np.rint(x), 0, cmax), cmax).astype(np.int32)
    return code, np.ldexp(F64(1.0), -code)


def f16_round(x: np.ndarray) -> np.ndarray:
    """Round to nearest-even fp16, returned as float64."""
    return np.asarray(x).astype(np.float16).astype(F64)


# ----------------------------------------------------------------------------------------------
# The layer
# ----------------------------------------------------------------------------------------------

@dataclass
class TaqConfig:
    heads: int
    w_bits: int = 8          # 0 = weights left unquantized
    w_group: int = 0
    q_bits: int = 8          # 8 = Eq. 2's Q~ = Q_a(Q); 0 = Q left unquantized
    kv_bits: int = 8         # 8 / 4 = non-trigger K/V rows int8 / 4-bit (qmax 7); 0 = no K/V quantization at all
    p_bits: int = 8          # 8 / 4 = non-trigger probabilities uint8 / 4-bit (15 levels); 0 = no probability quantization
    a_bits: int = 0          # 8 = inputs of the projections (X, ctx, O) int8 per token; 0 = left in fp16
    p_log: bool = False      # non-trigger probabilities through the logarithmic quantizer (p_bits levels) instead of the linear one
    contract: bool = True    # fp16 storage roundings on (contract) or off (ideal)


def effective_weight(W: np.ndarray, cfg: TaqConfig) -> np.ndarray:
    """The weight matrix the projections actually multiply by (float64)."""
    if cfg.w_bits == 0:
        return np.asarray(W, dtype=F64)
    codes, scales = quantize_weights(W, cfg.w_bits, cfg.w_group)
    return dequantize_weights(codes, scales, cfg.w_group, cfg.contract)


def quantize_activations(x: np.ndarray, cfg: TaqConfig) -> np.ndarray:
    """Input of a projection under ``a_bits``: x~ = q * s with (q, s) = Q_a(row), one row per token over all of
    its channels; the product is exact (the projection multiplies the integer codes and applies s afterwards)."""
    x = np.asarray(x, dtype=F64)
    if cfg.a_bits == 0:
        return x
    if cfg.a_bits != 8:
        raise ValueError("a_bits must be 0 or 8")
    codes, scales = quantize_rows(x.astype(F32), 127)
    return codes.astype(F64) * scales.astype(F64)[..., None]


def split_heads(x: np.ndarray, heads: int) -> np.ndarray:
    """[B, L, C] -> [B, H, L, d] with head h owning channels h*d .. (h+1)*d-1."""
    B, L, C = x.shape
    d = C // heads
    return x.reshape(B, L, heads, d).transpose(0, 2, 1, 3)


def merge_heads(x: np.ndarray) -> np.ndarray:
    B, H, L, d = x.shape
    return x.transpose(0, 2, 1, 3).reshape(B, L, H * d)


def taq_kv(ctx: np.ndarray, Wk: np.ndarray, Wv: np.ndarray, mask_kv: np.ndarray, cfg: TaqConfig) -> Dict[str, np.ndarray]:
    """Text keys/values and Eq. 2 (first two lines).

    ctx [B,T,Dc] (fp16 data), Wk/Wv [C,Dc] float32, mask_kv [B,T] (1 = trigger row kept).
    Returns K~, V~ as float64 [B,H,T,d] plus the integer codes / scales of the quantized rows.
    """
    ctx = quantize_activations(ctx, cfg)
    K = split_heads(ctx @ effective_weight(Wk, cfg).T, cfg.heads)
    V = split_heads(ctx @ effective_weight(Wv, cfg).T, cfg.heads)
    M = (np.asarray(mask_kv) != 0)[:, None, :, None]           # broadcast over heads and channels
    out: Dict[str, np.ndarray] = {"K": K, "V": V}
    for name, Z in (("K", K), ("V", V)):
        kept = f16_round(Z) if cfg.contract else Z               # trigger rows: stored fp16
        if cfg.kv_bits == 0:
            Zt = np.where(M, kept, Z)
            codes = np.zeros(Z.shape, dtype=np.int32)
            scales = np.zeros(Z.shape[:-1], dtype=F32)
        else:
            if cfg.kv_bits not in (4, 8):
                raise ValueError("kv_bits must be 0, 4 or 8")
            codes, scales = quantize_rows(Z.astype(F32), 127 if cfg.kv_bits == 8 else 7)
            Zq = dequantize_rows(codes, scales).astype(F64)
            Zt = np.where(M, kept, Zq)                            # Eq. 2
        out[name + "_tilde"] = Zt
        out[name + "_codes"] = codes
        out[name + "_scales"] = scales
    return out


def taq_q(X: np.ndarray, Wq: np.ndarray, cfg: TaqConfig) -> Dict[str, np.ndarray]:
    """Query projection and Eq. 2 (third line): Q~ = Q_a(Q) per (batch, head, token) row."""
    X = quantize_activations(X, cfg)
    Q = split_heads(X @ effective_weight(Wq, cfg).T, cfg.heads)
    if cfg.q_bits == 0:
        Qt = f16_round(Q) if cfg.contract else Q                  # unquantized Q is an fp16 tensor
        return {"Q": Q, "Q_tilde": Qt}
    codes, scales = quantize_rows(Q.astype(F32), 127)
    return {"Q": Q, "Q_tilde": dequantize_rows(codes, scales).astype(F64), "Q_codes": codes, "Q_scales": scales}


def taq_attention(Q_tilde: np.ndarray, K_tilde: np.ndarray, V_tilde: np.ndarray, mask_a: np.ndarray,
                  cfg: TaqConfig, return_probs: bool = False):
    """A = softmax(Q~ K~^T / sqrt(d)), Eq. 3, O = A^ V~.

    Q~ [B,H,N,d], K~/V~ [B,H,T,d] float64; mask_a [B,T] (1 = trigger column kept), the same for
    every head and query row.  Returns O [B,N,C] float64 (fp16-rounded in contract mode).
    """
    B, H, N, d = Q_tilde.shape
    M = (np.asarray(mask_a) != 0)[:, None, None, :]
    S = np.einsum("bhnd,bhtd->bhnt", Q_tilde, K_tilde) / np.sqrt(F64(d))
    S = S - S.max(axis=-1, keepdims=True)
    E = np.exp(S)
    A = E / E.sum(axis=-1, keepdims=True)
    # Trigger columns are kept in fp16.  The stored probability tensor uses one unit for all columns, 1/pmax
    # (1/255 for uint8 codes): ordinary columns hold the integer code, trigger columns hold fp16(pmax A).
    if cfg.p_bits not in (0, 4, 8):
        raise ValueError("p_bits must be 0, 4 or 8")
    pmax = float(2 ** cfg.p_bits - 1) if cfg.p_bits else 255.0
    if cfg.p_log and cfg.p_bits:
        pmax = 256.0                                              # power-of-two codes sit on a power-of-two unit
    kept = f16_round(A * pmax) / pmax if cfg.contract else A
    if cfg.p_bits == 0:
        A_hat = np.where(M, kept, A)
    elif cfg.p_log:
        _, Aq = quantize_prob_log(A, cfg.p_bits)
        if cfg.contract:
            Aq = f16_round(Aq * pmax) / pmax                      # fp16 operand: codes beyond 32 flush to zero
        A_hat = np.where(M, kept, Aq)
    else:
        _, Aq = quantize_prob(A, cfg.p_bits)
        A_hat = np.where(M, kept, Aq)                             # Eq. 3
    if cfg.contract:
        # Dequantized non-trigger V rows are fp16 matrix operands; trigger rows already are fp16.
        V_tilde = f16_round(V_tilde)
    O = merge_heads(np.einsum("bhnt,bhtd->bhnd", A_hat, V_tilde))
    if cfg.contract:
        O = f16_round(O)
    return (O, A, A_hat) if return_probs else O


def taq_out(O: np.ndarray, Wout: np.ndarray, bout: Optional[np.ndarray], cfg: TaqConfig) -> np.ndarray:
    Y = quantize_activations(O, cfg) @ effective_weight(Wout, cfg).T
    if bout is not None:
        Y = Y + np.asarray(bout, dtype=F64)
    return f16_round(Y) if cfg.contract else Y


def taq_layer(X, ctx, Wq, Wk, Wv, Wout, bout, mask, cfg: TaqConfig, mask_a=None) -> Dict[str, np.ndarray]:
    """One full TAQ cross-attention layer: to_q, to_k/to_v on the text, Eq. 2, softmax, Eq. 3,
    P.V, to_out.  ``mask`` [B,T] marks the trigger span (M_KV); ``mask_a`` defaults to the same
    positions (M_A marks the same token indices)."""
    mask_a = mask if mask_a is None else mask_a
    kv = taq_kv(ctx, Wk, Wv, mask, cfg)
    q = taq_q(X, Wq, cfg)
    O = taq_attention(q["Q_tilde"], kv["K_tilde"], kv["V_tilde"], mask_a, cfg)
    Y = taq_out(O, Wout, bout, cfg)
    return {"Y": Y, "O": O, **{k: v for k, v in q.items()}, **{k: v for k, v in kv.items()}}


def token_sensitivity(X, ctx, Wq, Wk, Wv, Wout, bout, cfg: TaqConfig, bits: int) -> np.ndarray:
    """Per-token quantization sensitivity, Eq. 1, restated at the level of one layer: Delta_i(b) is the mean
    squared difference between the layer output with ONLY the K and V rows of text token i quantized to b bits
    and the output y* with no K/V row quantized.  Everything else is as ``cfg`` says in both runs (the paper
    keeps it in full precision: pass w_bits = q_bits = 0); attention probabilities are not quantized in either
    run (M_A all ones: the experiment touches K and V only).  Returns Delta [T], averaged over the batch."""
    from dataclasses import replace
    B, T = np.asarray(ctx).shape[:2]
    ones = np.ones((B, T), dtype=np.uint8)
    c = replace(cfg, kv_bits=bits)
    y_star = taq_layer(X, ctx, Wq, Wk, Wv, Wout, bout, ones, c, mask_a=ones)["Y"]
    delta = np.zeros(T, dtype=F64)
    for i in range(T):
        m = ones.copy()
        m[:, i] = 0                                                # only token i's K/V rows pass through Q_b
        y = taq_layer(X, ctx, Wq, Wk, Wv, Wout, bout, m, c, mask_a=ones)["Y"]
        delta[i] = np.mean((y - y_star) ** 2)
    return delta


# ----------------------------------------------------------------------------------------------
# Cost accounting quoted by the paper
# ----------------------------------------------------------------------------------------------

def bops(flops: float, b_w: int, b_a: int) -> float:
    """BOPs = FLOPs * b_w * b_a (paper, "Automatic Benchmarks")."""
    return flops * b_w * b_a


def packed_weight_bits(n_out: int, k_in: int, bits: int, group: int) -> int:
    """Storage of one packed matrix: codes plus one fp32 scale per (channel, group)."""
    g = k_in if group == 0 else group
    return n_out * k_in * bits + n_out * ((k_in + g - 1) // g) * 32
