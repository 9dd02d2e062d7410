"""CPU fp64 oracle for the VeriLLM verifier path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, obviously-correct numpy implementation of what the verifier computes:
the teacher-forced causal forward pass of a Llama-style decoder over [prompt || output]
(paper Eq. 1 and the "Prefill Computation" paragraph: S_{i+1}^{(t)} = F_i(S_i^{(t)}; W_i)
for all t at once), its token-by-token twin with a KV cache (the prover's decode loop of
the "Inference Scheme" section), the element-wise comparison statistics (the
"Comparison and On-Chain Commitment" paragraph, the offline test battery T_off of the
quantization-attack analysis, and the bit-aware statistical comparison of the evaluation
section) and the accept/reject verdict (b = 1[T_v <= tau]; Slash iff some delta > eps).

Only tests, the smoke check and the benchmark's CPU-baseline leg may import this file.
It shares no code with the CUDA path and never receives values computed by it.

Arithmetic is float64 throughout; weights given as bf16 bit patterns (uint16) or float32
are widened exactly.  No blocking, fusion or reordering beyond the definitions.

Parity pins (tests/test_oracle_pins.py): prefill == decode position by position, causal
prefix invariance, softmax rows sum to one, T=1 closed form, RoPE relative-position
invariance / identity at 0 / norm preservation, RMSNorm scale invariance, GQA == MHA with
replicated K/V heads, zeroed-projection closed forms, batch independence, an independent
library implementation of the same architecture (transformers' LlamaModel in float64),
hand-worked comparison vectors, and the bin bookkeeping of the paper's Tables 1-2.
"parity unpinned": the numeric acceptance thresholds of the bit-aware test (P_e, P_m, P_w,
e) were calibrated by the paper on its own model and hardware; nothing in the paper fixes
what they should be for bf16 random-init traces, so only their direction and bookkeeping
are pinned.
"""
from __future__ import annotations

import dataclasses
from typing import Dict, List, Optional, Sequence

import numpy as np

TINY = 1e-30

# ----------------------------------------------------------------------------- number formats


def widen_bf16_bits(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exactly (bf16 is the top half of a float32)."""
    u32 = bits.astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


def as_f64(w: np.ndarray) -> np.ndarray:
    if w.dtype == np.uint16:
        return widen_bf16_bits(w)
    return np.asarray(w, dtype=np.float64)


def round_to_bf16(x: np.ndarray) -> np.ndarray:
    """Round float64 values to the nearest bf16 value (ties to even); result kept as float64.

    bf16: 1 sign, 8 exponent, 7 mantissa bits.  A normal value m*2^e (0.5 <= |m| < 1) is a
    multiple of 2^(e-8); below 2^-126 the spacing stays 2^-133 (subnormals)."""
    x = np.asarray(x, dtype=np.float64)
    out = np.array(x, copy=True)
    fin = np.isfinite(x) & (x != 0.0)
    if np.any(fin):
        xf = x[fin]
        _, e = np.frexp(xf)
        q = np.ldexp(1.0, np.maximum(e - 8, -133))
        r = np.rint(xf / q) * q
        r = np.where(np.abs(r) >= np.ldexp(1.0, 128), np.copysign(np.inf, r), r)
        out[fin] = r
    return out


def round_to_f32(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)


def round_to(x: np.ndarray, dtype: str) -> np.ndarray:
    if dtype == "bf16":
        return round_to_bf16(x)
    if dtype == "f32":
        return round_to_f32(x)
    raise ValueError(dtype)


def float_fields(x_rounded: np.ndarray, dtype: str):
    """(sign, raw biased exponent field, mantissa field, mantissa bits) of values that are
    already representable in `dtype`."""
    with np.errstate(over="ignore"):
        u = np.asarray(x_rounded, dtype=np.float64).astype(np.float32).view(np.uint32).astype(np.int64)
    sign = (u >> 31) & 1
    expo = (u >> 23) & 0xFF
    if dtype == "bf16":
        return sign, expo, (u >> 16) & 0x7F, 7
    return sign, expo, u & 0x7FFFFF, 23


# ----------------------------------------------------------------------------- model


@dataclasses.dataclass
class Model:
    """`layers` is any sequence of per-layer weight dicts (float64); it may generate them on access."""

    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    rope_base: float
    rms_eps: float
    embed: np.ndarray  # [vocab or n_rows, d_model]
    final_norm: np.ndarray
    layers: List[Dict[str, np.ndarray]]  # each: attn_norm, wq, wk, wv, wo, ffn_norm, w_gate, w_up, w_down
    embed_rows: Optional[Dict[int, int]] = None  # token id -> row of `embed` when only some rows are held


def make_model(shape, embed, final_norm, layers, embed_rows=None) -> Model:
    """`shape`: any object with the ModelShape attribute names.  Weights: float arrays or bf16 bits,
    every projection [out_features, in_features]."""
    return Model(
        shape.n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
        shape.vocab, float(shape.rope_base), float(shape.rms_eps),
        as_f64(embed), as_f64(final_norm), [{k: as_f64(v) for k, v in lw.items()} for lw in layers],
        embed_rows,
    )


def embed_tokens(m: Model, tokens: np.ndarray) -> np.ndarray:
    """S_1 = Embed(x) (Inference Scheme, first line of the per-step equations)."""
    if m.embed_rows is not None:
        idx = np.array([m.embed_rows[int(t)] for t in tokens], dtype=np.int64)
    else:
        idx = np.asarray(tokens, dtype=np.int64)
    return m.embed[idx].copy()


def rmsnorm(x: np.ndarray, gamma: np.ndarray, eps: float) -> np.ndarray:
    """x * rsqrt(mean(x^2) + eps) * gamma over the last axis."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps) * gamma


def rope(x: np.ndarray, positions: np.ndarray, base: float) -> np.ndarray:
    """Rotary embedding, half-split pairing: element i pairs with i + dh/2, angle p * base^(-2i/dh).

    x: [T, n_heads, dh]; positions: [T]."""
    dh = x.shape[-1]
    half = dh // 2
    inv_freq = base ** (-2.0 * np.arange(half, dtype=np.float64) / dh)
    ang = np.asarray(positions, dtype=np.float64)[:, None] * inv_freq[None, :]  # [T, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    x1, x2 = x[..., :half], x[..., half:]
    return np.concatenate([x1 * c - x2 * s, x2 * c + x1 * s], axis=-1)


def softmax_rows(s: np.ndarray) -> np.ndarray:
    s = s - np.max(s, axis=-1, keepdims=True)
    e = np.exp(s)
    return e / np.sum(e, axis=-1, keepdims=True)


def causal_attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, probs_out: Optional[list] = None) -> np.ndarray:
    """softmax(q k^T / sqrt(dh) + causal mask) v per head; query head g reads KV head g*KV//H.

    q: [T, H, dh]; k, v: [T, KV, dh] -> [T, H, dh]."""
    T, H, dh = q.shape
    KV = k.shape[1]
    out = np.empty_like(q)
    mask = np.triu(np.ones((T, T), dtype=bool), k=1)  # j > p is masked
    for g in range(H):
        kv = g * KV // H
        s = q[:, g, :] @ k[:, kv, :].T / np.sqrt(float(dh))
        s = np.where(mask, -np.inf, s)
        w = softmax_rows(s)
        if probs_out is not None:
            probs_out.append(w)
        out[:, g, :] = w @ v[:, kv, :]
    return out


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def layer_forward(m: Model, w: Dict[str, np.ndarray], h: np.ndarray, positions: np.ndarray) -> np.ndarray:
    """One pre-norm block F_l with weights w on a whole sequence h: [T, d_model] -> [T, d_model]."""
    T = h.shape[0]
    a = rmsnorm(h, w["attn_norm"], m.rms_eps)
    q = (a @ w["wq"].T).reshape(T, m.n_heads, m.head_dim)
    k = (a @ w["wk"].T).reshape(T, m.n_kv_heads, m.head_dim)
    v = (a @ w["wv"].T).reshape(T, m.n_kv_heads, m.head_dim)
    q = rope(q, positions, m.rope_base)
    k = rope(k, positions, m.rope_base)
    o = causal_attention(q, k, v).reshape(T, m.n_heads * m.head_dim)
    u = h + o @ w["wo"].T
    f = rmsnorm(u, w["ffn_norm"], m.rms_eps)
    return u + (silu(f @ w["w_gate"].T) * (f @ w["w_up"].T)) @ w["w_down"].T


def forward_segment_batch(m: Model, states_in: Sequence[np.ndarray], layer_begin: int, layer_end: int) -> List[np.ndarray]:
    """Segment-local pass: S_{i+1}^{(t)} = F_i(S_i^{(t)}; W_i) for all t, for the blocks layer_begin .. layer_end-1,
    starting from given input states (one [T_b, d_model] array per sequence: the recorded upstream states
    of a verifier's segment, or the embeddings for the first segment).

    Returns one [layer_end - layer_begin, T_b, d_model] array per sequence.  Sequences never interact; the
    loop runs layer by layer over all of them only so that `m.layers` may be a lazy sequence that
    materialises one layer's weights at a time."""
    hs = [np.array(h, dtype=np.float64, copy=True) for h in states_in]
    n = layer_end - layer_begin
    out = [np.empty((n, h.shape[0], m.d_model), dtype=np.float64) for h in hs]
    for l in range(layer_begin, layer_end):
        w = m.layers[l]
        for b in range(len(hs)):
            hs[b] = layer_forward(m, w, hs[b], np.arange(hs[b].shape[0]))
            out[b][l - layer_begin] = hs[b]
    return out


def forward_prefill_batch(m: Model, seqs: Sequence[np.ndarray]) -> List[np.ndarray]:
    """All layer-output states of every sequence, each in a single causal pass (Eq. 1).

    Returns one [n_layers, T_b, d_model] array per sequence: entry l is the residual stream after
    block l+1, i.e. the boundary state S_{l+2} in the paper's numbering, before the final norm."""
    return forward_segment_batch(m, [embed_tokens(m, np.asarray(t)) for t in seqs], 0, m.n_layers)


def forward_prefill(m: Model, tokens: np.ndarray) -> np.ndarray:
    """One sequence: [n_layers, T, d_model]."""
    return forward_prefill_batch(m, [tokens])[0]


def forward_decode_kvcache(m: Model, tokens: np.ndarray, precision: str = "f64") -> np.ndarray:
    """The prover's loop: one position at a time, keys/values of earlier positions taken from a cache.

    precision "f64": exact twin of forward_prefill (brute-force check of the paper's equivalence claim).
    precision "bf16": emulates a bf16 serving stack: the normed activations, rotated q/k, v, the
    attention output and the FFN product are rounded to bf16 where such a stack stores them
    (so the cache holds bf16 keys/values); accumulation and the residual stream stay wide.
    Returns [n_layers, T, d_model] (not rounded; the caller serialises)."""
    rnd = (lambda x: x) if precision == "f64" else round_to_bf16
    T = len(tokens)
    H, KV, dh = m.n_heads, m.n_kv_heads, m.head_dim
    kc = np.zeros((m.n_layers, T, KV, dh))
    vc = np.zeros((m.n_layers, T, KV, dh))
    states = np.empty((m.n_layers, T, m.d_model), dtype=np.float64)
    for t in range(T):
        h = embed_tokens(m, tokens[t : t + 1])[0]
        p = np.array([t])
        for l in range(m.n_layers):
            w = m.layers[l]
            a = rnd(rmsnorm(h, w["attn_norm"], m.rms_eps))
            q = rnd(rope((w["wq"] @ a).reshape(1, H, dh), p, m.rope_base))[0]
            kc[l, t] = rnd(rope((w["wk"] @ a).reshape(1, KV, dh), p, m.rope_base))[0]
            vc[l, t] = rnd((w["wv"] @ a).reshape(KV, dh))
            o = np.empty((H, dh))
            for g in range(H):
                kv = g * KV // H
                s = kc[l, : t + 1, kv, :] @ q[g] / np.sqrt(float(dh))
                wgt = softmax_rows(s[None, :])[0]
                o[g] = wgt @ vc[l, : t + 1, kv, :]
            u = h + w["wo"] @ rnd(o.reshape(-1))
            f = rnd(rmsnorm(u, w["ffn_norm"], m.rms_eps))
            h = u + w["w_down"] @ rnd(silu(w["w_gate"] @ f) * (w["w_up"] @ f))
            states[l, t] = h
    return states


# ----------------------------------------------------------------------------- comparison

STAT_NAMES = (
    "rel_l2", "max_abs", "mae", "mean_signed", "p_e", "p_m", "p_w", "q_small", "z_large",
    "n_exp_mismatch", "n_mant_large", "n_mant_small", "n_exact", "n_nonfinite", "l2_delta", "l2_ref",
)
NSTAT = len(STAT_NAMES)


@dataclasses.dataclass
class Tol:
    """Tolerances.  A float test with threshold <= 0 is disabled; the bit-aware tests run only
    when `bit_aware` is set (their thresholds were calibrated by the paper on its own setup)."""

    rel_l2: float = 5e-2
    max_abs: float = 0.0
    mae: float = 0.0
    pe_max: float = 0.05
    pm_min: float = 0.75
    pw_min: float = 0.80
    e_abs_max: float = 0.01
    e_w: float = 1e-2
    e_m: int = 7
    tau_large: float = 0.0
    z_large_max: float = -1.0  # < 0 disables
    q_small_min: float = 0.0  # <= 0 disables
    bit_aware: bool = False


def compare_stats(h: np.ndarray, c: np.ndarray, commit_dtype: str, tol: Tol) -> np.ndarray:
    """Deviation statistics of recomputed states h against committed states c.

    h, c: [..., d]; returns [..., NSTAT] in STAT_NAMES order.
    Delta = h - c (Comparison paragraph); mae is phi = mean |Delta|; mean_signed is the bit-aware
    test's mean discrepancy e; p_e / q_small / z_large / mae are the battery T_off; p_m and p_w
    follow the exponent-first checks: among exponent mismatches the fraction whose mantissa
    fields differ by more than e_m; among exponent matches the fraction whose significands
    differ by at most e_w * 2^mantissa_bits.  0/0 fractions are reported as 1 for p_w and p_m
    (a vacuous pass).  Threshold decisions on |Delta| are taken on the float32 difference of the
    float32 operands, the precision a GPU verifier holds them in."""
    h = np.asarray(h, dtype=np.float64)
    c = np.asarray(c, dtype=np.float64)
    d = h.shape[-1]
    finite = np.isfinite(h) & np.isfinite(c)
    n_nonfinite = np.sum(~finite, axis=-1)
    hz = np.where(finite, h, 0.0)
    cz = np.where(finite, c, 0.0)
    delta = hz - cz
    sum_sq = np.sum(delta * delta, axis=-1)
    ref_sq = np.sum(cz * cz, axis=-1)
    l2_delta, l2_ref = np.sqrt(sum_sq), np.sqrt(ref_sq)
    rel_l2 = l2_delta / np.maximum(l2_ref, TINY)
    max_abs = np.max(np.abs(delta), axis=-1)
    mae = np.sum(np.abs(delta), axis=-1) / d
    mean_signed = np.sum(delta, axis=-1) / d

    with np.errstate(over="ignore", invalid="ignore"):
        d32 = (hz.astype(np.float32) - cz.astype(np.float32)).astype(np.float32)
    a32 = np.abs(d32)
    q_small = np.sum(finite & (a32 <= np.float32(1e-5)), axis=-1) / d
    z_large = np.sum(finite & (a32 > np.float32(tol.tau_large)), axis=-1) / d

    hr, cr = round_to(hz, commit_dtype), round_to(cz, commit_dtype)
    sh, eh, mh, mbits = float_fields(hr, commit_dtype)
    sc, ec, mc, _ = float_fields(cr, commit_dtype)
    mismatch = finite & (eh != ec)
    match = finite & (eh == ec)
    one = 1 << mbits
    sig_h = np.where(eh != 0, one, 0) + mh
    sig_c = np.where(ec != 0, one, 0) + mc
    sig_h = np.where(sh == 1, -sig_h, sig_h)
    sig_c = np.where(sc == 1, -sig_c, sig_c)
    dev_match = np.abs(sig_h - sig_c)
    thr_w = float(np.float32(tol.e_w) * np.float32(one))
    small_in_match = match & (dev_match.astype(np.float64) <= thr_w)
    large_in_mismatch = mismatch & (np.abs(mh - mc) > int(tol.e_m))
    exact = finite & (sh == sc) & (eh == ec) & (mh == mc)

    n_mis = np.sum(mismatch, axis=-1)
    n_match = np.sum(match, axis=-1)
    n_large = np.sum(large_in_mismatch, axis=-1)
    n_small = np.sum(small_in_match, axis=-1)
    p_e = n_mis / d
    p_m = np.where(n_mis > 0, n_large / np.maximum(n_mis, 1), 1.0)
    p_w = np.where(n_match > 0, n_small / np.maximum(n_match, 1), 1.0)

    cols = [rel_l2, max_abs, mae, mean_signed, p_e, p_m, p_w, q_small, z_large,
            n_mis, n_large, n_small, np.sum(exact, axis=-1), n_nonfinite, l2_delta, l2_ref]
    return np.stack([np.asarray(x, dtype=np.float64) for x in cols], axis=-1)


def layer_passes(stats: np.ndarray, tol: Tol) -> np.ndarray:
    """Boolean per stats row: every enabled test holds.  Equality with a float threshold accepts
    (b = 1[T_v <= tau]; element passes iff Delta_j <= eps); the bit-aware thresholds keep the
    paper's strict direction (P_e < ., P_m > ., P_w > ., e within the closed interval)."""
    s = {n: stats[..., i] for i, n in enumerate(STAT_NAMES)}
    ok = s["n_nonfinite"] == 0
    if tol.rel_l2 > 0:
        ok &= s["rel_l2"] <= tol.rel_l2
    if tol.max_abs > 0:
        ok &= s["max_abs"] <= tol.max_abs
    if tol.mae > 0:
        ok &= s["mae"] <= tol.mae
    if tol.z_large_max >= 0:
        ok &= s["z_large"] <= tol.z_large_max
    if tol.q_small_min > 0:
        ok &= s["q_small"] >= tol.q_small_min
    if tol.bit_aware:
        ok &= s["p_e"] < tol.pe_max
        ok &= s["p_m"] > tol.pm_min
        ok &= s["p_w"] > tol.pw_min
        ok &= np.abs(s["mean_signed"]) <= tol.e_abs_max
    return ok


def threshold_sweep(stats: np.ndarray, is_attack: np.ndarray, variants: Sequence[Tol]) -> np.ndarray:
    """Threshold Sensitivity Analysis: for each tolerance set, how many honest and attack cells its tests accept
    and reject.  stats: [n_cells, NSTAT]; is_attack: [n_cells] bool.  Returns int64 [n_variants, 4] = honest
    accepted, honest rejected, attack accepted, attack rejected.  The thresholds are taken at float32
    precision, the precision a GPU verifier holds them in (the statistics it reports are float32 too)."""
    stats = np.asarray(stats, dtype=np.float64).reshape(-1, NSTAT)
    attack = np.asarray(is_attack).astype(bool).reshape(-1)
    out = np.zeros((len(variants), 4), dtype=np.int64)
    for v, tol in enumerate(variants):
        t32 = dataclasses.replace(tol, **{f.name: float(np.float32(getattr(tol, f.name)))
                                          for f in dataclasses.fields(tol) if isinstance(getattr(tol, f.name), float)})
        ok = layer_passes(stats, t32)
        out[v] = [np.sum(ok & ~attack), np.sum(~ok & ~attack), np.sum(ok & attack), np.sum(~ok & attack)]
    return out


def detection_rates(counts: np.ndarray) -> Dict[str, np.ndarray]:
    """FPR / FNR / TPR / TNR of the table in Threshold Sensitivity Analysis from threshold_sweep's counts
    (positive = attack detected, i.e. rejected)."""
    c = np.asarray(counts, dtype=np.float64)
    honest, attack = c[:, 0] + c[:, 1], c[:, 2] + c[:, 3]
    with np.errstate(invalid="ignore", divide="ignore"):
        fpr, fnr = c[:, 1] / honest, c[:, 2] / attack
    return {"FPR": fpr, "FNR": fnr, "TPR": 1.0 - fnr, "TNR": 1.0 - fpr}


@dataclasses.dataclass
class Report:
    stats: np.ndarray  # [n_check, n_layers, NSTAT]
    pos_ok: np.ndarray  # [n_check] uint8
    first_bad_layer: np.ndarray  # [n_check] int32, -1 if none
    seq_ok: np.ndarray  # [batch] uint8
    seq_score: np.ndarray  # [batch] float64
    hidden: np.ndarray  # [n_layers, n_check, d_model] recomputed states at the checked positions


def verdict(stats: np.ndarray, check_seq: np.ndarray, batch: int, tol: Tol):
    """stats [n_check, n_layers, NSTAT] -> (pos_ok, first_bad_layer, seq_ok, seq_score).

    A position is accepted iff every layer passes; a sequence iff all its checked positions are
    accepted (the slash rule: one deviation above tolerance suffices).  The score is
    T_v = Psi({phi}) with phi = MAE of a (position, layer) cell and Psi the mean over the
    sequence's checked positions and layers; a sequence without checked positions scores 0
    and is accepted."""
    n_check, n_layers, _ = stats.shape
    ok = layer_passes(stats, tol)  # [n_check, n_layers]
    pos_ok = np.all(ok, axis=1)
    first_bad = np.where(pos_ok, -1, np.argmax(~ok, axis=1)).astype(np.int32)
    seq_ok = np.ones(batch, dtype=np.uint8)
    seq_score = np.zeros(batch, dtype=np.float64)
    mae_idx = STAT_NAMES.index("mae")
    for b in range(batch):
        sel = np.asarray(check_seq) == b
        if np.any(sel):
            seq_ok[b] = np.uint8(np.all(pos_ok[sel]))
            seq_score[b] = float(np.mean(stats[sel][:, :, mae_idx]))
    return pos_ok.astype(np.uint8), first_bad, seq_ok, seq_score


def verify_segment(
    m: Model, states_in: Sequence[np.ndarray], layer_begin: int, layer_end: int, committed: np.ndarray,
    check_seq: np.ndarray, check_pos: np.ndarray, tol: Tol, commit_dtype: str = "bf16",
) -> Report:
    """Segment verifier: recompute blocks layer_begin .. layer_end-1 from the recorded upstream states of every
    position, compare at the checked positions with the committed outputs [layer_end - layer_begin, n_check,
    d_model] and decide.  Layer indices in the report count from layer_begin."""
    committed = as_f64(committed)
    n_check = len(check_seq)
    n = layer_end - layer_begin
    hidden = np.zeros((n, n_check, m.d_model), dtype=np.float64)
    outs = forward_segment_batch(m, states_in, layer_begin, layer_end)
    for slot in range(n_check):
        hidden[:, slot, :] = outs[int(check_seq[slot])][:, int(check_pos[slot]), :]
    stats = np.transpose(compare_stats(hidden, committed, commit_dtype, tol), (1, 0, 2)).copy()
    pos_ok, first_bad, seq_ok, seq_score = verdict(stats, np.asarray(check_seq), len(states_in), tol)
    return Report(stats, pos_ok, first_bad, seq_ok, seq_score, hidden)


def merkle_root(vec: np.ndarray) -> bytes:
    """Merkle root of one hidden-state vector: leaves are SHA-256 of each entry's canonical float32 serialisation
    (4 bytes, little endian), inner nodes SHA-256(left || right); a level with an odd number of nodes pairs its
    last node with itself; a single leaf is its own root."""
    import hashlib
    import struct

    level = [hashlib.sha256(struct.pack("<f", float(np.float32(x)))).digest() for x in np.asarray(vec).reshape(-1)]
    while len(level) > 1:
        if len(level) % 2:
            level.append(level[-1])
        level = [hashlib.sha256(level[i] + level[i + 1]).digest() for i in range(0, len(level), 2)]
    return level[0]


def merkle_path(vec: np.ndarray, index: int):
    """Inclusion proof of leaf `index`: the sibling digests from the leaf level up."""
    import hashlib
    import struct

    level = [hashlib.sha256(struct.pack("<f", float(np.float32(x)))).digest() for x in np.asarray(vec).reshape(-1)]
    path = []
    while len(level) > 1:
        if len(level) % 2:
            level.append(level[-1])
        path.append(level[index ^ 1])
        level = [hashlib.sha256(level[i] + level[i + 1]).digest() for i in range(0, len(level), 2)]
        index //= 2
    return path


def spot_check(hidden: np.ndarray, sample_row, sample_col, reference, eps: float, theta: float):
    """Relaxed on-chain test on sampled scalars: Delta_j = |v_j - V_j| <= eps, p_hat = mean 1[Delta_j <= eps],
    verdict = p_hat >= theta.  The threshold decision is taken on float32 values, the precision in which the
    entries are serialised.  Returns (agree [n] uint8, p_hat, verdict)."""
    v = np.asarray(hidden)[np.asarray(sample_row), np.asarray(sample_col)].astype(np.float32)
    with np.errstate(invalid="ignore"):
        agree = np.abs(v - np.asarray(reference, dtype=np.float32)) <= np.float32(eps)
    p_hat = float(np.float32(agree.sum()) / np.float32(len(agree)))
    return agree.astype(np.uint8), p_hat, bool(np.float32(p_hat) >= np.float32(theta))


def token_match(m: Model, last_hidden: np.ndarray, lm_head: np.ndarray, claimed: np.ndarray):
    """Tail token check: TokenMatch(argmax f_LM(S_{L+1}), y) with f_LM = output head after the final RMSNorm.

    last_hidden [n, d_model] (states after the last block), lm_head [vocab, d_model] (float or bf16 bits),
    claimed [n].  Returns (argmax [n], match [n] uint8, margin [n] = best logit - runner-up).  np.argmax
    takes the lowest index among equal maxima."""
    logits = rmsnorm(np.asarray(last_hidden, dtype=np.float64), m.final_norm, m.rms_eps) @ as_f64(lm_head).T
    arg = np.argmax(logits, axis=-1)
    top2 = np.partition(logits, -2, axis=-1)[:, -2:]
    margin = top2[:, 1] - top2[:, 0]
    return arg.astype(np.int32), (arg == np.asarray(claimed)).astype(np.uint8), margin


def verify_prefill(
    m: Model, seqs: Sequence[np.ndarray], committed: np.ndarray, check_seq: np.ndarray,
    check_pos: np.ndarray, tol: Tol, commit_dtype: str = "bf16", prefix_only: bool = False,
) -> Report:
    """The verifier: recompute every sequence by one causal pass, gather the checked positions,
    compare with the committed states [n_layers, n_check, d_model] (float values already rounded
    to commit_dtype, or bf16 bits), and decide.

    prefix_only=True recomputes each sequence only up to its last checked position; under the
    causal mask later tokens cannot change earlier states (pinned by the prefix-invariance
    test), and it is what makes sampled checks of long sequences affordable on a CPU."""
    committed = as_f64(committed)
    n_check = len(check_seq)
    hidden = np.zeros((m.n_layers, n_check, m.d_model), dtype=np.float64)
    todo, prefixes = [], []
    for b, toks in enumerate(seqs):
        sel = np.nonzero(np.asarray(check_seq) == b)[0]
        if sel.size == 0:
            continue
        upto = int(np.max(np.asarray(check_pos)[sel])) + 1 if prefix_only else len(toks)
        todo.append(sel)
        prefixes.append(np.asarray(toks)[:upto])
    for sel, states in zip(todo, forward_prefill_batch(m, prefixes)):
        for slot in sel:
            hidden[:, slot, :] = states[:, int(check_pos[slot]), :]
    stats = compare_stats(hidden, committed, commit_dtype, tol)  # [n_layers, n_check, NSTAT]
    stats = np.transpose(stats, (1, 0, 2)).copy()
    pos_ok, first_bad, seq_ok, seq_score = verdict(stats, np.asarray(check_seq), len(seqs), tol)
    return Report(stats, pos_ok, first_bad, seq_ok, seq_score, hidden)
