"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU)."""
import dataclasses
import os

import numpy as np
import pytest
import torch

from oracle import verillm_oracle as vo
from paper_2509_24257_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_shape(n_layers=2, H=4, KV=2, dh=16, d=32, F=48, vocab=50):
    return synth.ModelShape(n_layers, d, H, KV, dh, F, vocab, 10000.0, 1e-5)


def random_model(shape, seed=0, std=0.2):
    rng = np.random.default_rng(seed)
    layers = []
    for _ in range(shape.n_layers):
        lw = {}
        for name, shp in synth.layer_tensor_shapes(shape).items():
            lw[name] = 1.0 + 0.1 * rng.standard_normal(shp) if name.endswith("norm") else std * rng.standard_normal(shp)
        layers.append(lw)
    embed = rng.standard_normal((shape.vocab, shape.d_model))
    final = 1.0 + 0.1 * rng.standard_normal(shape.d_model)
    return vo.make_model(shape, embed, final, layers)


def test_prefill_equals_decode_position_by_position():
    # the paper's core claim: one causal pass reproduces every decode-step state
    shape = small_shape()
    m = random_model(shape, 1)
    toks = np.random.default_rng(2).integers(0, shape.vocab, 13)
    a = vo.forward_prefill(m, toks)
    b = vo.forward_decode_kvcache(m, toks, "f64")
    assert a.shape == (shape.n_layers, 13, shape.d_model)
    assert np.max(np.abs(a - b)) <= 1e-12 * np.max(np.abs(a))


def test_causal_prefix_invariance():
    shape = small_shape()
    m = random_model(shape, 3)
    toks = np.random.default_rng(4).integers(0, shape.vocab, 12)
    base = vo.forward_prefill(m, toks)
    other = toks.copy()
    other[7] = (other[7] + 1) % shape.vocab
    moved = vo.forward_prefill(m, other)
    assert np.array_equal(base[:, :7], moved[:, :7])  # earlier positions bit-identical
    assert np.max(np.abs(base[:, 7:] - moved[:, 7:])) > 1e-3  # position 7 and later do move
    # a truncated sequence gives the same states on the shared prefix
    short = vo.forward_prefill(m, toks[:9])
    assert np.max(np.abs(short - base[:, :9])) <= 1e-13 * np.max(np.abs(base))


def test_softmax_rows_sum_to_one_and_single_token_closed_form():
    rng = np.random.default_rng(5)
    T, H, KV, dh = 9, 4, 2, 8
    q, k, v = rng.standard_normal((T, H, dh)), rng.standard_normal((T, KV, dh)), rng.standard_normal((T, KV, dh))
    probs = []
    out = vo.causal_attention(q, k, v, probs)
    for w in probs:
        assert np.max(np.abs(w.sum(axis=-1) - 1.0)) <= 1e-14
        assert np.all(np.triu(w, 1) == 0.0)  # nothing attends to the future
    # first position attends to itself only: output = v_0 of its KV head
    for g in range(H):
        assert np.array_equal(out[0, g], v[0, g * KV // H])
    one = vo.causal_attention(q[:1], k[:1], v[:1])
    assert np.array_equal(one[0, 3], v[0, 1])


def test_attention_matches_library_sdpa():
    rng = np.random.default_rng(6)
    T, H, KV, dh = 17, 6, 2, 16
    q, k, v = rng.standard_normal((T, H, dh)), rng.standard_normal((T, KV, dh)), rng.standard_normal((T, KV, dh))
    ours = vo.causal_attention(q, k, v)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(k).permute(1, 0, 2)[None].repeat_interleave(H // KV, dim=1)
    tv = torch.from_numpy(v).permute(1, 0, 2)[None].repeat_interleave(H // KV, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2).numpy()
    assert np.max(np.abs(ours - ref)) <= 1e-12


def test_rope_properties():
    rng = np.random.default_rng(7)
    dh = 32
    q, k = rng.standard_normal((1, 1, dh)), rng.standard_normal((1, 1, dh))
    base = 500000.0

    def dot(m, n):
        return float(np.sum(vo.rope(q, np.array([m]), base) * vo.rope(k, np.array([n]), base)))

    assert abs(dot(5, 2) - dot(103, 100)) <= 1e-11  # depends on m - n only
    assert abs(dot(40, 40) - dot(0, 0)) <= 1e-11
    assert abs(dot(5, 2) - dot(2, 5)) > 1e-3  # and on its sign
    assert np.array_equal(vo.rope(q, np.array([0]), base), q)  # identity at position 0
    r = vo.rope(q, np.array([77]), base)
    assert abs(np.linalg.norm(r) - np.linalg.norm(q)) <= 1e-13
    # pairing (i, i + dh/2) and the frequency ladder, worked by hand for one pair
    x = np.zeros((1, 1, dh))
    x[0, 0, 3] = 1.0
    y = vo.rope(x, np.array([10]), base)
    ang = 10.0 * base ** (-2.0 * 3 / dh)
    expect = np.zeros(dh)
    expect[3], expect[3 + dh // 2] = np.cos(ang), np.sin(ang)
    assert np.max(np.abs(y[0, 0] - expect)) <= 1e-15


def test_rmsnorm_properties():
    rng = np.random.default_rng(8)
    x = rng.standard_normal((5, 64)) * 3.0
    g = np.ones(64)
    y = vo.rmsnorm(x, g, 0.0)
    assert np.max(np.abs(np.sqrt(np.mean(y * y, axis=-1)) - 1.0)) <= 1e-14
    assert np.max(np.abs(vo.rmsnorm(7.5 * x, g, 0.0) - y)) <= 1e-14
    g2 = 1.0 + rng.standard_normal(64)
    assert np.max(np.abs(vo.rmsnorm(x, g2, 1e-5) - vo.rmsnorm(x, g, 1e-5) * g2)) <= 1e-14
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (64,), torch.from_numpy(g2), 1e-5).numpy()
    assert np.max(np.abs(vo.rmsnorm(x, g2, 1e-5) - ref)) <= 1e-13


def test_gqa_equals_mha_with_replicated_kv_heads():
    shape = small_shape(H=4, KV=2)
    m = random_model(shape, 9)
    rep = shape.n_heads // shape.n_kv_heads
    mha_shape = dataclasses.replace(shape, n_kv_heads=shape.n_heads)
    layers = []
    for lw in m.layers:
        lw2 = dict(lw)
        for nm in ("wk", "wv"):
            w = lw[nm].reshape(shape.n_kv_heads, shape.head_dim, shape.d_model)
            lw2[nm] = np.repeat(w, rep, axis=0).reshape(shape.n_heads * shape.head_dim, shape.d_model)
        layers.append(lw2)
    m2 = vo.make_model(mha_shape, m.embed, m.final_norm, layers)
    toks = np.random.default_rng(10).integers(0, shape.vocab, 11)
    a, b = vo.forward_prefill(m, toks), vo.forward_prefill(m2, toks)
    assert np.max(np.abs(a - b)) <= 1e-12 * np.max(np.abs(a))


def test_zeroed_projection_closed_forms():
    shape = small_shape()
    m = random_model(shape, 11)
    toks = np.random.default_rng(12).integers(0, shape.vocab, 9)
    for lw in m.layers:
        lw["wo"][:] = 0.0
        lw["w_down"][:] = 0.0
    st = vo.forward_prefill(m, toks)
    for l in range(shape.n_layers):
        assert np.array_equal(st[l], m.embed[toks])  # every block is the identity
    m = random_model(shape, 11)
    for lw in m.layers:
        lw["w_gate"][:] = 0.0  # silu(0) = 0: the FFN adds nothing
    st = vo.forward_prefill(m, toks)
    h = m.embed[toks]
    w = m.layers[0]
    a = vo.rmsnorm(h, w["attn_norm"], m.rms_eps)
    T = len(toks)
    q = vo.rope((a @ w["wq"].T).reshape(T, 4, 16), np.arange(T), m.rope_base)
    k = vo.rope((a @ w["wk"].T).reshape(T, 2, 16), np.arange(T), m.rope_base)
    v = (a @ w["wv"].T).reshape(T, 2, 16)
    u = h + vo.causal_attention(q, k, v).reshape(T, -1) @ w["wo"].T
    assert np.max(np.abs(st[0] - u)) <= 1e-13


def test_against_transformers_llama_float64():
    """The whole forward against an independent library implementation of the architecture."""
    from transformers import LlamaConfig, LlamaModel

    shape = synth.ModelShape(3, 64, 4, 2, 16, 96, 101, 500000.0, 1e-5)
    m = random_model(shape, 13, std=0.15)
    cfg = LlamaConfig(
        vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.d_ffn,
        num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_heads,
        num_key_value_heads=shape.n_kv_heads, head_dim=shape.head_dim, rms_norm_eps=shape.rms_eps,
        rope_theta=shape.rope_base, attention_bias=False, mlp_bias=False, max_position_embeddings=256,
        tie_word_embeddings=False,
    )
    hf = LlamaModel(cfg).double().eval()
    sd = {"embed_tokens.weight": m.embed, "norm.weight": m.final_norm}
    names = {"attn_norm": "input_layernorm", "wq": "self_attn.q_proj", "wk": "self_attn.k_proj",
             "wv": "self_attn.v_proj", "wo": "self_attn.o_proj", "ffn_norm": "post_attention_layernorm",
             "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj", "w_down": "mlp.down_proj"}
    for l, lw in enumerate(m.layers):
        for k, v in lw.items():
            sd[f"layers.{l}.{names[k]}.weight"] = v
    missing = hf.load_state_dict({k: torch.from_numpy(np.ascontiguousarray(v)) for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k]
    toks = np.random.default_rng(14).integers(0, shape.vocab, 37)
    with torch.no_grad():
        out = hf(input_ids=torch.from_numpy(toks)[None], output_hidden_states=True, use_cache=False)
    ours = vo.forward_prefill(m, toks)
    for l in range(shape.n_layers - 1):
        ref = out.hidden_states[l + 1][0].numpy()
        assert np.linalg.norm(ours[l] - ref) <= 1e-5 * np.linalg.norm(ref), l
    last = vo.rmsnorm(ours[-1], m.final_norm, m.rms_eps)  # the library applies the final norm to the last state
    ref = out.last_hidden_state[0].numpy()
    assert np.linalg.norm(last - ref) <= 1e-5 * np.linalg.norm(ref)


def test_batch_independence_and_zero_deviation_accept():
    shape = small_shape()
    m = random_model(shape, 15)
    rng = np.random.default_rng(16)
    seqs = [rng.integers(0, shape.vocab, 10), rng.integers(0, shape.vocab, 7), rng.integers(0, shape.vocab, 12)]
    check_seq = np.array([2, 0, 0, 2], dtype=np.int32)
    check_pos = np.array([11, 3, 9, 0], dtype=np.int32)
    own = np.stack([np.stack([vo.forward_prefill(m, seqs[s])[l, p] for s, p in zip(check_seq, check_pos)])
                    for l in range(shape.n_layers)])
    tol = vo.Tol(bit_aware=True)
    rep = vo.verify_prefill(m, seqs, own, check_seq, check_pos, tol, "f32")
    # against its own float64 states rounded to f32 the only deviation is that rounding
    assert rep.pos_ok.tolist() == [1, 1, 1, 1] and rep.seq_ok.tolist() == [1, 1, 1]
    assert rep.first_bad_layer.tolist() == [-1] * 4
    assert np.max(rep.stats[..., vo.STAT_NAMES.index("rel_l2")]) == 0.0
    assert rep.seq_score[1] == 0.0  # a sequence without checked positions: accepted, score 0
    # order of sequences in the batch does not matter
    rep2 = vo.verify_prefill(m, [seqs[2], seqs[1], seqs[0]], own, np.array([0, 2, 2, 0]), check_pos, tol, "f32")
    assert np.array_equal(rep.stats, rep2.stats)
    # prefix-only recomputation gives the same report
    rep3 = vo.verify_prefill(m, seqs, own, check_seq, check_pos, tol, "f32", prefix_only=True)
    assert np.max(np.abs(rep3.hidden - rep.hidden)) <= 1e-13 * np.max(np.abs(rep.hidden))


def test_round_to_bf16_matches_library_conversion():
    rng = np.random.default_rng(17)
    x = np.concatenate([
        rng.standard_normal(20000) * np.exp(rng.uniform(-60, 60, 20000)),
        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895313892515355e38, 1e-40, -1e-39, 65280.0, 65408.0]),
    ]).astype(np.float32)  # float32 inputs: the library rounds float32 -> bf16 once
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float64).numpy()
    got = vo.round_to_bf16(x.astype(np.float64))
    assert np.array_equal(ref, got)
    bits = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(vo.widen_bf16_bits(bits), ref)
    # ties go to even: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    assert vo.round_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert vo.round_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6


def test_compare_stats_hand_worked_vectors():
    tol = vo.Tol(tau_large=0.25, e_w=1e-2, e_m=7)
    u = 2.0 ** -7  # one bf16 step in [1, 2)
    #            exact  +1 step  +8 steps  binade cross   other binade   tiny     sign flip
    c = np.array([1.5, 1.5, 1.5, 1.0, 1.0, 0.0, 1.25])
    h = np.array([1.5, 1.5 + u, 1.5 + 8 * u, 1.0 - u / 2, 0.5, 4e-6, -1.25])
    s = dict(zip(vo.STAT_NAMES, vo.compare_stats(h, c, "bf16", tol)))
    d = h - c
    assert s["n_exact"] == 1 and s["n_nonfinite"] == 0
    assert s["n_exp_mismatch"] == 3  # 1-u/2 (exp 126), 0.5 (exp 126), 4e-6 vs 0 (exp field 0)
    assert s["p_e"] == 3 / 7
    # mismatches: (1 - u/2) has mantissa 127 vs 0 -> large; 0.5 has mantissa 0 vs 0 -> small;
    # 4e-6 = 1.0000110...b * 2^-18 rounds to mantissa 6 vs 0 -> small
    assert s["n_mant_large"] == 1 and s["p_m"] == 1 / 3
    # matches: exact (0 steps), +1 step (<= 1.28), +8 steps (large), sign flip (2*(128+32) steps, large)
    assert s["n_mant_small"] == 2 and s["p_w"] == 2 / 4
    assert s["max_abs"] == 2.5
    assert abs(s["mae"] - np.sum(np.abs(d)) / 7) <= 1e-15
    assert abs(s["mean_signed"] - np.sum(d) / 7) <= 1e-15
    assert abs(s["rel_l2"] - np.linalg.norm(d) / np.linalg.norm(c)) <= 1e-15
    assert s["q_small"] == 2 / 7  # the exact element and the 4e-6 one
    assert s["z_large"] == 2 / 7  # |d| > 0.25: the 0.5 and the 2.5
    # f32 serialisation: 23 mantissa bits, one bf16 step is 65536 f32 steps (<= 0.01 * 2^23 = 83886)
    s32 = dict(zip(vo.STAT_NAMES, vo.compare_stats(h, c, "f32", tol)))
    assert s32["n_mant_small"] == 2 and s32["n_exp_mismatch"] == 3
    # non-finite values are counted and force a reject
    hn = h.copy()
    hn[2] = np.nan
    sn = vo.compare_stats(hn, c, "bf16", tol)
    assert sn[vo.STAT_NAMES.index("n_nonfinite")] == 1
    assert not vo.layer_passes(sn, vo.Tol(rel_l2=0.0))
    # reference of norm zero: relative error stays finite through the tiny floor
    z = vo.compare_stats(np.array([1.0, 0.0]), np.array([0.0, 0.0]), "bf16", tol)
    assert np.isfinite(z[0]) and z[0] > 1e20


def test_threshold_directions():
    tol = vo.Tol(rel_l2=0.25, max_abs=0.5, mae=0.0)
    c = np.array([2.0, 0.0, 0.0, 0.0])
    at = vo.compare_stats(np.array([2.5, 0.0, 0.0, 0.0]), c, "f32", tol)  # rel_l2 = 0.25, max_abs = 0.5 exactly
    assert vo.layer_passes(at, tol)  # equality accepts
    above = vo.compare_stats(np.array([2.5000001, 0.0, 0.0, 0.0]), c, "f32", tol)
    assert not vo.layer_passes(above, tol)
    # one bad layer rejects the position, one bad position rejects its sequence only
    good = vo.compare_stats(c, c, "f32", tol)
    stats = np.stack([np.stack([good, good, good]), np.stack([good, above, above]), np.stack([good, good, good])])
    pos_ok, first_bad, seq_ok, score = vo.verdict(stats, np.array([0, 1, 1]), 3, tol)
    assert pos_ok.tolist() == [1, 0, 1] and first_bad.tolist() == [-1, 1, -1]
    assert seq_ok.tolist() == [1, 0, 1]
    mae_bad = above[vo.STAT_NAMES.index("mae")]
    assert abs(score[1] - (2 * mae_bad) / 6) <= 1e-15 and score[0] == 0.0 and score[2] == 0.0


def _table_rows():
    rows = []
    for line in open(os.path.join(GOLDEN, "paper_table_bins.txt")):
        if line.strip() and not line.startswith("#"):
            rows.append([int(x) for x in line.split()])
    return rows


@pytest.mark.parametrize("row", _table_rows())
def test_bit_aware_bookkeeping_reproduces_paper_table_bins(row):
    """Elements realising one printed table row must give back the row's ratios, and the paper's
    off-chain thresholds must separate the honest table from the quantised one."""
    table, n, exact, m_large, m_small, x_large, x_small = row
    assert m_large + m_small + x_large + x_small == n and exact <= m_small
    u = 2.0 ** -7
    c, h = [], []
    for i in range(exact):
        c.append(1.5); h.append(1.5)
    for i in range(m_small - exact):
        c.append(1.5); h.append(1.5 + u * (1 if i % 2 else -1))
    for i in range(m_large):
        c.append(1.5); h.append(1.5 + 8 * u * (1 if i % 2 else -1))
    for i in range(x_large):  # just across a binade boundary: mantissa fields 0 and 127
        if i % 2:
            c.append(1.0); h.append(1.0 - u / 2)
        else:
            c.append(1.0 - u / 2); h.append(1.0)
    for i in range(x_small):  # a factor of two apart: equal mantissa fields
        if i % 2:
            c.append(1.0); h.append(0.5)
        else:
            c.append(0.5); h.append(1.0)
    perm = np.random.default_rng(n).permutation(n)
    c, h = np.array(c)[perm], np.array(h)[perm]
    tol = vo.Tol(rel_l2=0.0, bit_aware=True)  # the paper's off-chain thresholds are the defaults
    st = vo.compare_stats(h, c, "bf16", tol)
    s = dict(zip(vo.STAT_NAMES, st))
    assert s["n_exact"] == exact
    assert s["p_e"] == (x_large + x_small) / n
    assert s["p_m"] == x_large / (x_large + x_small)
    assert s["p_w"] == m_small / (m_large + m_small)
    accept = bool(vo.layer_passes(st, tol))
    if table == 2:
        assert s["p_e"] > 0.05 and not accept  # quantised prover: rejected on P_e alone
    elif n == 256:
        assert accept  # 9/256 < 0.05, 7/9 > 0.75, 201/247 > 0.80
    else:
        assert s["p_e"] < 0.05 and s["p_m"] < 0.75 and not accept  # 64-element row: 2/3 and 48/61 miss the paper's own cut


def test_bf16_decode_trace_is_close_but_not_identical():
    shape = small_shape(d=64, dh=16, H=4, KV=2, F=96)
    m = random_model(shape, 18)
    toks = np.random.default_rng(19).integers(0, shape.vocab, 16)
    exact = vo.forward_prefill(m, toks)
    noisy = vo.forward_decode_kvcache(m, toks, "bf16")
    rel = np.linalg.norm(noisy - exact, axis=-1) / np.linalg.norm(exact, axis=-1)
    assert 1e-5 < rel.max() < 2e-2


def test_synth_generator_is_reproducible_and_distributed_as_stated():
    wl = synth.WORKLOADS["tiny"]
    a = synth.layer_weights(wl, 0)
    b = synth.layer_weights(wl, 0)
    assert all(torch.equal(a[k], b[k]) for k in a)
    w32 = synth.layer_weights(wl, 0, dtype=torch.float32)
    assert torch.equal(w32["wq"].to(torch.bfloat16), a["wq"])  # bf16 copy = RNE of the fp32 master
    assert abs(float(w32["w_gate"].std()) - 0.02) < 5e-4 and abs(float(w32["w_gate"].mean())) < 2e-4
    assert abs(float(w32["ffn_norm"].mean()) - 1.0) < 0.02
    assert not torch.equal(a["wk"], a["wv"])
    toks = synth.token_streams(wl)
    assert toks.shape == (1, 64) and toks.min() >= 0 and toks.max() < 1024
    big = synth.token_streams(synth.WORKLOADS["small"])
    assert big.shape == (4, 512) and len(np.unique(big)) > 1900
    cs, cp = synth.check_positions(synth.WORKLOADS["small"])
    assert len(cs) == 20 and len(set(zip(cs.tolist(), cp.tolist()))) == 20
    rows = synth.embed_weights(wl, rows=torch.tensor([5, 1000]))
    full = synth.embed_weights(wl)
    assert torch.equal(rows, full[[5, 1000]])


def test_token_match_against_transformers_causal_lm():
    """Final norm + output head + arg-max against the library's causal-LM logits."""
    from transformers import LlamaConfig, LlamaForCausalLM

    shape = synth.ModelShape(2, 64, 4, 2, 16, 96, 211, 10000.0, 1e-5)
    m = random_model(shape, 21, std=0.15)
    rng = np.random.default_rng(22)
    lm_head = 0.2 * rng.standard_normal((shape.vocab, shape.d_model))
    cfg = LlamaConfig(
        vocab_size=shape.vocab, hidden_size=shape.d_model, intermediate_size=shape.d_ffn,
        num_hidden_layers=shape.n_layers, num_attention_heads=shape.n_heads, num_key_value_heads=shape.n_kv_heads,
        head_dim=shape.head_dim, rms_norm_eps=shape.rms_eps, rope_theta=shape.rope_base, attention_bias=False,
        mlp_bias=False, max_position_embeddings=256, tie_word_embeddings=False,
    )
    hf = LlamaForCausalLM(cfg).double().eval()
    names = {"attn_norm": "input_layernorm", "wq": "self_attn.q_proj", "wk": "self_attn.k_proj",
             "wv": "self_attn.v_proj", "wo": "self_attn.o_proj", "ffn_norm": "post_attention_layernorm",
             "w_gate": "mlp.gate_proj", "w_up": "mlp.up_proj", "w_down": "mlp.down_proj"}
    sd = {"model.embed_tokens.weight": m.embed, "model.norm.weight": m.final_norm, "lm_head.weight": lm_head}
    for l, lw in enumerate(m.layers):
        for k, v in lw.items():
            sd[f"model.layers.{l}.{names[k]}.weight"] = v
    missing = hf.load_state_dict({k: torch.from_numpy(np.ascontiguousarray(v)) for k, v in sd.items()}, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k]
    toks = rng.integers(0, shape.vocab, 29)
    with torch.no_grad():
        ref_logits = hf(input_ids=torch.from_numpy(toks)[None], use_cache=False).logits[0].numpy()
    last = vo.forward_prefill(m, toks)[-1]
    claimed = np.argmax(ref_logits, axis=-1)
    claimed[5] = (claimed[5] + 1) % shape.vocab  # one forged token
    arg, match, margin = vo.token_match(m, last, lm_head, claimed)
    assert np.array_equal(arg, np.argmax(ref_logits, axis=-1))
    assert match.tolist() == [0 if i == 5 else 1 for i in range(29)]
    srt = np.sort(ref_logits, axis=-1)
    assert np.allclose(margin, srt[:, -1] - srt[:, -2], rtol=0, atol=2e-5)  # the library keeps its rotary table in float32
    # a duplicated head row ties (up to the summation order of the matrix product): margin vanishes
    a2, _, m2 = vo.token_match(m, last[:1], np.concatenate([lm_head[:3], lm_head[:3]]), np.array([0]))
    assert a2[0] % 3 == int(np.argmax(lm_head[:3] @ vo.rmsnorm(last[0], m.final_norm, m.rms_eps))) and m2[0] < 1e-12


def test_segments_compose_to_the_full_pass():
    """Running blocks [0, a) and then [a, L) from the first segment's output reproduces the single pass bit
    for bit, and a segment's result depends only on its input states."""
    shape = small_shape(n_layers=4)
    m = random_model(shape, 23)
    rng = np.random.default_rng(24)
    seqs = [rng.integers(0, shape.vocab, 11), rng.integers(0, shape.vocab, 6)]
    full = vo.forward_prefill_batch(m, seqs)
    first = vo.forward_segment_batch(m, [vo.embed_tokens(m, t) for t in seqs], 0, 3)
    second = vo.forward_segment_batch(m, [f[-1] for f in first], 3, 4)
    for b in range(2):
        assert np.array_equal(np.concatenate([first[b], second[b]]), full[b])
    # verify_segment on its own outputs accepts with zero deviation; a perturbed upstream state is caught downstream
    cs, cp = np.array([0, 1, 0]), np.array([10, 2, 4])
    own = np.stack([second[s][:, p] for s, p in zip(cs, cp)], axis=1)
    rep = vo.verify_segment(m, [f[-1] for f in first], 3, 4, own, cs, cp, vo.Tol(), "f32")
    assert rep.pos_ok.all() and rep.stats[..., 0].max() < 1e-6
    bad_in = [f[-1].copy() for f in first]
    bad_in[0][4] += rng.standard_normal(shape.d_model) * np.sqrt(np.mean(bad_in[0][4] ** 2))  # not a rescaling: the norm would undo it
    rep = vo.verify_segment(m, bad_in, 3, 4, own, cs, cp, vo.Tol(), "f32")
    rel = rep.stats[:, 0, 0]
    assert rep.pos_ok[2] == 0 and rel[2] > 0.1  # the perturbed position itself
    assert rel[1] < 1e-6  # another sequence: untouched
    assert 1e-6 < rel[0] < rel[2]  # a later position of the same sequence attends to it and moves, but less


def test_spot_check_worked_example():
    """Eight sampled scalars, tolerance 0.01: worked by hand."""
    hidden = np.arange(12, dtype=np.float64).reshape(3, 4) / 8.0
    rows, cols = [0, 0, 1, 1, 2, 2, 2, 0], [0, 3, 1, 2, 0, 3, 1, 1]
    ref = hidden[rows, cols].copy()
    ref[1] += 0.01      # exactly at the tolerance: agrees (<=)
    ref[2] -= 0.0101    # just beyond: disagrees
    ref[5] = np.nan     # never agrees
    ref[7] += 1.0
    agree, p_hat, ok = vo.spot_check(hidden, rows, cols, ref, 0.01, 0.625)
    assert agree.tolist() == [1, 1, 0, 1, 1, 0, 1, 0] and p_hat == 5 / 8 and ok  # 0.625 >= theta
    assert not vo.spot_check(hidden, rows, cols, ref, 0.01, 0.63)[2]


def test_merkle_root_structure_and_inclusion_proofs():
    """The tree against an independent verifier that only knows 'hash the leaf, then fold the path'."""
    import hashlib
    import struct

    def verify(root, value, index, path):  # MerkleVerify as a contract would run it
        h = hashlib.sha256(struct.pack("<f", value)).digest()
        for sib in path:
            h = hashlib.sha256(sib + h).digest() if index & 1 else hashlib.sha256(h + sib).digest()
            index >>= 1
        return h == root

    rng = np.random.default_rng(41)
    for n in (1, 2, 3, 5, 8, 13, 64):
        v = rng.standard_normal(n).astype(np.float32)
        root = vo.merkle_root(v)
        assert len(root) == 32
        for j in range(n):
            path = vo.merkle_path(v, j)
            assert len(path) == int(np.ceil(np.log2(n))) if n > 1 else path == []
            assert verify(root, float(v[j]), j, path)
            assert not verify(root, float(v[j]) + 1.0, j, path)
        w = v.copy()
        w[n // 2] = np.nextafter(w[n // 2], np.float32(10.0))  # one ulp in one leaf
        assert vo.merkle_root(w) != root
    # serialisation: float32 little endian, so -0.0 and 0.0 commit differently and float64 input is narrowed first
    assert vo.merkle_root(np.array([0.0])) == hashlib.sha256(bytes(4)).digest()
    assert vo.merkle_root(np.array([-0.0])) == hashlib.sha256(bytes.fromhex("00000080")).digest()
    assert vo.merkle_root(np.array([1.0])) == hashlib.sha256(bytes.fromhex("0000803f")).digest()
    assert vo.merkle_root(np.array([0.1], dtype=np.float64)) == vo.merkle_root(np.array([np.float32(0.1)]))
    two = vo.merkle_root(np.array([1.0, 2.0]))
    assert two == hashlib.sha256(hashlib.sha256(bytes.fromhex("0000803f")).digest()
                                 + hashlib.sha256(bytes.fromhex("00000040")).digest()).digest()


# ----------------------------------------------------------------------------- threshold sensitivity


def _cell(**kw):
    row = np.zeros(vo.NSTAT)
    row[vo.STAT_NAMES.index("p_m")] = 1.0
    row[vo.STAT_NAMES.index("p_w")] = 1.0
    for k, v in kw.items():
        row[vo.STAT_NAMES.index(k)] = v
    return row


def test_threshold_sweep_hand_worked_cells():
    """Seven cells whose verdict under three tolerance sets is worked out by hand (strict P_e / P_m / P_w,
    closed |e| and rel-L2 intervals, a non-finite element rejects, equality with a strict bound rejects)."""
    f32 = lambda x: float(np.float32(x))
    stats = np.stack([
        _cell(rel_l2=0.01, p_e=0.01, p_m=1.0, p_w=0.9, mean_signed=0.001),     # honest, clean
        _cell(rel_l2=0.03, p_e=0.06, p_m=0.8, p_w=0.85),                       # honest, P_e above 0.05
        _cell(rel_l2=0.01, p_e=0.02, p_m=0.7, p_w=0.95, mean_signed=-0.02),    # honest, P_m low and |e| high
        _cell(rel_l2=0.0, p_e=f32(0.05)),                                      # honest, P_e exactly at the strict bound
        _cell(rel_l2=0.02, p_e=0.08, p_m=0.95, p_w=0.3),                       # attack inside the rel-L2 tolerance
        _cell(rel_l2=0.2, p_e=0.5, p_m=0.9, p_w=0.05),                         # gross attack
        _cell(rel_l2=0.01, p_e=0.01, p_m=1.0, p_w=0.9, n_nonfinite=1),         # attack hiding behind a NaN
    ])
    attack = np.array([0, 0, 0, 0, 1, 1, 1], dtype=bool)
    variants = [
        vo.Tol(),                                                                               # rel-L2 <= 5e-2 only
        vo.Tol(bit_aware=True),                                                                 # + the paper's selected set
        vo.Tol(rel_l2=0.0, bit_aware=True, pe_max=0.07, pm_min=0.6, pw_min=0.5, e_abs_max=0.05),
    ]
    counts = vo.threshold_sweep(stats, attack, variants)
    assert counts.tolist() == [[4, 0, 1, 2], [1, 3, 0, 3], [4, 0, 0, 3]]
    r = vo.detection_rates(counts)
    assert r["FPR"].tolist() == [0.0, 0.75, 0.0] and r["FNR"].tolist() == [1 / 3, 0.0, 0.0]
    assert np.allclose(r["TPR"] + r["FNR"], 1.0) and np.allclose(r["TNR"] + r["FPR"], 1.0)


def test_threshold_sweep_is_monotone_and_agrees_with_the_verdict():
    rng = np.random.default_rng(5)
    n = 400
    stats = np.zeros((n, vo.NSTAT))
    for name, lo, hi in (("rel_l2", 0, 0.1), ("p_e", 0, 0.2), ("p_m", 0.4, 1), ("p_w", 0, 1), ("mean_signed", -0.03, 0.03)):
        stats[:, vo.STAT_NAMES.index(name)] = rng.uniform(lo, hi, n).astype(np.float32)
    attack = rng.random(n) < 0.5
    base = dict(rel_l2=0.0, bit_aware=True)
    # loosening a threshold never turns an accept into a reject
    for field, values in (("pe_max", (0.02, 0.05, 0.1)), ("pm_min", (0.9, 0.75, 0.5)), ("pw_min", (0.9, 0.8, 0.3)),
                          ("e_abs_max", (0.005, 0.01, 0.02))):
        c = vo.threshold_sweep(stats, attack, [vo.Tol(**base, **{field: v}) for v in values])
        assert np.all(np.diff(c[:, 0]) >= 0) and np.all(np.diff(c[:, 2]) >= 0)
        assert np.all(c.sum(axis=1) == n)
    # one layer per position: a cell passes the sweep iff the position verdict accepts it
    tol = vo.Tol(bit_aware=True)
    pos_ok, _, _, _ = vo.verdict(stats.reshape(n, 1, vo.NSTAT), np.zeros(n, dtype=np.int32), 1, tol)
    c = vo.threshold_sweep(stats, np.zeros(n, dtype=bool), [tol])
    assert c[0, 0] == int(pos_ok.sum()) and c[0, 1] == n - int(pos_ok.sum())


def test_fake_quantise_grid_and_error_bound():
    """The attack model of the sensitivity analysis: values land on a symmetric integer grid per row, the row
    maximum is kept, and the error is at most half a step."""
    w = torch.from_numpy(np.random.default_rng(3).standard_normal((7, 64)).astype(np.float32))
    for bits in (8, 4):
        q = synth.fake_quantise(w, bits)
        qmax = 2 ** (bits - 1) - 1
        step = w.abs().amax(dim=1, keepdim=True) / qmax
        k = q / step
        assert torch.allclose(k, torch.round(k), atol=1e-4) and float(k.abs().max()) <= qmax + 1e-4
        assert float(((q - w).abs() / step).max()) <= 0.5 + 1e-5
        assert torch.allclose(q.abs().amax(dim=1), w.abs().amax(dim=1))


# ----------------------------------------------------------------------------- every branch of the verdict


def _worked_row():
    """Eight deviations whose statistics are exact binary fractions: 0.5, -0.25, 2^-18 and 0.125 beside four
    zeros.  MAE = (0.875 + 2^-18) / 8, Q_small = 5/8 (the zeros and 2^-18 <= 1e-5), Z_large at tau = 0.125 is
    2/8 (0.125 itself is not above tau), max |Delta| = 0.5."""
    c = np.array([1.0, -2.0, 0.5, 0.0, 3.0, -1.0, 0.25, 1.5])
    delta = np.array([0.5, -0.25, 0.0, 0.0, 0.0, 0.0, 2.0 ** -18, 0.125])
    return c + delta, c


def test_each_float_test_of_the_verdict_at_and_past_its_threshold():
    """Offline battery T_off (MAE, Z_large, Q_small) and max |Delta|, one test enabled at a time: the value exactly
    at the threshold accepts (b = 1[T_v <= tau]), the next representable threshold on the wrong side rejects,
    and the documented "off" values switch the test off."""
    h, c = _worked_row()
    base = dict(rel_l2=0.0, tau_large=0.125)
    s = vo.compare_stats(h, c, "f32", vo.Tol(**base))
    v = dict(zip(vo.STAT_NAMES, s))
    mae = 0.109375 + 2.0 ** -21
    assert v["mae"] == mae and v["q_small"] == 0.625 and v["z_large"] == 0.25 and v["max_abs"] == 0.5
    ok = lambda **kw: bool(vo.layer_passes(s, vo.Tol(**{**base, **kw})))
    assert ok()  # nothing enabled: accept
    # MAE <= tau
    assert ok(mae=mae) and ok(mae=1.0) and not ok(mae=np.nextafter(mae, 0.0)) and not ok(mae=0.05)
    assert ok(mae=0.0) and ok(mae=-1.0)  # <= 0 disables
    # max |Delta| <= tau
    assert ok(max_abs=0.5) and not ok(max_abs=np.nextafter(0.5, 0.0)) and ok(max_abs=0.0) and ok(max_abs=-3.0)
    # Z_large <= z_large_max (a fraction of large deviations that is too high rejects)
    assert ok(z_large_max=0.25) and ok(z_large_max=0.9) and not ok(z_large_max=np.nextafter(0.25, 0.0))
    assert not ok(z_large_max=0.0)  # zero is an enabled threshold: no large deviation allowed at all
    assert ok(z_large_max=-1.0) and ok(z_large_max=-1e-9)  # negative disables
    # Q_small >= q_small_min (too few tiny deviations rejects)
    assert ok(q_small_min=0.625) and ok(q_small_min=0.1) and not ok(q_small_min=np.nextafter(0.625, 1.0))
    assert not ok(q_small_min=1.0)
    assert ok(q_small_min=0.0) and ok(q_small_min=-0.5)  # <= 0 disables
    # an identical pair passes every enabled test at its strictest setting
    z = vo.compare_stats(c, c, "f32", vo.Tol(**base))
    assert vo.layer_passes(z, vo.Tol(rel_l2=1e-30, max_abs=1e-30, mae=1e-30, tau_large=0.0, z_large_max=0.0, q_small_min=1.0))
    # the tests combine by AND: one failing test rejects whatever the others say
    assert ok(mae=1.0, max_abs=1.0, z_large_max=1.0, q_small_min=0.5)
    assert not ok(mae=1.0, max_abs=1.0, z_large_max=1.0, q_small_min=0.7)
    assert not ok(mae=1.0, max_abs=0.4, z_large_max=1.0, q_small_min=0.5)


def test_relaxed_value_test_is_the_z_large_test_on_a_full_row():
    """The relaxed on-chain test (|v_j - V_j| <= eps on sampled entries, agreement rate p_hat >= theta) applied to
    every entry of a row decides like Z_large with tau_large = eps and z_large_max = 1 - theta: Z_large is the
    fraction above eps, p_hat the fraction at or below it."""
    rng = np.random.default_rng(11)
    d, eps = 64, 0.125
    cols = np.arange(d)
    for n_far in (0, 5, 16, 17, 40, 64):
        c = rng.standard_normal(d)
        delta = rng.uniform(-0.1, 0.1, d)
        far = rng.choice(d, n_far, replace=False)
        delta[far] = rng.choice([-1.0, 1.0], n_far) * rng.uniform(0.2, 0.9, n_far)
        if n_far:
            delta[far[0]] = 0.125 if n_far == 64 else 0.5  # exactly eps agrees (<=), it is not "large" (>)
        h = (c + delta).astype(np.float32).astype(np.float64)
        c = c.astype(np.float32).astype(np.float64)
        agree, p_hat, _ = vo.spot_check(h[None, :], np.zeros(d, int), cols, c, eps, 0.5)
        for theta in (0.25, 0.5, 0.75, 0.9, 1.0):  # 1 - theta is exact for these in binary except 0.9
            tol = vo.Tol(rel_l2=0.0, tau_large=eps, z_large_max=1.0 - theta)
            s = vo.compare_stats(h, c, "f32", tol)
            z = s[vo.STAT_NAMES.index("z_large")]
            assert z == 1.0 - agree.sum() / d
            on_chain = vo.spot_check(h[None, :], np.zeros(d, int), cols, c, eps, theta)[2]
            if abs((1.0 - z) - theta) > 1e-6:  # away from the rounding of 1 - 0.9
                assert bool(vo.layer_passes(s, tol)) == on_chain, (n_far, theta)
    # the boundary itself with exact fractions: 16 of 64 far -> p_hat = 0.75 = theta accepts, 17 rejects
    for n_far, expect in ((16, True), (17, False)):
        c = np.zeros(d)
        h = np.where(np.arange(d) < n_far, 1.0, 0.0)
        tol = vo.Tol(rel_l2=0.0, tau_large=eps, z_large_max=0.25)
        assert bool(vo.layer_passes(vo.compare_stats(h, c, "f32", tol), tol)) is expect
        assert vo.spot_check(h[None, :], np.zeros(d, int), cols, c, eps, 0.75)[2] is expect


def test_synthetic_weight_scale_keeps_bf16_rounding_noise_from_growing():
    """Input recipe evidence: at d_model = 4096 a plain N(0, 0.02) initialisation gives every projection a gain of
    0.02 * sqrt(4096) = 1.28, and such a random network amplifies bf16 rounding noise from block to block; with the
    constant-gain scale 0.02 * sqrt(256 / d_model) it does not.  Measured on the oracle alone: its bf16-emulating
    decode against its own float64 prefill, 16 tokens, 3 blocks of width 4096 (narrow FFN to keep this quick)."""
    shape = synth.ModelShape(3, 4096, 8, 2, 128, 1024, 64, 500000.0)
    tokens = np.arange(16) % shape.vocab

    def drift(std):
        rng = np.random.default_rng(3)
        r = lambda *s: rng.standard_normal(s) * std
        layers = [{"attn_norm": 1 + 0.1 * rng.standard_normal(shape.d_model), "wq": r(shape.d_q, shape.d_model),
                   "wk": r(shape.d_kv, shape.d_model), "wv": r(shape.d_kv, shape.d_model), "wo": r(shape.d_model, shape.d_q),
                   "ffn_norm": 1 + 0.1 * rng.standard_normal(shape.d_model), "w_gate": r(shape.d_ffn, shape.d_model),
                   "w_up": r(shape.d_ffn, shape.d_model), "w_down": r(shape.d_model, shape.d_ffn)}
                  for _ in range(shape.n_layers)]
        layers = [{k: vo.round_to_bf16(v) for k, v in lw.items()} for lw in layers]
        m = vo.make_model(shape, vo.round_to_bf16(rng.standard_normal((shape.vocab, shape.d_model)) * 0.02),
                          np.ones(shape.d_model), layers)
        exact = vo.forward_prefill(m, tokens)
        emul = vo.forward_decode_kvcache(m, tokens, "bf16")
        rel = np.linalg.norm(emul - exact, axis=-1) / np.linalg.norm(exact, axis=-1)  # [layers, tokens]
        return rel.max(axis=1)

    plain = drift(0.02)
    scaled = drift(synth.weight_std(shape))
    assert synth.weight_std(shape) == 0.02 * (256 / 4096) ** 0.5
    assert np.all(np.diff(plain) > 0) and plain[-1] > 2 * scaled[-1], (plain, scaled)
    assert scaled.max() <= 5e-3, scaled
    assert plain[-1] >= 8e-3, plain
