"""End-to-end parity of the verifier path (C ABI on a B200) against the CPU oracle on the same seeded inputs.

Bars: recomputed hidden states within relative L2 <= 2e-2 per checked position and layer; verdicts,
first failing layers and indices identical for every cell outside the gray band (oracle rel-L2 <= tol/2
or >= 2 tol; the traces are built so that no intended cell lies inside it); integer work bit-exact.
"""
import numpy as np
import pytest
import torch

from oracle import verillm_oracle as vo
from paper_2509_24257_b200 import binding as vb
from paper_2509_24257_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
HIDDEN_TOL = 2e-2
TOL = 5e-2
REL = vo.STAT_NAMES.index("rel_l2")


def run_both(model, om, wl, tokens, committed64, check_seq, check_pos, commit="bf16", prefix_only=False,
             tol_kw=None, seqs=None, cu=None):
    """Feeds the same tokens / committed states / check set to the CUDA path and to the oracle."""
    tol_kw = tol_kw or {}
    comm_t = synth.to_commit_dtype(committed64, commit)
    seqs = list(tokens) if seqs is None else seqs
    cu = synth.cu_seqlens(wl) if cu is None else cu
    flat = torch.from_numpy(np.concatenate([np.asarray(s) for s in seqs]).astype(np.int32)).to(DEV)
    rep = model.verify_prefill(flat, cu, comm_t.to(DEV), check_seq, check_pos, vb.default_tol(**tol_kw), want_hidden=True)
    torch.cuda.synchronize()
    g = rep.cpu()
    o = vo.verify_prefill(om, seqs, comm_t.to(torch.float64).numpy(), check_seq, check_pos, vo.Tol(**tol_kw), commit,
                          prefix_only=prefix_only)
    return g, o


def assert_parity(g, o, tol=TOL, expect_reject=(), expect_gray=()):
    assert g["status"] == 0
    # hidden states: the first gate
    rel = H.rel_l2(g["hidden"], o.hidden)
    assert rel.max() <= HIDDEN_TOL, f"hidden-state rel-L2 {rel.max():.3e}"
    # verdicts: identical wherever the oracle's cell is outside the gray band
    o_rel = o.stats[..., REL]  # [n_check, n_layers]
    gray = (o_rel > tol / 2) & (o_rel < 2 * tol)
    gray_pos = gray.any(axis=1)
    for s in np.nonzero(gray_pos)[0]:
        assert s in expect_gray, f"slot {s} unexpectedly inside the gray band ({o_rel[s].max():.3e})"
    clear = ~gray_pos
    assert np.array_equal(g["pos_ok"][clear], o.pos_ok[clear])
    assert np.array_equal(g["first_bad_layer"][clear], o.first_bad_layer[clear])
    for s in expect_reject:
        assert o.pos_ok[s] == 0 and g["pos_ok"][s] == 0
    if not gray_pos.any():
        assert np.array_equal(g["seq_ok"], o.seq_ok)
        # |MAE_gpu - MAE_oracle| <= mean|h_gpu - h_oracle| <= rms(h_gpu - h_oracle) <= 2e-2 rms(h)
        bound = HIDDEN_TOL * float(np.sqrt(np.mean(o.hidden ** 2))) * 1.5 + 1e-7
        assert np.all(np.abs(g["seq_score"] - o.seq_score) <= bound)
    # statistics: same quantity computed from states that differ by <= 2e-2 of the state norm
    g_rel = g["stats"][..., REL]
    assert np.all(np.abs(g_rel - o_rel) <= HIDDEN_TOL * 1.2 + 1e-6)


@pytest.fixture(scope="module")
def tiny():
    wl = synth.WORKLOADS["tiny"]
    tokens = synth.token_streams(wl)
    om = H.oracle_model(wl)
    cs, cp = synth.check_positions(wl)  # all 64 positions, in draw order
    committed = H.oracle_committed(om, tokens, cs, cp, "bf16")
    model = H.gpu_model(wl, len(cs))
    yield wl, tokens, om, cs, cp, committed, model
    model.close()


def test_tiny_honest_trace_accepts_everywhere(tiny):
    wl, tokens, om, cs, cp, committed, model = tiny
    assert len(cs) == 64 and sorted(cp.tolist()) == list(range(64))
    g, o = run_both(model, om, wl, tokens, committed, cs, cp)
    assert_parity(g, o)
    assert g["pos_ok"].all() and g["seq_ok"].tolist() == [1]
    assert model.last_launch_count() == 3 + 7 * wl.shape.n_layers + 2


def test_tiny_noise_at_three_positions_is_rejected_exactly_there(tiny):
    wl, tokens, om, cs, cp, committed, model = tiny
    rng = synth.tamper_rng(wl)
    bad = sorted(rng.choice(len(cs), size=3, replace=False).tolist())
    tampered = synth.add_state_noise(committed, bad, None, 0.5, rng)  # 0.5 x RMS = 10 x tol
    g, o = run_both(model, om, wl, tokens, tampered, cs, cp)
    assert_parity(g, o, expect_reject=bad)
    assert sorted(np.nonzero(g["pos_ok"] == 0)[0].tolist()) == bad
    assert g["seq_ok"].tolist() == [0] and (g["first_bad_layer"][bad] == 0).all()


def test_tiny_f32_trace_and_bit_aware_statistics(tiny):
    wl, tokens, om, cs, cp, committed, model = tiny
    g, o = run_both(model, om, wl, tokens, committed, cs, cp, commit="f32", tol_kw=dict(tau_large=0.05))
    assert_parity(g, o)
    # the counts are integers of d_model elements and partition it
    st = g["stats"]
    n_mis = st[..., vo.STAT_NAMES.index("n_exp_mismatch")]
    assert np.all(n_mis == np.round(n_mis)) and np.all(n_mis <= wl.shape.d_model)
    assert np.allclose(st[..., vo.STAT_NAMES.index("p_e")], n_mis / wl.shape.d_model)
    # honest noise: few exponent mismatches on either side
    assert st[..., vo.STAT_NAMES.index("p_e")].mean() < 0.05 and o.stats[..., vo.STAT_NAMES.index("p_e")].mean() < 0.05


def test_tiny_results_are_deterministic(tiny):
    wl, tokens, om, cs, cp, committed, model = tiny
    comm = synth.to_commit_dtype(committed, "bf16").to(DEV)
    flat = torch.from_numpy(tokens.reshape(-1)).to(DEV)
    a = model.verify_prefill(flat, synth.cu_seqlens(wl), comm, cs, cp, want_hidden=True).cpu()
    b = model.verify_prefill(flat, synth.cu_seqlens(wl), comm, cs, cp, want_hidden=True).cpu()
    assert np.array_equal(a["stats"], b["stats"]) and np.array_equal(a["hidden"], b["hidden"])


def test_ragged_batch_duplicates_and_order(tiny):
    """Sequences of different lengths (one of length 1), duplicate and unsorted check positions."""
    wl, tokens, om, _, _, _, _ = tiny
    rng = np.random.default_rng(5)
    lens = [57, 1, 130, 64]
    seqs = [rng.integers(0, wl.shape.vocab, n).astype(np.int32) for n in lens]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    cs = np.array([2, 0, 2, 1, 3, 2, 0, 2], dtype=np.int32)
    cp = np.array([129, 0, 5, 0, 63, 129, 56, 77], dtype=np.int32)  # slot 0 and 5 name the same position
    committed = np.zeros((wl.shape.n_layers, len(cs), wl.shape.d_model))
    for i, (s, p) in enumerate(zip(cs, cp)):
        committed[:, i] = vo.forward_decode_kvcache(om, seqs[s][: p + 1], "bf16")[:, p]
    committed = synth.add_state_noise(committed, [5], None, 0.5, rng)  # tamper one of the two duplicates
    model = vb.Model(wl.shape, int(cu[-1]), len(cs), len(lens), DEV)
    model.load_globals(synth.embed_weights(wl, DEV), synth.final_norm_weights(wl, DEV))
    model.load_layer(0, synth.layer_weights(wl, 0, DEV))
    g, o = run_both(model, om, wl, None, committed, cs, cp, commit="f32", seqs=seqs, cu=cu)
    assert_parity(g, o, expect_reject=[5])
    assert g["pos_ok"].tolist() == [1, 1, 1, 1, 1, 0, 1, 1]
    assert g["seq_ok"].tolist() == [1, 1, 0, 1]
    assert np.array_equal(g["hidden"][:, 0], g["hidden"][:, 5])  # same position gathered twice, bit-identical
    # no checks at all: every sequence accepted with score 0
    flat = torch.from_numpy(np.concatenate(seqs)).to(DEV)
    rep = model.verify_prefill(flat, cu, None, [], []).cpu()
    assert rep["seq_ok"].tolist() == [1, 1, 1, 1] and rep["seq_score"].tolist() == [0, 0, 0, 0]
    model.close()


def test_argument_errors_launch_nothing(tiny):
    wl, tokens, om, cs, cp, committed, model = tiny
    comm = synth.to_commit_dtype(committed, "bf16").to(DEV)
    flat = torch.from_numpy(tokens.reshape(-1)).to(DEV)
    cu = synth.cu_seqlens(wl)

    def code(**kw):
        args = dict(tokens=flat, cu_seqlens=cu, committed=comm, check_seq=cs, check_pos=cp)
        args.update(kw)
        with pytest.raises(vb.VerillmError) as e:
            model.verify_prefill(**args)
        return e.value.code

    bad_pos = cp.copy(); bad_pos[3] = 64
    assert code(check_pos=bad_pos) == vb.E_RANGE
    bad_seq = cs.copy(); bad_seq[0] = 1
    assert code(check_seq=bad_seq) == vb.E_RANGE
    assert code(cu_seqlens=[0, 65]) == vb.E_SHAPE  # more tokens than the handle was sized for
    assert code(cu_seqlens=[0, 40, 30]) in (vb.E_RANGE, vb.E_SHAPE)
    assert code(cu_seqlens=[1, 64]) == vb.E_RANGE
    with pytest.raises(vb.VerillmError) as e:
        vb.Model(synth.ModelShape(1, 256, 4, 4, 96, 768, 1024), 64, 4, 1, DEV)  # head_dim 96
    assert e.value.code == vb.E_SHAPE
    # a token id outside the vocabulary is clamped on the device, flagged, and rejects everything
    bad_tok = flat.clone(); bad_tok[10] = wl.shape.vocab + 5
    rep = model.verify_prefill(bad_tok, cu, comm, cs, cp).cpu()
    assert rep["status"] == vb.DEV_TOKEN_RANGE and not rep["pos_ok"].any() and rep["seq_ok"].tolist() == [0]
    # and the handle keeps working afterwards
    assert model.verify_prefill(flat, cu, comm, cs, cp).cpu()["pos_ok"].all()


@pytest.fixture(scope="module")
def small():
    wl = synth.WORKLOADS["small"]
    tokens = synth.token_streams(wl)
    om = H.oracle_model(wl)
    rng = synth.tamper_rng(wl)
    # the token-swap position is forced into the check set (its later positions move only slightly)
    swap_seq, swap_pos = 1, wl.prompt_len + int(rng.integers(0, wl.gen_len))
    cs, cp = synth.check_positions(wl, force=[(swap_seq, swap_pos)])
    committed = H.oracle_committed(om, tokens, cs, cp, "bf16")
    model = H.gpu_model(wl, len(cs))
    yield wl, tokens, om, cs, cp, committed, model, rng, (swap_seq, swap_pos)
    model.close()


def test_small_honest_trace(small):
    wl, tokens, om, cs, cp, committed, model, rng, _ = small
    assert len(cs) == 20
    g, o = run_both(model, om, wl, tokens, committed, cs, cp, prefix_only=True)
    assert_parity(g, o)
    assert g["pos_ok"].all() and g["seq_ok"].all()


def test_small_ragged_batch_spanning_several_row_tiles(small):
    """890 packed tokens = three full 256-row tiles and a ragged one through the CTA-pair GEMMs (coalesced
    residual epilogue, fused compare), sequences that end inside a tile, checks on first and last rows."""
    wl, _, om, _, _, _, model, _, _ = small
    rng = np.random.default_rng(17)
    lens = [300, 77, 513]
    seqs = [rng.integers(0, wl.shape.vocab, n).astype(np.int32) for n in lens]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    cs = np.array([2, 0, 1, 2, 0, 2], dtype=np.int32)
    cp = np.array([512, 299, 76, 0, 0, 255], dtype=np.int32)
    committed = np.zeros((wl.shape.n_layers, len(cs), wl.shape.d_model))
    for i, (b, q) in enumerate(zip(cs, cp)):
        committed[:, i] = vo.forward_decode_kvcache(om, seqs[b][: q + 1], "bf16")[:, q]
    committed = synth.add_state_noise(committed, [0], [wl.shape.n_layers - 1], 10 * TOL, rng)
    g, o = run_both(model, om, wl, None, committed, cs, cp, seqs=seqs, cu=cu)
    assert_parity(g, o, expect_reject=[0])
    assert g["pos_ok"].tolist() == [0, 1, 1, 1, 1, 1] and g["first_bad_layer"][0] == wl.shape.n_layers - 1
    assert g["seq_ok"].tolist() == [1, 1, 0]


def test_small_substituted_token_is_caught_at_its_position(small):
    wl, tokens, om, cs, cp, committed, model, rng, (sq, sp) = small
    forged = synth.swap_token(tokens, sq, sp, wl.shape.vocab, rng)
    later = [i for i in range(len(cs)) if cs[i] == sq and cp[i] > sp]  # may drift into the gray band
    g, o = run_both(model, om, wl, forged, committed, cs, cp, prefix_only=True)
    assert_parity(g, o, expect_reject=[0], expect_gray=later)
    assert g["seq_ok"][sq] == 0 and o.seq_ok[sq] == 0
    others = [b for b in range(wl.batch) if b != sq]
    assert g["seq_ok"][others].all() and o.seq_ok[others].all()


def test_small_layer_output_perturbation_of_ten_times_tolerance(small):
    wl, tokens, om, cs, cp, committed, model, rng, _ = small
    slot, layer = 7, 2
    tampered = synth.add_state_noise(committed, [slot], [layer], 10 * TOL, rng)
    g, o = run_both(model, om, wl, tokens, tampered, cs, cp, prefix_only=True)
    assert_parity(g, o, expect_reject=[slot])
    assert g["first_bad_layer"][slot] == layer and (np.delete(g["pos_ok"], slot) == 1).all()


def test_decode_commit_matches_oracle_decode_and_verifies_as_honest(small):
    wl, tokens, om, cs, cp, committed, model, rng, _ = small
    ref = H.oracle_committed(om, tokens, cs, cp, "f64")
    flat = torch.from_numpy(tokens.reshape(-1)).to(DEV)
    for n_prefill in (wl.prompt_len, 0, 300):
        trace = model.decode_commit(flat, synth.cu_seqlens(wl), n_prefill, cs, cp, torch.float32)
        rel = H.rel_l2(trace.double().cpu().numpy(), ref)
        assert rel.max() <= HIDDEN_TOL, (n_prefill, rel.max())
    trace = model.decode_commit(flat, synth.cu_seqlens(wl), wl.prompt_len, cs, cp, torch.bfloat16)
    rep = model.verify_prefill(flat, synth.cu_seqlens(wl), trace.contiguous(), cs, cp).cpu()
    assert rep["status"] == 0 and rep["pos_ok"].all() and rep["seq_ok"].all()
    assert 0 < rep["stats"][..., REL].max() <= TOL / 2  # decode and prefill differ, but only by rounding noise


def test_llama8b_width_reduced_depth():
    """Full layer widths (d 4096, 32/8 heads of 128, FFN 14336), two layers, ragged check set."""
    wl = synth.WORKLOADS["llama8b"].with_layers(2).with_batch(3, 200, 184)
    tokens = synth.token_streams(wl)
    cs = np.array([0, 0, 1, 2, 2, 1], dtype=np.int32)
    cp = np.array([0, 95, 130, 17, 127, 64], dtype=np.int32)
    om = H.oracle_model_streamed(wl, tokens, DEV)
    model = H.gpu_model(wl, len(cs))
    pre = vo.verify_prefill(om, list(tokens), np.zeros((2, len(cs), wl.shape.d_model)), cs, cp, vo.Tol(), "bf16",
                            prefix_only=True)
    honest = vo.round_to_bf16(pre.hidden)  # a prover that ran the same pass and serialised to bf16
    rng = synth.tamper_rng(wl)
    tampered = synth.add_state_noise(honest, [3], [1], 10 * TOL, rng)
    g, o = run_both(model, om, wl, tokens, tampered, cs, cp, prefix_only=True)
    assert_parity(g, o, expect_reject=[3])
    assert g["pos_ok"].tolist() == [1, 1, 1, 0, 1, 1] and g["seq_ok"].tolist() == [1, 1, 0]
    assert g["first_bad_layer"][3] == 1
    model.close()


def test_tail_token_match_same_states_and_end_to_end(small):
    """Arg-max of the output head on the last-layer states against the oracle: on identical states (single-CTA
    and CTA-pair product), and end to end on the states each side recomputed itself."""
    wl, tokens, om, cs, cp, committed, model, rng, _ = small
    lm = synth.lm_head_weights(wl, DEV)
    model.load_lm_head(lm)
    lm64 = vo.as_f64(H.bits(lm))
    wide = H.gpu_model(wl, 256)  # a handle sized for more checked rows than the configured 1 %
    wide.load_lm_head(lm)
    # (a) identical inputs: oracle last-layer states of 200 positions (pair kernel) and of 20 (single CTA)
    states = [vo.forward_prefill(om, tokens[b][:256])[-1] for b in range(2)]
    last = np.concatenate(states)[::2][:200].astype(np.float32)
    arg_o, _, margin_o = vo.token_match(om, last.astype(np.float64), lm64, np.zeros(len(last), np.int64))
    claimed = arg_o.copy()
    forged = [3, 77, 150]
    claimed[forged] = (claimed[forged] + 1) % wl.shape.vocab
    for n in (200, 20):
        arg, match, margin = wide.token_match(torch.from_numpy(last[:n]).to(DEV), claimed[:n])
        arg, match, margin = arg.cpu().numpy(), match.cpu().numpy(), margin.cpu().numpy()
        clear = margin_o[:n] > 5e-3  # bf16 rounding of the normed state moves logits by ~1e-3 here
        assert clear.mean() > 0.8
        assert np.array_equal(arg[clear], arg_o[:n][clear])
        want = (arg_o[:n] == claimed[:n]).astype(np.uint8)
        assert np.array_equal(match[clear], want[clear])
        assert all(match[i] == 0 for i in forged if i < n and clear[i])
        assert np.all(np.abs(margin - margin_o[:n])[clear] <= 5e-3)
    wide.close()
    # (b) end to end: each side uses the last-layer states it recomputed at the checked positions
    g, o = run_both(model, om, wl, tokens, committed, cs, cp, prefix_only=True)
    arg_o, _, margin_o = vo.token_match(om, o.hidden[-1], lm64, np.zeros(len(cs), np.int64))
    h_last = torch.from_numpy(np.ascontiguousarray(g["hidden"][-1])).to(DEV)
    arg, match, _ = model.token_match(h_last, arg_o)
    clear = margin_o > 3e-2  # states differ by up to 2e-2 relative
    assert clear.sum() >= len(cs) // 2
    assert np.array_equal(arg.cpu().numpy()[clear], arg_o[clear]) and match.cpu().numpy()[clear].all()
    with pytest.raises(vb.VerillmError):
        model.token_match(torch.zeros(len(cs) + 1, wl.shape.d_model, device=DEV), np.zeros(len(cs) + 1, np.int32))


def test_segment_local_verification_matches_oracle(small):
    """Blocks 2..3 recomputed from the recorded states entering block 2 (all positions), as a segment verifier
    does; committed outputs from the oracle's own segment pass, one of them tampered."""
    wl, tokens, om, cs, cp, _, model, rng, _ = small
    full = vo.forward_prefill_batch(om, list(tokens))
    upstream = [vo.round_to_bf16(f[1]) for f in full]  # recorded S entering block 2, serialised as bf16
    outs = vo.forward_segment_batch(om, upstream, 2, 4)
    honest = np.stack([outs[s][:, p] for s, p in zip(cs, cp)], axis=1)
    tampered = synth.add_state_noise(honest, [4], [1], 10 * TOL, rng)
    comm_t = synth.to_commit_dtype(tampered, "bf16")
    states = synth.to_commit_dtype(np.concatenate(upstream), "bf16").to(DEV)
    rep = model.verify_segment(states, 2, 4, synth.cu_seqlens(wl), comm_t.to(DEV), cs, cp, want_hidden=True)
    g = rep.cpu()
    o = vo.verify_segment(om, upstream, 2, 4, comm_t.to(torch.float64).numpy(), cs, cp, vo.Tol(), "bf16")
    assert g["stats"].shape == (len(cs), 2, vb.NSTAT)
    assert_parity(g, o, expect_reject=[4])
    assert g["first_bad_layer"][4] == 1 and g["pos_ok"].sum() == len(cs) - 1  # index counted from layer_begin
    # the same entry point from the embeddings reproduces the full pass over the first blocks
    with pytest.raises(vb.VerillmError) as e:
        model.verify_segment(states, 3, 3, synth.cu_seqlens(wl), comm_t.to(DEV), cs, cp)
    assert e.value.code == vb.E_RANGE


def test_nonfinite_recorded_states_reject_only_their_sequence(tiny):
    """Two packed sequences whose lengths are not multiples of the 64-key tile: the last key tile of the first
    covers the first rows of the second.  Inf / NaN (and an absurdly large value) in the second sequence's
    recorded input states reject that sequence as a whole, as the exact recomputation does (one such entry
    makes every state of its sequence non-finite), while the first sequence's statistics and verdict are those
    of the clean run, bit for bit; a following, smaller clean call on the same handle is unaffected."""
    wl, _, om, _, _, _, _ = tiny
    rng = np.random.default_rng(21)
    lens = [37, 45]
    states = [vo.round_to_bf16(rng.standard_normal((n, wl.shape.d_model)) * 0.5) for n in lens]
    cu = np.array([0, 37, 82], np.int32)
    cs = np.array([0, 0, 1, 1, 0], np.int32)
    cp = np.array([36, 3, 0, 44, 20], np.int32)
    outs = vo.forward_segment_batch(om, states, 0, 1)
    honest = np.stack([outs[s][:, p] for s, p in zip(cs, cp)], axis=1)
    comm = synth.to_commit_dtype(honest, "bf16").to(DEV)
    model = vb.Model(wl.shape, 128, len(cs), 2, DEV)
    model.load_globals(synth.embed_weights(wl, DEV), synth.final_norm_weights(wl, DEV))
    model.load_layer(0, synth.layer_weights(wl, 0, DEV))
    clean_in = synth.to_commit_dtype(np.concatenate(states), "f32")
    clean = model.verify_segment(clean_in.to(DEV), 0, 1, cu, comm, cs, cp, want_hidden=True).cpu()
    assert clean["pos_ok"].all() and clean["seq_ok"].tolist() == [1, 1]
    for bad_value, where in ((float("inf"), (37 + 5, 7)), (float("nan"), (37 + 44, 255)), (-3e20, (37 + 0, 0))):
        bad_in = clean_in.clone()
        bad_in[where] = bad_value
        g = model.verify_segment(bad_in.to(DEV), 0, 1, cu, comm, cs, cp, want_hidden=True).cpu()
        assert g["status"] == 0
        assert g["seq_ok"].tolist() == [1, 0]
        assert g["pos_ok"].tolist() == [1, 1, 0, 0, 1] and g["first_bad_layer"].tolist() == [-1, -1, 0, 0, -1]
        first = [0, 1, 4]
        assert np.array_equal(g["stats"][first], clean["stats"][first])
        assert np.array_equal(g["hidden"][:, first], clean["hidden"][:, first])
        assert np.isfinite(g["hidden"]).all()
        assert g["seq_score"][0] == clean["seq_score"][0]
        # the oracle on the same input: every state of the poisoned sequence is non-finite, the other is untouched
        bad_states = [states[0], bad_in[37:].to(torch.float64).numpy()]
        with np.errstate(all="ignore"):
            o = vo.verify_segment(om, bad_states, 0, 1, comm.cpu().to(torch.float64).numpy(), cs, cp, vo.Tol(), "bf16")
        if abs(bad_value) > 1e30 or bad_value != bad_value:
            assert np.array_equal(g["pos_ok"], o.pos_ok) and np.array_equal(g["seq_ok"], o.seq_ok)
            assert np.array_equal(g["first_bad_layer"], o.first_bad_layer)
        # a smaller clean call afterwards (the first sequence alone) reproduces the clean result
        sub = model.verify_segment(clean_in[:37].to(DEV), 0, 1, cu[:2], comm[:, first].contiguous(), cs[first], cp[first],
                                   want_hidden=True).cpu()
        assert np.array_equal(sub["stats"], clean["stats"][first]) and sub["seq_ok"].tolist() == [1]
    model.close()


def test_device_error_rejects_sequences_without_checked_positions(tiny):
    """An out-of-vocabulary token invalidates the whole call: also a sequence that has no checked position, and a
    call without any check, must come back rejected."""
    wl, tokens, om, cs, cp, committed, model = tiny
    small = vb.Model(wl.shape, 64, 4, 2, DEV)
    small.load_globals(synth.embed_weights(wl, DEV), synth.final_norm_weights(wl, DEV))
    small.load_layer(0, synth.layer_weights(wl, 0, DEV))
    toks = torch.from_numpy(tokens.reshape(-1)[:64].copy()).to(DEV)
    cu = np.array([0, 40, 64], np.int32)
    comm = synth.to_commit_dtype(committed[:, :2], "bf16").to(DEV)
    ok = small.verify_prefill(toks, cu, comm, [0, 0], [int(cp[0]) % 40, int(cp[1]) % 40]).cpu()
    assert ok["status"] == 0 and ok["seq_ok"][1] == 1  # sequence 1 has no checked position
    bad = toks.clone()
    bad[50] = -7  # inside sequence 1
    rep = small.verify_prefill(bad, cu, comm, [0, 0], [int(cp[0]) % 40, int(cp[1]) % 40]).cpu()
    assert rep["status"] == vb.DEV_TOKEN_RANGE and rep["seq_ok"].tolist() == [0, 0] and not rep["pos_ok"].any()
    rep = small.verify_prefill(bad, cu, None, [], []).cpu()
    assert rep["status"] == vb.DEV_TOKEN_RANGE and rep["seq_ok"].tolist() == [0, 0]
    small.close()


def test_pinned_host_arrays_may_be_overwritten_when_the_call_returns(tiny):
    """The header's promise: host arrays are free again at return.  With page-locked arrays a direct asynchronous
    copy would still be queued behind the work already on the stream; the library copies them first."""
    wl, tokens, om, cs, cp, committed, model = tiny
    comm = synth.to_commit_dtype(committed, "bf16").to(DEV)
    flat = torch.from_numpy(tokens.reshape(-1)).to(DEV)
    ref = model.verify_prefill(flat, synth.cu_seqlens(wl), comm, cs, cp, want_hidden=True).cpu()
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).pin_memory()
    cu_p, cs_p, cp_p = pin(synth.cu_seqlens(wl)), pin(cs), pin(cp)
    # keep the stream busy so that the call's own copies cannot have run when it returns
    a = torch.randn(4096, 4096, device=DEV)
    for _ in range(20):
        a = a @ a * 1e-2
    rep = model.verify_prefill(flat, cu_p.numpy(), comm, cs_p.numpy(), cp_p.numpy(), want_hidden=True)
    cu_p.fill_(0); cs_p.fill_(0); cp_p.fill_(63)  # the caller reuses its arrays at once
    torch.cuda.synchronize()
    g = rep.cpu()
    assert np.array_equal(g["stats"], ref["stats"]) and np.array_equal(g["hidden"], ref["hidden"])
    assert np.array_equal(g["seq_ok"], ref["seq_ok"]) and np.array_equal(g["seq_score"], ref["seq_score"])
    # the standalone comparison keeps the same promise for its slot-to-sequence map
    hid = torch.from_numpy(ref["hidden"]).to(DEV)
    seq_of = (np.arange(len(cs)) % 2).astype(np.int32)
    ref2 = vb.compare(hid, comm, seq_of, 2).cpu()
    seq_p = pin(seq_of)
    for _ in range(20):
        a = a @ a * 1e-2
    r2 = vb.compare(hid, comm, seq_p.numpy(), 2)
    seq_p.fill_(1)  # every slot would move to sequence 1
    torch.cuda.synchronize()
    r2 = r2.cpu()
    assert np.array_equal(r2["stats"], ref2["stats"]) and np.array_equal(r2["seq_score"], ref2["seq_score"])
    assert ref2["seq_score"][0] != ref2["seq_score"][1]


def test_bounded_wait_runs_out_and_the_context_stays_usable(tiny):
    """Failure detection: the wait every pipeline uses, given a short limit and a barrier nothing signals, gives
    up, records VERILLM_DEV_WAIT_TIMEOUT and returns; the next verification on the same context is correct."""
    wl, tokens, om, cs, cp, committed, model = tiny
    status, gave_up = vb.selftest_wait_timeout(200_000, DEV)  # about 0.1 ms of SM clocks
    torch.cuda.synchronize()
    assert int(status.item()) == vb.DEV_WAIT_TIMEOUT and int(gave_up.item()) == 1
    with pytest.raises(vb.VerillmError):
        vb.selftest_wait_timeout(0, DEV)
    with pytest.raises(vb.VerillmError):
        vb.selftest_wait_timeout(10 ** 12, DEV)  # limits beyond a second or so are refused
    g, o = run_both(model, om, wl, tokens, committed, cs, cp)
    assert_parity(g, o)
    assert g["pos_ok"].all()
