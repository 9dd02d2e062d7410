"""Parity with the oracle at the full size of the three large configurations, in the launch configuration
bench.py times.

The oracle recomputes every checked position it is asked for by one causal pass over the prefix that ends
there (under the causal mask later tokens cannot change earlier states; pinned by the prefix-invariance
test), one layer of weights at a time.  Committed states are the oracle's own states rounded to bf16; no
oracle input and no expected value comes from the CUDA path.

 - Llama-3-8B shape, 8 x 1024 tokens, 32 layers: all 82 positions of the seeded check set, with the
   configuration's tampering (one of eight sequences) in both forms: noise of 10 x the tolerance on one
   committed state, and a substituted token at a checked position.
 - Long context, 2 x 4096 tokens, 32 layers: sampled positions, one of them beyond position 2048; the other
   positions of the seeded check set carry the decode entry point's trace (properties only).
 - Llama-3-70B widths, 1 x 2048 tokens: 8 layers always; all 80 layers when VERILLM_SLOW=1 (a quarter of an
   hour of oracle time, most of it spent materialising 80 x 6.8 GB of float64 weights).
"""
import os

import numpy as np
import pytest
import torch

from oracle import verillm_oracle as vo
from paper_2509_24257_b200 import binding as vb
from paper_2509_24257_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
REL = vo.STAT_NAMES.index("rel_l2")
TOL = 5e-2
HIDDEN_TOL = 2e-2


def _oracle_states(wl, seqs, check_seq, check_pos):
    """Oracle states [n_layers, n_check, d] at the given (index into seqs, position) pairs, prefixes only."""
    need = np.concatenate([np.asarray(seqs[s])[: p + 1] for s, p in zip(check_seq, check_pos)])
    om = H.oracle_model_streamed(wl, need, DEV)
    zeros = np.zeros((wl.shape.n_layers, len(check_seq), wl.shape.d_model))
    return vo.verify_prefill(om, seqs, zeros, np.asarray(check_seq), np.asarray(check_pos), vo.Tol(), "bf16",
                             prefix_only=True).hidden


def _oracle_verdict(hidden, comm_t, check_seq, batch):
    stats = np.transpose(vo.compare_stats(hidden, comm_t.to(torch.float64).numpy(), "bf16", vo.Tol()), (1, 0, 2))
    return (stats,) + vo.verdict(stats, np.asarray(check_seq), batch, vo.Tol())


def _report(name, rel):
    print(f"\n[{name}] GPU vs oracle hidden rel-L2: max {rel.max():.3e}; per-layer max "
          + " ".join(f"{x:.2e}" for x in rel.max(axis=1)))


def test_llama8b_every_checked_position_with_noise_and_token_swap():
    wl = synth.WORKLOADS["llama8b"]
    L, B = wl.shape.n_layers, wl.batch
    tokens = synth.token_streams(wl)
    cs, cp = synth.check_positions(wl)
    assert len(cs) == wl.n_check == 82
    rng = synth.tamper_rng(wl)
    bad_seq = int(rng.choice(B, size=int(np.ceil(0.1 * B)), replace=False)[0])
    in_bad = np.nonzero(cs == bad_seq)[0]
    assert len(in_bad) >= 3
    by_pos = in_bad[np.argsort(cp[in_bad])]
    swap_slot = int(by_pos[len(by_pos) // 2])  # checked positions of that sequence lie before and after it
    noise_slot, noise_layer = int(by_pos[0]), int(rng.integers(0, L))
    forged = synth.swap_token(tokens, bad_seq, int(cp[swap_slot]), wl.shape.vocab, rng)

    # one oracle pass: the eight served sequences plus the forged copy of the tampered one
    seqs = list(tokens) + [forged[bad_seq]]
    cs_x = np.concatenate([cs, np.full(len(in_bad), B, np.int32)])
    cp_x = np.concatenate([cp, cp[in_bad]])
    states = _oracle_states(wl, seqs, cs_x, cp_x)
    honest = states[:, : len(cs)]
    forged_states = honest.copy()
    forged_states[:, in_bad] = states[:, len(cs):]

    trace = vo.round_to_bf16(honest)  # what the prover committed: the original tokens' states
    comm_honest = synth.to_commit_dtype(trace, "bf16")
    comm_noise = synth.to_commit_dtype(synth.add_state_noise(trace, [noise_slot], [noise_layer], 10 * TOL, rng), "bf16")

    model = H.gpu_model(wl, len(cs))
    cu = synth.cu_seqlens(wl)
    flat = torch.from_numpy(tokens.reshape(-1)).to(DEV)
    flat_forged = torch.from_numpy(forged.reshape(-1)).to(DEV)

    # ---- (a) state noise of 10 x tol at one (position, layer)
    g = model.verify_prefill(flat, cu, comm_noise.to(DEV), cs, cp, want_hidden=True).cpu()
    assert g["status"] == 0 and model.last_launch_count() == 3 + 1 + 5 * L + 2
    rel = H.rel_l2(g["hidden"], honest)
    _report("llama8b 8x1024 L32, 82 slots", rel)
    assert rel.max() <= HIDDEN_TOL
    stats_o, pos_ok_o, first_bad_o, seq_ok_o, score_o = _oracle_verdict(honest, comm_noise, cs, B)
    o_rel = stats_o[..., REL]
    assert not ((o_rel > TOL / 2) & (o_rel < 2 * TOL)).any()  # no cell inside the gray band
    assert np.array_equal(g["pos_ok"], pos_ok_o) and np.array_equal(g["first_bad_layer"], first_bad_o)
    assert np.array_equal(g["seq_ok"], seq_ok_o)
    assert pos_ok_o.sum() == len(cs) - 1 and pos_ok_o[noise_slot] == 0 and first_bad_o[noise_slot] == noise_layer
    assert seq_ok_o.tolist() == [0 if b == bad_seq else 1 for b in range(B)]
    assert np.all(np.abs(g["stats"][..., REL] - o_rel) <= 1.2 * HIDDEN_TOL)

    # ---- (b) a substituted token at a checked position: the verifier sees the forged sequence, the trace is
    # the original one's
    g = model.verify_prefill(flat_forged, cu, comm_honest.to(DEV), cs, cp, want_hidden=True).cpu()
    assert g["status"] == 0
    rel = H.rel_l2(g["hidden"], forged_states)
    assert rel.max() <= HIDDEN_TOL
    stats_o, pos_ok_o, first_bad_o, seq_ok_o, _ = _oracle_verdict(forged_states, comm_honest, cs, B)
    o_rel = stats_o[..., REL]
    gray_pos = ((o_rel > TOL / 2) & (o_rel < 2 * TOL)).any(axis=1)
    later = (cs == bad_seq) & (cp > cp[swap_slot])
    print(f"[token swap at position {int(cp[swap_slot])}] oracle rel-L2 at the swapped position, layer 0: "
          f"{o_rel[swap_slot, 0]:.3f}; later checked positions of the sequence: "
          + " ".join(f"{int(p)}:{o_rel[s].max():.3f}" for s, p in zip(np.nonzero(later)[0], cp[later])))
    assert not gray_pos[~later].any()  # only positions after the swap may fall inside the band
    clear = ~gray_pos
    assert np.array_equal(g["pos_ok"][clear], pos_ok_o[clear])
    assert np.array_equal(g["first_bad_layer"][clear], first_bad_o[clear])
    assert o_rel[swap_slot, 0] >= 2 * TOL and g["pos_ok"][swap_slot] == 0 and g["first_bad_layer"][swap_slot] == 0
    earlier = (cs == bad_seq) & (cp < cp[swap_slot])
    assert earlier.any() and g["pos_ok"][earlier].all() and g["pos_ok"][cs != bad_seq].all()
    assert g["seq_ok"].tolist() == seq_ok_o.tolist() == [0 if b == bad_seq else 1 for b in range(B)]
    model.close()


def _sampled_parity(wl, sampled, bad_slot, bad_layer, with_decode_trace=False):
    """Whole batch on the GPU, the oracle on the sampled (sequence, position) pairs.  With the decode trace,
    the rest of the seeded check set rides along, carrying the trace of the decode entry point."""
    tokens = synth.token_streams(wl)
    n_s = len(sampled)
    cs = np.array([s for s, _ in sampled], np.int32)
    cp = np.array([p for _, p in sampled], np.int32)
    if with_decode_trace:
        cs_all, cp_all = synth.check_positions(wl)
        keep = [i for i in range(len(cs_all)) if (int(cs_all[i]), int(cp_all[i])) not in sampled][: len(cs_all) - n_s]
        cs, cp = np.concatenate([cs, cs_all[keep]]), np.concatenate([cp, cp_all[keep]])
        assert len(cs) == wl.n_check
    hidden_o = _oracle_states(wl, list(tokens), cs[:n_s], cp[:n_s])
    honest = vo.round_to_bf16(hidden_o)
    tampered = synth.add_state_noise(honest, [bad_slot], [bad_layer], 10 * TOL, synth.tamper_rng(wl))
    comm_s = synth.to_commit_dtype(tampered, "bf16")

    model = H.gpu_model(wl, len(cs))
    flat = torch.from_numpy(tokens.reshape(-1)).to(DEV)
    cu = synth.cu_seqlens(wl)
    if with_decode_trace:
        committed = model.decode_commit(flat, cu, wl.prompt_len, cs, cp, torch.bfloat16).contiguous().clone()
        committed[:, :n_s] = comm_s.to(DEV)
    else:
        committed = comm_s.to(DEV)
    g = model.verify_prefill(flat, cu, committed, cs, cp, want_hidden=True).cpu()
    model.close()
    assert g["status"] == 0
    rel = H.rel_l2(g["hidden"][:, :n_s], hidden_o)
    _report(f"{wl.name} {wl.batch}x{wl.seq_len} L{wl.shape.n_layers}, {n_s} sampled slots", rel)
    assert rel.max() <= HIDDEN_TOL, rel.max()
    stats_o, pos_ok_o, first_bad_o, _, _ = _oracle_verdict(hidden_o, comm_s, cs[:n_s], wl.batch)
    o_rel = stats_o[..., REL]
    assert not ((o_rel > TOL / 2) & (o_rel < 2 * TOL)).any()
    assert np.array_equal(g["pos_ok"][:n_s], pos_ok_o) and np.array_equal(g["first_bad_layer"][:n_s], first_bad_o)
    assert pos_ok_o.sum() == n_s - 1 and pos_ok_o[bad_slot] == 0 and first_bad_o[bad_slot] == bad_layer
    assert np.all(np.abs(g["stats"][:n_s, :, REL] - o_rel) <= 1.2 * HIDDEN_TOL)
    bad_seq = int(cs[bad_slot])
    if with_decode_trace:
        # the honest decode trace of the remaining slots is accepted, with deviations in the rounding-noise range
        assert g["pos_ok"][n_s:].all() and (g["first_bad_layer"][n_s:] == -1).all()
        assert 0 < g["stats"][n_s:, :, REL].max() <= 2.5e-2
    assert g["seq_ok"].tolist() == [0 if b == bad_seq else 1 for b in range(wl.batch)]
    return g


def test_long_context_8b_full_depth_with_a_position_beyond_2048():
    """2 x 4096 tokens at the 8B shape, all 32 layers: up to 64 key tiles per query tile in attention, one check
    per two hundred rows, one sampled position past the middle of its sequence and one at a tile boundary."""
    wl = synth.WORKLOADS["llama8b_long"]
    _sampled_parity(wl, [(0, 5), (0, 700), (1, 2100), (1, 63)], bad_slot=2, bad_layer=17, with_decode_trace=True)


def test_long_context_8b_width_last_position_two_layers():
    """The very last position of a 4096-token sequence (prefix of the full length), at reduced depth."""
    wl = synth.WORKLOADS["llama8b_long"].with_layers(2)
    _sampled_parity(wl, [(0, 5), (1, 2048), (1, 4095)], bad_slot=1, bad_layer=1)


def test_llama70b_width_eight_layers():
    """Llama-3-70B widths (d 8192, 64/8 heads, FFN 28672), 8 layers, the configured 1 x 2048 batch."""
    wl = synth.WORKLOADS["llama70b"].with_layers(8)
    _sampled_parity(wl, [(0, 0), (0, 63), (0, 129), (0, 300)], bad_slot=2, bad_layer=5)


@pytest.mark.skipif(os.environ.get("VERILLM_SLOW") != "1", reason="all 80 layers of the 70B shape: set VERILLM_SLOW=1")
def test_llama70b_all_eighty_layers():
    wl = synth.WORKLOADS["llama70b"]
    _sampled_parity(wl, [(0, 0), (0, 63), (0, 129)], bad_slot=1, bad_layer=60)
