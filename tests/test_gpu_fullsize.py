"""Parity at the full Llama-3-8B-shaped configuration (32 layers, 8 x 1024 tokens, 82 checked positions),
in the launch configuration bench.py times.

The oracle cannot recompute 8192 tokens x 32 layers in fp64 in test time, so it recomputes sampled outputs
one by one: a handful of positions whose causal prefixes are short (weights streamed one layer at a
time).  Their committed states are the oracle's own states rounded to bf16, one of them tampered with
noise of 10 x the tolerance.  The other check slots of the configuration carry the trace produced by the
decode entry point and are checked through properties that hold at any size: an honest trace is
accepted everywhere, its deviation stays inside the rounding-noise range, and results do not depend on
which other positions are checked.
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
REL = vo.STAT_NAMES.index("rel_l2")


def test_llama8b_full_depth_sampled_positions_and_honest_trace():
    wl = synth.WORKLOADS["llama8b"]
    tokens = synth.token_streams(wl)
    cs_all, cp_all = synth.check_positions(wl)
    # sampled outputs: short causal prefixes in three sequences (first, ragged middle, tile boundaries)
    sampled = [(0, 0), (0, 63), (3, 17), (3, 127), (7, 100), (7, 64)]
    keep = [i for i in range(len(cs_all)) if (int(cs_all[i]), int(cp_all[i])) not in sampled][: len(cs_all) - len(sampled)]
    cs = np.concatenate([np.array([s for s, _ in sampled], np.int32), cs_all[keep]])
    cp = np.concatenate([np.array([p for _, p in sampled], np.int32), cp_all[keep]])
    n_s = len(sampled)
    assert len(cs) == wl.n_check == 82

    model = H.gpu_model(wl, len(cs))
    flat = torch.from_numpy(tokens.reshape(-1)).to(DEV)
    cu = synth.cu_seqlens(wl)

    # oracle on the sampled slots only (prefix recomputation, one layer of weights at a time)
    om = H.oracle_model_streamed(wl, np.concatenate([tokens[s][: p + 1] for s, p in sampled]), DEV)
    zeros = np.zeros((wl.shape.n_layers, n_s, wl.shape.d_model))
    pre = vo.verify_prefill(om, list(tokens), zeros, cs[:n_s], cp[:n_s], vo.Tol(), "bf16", prefix_only=True)
    honest = vo.round_to_bf16(pre.hidden)
    rng = synth.tamper_rng(wl)
    bad_slot, bad_layer = 3, 20
    tampered = synth.add_state_noise(honest, [bad_slot], [bad_layer], 10 * 5e-2, rng)
    comm_sampled = synth.to_commit_dtype(tampered, "bf16")

    # the remaining slots: the prover-side decode trace (GPU), honest
    trace = model.decode_commit(flat, cu, wl.prompt_len, cs, cp, torch.bfloat16).contiguous()
    committed = trace.clone()
    committed[:, :n_s] = comm_sampled.to(DEV)

    rep = model.verify_prefill(flat, cu, committed, cs, cp, want_hidden=True)
    torch.cuda.synchronize()
    g = rep.cpu()
    assert g["status"] == 0 and model.last_launch_count() == 3 + 1 + 5 * 32 + 2

    # --- sampled outputs against the oracle
    stats_o = np.transpose(vo.compare_stats(pre.hidden, comm_sampled.to(torch.float64).numpy(), "bf16", vo.Tol()), (1, 0, 2))
    pos_ok_o, first_bad_o, _, _ = vo.verdict(stats_o, cs[:n_s], wl.batch, vo.Tol())
    rel = H.rel_l2(g["hidden"][:, :n_s], pre.hidden)
    assert rel.max() <= 2e-2, f"hidden-state rel-L2 {rel.max():.3e} (per layer max {rel.max(axis=1)})"
    o_rel = stats_o[..., REL]
    assert not ((o_rel > 2.5e-2) & (o_rel < 1e-1)).any()  # nothing inside the gray band
    assert np.array_equal(g["pos_ok"][:n_s], pos_ok_o) and np.array_equal(g["first_bad_layer"][:n_s], first_bad_o)
    assert pos_ok_o.tolist() == [1, 1, 1, 0, 1, 1] and first_bad_o[bad_slot] == bad_layer
    assert np.all(np.abs(g["stats"][:n_s, :, REL] - o_rel) <= 2.4e-2)

    # --- properties on the honest decode trace of the remaining slots
    assert g["pos_ok"][n_s:].all() and (g["first_bad_layer"][n_s:] == -1).all()
    honest_rel = g["stats"][n_s:, :, REL]
    assert 0 < honest_rel.max() <= 2.5e-2, honest_rel.max()
    seq_ok = g["seq_ok"].tolist()
    assert seq_ok[3] == 0 and all(seq_ok[b] == 1 for b in range(wl.batch) if b != 3)
    # a state does not depend on which other positions are checked, nor on the batch around it:
    # the same positions verified alone give bit-identical hidden states
    sub = [0, 3, n_s, len(cs) - 1]
    rep2 = model.verify_prefill(flat, cu, committed[:, sub].contiguous(), cs[sub], cp[sub], want_hidden=True).cpu()
    assert np.array_equal(rep2["hidden"], g["hidden"][:, sub])
    assert np.array_equal(rep2["stats"], g["stats"][sub])
    model.close()


def _sampled_parity(wl, sampled, bad_slot, bad_layer, oracle_device=DEV):
    """Runs the whole batch on the GPU and the oracle on the sampled (sequence, position) pairs only."""
    tokens = synth.token_streams(wl)
    cs = np.array([s for s, _ in sampled], np.int32)
    cp = np.array([p for _, p in sampled], np.int32)
    model = H.gpu_model(wl, len(cs))
    om = H.oracle_model_streamed(wl, np.concatenate([tokens[s][: p + 1] for s, p in sampled]), oracle_device)
    zeros = np.zeros((wl.shape.n_layers, len(cs), wl.shape.d_model))
    pre = vo.verify_prefill(om, list(tokens), zeros, cs, cp, vo.Tol(), "bf16", prefix_only=True)
    honest = vo.round_to_bf16(pre.hidden)
    tampered = synth.add_state_noise(honest, [bad_slot], [bad_layer], 10 * 5e-2, synth.tamper_rng(wl))
    comm = synth.to_commit_dtype(tampered, "bf16")
    flat = torch.from_numpy(tokens.reshape(-1)).to(DEV)
    g = model.verify_prefill(flat, synth.cu_seqlens(wl), comm.to(DEV), cs, cp, want_hidden=True).cpu()
    model.close()
    stats_o = np.transpose(vo.compare_stats(pre.hidden, comm.to(torch.float64).numpy(), "bf16", vo.Tol()), (1, 0, 2))
    pos_ok_o, first_bad_o, seq_ok_o, _ = vo.verdict(stats_o, cs, wl.batch, vo.Tol())
    assert g["status"] == 0
    rel = H.rel_l2(g["hidden"], pre.hidden)
    assert rel.max() <= 2e-2, rel.max()
    assert np.array_equal(g["pos_ok"], pos_ok_o) and np.array_equal(g["first_bad_layer"], first_bad_o)
    assert np.array_equal(g["seq_ok"], seq_ok_o)
    assert g["pos_ok"][bad_slot] == 0 and g["pos_ok"].sum() == len(cs) - 1 and g["first_bad_layer"][bad_slot] == bad_layer
    assert np.all(np.abs(g["stats"][..., REL] - stats_o[..., REL]) <= 2.4e-2)


def test_long_context_8b_width_sparse_checks():
    """2 sequences of 4096 tokens at the 8B widths (two layers): 64 key tiles per query tile in attention, and
    checks as sparse as one per thousand rows, among them the very last position of a sequence."""
    wl = synth.WORKLOADS["llama8b_long"].with_layers(2)
    _sampled_parity(wl, [(0, 5), (0, 700), (1, 2048), (1, 4095)], bad_slot=1, bad_layer=1)


def test_llama70b_width_single_layer():
    """Llama-3-70B widths (d 8192, 64/8 heads, FFN 28672), one layer, the configured 1 x 2048 batch."""
    wl = synth.WORKLOADS["llama70b"].with_layers(1)
    _sampled_parity(wl, [(0, 0), (0, 63), (0, 129), (0, 300)], bad_slot=2, bad_layer=0)
