"""Threshold sensitivity of the bit-aware tests on honest and quantised-prover traces.

    python -m paper_2509_24257_b200.calibrate [--workload small] [--bits 8] [--check-frac 0.25]

Follows the paper's "Threshold Sensitivity Analysis": each of the four thresholds (P_e, |e|, P_m, P_w) is
varied while the others stay at their selected values, and FPR / FNR / TPR / TNR are read off cells of
honest traces and of attack traces.  Here the honest prover is the library's bf16 KV-cache decode, the
attacker is the same decode on fake-quantised weights (synth.fake_quantise), the verifier recomputes with
the true weights; every step runs in the library's kernels (decode_commit, verify_prefill,
threshold_sweep), this module only arranges the calls and prints the table.
"""
from __future__ import annotations

import argparse
import dataclasses
from typing import Dict, List, Sequence, Tuple

import numpy as np
import torch

from . import binding as vb
from . import synth

# selected thresholds for bf16 traces of the synthetic models and the grid around them
SELECTED = {"pe_max": 0.035, "e_abs_max": 0.01, "pm_min": 0.75, "pw_min": 0.55}
GRID = {
    "pe_max": (0.02, 0.03, 0.035, 0.05, 0.08),
    "e_abs_max": (0.0005, 0.002, 0.01, 0.05),
    "pm_min": (0.50, 0.75, 0.90, 0.95),
    "pw_min": (0.30, 0.45, 0.55, 0.70, 0.80),
}


def variants(selected: Dict[str, float] = SELECTED, grid: Dict[str, Sequence[float]] = GRID) -> Tuple[List[vb.Tol], List[Tuple[str, float]]]:
    """One tolerance set per (parameter, value) of the grid, the other parameters at their selected values;
    only the bit-aware tests are enabled."""
    tols, labels = [], []
    for name, values in grid.items():
        for val in values:
            kw = dict(selected)
            kw[name] = val
            tols.append(vb.default_tol(rel_l2=0.0, bit_aware=True, **kw))
            labels.append((name, float(val)))
    return tols, labels


def trace_stats(wl: synth.Workload, bits: int, device: torch.device):
    """Statistics [n_cells][NSTAT] (device) of honest cells followed by attack cells, and the class flags."""
    w = synth.model_weights(wl, device)
    cs, cp = synth.check_positions(wl)
    cu = synth.cu_seqlens(wl)
    flat = torch.from_numpy(synth.token_streams(wl).reshape(-1)).to(device)
    verifier = vb.Model.from_weights(wl.shape, w, wl.n_tokens, len(cs), wl.batch, device)
    attacker = vb.Model.from_weights(wl.shape, synth.quantised_model_weights(w, bits), wl.n_tokens, len(cs), wl.batch, device)
    tol = vb.default_tol()
    parts = []
    for prover in (verifier, attacker):
        committed = prover.decode_commit(flat, cu, wl.prompt_len, cs, cp, torch.bfloat16).contiguous()
        rep = verifier.verify_prefill(flat, cu, committed, cs, cp, tol)
        parts.append(rep.stats.reshape(-1, vb.NSTAT).clone())
    attacker.close()
    verifier.close()
    stats = torch.cat(parts).contiguous()
    is_attack = torch.zeros(stats.shape[0], dtype=torch.uint8, device=device)
    is_attack[parts[0].shape[0]:] = 1
    return stats, is_attack


def sensitivity_rows(stats: torch.Tensor, is_attack: torch.Tensor, selected=SELECTED, grid=GRID):
    """[(parameter, value, FPR, FNR, TPR, TNR)] from one verillm_threshold_sweep call."""
    tols, labels = variants(selected, grid)
    counts = vb.threshold_sweep(stats, is_attack, tols).cpu().numpy().astype(np.float64)
    rows = []
    for (name, val), c in zip(labels, counts):
        fpr, fnr = c[1] / max(c[0] + c[1], 1.0), c[2] / max(c[2] + c[3], 1.0)
        rows.append((name, val, fpr, fnr, 1.0 - fnr, 1.0 - fpr))
    return rows


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="small")
    ap.add_argument("--bits", type=int, default=8)
    ap.add_argument("--check-frac", type=float, default=0.25)
    args = ap.parse_args()
    wl = dataclasses.replace(synth.WORKLOADS[args.workload], check_frac=args.check_frac)
    stats, is_attack = trace_stats(wl, args.bits, torch.device("cuda", 0))
    print(f"{wl.name}: {int((is_attack == 0).sum())} honest and {int(is_attack.sum())} int{args.bits} attack cells")
    print(f"{'threshold':>22} {'FPR':>8} {'FNR':>8} {'TPR':>8} {'TNR':>8}")
    for name, val, fpr, fnr, tpr, tnr in sensitivity_rows(stats, is_attack):
        mark = " (selected)" if SELECTED[name] == val else ""
        print(f"{name + ' = ' + format(val, 'g'):>22} {100 * fpr:7.2f}% {100 * fnr:7.2f}% {100 * tpr:7.2f}% {100 * tnr:7.2f}%{mark}")


if __name__ == "__main__":
    main()
