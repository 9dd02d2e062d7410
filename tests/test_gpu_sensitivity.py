"""Threshold sensitivity sweep (verillm_threshold_sweep) on a B200: counts bit-exact against the oracle on the same
seeded statistics, decisions identical to the verdict kernel's, and the honest / quantised-prover separation that
the analysis is meant to show."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import verillm_oracle as vo
from paper_2509_24257_b200 import binding as vb
from paper_2509_24257_b200 import calibrate, synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _gpu_tol(t: vo.Tol) -> vb.Tol:
    return vb.default_tol(rel_l2=t.rel_l2, max_abs=t.max_abs, mae=t.mae, pe_max=t.pe_max, pm_min=t.pm_min,
                          pw_min=t.pw_min, e_abs_max=t.e_abs_max, z_large_max=t.z_large_max,
                          q_small_min=t.q_small_min, bit_aware=t.bit_aware)


def test_sweep_counts_match_the_oracle_bit_for_bit():
    """Statistics from the oracle's own comparison of seeded (recomputed, committed) pairs, with values placed
    exactly on thresholds; 64 tolerance sets; a cell count that is not a multiple of the block size."""
    rng = np.random.default_rng(11)
    n, d = 1000, 256
    c = rng.standard_normal((n, d)).astype(np.float32)
    noise = np.where(rng.random((n, 1)) < 0.5, 2e-3, 2e-2)  # "honest" and "attack" deviation levels
    h = (c.astype(np.float64) * (1 + noise * rng.standard_normal((n, d)))).astype(np.float32)
    h[5, 7] = np.nan
    stats = vo.compare_stats(h, vo.round_to(c.astype(np.float64), "bf16"), "bf16", vo.Tol()).astype(np.float32)
    attack = (noise[:, 0] > 1e-2)
    pe, pw = vo.STAT_NAMES.index("p_e"), vo.STAT_NAMES.index("p_w")
    stats[10, pe] = np.float32(0.05)   # exactly on a strict bound
    stats[11, pw] = np.float32(0.80)
    variants = [vo.Tol()] + [vo.Tol(rel_l2=0.0, bit_aware=True, pe_max=float(a), pw_min=float(b), pm_min=float(m), e_abs_max=float(e))
                             for a, b, m, e in zip(rng.uniform(0.0, 0.2, 63), rng.uniform(0.0, 1.0, 63),
                                                   rng.uniform(0.3, 1.0, 63), rng.uniform(0.0, 0.01, 63))]
    variants[1] = vo.Tol(bit_aware=True)
    want = vo.threshold_sweep(stats, attack, variants)
    got = vb.threshold_sweep(torch.from_numpy(stats).to(DEV), torch.from_numpy(attack.astype(np.uint8)).to(DEV),
                             [_gpu_tol(t) for t in variants])
    assert np.array_equal(got.cpu().numpy().astype(np.int64), want)
    assert want[0, 3] >= 1  # the NaN cell is rejected even by the loosest set

    # same tests, two kernels: with one layer per position, verdict_kernel accepts a position iff the sweep accepts
    # its cell (statistics produced on the device by the comparison path from the same pairs)
    tol = vb.default_tol(bit_aware=True, pe_max=0.06, pw_min=0.4)
    rep = vb.compare(torch.from_numpy(h[None]).to(DEV), torch.from_numpy(c[None]).to(DEV).to(torch.bfloat16),
                     np.zeros(n, dtype=np.int32), 1, tol)
    torch.cuda.synchronize()
    pos_ok = rep.pos_ok.cpu().numpy().astype(bool)
    cnt = vb.threshold_sweep(rep.stats.reshape(n, vb.NSTAT).contiguous(), torch.from_numpy(attack.astype(np.uint8)).to(DEV),
                             [tol]).cpu().numpy()[0]
    assert cnt.tolist() == [int(np.sum(pos_ok & ~attack)), int(np.sum(~pos_ok & ~attack)),
                            int(np.sum(pos_ok & attack)), int(np.sum(~pos_ok & attack))]
    assert 0 < pos_ok.sum() < n
    with pytest.raises(vb.VerillmError) as e:
        vb.threshold_sweep(torch.from_numpy(stats).to(DEV), torch.from_numpy(attack.astype(np.uint8)).to(DEV),
                           [_gpu_tol(vo.Tol())] * 65)
    assert e.value.code == vb.E_SHAPE


def test_sensitivity_on_quantised_prover_traces():
    """Honest bf16 decode against a prover that serves int8-quantised weights (small configuration, a quarter of the
    positions checked): the sweep's decisions equal the verdict kernel's, the attack passes the plain rel-L2
    tolerance, and the bit-aware thresholds separate the two classes."""
    wl = dataclasses.replace(synth.WORKLOADS["small"], check_frac=0.25)
    stats, is_attack = calibrate.trace_stats(wl, 8, torch.device(DEV))
    L = wl.shape.n_layers
    n_cells = stats.shape[0]
    assert n_cells == 2 * wl.n_check * L and int(is_attack.sum()) == n_cells // 2

    tol = vb.default_tol(bit_aware=True, pe_max=0.035, pw_min=0.55)
    counts = vb.threshold_sweep(stats, is_attack, [vb.default_tol(), tol]).cpu().numpy()
    assert np.all(counts.sum(axis=1) == n_cells)

    # the quantised prover stays inside the plain tolerance: every attack cell passes rel-L2 <= 5e-2 ...
    assert counts[0, 3] == 0 and counts[0, 1] == 0
    # ... and the calibrated bit-aware set catches it while keeping honest cells
    n_h = counts[1, 0] + counts[1, 1]
    n_a = counts[1, 2] + counts[1, 3]
    assert counts[1, 1] / n_h <= 0.10, counts
    assert counts[1, 2] / n_a <= 0.02, counts

    rows = calibrate.sensitivity_rows(stats, is_attack)
    table = {(name, val): (fpr, fnr) for name, val, fpr, fnr, _, _ in rows}
    # loosening P_e lowers the false-positive rate and raises the false-negative rate (the table's trend)
    fprs = [table[("pe_max", v)][0] for v in calibrate.GRID["pe_max"]]
    fnrs = [table[("pe_max", v)][1] for v in calibrate.GRID["pe_max"]]
    assert all(a >= b for a, b in zip(fprs, fprs[1:])) and all(a <= b for a, b in zip(fnrs, fnrs[1:]))
