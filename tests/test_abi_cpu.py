"""Host-side checks that need no GPU: the library builds, loads and exports the declared ABI, rejects bad
arguments before touching a device, and the multi-process replica plumbing works over gloo."""
import ctypes
import os
import re
import sys

import pytest

from paper_2509_24257_b200 import binding as vb
from paper_2509_24257_b200 import build, dist as vdist, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def library():
    build.build_library()
    return vb.lib()


def test_library_exports_every_declared_symbol(library):
    header = open(os.path.join(ROOT, "include", "verillm.h")).read()
    declared = set(re.findall(r"\b(verillm_[a-z_0-9]+)\s*\(", header))
    assert declared == set(vb.EXPORTS)
    for name in declared:
        assert hasattr(library, name), name


def test_error_strings_and_default_tolerances(library):
    assert vb.strerror(0) == "ok"
    assert "range" in vb.strerror(vb.E_RANGE) and "shape" in vb.strerror(vb.E_SHAPE)
    t = vb.default_tol()
    assert abs(t.rel_l2 - 5e-2) < 1e-9 and t.flags == 0 and t.e_m == 7
    assert (round(t.pe_max, 4), round(t.pm_min, 4), round(t.pw_min, 4), round(t.e_abs_max, 4)) == (0.05, 0.75, 0.8, 0.01)
    assert vb.default_tol(bit_aware=True).flags == vb.TOL_BIT_AWARE


def test_bad_arguments_are_rejected_on_the_host(library):
    h = ctypes.c_void_p()
    bad = vb.Config(1, 256, 4, 4, 96, 768, 1024, 10000.0, 1e-5, 64, 4, 1)  # head_dim 96
    assert library.verillm_load_weights(ctypes.byref(bad), None, ctypes.byref(h)) == vb.E_SHAPE
    bad = vb.Config(1, 250, 4, 4, 64, 768, 1024, 10000.0, 1e-5, 64, 4, 1)  # d_model not a multiple of 64
    assert library.verillm_load_weights(ctypes.byref(bad), None, ctypes.byref(h)) == vb.E_SHAPE
    assert library.verillm_load_weights(None, None, ctypes.byref(h)) == vb.E_INVAL
    tol, rep = vb.default_tol(), vb.ReportC()
    assert library.verillm_verify_prefill(None, None, None, 1, None, 0, None, None, 0, ctypes.byref(tol), ctypes.byref(rep), None) == vb.E_INVAL
    assert library.verillm_compare(None, None, 0, 1, 1, 64, None, 1, ctypes.byref(tol), ctypes.byref(rep), None) == vb.E_INVAL
    assert library.verillm_op_gemm(None, None, None, 1, 1, 1, 0, None, None) == vb.E_INVAL
    z = ctypes.c_void_p()
    assert library.verillm_spot_check(None, 1, 1, None, None, None, 1, ctypes.c_float(0.1), ctypes.c_float(0.5), None, None, None, None) == vb.E_INVAL
    assert library.verillm_merkle_roots(None, 1, 8, None, None) == vb.E_INVAL
    assert library.verillm_token_match(None, None, None, 1, None, None, None, None) == vb.E_INVAL
    assert library.verillm_load_lm_head(None, None, 0) == vb.E_INVAL
    assert library.verillm_verify_segment(None, None, 0, 0, 1, None, 1, None, 0, None, None, 0, ctypes.byref(tol), ctypes.byref(rep), None) == vb.E_INVAL
    assert library.verillm_compare_noalloc(None, None, 0, 1, 1, 64, None, 1, ctypes.byref(tol), ctypes.byref(rep), None) == vb.E_INVAL
    library.verillm_free(None)  # a no-op


def test_missing_library_fails_loudly(monkeypatch):
    monkeypatch.setattr(vb, "_lib", None)
    monkeypatch.setattr(vb, "LIB_PATH", os.path.join(ROOT, "no_such_dir", "libverillm.so"))
    with pytest.raises(FileNotFoundError):
        vb.default_tol()


def test_product_never_touches_the_oracle():
    pkg = os.path.join(ROOT, "paper_2509_24257_b200")
    for dirpath, _, files in os.walk(pkg):
        if "_build" in dirpath:
            continue
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", text, re.M), f
                assert "verillm_oracle" not in text and "oracle/" not in text, f
    assert "paper_2509_24257_b200" not in open(os.path.join(ROOT, "oracle", "verillm_oracle.py")).read()


def _replica_worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    vdist.init("gloo")
    wl = vdist.replica_workload(synth.WORKLOADS["tiny"], rank)
    toks = synth.token_streams(wl)
    vdist.barrier()
    seconds = 0.5 * (rank + 1)  # rank 1 is the slow one
    value = vdist.aggregate_throughput(float(wl.n_tokens), seconds)
    out[rank] = (value, int(toks.sum()), vdist.max_over_ranks(float(rank)))
    vdist.shutdown()


def test_two_replicas_over_gloo_aggregate_tokens_over_slowest_rank():
    import torch.multiprocessing as mp

    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_replica_worker, args=(2, 29517, out), nprocs=2, join=True)
    (v0, s0, m0), (v1, s1, m1) = out[0], out[1]
    assert v0 == v1 == pytest.approx(2 * 64 / 1.0)  # all tokens of both replicas over the slower rank's second
    assert s0 != s1  # replicas verify different sequences
    assert m0 == m1 == 1.0


def test_workload_table_matches_the_stated_configs():
    w = synth.WORKLOADS
    names = ("tiny", "small", "llama8b", "llama8b_long", "llama70b")
    assert tuple(w[n].n_tokens for n in names) == (64, 2048, 8192, 8192, 2048)
    assert tuple(w[n].n_check for n in names) == (64, 20, 82, 41, 20)
    assert abs(w["llama8b"].total_flops() / 1e12 - 116.6) < 0.2 and abs(w["llama70b"].total_flops() / 1e12 - 285.9) < 0.5
    assert abs(w["llama8b"].shape.n_params() / 1e9 - 7.505) < 0.01  # embedding + 32 blocks, no output head


def test_reference_arm_prints_the_contract_line():
    """`bench.py --impl reference` times the oracle on the host cores and prints one JSON line with the same metric,
    unit and workload keys as the GPU arm, `impl`, a `cpu_baseline` describing the run and an `e2e` block without copies."""
    import json
    import subprocess

    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--workload", "tiny",
                          "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=300, cwd=root)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [l for l in out.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "verified_tokens_per_sec" and d["unit"] == "tokens/s"
    assert d["higher_is_better"] is True and d["vs_baseline"] is None and d["dtype"] == "f64" and d["gpu_launches"] == 0
    assert d["config"]["workload"] == "tiny" and d["value"] > 0 and d["steps"] == 1
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["value"] == d["value"] and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"] == {"value": d["value"], "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}
