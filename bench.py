#!/usr/bin/env python
"""Benchmark of the verifier prefill: verified tokens/s at the Llama-3-8B shape on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload llama8b]

A step is one verillm_verify_prefill call over one synthetic batch (8 sequences of 512 prompt + 512
generated tokens, 1 % of positions checked at every layer, 10 % of sequences tampered): embedding,
32 transformer blocks with the fused gather-and-compare epilogue, verdict.  Weights (15 GB) are
re-streamed from HBM every step, far more than the 126 MB L2, so no flush is needed between steps.
With N > 1 (torchrun) every rank runs an independent replica on its own sequences; there is no
collective on the data path.  Prints one JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC, UNIT = "verified_tokens_per_sec", "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
TOL_REL_L2 = 5e-2
# 32-bit integer instructions of one SHA-256 compression written out in full (64 rounds x 14, 48 schedule words
# x 10, 8 final adds), and the average the Merkle kernel executes per compression of a 4096-entry tree (profiler
# instruction count: the padding block of every inner node has a constant schedule, most of a leaf's folds away)
SHA256_INT_OPS = 64 * 14 + 48 * 10 + 8
SHA256_INT_OPS_EXECUTED = 1286
# of which funnel shifts (rotations): 6 per round everywhere, 4 per schedule word where a schedule is computed
# (all 48 words of an inner node's first block, about a third of a leaf's): about 490 on average
SHA256_FUNNEL_SHIFTS_EXECUTED = 490
GATE_UP_DRAM_BYTES_8B = 668.7e6 + 227.9e6  # measured, per launch, M = 8192 tokens at the 8B widths


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {k: float(p[k]) for k in FALLBACK_PEAKS if k in p}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index, self.proc, self.lines = gpu_index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100", "-i",
                 str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], None, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for ts, line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7 or not (t0 <= ts <= t1 + 0.2):
                continue
            try:
                sm.append(float(parts[0]))
                mx = float(parts[1])
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(sm)}


# ----------------------------------------------------------------------------------------------- CPU arm


def oracle_sample(wl, budget_s: float, device_for_weights: str):
    """Builds a bounded sample of the workload for the CPU oracle: one sequence prefix and the first
    layers, sized from a short calibration run so that one pass costs about `budget_s` seconds.
    Returns (run, description) where run() executes one pass and returns (tokens, seconds, layers)."""
    import torch
    from oracle import verillm_oracle as vo
    from paper_2509_24257_b200 import synth

    def bits(t):
        return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)

    shape = wl.shape
    tokens = synth.token_streams(wl)[0]
    ids = sorted(set(int(t) for t in tokens))
    embed = vo.as_f64(bits(synth.embed_weights(wl, device_for_weights, rows=torch.tensor(ids))))
    rows = {t: i for i, t in enumerate(ids)}
    final = vo.as_f64(bits(synth.final_norm_weights(wl, "cpu")))
    layer0 = {k: vo.as_f64(bits(v)) for k, v in synth.layer_weights(wl, 0, device_for_weights).items()}

    def model(n_layers):
        return vo.Model(n_layers, shape.d_model, shape.n_heads, shape.n_kv_heads, shape.head_dim, shape.d_ffn,
                        shape.vocab, float(shape.rope_base), float(shape.rms_eps), embed, final,
                        [layer0] * n_layers, rows)

    # calibration: one layer on 64 tokens (the cost is close to linear in tokens x layers)
    t0 = time.perf_counter()
    vo.forward_prefill_batch(model(1), [tokens[:64]])
    per_token_layer = (time.perf_counter() - t0) / 64.0
    n_layers = 2 if shape.n_layers >= 2 else 1
    T = int(min(len(tokens), max(64, (budget_s / (per_token_layer * n_layers)) // 64 * 64)))
    om = model(n_layers)
    n_chk = max(1, int(round(wl.check_frac * T)))
    check_pos = np.linspace(0, T - 1, n_chk).astype(np.int32)
    check_seq = np.zeros(n_chk, dtype=np.int32)
    committed = np.zeros((n_layers, n_chk, shape.d_model))
    tol = vo.Tol(rel_l2=TOL_REL_L2)

    def run():
        t0 = time.perf_counter()
        vo.verify_prefill(om, [tokens[:T]], committed, check_seq, check_pos, tol, "bf16")
        return T, time.perf_counter() - t0, n_layers

    desc = (f"oracle (numpy fp64) on 1 sequence x {T} tokens x {n_layers} of {shape.n_layers} layers at full width, "
            f"{n_chk} checked positions; tokens/s scaled by {n_layers}/{shape.n_layers} to the full depth")
    return run, desc


def cpu_cores() -> int:
    try:
        from threadpoolctl import threadpool_info

        n = max((p.get("num_threads", 1) for p in threadpool_info()), default=1)
    except Exception:
        n = 1
    return int(min(n, len(os.sched_getaffinity(0))))


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", 0))
    if rank != 0:
        return
    import torch

    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    budget = max(1.0, min(20.0, 150.0 / (args.steps + args.warmup)))
    run, desc = oracle_sample(wl, budget, dev)
    for _ in range(args.warmup):
        run()
    tot_tokens, tot_s = 0.0, 0.0
    for _ in range(args.steps):
        T, s, nl = run()
        tot_tokens += T * nl / wl.shape.n_layers
        tot_s += s
    value = tot_tokens / tot_s
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * tot_s / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "timing": "host wall clock; the oracle runs on the host cores"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_cores(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------- GPU arm


def build_job(wl, device, max_checks: int = 0):
    """Model handle plus one batch of inputs resident on the device (weights generated in place)."""
    import torch
    from paper_2509_24257_b200 import binding as vb, synth

    cs, cp = synth.check_positions(wl)
    model = vb.Model(wl.shape, wl.n_tokens, max_checks or len(cs), wl.batch, device)
    model.load_globals(synth.embed_weights(wl, device), synth.final_norm_weights(wl, device))
    for l in range(wl.shape.n_layers):
        model.load_layer(l, synth.layer_weights(wl, l, device))
    torch.cuda.empty_cache()
    tokens = synth.token_streams(wl)
    cu = synth.cu_seqlens(wl)
    flat = torch.from_numpy(tokens.reshape(-1)).to(device)
    # the prover's trace: teacher-forced bf16 KV-cache decode after a parallel pass over the prompts
    t0 = time.perf_counter()
    committed = model.decode_commit(flat, cu, wl.prompt_len, cs, cp, torch.bfloat16).contiguous()
    trace_s = time.perf_counter() - t0
    # tamper ceil(10 %) of the sequences, alternating a substituted token and state noise of 10 x tol
    rng = synth.tamper_rng(wl)
    n_bad = int(math.ceil(0.1 * wl.batch))
    bad_seqs = sorted(rng.choice(wl.batch, size=n_bad, replace=False).tolist())
    tampered_tokens = tokens
    comm_host = committed.float().cpu().numpy().astype(np.float64)
    for i, b in enumerate(bad_seqs):
        slots = np.nonzero(cs == b)[0]
        if slots.size == 0:
            continue
        slot = int(slots[0])
        if i % 2 == 0:
            tampered_tokens = synth.swap_token(tampered_tokens, b, int(cp[slot]), wl.shape.vocab, rng)
        else:
            comm_host = synth.add_state_noise(comm_host, [slot], [int(rng.integers(0, wl.shape.n_layers))],
                                              10 * TOL_REL_L2, rng)
    committed = synth.to_commit_dtype(comm_host, "bf16").to(device)
    flat = torch.from_numpy(tampered_tokens.reshape(-1)).to(device)
    return model, flat, tampered_tokens, cu, cs, cp, committed, bad_seqs, trace_s


def bench_compare_path(wl, device, tol, peaks, stream, iters: int = 40):
    """The comparison path alone at full coverage (every position of 2 sequences checked at every layer): the
    standalone compare + verdict kernels stream hidden (fp32) and committed (bf16) states once."""
    import torch
    from paper_2509_24257_b200 import binding as vb

    s = wl.shape
    n_rows = min(2 * wl.seq_len, wl.n_tokens)
    hid = torch.randn(s.n_layers, n_rows, s.d_model, device=device)
    com = (hid * (1 + 4e-3 * torch.randn_like(hid))).to(torch.bfloat16)
    seq_of = (np.arange(n_rows) // wl.seq_len).astype(np.int32)
    cmp_rep = vb.Report(n_rows, s.n_layers, 2, s.d_model, device, False)
    cmp_call = vb.compare_noalloc if s.n_layers * n_rows <= 65536 else vb.compare
    kw = {"report": cmp_rep} if cmp_call is vb.compare_noalloc else {}
    cmp_ms = timed_light(lambda: cmp_call(hid, com, seq_of, 2, tol, **kw), stream, iters)
    cmp_bytes = hid.numel() * 6
    # the kernel reads each byte once; the statistics cost a few tens of instructions per element, so instruction
    # issue, not HBM, is what it runs into first
    return {"rows": int(s.n_layers * n_rows), "ms": round(cmp_ms, 4), "bound": "hbm",
            "achieved_gbs": round(cmp_bytes / (cmp_ms * 1e-3) / 1e9, 1), "peak_gbs": peaks["hbm_gbs"],
            "frac": round(cmp_bytes / (cmp_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4),
            "limiter": "instruction issue"}


def timed_light(fn, stream, iters: int, warm_ms: float = 200.0):
    """Mean time of fn() on `stream` over `iters` calls.  Kernels that are bound by instruction issue or integer
    arithmetic follow the SM clock, which the power-capped transformer steps before them pull far below its
    maximum; the warm-up therefore runs the light kernel itself for `warm_ms` so that the clock has recovered."""
    import torch

    t0 = time.perf_counter()
    n = 0
    while n < 3 or (time.perf_counter() - t0) * 1e3 < warm_ms:
        fn()
        n += 1
        if n % 8 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(iters):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / iters


def per_kernel_ms(model, step, n_steps):
    """Mean time per launch of every kernel class over n_steps profiled steps (one CUDA event per launch)."""
    model.profile_enable(True)
    acc = {}
    for _ in range(n_steps):
        step()
        for k, (ms, n) in model.profile_read().items():
            a = acc.setdefault(k, [0.0, 0])
            a[0] += ms
            a[1] += n
    model.profile_enable(False)
    return acc


def bench_full_coverage(model, wl, flat, cu, tol, device, stream, peaks, down_ms_sampled, steps: int = 3):
    """The same step with EVERY position checked at every layer: the gather-and-compare epilogue of the down
    projection then reads a committed slab as large as the layer's output.  The committed states are the
    verifier's own recomputed states rounded to bf16 (an honest trace up to rounding), taken from one untimed
    pass.  Reports the step, the down projection with and without the full comparison, and the comparison's
    bytes (committed bf16 + recomputed fp32 re-read) over the time it adds."""
    import torch
    from paper_2509_24257_b200 import binding as vb

    s = wl.shape
    M = wl.n_tokens
    cs = np.repeat(np.arange(wl.batch, dtype=np.int32), wl.seq_len)
    cp = np.tile(np.arange(wl.seq_len, dtype=np.int32), wl.batch)
    empty = torch.zeros(s.n_layers, M, s.d_model, dtype=torch.bfloat16, device=device)
    rep = model.verify_prefill(flat, cu, empty, cs, cp, tol, want_hidden=True, stream=stream)
    torch.cuda.synchronize()
    committed = rep.hidden.to(torch.bfloat16)
    del rep, empty
    torch.cuda.empty_cache()
    report = vb.Report(M, s.n_layers, wl.batch, s.d_model, device, False)

    def step():
        model.verify_prefill(flat, cu, committed, cs, cp, tol, report=report, stream=stream)

    for _ in range(3):
        step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    acc = per_kernel_ms(model, step, steps)
    down = acc["gemm_down_resid_compare"]
    down_ms = down[0] / down[1]
    res = report.cpu()
    # HBM traffic the comparison adds: the committed slab (bf16).  The recomputed values are re-read by the thread
    # that has just written them (cache hits), and the whole epilogue of a tile runs under the next tile's MMAs, so
    # the time it adds to the projection is small and the rate below is a lower bound on what the path sustains.
    cmp_bytes = float(M) * s.d_model * 2
    added = max(down_ms - down_ms_sampled, 1e-6)
    gbs = cmp_bytes / (added * 1e-3) / 1e9
    return {"checked_positions": int(M), "committed_gb": round(committed.numel() * 2 / 1e9, 2),
            "ms_per_step": round(ms, 3), "gemm_down_ms": round(down_ms, 4), "gemm_down_ms_sampled": round(down_ms_sampled, 4),
            "added_ms_per_layer": round(down_ms - down_ms_sampled, 4),
            "added_frac_of_down_projection": round((down_ms - down_ms_sampled) / down_ms_sampled, 4),
            "committed_bytes_per_layer": int(cmp_bytes),
            "bound": "hbm", "achieved_gbs": round(gbs, 1), "peak_gbs": peaks["hbm_gbs"],
            "frac": round(gbs / peaks["hbm_gbs"], 4),
            "note": "committed bytes over the time the comparison adds to the down projection (it overlaps the next tile's main loop)",
            "positions_accepted": int((res["pos_ok"] == 1).sum()), "status": res["status"]}


def bench_merkle(n_vec, d_model, device, stream, clocks, iters: int = 10):
    """Merkle commitment of n_vec state vectors (one SHA-256 tree per (layer, position) vector): integer ALU work."""
    import torch
    from paper_2509_24257_b200 import binding as vb

    mk_in = torch.randn(n_vec, d_model, device=device)
    mk_out = torch.empty(mk_in.shape[0], 32, dtype=torch.uint8, device=device)
    mk_ms = timed_light(lambda: vb.merkle_roots(mk_in, stream, out=mk_out), stream, iters)
    n_compress = mk_in.shape[0] * (4 * ((d_model + 1) // 2) + 2 * ((d_model + 1) // 2 - 1))
    # ALU peak: one SHA-256 compression is 1384 32-bit integer instructions as written (64 rounds x 14, 48 schedule
    # words x 10, 8 final adds); an SM issues 4 warp instructions = 128 lane operations per clock
    props = torch.cuda.get_device_properties(device)
    sm_clock_hz = 1e6 * float(clocks.get("sm_max_mhz") or 1965.0)
    lane_ops_peak = props.multi_processor_count * 128 * sm_clock_hz
    mk_peak = lane_ops_peak / SHA256_INT_OPS
    mk_rate = n_compress / (mk_ms * 1e-3)
    # funnel shifts (every rotation: 6 of a round's 14 instructions, 4 of a schedule word's 10) issue at half
    # rate on this part (64 lanes per clock per SM, measured), so a full-rate count overstates what the ALUs can do
    merkle = {"vectors": int(mk_in.shape[0]), "scalars_per_vector": d_model, "ms": round(mk_ms, 4), "bound": "alu",
              "ns_per_scalar": round(mk_ms * 1e6 / mk_in.numel(), 4),
              "sha256_compressions_per_s": round(mk_rate, 0), "peak_compressions_per_s": round(mk_peak, 0),
              "frac": round(mk_rate / mk_peak, 4),
              "peak_kind": "derived: SMs x 128 integer lane-ops per clock x max SM clock / 1384 ops per full compression",
              "ops_executed_per_compression": SHA256_INT_OPS_EXECUTED,
              "frac_of_lane_op_peak_executed": round(mk_rate * SHA256_INT_OPS_EXECUTED / lane_ops_peak, 4),
              "frac_with_half_rate_rotations": round(
                  mk_rate * (SHA256_INT_OPS_EXECUTED + SHA256_FUNNEL_SHIFTS_EXECUTED) / lane_ops_peak, 4)}
    return merkle


def run_compare_only(args, wl):
    """Runs only the comparison path (no model): a small process for profiler captures of its kernels."""
    import torch
    from paper_2509_24257_b200 import binding as vb

    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    peaks, _ = measured_peaks()
    tol = vb.default_tol(rel_l2=TOL_REL_L2)
    print(json.dumps({"compare_path": bench_compare_path(wl, device, tol, peaks, torch.cuda.current_stream(),
                                                         iters=max(args.steps, 1))}))


def run_merkle_only(args, wl):
    """Runs only the Merkle commitment kernel (no model): a small process for profiler captures."""
    import torch

    device = torch.device("cuda", 0)
    torch.cuda.set_device(device)
    n_vec = wl.shape.n_layers * max(1, int(round(wl.check_frac * wl.n_tokens)))
    print(json.dumps({"merkle": bench_merkle(n_vec, wl.shape.d_model, device, torch.cuda.current_stream(), {},
                                            iters=max(args.steps, 1))}))


def run_ours(args, wl):
    import torch
    from paper_2509_24257_b200 import binding as vb, dist as vdist

    rank, world, local = vdist.init()
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}")
    device = torch.device("cuda", local)
    torch.cuda.set_device(device)
    wl_r = vdist.replica_workload(wl, rank)
    # the full-coverage supplementary (every position checked) needs the slot tables sized for it
    full_cov = args.gpus == 1 and not args.no_full_coverage and wl.n_tokens * wl.shape.n_layers * wl.shape.d_model <= 2 ** 31
    model, flat, tokens_host, cu, cs, cp, committed, bad_seqs, trace_s = build_job(wl_r, device, wl.n_tokens if full_cov else 0)
    tol = vb.default_tol(rel_l2=TOL_REL_L2)
    report = vb.Report(len(cs), wl.shape.n_layers, wl.batch, wl.shape.d_model, device, False)
    stream = torch.cuda.current_stream()

    def step():
        model.verify_prefill(flat, cu, committed, cs, cp, tol, report=report, stream=stream)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    # ---- device-resident timing: exactly K steps between two events
    sampler = ClockSampler(int(os.environ.get("CUDA_VISIBLE_DEVICES", "0").split(",")[local]) if
                           os.environ.get("CUDA_VISIBLE_DEVICES") else local)
    sampler.start()
    time.sleep(0.3)
    vdist.barrier()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    torch.cuda.profiler.start()  # a profiler started with --profile-from-start off sees only the timed steps
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize()
    torch.cuda.profiler.stop()
    t_wall1 = time.time()
    vdist.barrier()
    seconds = e0.elapsed_time(e1) / 1e3
    clocks = sampler.stop(t_wall0, t_wall1)
    res = report.cpu()
    launches = model.last_launch_count() * args.steps
    value = vdist.aggregate_throughput(float(wl.n_tokens * args.steps), seconds)
    slowest = vdist.max_over_ranks(seconds)

    # ---- end to end: host buffers in, report out, every step.  Inputs of step i + 1 are uploaded from pinned memory
    # on a copy stream while step i computes (two device buffers); every upload, every call and every read-back of
    # the report lies inside the timed region, and the host waits for each step's report before it goes on.
    pin = lambda t: t.cpu().pin_memory()
    tok_pin, comm_pin = pin(flat), pin(committed)
    out_pin = {k: torch.empty_like(getattr(report, k), device="cpu").pin_memory()
               for k in ("stats", "pos_ok", "first_bad_layer", "seq_ok", "seq_score", "status")}
    in_dev = [(torch.empty_like(flat), torch.empty_like(committed)) for _ in range(2)]
    copy_stream = torch.cuda.Stream(device=device)
    uploaded = [torch.cuda.Event() for _ in range(2)]
    consumed = [torch.cuda.Event() for _ in range(2)]

    def upload(i):
        tok_dev, comm_dev = in_dev[i % 2]
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(consumed[i % 2])  # the step that last read this buffer has finished with it
            tok_dev.copy_(tok_pin, non_blocking=True)
            comm_dev.copy_(comm_pin, non_blocking=True)
            uploaded[i % 2].record(copy_stream)

    def e2e_run(n):
        upload(0)
        for i in range(n):
            if i + 1 < n:
                upload(i + 1)
            tok_dev, comm_dev = in_dev[i % 2]
            stream.wait_event(uploaded[i % 2])
            model.verify_prefill(tok_dev, cu, comm_dev, cs, cp, tol, report=report, stream=stream)
            consumed[i % 2].record(stream)
            for k, buf in out_pin.items():
                buf.copy_(getattr(report, k), non_blocking=True)
            stream.synchronize()

    for ev in consumed:
        ev.record(stream)
    e2e_run(2)
    torch.cuda.synchronize()
    vdist.barrier()
    t0 = time.perf_counter()
    e2e_run(args.steps)
    torch.cuda.synchronize()
    e2e_seconds = time.perf_counter() - t0
    vdist.barrier()
    e2e_value = vdist.aggregate_throughput(float(wl.n_tokens * args.steps), e2e_seconds)
    h2d = tok_pin.numel() * 4 + comm_pin.numel() * comm_pin.element_size() + 4 * (len(cu) + 2 * len(cs))
    d2h = sum(b.numel() * b.element_size() for b in out_pin.values())

    # ---- per-kernel times (second pass with one event per launch) for the roofline of the dominant kernel
    peaks, peaks_kind = measured_peaks()
    acc = per_kernel_ms(model, step, min(args.steps, 5))
    s = wl.shape
    M = wl.n_tokens
    flops_per_launch = {
        "gemm_qkv_rope": 2.0 * M * (s.d_q + 2 * s.d_kv) * s.d_model,
        "gemm_o_resid": 2.0 * M * s.d_model * s.d_q,
        "gemm_gate_up_swiglu": 2.0 * M * 2 * s.d_ffn * s.d_model,
        "gemm_down_resid_compare": 2.0 * M * s.d_model * s.d_ffn,
        "attention": 4.0 * s.n_heads * s.head_dim * M * (wl.seq_len + 1) / 2.0,
    }
    kernels = {}
    for k, (ms, n) in acc.items():
        if n == 0:
            continue
        per = ms / n
        kernels[k] = {"launches_per_step": n // min(args.steps, 5), "ms_per_launch": round(per, 4)}
        if k in flops_per_launch:
            kernels[k]["tflops"] = round(flops_per_launch[k] / (per * 1e-3) / 1e12, 1)
    dom = "gemm_gate_up_swiglu"
    achieved = flops_per_launch[dom] / (acc[dom][0] / acc[dom][1] * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"]
    # DRAM bytes of one launch of that kernel: dram__bytes_read.sum + dram__bytes_write.sum of a stored profiler
    # capture of the same launch (same M, N, K, grid and tile walk), not measured by this run; only valid for the
    # shape it was taken on
    traffic = GATE_UP_DRAM_BYTES_8B if (s.d_model, s.d_ffn, M) == (4096, 14336, 8192) else None
    roofline = {"bound": "tensor", "kernel": dom, "achieved": round(achieved, 1), "peak": peak, "unit": "TFLOP/s",
                "frac": round(achieved / peak, 4), "traffic": traffic,
                "traffic_source": "stored ncu capture of one launch at this shape" if traffic else None,
                "peak_kind": f"bf16 sustained (the kernel is timed inside a long power-capped step), of {peaks_kind}",
                "frac_of_burst_peak": round(achieved / peaks["bf16_tflops"], 4),
                "frac_of_nominal_2250": round(achieved / 2250.0, 4), "kernels": kernels}

    # ---- tail token check (next row of the scope table): final norm + output head + arg-max on the checked rows;
    # it streams the [vocab][d_model] head once, so it is reported against the measured copy bandwidth
    from paper_2509_24257_b200 import synth as _synth
    model.load_lm_head(_synth.lm_head_weights(wl, device))
    last_hidden = torch.randn(len(cs), s.d_model, device=device)
    claimed = np.zeros(len(cs), dtype=np.int32)
    tm_ms = timed_light(lambda: model.token_match(last_hidden, claimed, stream), stream, 20)
    tm_bytes = s.vocab * s.d_model * 2 + len(cs) * s.d_model * 6
    token_match = {"rows": int(len(cs)), "ms": round(tm_ms, 4), "bound": "hbm",
                   "achieved_gbs": round(tm_bytes / (tm_ms * 1e-3) / 1e9, 1), "peak_gbs": peaks["hbm_gbs"],
                   "frac": round(tm_bytes / (tm_ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)}

    compare_path = bench_compare_path(wl, device, tol, peaks, stream)
    full_coverage = None
    if full_cov:
        down_sampled = acc["gemm_down_resid_compare"][0] / acc["gemm_down_resid_compare"][1]
        full_coverage = bench_full_coverage(model, wl, flat, cu, tol, device, stream, peaks, down_sampled)

    merkle = bench_merkle(s.n_layers * len(cs), s.d_model, device, stream, clocks)

    if rank == 0:
        run, desc = oracle_sample(wl, 12.0, str(device)) if args.gpus == 1 else (None, None)
        cpu_baseline = None
        if run is not None:
            T, sec, nl = run()
            cpu_baseline = {"value": T * nl / wl.shape.n_layers / sec, "unit": UNIT, "cores": cpu_cores(),
                            "kind": "oracle", "sample": desc}
        total_tflops = wl.total_flops() * args.gpus * args.steps / slowest / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * slowest / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {
                "workload": wl.name, "batch": wl.batch, "seq_len": wl.seq_len, "n_check": int(len(cs)),
                "tampered_sequences": bad_seqs, "parallelism": f"replicas x{args.gpus}",
                "l2": "inputs larger than L2 (15 GB of weights streamed per step)",
                "trace": f"committed states from verillm_decode_commit ({trace_s:.1f} s, untimed)",
            },
            "model_tflops": round(total_tflops, 1),
            "pct_of_bf16_peak": {"of_measured_burst": round(total_tflops / args.gpus / peaks["bf16_tflops"], 4),
                                 "of_measured_sustained": round(total_tflops / args.gpus / peaks["bf16_tflops_sustained"], 4),
                                 "of_nominal_2250": round(total_tflops / args.gpus / 2250.0, 4), "peaks": peaks_kind},
            "verdicts": {"seq_ok": res["seq_ok"].tolist(), "positions_rejected": int((res["pos_ok"] == 0).sum()),
                         "status": res["status"]},
            "clocks": clocks, "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                                     "d2h_bytes_per_step": int(d2h),
                                     "pipelining": "inputs of step i+1 are uploaded on a copy stream while step i runs; "
                                                   "the host waits for every step's report"},
            "gpu_launches": int(launches), "roofline": roofline, "token_match": token_match, "compare_path": compare_path,
            "full_coverage": full_coverage, "merkle": merkle,
            "cpu_baseline": cpu_baseline,
        }
        print(json.dumps(line))
    model.close()
    vdist.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama8b")
    ap.add_argument("--compare-only", action="store_true",
                    help="time only the standalone comparison path at the workload's widths (no model is built)")
    ap.add_argument("--merkle-only", action="store_true",
                    help="time only the Merkle commitment of the workload's checked states (no model is built)")
    ap.add_argument("--no-full-coverage", action="store_true",
                    help="skip the supplementary run that checks every position (it holds 6 GB more on the device)")
    ap.add_argument("--layers", type=int, default=0,
                    help="reduced depth at full width (same launches per layer; for small profiler captures)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    from paper_2509_24257_b200 import synth

    wl = synth.WORKLOADS[args.workload]
    if args.layers > 0:
        wl = wl.with_layers(args.layers)
    if args.impl == "reference":
        run_reference(args, wl)
    elif args.compare_only:
        run_compare_only(args, wl)
    elif args.merkle_only:
        run_merkle_only(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
