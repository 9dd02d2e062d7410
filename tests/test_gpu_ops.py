"""Single steps of the CUDA path against the oracle's pieces, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

from oracle import verillm_oracle as vo
from paper_2509_24257_b200 import binding as vb
from paper_2509_24257_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _rand_bf16(shape, seed, scale=0.5):
    g = torch.Generator().manual_seed(seed)
    return (torch.randn(*shape, generator=g) * scale).to(torch.bfloat16)


@pytest.mark.parametrize("M,N,K", [(64, 768, 256), (300, 96, 72), (129, 32, 8), (1000, 512, 4096), (2049, 2816, 1024)])
def test_gemm_matches_textbook_product(M, N, K):
    # several 128x256 tiles, ragged last row tile, N and K tails
    a, b = _rand_bf16((M, K), 1), _rand_bf16((N, K), 2)
    ref = vo.as_f64(H.bits(a)) @ vo.as_f64(H.bits(b)).T
    c32 = vb.op_gemm(a.to(DEV), b.to(DEV), out_f32=True).cpu().numpy().astype(np.float64)
    c16 = vb.op_gemm(a.to(DEV), b.to(DEV), out_f32=False).float().cpu().numpy().astype(np.float64)
    # fp32 accumulation of K products: error ~ sqrt(K) * 2^-24 relative to the row scale
    assert np.linalg.norm(c32 - ref) <= 2e-5 * np.linalg.norm(ref)
    assert np.max(H.rel_l2(c32, ref)) <= 5e-5
    assert np.max(H.rel_l2(c16, ref)) <= 4e-3  # one bf16 rounding of the result
    assert np.array_equal(c16, vo.round_to_bf16(c32))  # bf16 output = RNE of the fp32 accumulator


def test_gemm_rejects_unsupported_shapes():
    a, b = _rand_bf16((16, 12), 1).to(DEV), _rand_bf16((32, 12), 2).to(DEV)
    with pytest.raises(vb.VerillmError) as e:
        vb.op_gemm(a, b)
    assert e.value.code == vb.E_SHAPE


@pytest.mark.parametrize("M,d", [(77, 1024), (5, 4096), (3, 64)])
def test_rmsnorm_matches_oracle(M, d):
    g = torch.Generator().manual_seed(3)
    x = torch.randn(M, d, generator=g) * 3.0
    gain = (1 + 0.1 * torch.randn(d, generator=g)).to(torch.bfloat16)
    y = vb.op_rmsnorm(x.to(DEV), gain.to(DEV), 1e-5).float().cpu().numpy().astype(np.float64)
    ref = vo.rmsnorm(x.numpy().astype(np.float64), vo.as_f64(H.bits(gain)), 1e-5)
    assert np.max(np.abs(y - ref) / np.maximum(np.abs(ref), 1e-30)) <= 2.0 ** -7  # at most one bf16 step apart
    assert np.max(H.rel_l2(y, ref)) <= 3e-3


@pytest.mark.parametrize("Hq,KV,dh,lens", [
    (4, 4, 64, [64]), (4, 2, 64, [100, 37, 300, 1]), (8, 2, 128, [129, 64, 515]), (2, 1, 128, [1, 2, 127, 128, 130]),
])
def test_attention_matches_oracle(Hq, KV, dh, lens):
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    qkv = _rand_bf16((int(cu[-1]), (Hq + 2 * KV) * dh), 4, 1.0)
    out = vb.op_attention(qkv.to(DEV), cu, Hq, KV, dh).float().cpu().numpy().astype(np.float64)
    x = vo.as_f64(H.bits(qkv))
    for b in range(len(lens)):
        s, e = int(cu[b]), int(cu[b + 1])
        q = x[s:e, : Hq * dh].reshape(-1, Hq, dh)
        k = x[s:e, Hq * dh : (Hq + KV) * dh].reshape(-1, KV, dh)
        v = x[s:e, (Hq + KV) * dh :].reshape(-1, KV, dh)
        ref = vo.causal_attention(q, k, v).reshape(e - s, Hq, dh)
        got = out[s:e].reshape(e - s, Hq, dh)
        assert np.max(H.rel_l2(got, ref)) <= 1e-2  # bf16 probabilities and output
        assert np.array_equal(got[0], v[0, [g * KV // Hq for g in range(Hq)]])  # first row = v_0 exactly


def test_attention_many_units_per_cta():
    """More (sequence, head, query tile) units than the persistent CTAs keep in their shared-memory table, so the
    later units are looked up on the spot, over several dealing rounds: sampled sequences against the oracle,
    and the closed form row 0 = v_0 on every sequence and head."""
    Hq, KV, dh = 32, 8, 64
    rng = np.random.default_rng(77)
    lens = rng.integers(1, 161, size=480)
    lens[:4] = [160, 129, 128, 1]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    assert 2 * Hq * len(lens) > 48 * 2 * torch.cuda.get_device_properties(0).multi_processor_count
    qkv = _rand_bf16((int(cu[-1]), (Hq + 2 * KV) * dh), 12, 1.0)
    out = vb.op_attention(qkv.to(DEV), cu, Hq, KV, dh).float().cpu().numpy().astype(np.float64)
    x = vo.as_f64(H.bits(qkv))
    assert np.all(np.isfinite(out))
    v_first = x[cu[:-1], (Hq + KV) * dh :].reshape(len(lens), KV, dh)
    assert np.array_equal(out[cu[:-1]].reshape(len(lens), Hq, dh), v_first[:, [g * KV // Hq for g in range(Hq)]])
    for b in list(range(4)) + rng.choice(len(lens), 12, replace=False).tolist():
        s, e = int(cu[b]), int(cu[b + 1])
        q = x[s:e, : Hq * dh].reshape(-1, Hq, dh)
        k = x[s:e, Hq * dh : (Hq + KV) * dh].reshape(-1, KV, dh)
        v = x[s:e, (Hq + KV) * dh :].reshape(-1, KV, dh)
        ref = vo.causal_attention(q, k, v).reshape(e - s, Hq, dh)
        assert np.max(H.rel_l2(out[s:e].reshape(e - s, Hq, dh), ref)) <= 1e-2


def _engineered_pairs(d, seed):
    """Hidden/committed rows that exercise every branch of the comparison."""
    rng = np.random.default_rng(seed)
    c = rng.standard_normal(d).astype(np.float32) * 2.0
    h = (c.astype(np.float64) * (1 + 3e-3 * rng.standard_normal(d))).astype(np.float32)
    h[0:4] = [1.0 - 2.0 ** -9, 0.5, -1.25, 4e-6]
    c[0:4] = [1.0, 1.0, 1.25, 0.0]
    h[4:8] = [0.0, -0.0, 3.0, 1e-41]
    c[4:8] = [-0.0, 0.0, 3.0, 0.0]
    return h, c


@pytest.mark.parametrize("commit", ["bf16", "f32"])
def test_compare_same_inputs_counts_are_bit_exact(commit):
    L, n, d = 3, 37, 1024
    hs, cs = [], []
    for i in range(L * n):
        h, c = _engineered_pairs(d, 100 + i)
        hs.append(h)
        cs.append(c)
    hidden = np.stack(hs).reshape(L, n, d)
    comm = np.stack(cs).reshape(L, n, d)
    hidden[1, 5, 17] = np.nan
    comm[2, 9, 3] = np.inf
    comm[0, 3] = hidden[0, 3]  # an identical row
    hidden[2, 11] += 0.5  # a grossly wrong row
    comm_t = synth.to_commit_dtype(comm.astype(np.float64), commit)
    comm64 = comm_t.to(torch.float64).numpy()
    check_seq = (np.arange(n) % 4).astype(np.int32)
    tol_o = vo.Tol(rel_l2=8e-2, tau_large=0.01, bit_aware=False)
    tol_g = vb.default_tol(rel_l2=8e-2, tau_large=0.01)
    rep = vb.compare(torch.from_numpy(hidden).to(DEV), comm_t.to(DEV), check_seq, 4, tol_g).cpu()
    stats_o = np.transpose(vo.compare_stats(hidden.astype(np.float64), comm64, commit, tol_o), (1, 0, 2))
    pos_ok, first_bad, seq_ok, score = vo.verdict(stats_o, check_seq, 4, tol_o)
    for j, nm in enumerate(vo.STAT_NAMES):
        g, o = rep["stats"][..., j].astype(np.float64), stats_o[..., j]
        if nm.startswith("n_"):
            assert np.array_equal(g, o), nm  # integer counts: bit-exact
        elif nm in ("p_e", "q_small", "z_large", "p_m", "p_w"):
            assert np.allclose(g, o, rtol=1e-6, atol=0), nm  # ratios of identical integers
        else:
            assert np.allclose(g, o, rtol=5e-6, atol=1e-9), nm  # fp32 sums of 1024 terms vs fp64
    assert np.array_equal(rep["pos_ok"], pos_ok)
    assert np.array_equal(rep["first_bad_layer"], first_bad)
    assert np.array_equal(rep["seq_ok"], seq_ok)
    assert np.allclose(rep["seq_score"], score, rtol=1e-5)
    assert rep["pos_ok"][3] == 1 and rep["pos_ok"][5] == 0 and rep["pos_ok"][9] == 0 and rep["pos_ok"][11] == 0


def test_bit_aware_verdict_matches_oracle_on_same_inputs():
    L, n, d = 2, 16, 512
    rng = np.random.default_rng(7)
    comm = rng.standard_normal((L, n, d)).astype(np.float32)
    hidden = comm.copy()
    # rows 0..7: honest-like (tiny relative noise); rows 8..15: heavy noise that scrambles exponents
    hidden[:, :8] *= (1 + 1e-4 * rng.standard_normal((L, 8, d))).astype(np.float32)
    hidden[:, 8:] *= (1 + 0.4 * rng.standard_normal((L, 8, d))).astype(np.float32)
    comm_t = synth.to_commit_dtype(comm.astype(np.float64), "f32")
    kw = dict(rel_l2=0.0, bit_aware=True, pw_min=0.5, pm_min=-1.0, e_w=1e-3)
    rep = vb.compare(torch.from_numpy(hidden).to(DEV), comm_t.to(DEV), np.zeros(n, np.int32), 1, vb.default_tol(**kw)).cpu()
    tol_o = vo.Tol(**kw)
    stats_o = np.transpose(vo.compare_stats(hidden.astype(np.float64), comm.astype(np.float64), "f32", tol_o), (1, 0, 2))
    pos_ok, first_bad, _, _ = vo.verdict(stats_o, np.zeros(n, np.int32), 1, tol_o)
    assert np.array_equal(rep["pos_ok"], pos_ok) and np.array_equal(rep["first_bad_layer"], first_bad)
    assert pos_ok[:8].all() and not pos_ok[8:].any()


def test_seeded_generator_is_identical_on_device():
    wl = synth.WORKLOADS["small"]
    cpu = synth.layer_weights(wl, 1, "cpu")
    gpu = synth.layer_weights(wl, 1, DEV)
    assert all(torch.equal(cpu[k], gpu[k].cpu()) for k in cpu)
    rows = torch.tensor([0, 31999, 17])
    assert torch.equal(synth.embed_weights(wl, DEV, rows=rows).cpu(), synth.embed_weights(wl, "cpu")[rows])


def test_tensor_core_kernels_are_bit_reproducible_over_many_launches():
    """A missed wait inside a pipelined kernel shows up as a rare run-to-run difference, long before it
    shows up as an error against the oracle: repeat the launches and compare bit for bit."""
    qkv = _rand_bf16((4 * 640, (8 + 2 * 2) * 128), 9, 0.3).to(DEV)
    cu = np.arange(5, dtype=np.int32) * 640
    ref = vb.op_attention(qkv, cu, 8, 2, 128)
    for _ in range(1500):
        assert torch.equal(vb.op_attention(qkv, cu, 8, 2, 128), ref)
    a, b = _rand_bf16((2048, 1024), 10).to(DEV), _rand_bf16((1536, 1024), 11).to(DEV)
    ref = vb.op_gemm(a, b)
    for _ in range(300):
        assert torch.equal(vb.op_gemm(a, b), ref)


def test_spot_check_matches_oracle_bit_for_bit():
    rng = np.random.default_rng(31)
    hidden = rng.standard_normal((82, 4096)).astype(np.float32)
    n = 3584  # the largest sample count in the paper's tables
    rows, cols = rng.integers(0, 82, n), rng.integers(0, 4096, n)
    ref = hidden[rows, cols] + (rng.standard_normal(n) * 0.01).astype(np.float32)
    ref[::97] = np.nan
    for eps, theta in ((0.01, 0.6), (0.02, 0.99), (0.0, 0.0)):
        agree_o, p_o, ok_o = vo.spot_check(hidden, rows, cols, ref, eps, theta)
        agree, p_hat, ok = vb.spot_check(torch.from_numpy(hidden).to(DEV), rows, cols, ref, eps, theta)
        assert np.array_equal(agree.cpu().numpy(), agree_o)
        assert float(p_hat.item()) == np.float32(p_o) and bool(ok.item()) == ok_o
    with pytest.raises(vb.VerillmError) as e:
        vb.spot_check(torch.from_numpy(hidden).to(DEV), [82], [0], [0.0], 0.1, 0.5)
    assert e.value.code == vb.E_RANGE


@pytest.mark.parametrize("n_vec,d", [(5, 1), (7, 2), (3, 3), (4, 257), (6, 1024), (3, 4096), (2, 8192), (2, 5000)])
def test_merkle_roots_are_bit_exact(n_vec, d):
    rng = np.random.default_rng(100 + d)
    x = rng.standard_normal((n_vec, d)).astype(np.float32)
    x[0, 0] = -0.0
    if d > 2:
        x[-1, 1], x[-1, 2] = np.inf, np.nan  # every bit pattern is just four bytes to the hash
    roots = vb.merkle_roots(torch.from_numpy(x).to(DEV)).cpu().numpy()
    for i in range(n_vec):
        assert roots[i].tobytes() == vo.merkle_root(x[i]), (i, d)
    with pytest.raises(vb.VerillmError) as e:
        vb.merkle_roots(torch.zeros(1, 12801, device=DEV))
    assert e.value.code == vb.E_SHAPE


def _exact_rows(L, n, d, seed):
    """Committed rows and deviations whose statistics are exact in float32: every value is a small multiple of
    2^-10, most deviations are zero, a few are +-2^-18 (below the 1e-5 of Q_small) or multiples of 1/8."""
    rng = np.random.default_rng(seed)
    c = rng.integers(-2048, 2048, (L, n, d)) / 1024.0
    delta = np.zeros((L, n, d))
    for l in range(L):
        for i in range(n):
            k = rng.integers(0, d // 2 + 1)
            idx = rng.choice(d, k, replace=False)
            delta[l, i, idx] = rng.choice([2.0 ** -18, -2.0 ** -18, 0.125, -0.125, 0.25, 0.5, -0.75], k)
    return (c + delta).astype(np.float32), c.astype(np.float32)


def test_every_float_test_of_the_verdict_matches_oracle_bit_for_bit():
    """max |Delta|, MAE, Z_large and Q_small enabled in the standalone comparison and in the threshold sweep, on
    rows whose statistics are exact in float32, with each threshold set to a value some row attains exactly:
    verdicts, first failing layers and sweep counts equal the oracle's."""
    L, n, d = 3, 40, 64
    hidden, comm = _exact_rows(L, n, d, 77)
    check_seq = (np.arange(n) % 3).astype(np.int32)
    base = dict(rel_l2=0.0, tau_large=0.125)
    stats_o = np.transpose(vo.compare_stats(hidden.astype(np.float64), comm.astype(np.float64), "f32", vo.Tol(**base)), (1, 0, 2))
    med = lambda name: float(np.median(stats_o[..., vo.STAT_NAMES.index(name)]))
    variants = [
        dict(max_abs=0.5), dict(mae=med("mae")), dict(z_large_max=med("z_large")), dict(q_small_min=med("q_small")),
        dict(z_large_max=0.0), dict(q_small_min=1.0),
        dict(max_abs=0.5, mae=med("mae"), z_large_max=med("z_large"), q_small_min=med("q_small")),
    ]
    hid_t, com_t = torch.from_numpy(hidden).to(DEV), torch.from_numpy(comm).to(DEV)
    seen = set()
    for kw in variants:
        tol_o, tol_g = vo.Tol(**base, **kw), vb.default_tol(**base, **kw)
        rep = vb.compare(hid_t, com_t, check_seq, 3, tol_g).cpu()
        for j, nm in enumerate(vo.STAT_NAMES):
            if nm not in ("rel_l2", "l2_delta", "l2_ref"):  # everything but the square roots is exact here:
                # sums and counts exactly, ratios of counts (P_w, P_m) as the correctly rounded float32 quotient
                assert np.array_equal(rep["stats"][..., j].astype(np.float32), stats_o[..., j].astype(np.float32)), nm
        pos_ok, first_bad, seq_ok, _ = vo.verdict(stats_o, check_seq, 3, tol_o)
        assert np.array_equal(rep["pos_ok"], pos_ok) and np.array_equal(rep["first_bad_layer"], first_bad), kw
        assert np.array_equal(rep["seq_ok"], seq_ok), kw
        seen.add((int(pos_ok.sum()) > 0, int(pos_ok.sum()) < n))
    assert (True, True) in seen  # thresholds that split the rows, not all-or-nothing
    # the same tests applied afterwards to the reported statistics
    rep = vb.compare(hid_t, com_t, check_seq, 3, vb.default_tol(**base))
    cells = rep.stats[:n].reshape(-1, vb.NSTAT).contiguous()
    attack = torch.from_numpy((np.arange(n * L) % 2).astype(np.uint8)).to(DEV)
    counts = vb.threshold_sweep(cells, attack, [vb.default_tol(**base, **kw) for kw in variants]).cpu().numpy()
    counts_o = vo.threshold_sweep(cells.cpu().numpy(), attack.cpu().numpy(), [vo.Tol(**base, **kw) for kw in variants])
    assert np.array_equal(counts, counts_o)
    assert (counts[:4, 0] > 0).all() and (counts[:4, 1] > 0).all()


def test_relaxed_value_test_on_a_full_row_equals_the_spot_check():
    """Position-granular form of the relaxed on-chain test: tau_large = eps, z_large_max = 1 - theta on a whole
    row decides like the sampled-scalar spot check over all d entries of that row, on the GPU and in the oracle."""
    rng = np.random.default_rng(13)
    n, d, eps = 24, 256, 0.125
    comm = (rng.integers(-4096, 4096, (1, n, d)) / 1024.0).astype(np.float32)
    hidden = comm.copy()
    for i in range(n):
        far = rng.choice(d, int(rng.integers(0, d // 2)), replace=False)
        hidden[0, i, far] += rng.choice([-0.5, 0.25, 1.0], len(far)).astype(np.float32)
        hidden[0, i, (far + 1) % d] += np.float32(0.125)  # exactly eps: agrees
    hidden[0, 0] = comm[0, 0]
    hidden[0, 1, : d // 4] = comm[0, 1, : d // 4] + 1.0  # p_hat = 0.75 exactly (the rest of row 1 is reset below)
    hidden[0, 1, d // 4:] = comm[0, 1, d // 4:]
    hid_t, com_t = torch.from_numpy(hidden).to(DEV), torch.from_numpy(comm).to(DEV)
    cols = np.arange(d)
    for theta in (0.5, 0.75, 1.0):
        kw = dict(rel_l2=0.0, tau_large=eps, z_large_max=1.0 - theta)
        rep = vb.compare(hid_t, com_t, np.zeros(n, np.int32), 1, vb.default_tol(**kw)).cpu()
        stats_o = vo.compare_stats(hidden[0].astype(np.float64), comm[0].astype(np.float64), "f32", vo.Tol(**kw))
        for i in range(n):
            _, p_hat, ok = vb.spot_check(hid_t[0], np.full(d, i), cols, comm[0, i], eps, theta)
            _, p_hat_o, ok_o = vo.spot_check(hidden[0], np.full(d, i), cols, comm[0, i], eps, theta)
            assert float(p_hat.item()) == p_hat_o and bool(ok.item()) == ok_o
            assert bool(rep["pos_ok"][i]) == ok_o == bool(vo.layer_passes(stats_o[i], vo.Tol(**kw))), (theta, i)
    assert rep["pos_ok"][0] == 1
