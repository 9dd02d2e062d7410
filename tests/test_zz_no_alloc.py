"""The allocation-free comparison entry point against the regular one (needs a B200).

verillm_compare_noalloc exists for callers that cannot allocate device memory while they run (a serving
loop that must not hit cudaMalloc's device-wide synchronisation, or a process whose memory all belongs to
a pool).  It keeps its scratch in a fixed array inside the library, shared by all calls, so this test
makes two calls in a row, the second one smaller than the first, to show that what the first call left
in the array does not leak into the second.  This file is collected last on purpose.
"""
import numpy as np
import pytest
import torch

from paper_2509_24257_b200 import binding as vb

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(L, n, d, seed, dtype):
    g = torch.Generator().manual_seed(seed)
    committed = torch.randn(L, n, d, generator=g).to(dtype)
    hidden = committed.float() * (1 + 4e-3 * torch.randn(L, n, d, generator=g))
    hidden[L - 1, n // 2] += 0.7  # one grossly wrong cell
    hidden[0, 1, 5] = float("nan")
    check_seq = (np.arange(n) % 3).astype(np.int32)
    return hidden.to(DEV), committed.to(DEV).contiguous(), check_seq


def _same(a, b):
    for k in ("pos_ok", "first_bad_layer", "seq_ok"):
        assert np.array_equal(a[k], b[k]), k
    # both entry points run the same kernels in the same order: the floats agree to the last bit,
    # which is inside the 5e-6 relative tolerance the comparison tests use
    assert np.allclose(a["stats"], b["stats"], rtol=5e-6, atol=1e-9, equal_nan=True)
    assert np.array_equal(a["stats"], b["stats"], equal_nan=True)
    assert np.allclose(a["seq_score"], b["seq_score"], rtol=1e-5)
    assert a["status"] == b["status"] == 0


def test_two_calls_in_a_row_match_the_allocating_entry_point():
    tol = vb.default_tol(tau_large=0.02)
    first = _case(6, 301, 1024, 1, torch.bfloat16)
    second = _case(3, 40, 512, 2, torch.float32)  # fewer rows: reads a part of the array the first call filled
    want1 = vb.compare(*first[:2], first[2], 3, tol).cpu()
    want2 = vb.compare(*second[:2], second[2], 3, tol).cpu()
    got1 = vb.compare_noalloc(*first[:2], first[2], 3, tol)
    got2 = vb.compare_noalloc(*second[:2], second[2], 3, tol)  # enqueued behind the first on the same stream
    torch.cuda.synchronize()
    _same(got1.cpu(), want1)
    _same(got2.cpu(), want2)
    assert want1["pos_ok"][301 // 2] == 0 and want1["pos_ok"][1] == 0 and want1["pos_ok"].sum() == 299


def test_sizes_beyond_the_fixed_scratch_are_refused():
    h = torch.zeros(2, 8, 64, device=DEV)
    c = torch.zeros(2, 8, 64, device=DEV)
    rep = vb.Report(8, 2, 1, 64, DEV, False)
    st, tol = rep.c_struct(), vb.default_tol()
    seq = np.zeros(8, dtype=np.int32)
    import ctypes as C
    # 70000 layers x 8 slots would need more rows than the array holds: rejected before any launch
    code = vb.lib().verillm_compare_noalloc(h.data_ptr(), c.data_ptr(), vb.F32, 70000, 8, 64, seq.ctypes.data, 1,
                                            C.byref(tol), C.byref(st), None)
    assert code == vb.E_SHAPE
