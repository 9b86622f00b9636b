"""tb_factor_static: the factor for callers that cannot allocate device memory
(all free memory already given to a pool of their own, or a loop in which
cudaMalloc is banned because it synchronises the device).  The library keeps
the scratch in a fixed 32 MiB device array instead of taking a workspace.

Checked here through the C ABI: two calls in a row, on different inputs, must
each reproduce tb_factor (same arithmetic, so the tolerance of the factor
parity test, 1e-6 relative, is met with room), the second call must not be
disturbed by what the first left in the shared array, and a problem larger
than the array must be refused.  This file sorts last on purpose: a run that
stops at the first failure has then already run every other test."""
import ctypes

import numpy as np
import pytest

import tb_inputs

pytestmark = pytest.mark.gpu


def _rel(a, b):
    return float(np.linalg.norm(a.astype(np.float64) - b.astype(np.float64)) / np.linalg.norm(b.astype(np.float64)))


def test_static_scratch_factor_matches_tb_factor_twice():
    import torch
    import paper_2602_04929_b200 as tb
    lib = tb.load()
    assert lib.tb_factor_static_capacity() == 32 << 20
    dev = torch.device("cuda:0")
    # per-head H_out shape, a ragged size, and the largest single matrix that fits: at 1024 columns
    # tb_factor splits its trailing updates over a helper stream and this entry point does not, yet
    # every entry receives the same updates in the same order
    cases = [(32, 128, 1e3, 40), (3, 200, 1e4, 50), (1, 1024, 1e4, 60)]
    for n_batch, d, cond, seed in cases:
        H = np.stack([tb_inputs.spd_matrix(seed + b, d, cond=cond) for b in range(n_batch)])
        Hd = torch.from_numpy(H).to(dev)
        U_ref, info_ref = tb.tb_factor(Hd)
        # outputs allocated up front; the call itself takes only pointers
        U = torch.full_like(Hd, float("nan"))
        info = torch.full((n_batch,), -1, dtype=torch.int32, device=dev)
        st = lib.tb_factor_static(ctypes.c_void_p(Hd.data_ptr()), n_batch, d, ctypes.c_void_p(U.data_ptr()),
                                  ctypes.c_void_p(info.data_ptr()),
                                  ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert st == 0, tb.status_string(st)
        torch.cuda.synchronize()
        assert info.cpu().tolist() == info_ref.cpu().tolist() == [0] * n_batch
        for b in range(n_batch):
            assert _rel(U[b].cpu().numpy(), U_ref[b].cpu().numpy()) <= 1e-6
        assert torch.equal(U, U_ref)
        assert torch.equal(torch.tril(U, -1), torch.zeros_like(U))
        # the array exists by now (the call above was at least the first on this device): one more call
        # must leave the device's free memory exactly as it found it
        free_before, _ = torch.cuda.mem_get_info(dev)
        st = lib.tb_factor_static(ctypes.c_void_p(Hd.data_ptr()), n_batch, d, ctypes.c_void_p(U.data_ptr()),
                                  ctypes.c_void_p(info.data_ptr()),
                                  ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
        assert st == 0, tb.status_string(st)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info(dev)
        assert free_after == free_before
        assert torch.equal(U, U_ref)


def test_static_scratch_rejects_what_does_not_fit():
    import paper_2602_04929_b200 as tb
    lib = tb.load()
    one = ctypes.c_void_p(256)   # never dereferenced: the size check comes first
    assert lib.tb_factor_workspace(1, 4096) > lib.tb_factor_static_capacity()
    assert lib.tb_factor_static(one, 1, 4096, one, one, None) == 2      # TB_ERR_UNSUPPORTED
    assert lib.tb_factor_static(one, 128, 128, one, one, None) == 2
    assert lib.tb_factor_static(None, 1, 64, one, one, None) == 1       # TB_ERR_INVALID_ARG
