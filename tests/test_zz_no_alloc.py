"""The allocation-free loss entry point gives the same results as the workspace one.

twist_mse_fwd_bwd_noalloc is for callers that are not allowed to allocate device memory (no
cudaMalloc in a serving loop, a host application that hands over fixed buffers only): it keeps its
scratch inside the library.  Here it is called through the C ABI twice in a row -- the second call
with other data and fewer subnets, so that stale scratch contents from the first call would show --
and each time compared with twist_mse_fwd_bwd on the same inputs.  The file name sorts last so that
a run that stops at the first failure has already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2511_03983_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _both(B, dtype, S, T, width, valid, seg_begin, seg_width, seed):
    td = torch.bfloat16 if dtype == I.DTYPE_BF16 else torch.float32
    y = torch.from_numpy(I.normal(seed, 1, (S, T, width), 1.0, dtype)).to(td).cuda()
    t = torch.from_numpy(I.normal(seed, 2, (S, T, width), 1.0, dtype)).to(td).cuda()
    vc = None if valid is None else torch.tensor(valid, dtype=torch.int32, device="cuda")
    ws = torch.empty(B.twist_mse_workspace_bytes(S), dtype=torch.uint8, device="cuda")
    dy_a, dy_b = torch.zeros_like(y), torch.zeros_like(y)
    loss_a = torch.zeros(S, dtype=torch.float32, device="cuda")
    loss_b = torch.zeros(S, dtype=torch.float32, device="cuda")
    B.twist_mse_fwd_bwd(y, t, dy_a, loss_a, S, T, width, vc, seg_begin, seg_width, dtype, ws)
    B.twist_mse_fwd_bwd_noalloc(y, t, dy_b, loss_b, S, T, width, vc, seg_begin, seg_width, dtype)
    torch.cuda.synchronize()
    # same kernels, same launch shape, same summation order: the tolerance of the other tests
    # (1e-5 relative on the loss) is met with equality
    assert torch.allclose(loss_a, loss_b, rtol=1e-5, atol=0)
    assert torch.equal(dy_a, dy_b)
    assert float(loss_a.min()) > 0.5      # N(0,1) - N(0,1): the loss is about 2, not a stale zero


def test_noalloc_matches_workspace_entry_point_twice_in_a_row():
    from paper_2511_03983_b200 import binding as B
    B.lib()
    _both(B, I.DTYPE_BF16, 8, 1024, 512, None, 0, 0, seed=61)                      # many blocks per subnet
    _both(B, I.DTYPE_BF16, 3, 77, 72, [8, 16, 24], 24, 24, seed=62)                # fewer subnets, ragged columns
    _both(B, I.DTYPE_FP32, 2, 50, 20, None, 0, 0, seed=63)
    assert B.twist_device_status() == 0


def test_noalloc_call_allocates_no_device_memory():
    """What the entry point is for: once its first call on the device has happened, a call leaves the device's free
    memory and the allocator's books exactly as they were."""
    from paper_2511_03983_b200 import binding as B
    B.lib()
    S, T, width = 4, 256, 128
    y = torch.randn(S, T, width, device="cuda").to(torch.bfloat16)
    t = torch.randn(S, T, width, device="cuda").to(torch.bfloat16)
    dy = torch.zeros_like(y)
    loss = torch.zeros(S, dtype=torch.float32, device="cuda")
    B.twist_mse_fwd_bwd_noalloc(y, t, dy, loss, S, T, width, None, 0, 0, I.DTYPE_BF16)      # warm-up: first call
    torch.cuda.synchronize()
    free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
    for _ in range(3):
        B.twist_mse_fwd_bwd_noalloc(y, t, dy, loss, S, T, width, None, 0, 0, I.DTYPE_BF16)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free0
    assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    assert float(loss.min()) > 0.5


def test_noalloc_rejects_more_subnets_than_its_scratch_holds():
    from paper_2511_03983_b200 import binding as B
    h = B.lib()
    x = torch.zeros(64, dtype=torch.bfloat16, device="cuda")
    loss = torch.zeros(64, dtype=torch.float32, device="cuda")
    rc = h.twist_mse_fwd_bwd_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), loss.data_ptr(), 33, 1, 8, None, 0, 0,
                                     B.BF16, None)
    assert rc == B.ERR_UNSUPPORTED
    assert b"implemented range" in h.twist_strerror(rc)
