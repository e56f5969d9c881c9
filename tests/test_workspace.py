"""The optimizer's state in caller memory: compams_workspace_bytes (host arithmetic, no GPU needed) and
compams_create_in_workspace (a handle whose every device buffer is cut from one caller-owned region)."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2205_05632_b200 import BLOCKSIGN, RANDK, TOPK, CompAMS, CompAMSError, load_library, workspace_bytes

D = 11_173_962


def test_workspace_size_is_host_arithmetic_and_covers_the_named_buffers():
    for comp, ratio in ((TOPK, 0.01), (BLOCKSIGN, 1.0), (RANDK, 0.01)):
        b16, b32 = workspace_bytes(16, D, [0, D], comp, ratio), workspace_bytes(32, D, [0, D], comp, ratio)
        assert b16 % 256 == 0 and b32 % 256 == 0
        # e [n, d] and m, v, vhat, gbar [d] are in there, and the size grows by at least one row of e per worker
        assert b16 >= (16 + 4) * D * 4
        assert b32 - b16 >= 16 * D * 4
    # k = d: no error accumulators, only the server's vectors and the status words
    assert workspace_bytes(16, D, [0, D], TOPK, 1.0) < 5 * D * 4
    # sharded handle: e for the local workers, messages for all
    assert workspace_bytes(4, D, [0, D], BLOCKSIGN, 1.0, n_total=16) < workspace_bytes(16, D, [0, D], BLOCKSIGN)


def test_workspace_size_rejects_what_create_rejects():
    L = load_library()
    out = ctypes.c_size_t(0)
    offs = (ctypes.c_int64 * 2)(0, 10)
    assert L.compams_workspace_bytes(ctypes.byref(out), 0, 0, 10, offs, 1, 0, 0.5) == -1       # n < 1
    assert L.compams_workspace_bytes(ctypes.byref(out), 2, 2, 11, offs, 1, 0, 0.5) == -1       # last offset != d
    assert L.compams_workspace_bytes(ctypes.byref(out), 2, 2, 10, offs, 1, 7, 0.5) == -1       # unknown compressor
    assert L.compams_workspace_bytes(None, 2, 2, 10, offs, 1, 0, 0.5) == -1
    assert L.compams_workspace_bytes(ctypes.byref(out), 2, 2, 10, offs, 1, 0, 0.5) == 0 and out.value > 0


@pytest.mark.gpu
@pytest.mark.parametrize("comp,ratio", [(TOPK, 0.02), (BLOCKSIGN, 1.0), (RANDK, 0.02), (TOPK, 1.0)])
def test_handle_in_caller_memory_matches_the_self_allocating_handle(comp, ratio):
    n, d = 3, 5 * 8192 + 1234
    offs = [0, 3000, 20000, d]
    need = workspace_bytes(n, d, offs, comp, ratio)
    ws = torch.full((need,), 0xA5, dtype=torch.uint8, device="cuda")  # garbage: the handle must initialise its state
    assert ws.data_ptr() % 256 == 0
    a = CompAMS(n, d, offs, comp, ratio, workspace=ws, record_average=True)
    b = CompAMS(n, d, offs, comp, ratio, record_average=True)
    gen = torch.Generator(device="cuda").manual_seed(4)
    ta, tb = torch.zeros(d, device="cuda"), torch.zeros(d, device="cuda")
    for _ in range(4):
        G = torch.randn(n, d, generator=gen, device="cuda")
        a.step(G, ta)
        b.step(G, tb)
    assert a.check_status() == 0
    assert torch.equal(ta, tb)
    for name in ("E", "m", "v", "vhat", "gbar"):
        assert torch.equal(a.buffer(name), b.buffer(name)), name
    # every buffer of the handle lies inside the caller's region
    lo, hi = ws.data_ptr(), ws.data_ptr() + need
    for name in ("m", "v", "vhat", "gbar", "status"):
        p = a.buffer(name).data_ptr()
        assert lo <= p < hi, name
    a.close()
    b.close()
    # too small a region, or one off the 256-byte grid, is refused
    with pytest.raises(CompAMSError):
        CompAMS(n, d, offs, comp, ratio, workspace=ws[:need - 256])
    with pytest.raises(CompAMSError):
        CompAMS(n, d, offs, comp, ratio, workspace=torch.empty(need + 16, dtype=torch.uint8, device="cuda")[16:])
