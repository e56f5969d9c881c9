"""The allocation-free Block-Sign sweep (compams_blocksign_sweep_static) against the handle-based path.

Some users of the library run where device allocation is impossible (an allocator callback of
another framework, a process with pre-partitioned device memory, a latency-critical stream). For
them the library offers one entry point whose scratch is a fixed array inside the library. This
test drives it through the C ABI with caller-owned buffers only, twice in a row (the second call
sees whatever the first left in the shared scratch), and checks scales, sign bits and the
residual against what compams_step produces for the same gradients, and against Definition 2 written out
on the CPU (the oracle's exact block scale, the sign bit of g + e).

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

import oracle

from paper_2205_05632_b200 import BLOCKSIGN, CompAMS, CompAMSError
from paper_2205_05632_b200.binding import blocksign_sweep_static, blocksign_sweep_static_limits

pytestmark = pytest.mark.gpu

ATOL, RTOL = 1e-7, 1e-6  # the float tolerance of the parity tests


def _close(a, b):
    return bool(((a - b).abs() <= ATOL + RTOL * b.abs()).all())


def _unpack(bits, d):
    """[n, ceil(d/32)] int32 words, LSB first -> [n, d] booleans; the padding bits must be zero."""
    u8 = np.ascontiguousarray(bits.cpu().numpy()).view(np.uint8)
    b = np.unpackbits(u8, axis=1, bitorder="little")
    assert not b[:, d:].any(), "padding bits are not zero"
    return b[:, :d].astype(bool)


# d = 0, 1, 2 and 3 mod 4: the rows of the packed [n, d] buffers then start in every 16-byte phase, so the
# 128-, 64- and 32-bit access branches of the kernel all run; `shift` moves the caller's buffers off the
# 16-byte grid as a whole
@pytest.mark.parametrize("n,d,shift", [(3, 3 * 8192 + 1234, 0), (2, 5000, 0), (4, 2 * 8192 + 2, 0), (4, 2 * 8192 + 4101, 0),
                                       (5, 8192 + 3, 0), (3, 2 * 8192 + 77, 1), (2, 8192 + 6, 3), (1, 31, 2)])
def test_static_sweep_matches_the_handle_path_on_two_calls_in_a_row(n, d, shift):
    gen = torch.Generator(device="cuda").manual_seed(99)
    ref = CompAMS(n, d, [0, d], BLOCKSIGN)
    theta = torch.zeros(d, device="cuda")
    # caller-owned buffers of the allocation-free path, created before the first call
    g_store = torch.zeros(n * d + 8, device="cuda")
    x_store = torch.zeros(n * d + 8, device="cuda")
    G_in = g_store[shift:shift + n * d].view(n, d)
    x_state = x_store[shift:shift + n * d].view(n, d)
    assert x_state.data_ptr() % 16 == (4 * shift) % 16
    scales = [torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")]
    bits = torch.zeros(n, (d + 31) // 32, dtype=torch.int32, device="cuda")
    e_cpu = np.zeros((n, d), dtype=np.float32)  # the error accumulators as the definitions give them
    for t in range(2):
        G = torch.randn(n, d, generator=gen, device="cuda")
        G_in.copy_(G)
        ref.step(G, theta)
        blocksign_sweep_static(G_in, x_state, scales[(t + 1) % 2] if t else None, scales[t % 2], bits, deferred=t > 0)
        torch.cuda.synchronize()
        # against the handle-based entry point
        want_scales = ref.buffer("scales").flatten()
        assert _close(scales[t % 2], want_scales)
        assert torch.equal(bits, ref.buffer("sign_bits"))
        # the residual the next call will reconstruct: e = x - sign(x) * scale
        e = x_state - torch.copysign(scales[t % 2][:, None].expand(n, d), x_state)
        assert _close(e, ref.buffer("E"))
        # against the definitions themselves: x = g + e (Algorithm 2), sign bit of x, scale = ||x||_1 / d (Definition 2)
        x_cpu = G.cpu().numpy() + e_cpu
        assert np.array_equal(x_state.cpu().numpy().view(np.int32), x_cpu.view(np.int32))
        assert np.array_equal(_unpack(bits, d), np.signbit(x_cpu))
        s_cpu = np.array([oracle.blocksign_scale(x_cpu[i]) for i in range(n)], dtype=np.float32)
        assert _close(scales[t % 2], torch.from_numpy(s_cpu).cuda())
        e_cpu = x_cpu - np.copysign(s_cpu[:, None], x_cpu)
    assert ref.check_status() == 0
    ref.close()


def test_static_sweep_rejects_sizes_beyond_its_fixed_scratch():
    max_workers, max_tiles = blocksign_sweep_static_limits()
    assert max_workers == 1024 and max_tiles == 65536
    n, d = 2, 64
    g = torch.zeros(n, d, device="cuda")
    x = torch.zeros(n, d, device="cuda")
    s = torch.zeros(n, device="cuda")
    b = torch.zeros(n, 2, dtype=torch.int32, device="cuda")
    from paper_2205_05632_b200 import load_library
    import ctypes
    L = load_library()
    # too many workers / too many tiles: refused with the dedicated status, nothing is launched
    rc = L.compams_blocksign_sweep_static(g.data_ptr(), x.data_ptr(), None, s.data_ptr(), b.data_ptr(),
                                          max_workers + 1, d, 0, None)
    assert rc == -5
    rc = L.compams_blocksign_sweep_static(g.data_ptr(), x.data_ptr(), None, s.data_ptr(), b.data_ptr(),
                                          16, 8192 * (max_tiles // 16) + 1, 0, None)
    assert rc == -5
    assert L.compams_error_string(-5) == b"problem size exceeds the fixed scratch capacity"
    with pytest.raises(CompAMSError):
        blocksign_sweep_static(g, x, None, s, b[:, :1].contiguous(), deferred=False)
