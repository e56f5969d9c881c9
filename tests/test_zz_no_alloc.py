"""The allocation-free Block-Sign sweep (compams_blocksign_sweep_static) against the handle-based path.

Some users of the library run where device allocation is impossible (an allocator callback of
another framework, a process with pre-partitioned device memory, a latency-critical stream). For
them the library offers one entry point whose scratch is a fixed array inside the library. This
test drives it through the C ABI with caller-owned buffers only, twice in a row (the second call
sees whatever the first left in the shared scratch), and checks scales, sign bits and the
residual against what compams_step produces for the same gradients.

The file name sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import pytest
import torch

from paper_2205_05632_b200 import BLOCKSIGN, CompAMS, CompAMSError
from paper_2205_05632_b200.binding import blocksign_sweep_static, blocksign_sweep_static_limits

pytestmark = pytest.mark.gpu

ATOL, RTOL = 1e-7, 1e-6  # the float tolerance of the parity tests


def _close(a, b):
    return bool(((a - b).abs() <= ATOL + RTOL * b.abs()).all())


@pytest.mark.parametrize("n,d", [(3, 3 * 8192 + 1234), (2, 5000), (4, 2 * 8192 + 2)])
def test_static_sweep_matches_the_handle_path_on_two_calls_in_a_row(n, d):
    gen = torch.Generator(device="cuda").manual_seed(99)
    ref = CompAMS(n, d, [0, d], BLOCKSIGN)
    theta = torch.zeros(d, device="cuda")
    # caller-owned buffers of the allocation-free path, created before the first call
    x_state = torch.zeros(n, d, device="cuda")
    scales = [torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")]
    bits = torch.zeros(n, (d + 31) // 32, dtype=torch.int32, device="cuda")
    for t in range(2):
        G = torch.randn(n, d, generator=gen, device="cuda")
        ref.step(G, theta)
        blocksign_sweep_static(G, x_state, scales[(t + 1) % 2] if t else None, scales[t % 2], bits, deferred=t > 0)
        torch.cuda.synchronize()
        want_scales = ref.buffer("scales").flatten()
        assert _close(scales[t % 2], want_scales)
        assert torch.equal(bits, ref.buffer("sign_bits"))
        # the residual the next call will reconstruct: e = x - sign(x) * scale
        e = x_state - torch.copysign(scales[t % 2][:, None].expand(n, d), x_state)
        assert _close(e, ref.buffer("E"))
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
