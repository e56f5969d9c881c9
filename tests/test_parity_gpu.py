"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle."""
import numpy as np
import pytest
import torch

from paper_2205_05632_b200 import BLOCKSIGN, RANDK, TOPK, CompAMS, CompAMSError
from paper_2205_05632_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _pair_run(n, d, offsets, comp, ratio, make_g, steps=4, theta_sigma=0.1, check_e_every=1, **hp):
    from parity import Pair
    gen = torch.Generator(device="cuda").manual_seed(1234)
    if comp == RANDK:
        hp.setdefault("seed", 2022)
    p = Pair(n, d, offsets, comp, ratio, **hp)
    try:
        p.start(theta_sigma * torch.randn(d, generator=gen, device="cuda"))
        for t in range(steps):
            p.step(make_g(gen, t), check_e=(t % check_e_every == 0) or t == steps - 1)
        return p.inexact
    finally:
        p.close()


def _randn(n, d):
    return lambda gen, t: torch.randn(n, d, generator=gen, device="cuda")


def _randn_bf16(n, d):
    return lambda gen, t: torch.randn(n, d, generator=gen, device="cuda").bfloat16()


# ------------------------------------------------------------------ mid-size cases: several tiles, ragged tails

RAGGED = [0, 10, 74, 1098, 5194, 5195, 13387 + 5, 13392 + 3 * 8192 + 1234, 13392 + 3 * 8192 + 1234 + 4097]


@pytest.mark.parametrize("n", [1, 3])
@pytest.mark.parametrize("ratio", [0.01, 0.3, 1.0])
def test_topk_ragged_blocks(n, ratio):
    d = RAGGED[-1]
    _pair_run(n, d, RAGGED, TOPK, ratio, _randn(n, d))


@pytest.mark.parametrize("n", [1, 5])
@pytest.mark.parametrize("check_e_every", [1, 100])
def test_blocksign_ragged_blocks(n, check_e_every):
    d = RAGGED[-1]
    _pair_run(n, d, RAGGED, BLOCKSIGN, 1.0, _randn(n, d), steps=5, check_e_every=check_e_every)


@pytest.mark.parametrize("n", [2, 7, 31, 32, 33, 70])
def test_blocksign_worker_counts_around_the_transposition_width(n):
    # the server kernel transposes the sign words of up to 32 workers at a time and looks up the scales of 4
    # workers at once: worker counts below, at and above those widths, blocks that end inside a word
    d = 2 * 8192 + 1234
    _pair_run(n, d, [0, 37, 5000, 8192 + 100, d], BLOCKSIGN, 1.0, _randn(n, d), steps=3)


@pytest.mark.parametrize("d", [1, 2, 3, 5, 31, 33, 4096, 4097, 8191, 8192, 8193, 3 * 8192 + 2])
@pytest.mark.parametrize("comp", [TOPK, BLOCKSIGN])
def test_single_block_sizes_around_tile_edges(d, comp):
    _pair_run(2, d, [0, d], comp, 0.1, _randn(2, d), steps=3)


@pytest.mark.parametrize("comp,ratio", [(TOPK, 0.01), (TOPK, 0.3), (TOPK, 1.0), (BLOCKSIGN, 1.0), (RANDK, 0.05)])
@pytest.mark.parametrize("n", [1, 3, 4])
def test_bfloat16_gradients_ragged_blocks(comp, ratio, n):
    # d = 3 mod 4 and odd block offsets: rows and blocks of the bfloat16 tensor start in every alignment class
    d = RAGGED[-1]
    assert d % 4 == 3
    _pair_run(n, d, RAGGED, comp, ratio, _randn_bf16(n, d))


def test_bfloat16_and_fp32_gradients_may_alternate():
    d = 3 * 8192 + 77
    mixed = lambda gen, t: (torch.randn(2, d, generator=gen, device="cuda").bfloat16() if t % 2 else
                            torch.randn(2, d, generator=gen, device="cuda"))
    for comp in (TOPK, BLOCKSIGN):
        _pair_run(2, d, [0, d], comp, 0.02, mixed, steps=5)


def test_bfloat16_gradients_resnet18_shapes_blocksign_and_topk():
    w = W.config2("cuda")
    theta = w.start()
    from parity import Pair
    for comp, ratio, offs in ((BLOCKSIGN, 1.0, w.block_offsets), (TOPK, 0.01, np.array([0, w.d]))):
        p = Pair(4, w.d, offs, comp, ratio)
        try:
            p.start(theta)
            for t in range(3):
                p.step(w.grads()[:4].contiguous().bfloat16(), check_e=(t == 2))
        finally:
            p.close()


def test_rows_not_multiple_of_four_use_all_alignment_classes():
    # d = 1 mod 4: rows 0..3 start at four different 16-byte phases
    d = 2 * 8192 + 4101
    for comp in (TOPK, BLOCKSIGN):
        _pair_run(4, d, [0, 4099, d], comp, 0.05, _randn(4, d), steps=3)
    _pair_run(4, d, [0, d], TOPK, 1.0, _randn(4, d), steps=3)


@pytest.mark.parametrize("shift", [1, 2, 3])
def test_gradient_buffer_off_the_16_byte_grid(shift):
    # the caller's G may start anywhere on the 4-byte grid, while E is the library's own: the two no
    # longer share their alignment and G is read with narrower loads; results must not change
    n, d = 3, 2 * 8192 + 4101
    offs = [0, 4099, d]
    for comp, ratio in ((TOPK, 0.05), (BLOCKSIGN, 1.0), (TOPK, 1.0)):
        a = CompAMS(n, d, offs, comp, ratio, record_average=True)
        b = CompAMS(n, d, offs, comp, ratio, record_average=True)
        ta = torch.zeros(d, device="cuda")
        tb = torch.zeros(d, device="cuda")
        gen = torch.Generator(device="cuda").manual_seed(77)
        for t in range(3):
            G = torch.randn(n, d, generator=gen, device="cuda")
            store = torch.empty(n * d + 8, device="cuda")
            Gs = store[shift:shift + n * d].view(n, d)
            Gs.copy_(G)
            assert Gs.data_ptr() % 16 == 4 * shift
            a.step(G, ta)
            b.step(Gs, tb)
        for name in ("E", "m", "v", "vhat", "gbar"):
            assert torch.equal(a.buffer(name).view(torch.int32), b.buffer(name).view(torch.int32)), name
        assert torch.equal(ta.view(torch.int32), tb.view(torch.int32))
        a.close()
        b.close()


def test_blocks_of_size_one_and_tiny():
    d = 200
    offs = list(range(0, 101)) + [110, 150, 200]
    for comp in (TOPK, BLOCKSIGN):
        _pair_run(3, d, offs, comp, 0.2, _randn(3, d), steps=3)


def test_more_tiled_blocks_than_the_kernel_argument_block_list_holds():
    # the sweeps find a tile's block in a kernel-argument copy of the block list when it has at most 168
    # entries; beyond that they read a per-tile table in global memory
    sizes = [4097 + 37 * (b % 23) for b in range(181)]   # Top-k: 181 tiled blocks (each above 4096 coordinates)
    offs = np.concatenate([[0], np.cumsum(sizes)]).tolist()
    _pair_run(2, offs[-1], offs, TOPK, 0.01, _randn(2, offs[-1]), steps=4)
    sizes = [1 + (7 * b) % 300 for b in range(400)] + [9000, 3, 8192, 1]   # Block-Sign: every block is tiled
    offs = np.concatenate([[0], np.cumsum(sizes)]).tolist()
    _pair_run(3, offs[-1], offs, BLOCKSIGN, 1.0, _randn(3, offs[-1]), steps=4)


# ------------------------------------------------------------------ degenerate inputs: ties everywhere

def _quantised(n, d, levels):
    def make(gen, t):
        return torch.randint(-levels, levels + 1, (n, d), generator=gen, device="cuda").float()
    return make


@pytest.mark.parametrize("levels", [0, 1, 3])
@pytest.mark.parametrize("d,offs", [(3000, [0, 3000]), (40000, [0, 40000]), (60000, [0, 100, 30000, 60000])])
def test_topk_with_massive_ties(levels, d, offs):
    # all zeros (levels = 0) or a tiny alphabet: the threshold is tied many times over and the
    # lower indices must win, tile after tile
    _pair_run(2, d, offs, TOPK, 0.07, _quantised(2, d, levels), steps=3)


def test_topk_ties_straddling_tiles_with_k_one():
    d = 5 * 8192
    def make(gen, t):
        g = torch.zeros(2, d, device="cuda")
        g[0, 3 * 8192 + 5] = 2.0
        g[0, 4 * 8192 + 7] = -2.0   # equal magnitude further right: must lose
        g[1, :] = 1.0
        return g
    _pair_run(2, d, [0, d], TOPK, 1.0 / d, make, steps=3)


def test_blocksign_zero_and_signed_zero_inputs():
    d = 10000
    def make(gen, t):
        g = torch.randn(2, d, generator=gen, device="cuda")
        g[0, ::3] = 0.0
        g[1, ::5] = -0.0
        if t == 1:
            g[1] = 0.0
        return g
    _pair_run(2, d, [0, 777, d], BLOCKSIGN, 1.0, make, steps=4, check_e_every=2)


def test_heavy_tails_and_wide_dynamic_range():
    d = 50000
    def make(gen, t):
        e = torch.randint(-40, 40, (3, d), generator=gen, device="cuda").float()
        return torch.randn(3, d, generator=gen, device="cuda") * torch.exp2(e)
    for comp in (TOPK, BLOCKSIGN):
        _pair_run(3, d, [0, 20000, d], comp, 0.01, make, steps=3)


# ------------------------------------------------------------------ reductions

def test_n_one_and_identity_mode_have_zero_error_buffer():
    d = 3 * 8192 + 77
    opt = CompAMS(2, d, [0, d], TOPK, 1.0)
    theta = torch.zeros(d, device="cuda")
    opt.step(torch.randn(2, d, device="cuda"), theta)
    assert not opt.buffer("E").any()
    assert opt.buffer("topk_idx").numel() == 0
    opt.close()


def test_run_to_run_determinism():
    d = 6 * 8192 + 3
    G = [torch.randn(4, d, device="cuda") for _ in range(3)]
    for comp, ratio in ((TOPK, 0.02), (BLOCKSIGN, 1.0)):
        outs = []
        for rep in range(2):
            opt = CompAMS(4, d, [0, 5000, d], comp, ratio)
            theta = torch.zeros(d, device="cuda")
            for g in G:
                opt.step(g, theta)
            outs.append((theta.clone(), opt.buffer("E").clone(), opt.buffer("vhat").clone()))
            opt.close()
        for a, b in zip(*outs):
            assert torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_step_host_matches_step():
    d = 2 * 8192 + 10
    G = torch.randn(3, d)
    theta0 = torch.randn(d)
    a = CompAMS(3, d, [0, d], TOPK, 0.05)
    b = CompAMS(3, d, [0, d], TOPK, 0.05)
    th_dev = theta0.cuda()
    a.step(G.cuda(), th_dev)
    th_host = theta0.clone()
    b.step_host(G, th_host)
    assert torch.equal(th_dev.cpu(), th_host)
    a.close()
    b.close()


def test_argument_errors_are_reported_not_fatal():
    with pytest.raises(CompAMSError):
        CompAMS(0, 10, [0, 10], TOPK, 0.1)
    with pytest.raises(CompAMSError):
        CompAMS(2, 10, [0, 5, 5, 10], TOPK, 0.1)
    with pytest.raises(CompAMSError):
        CompAMS(2, 10, [0, 10], TOPK, 0.0)
    with pytest.raises(CompAMSError):
        CompAMS(2, 10, [0, 10], 7, 0.5)
    opt = CompAMS(2, 10, [0, 10], TOPK, 0.5)
    with pytest.raises(CompAMSError):
        opt.step(torch.zeros(2, 11, device="cuda"), torch.zeros(10, device="cuda"))
    opt.close()


# ------------------------------------------------------------------ the named configurations, 10 chained steps

def test_config1_topk_small_dense_gaussian():
    from parity import run_workload
    run_workload(W.config1("cuda"))


def test_config2_blocksign_resnet18_shapes():
    from parity import run_workload
    run_workload(W.config2("cuda"), check_e_every=3)


@pytest.mark.parametrize("ratio", [0.001, 0.01])
def test_config3_topk_whole_vector_with_zeros(ratio):
    from parity import run_workload
    run_workload(W.config3(ratio, "cuda"), check_e_every=3)


@pytest.mark.parametrize("comp", [TOPK, BLOCKSIGN])
def test_config4_resnet50_shapes_layerwise(comp):
    from parity import run_workload
    run_workload(W.config4(comp, "cuda"), check_e_every=5)


@pytest.mark.parametrize("mode", ["topk", "sign", "dense"])
@pytest.mark.parametrize("n", [1, 8, 32])
def test_config5_sweep_points_oracle_sized(mode, n):
    from parity import run_workload
    run_workload(W.sweep_point(1 << 20, n, mode, "cuda"), steps=10, check_e_every=3)


@pytest.mark.parametrize("mode", ["topk", "sign", "dense"])
def test_config5_sweep_point_d_2_24_n_8_against_the_full_oracle(mode):
    from parity import run_workload
    run_workload(W.sweep_point(1 << 24, 8, mode, "cuda"), steps=10, check_e_every=5)


@pytest.mark.parametrize("mode", ["topk", "sign", "dense", "randk"])
def test_config5_largest_point_d_2_27_n_32_against_the_full_oracle(mode):
    # the largest configuration: n d = 2^32 elements (16 GiB per [n, d] buffer), every index beyond 32 bits.
    # Two chained steps: the first Top-k selection runs the dense passes, the second the candidate path.
    free, _ = torch.cuda.mem_get_info()
    if free < 80 * (1 << 30):
        pytest.skip("needs about 80 GiB of free device memory")
    import psutil
    if psutil.virtual_memory().available < 120 * (1 << 30):
        pytest.skip("needs about 120 GiB of free host memory for the oracle")
    from parity import run_workload
    run_workload(W.sweep_point(1 << 27, 32, mode, "cuda"), steps=2, check_e_every=2)
    torch.cuda.empty_cache()


# ------------------------------------------------------------------ the candidate path and its fallbacks

def _status(opt):
    return opt.buffer("status").cpu().tolist()


def test_topk_candidate_path_is_taken_in_steady_state():
    # after the first steps the threshold prediction must carry the selection: the dense passes stop
    from parity import Pair
    n, d = 4, 40 * 8192 + 321
    gen = torch.Generator(device="cuda").manual_seed(5)
    p = Pair(n, d, [0, d], TOPK, 0.01)
    try:
        p.start(torch.zeros(d, device="cuda"))
        for t in range(8):
            p.step(torch.randn(n, d, generator=gen, device="cuda"), check_e=(t % 3 == 0))
        st = _status(p.gpu)
        assert st[0] == 0
        assert st[1] + st[2] == 8 * n
        assert st[1] <= 3 * n, "dense passes ran on %d of %d selections" % (st[1], 8 * n)
    finally:
        p.close()


@pytest.mark.parametrize("d", [40 * 8192 + 321, (1 << 21) + 5])
def test_topk_candidate_path_survives_gradients_that_alternate_between_two_batches(d):
    # the same two gradient tensors in turn (what a benchmark ring does, and what a data loader with two
    # shards does): the threshold then alternates between two levels instead of drifting. The prediction must
    # keep the selection inside the candidate lists (short list: one CTA; long list: slices) - and stay exact
    from parity import Pair
    n = 4
    gen = torch.Generator(device="cuda").manual_seed(8)
    ring = [torch.randn(n, d, generator=gen, device="cuda") for _ in range(2)]
    p = Pair(n, d, [0, d], TOPK, 0.01)
    try:
        p.start(torch.zeros(d, device="cuda"))
        for t in range(12):
            p.step(ring[t % 2], check_e=(t % 4 == 3))
        st = _status(p.gpu)
        assert st[0] == 0 and st[1] + st[2] == 12 * n
        assert st[1] <= 3 * n, "dense passes ran on %d of %d selections: %r" % (st[1], 12 * n, st)
    finally:
        p.close()


@pytest.mark.parametrize("blocks", [1, 24])
def test_topk_dense_passes_stay_rare_over_hundreds_of_alternating_steps(blocks):
    # Two alternating batches over 400 steps: under error feedback the threshold then swings between two levels
    # and the magnitudes pile up just below it. A smaller candidate margin is probed again and again; a probe that
    # fails costs a dense-pass step, so failed probes must back off, and a segment sent to the dense passes must
    # come back with a threshold fine enough not to return there on the next step.
    n, d = 4, 48 * 8192
    offs = [d // blocks * b for b in range(blocks)] + [d]
    gen = torch.Generator(device="cuda").manual_seed(11)
    ring = [torch.randn(n, d, generator=gen, device="cuda") for _ in range(2)]
    theta = torch.zeros(d, device="cuda")
    opt = CompAMS(n, d, offs, TOPK, 0.01)
    try:
        steps, after = 400, 8
        for t in range(steps):
            if t == after:
                st0 = _status(opt)
            opt.step(ring[t % 2], theta)
        st = _status(opt)
        opt.check_status()
        selections = (steps - after) * n * blocks
        assert (st[1] - st0[1]) + (st[2] - st0[2]) == selections
        dense = st[1] - st0[1]
        # a fixed wait of 32 selections between probes gives one dense-pass selection in 33: 3 %
        assert dense <= 0.015 * selections, "dense passes decided %d of %d selections: %r" % (dense, selections, st)
    finally:
        opt.close()


def test_topk_no_dense_pass_after_the_first_steps_with_a_new_batch_every_step():
    # independent gradients every step, 300 steps, a long list (slices) and short ones (one CTA each): once the
    # error accumulators have filled, every selection is decided inside its candidate list, through every change
    # of the candidate margin
    n, d = 4, 1 << 22
    offs = [0, 1 << 21, (1 << 21) + 300000, d]
    gen = torch.Generator(device="cuda").manual_seed(12)
    theta = torch.zeros(d, device="cuda")
    G = torch.empty(n, d, device="cuda")
    opt = CompAMS(n, d, offs, TOPK, 0.01)
    try:
        steps, after = 300, 40
        for t in range(steps):
            if t == after:
                st0 = _status(opt)
            G.normal_(generator=gen)
            opt.step(G, theta)
        st = _status(opt)
        opt.check_status()
        assert st[2] - st0[2] == (steps - after) * n * 3 and st[1] == st0[1], "dense passes after step %d: %r -> %r" % (after, st0, st)
    finally:
        opt.close()


@pytest.mark.parametrize("name,n,blocks,block_len,ring,steps", [
    ("one block, two alternating batches", 4, 1, 48 * 8192 + 77, 2, 100),
    ("24 blocks, two alternating batches", 3, 24, 20000, 2, 100),
    ("one block, a new batch every step", 4, 1, 40 * 8192 + 5, 0, 80),
    ("720 lists layer-wise", 8, 90, 9000, 2, 40)])
def test_topk_long_chained_runs_against_the_oracle(name, n, blocks, block_len, ring, steps):
    # long enough for the candidate margin to be raised, probed and taken back several times (alternating batches
    # make lists come up short and nearly short), and with enough lists for the narrower select CTAs: every step
    # against the oracle, E on every seventh
    d = blocks * block_len
    offs = [block_len * b for b in range(blocks + 1)]
    gen0 = torch.Generator(device="cuda").manual_seed(77)
    batches = [torch.randn(n, d, generator=gen0, device="cuda") for _ in range(ring)]

    def make(gen, t):
        return batches[t % ring] if ring else torch.randn(n, d, generator=gen, device="cuda")
    _pair_run(n, d, offs, TOPK, 0.01, make, steps=steps, check_e_every=7)


def test_topk_prediction_failures_fall_back_exactly():
    # the gradient scale jumps by orders of magnitude between steps: too few candidates, too many,
    # thresholds far above the predicted range - every case must still give the exact Top-k
    scales = [1.0, 1.0, 1.0, 1.0, 300.0, 1.0, 1.0, 1e-3, 1e-3, 50.0, 1.0, 1.0]
    n, d = 3, 25 * 8192 + 77
    def make(gen, t):
        return scales[t] * torch.randn(n, d, generator=gen, device="cuda")
    _pair_run(n, d, [0, 6000, d], TOPK, 0.01, make, steps=len(scales), check_e_every=2)


def test_topk_candidate_path_with_heavily_duplicated_values():
    # a tiny alphabet: thousands of candidates share the threshold key, which neither the candidate
    # list's threshold bin nor a plain radix pass can separate without the index order
    n, d = 2, 30 * 8192
    def make(gen, t):
        return torch.randint(-20, 21, (n, d), generator=gen, device="cuda").float()
    _pair_run(n, d, [0, d], TOPK, 0.01, make, steps=6, check_e_every=2)


def test_topk_long_list_with_thousands_of_candidates_in_the_threshold_bin():
    # whole-vector selection over a long list whose threshold bin holds more candidates than shared
    # memory can rank pair by pair: (a) thousands of exact duplicates of the threshold value, told apart
    # by index only; (b) a very large k, where the bin's candidates differ in their low key bits
    n, d = 2, 320 * 8192
    def dup(gen, t):
        return torch.randint(-400, 401, (n, d), generator=gen, device="cuda").float()
    _pair_run(n, d, [0, d], TOPK, 0.01, dup, steps=5, check_e_every=2)
    d = 48 * (1 << 20) + 13
    p_steps = 4
    from parity import Pair
    gen = torch.Generator(device="cuda").manual_seed(11)
    p = Pair(n, d, [0, d], TOPK, 0.03)
    try:
        p.start(torch.zeros(d, device="cuda"))
        for t in range(p_steps):
            p.step(torch.randn(n, d, generator=gen, device="cuda"), check_e=(t == p_steps - 1))
        st = _status(p.gpu)
        assert st[0] == 0 and st[1] + st[2] == p_steps * n
        assert st[2] >= n, "the candidate path never decided a selection: %r" % (st,)
    finally:
        p.close()


def test_topk_layerwise_many_lists_single_cta_select():
    # many long candidate lists at once: the select runs one CTA per list instead of clusters
    n = 8
    offs = [0] + [int(x) for x in np.cumsum([120000] * 9)]
    d = offs[-1]
    _pair_run(n, d, offs, TOPK, 0.03, _randn(n, d), steps=5, check_e_every=2)


@pytest.mark.parametrize("n", [3, 5])
def test_topk_long_list_select_with_a_worker_count_that_is_not_a_power_of_two(n):
    # one block long enough that its candidate list is cut into slices (two kernels over the slices); with
    # n = 3 or 5 the mean over workers is an IEEE division, not a multiplication by 1 / n
    d = 1_500_003
    inexact = _pair_run(n, d, [0, d], TOPK, 0.01, _randn(n, d), steps=6, check_e_every=3)
    assert inexact.get("gbar", 0) == 0


@pytest.mark.parametrize("comp", [TOPK, BLOCKSIGN])
def test_layerwise_over_more_than_two_hundred_large_blocks(comp):
    # 230 blocks of 5,000 to 60,000 coordinates, n = 8: every block is tiled, the block list does not fit the
    # kernel-argument copy (the per-tile table in global memory is used), and the selection runs over
    # 8 x 230 candidate lists
    sizes = [5000 + (7919 * b) % 55001 for b in range(230)]
    offs = np.concatenate([[0], np.cumsum(sizes)]).tolist()
    n, d = 8, offs[-1]
    _pair_run(n, d, offs, comp, 0.01, _randn(n, d), steps=5, check_e_every=2)


@pytest.mark.parametrize("comp,ratio", [(TOPK, 0.02), (BLOCKSIGN, 1.0), (TOPK, 1.0)])
def test_learning_rate_schedule_matches_the_oracle(comp, ratio):
    # eta_t varies (Algorithm 2): divided by 10 in mid-run as in Section 5.1, then changed at every step;
    # both sides are given the same eta_t before the same step
    from parity import Pair
    n, d = 3, 3 * 8192 + 517
    gen = torch.Generator(device="cuda").manual_seed(21)
    p = Pair(n, d, [0, 5000, d], comp, ratio, lr=1e-2)
    schedule = [None, None, 1e-3, None, 1e-4, 3e-2, 0.0, 7e-3, 1e-3, 5e-4]
    try:
        p.start(0.1 * torch.randn(d, generator=gen, device="cuda"))
        for t, lr in enumerate(schedule):
            if lr is not None:
                p.set_lr(lr)
            before = p.theta_gpu.clone()
            p.step(torch.randn(n, d, generator=gen, device="cuda"), check_e=(t % 3 == 0))
            if lr == 0.0:
                assert torch.equal(p.theta_gpu, before)  # eta_t = 0: the parameters rest, the moments move on
    finally:
        p.close()


@pytest.mark.parametrize("comp,ratio", [(TOPK, 0.01), (TOPK, 1.0), (BLOCKSIGN, 1.0), (RANDK, 0.02)])
def test_the_average_is_stored_only_on_request_and_changes_nothing_else(comp, ratio):
    # gbar_t is an intermediate of the server's update: a new handle does not store it, asking for it is refused,
    # and every result of the step is the same bits with and without it
    n, d = 3, 5 * 8192 + 77   # the last bucket and the last float4 group are partial
    offs = [0, 4099, 30001, d]
    gen = torch.Generator(device="cuda").manual_seed(8)
    G = [torch.randn(n, d, generator=gen, device="cuda") for _ in range(4)]
    plain, rec = CompAMS(n, d, offs, comp, ratio), CompAMS(n, d, offs, comp, ratio, record_average=True)
    tp, tr = torch.zeros(d, device="cuda"), torch.zeros(d, device="cuda")
    for t, g in enumerate(G):
        plain.step(g, tp)
        rec.step(g, tr)
        if t == 1:
            with pytest.raises(CompAMSError):
                plain.buffer("gbar")
            rec.buffer("gbar")
    assert torch.equal(tp.view(torch.int32), tr.view(torch.int32))
    for name in ("E", "m", "v", "vhat"):
        assert torch.equal(plain.buffer(name).view(torch.int32), rec.buffer(name).view(torch.int32)), name
    # switched on later, the next step stores it; it equals the recorded handle's
    plain.record_average(True)
    g = torch.randn(n, d, generator=gen, device="cuda")
    plain.step(g, tp)
    rec.step(g, tr)
    assert torch.equal(plain.buffer("gbar").view(torch.int32), rec.buffer("gbar").view(torch.int32))
    assert plain.check_status() == 0 and rec.check_status() == 0
    plain.close()
    rec.close()


def test_calls_out_of_order_are_rejected():
    # compress opens an iteration and apply closes it: in between the residual is not final, so the
    # state cannot be read or replaced, and neither call may come twice in a row
    n, d = 2, 3 * 8192
    for comp, ratio in ((TOPK, 0.01), (BLOCKSIGN, 1.0)):
        opt = CompAMS(n, d, [0, d], comp, ratio)
        theta = torch.zeros(d, device="cuda")
        G = torch.randn(n, d, device="cuda")
        with pytest.raises(CompAMSError):
            opt.apply(theta)                  # nothing compressed yet
        opt.compress(G)
        for call in (lambda: opt.compress(G), lambda: opt.step(G, theta), lambda: opt.buffer("E"),
                     lambda: opt.get_state(), lambda: opt.set_state({"m": torch.zeros(d, device="cuda")})):
            with pytest.raises(CompAMSError):
                call()
        opt.buffer("m")                       # buffers that the open iteration does not touch stay readable
        opt.apply(theta)
        opt.step(G, theta)                    # and the handle goes on as usual
        assert opt.check_status() == 0
        ref = CompAMS(n, d, [0, d], comp, ratio)
        theta_ref = torch.zeros(d, device="cuda")
        ref.step(G, theta_ref)
        ref.step(G, theta_ref)
        assert torch.equal(theta, theta_ref) and torch.equal(opt.buffer("E"), ref.buffer("E"))
        opt.close()
        ref.close()


# ------------------------------------------------------------------ randomised shapes and value distributions

@pytest.mark.parametrize("seed", range(30))
def test_randomised_partitions_ratios_and_distributions(seed):
    # random block partitions (tiny, small and tiled blocks mixed), worker counts, keep ratios and gradient
    # distributions that change from step to step - continuous, heavy-tailed, quantised to a few levels (ties at
    # the threshold, kept and cut), exact zeros, scale jumps - for the three compressors, every step against the
    # oracle; reading E on some steps only exercises the deferred residual on the others
    rng = np.random.default_rng(1000 + seed)
    n = int(rng.choice([1, 2, 3, 5, 8]))
    sizes = []
    for _ in range(int(rng.integers(1, 9))):
        kind = rng.integers(0, 4)
        sizes.append(int(rng.integers(1, 40)) if kind == 0 else int(rng.integers(40, 4097)) if kind == 1
                     else int(rng.integers(4097, 30000)) if kind == 2 else int(rng.integers(30000, 120000)))
    offs = np.concatenate([[0], np.cumsum(sizes)]).tolist()
    d = offs[-1]
    comp = [TOPK, BLOCKSIGN, RANDK][seed % 3]
    ratio = float(rng.choice([0.001, 0.01, 0.05, 0.3]))
    kinds = rng.integers(0, 5, size=8)
    scales = 10.0 ** rng.integers(-3, 3, size=8)

    def make(gen, t):
        kind, sc = int(kinds[t]), float(scales[t]) if t % 3 == 2 else 1.0
        if kind == 0:
            g = torch.randn(n, d, generator=gen, device="cuda")
        elif kind == 1:
            z = torch.randn(2, n, d, generator=gen, device="cuda")
            g = z[0] / z[1].abs().clamp_min(1e-3)                      # heavy tails
        elif kind == 2:
            g = torch.randint(-3, 4, (n, d), generator=gen, device="cuda").float()   # seven levels: ties everywhere
        elif kind == 3:
            g = torch.randn(n, d, generator=gen, device="cuda")
            g[torch.rand(n, d, generator=gen, device="cuda") < 0.5] = 0.0  # half exact zeros
        else:
            g = torch.randint(-40, 41, (n, d), generator=gen, device="cuda").float() * 0.25
        return g * sc

    _pair_run(n, d, offs, comp, ratio, make, steps=8, check_e_every=3)


# ------------------------------------------------------------------ Random-k

@pytest.mark.parametrize("n", [1, 3])
@pytest.mark.parametrize("ratio", [0.01, 0.3, 1.0])
def test_randk_ragged_blocks(n, ratio):
    d = RAGGED[-1]
    _pair_run(n, d, RAGGED, RANDK, ratio, _randn(n, d), steps=5)


@pytest.mark.parametrize("d", [1, 2, 5, 33, 4097, 8193, 3 * 8192 + 2])
def test_randk_single_block_sizes(d):
    _pair_run(2, d, [0, d], RANDK, 0.1, _randn(2, d), steps=3)


def test_randk_resnet18_shapes_layerwise_and_whole_vector():
    # large enough that the step is overlapped (groups of workers, messages delivered behind the sweeps)
    w = W.config2("cuda")
    theta = w.start()
    from parity import Pair
    for offs, ratio in ((w.block_offsets, 0.01), (np.array([0, w.d]), 0.001)):
        p = Pair(8, w.d, offs, RANDK, ratio, seed=5)
        try:
            p.start(theta)
            for t in range(4):
                p.step(w.grads()[:8].contiguous(), check_e=(t % 2 == 1))
        finally:
            p.close()


def _long_row_offsets():
    # rows of more than 2^21 coordinates; the first 2^16 are 8192 blocks of 8 coordinates, each keeping one (most
    # CTAs of the emit kernel then hold many blocks' first slots), then blocks of very different lengths
    offs = list(range(0, 65536 + 1, 8))
    for step in (100000, 31, 700001, 65536, 1234567, 5):
        offs.append(offs[-1] + step)
    return offs


@pytest.mark.parametrize("n", [1, 3])
def test_randk_long_rows_many_tiny_blocks_then_large_ones(n):
    offs = _long_row_offsets()
    d = offs[-1]
    assert d >= 1 << 21
    _pair_run(n, d, offs, RANDK, 0.01, _randn(n, d), steps=4)


def test_randk_long_row_single_block_many_steps():
    d = (1 << 21) + 4099
    _pair_run(2, d, [0, d], RANDK, 0.02, _randn(2, d), steps=7, check_e_every=3)


def test_randk_sets_follow_seed_and_iteration_count():
    n, d = 2, 50000
    gen = torch.Generator(device="cuda").manual_seed(3)
    G = [torch.randn(n, d, generator=gen, device="cuda") for _ in range(3)]

    def run(seed, start):
        opt = CompAMS(n, d, [0, 20000, d], RANDK, 0.01)
        opt.set_seed(seed, start)
        theta = torch.zeros(d, device="cuda")
        sets = []
        for g in G:
            opt.step(g, theta)
            sets.append(torch.sort(opt.buffer("topk_idx"), dim=1).values.clone())
        opt.close()
        return sets

    a, b, c, late = run(1, 0), run(1, 0), run(2, 0), run(1, 1)
    assert all(torch.equal(x, y) for x, y in zip(a, b))
    assert not torch.equal(a[0], c[0])
    assert torch.equal(a[1], late[0]) and torch.equal(a[2], late[1])  # iteration t + 1 of one run = iteration t of a run started one later


# ------------------------------------------------------------------ streams

@pytest.mark.parametrize("comp,ratio", [(TOPK, 0.01), (BLOCKSIGN, 1.0), (RANDK, 0.01), (TOPK, 1.0)])
def test_steps_on_a_side_stream_match_the_default_stream(comp, ratio):
    # everything a step enqueues - programmatic dependents, the cooperative dense-pass kernel, the host-buffer
    # copies - goes to the handle's stream: a handle on a side stream, fed by producers on that stream, must give
    # the bits of a handle on the default stream; moving a handle to another stream (ordered by an event) too
    n, d = 3, 6 * 8192 + 321
    offs = [0, 3000, 30000, d]
    gen = torch.Generator(device="cuda").manual_seed(12)
    G = [torch.randn(n, d, generator=gen, device="cuda") for _ in range(5)]
    ref = CompAMS(n, d, offs, comp, ratio, record_average=True)
    theta_ref = torch.zeros(d, device="cuda")
    for g in G:
        ref.step(g, theta_ref)
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    theta = torch.zeros(d, device="cuda")
    with torch.cuda.stream(s1):
        opt = CompAMS(n, d, offs, comp, ratio, stream=s1, record_average=True)
        for g in G[:3]:
            staged = g.clone()          # produced on s1, consumed by the step on s1
            opt.step(staged, theta)
        done = torch.cuda.Event()
        done.record(s1)
    s2.wait_event(done)
    opt.set_stream(s2)
    with torch.cuda.stream(s2):
        for g in G[3:]:
            opt.step(g.clone(), theta)
        e_side = opt.buffer("E").clone()
    s2.synchronize()
    assert opt.check_status() == 0
    assert torch.equal(theta, theta_ref)
    assert torch.equal(e_side, ref.buffer("E"))
    for name in ("m", "v", "vhat", "gbar"):
        assert torch.equal(opt.buffer(name), ref.buffer(name)), name
    opt.close()
    ref.close()


# ------------------------------------------------------------------ checkpoint / restore, traffic accounting

@pytest.mark.parametrize("comp,ratio", [(TOPK, 0.02), (BLOCKSIGN, 1.0), (TOPK, 1.0)])
def test_restored_state_continues_bit_identically(comp, ratio):
    n, d = 3, 5 * 8192 + 1234
    offs = [0, 3000, 20000, d]
    gen = torch.Generator(device="cuda").manual_seed(9)
    G = [torch.randn(n, d, generator=gen, device="cuda") for _ in range(6)]
    a = CompAMS(n, d, offs, comp, ratio)
    theta_a = torch.zeros(d, device="cuda")
    for g in G[:3]:
        a.step(g, theta_a)
    saved = {k: v.clone() for k, v in a.get_state().items()}
    theta_saved = theta_a.clone()
    for g in G[3:]:
        a.step(g, theta_a)
    # the saved e is what the residual update defines, not the library's deferred form of it
    b = CompAMS(n, d, offs, comp, ratio)
    b.set_state(saved)
    if not (comp == TOPK and ratio == 1.0):
        assert torch.equal(b.buffer("E"), saved["e"])
    else:
        assert not saved["e"].any()
    theta_b = theta_saved.clone()
    for g in G[3:]:
        b.step(g, theta_b)
    assert torch.equal(theta_a.view(torch.int32), theta_b.view(torch.int32))
    sa, sb = a.get_state(), b.get_state()
    for k in sa:
        assert torch.equal(sa[k].view(torch.int32), sb[k].view(torch.int32)), k
    assert a.check_status() == 0 and b.check_status() == 0
    a.close()
    b.close()


def test_get_state_matches_the_oracle_and_leaves_the_run_unchanged():
    from parity import Pair, close
    n, d = 2, 3 * 8192 + 17
    for comp, ratio in ((TOPK, 0.01), (BLOCKSIGN, 1.0)):
        gen = torch.Generator(device="cuda").manual_seed(3)
        p = Pair(n, d, [0, 5000, d], comp, ratio)
        try:
            p.start(torch.zeros(d, device="cuda"))
            for t in range(4):
                p.step(torch.randn(n, d, generator=gen, device="cuda"), check_e=False)
                st = p.gpu.get_state()   # every step: reading the state must not disturb the next one
                close(st["e"], p.cpu.buffer("E"), "e from get_state", t + 1)
                close(st["m"], p.cpu.buffer("m"), "m from get_state", t + 1)
                close(st["vhat"], p.cpu.buffer("vhat"), "vhat from get_state", t + 1)
        finally:
            p.close()


def test_bits_transmitted_follow_the_32_bit_accounting():
    n, d = 4, 100000
    offs = [0, 30000, d]
    g = torch.zeros(n, d, device="cuda")
    theta = torch.zeros(d, device="cuda")
    t = CompAMS(n, d, offs, TOPK, 0.01)
    for _ in range(3):
        t.step(g, theta)
    k = 300 + 700
    assert t.bits_transmitted() == {"full_precision": 3 * 32 * n * d, "payload": 3 * 32 * n * k,
                                    "topk_indices": 3 * 32 * n * k}
    t.close()
    s = CompAMS(n, d, offs, BLOCKSIGN)
    s.step(g, theta)
    s.step(g, theta)
    assert s.bits_transmitted() == {"full_precision": 2 * 32 * n * d, "payload": 2 * n * (d + 32 * 2), "topk_indices": 0}
    s.close()
    f = CompAMS(n, d, offs, TOPK, 1.0)
    f.step(g, theta)
    assert f.bits_transmitted() == {"full_precision": 32 * n * d, "payload": 32 * n * d, "topk_indices": 0}
    f.close()
