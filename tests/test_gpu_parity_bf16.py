"""GPU parity, bf16-operand tensor-core path (tcgen05 + TMA), through the C ABI.

The oracle runs in fp64 on the same inputs the GPU sees (data pool rounded to
bf16 once, fp32 initial parameters).  Tolerance: relative L2 of the stacked
parameters <= 2e-2 after one full averaging period from a synchronised state.
Because one period moves the parameters by only a few percent, the tests also
bound the relative L2 error of the *update* x^t - x^0, which a wrong or
missing gradient cannot pass.

bf16 rounding of the weights moves a hidden pre-activation by ~2^-9 of its
scale, so a fraction p ~ 1e-3 of the ReLU units sits close enough to zero to
switch on one side only; each such unit is a whole wrong entry of dZ and the
update error it causes is ~sqrt(p), a few percent.  Random-init runs therefore
use TOL_UPDATE; runs whose hidden biases are +-6 (every unit firmly on or off,
no switch possible) must meet the much tighter TOL_UPDATE_MARGIN.
"""
import numpy as np
import pytest

from oracle import prsgd_oracle as orc
from paper_1807_06629_b200 import synth
from helpers import make_ctx, make_inputs, oracle_run, rel_l2

pytestmark = pytest.mark.gpu

TOL_PERIOD = 2e-2
TOL_UPDATE = 1e-1
TOL_UPDATE_MARGIN = 1e-2


def with_margin(x0, dims):
    """Hidden biases alternate +6 / -6: half the units always fire, half never do."""
    x = x0.copy()
    off = 0
    for l in range(len(dims) - 1):
        off += dims[l] * dims[l + 1]
        if l < len(dims) - 2:
            x[off:off + dims[l + 1]] = np.where(np.arange(dims[l + 1]) % 2 == 0, 6.0, -6.0)
        off += dims[l + 1]
    return x


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch


def _w(name, N, dims, B, I=2, gamma=0.05, P=None, shift=0.5, seed=31):
    return synth.Workload(name, N, dims, B, gamma, I, 2 * I, 1, P if P else 4 * B, mean_shift=shift, seed=seed)


SMALL = [
    _w("tc-logistic", 2, (64, 10), 32),
    _w("tc-two-layer", 3, (128, 256, 10), 32),
    _w("tc-b16", 2, (64, 128, 64, 10), 16),
    _w("tc-b64", 2, (128, 128, 100), 64),
    _w("tc-ragged-tiles", 2, (192, 320, 100), 32),
    _w("tc-many-kblocks", 1, (1024, 128, 10), 32),
    _w("tc-deep", 2, (64,) * 7 + (10,), 32),
]


@pytest.mark.parametrize("w", SMALL, ids=[w.name for w in SMALL])
def test_every_gemm_is_tight_when_no_relu_can_switch(torch_cuda, w):
    X, Y, x0 = make_inputs(w)
    x0 = with_margin(x0, w.dims)
    p = make_ctx(w, X, Y, x0, I=0)
    x0s = np.tile(x0, (w.N, 1)).astype(np.float64)
    losses = {}
    want = oracle_run(w, X, Y, x0s, 0, 1, I=0, losses=losses)
    p.local_steps(1)
    got = p.get_params_stacked()
    assert np.allclose(p.get_losses(), [losses[(i, 1)] for i in range(w.N)], rtol=1e-2, atol=1e-3)
    off = 0
    for l in range(len(w.dims) - 1):                      # every layer's W and b on its own
        for cnt in (w.dims[l] * w.dims[l + 1], w.dims[l + 1]):
            g, t = got[:, off:off + cnt] - x0s[:, off:off + cnt], want[:, off:off + cnt] - x0s[:, off:off + cnt]
            assert np.linalg.norm(t) > 0
            # dZ is rounded to bf16 once per layer on its way down: allow the noise to grow with the depth below
            depth = len(w.dims) - 1 - l
            assert rel_l2(g, t) <= TOL_UPDATE_MARGIN * max(1.0, depth / 2), (l, cnt, rel_l2(g, t))
            off += cnt


@pytest.mark.parametrize("w", SMALL, ids=[w.name for w in SMALL])
def test_one_step_and_one_period(torch_cuda, w):
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    x0s = np.tile(x0, (w.N, 1)).astype(np.float64)
    # one iteration
    losses = {}
    want1 = oracle_run(w, X, Y, x0s, 0, 1, I=0, losses=losses)
    p.set_interval(0)
    p.local_steps(1)
    got1 = p.get_params_stacked()
    assert p.get_draws().tolist() == [orc.draw_block(w.seed, i, 1, w.n_blocks) for i in range(w.N)]
    gl, wl = p.get_losses(), np.array([losses[(i, 1)] for i in range(w.N)])
    assert np.allclose(gl, wl, rtol=2e-2, atol=2e-3), (gl, wl)
    assert rel_l2(got1 - x0s, want1 - x0s) <= TOL_UPDATE, rel_l2(got1 - x0s, want1 - x0s)
    assert rel_l2(got1, want1) <= TOL_PERIOD
    # one full period from the synchronised start
    p.set_params(x0)
    p.set_step(0)
    p.set_interval(w.I)
    p.local_steps(w.I)
    got = p.get_params_stacked()
    want = oracle_run(w, X, Y, x0s, 0, w.I)
    assert all(np.array_equal(got[i], got[0]) for i in range(w.N))
    assert rel_l2(got, want) <= TOL_PERIOD
    assert rel_l2(got - x0s, want - x0s) <= TOL_UPDATE, rel_l2(got - x0s, want - x0s)


def test_fused_average_equals_update_then_average_bit_for_bit(torch_cuda):
    from paper_1807_06629_b200 import binding
    for w in (SMALL[1], SMALL[4], _w("tc-n5", 5, (64, 128, 10), 32, I=3)):
        X, Y, x0 = make_inputs(w)
        outs = []
        for fused, tile in ((1, 0), (0, 0), (1, 64), (0, 64), (1, 128), (0, 128)):   # tile width changes no bit either
            p = make_ctx(w, X, Y, x0)
            p.set_option(binding.OPT_FUSED_AVERAGE, fused)
            p.set_option(binding.OPT_UPDATE_TILE, tile)
            p.local_steps(2 * w.I + 1)
            outs.append(p.get_params_stacked())
        for o in outs[1:]:
            assert np.array_equal(outs[0], o)


@pytest.mark.parametrize("avg_v", [False, True])
def test_fused_average_with_momentum_equals_update_then_average_bit_for_bit(torch_cuda, avg_v):
    """The momentum step inside the fused update + average (every worker's new buffer tile written back to its
    own row, or a second set of running sums when the buffers are averaged too) against the momentum update
    followed by the stand-alone average: identical parameters and momentum buffers, also with a worker mask
    (an inactive worker contributes its unchanged point and keeps its buffer) and replayed periods."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    for w in (SMALL[1], SMALL[4], _w("tc-n5", 5, (64, 128, 10), 32, I=3), _w("tc-mom-I1", 4, (192, 320, 100), 16, I=1)):
        X, Y, x0 = make_inputs(w)
        for mask in (None, [1 if i != 1 else 0 for i in range(w.N)]):
            outs = []
            for fused, graph in ((0, 0), (1, 0), (1, 1)):
                with torch.cuda.stream(torch.cuda.Stream()):
                    p = make_ctx(w, X, Y, x0)
                    p.enable_momentum(0.9, average_velocity=avg_v)
                    p.set_option(binding.OPT_FUSED_AVERAGE, fused)
                    p.set_option(binding.OPT_GRAPH, graph)
                    if mask is not None:
                        p.set_active(mask)
                    n0 = p.get_launch_count()
                    p.local_steps(3 * w.I + 1)
                    outs.append((p.get_params_stacked(), p.get_velocity_stacked(), p.get_launch_count() - n0))
                    torch.cuda.current_stream().synchronize()
                    p.close()
            for o in outs[1:]:
                assert np.array_equal(outs[0][0], o[0]), (w.name, mask)
                assert np.array_equal(outs[0][1], o[1]), (w.name, mask)
            if not avg_v:
                assert len({tuple(v) for v in outs[0][1][:, :8]}) > 1      # local buffers stay apart


def test_early_weight_loads_change_no_bit(torch_cuda):
    """Tiles requested ahead of a kernel's dependency wait (weights nobody is writing at that time) against
    the same run with every load after the wait: identical bits over several periods, direct and replayed."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    for w in (SMALL[1], SMALL[4], SMALL[6], _w("tc-n5", 5, (64, 128, 10), 32, I=3)):
        X, Y, x0 = make_inputs(w)
        outs = []
        for early, graph in ((1, 0), (0, 0), (1, 1), (0, 1)):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                p.set_option(binding.OPT_EARLY_LOADS, early)
                p.set_option(binding.OPT_GRAPH, graph)
                p.local_steps(3 * w.I + 1)
                outs.append((p.get_params_stacked(), p.get_losses()))
                torch.cuda.current_stream().synchronize()
        for o in outs[1:]:
            assert np.array_equal(outs[0][0], o[0]) and np.array_equal(outs[0][1], o[1])


def test_next_forward_folded_into_the_first_layers_update_changes_no_bit(torch_cuda):
    """The update of layer 1 also forms a_1 of the following iteration from its freshly stepped tiles (and leaves
    W_1's bf16 copy unwritten meanwhile) against the separate forward launch: identical parameters, losses and
    draws, direct and replayed, for both tile widths, ragged tiles and calls that end in the middle of a period;
    the bf16 copy of every layer equals bf16(master) whenever a call has returned."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    cases = (SMALL[1], SMALL[2], SMALL[3], SMALL[4], SMALL[5], SMALL[6], _w("tc-n5-I5", 5, (192, 128, 10), 32, I=5),
             _w("tc-wide-in", 3, (448, 256, 10), 16, I=4))
    for w in cases:
        X, Y, x0 = make_inputs(w)
        outs = []
        for nxt, graph, tile in ((0, 0, 0), (1, 0, 0), (1, 1, 0), (1, 0, 64), (1, 1, 128)):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                p.set_option(binding.OPT_NEXT_FORWARD, nxt)
                p.set_option(binding.OPT_GRAPH, graph)
                p.set_option(binding.OPT_UPDATE_TILE, tile)
                n0 = p.get_launch_count()
                p.local_steps(2)                       # ends inside a period
                p.local_steps(2 * w.I + 1)             # crosses two averages
                launches = p.get_launch_count() - n0
                p.sync()
                store = p.params.cpu().numpy().reshape(w.N, p.m_pad)
                shadow = p.shadow.view(torch.int16).cpu().numpy().view(np.uint16).reshape(w.N, p.m_pad)
                for l in range(len(w.dims) - 1):
                    a, n = p.layout.w_off[l], w.dims[l] * w.dims[l + 1]
                    assert np.array_equal(shadow[:, a:a + n], synth.bf16_bits(store[:, a:a + n])), (w.name, l)
                outs.append((p.get_params_stacked(), p.get_losses(), p.get_draws().tolist(), launches))
                torch.cuda.current_stream().synchronize()
        for o in outs[1:]:
            assert np.array_equal(outs[0][0], o[0]), w.name
            assert np.array_equal(outs[0][1], o[1]) and outs[0][2] == o[2]
        assert outs[1][3] < outs[0][3]                 # forward launches were saved


def test_dx_folded_into_the_update_changes_no_bit(torch_cuda):
    """dZ of the layer below formed inside the update launch (from the bf16 values the weights had before the
    step) against the separate dX launch: identical parameters, losses and bias steps over several periods,
    direct and replayed, with and without the folded next forward."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    cases = (SMALL[1], SMALL[2], SMALL[3], SMALL[4], SMALL[6], _w("tc-n5-I5", 5, (192, 128, 10), 32, I=5),
             _w("tc-wide-hidden", 3, (64, 448, 320, 10), 16, I=4))
    for w in cases:
        X, Y, x0 = make_inputs(w)
        outs = []
        # dxu 2 = every layer, whatever its size; the tile width only concerns layer 1's update here
        for dxu, nxt, graph, tile in ((0, 0, 0, 0), (2, 0, 0, 64), (2, 1, 0, 128), (2, 1, 1, 64), (2, 0, 1, 128)):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                p.set_option(binding.OPT_DX_IN_UPDATE, dxu)
                p.set_option(binding.OPT_NEXT_FORWARD, nxt)
                p.set_option(binding.OPT_GRAPH, graph)
                p.set_option(binding.OPT_UPDATE_TILE, tile)
                n0 = p.get_launch_count()
                p.local_steps(2)
                p.local_steps(2 * w.I + 1)
                launches = p.get_launch_count() - n0
                p.sync()
                store = p.params.cpu().numpy().reshape(w.N, p.m_pad)
                shadow = p.shadow.view(torch.int16).cpu().numpy().view(np.uint16).reshape(w.N, p.m_pad)
                for l in range(len(w.dims) - 1):          # the bf16 copy follows the master through either store path
                    a, n = p.layout.w_off[l], w.dims[l] * w.dims[l + 1]
                    assert np.array_equal(shadow[:, a:a + n], synth.bf16_bits(store[:, a:a + n])), (w.name, l, tile)
                outs.append((p.get_params_stacked(), p.get_losses(), launches))
                torch.cuda.current_stream().synchronize()
        for o in outs[1:]:
            assert np.array_equal(outs[0][0], o[0]), w.name
            assert np.array_equal(outs[0][1], o[1])
        assert outs[1][2] < outs[0][2]


HEAD_CASES = [
    _w("tc-head-cl2", 3, (128, 256, 10), 32, I=3),
    _w("tc-head-cl1-c100", 2, (128, 128, 100), 64),
    _w("tc-head-cl8-b64", 3, (192, 1024, 10), 64, I=3),
    _w("tc-head-cl4-c100", 5, (64, 512, 100), 32, I=3),
    _w("tc-head-cl8-b16-c128", 2, (64, 128, 1024, 128), 16),
    _w("tc-head-cl8-c100", 4, (128, 1024, 100), 32),
]


@pytest.mark.parametrize("w", HEAD_CASES, ids=[w.name for w in HEAD_CASES])
def test_class_layer_in_one_launch_of_clusters(torch_cuda, w):
    """The class layer as one launch (a cluster per worker: logits summed slice by slice through the cluster's
    shared memory, softmax-CE gradient, step of W_L and b_L, dZ of the layer below) against the forward GEMM and
    the update launch it replaces.  The logits are summed in another order, so the two agree to rounding (a bf16
    entry of dZ_L may fall on the other side of a rounding boundary), not bit for bit; the launch itself is
    deterministic (direct, replayed and with a worker mask), keeps every bf16 copy equal to bf16(master), leaves
    an inactive worker alone, saves one launch per iteration and meets the oracle's per-layer bounds."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    X, Y, x0 = make_inputs(w)
    x0s = np.tile(x0, (w.N, 1))
    T = 2 * w.I + 2
    runs = {}
    for head, graph in ((0, 0), (1, 0), (1, 1)):
        with torch.cuda.stream(torch.cuda.Stream()):
            p = make_ctx(w, X, Y, x0)
            p.set_option(binding.OPT_HEAD_KERNEL, head)
            p.set_option(binding.OPT_HEAD_FORWARD, 0)        # (the forward GEMM below it stays a launch: it has a test of its own)
            p.set_option(binding.OPT_GRAPH, graph)
            n0 = p.get_launch_count()
            p.local_steps(1)
            first, first_losses = p.get_params_stacked(), p.get_losses()
            p.local_steps(T - 1)
            launches = p.get_launch_count() - n0
            p.sync()
            store = p.params.cpu().numpy().reshape(w.N, p.m_pad)
            shadow = p.shadow.view(torch.int16).cpu().numpy().view(np.uint16).reshape(w.N, p.m_pad)
            for l in range(len(w.dims) - 1):
                a, n = p.layout.w_off[l], w.dims[l] * w.dims[l + 1]
                assert np.array_equal(shadow[:, a:a + n], synth.bf16_bits(store[:, a:a + n])), (w.name, l, head)
            runs[(head, graph)] = (first, p.get_params_stacked(), p.get_losses(), p.get_draws().tolist(), launches, first_losses)
            torch.cuda.current_stream().synchronize()
            p.close()
    off, on, replay = runs[(0, 0)], runs[(1, 0)], runs[(1, 1)]
    assert np.array_equal(on[1], replay[1]) and np.array_equal(on[2], replay[2]) and on[3] == replay[3]
    assert on[4] == off[4] - T                             # one launch fewer per iteration
    assert on[3] == off[3]
    assert np.allclose(on[5], off[5], rtol=1e-4, atol=1e-5)        # the first iteration starts from the same point
    assert np.allclose(on[2], off[2], rtol=5e-3, atol=1e-4)        # later ones from points a rounding apart
    assert rel_l2(on[0] - x0s, off[0] - x0s) <= 5e-3, rel_l2(on[0] - x0s, off[0] - x0s)
    assert rel_l2(on[1] - x0s, off[1] - x0s) <= 2e-2, rel_l2(on[1] - x0s, off[1] - x0s)
    # against the oracle, every segment on its own, with no ReLU able to switch: the per-layer bound, or (for the
    # shapes whose bf16 noise exceeds it with the separate launches too) no worse than the separate launches
    xm = with_margin(x0, w.dims)
    xms = np.tile(xm, (w.N, 1)).astype(np.float64)
    losses = {}
    want = oracle_run(w, X, Y, xms, 0, 1, I=0, losses=losses)
    errs = {}
    for head in (0, 1):
        p = make_ctx(w, X, Y, xm, I=0)
        p.set_option(binding.OPT_HEAD_KERNEL, head)
        p.local_steps(1)
        got = p.get_params_stacked()
        assert np.allclose(p.get_losses(), [losses[(i, 1)] for i in range(w.N)], rtol=1e-2, atol=1e-3)
        errs[head] = [rel_l2(got[:, lo:hi] - xms[:, lo:hi], want[:, lo:hi] - xms[:, lo:hi]) for _, lo, hi in _segments(w.dims)]
        p.close()
    for l, e in enumerate(errs[1]):
        depth = len(w.dims) - 1 - l // 2
        assert e <= max(TOL_UPDATE_MARGIN * max(1.0, depth / 2), 1.05 * errs[0][l]), (l, e, errs[0][l])
    # a worker mask: the inactive worker's row stays where it was, the others do what they do without a mask
    mask = [1 if i != 1 else 0 for i in range(w.N)]
    outs = []
    for graph in (0, 1):
        with torch.cuda.stream(torch.cuda.Stream()):
            p = make_ctx(w, X, Y, x0, I=0)
            p.set_option(binding.OPT_GRAPH, graph)
            p.set_active(mask)
            p.local_steps(3)
            outs.append(p.get_params_stacked())
            torch.cuda.current_stream().synchronize()
            p.close()
    assert np.array_equal(outs[0], outs[1])
    assert np.array_equal(outs[0][1], x0s[1])
    p = make_ctx(w, X, Y, x0, I=0)
    p.local_steps(3)
    free = p.get_params_stacked()
    p.close()
    keep = [i for i in range(w.N) if mask[i]]
    assert np.array_equal(outs[0][keep], free[keep])


def test_stage_layouts_of_the_update_dx_kernel_change_no_bit(torch_cuda):
    """64-wide update + dX with one shared pair of bf16 tiles behind a deeper pipeline against a pair per stage:
    identical parameters, losses and bf16 copies for B = 16, 32, 64, single- and multi-tile column blocks, ragged
    widths, a worker mask, direct and replayed."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    cases = (SMALL[1], SMALL[2], SMALL[3], SMALL[4], SMALL[6], _w("tc-pair-b64", 3, (128, 320, 192, 10), 64, I=3),
             _w("tc-pair-wide", 3, (64, 448, 320, 10), 16, I=4))
    for w in cases:
        X, Y, x0 = make_inputs(w)
        for mask in (None, [1 if i != 1 else 0 for i in range(w.N)]):
            outs = []
            for shared, graph in ((0, 0), (1, 0), (1, 1)):
                with torch.cuda.stream(torch.cuda.Stream()):
                    p = make_ctx(w, X, Y, x0)
                    p.set_option(binding.OPT_DX_IN_UPDATE, 2)          # every layer >= 2 takes the folded kernel
                    p.set_option(binding.OPT_UPDATE_TILE, 64)
                    p.set_option(binding.OPT_DX_SHARED_PAIR, shared)
                    p.set_option(binding.OPT_GRAPH, graph)
                    if mask is not None:
                        p.set_active(mask)
                    p.local_steps(2)
                    p.local_steps(2 * w.I + 1)
                    p.sync()
                    outs.append((p.get_params_stacked(), p.get_losses(), p.shadow.view(torch.int16).cpu().numpy().copy()))
                    torch.cuda.current_stream().synchronize()
                    p.close()
            keep = [i for i in range(w.N) if mask is None or mask[i]]
            for o in outs[1:]:
                assert np.array_equal(outs[0][0], o[0]), (w.name, mask)
                assert np.array_equal(outs[0][1][keep], o[1][keep]) and np.array_equal(outs[0][2], o[2])


@pytest.mark.parametrize("avg_v", [False, True])
def test_folded_kernels_with_momentum_change_no_bit(torch_cuda, avg_v):
    """The momentum step inside the two folded update kernels (dZ of the layer below, next forward of layer 1)
    against the separate launches: identical parameters, momentum buffers and losses across averages."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    for w in (SMALL[1], SMALL[3], SMALL[4], SMALL[6], _w("tc-wide-hidden", 3, (64, 448, 320, 10), 16, I=4)):
        X, Y, x0 = make_inputs(w)
        outs = []
        for dxu, nxt, graph in ((0, 0, 0), (2, 1, 0), (2, 0, 1), (0, 1, 1)):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                p.enable_momentum(0.9, average_velocity=avg_v)
                p.set_option(binding.OPT_DX_IN_UPDATE, dxu)
                p.set_option(binding.OPT_NEXT_FORWARD, nxt)
                p.set_option(binding.OPT_GRAPH, graph)
                p.local_steps(2)
                p.local_steps(2 * w.I + 1)
                outs.append((p.get_params_stacked(), p.get_velocity_stacked(), p.get_losses()))
                torch.cuda.current_stream().synchronize()
        for o in outs[1:]:
            assert np.array_equal(outs[0][0], o[0]), w.name
            assert np.array_equal(outs[0][1], o[1]), w.name
            assert np.array_equal(outs[0][2], o[2])


def test_folded_kernels_with_a_worker_mask_change_no_bit(torch_cuda):
    """Algorithm 3's worker mask inside the folded update kernels (an inactive worker's blocks are skipped by
    every role of the kernel) against the separate launches, several iterations per call so that the folded
    next forward runs too; the inactive workers' rows must not move between averages."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    for w in (_w("tc-mask5", 5, (192, 128, 10), 32, I=3), _w("tc-mask-deep", 4, (64, 448, 320, 10), 16, I=4), SMALL[3]):
        X, Y, x0 = make_inputs(w)
        mask = [1 if i % 2 == 0 else 0 for i in range(w.N)]
        outs = []
        for dxu, nxt, graph, tile in ((0, 0, 0, 0), (2, 1, 0, 64), (2, 1, 1, 128), (2, 0, 0, 128)):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                p.set_option(binding.OPT_DX_IN_UPDATE, dxu)
                p.set_option(binding.OPT_NEXT_FORWARD, nxt)
                p.set_option(binding.OPT_GRAPH, graph)
                p.set_option(binding.OPT_UPDATE_TILE, tile)
                p.set_active(mask)
                p.local_steps(w.I - 1)                     # stops just before the first average
                before = p.get_params_stacked()
                p.local_steps(2 * w.I + 2)
                outs.append((before, p.get_params_stacked(), p.get_losses()))
                torch.cuda.current_stream().synchronize()
        x0s = np.tile(x0, (w.N, 1))
        for i in range(w.N):
            if not mask[i]:
                assert np.array_equal(outs[0][0][i], x0s[i])           # an inactive worker has not moved
            else:
                assert not np.array_equal(outs[0][0][i], x0s[i])
        for o in outs[1:]:
            assert np.array_equal(outs[0][0], o[0]) and np.array_equal(outs[0][1], o[1]), w.name
            active = [i for i in range(w.N) if mask[i]]
            assert np.array_equal(outs[0][2][active], o[2][active])


def test_forward_chain_in_one_launch_changes_no_bit(torch_cuda):
    """The forward GEMMs of all layers as one launch whose items wait per (layer, worker) for the activations
    below them, against one launch per layer: identical parameters, losses and draws over several periods,
    direct and replayed, with a worker mask, with momentum, for deep and ragged nets; fewer launches."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    cases = (SMALL[1], SMALL[2], SMALL[3], SMALL[4], SMALL[6], _w("tc-chain-n7", 7, (192, 128, 256, 10), 32, I=3),
             _w("tc-chain-200", 2, (64, 128, 200), 32), _w("tc-chain-wide", 3, (64, 448, 320, 10), 16, I=4))
    for w in cases:
        X, Y, x0 = make_inputs(w)
        for variant in ("plain", "mask", "momentum"):
            outs = []
            for chain, graph in ((0, 0), (1, 0), (1, 1)):
                with torch.cuda.stream(torch.cuda.Stream()):
                    p = make_ctx(w, X, Y, x0)
                    p.set_option(binding.OPT_FORWARD_CHAIN, chain)
                    p.set_option(binding.OPT_GRAPH, graph)
                    if variant == "mask":
                        p.set_active([1 if i % 2 == 0 else 0 for i in range(w.N)])
                    if variant == "momentum":
                        p.enable_momentum(0.9)
                    n0 = p.get_launch_count()
                    p.local_steps(2)
                    p.local_steps(3 * w.I + 1)
                    outs.append((p.get_params_stacked(), p.get_losses(), p.get_draws().tolist(), p.get_launch_count() - n0))
                    torch.cuda.current_stream().synchronize()
                    p.close()
            keep = [i for i in range(w.N) if variant != "mask" or i % 2 == 0]
            for o in outs[1:]:
                assert np.array_equal(outs[0][0], o[0]), (w.name, variant)
                assert np.array_equal(outs[0][1][keep], o[1][keep])
                assert [outs[0][2][i] for i in keep] == [o[2][i] for i in keep]
            # (with the class layer a launch of its own kind the chain ends below it: a two-layer net then has
            # nothing to chain and a longer one chains only while layer 1's forward is not folded away)
            head = variant != "momentum" and len(w.dims) > 2 and w.dims[-1] <= 128 and w.dims[-2] in (128, 256, 512, 1024)
            assert outs[1][3] < outs[0][3] or (head and outs[1][3] == outs[0][3] and len(w.dims) == 3)


def test_worker_groups_on_their_own_streams_change_no_bit(torch_cuda):
    """The plain iterations of a period as 2, 3 or 4 independent launch chains (one per group of workers, each on
    a stream of the library's own, forked from and joined to the context's stream) against one chain for all
    workers: identical parameters, losses, draws and momentum buffers over several periods, direct and replayed,
    with calls that end in the middle of a period and group sizes that do not divide N."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    cases = (_w("tc-groups-n8", 8, (128, 256, 10), 32, I=4), _w("tc-groups-n7", 7, (192, 128, 256, 10), 32, I=5),
             _w("tc-groups-wide", 9, (64, 448, 320, 10), 16, I=3), _w("tc-groups-b64", 8, (128, 128, 100), 64, I=4))
    for w in cases:
        X, Y, x0 = make_inputs(w)
        for mu in (None, 0.9):
            outs = []
            for groups, graph in ((1, 0), (2, 0), (2, 1), (3, 1), (4, 0)):
                with torch.cuda.stream(torch.cuda.Stream()):
                    p = make_ctx(w, X, Y, x0)
                    p.set_option(binding.OPT_WORKER_GROUPS, groups)
                    p.set_option(binding.OPT_GRAPH, graph)
                    if mu is not None:
                        p.enable_momentum(mu)
                    p.local_steps(2)                       # ends inside a period
                    p.local_steps(3 * w.I + 2)             # crosses three averages, ends inside a period again
                    p.local_steps(w.I - 1)
                    outs.append((p.get_params_stacked(), p.get_losses(), p.get_draws().tolist(), p.get_step(),
                                 p.get_velocity_stacked() if mu is not None else None))
                    torch.cuda.current_stream().synchronize()
                    p.close()
            for o in outs[1:]:
                assert np.array_equal(outs[0][0], o[0]), (w.name, mu)
                assert np.array_equal(outs[0][1], o[1]) and outs[0][2] == o[2] and outs[0][3] == o[3]
                if mu is not None:
                    assert np.array_equal(outs[0][4], o[4])
    with pytest.raises(binding.PRSGDError):
        make_ctx(cases[0], *make_inputs(cases[0])).set_option(binding.OPT_WORKER_GROUPS, 5)


def test_reading_the_common_restart_point_once_changes_no_bit(torch_cuda):
    """After a node average all N rows hold the same bits, so the following iteration's forward, dX and fused
    update + average launches read worker 0's weights for every worker (PRSGD_OPT_SHARED_RESTART).  Against
    the same runs with the option off: identical parameters, losses and momentum buffers for I = 1 (every
    iteration follows an average), I = 3, replayed periods, a start from N different points (nothing may be
    shared before the first average), momentum, and the two halves of the multi-GPU average."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    cases = [(_w("tc-share-I1", 5, (192, 320, 100), 32, I=1), None), (_w("tc-share-I3", 4, (64, 448, 320, 10), 16, I=3), None),
             (SMALL[3].with_(I=1), None), (_w("tc-share-mom", 3, (128, 256, 10), 32, I=1), 0.9), (SMALL[6], None)]
    for w, mu in cases:
        X, Y, x0 = make_inputs(w)
        rng = np.random.default_rng(1)
        apart = np.tile(x0, (w.N, 1)) * (1.0 + 0.01 * rng.standard_normal((w.N, 1))).astype(np.float32)
        outs = []
        for share, graph, start in ((0, 0, "same"), (1, 0, "same"), (1, 1, "same"), (0, 0, "apart"), (1, 1, "apart")):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                p.set_option(binding.OPT_SHARED_RESTART, share)
                p.set_option(binding.OPT_COMMON_POINT, 0)      # (one GEMM over all workers rounds differently: its own test)
                p.set_option(binding.OPT_GRAPH, graph)
                if mu is not None:
                    p.enable_momentum(mu)
                if start == "apart":
                    p.set_params_stacked(apart)
                p.local_steps(2 * w.I + 1)
                p.local_steps(3 * w.I)
                # the multi-GPU halves leave N equal rows too: the iteration after them shares its reads
                row = p.new_row()
                half = (p.m_pad // 8) * 4
                p.partial_sum(row)
                p.assign_rows(row, float(w.N), 0, half)
                p.assign_rows(row, float(w.N), half, p.m_pad - half)
                p.local_steps(2)
                outs.append((start, p.get_params_stacked(), p.get_losses(),
                             p.get_velocity_stacked() if mu is not None else None))
                torch.cuda.current_stream().synchronize()
                p.close()
        for start in ("same", "apart"):
            grp = [o for o in outs if o[0] == start]
            for o in grp[1:]:
                assert np.array_equal(grp[0][1], o[1]), (w.name, start)
                assert np.array_equal(grp[0][2], o[2])
                if mu is not None:
                    assert np.array_equal(grp[0][3], o[3])


def test_small_weight_segments_averaged_by_the_bias_average_launch_change_no_bit(torch_cuda):
    """On a fused averaging iteration the weight segments too small for the fused update + average (every layer
    of these small nets; the class layer of the large ones) are averaged by the launch that averages the bias
    segments instead of by launches of their own: identical parameters, bf16 copies and momentum buffers over
    several periods, direct and replayed, with and without the cluster launch, also in the row-sum form; fewer
    launches."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    cases = ((SMALL[1], None), (SMALL[4], None), (_w("tc-merge-I1", 3, (640, 1024, 10), 32, I=1), None),
             (_w("tc-merge-mom", 4, (128, 256, 10), 32, I=2), 0.9))
    for w, mu in cases:
        X, Y, x0 = make_inputs(w)
        outs = []
        for merged, graph, head in ((0, 0, 1), (1, 0, 1), (1, 1, 1), (0, 0, 0), (1, 0, 0)):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                if mu is not None:
                    p.enable_momentum(mu, average_velocity=True)
                p.set_option(binding.OPT_MERGED_SMALL_AVERAGE, merged)
                p.set_option(binding.OPT_GRAPH, graph)
                p.set_option(binding.OPT_HEAD_KERNEL, head)
                n0 = p.get_launch_count()
                p.local_steps(3 * w.I + 1)
                launches = p.get_launch_count() - n0
                p.sync()
                shadow = p.shadow.view(torch.int16).cpu().numpy().copy()
                p.set_interval(0)
                if mu is None:
                    p.local_steps_sum(1)
                outs.append((head, p.get_params_stacked(), shadow, p.get_velocity_stacked() if mu is not None else None, launches, graph))
                torch.cuda.current_stream().synchronize()
                p.close()
        for head in (1, 0):
            grp = [o for o in outs if o[0] == head]
            for o in grp[1:]:
                assert np.array_equal(grp[0][1], o[1]) and np.array_equal(grp[0][2], o[2]), (w.name, head)
                if mu is not None:
                    assert np.array_equal(grp[0][3], o[3])
            assert grp[1][4] < grp[0][4]


TILED_CASES = [
    _w("tc-tiled-two-layer", 3, (128, 256, 10), 32, I=2),
    _w("tc-tiled-mixed", 2, (64, 128, 64, 10), 16, I=3),
    _w("tc-tiled-odd-width", 3, (448, 256, 10), 16, I=2),
    _w("tc-tiled-deep", 2, (192, 384, 256, 128, 100), 32, I=2),
    _w("tc-tiled-I1", 3, (640, 1024, 10), 32, I=1),
    _w("tc-tiled-b64", 2, (128, 1024, 256, 10), 64, I=2),
]


@pytest.mark.parametrize("w", TILED_CASES, ids=[w.name for w in TILED_CASES])
def test_tile_major_weight_segments_change_no_bit(torch_cuda, w):
    """Hidden layers' weight segments stored as 128 x 64 tiles (PRSGD_OPT_TILED_WEIGHTS) against row-major
    segments: the same arithmetic on the same numbers, so every result that crosses the interface -- stacked
    parameters, one worker's parameters, the node average (to the host, to the device, asynchronously), losses,
    momentum buffers -- is identical, for both tile widths, the folded and the separate launches, momentum, a
    worker mask and replayed periods; switching the order in the middle of a run changes nothing either; the bf16
    copy equals bf16(master) element for element in whichever order the rows are."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    X, Y, x0 = make_inputs(w)
    T = 2 * w.I + 1
    variants = [("plain", {}), ("tile64", {binding.OPT_UPDATE_TILE: 64}), ("tile128", {binding.OPT_UPDATE_TILE: 128}),
                ("separate", {binding.OPT_DX_IN_UPDATE: 0, binding.OPT_NEXT_FORWARD: 0}), ("fold-all", {binding.OPT_DX_IN_UPDATE: 2}),
                ("momentum", {}), ("mask", {}), ("head-forward", {binding.OPT_HEAD_FORWARD: 1}), ("chain", {binding.OPT_FORWARD_CHAIN: 1})]
    for name, opts in variants:
        outs = []
        for tiled, graph, switch in ((0, 0, False), (1, 0, False), (1, 1, False), (0, 0, True)):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                p.set_option(binding.OPT_TILED_WEIGHTS, tiled)
                p.set_option(binding.OPT_GRAPH, graph)
                for k, v in opts.items():
                    p.set_option(k, v)
                if name == "momentum":
                    p.enable_momentum(0.9, average_velocity=True)
                if name == "mask":
                    p.set_active([1 if i != 1 else 0 for i in range(w.N)])
                p.local_steps(2)
                if switch:
                    p.set_option(binding.OPT_TILED_WEIGHTS, 1)          # re-orders the store (and the momentum buffers) in place
                p.local_steps(T - 2)
                p.sync()
                store = p.params.cpu().numpy().reshape(w.N, p.m_pad)
                shadow = p.shadow.view(torch.int16).cpu().numpy().view(np.uint16).reshape(w.N, p.m_pad)
                for l in range(len(w.dims) - 1):
                    a, n = p.layout.w_off[l], w.dims[l] * w.dims[l + 1]
                    assert np.array_equal(shadow[:, a:a + n], synth.bf16_bits(store[:, a:a + n])), (w.name, name, l)
                avg_dev = torch.empty(p.m, dtype=torch.float32, device="cuda")
                p.get_average(avg_dev)
                pinned = torch.empty(p.m, dtype=torch.float32).pin_memory()
                side = torch.cuda.Stream()
                p.get_average_async(pinned, side)
                side.synchronize()
                outs.append((p.get_params_stacked(), p.get_losses(), p.get_average(), avg_dev.cpu().numpy(), pinned.numpy().copy(),
                             p.get_params(w.N - 1), p.get_velocity_stacked() if name == "momentum" else None))
                torch.cuda.current_stream().synchronize()
                p.close()
        keep = [i for i in range(w.N) if name != "mask" or i != 1]
        for o in outs[1:]:
            assert np.array_equal(outs[0][0], o[0]), (w.name, name)
            assert np.array_equal(outs[0][1][keep], o[1][keep])
            assert np.array_equal(outs[0][2], o[2]) and np.array_equal(o[2], o[3]) and np.array_equal(o[2], o[4])
            assert np.array_equal(outs[0][5], o[5]) and np.array_equal(o[5], o[0][w.N - 1])
            if name == "momentum":
                assert np.array_equal(outs[0][6], o[6])


OVERLAP_CASES = [
    _w("tc-overlap-small", 3, (128, 256, 256, 10), 32, I=3),
    _w("tc-overlap-b64", 2, (192, 1024, 256, 10), 64, I=4),
    _w("tc-overlap-deep", 2, (64, 256, 384, 256, 100), 16, I=2),
    _w("tc-overlap-many", 20, (256, 1024, 512, 10), 32, I=5),
    _w("tc-overlap-I1", 4, (128, 1024, 256, 10), 32, I=1),
]


@pytest.mark.parametrize("w", OVERLAP_CASES, ids=[w.name for w in OVERLAP_CASES])
def test_second_layers_update_beside_the_first_layers_changes_no_bit(torch_cuda, w):
    """Layer 2's update enqueued after layer 1's update + next forward and started beside it, tiles claimed from a
    device counter, the next a_1 in a second buffer, and on fused averaging iterations the last big launch started
    beside the averages of the small segments (PRSGD_OPT_OVERLAP_UPDATE), against the launches one after the
    other: every tile is formed from the same numbers in the same order, so parameters, bf16 copy, losses and node
    average are identical; with direct launches and replayed periods, both tile widths, the momentum step, calls
    that end inside a period, and more row blocks than SMs."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    X, Y, x0 = make_inputs(w)
    T = 2 * w.I + 2
    for name, opts in (("plain", {}), ("tile128", {binding.OPT_UPDATE_TILE: 128}), ("no-head", {binding.OPT_HEAD_KERNEL: 0}), ("momentum", {}),
                       ("momentum-averaged", {})):
        outs = []
        for overlap, graph in ((0, 0), (1, 0), (1, 1)):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                p.set_option(binding.OPT_OVERLAP_UPDATE, overlap)
                p.set_option(binding.OPT_GRAPH, graph)
                for k, v in opts.items():
                    p.set_option(k, v)
                if name.startswith("momentum"):
                    p.enable_momentum(0.9, average_velocity=name.endswith("averaged"))
                n0 = p.get_launch_count()
                p.local_steps(w.I + 1)           # ends inside the second period
                mid = p.get_params_stacked()
                p.local_steps(T - w.I - 1)
                p.sync()
                store = p.params.cpu().numpy().reshape(w.N, p.m_pad)
                shadow = p.shadow.view(torch.int16).cpu().numpy().view(np.uint16).reshape(w.N, p.m_pad)
                for l in range(len(w.dims) - 1):
                    a, n = p.layout.w_off[l], w.dims[l] * w.dims[l + 1]
                    assert np.array_equal(shadow[:, a:a + n], synth.bf16_bits(store[:, a:a + n])), (w.name, name, l)
                outs.append((p.get_params_stacked(), mid, p.get_losses(), p.get_average(), p.get_launch_count() - n0,
                             p.get_velocity_stacked() if name.startswith("momentum") else None))
                torch.cuda.current_stream().synchronize()
                p.close()
        for o in outs[1:]:
            assert np.array_equal(outs[0][0], o[0]), (w.name, name)
            assert np.array_equal(outs[0][1], o[1]), (w.name, name)
            assert np.array_equal(outs[0][2], o[2]) and np.array_equal(outs[0][3], o[3])
            if name.startswith("momentum"):
                assert np.array_equal(outs[0][5], o[5])
        assert outs[0][4] == outs[1][4]


@pytest.mark.parametrize("I,T", [(16, 40), (1, 12), (3, 20)])
def test_overlapped_launches_at_full_size_change_no_bit(torch_cuda, I, T):
    """The 16-worker 3072-1024-1024-10 configuration as the benchmark runs it (replayed periods, 128 row-block CTAs
    of layer 1's launch beside the claimed tiles of layer 2's update, the last big launch of an averaging iteration
    beside the small averages) against the launches one after the other: identical parameters and losses, also
    across calls that end inside a period and an odd number of iterations per period."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    w = synth.WORKLOADS["cfg3"].with_(pool_samples=256, I=I)
    X, Y, x0 = make_inputs(w)
    outs = []
    for overlap, graph in ((0, 0), (1, 1), (1, 0)):
        with torch.cuda.stream(torch.cuda.Stream()):
            p = make_ctx(w, X, Y, x0)
            p.set_option(binding.OPT_OVERLAP_UPDATE, overlap)
            p.set_option(binding.OPT_GRAPH, graph)
            p.local_steps(5)
            p.local_steps(T - 5)
            p.sync()
            outs.append((p.params.cpu().numpy().copy(), p.get_losses().copy()))
            torch.cuda.current_stream().synchronize()
            p.close()
    for o in outs[1:]:
        assert np.array_equal(outs[0][0], o[0]) and np.array_equal(outs[0][1], o[1])


HEAD_FWD_CASES = [
    _w("tc-tail-small", 3, (128, 256, 128, 10), 32, I=3),
    _w("tc-tail-ragged-k", 2, (192, 320, 1024, 10), 64, I=2),
    _w("tc-tail-b16-c100", 5, (64, 128, 512, 100), 16, I=3),
    _w("tc-tail-deep", 2, (64, 192, 256, 256, 10), 32, I=2),
    _w("tc-tail-I1", 4, (128, 1024, 256, 10), 32, I=1),
]


@pytest.mark.parametrize("w", HEAD_FWD_CASES, ids=[w.name for w in HEAD_FWD_CASES])
def test_forward_below_the_class_layer_inside_the_cluster_launch(torch_cuda, w):
    """The forward GEMM of layer L - 1 done by the class layer's cluster launch (every CTA forms the 128 features of
    a_{L-1} it needs and keeps them in shared memory) against the separate forward launch: the same products in
    the same order, so identical parameters, losses and draws over several periods, direct and replayed, with a
    worker mask, from a common restart point (I = 1) and with the option that shares one copy of the weights
    off; one launch fewer per iteration."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    X, Y, x0 = make_inputs(w)
    T = 2 * w.I + 2
    for variant in ("plain", "mask", "no-shared-restart"):
        outs = []
        for fwd, graph in ((0, 0), (1, 0), (1, 1)):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                p.set_option(binding.OPT_HEAD_FORWARD, fwd)
                p.set_option(binding.OPT_GRAPH, graph)
                if variant == "mask":
                    p.set_active([1 if i != 1 else 0 for i in range(w.N)])
                if variant == "no-shared-restart":
                    p.set_option(binding.OPT_SHARED_RESTART, 0)
                n0 = p.get_launch_count()
                p.local_steps(1)
                p.local_steps(T - 1)
                outs.append((p.get_params_stacked(), p.get_losses(), p.get_draws().tolist(), p.get_launch_count() - n0))
                torch.cuda.current_stream().synchronize()
                p.close()
        keep = [i for i in range(w.N) if variant != "mask" or i != 1]
        for o in outs[1:]:
            assert np.array_equal(outs[0][0], o[0]), (w.name, variant)
            assert np.array_equal(outs[0][1][keep], o[1][keep])
            assert [outs[0][2][i] for i in keep] == [o[2][i] for i in keep]
        assert outs[1][3] == outs[0][3] - T, (outs[0][3], outs[1][3])


SPLIT_CASES = [
    (_w("tc-split-ragged", 2, (192, 320, 100), 32, I=3), None),
    (_w("tc-split-wide-in", 3, (448, 256, 10), 16, I=4), None),
    (_w("tc-split-one-block", 1, (1024, 128, 10), 32, I=2), None),
    (_w("tc-split-b64", 2, (128, 128, 100), 64, I=2), None),
    (_w("tc-split-mom", 3, (320, 256, 10), 32, I=3), 0.9),
]


@pytest.mark.parametrize("w,mu", SPLIT_CASES, ids=[c[0].name for c in SPLIT_CASES])
def test_row_blocks_cut_at_run_boundaries(torch_cuda, w, mu):
    """Layer 1's update + next forward with its column tiles dealt out in equal runs (PRSGD_OPT_SPLIT_BLOCKS = 2
    forces it on small shapes): a row block cut by a run boundary gets its a_1 from partial sums added in run
    order by the last of its CTAs.  The step of an iteration does not depend on it (bit-identical weights after
    the first iteration); later iterations start from an a_1 summed in another order, so they agree to rounding;
    the form is deterministic (two runs, direct and replayed, same bits), works for both tile widths, and a period
    meets the oracle's bounds."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    X, Y, x0 = make_inputs(w)
    x0s = np.tile(x0, (w.N, 1))
    T = 2 * w.I + 2
    runs = {}
    for split, graph, tile in ((0, 0, 0), (2, 0, 0), (2, 1, 0), (2, 0, 64), (2, 0, 128), (2, 0, 0)):
        with torch.cuda.stream(torch.cuda.Stream()):
            p = make_ctx(w, X, Y, x0)
            if mu is not None:
                p.enable_momentum(mu)
            p.set_option(binding.OPT_SPLIT_BLOCKS, split)
            p.set_option(binding.OPT_GRAPH, graph)
            p.set_option(binding.OPT_UPDATE_TILE, tile)
            n0 = p.get_launch_count()
            p.local_steps(2)
            second = p.get_params_stacked()
            p.local_steps(T - 2)
            runs.setdefault((split, graph, tile), []).append(
                (second, p.get_params_stacked(), p.get_losses(), p.get_draws().tolist(), p.get_launch_count() - n0))
            torch.cuda.current_stream().synchronize()
            p.close()
    off = runs[(0, 0, 0)][0]
    on = runs[(2, 0, 0)]
    assert np.array_equal(on[0][1], on[1][1]) and np.array_equal(on[0][2], on[1][2])        # deterministic
    for key in ((2, 1, 0), (2, 0, 64), (2, 0, 128)):
        o = runs[key][0]
        if key[2] == 0 or mu is not None:                  # (a tile width of its own cuts the blocks elsewhere)
            assert np.array_equal(on[0][1], o[1]), key
        assert rel_l2(o[1] - x0s, off[1] - x0s) <= 2e-2, key
        assert o[3] == off[3] and (key[1] == 1 or o[4] == off[4])
    # iteration 1 has no folded forward before it and iteration 2 starts from the a_1 it formed: the first step is
    # bit-identical, the second within rounding
    assert rel_l2(on[0][0] - x0s, off[0] - x0s) <= 5e-3, rel_l2(on[0][0] - x0s, off[0] - x0s)
    assert np.allclose(on[0][2], off[2], rtol=5e-3, atol=1e-4)
    want = oracle_run(w, X, Y, x0s.astype(np.float64), 0, T) if mu is None else None
    if want is not None:
        assert rel_l2(on[0][1], want) <= TOL_PERIOD
        assert rel_l2(on[0][1] - x0s, want - x0s) <= TOL_UPDATE


COMMON_CASES = [
    _w("tc-common-b32", 3, (640, 1024, 10), 32, I=1),
    _w("tc-common-b64-n5", 5, (1024, 768, 100), 64, I=1),
    _w("tc-common-b16-deep", 2, (704, 1024, 640, 10), 16, I=1),
    _w("tc-common-cut-tail", 3, (1280, 1280, 10), 32, I=1),       # 200 tiles: the 52 of the second round are cut in two
]


@pytest.mark.parametrize("w", COMMON_CASES, ids=[w.name for w in COMMON_CASES])
def test_average_from_a_common_point_as_one_gemm_over_all_workers(torch_cuda, w):
    """An averaging iteration that starts from N equal rows (every iteration when I = 1: parallel mini-batch SGD)
    forms the new average as x - (gamma / N) sum_i G_i with one weight-gradient GEMM over the minibatches of all
    workers, against the N stepped models summed one by one: equal to fp32 rounding, not bit for bit; rows
    identical, bf16 copies equal to bf16(master), replay identical to direct launches, the row-sum form of a
    sharded average, and every segment's step against the oracle."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    X, Y, x0 = make_inputs(w)
    x0s = np.tile(x0, (w.N, 1))
    runs = {}
    for common, graph in ((0, 0), (1, 0), (1, 1), (2, 0)):
        with torch.cuda.stream(torch.cuda.Stream()):
            p = make_ctx(w, X, Y, x0)
            p.set_option(binding.OPT_COMMON_POINT, common)
            p.set_option(binding.OPT_GRAPH, graph)
            n0 = p.get_launch_count()
            p.local_steps(1)
            first = p.get_params_stacked()
            p.local_steps(3)
            launches = p.get_launch_count() - n0
            p.sync()
            store = p.params.cpu().numpy().reshape(w.N, p.m_pad)
            shadow = p.shadow.view(torch.int16).cpu().numpy().view(np.uint16).reshape(w.N, p.m_pad)
            for l in range(len(w.dims) - 1):
                a, n = p.layout.w_off[l], w.dims[l] * w.dims[l + 1]
                assert np.array_equal(shadow[:, a:a + n], synth.bf16_bits(store[:, a:a + n])), (w.name, l, common)
            assert all(np.array_equal(store[i], store[0]) for i in range(w.N))
            # the row-sum form (first half of an average whose other rows live on other GPUs), from equal rows
            p.set_interval(0)
            p.local_steps_sum(1)
            sums = p.get_params_stacked()
            runs[(common, graph)] = (first, store.copy(), launches, sums)
            torch.cuda.current_stream().synchronize()
            p.close()
    off, on, replay, whole = runs[(0, 0)], runs[(1, 0)], runs[(1, 1)], runs[(2, 0)]
    assert np.array_equal(on[1], replay[1]) and np.array_equal(on[3], replay[3])
    assert np.array_equal(on[1], whole[1]) and np.array_equal(on[3], whole[3])      # who stores a row changes no bit
    assert on[2] <= off[2]                                 # (several such layers share one launch)
    assert not np.array_equal(on[0], x0s)
    assert rel_l2(on[0] - x0s, off[0] - x0s) <= 1e-4, rel_l2(on[0] - x0s, off[0] - x0s)
    assert rel_l2(on[1], off[1]) <= 1e-4
    assert rel_l2(on[3], off[3]) <= 1e-4 and np.linalg.norm(on[3][0]) > 1.5 * np.linalg.norm(on[1][0])
    # one averaging step from x0 against the oracle, every segment on its own, no ReLU able to switch
    xm = with_margin(x0, w.dims)
    xms = np.tile(xm, (w.N, 1)).astype(np.float64)
    want = oracle_run(w, X, Y, xms, 0, 1)
    errs = {}
    for common in (0, 1):
        p = make_ctx(w, X, Y, xm)
        p.set_option(binding.OPT_COMMON_POINT, common)
        p.local_steps(1)
        got = p.get_params_stacked()
        errs[common] = [rel_l2(got[:, lo:hi] - xms[:, lo:hi], want[:, lo:hi] - xms[:, lo:hi]) for _, lo, hi in _segments(w.dims)]
        p.close()
    for l, e in enumerate(errs[1]):
        depth = len(w.dims) - 1 - l // 2
        assert e <= max(TOL_UPDATE_MARGIN * max(1.0, depth / 2), 1.05 * errs[0][l]), (l, e, errs[0][l])


def _segments(dims):
    """[(is_weight, start, stop)] of a canonical parameter vector."""
    out, off = [], 0
    for l in range(len(dims) - 1):
        for is_w, cnt in ((True, dims[l] * dims[l + 1]), (False, dims[l + 1])):
            out.append((is_w, off, off + cnt))
            off += cnt
    return out


@pytest.mark.parametrize("w", [SMALL[0], SMALL[3], SMALL[4], SMALL[6]], ids=lambda w: w.name)
def test_epilogue_softmax_and_bias_steps_equal_the_standalone_kernels(torch_cuda, w):
    """Softmax-CE gradient in the last forward GEMM's epilogue and bias steps in the dZ epilogues against the
    same work done by kernels of their own: identical dZ, so identical weights after one iteration; the bias
    steps differ only in summing dZ before instead of after its rounding to bf16."""
    from paper_1807_06629_b200 import binding
    X, Y, x0 = make_inputs(w)
    outs = []
    for fused in (1, 0):
        p = make_ctx(w, X, Y, x0, I=0)
        p.set_option(binding.OPT_FUSED_EPILOGUES, fused)
        p.set_option(binding.OPT_DX_IN_UPDATE, 0)         # (needs the epilogue form; off in both arms)
        n0 = p.get_launch_count()
        p.local_steps(1)
        outs.append((p.get_params_stacked(), p.get_losses(), p.get_draws().tolist(), p.get_launch_count() - n0))
    (a, la, da, na), (b, lb, db, nb) = outs
    assert nb == na + 2                                   # the softmax kernel and the bias kernel
    assert da == db and np.array_equal(la, lb)
    x0s = np.tile(x0, (w.N, 1))
    for is_w, lo, hi in _segments(w.dims):
        if is_w:
            assert np.array_equal(a[:, lo:hi], b[:, lo:hi])
        else:
            assert rel_l2(a[:, lo:hi] - x0s[:, lo:hi], b[:, lo:hi] - x0s[:, lo:hi]) <= 5e-3


@pytest.mark.parametrize("fused", [1, 0])
def test_standalone_softmax_and_bias_kernels_against_the_oracle(torch_cuda, fused):
    """More than 128 classes do not fit one tile of the last GEMM, so the stand-alone kernels run whatever the
    option says; a 10-class net with the option off takes the same route."""
    from paper_1807_06629_b200 import binding
    for w in (_w("tc-200-classes", 2, (64, 128, 200), 32), SMALL[1]):
        X, Y, x0 = make_inputs(w)
        p = make_ctx(w, X, Y, x0)
        p.set_option(binding.OPT_FUSED_EPILOGUES, fused)
        if w.dims[-1] <= 128 and fused:
            continue                                      # that combination is every other test of this file
        x0s = np.tile(x0, (w.N, 1)).astype(np.float64)
        losses = {}
        want = oracle_run(w, X, Y, x0s, 0, w.I, losses=losses)
        p.local_steps(w.I)
        got = p.get_params_stacked()
        assert np.allclose(p.get_losses(), [losses[(i, w.I)] for i in range(w.N)], rtol=2e-2, atol=2e-3)
        assert all(np.array_equal(got[i], got[0]) for i in range(w.N))
        assert rel_l2(got, want) <= TOL_PERIOD
        assert rel_l2(got - x0s, want - x0s) <= TOL_UPDATE, rel_l2(got - x0s, want - x0s)


def test_shadow_tracks_master_and_padding_stays_zero(torch_cuda):
    torch = torch_cuda
    w = SMALL[4]
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    p.local_steps(2 * w.I + 1)
    p.sync()
    store = p.params.cpu().numpy().reshape(w.N, p.m_pad)
    shadow = p.shadow.view(torch.int16).cpu().numpy().view(np.uint16).reshape(w.N, p.m_pad)
    keep = np.zeros(p.m_pad, dtype=bool)
    for l in range(len(w.dims) - 1):
        a, n = p.layout.w_off[l], w.dims[l] * w.dims[l + 1]
        keep[a:a + n] = True
        assert np.array_equal(shadow[:, a:a + n], synth.bf16_bits(store[:, a:a + n]))   # weights: shadow = bf16(master)
        keep[p.layout.b_off[l]:p.layout.b_off[l] + w.dims[l + 1]] = True
    assert np.all(store[:, ~keep] == 0.0)


def test_inactive_workers_keep_their_point(torch_cuda):
    w = _w("tc-mask", 4, (64, 128, 10), 32, I=0)
    X, Y, x0 = make_inputs(w)
    fn = orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed)
    I_i, S = [3, 1, 2, 3], 2
    q = make_ctx(w, X, Y, x0, I=0)
    for s in range(S):
        q.average()
        for k in range(1, max(I_i) + 1):
            q.set_active([1 if k <= I_i[i] else 0 for i in range(w.N)])
            q.local_steps(1)
    want = orc.pr_sgd_heterogeneous(np.tile(x0, (w.N, 1)), w.gamma, I_i, S, fn)
    got = q.get_params_stacked()
    x0s = np.tile(x0, (w.N, 1))
    assert rel_l2(got - x0s, want - x0s) <= TOL_UPDATE
    # fused average with a mask: inactive workers contribute their unchanged point
    r = make_ctx(w, X, Y, x0, I=1)
    r.set_active([1, 0, 1, 0])
    r.local_steps(1)
    one = oracle_run(w, X, Y, x0s, 0, 1, I=0)
    one[1], one[3] = x0, x0
    assert rel_l2(r.get_params_stacked()[0] - x0, one.mean(0) - x0) <= TOL_UPDATE


@pytest.mark.parametrize("name,I", [("cfg3", 1), ("cfg3", 4), ("cfg3", 16), ("cfg4", 2), ("cfg4", 32)],
                         ids=lambda v: str(v))
def test_full_size_configs(torch_cuda, name, I):
    """cfg3 / cfg4 at their full N, widths, batch and averaging interval (cfg3: I = 1, 4, 16; cfg4: I = 32), one
    full averaging period from a synchronised state in ONE call on a side stream, i.e. in the launch
    configuration the benchmark times (folded kernels, fused update + average, graph replay), against the
    oracle: <= 2e-2 relative L2 of the stacked parameters, identical rows, exact draws."""
    torch = torch_cuda
    base = synth.WORKLOADS[name]
    w = base.with_(pool_samples=max(I, 4) * base.B, I=I)
    X, Y, x0 = make_inputs(w)
    x0s = np.tile(x0, (w.N, 1)).astype(np.float64)
    draws = {}
    want = oracle_run(w, X, Y, x0s, 0, w.I, draws=draws)
    with torch.cuda.stream(torch.cuda.Stream()):
        p = make_ctx(w, X, Y, x0)
        p.local_steps(w.I)
        got = p.get_params_stacked()
        assert p.get_step() == w.I
        assert p.get_draws().tolist() == [draws[(i, w.I)] for i in range(w.N)]
        assert all(np.array_equal(got[i], got[0]) for i in range(w.N))
        assert rel_l2(got, want) <= TOL_PERIOD, rel_l2(got, want)
        assert rel_l2(got - x0s, want - x0s) <= TOL_UPDATE, rel_l2(got - x0s, want - x0s)
        # the same period one iteration per call: the draw of every worker at every iteration is the oracle's,
        # and the separate launches leave the bits of the one-call run
        q = make_ctx(w, X, Y, x0)
        for t in range(1, w.I + 1):
            q.local_steps(1)
            assert q.get_draws().tolist() == [draws[(i, t)] for i in range(w.N)], t
        assert np.array_equal(q.get_params_stacked(), got)
        q.close()
        # the next (non-averaging) iteration of a few sampled workers: x_i^t - x_i^{t-1} = -gamma G_i^t
        fn = orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed)
        sample = list(range(0, w.N, max(1, w.N // 4)))
        G = np.stack([fn(i, w.I + 1, got[i].astype(np.float64)) for i in sample])
        p.set_interval(0)
        p.local_steps(1)
        nxt = p.get_params_stacked()
        for k, i in enumerate(sample):
            assert rel_l2(nxt[i] - got[i], -w.gamma * G[k]) <= TOL_UPDATE
        torch.cuda.current_stream().synchronize()
        p.close()


@pytest.mark.parametrize("name,T", [("cfg3", 64), ("cfg4", 64)])
def test_full_size_runs_of_whole_periods_keep_the_invariants(torch_cuda, name, T):
    """cfg3 / cfg4 at full size over several whole periods in one call (graph replay, folded kernels): after the
    last average every row holds the same bits, the bf16 copy equals bf16(master), the padding is still zero,
    and the loss has gone down."""
    torch = torch_cuda
    w = synth.WORKLOADS[name]
    w = w.with_(pool_samples=max(w.I, 4) * w.B)
    X, Y, x0 = make_inputs(w)
    with torch.cuda.stream(torch.cuda.Stream()):
        p = make_ctx(w, X, Y, x0)
        p.local_steps(1)
        first = p.get_losses().mean()
        p.local_steps(T - 1)
        assert p.get_step() == T and T % w.I == 0
        p.sync()
        rows = p.params.view(w.N, p.m_pad)
        assert bool((rows == rows[0:1]).all())             # the run ended on an average: one point, N copies
        p.local_steps(1)                                   # one more iteration for a loss at the averaged point
        last = p.get_losses().mean()
        p.sync()
        assert np.isfinite(last) and last < first - 0.05, (first, last)
        store = p.params.cpu().numpy().reshape(w.N, p.m_pad)
        shadow = p.shadow.view(torch.int16).cpu().numpy().view(np.uint16).reshape(w.N, p.m_pad)
        keep = np.zeros(p.m_pad, dtype=bool)
        for l in range(len(w.dims) - 1):
            a, n = p.layout.w_off[l], w.dims[l] * w.dims[l + 1]
            keep[a:a + n] = True
            keep[p.layout.b_off[l]:p.layout.b_off[l] + w.dims[l + 1]] = True
            assert np.array_equal(shadow[:, a:a + n], synth.bf16_bits(store[:, a:a + n])), l
        assert np.all(store[:, ~keep] == 0.0)
        torch.cuda.current_stream().synchronize()


@pytest.mark.parametrize("avg_v", [False, True])
def test_momentum_step_on_the_tensor_core_path(torch_cuda, avg_v):
    """v <- mu v + G, x <- x - gamma v in the update kernel's epilogue; hidden biases +-6 so no ReLU can switch."""
    for w in (SMALL[1], SMALL[3], SMALL[4]):
        X, Y, x0 = make_inputs(w)
        x0 = with_margin(x0, w.dims)
        p = make_ctx(w, X, Y, x0)
        if w is SMALL[3]:                                 # one workload takes the stand-alone bias kernel
            from paper_1807_06629_b200 import binding
            p.set_option(binding.OPT_FUSED_EPILOGUES, 0)
        p.enable_momentum(0.9, average_velocity=avg_v)
        fn = orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed)
        xs = np.tile(x0, (w.N, 1)).astype(np.float64)
        T = 2 * w.I + 1
        p.local_steps(T)
        want_x, want_v = orc.pr_sgd_momentum(xs, np.zeros_like(xs), w.gamma, 0.9, w.I, T, fn, average_velocity=avg_v)
        got_x, got_v = p.get_params_stacked(), p.get_velocity_stacked()
        assert rel_l2(got_x, want_x) <= TOL_PERIOD
        assert rel_l2(got_x - xs, want_x - xs) <= 2e-2, rel_l2(got_x - xs, want_x - xs)
        # averaged buffers keep only the common part of the gradients: smaller norm, same absolute bf16 noise
        assert rel_l2(got_v, want_v) <= (5e-2 if avg_v else 2e-2), rel_l2(got_v, want_v)
        # shadow still tracks the master
        import torch
        store = p.params.cpu().numpy().reshape(w.N, p.m_pad)
        shadow = p.shadow.view(torch.int16).cpu().numpy().view(np.uint16).reshape(w.N, p.m_pad)
        a, n = p.layout.w_off[0], w.dims[0] * w.dims[1]
        assert np.array_equal(shadow[:, a:a + n], synth.bf16_bits(store[:, a:a + n]))


def test_partial_sum_and_assign_rows_equal_average_on_the_bf16_store(torch_cuda):
    torch = torch_cuda
    w = SMALL[4]
    X, Y, x0 = make_inputs(w)
    a = make_ctx(w, X, Y, x0, I=0)
    b = make_ctx(w, X, Y, x0, I=0)
    a.local_steps(2); b.local_steps(2)
    a.average()
    r = b.new_row()
    b.partial_sum(r)
    b.assign_rows(r, float(w.N))
    b.sync()
    assert np.array_equal(a.get_params_stacked(), b.get_params_stacked())
    assert torch.equal(a.shadow.view(torch.int16), b.shadow.view(torch.int16))     # shadow rewritten too
    a.local_steps(1); b.local_steps(1)
    assert np.array_equal(a.get_params_stacked(), b.get_params_stacked())


def test_row_sums_fused_into_the_last_local_step_equal_the_separate_pass(torch_cuda):
    """prsgd_local_steps_sum (the period's last step in fused form with the division left out, every row = the
    local row sum) followed by prsgd_assign_rows(row 0, N) against the fused update + average, and against
    local steps + prsgd_partial_sum + prsgd_assign_rows: identical parameters and bf16 copy, plain and momentum
    step; the next period's iterations agree too (the restart point is flagged as common in all three)."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    for w in (SMALL[1], SMALL[4], _w("tc-sum-n5", 5, (64, 128, 10), 32, I=3), _w("tc-sum-wide", 3, (64, 448, 320, 10), 16, I=4)):
        X, Y, x0 = make_inputs(w)
        for mu in (None, 0.9):
            outs = []
            for how in ("fused average", "row sums in the last step", "separate row-sum pass"):
                p = make_ctx(w, X, Y, x0, I=w.I if how == "fused average" else 0)
                if mu is not None:
                    p.enable_momentum(mu)
                for period in range(2):
                    if how == "fused average":
                        p.local_steps(w.I)
                    elif how == "row sums in the last step":
                        p.local_steps_sum(w.I)
                        half = (p.m_pad // 8) * 4
                        p.assign_rows(p.row0(), float(w.N), 0, half)
                        p.assign_rows(p.row0(), float(w.N), half, p.m_pad - half)
                    else:
                        p.local_steps(w.I)
                        r = p.new_row()
                        p.partial_sum(r)
                        p.assign_rows(r, float(w.N))
                p.set_interval(0)
                p.local_steps(1)
                p.sync()
                shadow = p.shadow.view(torch.int16).cpu().numpy().reshape(w.N, p.m_pad)
                wcols = np.zeros(p.m_pad, dtype=bool)         # the bf16 copy matters (and is kept) for the weights only
                for l in range(len(w.dims) - 1):
                    wcols[p.layout.w_off[l]:p.layout.w_off[l] + w.dims[l] * w.dims[l + 1]] = True
                outs.append((p.get_params_stacked(), shadow[:, wcols].copy(), p.get_step(),
                             p.get_velocity_stacked() if mu is not None else None))
                p.close()
            for o in outs[1:]:
                assert np.array_equal(outs[0][0], o[0]), (w.name, mu)
                assert np.array_equal(outs[0][1], o[1]) and outs[0][2] == o[2] == 2 * w.I + 1
                if mu is not None:
                    assert np.array_equal(outs[0][3], o[3])
    q = make_ctx(SMALL[1], *make_inputs(SMALL[1]))              # I = 2: the library averages by itself
    with pytest.raises(binding.PRSGDError):
        q.local_steps_sum(2)


def test_training_run_tracks_the_oracle_loss_curve(torch_cuda):
    """48 iterations (12 periods) on the tensor-core path: draws exact, loss curve within bf16 noise of the
    oracle's, loss going down."""
    w = synth.Workload("tc-train", 4, (128, 256, 128, 10), 32, 0.1, 4, 48, 1, 32 * 32, mean_shift=0.5, seed=77)
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    losses, draws = {}, {}
    want = oracle_run(w, X, Y, np.tile(x0, (w.N, 1)), 0, w.T, losses=losses, draws=draws)
    curve = []
    for t in range(1, w.T + 1):
        p.local_steps(1)
        assert p.get_draws().tolist() == [draws[(i, t)] for i in range(w.N)]
        curve.append(p.get_losses())
    curve = np.array(curve)
    ref = np.array([[losses[(i, t)] for i in range(w.N)] for t in range(1, w.T + 1)])
    assert np.abs(curve - ref).max() <= 5e-2
    assert np.abs(curve.mean(1) - ref.mean(1)).max() <= 2e-2
    assert curve[-8:].mean() < curve[:8].mean() - 0.1
    assert rel_l2(p.get_params_stacked(), want) <= TOL_PERIOD


def test_graph_replay_of_whole_periods_is_bit_identical(torch_cuda):
    """On a non-default stream whole periods are replayed from a captured CUDA graph (iteration number read
    from a device counter); the bits, the draws and the step counter must equal direct launches."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    for w in (SMALL[1], _w("tc-n5", 5, (64, 128, 10), 32, I=3), synth.WORKLOADS["cfg1"]):
        X, Y, x0 = make_inputs(w)
        outs = []
        for use_graph in (0, 1):
            with torch.cuda.stream(torch.cuda.Stream()):
                p = make_ctx(w, X, Y, x0)
                p.set_option(binding.OPT_GRAPH, use_graph)
                n0 = p.get_launch_count()
                p.local_steps(1)                  # partial period: direct
                p.local_steps(w.I - 1)            # reaches the first average
                p.local_steps(3 * w.I + 1)        # three whole periods (replayed) and one more iteration
                p.set_lr(w.gamma * 0.5)           # a new setting keys a new capture
                p.local_steps(2 * w.I)
                outs.append((p.get_params_stacked(), p.get_draws().tolist(), p.get_step(), p.get_losses(),
                             p.get_launch_count() - n0))
                torch.cuda.current_stream().synchronize()
        assert np.array_equal(outs[0][0], outs[1][0])
        assert outs[0][1] == outs[1][1] and outs[0][2] == outs[1][2] == 6 * w.I + 1
        assert np.array_equal(outs[0][3], outs[1][3])
        # same kernels, plus one counter-set launch per run of replayed periods (a replay leaves the device counter
        # at the next period's start): one before the three periods, one after the new setting, whose request first
        # walks to the period boundary with direct launches
        assert outs[1][4] == outs[0][4] + 2


def test_expired_wait_is_reported_and_the_context_recovers(torch_cuda):
    """Failure path without a fault: a bounded wait runs out, the status word is set, later launches do
    nothing, the host sees PRSGD_ERR_DEVICE_TIMEOUT, and after clearing the context continues bit for bit."""
    from paper_1807_06629_b200 import binding
    w = SMALL[1]
    X, Y, x0 = make_inputs(w)
    ref = make_ctx(w, X, Y, x0)
    ref.local_steps(3)
    want = ref.get_params_stacked()
    p = make_ctx(w, X, Y, x0)
    p.local_steps(1)
    after1 = p.get_params_stacked()
    p.selftest_wait_expiry(500)                          # ~0.5 ms wait on a barrier nobody signals
    with pytest.raises(binding.PRSGDError) as e:
        p.sync()
    assert e.value.code == -6 and "expired" in str(e.value)
    p.local_steps(2)                                     # every tensor-core launch now sees the status word: no-ops
    with pytest.raises(binding.PRSGDError):
        p.get_params_stacked()
    p.clear_device_error()
    assert np.array_equal(p.get_params_stacked(), after1)   # the two skipped iterations changed nothing
    assert p.get_step() == 3
    # start over from a clean state: the context is fully usable again
    p.set_params(x0)
    p.set_step(0)
    p.local_steps(3)
    assert np.array_equal(p.get_params_stacked(), want)
