"""GPU parity, fp32-operand path and the averaging kernel, through the C ABI.

Tolerances (relative L2 over the stacked N*m parameter vector, from a state
synchronised with the oracle): <= 1e-5 after one iteration, <= 1e-4 after one
full averaging period.  Integer facts (draws, schedule, slot mapping) are exact.
"""
import numpy as np
import pytest

from oracle import prsgd_oracle as orc
from paper_1807_06629_b200 import synth
from helpers import make_ctx, make_inputs, oracle_run, rel_l2

pytestmark = pytest.mark.gpu

TOL_STEP, TOL_PERIOD = 1e-5, 1e-4
TOL_UPDATE = 1e-4          # relative L2 of the *change* x^t - x^{t-1} (a zero update cannot pass)


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch


def test_average_rows_matches_fp64_mean(torch_cuda):
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    for (N, m, stride) in [(8, 1_000_000, 1_000_000), (3, 1027, 1028), (1, 5, 8), (64, 40_003, 40_004), (7, 4, 4),
                           (256, 5000, 5000)]:
        V = synth.stacked_vectors(N, stride, seed=N * 7919 + m)
        P = torch.from_numpy(V).to("cuda:0")
        binding.prsgd_average_rows(P, N, m, stride)
        out = P.cpu().numpy()
        want = orc.node_average(V[:, :m].astype(np.float64))
        for i in range(1, N):
            assert np.array_equal(out[i, :m], out[0, :m])          # every slot holds the same bits
        assert np.array_equal(out[:, m:], V[:, m:])                # columns past m untouched
        assert np.abs(out[0, :m] - want).max() <= 2.0 ** -22 * np.abs(V[:, :m]).sum(0).max() / N + 1e-12
        assert rel_l2(out[0, :m], want) < 1e-6


def test_average_rows_empty_and_errors(torch_cuda):
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    P = torch.ones(4, 8, device="cuda:0")
    binding.prsgd_average_rows(P, 4, 0, 8)                         # m = 0: nothing to do
    assert torch.equal(P, torch.ones(4, 8, device="cuda:0"))
    with pytest.raises(binding.PRSGDError):
        binding.prsgd_average_rows(P, 4, 9, 8)


def test_set_get_roundtrip_and_padding_stays_zero(torch_cuda):
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    got = p.get_params_stacked()
    assert np.array_equal(got, np.tile(x0, (w.N, 1)))
    x1 = x0 + 1.0
    p.set_params(x1, worker=2)
    assert np.array_equal(p.get_params(2), x1) and np.array_equal(p.get_params(1), x0)
    p.set_params(x0)
    p.local_steps(9)                                               # includes two averages
    store = p.params.cpu().numpy().reshape(w.N, p.m_pad)
    keep = np.zeros(p.m_pad, dtype=bool)
    for l in range(len(w.dims) - 1):
        keep[p.layout.w_off[l]:p.layout.w_off[l] + w.dims[l] * w.dims[l + 1]] = True
        keep[p.layout.b_off[l]:p.layout.b_off[l] + w.dims[l + 1]] = True
    assert keep.sum() == w.m
    assert np.all(store[:, ~keep] == 0.0)
    assert np.array_equal(store[:, keep], p.get_params_stacked())


def test_draws_and_schedule_are_bit_exact(torch_cuda):
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    for t in range(1, 13):
        p.local_steps(1)
        assert p.get_step() == t
        want = [orc.draw_block(w.seed, i, t, w.n_blocks) for i in range(w.N)]
        assert p.get_draws().tolist() == want
        rows = p.get_params_stacked()
        identical = all(np.array_equal(rows[i], rows[0]) for i in range(1, w.N))
        assert identical == (t % w.I == 0)                          # averaged exactly at t = I, 2I, ...


@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_per_step_parity(torch_cuda, name):
    w = synth.WORKLOADS[name]
    if name == "cfg2":
        w = w.with_(pool_samples=32 * 16)
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    state = np.tile(x0, (w.N, 1)).astype(np.float64)
    for t in range(1, w.I + 2):                                     # a whole period and one step beyond
        losses = {}
        want = oracle_run(w, X, Y, state, t - 1, 1, losses=losses)
        p.set_params_stacked(state.astype(np.float32))              # synchronise with the oracle
        p.set_step(t - 1)
        p.local_steps(1)
        got = p.get_params_stacked()
        s32 = state.astype(np.float32).astype(np.float64)
        assert rel_l2(got, want) <= TOL_STEP, (t, rel_l2(got, want))
        assert rel_l2(got - s32, want - s32) <= TOL_UPDATE, (t, rel_l2(got - s32, want - s32))
        gl = p.get_losses()
        wl = np.array([losses[(i, t)] for i in range(w.N)])
        assert np.allclose(gl, wl, rtol=2e-5, atol=1e-6)
        state = want


@pytest.mark.parametrize("name", ["cfg1", "cfg2"])
def test_full_period_parity(torch_cuda, name):
    w = synth.WORKLOADS[name]
    if name == "cfg2":
        w = w.with_(pool_samples=32 * 16)
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    p.local_steps(w.I)
    got = p.get_params_stacked()
    want = oracle_run(w, X, Y, np.tile(x0, (w.N, 1)), 0, w.I)
    assert rel_l2(got, want) <= TOL_PERIOD
    assert rel_l2(got - x0[None, :], want - x0[None, :]) <= 10 * TOL_UPDATE
    for i in range(1, w.N):
        assert np.array_equal(got[i], got[0])
    # a second period, from the GPU's own state
    p.local_steps(w.I)
    want2 = oracle_run(w, X, Y, got, w.I, w.I)
    assert rel_l2(p.get_params_stacked(), want2) <= TOL_PERIOD


def test_fused_average_equals_update_then_average_bit_for_bit(torch_cuda):
    for name in ("cfg1", "cfg2"):
        w = synth.WORKLOADS[name]
        if name == "cfg2":
            w = w.with_(pool_samples=32 * 16)
        X, Y, x0 = make_inputs(w)
        from paper_1807_06629_b200 import binding
        outs = []
        for fused in (1, 0):
            p = make_ctx(w, X, Y, x0)
            p.set_option(binding.OPT_FUSED_AVERAGE, fused)
            p.local_steps(2 * w.I)
            outs.append(p.get_params_stacked())
        assert np.array_equal(outs[0], outs[1])
        # and a manual schedule (I = 0 plus explicit average) gives the same bits again
        p = make_ctx(w, X, Y, x0, I=0)
        for _ in range(2):
            p.local_steps(w.I)
            p.average()
        assert np.array_equal(p.get_params_stacked(), outs[0])


def test_local_steps_compose_and_resume(torch_cuda):
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    a = make_ctx(w, X, Y, x0)
    a.local_steps(11)
    b = make_ctx(w, X, Y, x0)
    b.local_steps(3)
    b.local_steps(0)
    b.local_steps(8)
    assert np.array_equal(a.get_params_stacked(), b.get_params_stacked())
    # checkpoint / resume: state + step counter reproduce the trajectory bit for bit
    c = make_ctx(w, X, Y, x0)
    c.local_steps(5)
    snap, t = c.get_params_stacked(), c.get_step()
    d = make_ctx(w, X, Y)
    d.set_params_stacked(snap)
    d.set_step(t)
    d.local_steps(6)
    assert np.array_equal(d.get_params_stacked(), a.get_params_stacked())


def test_get_average_is_the_mean_and_leaves_the_store_alone(torch_cuda):
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    p.local_steps(3)                                                # not an averaging iteration
    before = p.get_params_stacked()
    ybar = p.get_average()
    assert np.array_equal(p.get_params_stacked(), before)
    assert rel_l2(ybar, orc.node_average(before.astype(np.float64))) < 1e-6
    # mean dynamics (Eq. overline-x-update): xbar^t = xbar^{t-1} - gamma * mean_i G_i^t, also across an average
    fn = orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed)
    G = np.stack([fn(i, 4, before[i].astype(np.float64)) for i in range(w.N)])
    p.local_steps(1)                                                # t = 4 averages
    assert np.allclose(p.get_average(), ybar - w.gamma * G.mean(0), rtol=0, atol=2e-6)
    p.average()
    rows = p.get_params_stacked()
    assert all(np.array_equal(rows[i], rows[0]) for i in range(w.N))
    # right after an average the node average IS every row: returned as it stands, also for a worker count
    # that is no power of two (summing N copies and dividing would round)
    assert np.array_equal(p.get_average(), rows[0])
    w3 = w.with_(N=3)
    q = make_ctx(w3, X[:3], Y[:3], x0)
    q.local_steps(w3.I)                                             # ends on an averaging iteration
    assert np.array_equal(q.get_average(), q.get_params(0))
    q.local_steps(1)
    after = q.get_params_stacked().astype(np.float64)
    assert not np.array_equal(q.get_average(), q.get_params(0))     # workers differ again: the mean is formed
    assert rel_l2(q.get_average(), orc.node_average(after)) < 1e-6


def test_asynchronous_read_out_equals_get_average_while_training_goes_on(torch_cuda):
    """prsgd_get_average_async: the mean is snapshotted on the training stream and copied on another one; training
    that is queued right behind it must not leak into the snapshot, and back-to-back read-outs must not overwrite
    each other's staging row."""
    torch = torch_cuda
    w = synth.WORKLOADS["cfg2"].with_(pool_samples=8 * 32, I=3)
    X, Y, x0 = make_inputs(w)
    with torch.cuda.stream(torch.cuda.Stream()):
        ref = make_ctx(w, X, Y, x0)
        p = make_ctx(w, X, Y, x0)
        rs = torch.cuda.Stream()
        outs = [torch.empty(p.m, dtype=torch.float32).pin_memory() for _ in range(3)]
        want = []
        for k in range(3):
            ref.local_steps(2 + k)
            want.append(ref.get_average().copy())
            p.local_steps(2 + k)
            p.get_average_async(outs[k], rs)               # returns at once; more work follows immediately
        p.local_steps(4)
        rs.synchronize()
        for k in range(3):
            assert np.array_equal(outs[k].numpy(), want[k]), k
        ref.local_steps(4)
        assert np.array_equal(p.get_average(), ref.get_average())
        with pytest.raises(Exception):
            p.get_average_async(outs[0], torch.cuda.current_stream())   # needs a stream of its own
        torch.cuda.current_stream().synchronize()


def test_time_varying_rates_and_heterogeneous_epochs(torch_cuda):
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    fn = orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed)
    # Algorithm 2 with a short schedule driven through set_lr + explicit averages
    sched = [(2, 0.08), (1, 0.05), (3, 0.03)]
    p = make_ctx(w, X, Y, x0, I=0)
    for (K, g) in sched:
        p.average()
        p.set_lr(g)
        p.local_steps(K)
    want = orc.pr_sgd_time_varying(np.tile(x0, (w.N, 1)), sched, fn)
    assert rel_l2(p.get_params_stacked(), want) <= TOL_PERIOD
    # Algorithm 3: per-worker epoch lengths through the active mask
    I_i, S = [3, 1, 2, 3], 2
    q = make_ctx(w, X, Y, x0, I=0)
    for s in range(S):
        q.average()
        for k in range(1, max(I_i) + 1):
            q.set_active([1 if k <= I_i[i] else 0 for i in range(w.N)])
            q.local_steps(1)
    want = orc.pr_sgd_heterogeneous(np.tile(x0, (w.N, 1)), w.gamma, I_i, S, fn)
    assert rel_l2(q.get_params_stacked(), want) <= TOL_PERIOD
    q.set_active(None)


@pytest.mark.parametrize("N,dims,B", [(1, (5, 3), 1), (3, (7, 5, 3, 2), 5), (2, (130, 70, 33), 48), (5, (16, 300, 11), 100),
                                      (2, (12,) + (9,) * 15 + (4,), 256)])      # last: 16 layers, batch 256 (the maxima)
def test_ragged_shapes(torch_cuda, N, dims, B):
    w = synth.Workload("ragged", N, dims, B, 0.1, 3, 6, 0, 4 * B, mean_shift=0.3, seed=77)
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    p.local_steps(1)
    want1 = oracle_run(w, X, Y, np.tile(x0, (N, 1)), 0, 1)
    assert rel_l2(p.get_params_stacked(), want1) <= TOL_STEP
    p.set_params(x0)
    p.set_step(0)
    p.local_steps(w.I)
    want = oracle_run(w, X, Y, np.tile(x0, (N, 1)), 0, w.I)
    assert rel_l2(p.get_params_stacked(), want) <= TOL_PERIOD


@pytest.mark.parametrize("avg_v", [False, True])
def test_momentum_step_matches_oracle(torch_cuda, avg_v):
    """Local step of the paper's experiment (momentum 0.9): parameters and momentum buffers over two periods."""
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    p.enable_momentum(0.9, average_velocity=avg_v)
    fn = orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed)
    xs = np.tile(x0, (w.N, 1)).astype(np.float64)
    p.local_steps(1)
    x1, v1 = orc.pr_sgd_momentum(xs, np.zeros_like(xs), w.gamma, 0.9, w.I, 1, fn)
    assert rel_l2(p.get_params_stacked(), x1) <= TOL_STEP
    assert rel_l2(p.get_velocity_stacked(), v1) <= 1e-5
    p.local_steps(2 * w.I - 1)
    x2, v2 = orc.pr_sgd_momentum(xs, np.zeros_like(xs), w.gamma, 0.9, w.I, 2 * w.I, fn, average_velocity=avg_v)
    got_x, got_v = p.get_params_stacked(), p.get_velocity_stacked()
    assert rel_l2(got_x, x2) <= TOL_PERIOD and rel_l2(got_v, v2) <= 1e-3
    assert all(np.array_equal(got_x[i], got_x[0]) for i in range(w.N))
    assert all(np.array_equal(got_v[i], got_v[0]) for i in range(w.N)) == avg_v


def test_two_shards_on_one_gpu_reproduce_the_unsharded_run(torch_cuda):
    """The local halves of the multi-GPU average: two contexts hold workers 0-1 and 2-3 (worker offset
    2), their partial sums are added (standing in for the all-reduce) and assigned back."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    whole = make_ctx(w, X, Y, x0)
    whole.local_steps(2 * w.I)
    shards = []
    for first in (0, 2):
        ws = w.with_(N=2)
        p = make_ctx(ws, X[first:first + 2], Y[first:first + 2], x0, I=0)
        p.set_worker_offset(first)
        shards.append(p)
    for period in range(2):
        rows = []
        for k, p in enumerate(shards):
            p.local_steps(w.I)
            assert p.get_draws().tolist() == [orc.draw_block(w.seed, 2 * k + i, (period + 1) * w.I, w.n_blocks) for i in range(2)]
            r = p.new_row()
            p.partial_sum(r, 0, 1000)                     # two column chunks, as the pipelined all-reduce does
            p.partial_sum(r, 1000, p.m_pad - 1000)
            rows.append(r)
        total = rows[0] + rows[1]
        for p in shards:
            p.assign_rows(total, float(w.N), 0, 1000)
            p.assign_rows(total, float(w.N), 1000, p.m_pad - 1000)
    got = np.concatenate([p.get_params_stacked() for p in shards])
    want = whole.get_params_stacked()
    assert all(np.array_equal(got[i], got[0]) for i in range(w.N))
    assert rel_l2(got, want) <= 1e-6
    # the same job with the row sums formed by the period's last local step (prsgd_local_steps_sum): row 0 of each
    # shard is the buffer the all-reduce would work on
    fused = []
    for first in (0, 2):
        p = make_ctx(w.with_(N=2), X[first:first + 2], Y[first:first + 2], x0, I=0)
        p.set_worker_offset(first)
        p.set_global_workers(w.N)
        fused.append(p)
    for period in range(2):
        for p in fused:
            p.local_steps_sum(w.I)
        total = fused[0].row0() + fused[1].row0()
        for p in fused:
            p.assign_rows(total, float(w.N))
    got2 = np.concatenate([p.get_params_stacked() for p in fused])
    assert np.array_equal(got2, got)
    one = make_ctx(w, X, Y, x0, I=0)                      # one context: sums in place, then the division
    for period in range(2):
        one.local_steps_sum(w.I)
        one.assign_rows(one.row0(), float(w.N))
    assert np.array_equal(one.get_params_stacked(), want)
    # with a single context the two halves leave exactly the bits of prsgd_average
    a = make_ctx(w, X, Y, x0, I=0)
    b = make_ctx(w, X, Y, x0, I=0)
    a.local_steps(3); b.local_steps(3)
    a.average()
    r = b.new_row()
    b.partial_sum(r)
    b.assign_rows(r, float(w.N))
    assert np.array_equal(a.get_params_stacked(), b.get_params_stacked())
    with pytest.raises(binding.PRSGDError):
        b.partial_sum(r, 2, 8)                            # misaligned column range


@pytest.mark.parametrize("N,m", [(64, 11_000_000), (256, 25_000_000)])
def test_average_rows_at_full_sweep_sizes(torch_cuda, N, m):
    """The largest points of the averaging sweep (up to 25.6 GB): inputs are drawn on the device from a
    seed, the oracle checks a strided sample of columns, and every row must hold the same bits."""
    torch = torch_cuda
    from paper_1807_06629_b200 import binding
    g = torch.Generator(device="cuda:0")
    g.manual_seed(20180717 + N)
    P = torch.empty(N, m, device="cuda:0", dtype=torch.float32)
    for i in range(0, N, 16):                                    # fill in slabs: no second 25 GB temporary
        P[i:i + 16].normal_(generator=g)
    cols = torch.arange(0, m, 9973, device="cuda:0")
    cols = torch.cat([cols, torch.tensor([m - 4, m - 3, m - 2, m - 1], device="cuda:0")])
    before = P[:, cols].cpu().numpy().astype(np.float64)
    binding.prsgd_average_rows(P, N, m)
    after = P[:, cols].cpu().numpy()
    want = orc.node_average(before)
    assert all(np.array_equal(after[i], after[0]) for i in range(N))
    assert np.abs(after[0] - want).max() <= 2.0 ** -22 * np.abs(before).sum(0).max() / N + 1e-12
    for i in range(1, N, max(1, N // 8)):                        # whole rows, compared on the device
        assert bool(torch.equal(P[i], P[0]))


def test_staged_pool_upload_equals_direct_upload(torch_cuda):
    """Double-buffered upload: stage on a copy stream, swap, run -- same bits as uploading in place."""
    torch = torch_cuda
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    w2 = w.with_(seed=w.seed + 1)
    X2, Y2 = synth.make_pools(w2)
    hX = [torch.from_numpy(a).pin_memory() for a in (X, X2)]
    hY = [torch.from_numpy(a).pin_memory() for a in (Y, Y2)]
    a = make_ctx(w, X, Y, x0)
    b = make_ctx(w, X, Y, x0)
    cs = torch.cuda.Stream()
    for k in range(4):
        a.upload_data(hX[k % 2], hY[k % 2])
        a.local_steps(3)
        b.stage_data(hX[k % 2], hY[k % 2], cs)
        b.swap_data()
        b.local_steps(3)
    assert np.array_equal(a.get_params_stacked(), b.get_params_stacked())
    with pytest.raises(Exception):
        b.swap_data()                                  # nothing staged


def test_algorithm_2_and_3_drivers(torch_cuda):
    """prsgd_run_time_varying / prsgd_run_heterogeneous_epoch against the oracle's Algorithm 2 and 3."""
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    fn = orc.mlp_grad_fn(w.dims, X.astype(np.float64), Y, w.B, w.seed)
    xs = np.tile(x0, (w.N, 1))
    scale = 0.02
    p = make_ctx(w, X, Y, x0)
    p.run_time_varying(1, 70, scale)                      # K^s goes from 1 to 2 at s = 65 for N = 4
    sched = [(K, g * scale) for (K, g) in orc.alg2_schedule(w.N, 70)]
    assert sum(K for K, _ in sched) == p.get_step() and max(K for K, _ in sched) == 2
    want = orc.pr_sgd_time_varying(xs, sched, fn)
    assert rel_l2(p.get_params_stacked(), want) <= 2e-4
    q = make_ctx(w, X, Y, x0)
    I_i = [3, 1, 0, 2]
    for _ in range(2):
        q.run_heterogeneous_epoch(I_i)
    want = orc.pr_sgd_heterogeneous(xs, w.gamma, I_i, 2, fn)
    assert rel_l2(q.get_params_stacked(), want) <= TOL_PERIOD
    assert q.get_step() == 6


def test_non_finite_parameters_are_reported_not_trapped(torch_cuda):
    """A NaN (or an infinity) put into ONE worker's row through prsgd_set_params is found by the finite check
    before the average, and after the average, which spreads it to every row (Algorithm 1's averaging step),
    in all N rows; with PRSGD_OPT_CHECK_FINITE prsgd_sync reports it too.  Both precisions."""
    from paper_1807_06629_b200 import binding
    cases = [(synth.WORKLOADS["cfg1"], float("nan")), (synth.WORKLOADS["cfg1"], float("-inf")),
             (synth.Workload("tc-nonfinite", 3, (64, 128, 10), 32, 0.05, 2, 4, 1, 128, mean_shift=0.5, seed=5), float("nan"))]
    for w, poison in cases:
        X, Y, x0 = make_inputs(w)
        p = make_ctx(w, X, Y, x0, I=0)
        p.local_steps(1)
        assert p.check_finite() == (0, 0, -1)
        bad = p.get_params(w.N - 2)
        bad[[7, x0.size - 1]] = poison                   # a weight of the first layer and the last bias
        p.set_params(bad, worker=w.N - 2)
        rc, count, first = p.check_finite()
        assert (rc, count, first) == (binding.ERR_NONFINITE, 2, w.N - 2)
        assert b"non-finite" in binding.lib.prsgd_last_error(p.ctx)
        p.sync()                                         # the plain sync does not look for it ...
        p.set_option(binding.OPT_CHECK_FINITE, 1)
        with pytest.raises(binding.PRSGDError) as e:     # ... unless asked to
            p.sync()
        assert e.value.code == binding.ERR_NONFINITE
        p.set_option(binding.OPT_CHECK_FINITE, 0)
        p.average()
        rc, count, first = p.check_finite()
        assert (rc, count, first) == (binding.ERR_NONFINITE, 2 * w.N, 0)
        p.set_params(x0)                                 # a clean state again: the context is usable
        assert p.check_finite() == (0, 0, -1)
        p.enable_momentum(0.9)
        p.local_steps(1)
        assert p.check_finite() == (0, 0, -1)            # (the momentum buffers are read as well)


def test_expired_wait_stops_the_fp32_path_too(torch_cuda):
    """After a bounded wait has run out, the local-step kernels of an FP32 context leave the store alone."""
    from paper_1807_06629_b200 import binding
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    p.local_steps(1)
    after1 = p.get_params_stacked()
    p.selftest_wait_expiry(300)
    with pytest.raises(binding.PRSGDError) as e:
        p.sync()
    assert e.value.code == binding.ERR_DEVICE_TIMEOUT
    p.local_steps(2 * w.I)                               # forward, dX, update and averaging launches: all no-ops
    p.clear_device_error()
    assert np.array_equal(p.get_params_stacked(), after1)
    q = make_ctx(w, X, Y, x0)                            # and the context carries on like a fresh one
    q.local_steps(1 + 2 * w.I)
    p.set_step(1)
    p.local_steps(2 * w.I)
    assert np.array_equal(p.get_params_stacked(), q.get_params_stacked())


def test_time_varying_schedule_uses_the_global_worker_count(torch_cuda):
    """Theorem 2's K^s and gamma^s are functions of the N of the whole job: a context that is told it holds all
    of a larger job's rows is refused (its average would be a shard's), one that is the whole job runs."""
    from paper_1807_06629_b200 import binding
    w = synth.WORKLOADS["cfg1"]
    X, Y, x0 = make_inputs(w)
    p = make_ctx(w, X, Y, x0)
    with pytest.raises(binding.PRSGDError):
        p.set_global_workers(w.N - 1)
    p.set_global_workers(2 * w.N)
    with pytest.raises(binding.PRSGDError) as e:
        p.run_time_varying(1, 3, 0.02)
    assert e.value.code == -4
    p.set_global_workers(0)
    p.run_time_varying(1, 3, 0.02)
    assert p.get_step() == sum(K for K, _ in orc.alg2_schedule(w.N, 3))


def test_cfg1_whole_run_tracks_the_oracle(torch_cuda):
    """All T = 64 iterations of the tiny configuration (16 averaging periods), GPU against oracle:
    the same draws every iteration, the same loss curve, and parameters that stay together."""
    w = synth.WORKLOADS["cfg1"]
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
    assert np.abs(curve - ref).max() <= 1e-3
    assert curve[-8:].mean() < curve[:8].mean() - 0.05            # it trains
    got = p.get_params_stacked()
    assert rel_l2(got, want) <= 1e-3
    assert all(np.array_equal(got[i], got[0]) for i in range(w.N))  # T = 64 is an averaging iteration
