"""Pins for the fp64 oracle: every check here compares the oracle with something
other than itself (published values, closed forms, hand-worked numbers,
identities the paper states, finite differences, exact summation)."""
import math
import os

import numpy as np
import pytest

from oracle import prsgd_oracle as orc
from paper_1807_06629_b200 import synth


# ---------------------------------------------------------------- the draw
def test_splitmix64_published_vector(golden_dir):
    with open(os.path.join(golden_dir, "splitmix64_seed1234567.txt")) as f:
        want = [int(s) for s in f.read().split("\n") if s and not s.startswith("#")]
    assert orc.splitmix64_stream(1234567, len(want)) == want


def test_draw_block_is_two_nested_streams():
    # block = (i+1)-th output of the stream keyed by the t-th output of the seed's stream
    for seed, i, t, nb in [(20180717, 0, 1, 64), (20180717, 3, 17, 64), (5, 63, 256, 32), (2**63 + 11, 7, 1000, 250)]:
        u = orc.splitmix64_stream(seed, t)[-1]
        v = orc.splitmix64_stream(u, i + 1)[-1]
        assert orc.draw_block(seed, i, t, nb) == v % nb


def test_draw_block_spreads_and_decorrelates_workers():
    nb, T, N = 16, 4000, 4
    d = np.array([[orc.draw_block(99, i, t, nb) for t in range(1, T + 1)] for i in range(N)])
    assert d.min() == 0 and d.max() == nb - 1
    for i in range(N):
        cnt = np.bincount(d[i], minlength=nb)
        chi2 = ((cnt - T / nb) ** 2 / (T / nb)).sum()
        assert chi2 < 45.0  # 15 dof, P(chi2 > 45) ~ 8e-5
    # two workers must not draw the same block more often than chance (1/nb)
    same = (d[0] == d[1]).mean()
    assert abs(same - 1.0 / nb) < 0.02


# ------------------------------------------------- the gradient of the MLP loss
def test_loss_hand_worked_single_layer():
    # W = 0, b = (ln1, ln2, ln3): softmax = (1/6, 2/6, 3/6) for any input
    dims = (2, 3)
    x = np.zeros(orc.param_count(dims))
    x[6:] = np.log([1.0, 2.0, 3.0])
    Xb = np.array([[0.3, -1.2], [2.0, 0.5]])
    yb = np.array([2, 0])
    loss, g = orc.mlp_loss_grad(x, dims, Xb, yb)
    assert loss == pytest.approx(0.5 * (math.log(2.0) + math.log(6.0)), abs=1e-14)
    p = np.array([1 / 6, 2 / 6, 3 / 6])
    d0 = (p - np.array([0, 0, 1.0])) / 2
    d1 = (p - np.array([1.0, 0, 0])) / 2
    gW = np.outer(d0, Xb[0]) + np.outer(d1, Xb[1])
    assert np.allclose(g[:6].reshape(3, 2), gW, atol=1e-15)
    assert np.allclose(g[6:], d0 + d1, atol=1e-15)


def test_grad_hand_worked_two_layers():
    # x = (1,-2); z1 = (1,-2,-0.5) -> a1 = (1,0,0); z2 = (0, ln3) -> softmax (1/4, 3/4); label 0
    dims = (2, 3, 2)
    W1 = np.array([[1.0, 0.0], [0.0, 1.0], [1.0, 1.0]])
    b1 = np.array([0.0, 0.0, 0.5])
    W2 = np.array([[0.0, 5.0, -7.0], [math.log(3.0), 2.0, 9.0]])
    b2 = np.zeros(2)
    x = np.concatenate([W1.ravel(), b1, W2.ravel(), b2])
    loss, g = orc.mlp_loss_grad(x, dims, np.array([[1.0, -2.0]]), np.array([0]))
    assert loss == pytest.approx(math.log(4.0), abs=1e-14)
    (gW1, gb1), (gW2, gb2) = orc.unpack(g, dims)
    d1 = 0.75 * math.log(3.0)
    assert np.allclose(gW2, [[-0.75, 0, 0], [0.75, 0, 0]], atol=1e-15)
    assert np.allclose(gb2, [-0.75, 0.75], atol=1e-15)
    assert np.allclose(gW1, [[d1, -2 * d1], [0, 0], [0, 0]], atol=1e-15)
    assert np.allclose(gb1, [d1, 0, 0], atol=1e-15)


def test_uniform_logits_give_ln_C_and_zero_sum_delta():
    dims = (5, 7, 10)
    x = np.zeros(orc.param_count(dims))
    rng = np.random.default_rng(0)
    Xb = rng.standard_normal((6, 5))
    yb = rng.integers(0, 10, 6)
    loss, g = orc.mlp_loss_grad(x, dims, Xb, yb)
    assert loss == pytest.approx(math.log(10.0), abs=1e-14)
    gbL = orc.unpack(g, dims)[-1][1]
    assert abs(gbL.sum()) < 1e-15          # sum_c delta_L[b, c] = 0 for every sample
    want = np.full(10, 6 / 10 / 6) - np.bincount(yb, minlength=10) / 6
    assert np.allclose(gbL, want, atol=1e-15)


def test_single_layer_is_multinomial_logistic_regression():
    from scipy.special import log_softmax, softmax
    dims = (9, 4)
    rng = np.random.default_rng(1)
    x = rng.standard_normal(orc.param_count(dims))
    Xb = rng.standard_normal((11, 9))
    yb = rng.integers(0, 4, 11)
    W, b = x[:36].reshape(4, 9), x[36:]
    Z = Xb @ W.T + b
    loss, g = orc.mlp_loss_grad(x, dims, Xb, yb)
    assert loss == pytest.approx(-log_softmax(Z, axis=1)[np.arange(11), yb].mean(), rel=1e-13)
    R = softmax(Z, axis=1)
    R[np.arange(11), yb] -= 1
    assert np.allclose(g[:36].reshape(4, 9), R.T @ Xb / 11, atol=1e-13)
    assert np.allclose(g[36:], R.sum(0) / 11, atol=1e-13)


@pytest.mark.parametrize("dims,B", [((32, 64, 10), 16), ((6, 5, 4, 3), 3)])
def test_gradient_matches_central_differences(dims, B):
    rng = np.random.default_rng(7)
    x = synth.init_params(dims, seed=11).astype(np.float64)
    x += 0.05 * rng.standard_normal(x.shape)          # non-zero biases too
    Xb = rng.standard_normal((B, dims[0]))
    yb = rng.integers(0, dims[-1], B)
    # stay away from ReLU kinks: every hidden pre-activation at least 1e-4 from 0
    a = Xb
    for (W, b) in orc.unpack(x, dims)[:-1]:
        z = a @ W.T + b
        assert np.abs(z).min() > 1e-4
        a = np.maximum(z, 0)
    _, g = orc.mlp_loss_grad(x, dims, Xb, yb)
    fd = np.empty_like(g)
    for j in range(x.size):
        h = 1e-6 * max(1.0, abs(x[j]))
        xp, xm = x.copy(), x.copy()
        xp[j] += h
        xm[j] -= h
        fd[j] = (orc.mlp_loss_grad(xp, dims, Xb, yb)[0] - orc.mlp_loss_grad(xm, dims, Xb, yb)[0]) / (2 * h)
    rel = np.linalg.norm(g - fd) / np.linalg.norm(fd)
    assert rel < 1e-6
    assert np.abs(g - fd).max() < 1e-6 * max(1.0, np.abs(fd).max())


# --------------------------------------------------------- Algorithm 1 schedule
def _quad(a, c):
    return lambda i, t, xi: a[i] * (xi - c[i])


def test_brute_force_two_workers_scalar():
    # F_i(x) = a_i/2 (x - c_i)^2, N=2, m=1, I=2, T=4, worked with scalars
    a, c, g = [1.0, 3.0], [2.0, -1.0], 0.1
    x0 = x1 = 0.5
    for t in range(1, 5):
        x0 = x0 - g * a[0] * (x0 - c[0])
        x1 = x1 - g * a[1] * (x1 - c[1])
        if t % 2 == 0:
            x0 = x1 = (x0 + x1) / 2
    out = orc.pr_sgd(np.full((2, 1), 0.5), g, 2, 4, _quad(np.array(a), np.array(c)[:, None]))
    assert np.allclose(out[:, 0], [x0, x1], atol=1e-15)
    # and one more step leaves the two workers different again
    out5 = orc.pr_sgd(out, g, 2, 1, _quad(np.array(a), np.array(c)[:, None]), t0=4)
    assert out5[0, 0] == pytest.approx(x0 - g * a[0] * (x0 - c[0]), abs=1e-15)
    assert out5[1, 0] == pytest.approx(x1 - g * a[1] * (x1 - c[1]), abs=1e-15)


@pytest.mark.parametrize("I", [1, 3, 5])
def test_quadratic_closed_form_per_period(I):
    rng = np.random.default_rng(3)
    N, m, g = 5, 8, 0.07
    a = rng.uniform(0.5, 2.0, N)
    c = rng.standard_normal((N, m))
    y0 = rng.standard_normal(m)
    x = orc.pr_sgd(np.tile(y0, (N, 1)), g, I, I, _quad(a, c))
    want = np.mean([c[i] + (1 - g * a[i]) ** I * (y0 - c[i]) for i in range(N)], axis=0)
    assert np.allclose(x, want[None, :], atol=1e-13)


def test_quadratic_equal_curvature_independent_of_I():
    rng = np.random.default_rng(4)
    N, m, g, T = 4, 6, 0.1, 24
    c = rng.standard_normal((N, m))
    y0 = rng.standard_normal(m)
    want = c.mean(0) + (1 - g) ** T * (y0 - c.mean(0))
    for I in (1, 2, 4, 8, 24):
        x = orc.pr_sgd(np.tile(y0, (N, 1)), g, I, T, _quad(np.ones(N), c))
        assert np.allclose(x, want[None, :], atol=1e-13)


def _small_mlp_problem(N=3, dims=(6, 5, 4), B=4, P=16, seed=5):
    w = synth.Workload("t", N, dims, B, 0.05, 2, 8, 0, P, mean_shift=0.5, gumbel=True, seed=seed)
    X, Y = synth.make_pools(w)
    x0 = synth.init_params(dims, seed).astype(np.float64)
    return w, X.astype(np.float64), Y, x0


def test_I_equals_1_is_minibatch_sgd_on_the_concatenated_batch():
    # the third equivalent form of parallel mini-batch SGD (Introduction, footnote 1)
    w, X, Y, x0 = _small_mlp_problem()
    T = 6
    out = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, 1, T, orc.mlp_grad_fn(w.dims, X, Y, w.B, w.seed))

    def big_batch(i, t, xi):
        blks = [orc.draw_block(w.seed, k, t, w.n_blocks) for k in range(w.N)]
        Xc = np.concatenate([X[k, b * w.B:(b + 1) * w.B] for k, b in enumerate(blks)])
        Yc = np.concatenate([Y[k, b * w.B:(b + 1) * w.B] for k, b in enumerate(blks)])
        return orc.mlp_loss_grad(xi, w.dims, Xc, Yc)[1]

    single = orc.pr_sgd(x0[None, :], w.gamma, 0, T, big_batch)
    assert np.allclose(out, single, atol=1e-13)
    assert np.abs(out - x0).max() > 1e-3


def test_one_worker_is_plain_sgd_whatever_I():
    w, X, Y, x0 = _small_mlp_problem(N=1)
    fn = orc.mlp_grad_fn(w.dims, X, Y, w.B, w.seed)
    ref = orc.pr_sgd(x0[None, :], w.gamma, 0, 9, fn)
    for I in (1, 2, 4, 9):
        assert np.array_equal(orc.pr_sgd(x0[None, :], w.gamma, I, 9, fn), ref)
    x = x0.copy()
    for t in range(1, 10):                                    # SGD written out
        x = x - w.gamma * fn(0, t, x)
    assert np.allclose(ref[0], x, atol=1e-15)


def test_rows_identical_and_equal_exact_mean_after_average():
    w, X, Y, x0 = _small_mlp_problem(N=5)
    fn = orc.mlp_grad_fn(w.dims, X, Y, w.B, w.seed)
    pre = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, 0, 3, fn)
    assert np.abs(pre[0] - pre[1]).max() > 1e-6
    g4 = np.stack([fn(i, 4, pre[i]) for i in range(w.N)])
    post = orc.pr_sgd(pre, w.gamma, 4, 1, fn, t0=3)
    for i in range(1, w.N):
        assert np.array_equal(post[i], post[0])
    stepped = pre - w.gamma * g4
    exact = np.array([math.fsum(stepped[:, j]) / w.N for j in range(stepped.shape[1])])
    assert np.allclose(post[0], exact, rtol=0, atol=1e-15)
    assert np.allclose(orc.node_average(stepped), exact, rtol=0, atol=1e-15)


@pytest.mark.parametrize("literal", [False, True])
def test_mean_dynamics_telescoping_and_drift_bound(literal):
    w, X, Y, x0 = _small_mlp_problem(N=4)
    I, T = 3, 10
    fn = orc.mlp_grad_fn(w.dims, X, Y, w.B, w.seed)
    log = []
    orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, I, T, fn, literal=literal,
               on_step=lambda t, b, G, a, avg: log.append((t, b, G, a, avg)))
    assert [e[4] for e in log] == [t % I == 0 for t in range(1, T + 1)]
    ybar, acc, gmax, t0 = x0.copy(), np.zeros((w.N, x0.size)), 0.0, 0
    for (t, before, G, after, avg) in log:
        # Eq. (overline-x-update): holds on averaging and non-averaging iterations alike
        assert np.allclose(after.mean(0), before.mean(0) - w.gamma * G.mean(0), atol=1e-14)
        if literal:
            continue
        acc += G
        gmax = max(gmax, np.linalg.norm(G, axis=1).max())
        if avg:
            assert np.allclose(after, (ybar - w.gamma * acc.mean(0))[None, :], atol=1e-13)
            ybar, acc, gmax, t0 = after[0].copy(), np.zeros_like(acc), 0.0, t
        else:
            # proof of Lemma 1: x_i^t = ybar - gamma * sum_{tau=t0+1..t} G_i^tau
            assert np.allclose(after, ybar[None, :] - w.gamma * acc, atol=1e-13)
            drift = np.linalg.norm(after - after.mean(0)[None, :], axis=1).max()
            assert drift <= 2 * w.gamma * (t - t0) * gmax + 1e-12


def test_literal_reading_differs_from_restart_reading():
    w, X, Y, x0 = _small_mlp_problem(N=3)
    fn = orc.mlp_grad_fn(w.dims, X, Y, w.B, w.seed)
    a = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, 2, 4, fn)
    b = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, 2, 4, fn, literal=True)
    assert np.array_equal(a[0], a[1])
    assert np.abs(b[0] - b[1]).max() > 1e-6          # literal form: workers differ after an averaging iteration
    # both agree up to the first averaging iteration's gradient point
    a1 = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, 2, 1, fn)
    b1 = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, 2, 1, fn, literal=True)
    assert np.array_equal(a1, b1)


# ------------------------------------------------ Algorithms 2 and 3 reduce to 1
def test_alg2_schedule_values():
    s = orc.alg2_schedule(2, 27)
    assert s[0] == (1, 2.0)
    assert s[7][0] == 1 and s[7][1] == pytest.approx(2 / 4)
    assert s[26][0] == 2 and s[26][1] == pytest.approx(2 / 9)
    assert orc.alg2_schedule(1, 64)[63] == (4, pytest.approx(1 / 16))


def test_alg2_with_constant_schedule_is_alg1():
    w, X, Y, x0 = _small_mlp_problem(N=3)
    fn = orc.mlp_grad_fn(w.dims, X, Y, w.B, w.seed)
    a = orc.pr_sgd_time_varying(np.tile(x0, (w.N, 1)), [(3, w.gamma)] * 3, fn)
    b = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, 3, 6, fn)      # two full periods, then 3 free steps
    b = orc.pr_sgd(b, w.gamma, 0, 3, fn, t0=6)
    assert np.allclose(a, b, atol=1e-14)


def test_alg2_varying_schedule_matches_the_closed_form_per_epoch():
    """Algorithm 2 with Theorem 2's K^s = ceil(s^(1/3) / N), gamma^s = N / s^(2/3) (scaled) on the quadratic
    instance F_i(x) = a_i/2 |x - c_i|^2: epoch s starts every worker at the node average y of the previous
    epoch's end points and takes K^s gradient steps with rate gamma^s, so x_i = c_i + (1 - gamma^s a_i)^(K^s) (y - c_i).
    The epochs' rates and lengths both change inside the run, so using the wrong epoch's rate (the first one's
    throughout, or the neighbour's) or the wrong epoch length cannot pass."""
    rng = np.random.default_rng(11)
    N, m, S, scale = 2, 5, 30, 0.05
    a, c = rng.uniform(0.5, 2.0, N), rng.standard_normal((N, m))
    start = rng.standard_normal((N, m))                  # workers need not start equal: epoch 1 averages first
    Ks = [math.ceil(round(s ** (1 / 3), 12) / N) for s in range(1, S + 1)]     # written out here, not taken from the oracle
    gs = [scale * N / (s ** (1 / 3)) ** 2 for s in range(1, S + 1)]
    assert Ks[7] == 1 and Ks[8] == 2 and Ks[26] == 2 and Ks[27] == 2 and len(set(Ks)) == 2

    def closed_form(Ks, gs):
        x = start.copy()
        for K, g in zip(Ks, gs):
            y = x.mean(0)
            x = np.stack([c[i] + (1 - g * a[i]) ** K * (y - c[i]) for i in range(N)])
        return x
    sched = [(K, g * scale) for (K, g) in orc.alg2_schedule(N, S)]
    got = orc.pr_sgd_time_varying(start, sched, _quad(a, c))
    assert np.allclose(got, closed_form(Ks, gs), atol=1e-13)
    assert np.abs(got[0] - got[1]).max() > 1e-3          # the end points are not averaged
    # the pin discriminates: the mistakes it is there to catch move the result far beyond the tolerance
    for wrong in (closed_form(Ks, [gs[0]] * S), closed_form(Ks, gs[1:] + gs[-1:]), closed_form(Ks, gs[:1] + gs[:-1]),
                  closed_form([1] * S, gs), closed_form(Ks[1:] + Ks[-1:], gs)):
        assert np.abs(wrong - got).max() > 1e-6


def test_alg3_with_equal_lengths_is_alg1_and_slow_workers_stand_still():
    w, X, Y, x0 = _small_mlp_problem(N=3)
    fn = orc.mlp_grad_fn(w.dims, X, Y, w.B, w.seed)
    a = orc.pr_sgd_heterogeneous(np.tile(x0, (w.N, 1)), w.gamma, [2, 2, 2], 2, fn)
    b = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, 2, 2, fn)
    b = orc.pr_sgd(b, w.gamma, 0, 2, fn, t0=2)
    assert np.allclose(a, b, atol=1e-14)
    h = orc.pr_sgd_heterogeneous(np.tile(x0, (w.N, 1)), w.gamma, [3, 1, 2], 1, fn)
    one = orc.pr_sgd(np.tile(x0, (w.N, 1)), w.gamma, 0, 1, fn)
    assert np.allclose(h[1], one[1], atol=1e-15)                   # worker 1 took exactly one step


# ------------------------------------------------------------- momentum local step
def test_momentum_zero_is_plain_pr_sgd_and_first_step_is_a_gradient_step():
    w, X, Y, x0 = _small_mlp_problem(N=3)
    fn = orc.mlp_grad_fn(w.dims, X, Y, w.B, w.seed)
    xs = np.tile(x0, (w.N, 1))
    a, va = orc.pr_sgd_momentum(xs, np.zeros_like(xs), w.gamma, 0.0, 2, 6, fn)
    assert np.allclose(a, orc.pr_sgd(xs, w.gamma, 2, 6, fn), atol=1e-15)
    b, vb = orc.pr_sgd_momentum(xs, np.zeros_like(xs), w.gamma, 0.9, 0, 1, fn)
    assert np.allclose(b, orc.pr_sgd(xs, w.gamma, 0, 1, fn), atol=1e-15)     # v^1 = G^1
    assert np.allclose(vb, (xs - b) / w.gamma, atol=1e-12)


def test_momentum_on_a_quadratic_matches_the_linear_recurrence():
    # F(x) = a/2 (x - c)^2:  (x, v)_{t} = M (x - c, v)_{t-1},  M = [[1 - gamma a, -gamma mu], [a, mu]]
    a, c, gam, mu, T = 1.7, 0.4, 0.1, 0.9, 25
    x, v = orc.pr_sgd_momentum(np.array([[2.0]]), np.zeros((1, 1)), gam, mu, 0, T, lambda i, t, xi: a * (xi - c))
    M = np.array([[1 - gam * a, -gam * mu], [a, mu]])
    want = np.linalg.matrix_power(M, T) @ np.array([2.0 - c, 0.0])
    assert x[0, 0] == pytest.approx(want[0] + c, abs=1e-13) and v[0, 0] == pytest.approx(want[1], abs=1e-13)


def test_momentum_brute_force_and_velocity_choices():
    a, c, g, mu = np.array([1.0, 3.0]), np.array([[2.0], [-1.0]]), 0.1, 0.5
    x0_, x1_, v0_, v1_ = 0.5, 0.5, 0.0, 0.0
    for t in range(1, 5):
        v0_ = mu * v0_ + a[0] * (x0_ - c[0, 0]); x0_ = x0_ - g * v0_
        v1_ = mu * v1_ + a[1] * (x1_ - c[1, 0]); x1_ = x1_ - g * v1_
        if t % 2 == 0:
            x0_ = x1_ = (x0_ + x1_) / 2
    x, v = orc.pr_sgd_momentum(np.full((2, 1), 0.5), np.zeros((2, 1)), g, mu, 2, 4, _quad(a, c))
    assert np.allclose(x[:, 0], [x0_, x1_], atol=1e-15) and np.allclose(v[:, 0], [v0_, v1_], atol=1e-15)
    assert abs(v[0, 0] - v[1, 0]) > 1e-3                         # local momentum: buffers differ after the average
    x2, v2 = orc.pr_sgd_momentum(np.full((2, 1), 0.5), np.zeros((2, 1)), g, mu, 2, 4, _quad(a, c), average_velocity=True)
    assert v2[0, 0] == v2[1, 0] and x2[0, 0] == x2[1, 0]
    # mean dynamics with momentum on a non-averaging iteration: xbar moves by -gamma * mean(v)
    x3, v3 = orc.pr_sgd_momentum(x, v, g, mu, 2, 1, _quad(a, c), t0=4)
    assert np.allclose(x3.mean(0), x.mean(0) - g * v3.mean(0), atol=1e-15)


def test_averaged_momentum_buffers_value_pins():
    """average_velocity=True.  (a) Equal curvature: per worker (x_i - c_i, v_i) <- M (x_i - c_i, v_i) with
    M = [[1 - gamma a, -gamma mu], [a, mu]]; the map is linear, so the worker mean obeys it with c replaced by
    the mean of the c_i, and after an averaging iteration with averaged buffers EVERY worker holds that mean
    state: x_i = cbar + (M^T z0)_0, v_i = (M^T z0)_1 with z0 = (y0 - cbar, 0).  (b) Different curvatures:
    scalar recurrences worked in the test, buffers averaged by hand at t = 2, 4."""
    rng = np.random.default_rng(12)
    N, m, a, gam, mu, I, T = 4, 3, 1.3, 0.1, 0.9, 3, 9
    c, y0 = rng.standard_normal((N, m)), rng.standard_normal(m)
    x, v = orc.pr_sgd_momentum(np.tile(y0, (N, 1)), np.zeros((N, m)), gam, mu, I, T, _quad(np.full(N, a), c),
                               average_velocity=True)
    M = np.linalg.matrix_power(np.array([[1 - gam * a, -gam * mu], [a, mu]]), T)
    cbar = c.mean(0)
    want_x, want_v = cbar + M[0, 0] * (y0 - cbar), M[1, 0] * (y0 - cbar)
    assert np.allclose(x, want_x[None, :], atol=1e-13) and np.allclose(v, want_v[None, :], atol=1e-13)
    xl, vl = orc.pr_sgd_momentum(np.tile(y0, (N, 1)), np.zeros((N, m)), gam, mu, I, T, _quad(np.full(N, a), c))
    assert np.allclose(xl, want_x[None, :], atol=1e-13)           # same models (linear map, equal curvature) ...
    assert np.abs(vl - want_v[None, :]).max() > 1e-3              # ... but local buffers stay apart
    assert np.allclose(vl.mean(0), want_v, atol=1e-13)
    # (b)
    aa, cc, g, mu2 = [1.0, 3.0], [2.0, -1.0], 0.1, 0.5
    x0_ = x1_ = 0.5
    v0_ = v1_ = 0.0
    for t in range(1, 5):
        v0_ = mu2 * v0_ + aa[0] * (x0_ - cc[0]); x0_ -= g * v0_
        v1_ = mu2 * v1_ + aa[1] * (x1_ - cc[1]); x1_ -= g * v1_
        if t % 2 == 0:
            x0_ = x1_ = (x0_ + x1_) / 2
            v0_ = v1_ = (v0_ + v1_) / 2
    x2, v2 = orc.pr_sgd_momentum(np.full((2, 1), 0.5), np.zeros((2, 1)), g, mu2, 2, 4,
                                 _quad(np.array(aa), np.array(cc)[:, None]), average_velocity=True)
    assert np.allclose(x2[:, 0], [x0_, x1_], atol=1e-15) and np.allclose(v2[:, 0], [v0_, v1_], atol=1e-15)
    xk, _ = orc.pr_sgd_momentum(np.full((2, 1), 0.5), np.zeros((2, 1)), g, mu2, 2, 4,
                                _quad(np.array(aa), np.array(cc)[:, None]))
    assert abs(xk[0, 0] - x2[0, 0]) > 1e-4                        # with different curvatures the choice changes the models


# ------------------------------------------------------- planted mistakes are caught
def test_pins_catch_a_planted_mistake(monkeypatch):
    rng = np.random.default_rng(3)
    N, m, g, I = 5, 8, 0.07, 3
    a, c, y0 = rng.uniform(0.5, 2.0, N), rng.standard_normal((N, m)), rng.standard_normal(m)
    want = np.mean([c[i] + (1 - g * a[i]) ** I * (y0 - c[i]) for i in range(N)], axis=0)
    monkeypatch.setattr(orc, "node_average", lambda x: x.sum(0) / (x.shape[0] - 1))
    bad = orc.pr_sgd(np.tile(y0, (N, 1)), g, I, I, _quad(a, c))
    assert not np.allclose(bad, want[None, :], atol=1e-6)
