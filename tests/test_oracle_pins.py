"""Pins for the fp64 CPU oracle: it is checked against things other than itself.

Closed forms, invariants the paper states, library witnesses (numpy mean,
torch.optim, pandas ewm, scipy logsumexp), brute force on tiny inputs and the
few numbers the paper prints (tests/golden/paper_examples.txt).  Each pin is
chosen so that a plausible slip in oracle/ref_oracle.c -- a dropped term, a
wrong sign or index, a transposed operand, a stray 1/K -- fails it.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2305_12213_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_examples.txt")


def _grads(K, n, seed=7, std=1.0):
    return [g.numpy() for g in inputs.worker_gradients(K, n, std, seed)]


def _state(n, seed=99):
    p = inputs.normal(n, 0.02, seed).numpy().astype(np.float64)
    v = inputs.normal(n, 0.5, seed + 1).numpy().astype(np.float64)
    return p, v


# ---------------------------------------------------------------- weights, Eq. 2
def test_weights_sum_to_one_and_are_proportional():
    b = [16, 32, 80]
    lam = oracle.weights(b)
    assert abs(lam.sum() - 1.0) < 1e-15
    assert np.allclose(lam / lam[0], np.array(b) / b[0], rtol=1e-15)


def test_weights_reject_bad_batches():
    with pytest.raises(oracle.OracleError):
        oracle.weights([0, 0])
    with pytest.raises(oracle.OracleError):
        oracle.weights([4, -1])


# ---------------------------------------------------------------- aggregate, Eq. 2-3
@pytest.mark.parametrize("K", [1, 2, 3, 5, 8])
def test_equal_batches_reduce_to_plain_mean(K):
    """Eq. 1: with uniform batches the parameter server takes the plain average."""
    n = 257
    gs = _grads(K, n)
    p, v = np.zeros(n), np.zeros(n)
    g, _ = oracle.aggregate_update(gs, [32] * K, p, v, lr=1.0, mu=0.0, want_g=True)
    mean = np.mean(np.stack(gs).astype(np.float64), axis=0)
    assert np.allclose(g, mean, rtol=1e-14, atol=1e-16)
    # mu = 0, lr = 1, p0 = 0  =>  p = -g, v = g   (plain SGD step)
    assert np.array_equal(v, g) and np.array_equal(p, -g)


def test_single_worker_is_identity():
    n = 100
    gs = _grads(1, n)
    p, v = np.zeros(n), np.zeros(n)
    g, _ = oracle.aggregate_update(gs, [7], p, v, 1.0, 0.0, want_g=True)
    assert np.array_equal(g, gs[0].astype(np.float64))


def test_scaling_all_batches_changes_nothing():
    n = 300
    gs = _grads(4, n)
    outs = []
    for c in (1, 3, 10):
        p, v = _state(n)
        g, sq = oracle.aggregate_update(gs, [c * x for x in (24, 40, 64, 128)], p, v,
                                        0.1, 0.9, want_g=True)
        outs.append((g, p, v, sq))
    for o in outs[1:]:
        for a, b_ in zip(o[:3], outs[0][:3]):
            assert np.array_equal(a, b_)
        assert math.isclose(o[3], outs[0][3], rel_tol=1e-14)   # threaded sum order


def test_unequal_batches_weighted_not_uniform():
    """A worker with 3x the batch must count 3x: the uniform mean is a different number."""
    g0 = np.full(8, 1.0, dtype=np.float32)
    g1 = np.full(8, 5.0, dtype=np.float32)
    p, v = np.zeros(8), np.zeros(8)
    g, sq = oracle.aggregate_update([g0, g1], [30, 10], p, v, 1.0, 0.0, want_g=True)
    assert np.array_equal(g, np.full(8, 2.0))          # (30*1 + 10*5)/40
    assert sq == 8 * 4.0


def test_zero_batch_worker_is_never_read():
    n = 64
    gs = _grads(3, n)
    poisoned = [gs[0], np.full(n, np.nan, dtype=np.float32), gs[2]]
    p1, v1 = _state(n)
    p2, v2 = _state(n)
    g1, s1 = oracle.aggregate_update(poisoned, [5, 0, 9], p1, v1, 0.1, 0.9, want_g=True)
    g2, s2 = oracle.aggregate_update([gs[0], gs[2]], [5, 9], p2, v2, 0.1, 0.9, want_g=True)
    assert np.array_equal(g1, g2) and np.array_equal(p1, p2)
    assert math.isclose(s1, s2, rel_tol=1e-14)


def test_grad_sqnorm_closed_forms():
    n = 1000
    ones = [np.ones(n, dtype=np.float32)] * 4
    p, v = np.zeros(n), np.zeros(n)
    _, sq = oracle.aggregate_update(ones, [1, 2, 3, 4], p, v, 0.1, 0.9)
    assert abs(sq - n) < 1e-9
    gs = _grads(3, n)
    p, v = np.zeros(n), np.zeros(n)
    g, sq = oracle.aggregate_update(gs, [3, 4, 5], p, v, 0.1, 0.9, want_g=True)
    assert math.isclose(sq, float(np.dot(g, g)), rel_tol=1e-13)


def test_bf16_gradients_widen_exactly():
    n = 513
    g32 = inputs.worker_gradients(3, n, 1e-3, 11)
    g16 = [g.to(torch.bfloat16) for g in g32]
    as_bits = [inputs.bf16_bits(g) for g in g16]
    as_f32 = [g.to(torch.float32).numpy() for g in g16]
    pa, va = _state(n)
    pb, vb = _state(n)
    ga, sa = oracle.aggregate_update(as_bits, [8, 16, 40], pa, va, 0.05, 0.9, want_g=True)
    gb, sb = oracle.aggregate_update(as_f32, [8, 16, 40], pb, vb, 0.05, 0.9, want_g=True)
    assert np.array_equal(ga, gb) and np.array_equal(pa, pb) and np.array_equal(va, vb)
    assert math.isclose(sa, sb, rel_tol=1e-14)


# ---------------------------------------------------------------- momentum
def test_heavy_ball_matches_torch_sgd():
    """Witness: torch.optim.SGD(momentum, dampening 0, no Nesterov) in fp64 on CPU."""
    n, K, steps = 97, 3, 6
    b = [16, 32, 80]
    lam = np.array(b, dtype=np.float64) / sum(b)
    p0 = inputs.normal(n, 0.02, 5).numpy().astype(np.float64)
    w = torch.tensor(p0.copy(), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.SGD([w], lr=0.1, momentum=0.9, dampening=0.0, nesterov=False)
    p, v = p0.copy(), np.zeros(n)
    for it in range(steps):
        gs = [g.numpy() for g in inputs.worker_gradients(K, n, 1.0, 300, it)]
        oracle.aggregate_update(gs, b, p, v, 0.1, 0.9)
        agg = sum(l * g.astype(np.float64) for l, g in zip(lam, gs))
        w.grad = torch.tensor(agg)
        opt.step()
    assert np.allclose(p, w.detach().numpy(), rtol=1e-12, atol=1e-14)


def test_heavy_ball_constant_gradient_closed_form():
    """Constant g: v_t = g (1 - mu^t)/(1 - mu); p_t = p_0 - lr * sum_{s<=t} v_s."""
    n, mu, lr, T = 5, 0.9, 0.1, 12
    g = np.array([1.0, -2.0, 0.5, 0.0, 3.0], dtype=np.float32)
    p, v = np.zeros(n), np.zeros(n)
    acc = np.zeros(n)
    for t in range(1, T + 1):
        oracle.aggregate_update([g, g], [3, 9], p, v, lr, mu)
        vt = g.astype(np.float64) * (1 - mu ** t) / (1 - mu)
        acc += vt
        assert np.allclose(v, vt, rtol=1e-13)
        assert np.allclose(p, -lr * acc, rtol=1e-12)


def test_no_stray_one_over_K_in_the_step():
    """Reading of Eq. 3: the step is lr * weighted mean, not lr/K times it."""
    g = np.ones(4, dtype=np.float32)
    p, v = np.zeros(4), np.zeros(4)
    oracle.aggregate_update([g] * 5, [2] * 5, p, v, 0.5, 0.0)
    assert np.array_equal(p, np.full(4, -0.5))


# ---------------------------------------------------------------- Adam
def test_adam_matches_torch_adam():
    n, K, steps = 61, 2, 5
    b = [10, 30]
    lam = np.array(b, dtype=np.float64) / sum(b)
    p0 = inputs.normal(n, 0.02, 6).numpy().astype(np.float64)
    w = torch.tensor(p0.copy(), dtype=torch.float64, requires_grad=True)
    opt = torch.optim.Adam([w], lr=1e-4, betas=(0.9, 0.999), eps=1e-8)
    p, m, u = p0.copy(), np.zeros(n), np.zeros(n)
    for it in range(steps):
        gs = [g.numpy() for g in inputs.worker_gradients(K, n, 1.0, 400, it)]
        oracle.aggregate_adam(gs, b, p, m, u, 1e-4, 0.9, 0.999, 1e-8, it + 1)
        w.grad = torch.tensor(sum(l * g.astype(np.float64) for l, g in zip(lam, gs)))
        opt.step()
    assert np.allclose(p, w.detach().numpy(), rtol=1e-10, atol=1e-14)


def test_adam_reports_the_aggregate_and_its_squared_norm():
    """The Adam call returns the same g and sum g^2 as the momentum call: g_k = c_k everywhere gives
    g = sum lambda_k c_k and ||g||^2 = n g^2."""
    n, b, c = 37, [1, 3], [2.0, -6.0]                      # g = 0.25 * 2 - 0.75 * 6 = -4
    gs = [np.full(n, v, dtype=np.float32) for v in c]
    p, m, u = np.zeros(n), np.zeros(n), np.zeros(n)
    g, sq = oracle.aggregate_adam(gs, b, p, m, u, 1e-3, 0.9, 0.999, 1e-8, 1, want_g=True)
    assert np.array_equal(g, np.full(n, -4.0)) and sq == 16.0 * n
    # first step of Adam from zero state: mhat = g, uhat = g^2, so p = -lr * g / (|g| + eps)
    assert np.allclose(p, 1e-3 * 4.0 / (4.0 + 1e-8), rtol=1e-14)


# ---------------------------------------------------------------- linear-softmax gradient
def _brute_force_grad(X, y, W):
    """Per-sample definition in fp64: mean_i outer(x_i, softmax(x_i W) - onehot(y_i))."""
    X = X.astype(np.float64)
    W = W.astype(np.float64)
    n, D = X.shape
    C = W.shape[1]
    G = np.zeros((D, C))
    for i in range(n):
        z = np.array([sum(X[i, d] * W[d, c] for d in range(D)) for c in range(C)])
        e = np.exp(z - z.max())
        pr = e / e.sum()
        pr[y[i]] -= 1.0
        for d in range(D):
            for c in range(C):
                G[d, c] += X[i, d] * pr[c]
    return G / n


def _loss(X, y, W):
    from scipy.special import logsumexp
    Z = X.astype(np.float64) @ W
    return float(np.mean(logsumexp(Z, axis=1) - Z[np.arange(len(y)), y]))


def test_worker_grad_matches_per_sample_definition():
    X, y, W = inputs.softmax_problem([5], 6, 4, seed=21, w_std=0.5)
    X, y, W = X.numpy(), y.numpy(), W.numpy()
    G, loss = oracle.worker_grad(X, y, W)
    assert np.allclose(G, _brute_force_grad(X, y, W), rtol=1e-12, atol=1e-15)
    assert math.isclose(loss, _loss(X, y, W.astype(np.float64)), rel_tol=1e-12)


def test_worker_grad_is_the_derivative_of_the_loss():
    X, y, W = inputs.softmax_problem([7], 5, 3, seed=22, w_std=0.3)
    X, y, W = X.numpy(), y.numpy(), W.numpy()
    G, _ = oracle.worker_grad(X, y, W)
    W64 = W.astype(np.float64)
    h = 1e-6
    for d, c in itertools.product(range(5), range(3)):
        Wp, Wm = W64.copy(), W64.copy()
        Wp[d, c] += h
        Wm[d, c] -= h
        fd = (_loss(X, y, Wp) - _loss(X, y, Wm)) / (2 * h)
        assert abs(fd - G[d, c]) < 1e-8


def test_worker_grad_rows_sum_to_zero():
    X, y, W = inputs.softmax_problem([9], 16, 10, seed=23)
    G, _ = oracle.worker_grad(X.numpy(), y.numpy(), W.numpy())
    assert np.abs(G.sum(axis=1)).max() < 1e-15


def test_weighted_aggregate_equals_concatenated_batch_gradient():
    """Section 3.1: batch-proportional weights make the aggregate of per-worker mean
    gradients the mean gradient of the whole global batch (brute force, tiny sizes)."""
    bs = [1, 2, 5, 3]
    D, C = 4, 3
    X, y, W = inputs.softmax_problem(bs, D, C, seed=31, w_std=0.4)
    X, y, W = X.numpy(), y.numpy(), W.numpy()
    offs = np.concatenate([[0], np.cumsum(bs)])
    per_worker = [oracle.worker_grad(X[offs[i]:offs[i + 1]], y[offs[i]:offs[i + 1]], W)[0]
                  for i in range(len(bs))]
    # the aggregation oracle takes fp32 gradients; use exactly representable ones
    g32 = [g.astype(np.float32).reshape(-1) for g in per_worker]
    p, v = np.zeros(D * C), np.zeros(D * C)
    agg, _ = oracle.aggregate_update(g32, bs, p, v, 1.0, 0.0, want_g=True)
    full = _brute_force_grad(X, y, W).reshape(-1)
    assert np.allclose(agg, full, rtol=0, atol=2e-7)     # fp32 storage of the inputs
    # and in exact arithmetic on the fp64 gradients
    lam = oracle.weights(bs)
    exact = sum(l * g for l, g in zip(lam, per_worker)).reshape(-1)
    assert np.allclose(exact, full, rtol=1e-12, atol=1e-15)
    # the uniform average is measurably wrong here, so the pin has teeth
    uniform = np.mean(np.stack(per_worker), axis=0).reshape(-1)
    assert np.abs(uniform - full).max() > 1e-3


# ---------------------------------------------------------------- controller, Eq. 4-5
def test_controller_fixed_point():
    """All iteration times equal (b proportional to X) => no change."""
    for kp in (0.5, 1.0):
        assert oracle.controller_step([16, 32, 80], [1.0, 2.0, 5.0], kp).tolist() == [16, 32, 80]


def test_controller_one_step_closed_form():
    """Section 3.3: b1_k = b0_k * tbar / t_k; rescaled to the global batch this is S X_k / sum X."""
    b = np.array([32, 32, 32, 32])
    X = np.array([3.0, 9.0, 18.0, 6.0])
    t = b / X
    simplified = b * t.mean() / t
    q = oracle.controller_targets(b, X, 1.0)
    assert np.allclose(q / q.sum(), simplified / simplified.sum(), rtol=1e-14)
    assert np.allclose(q, b.sum() * X / X.sum(), rtol=1e-14)
    assert math.isclose(q.sum(), b.sum(), rel_tol=1e-14)


def test_controller_deviation_contracts_geometrically():
    """With fixed throughputs the distance e = b - S X / sum X obeys
    e' = (1-kp) s e,  s = S / (S + kp m sum X),  m = mean(e_k / X_k)."""
    b = np.array([40, 25, 63, 12, 116])
    X = np.array([1.5, 0.7, 2.2, 4.0, 3.1])
    S, kp = b.sum(), 0.35
    e = b - S * X / X.sum()
    m = np.mean(e / X)
    s = S / (S + kp * m * X.sum())
    q = oracle.controller_targets(b, X, kp)
    assert np.allclose(q - S * X / X.sum(), (1 - kp) * s * e, rtol=1e-12, atol=1e-12)


def test_controller_direction():
    """Slower-than-average workers shrink, faster ones grow (text below Eq. 5)."""
    b = np.array([32, 32, 32])
    X = np.array([1.0, 4.0, 10.0])
    t = b / X
    nb = oracle.controller_step(b, X, 1.0)
    assert nb[np.argmax(t)] < 32 and nb[np.argmin(t)] > 32
    assert nb.sum() == b.sum()


@pytest.mark.parametrize("seed", range(20))
def test_controller_conserves_global_batch_and_bounds(seed):
    K = 2 + seed % 9
    b = inputs.batch_sizes_uniform(K, 8, 256, seed)
    X = inputs.lognormal_throughputs(K, 0.5, seed + 100)
    for kp in (0.25, 0.5, 1.0):
        nb = oracle.controller_step(b, X, kp)
        assert nb.sum() == sum(b) and nb.min() >= 1


def test_controller_converges_to_throughput_proportional():
    """Fig. 4a: from a uniform start the batch sizes settle within two adjustments."""
    X = [10.0] * 4 + [1.0] * 4
    b = oracle.controller_step([32] * 8, X, 1.0)
    assert b.tolist() == [58] * 4 + [6] * 4          # 256*10/44 = 58.18, 256/44 = 5.8
    assert oracle.controller_step(b, X, 1.0).tolist() == b.tolist()
    half = [32] * 8
    seen = []
    for _ in range(6):
        half = oracle.controller_step(half, X, 0.5)
        seen.append((int(half[0]), int(half[7])))
    assert seen[:4] == [(52, 12), (56, 8), (57, 7), (58, 6)] and seen[-1] == (58, 6)


def _brute_force_best(q, S, lo, hi):
    best = None
    for cand in itertools.product(*[range(l, h + 1) for l, h in zip(lo, hi)]):
        if sum(cand) != S:
            continue
        cost = sum((c - x) ** 2 for c, x in zip(cand, q))
        if best is None or cost < best - 1e-12:
            best = cost
    return best


def test_integer_apportionment_is_optimal_exhaustively():
    """Enumerate every feasible integer vector for tiny K, S: the controller's rounding
    attains the least squared (and hence least max) distance to the real targets."""
    rng = np.random.default_rng(0)
    for trial in range(150):
        K = int(rng.integers(2, 5))
        b = rng.integers(1, 5, size=K)
        S = int(b.sum())
        X = rng.uniform(0.2, 5.0, size=K)
        kp = float(rng.choice([0.3, 0.5, 1.0]))
        lo = rng.integers(0, 2, size=K) if trial % 3 == 0 else np.ones(K, dtype=int)
        if trial % 5 == 1:
            lo = rng.integers(0, 4, size=K)          # lower bounds above the targets: units must be taken back
        hi = np.minimum(rng.integers(2, 9, size=K), S) if trial % 2 == 0 else np.full(K, S)
        hi = np.maximum(hi, lo)
        q = oracle.controller_targets(b, X, kp)
        feasible = lo.sum() <= S <= hi.sum()
        if not feasible:
            with pytest.raises(oracle.OracleError) as ei:
                oracle.controller_step(b, X, kp, lo, hi)
            assert ei.value.code == oracle.REF_ERR_INFEASIBLE
            continue
        nb = oracle.controller_step(b, X, kp, lo, hi)
        assert nb.sum() == S and (nb >= lo).all() and (nb <= hi).all()
        cost = float(((nb - q) ** 2).sum())
        assert cost <= _brute_force_best(q, S, lo, hi) + 1e-9


def test_apportionment_takes_surplus_units_back():
    """Lower bounds above the real targets leave too many units after the first pass; they come back from
    the workers above their lower bound, largest excess over the target first.
    (a) b = (4, 4, 4), X = (1, 1, 10): q = (1, 1, 10).  With b_min = (3, 1, 1) the start is (3, 1, 10) = 14;
        workers 0 and 1 sit on their bounds, so both units come from worker 2: (3, 1, 8).
    (b) X = (12, 13, 71), S = 24: q = X / 4 = (3, 3.25, 17.75) exactly.  With b_min = (5, 1, 1) the start is
        (5, 3, 17) = 25.  Worker 0 has the largest excess (2) but is on its bound; of the others worker 1
        (excess -0.25) gives the unit, not worker 2 (-0.75): (5, 2, 17), the nearest feasible vector.
    (c) q = (3, 3, 18), b_min = (6, 1, 1): start (6, 3, 18) = 27; equal excesses go lowest index first:
        worker 1, then worker 2 (0 against -1), then worker 1 again: (6, 1, 17)."""
    q = oracle.controller_targets([4, 4, 4], [1.0, 1.0, 10.0], 1.0)
    assert np.abs(q - [1.0, 1.0, 10.0]).max() < 1e-12
    assert oracle.controller_step([4, 4, 4], [1.0, 1.0, 10.0], 1.0, [3, 1, 1], [12, 12, 12]).tolist() == [3, 1, 8]
    assert oracle.static_allocate([12.0, 13.0, 71.0], 8, [5, 1, 1], [24, 24, 24]).tolist() == [5, 2, 17]
    assert oracle.static_allocate([1.0, 1.0, 6.0], 8, [6, 1, 1], [24, 24, 24]).tolist() == [6, 1, 17]


def test_apportionment_ties_go_to_lowest_index():
    # q = (2.5, 2.5, 7.5, 7.5): two spare units, four equal remainders
    assert oracle.static_allocate([1, 1, 3, 3], 5).tolist() == [3, 3, 7, 7]
    # q = (2.5, 2.5, 2.5, 2.5) from b = (2, 2, 3, 3) with equal throughputs
    assert oracle.controller_step([2, 2, 3, 3], [1.0, 1.0, 1.0, 1.0], 1.0).tolist() == [3, 3, 2, 2]


def test_without_bounds_every_worker_keeps_at_least_one_sample():
    """A worker 1000 times slower has a real target of 16/1001 < 0.5; with no bounds given it still
    holds one sample (a worker with b = 0 would drop out of the job), and b_min = 0 allows the zero."""
    assert oracle.controller_step([8, 8], [1000.0, 1.0], 1.0).tolist() == [15, 1]
    assert oracle.controller_step([8, 8], [1000.0, 1.0], 1.0, [0, 0], [16, 16]).tolist() == [16, 0]
    assert oracle.static_allocate([1000.0, 1.0], 8).tolist() == [15, 1]


def test_controller_rejects_bad_arguments():
    for bad in ([1.0, 0.0], [1.0, -2.0], [1.0, float("nan")], [1.0, float("inf")]):
        with pytest.raises(oracle.OracleError):
            oracle.controller_step([4, 4], bad, 1.0)
    for kp in (0.0, -0.5, 1.5, float("nan")):
        with pytest.raises(oracle.OracleError):
            oracle.controller_step([4, 4], [1.0, 2.0], kp)


# ---------------------------------------------------------------- the paper's printed numbers
def _golden():
    rows = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if not line:
                continue
            name, xs, total, expect = [s.strip() for s in line.split("|")]
            rows.append((name, [float(x) for x in xs.split()], int(total),
                         [int(x) for x in expect.split()]))
    return rows


@pytest.mark.parametrize("name,X,total,expect", _golden())
def test_static_allocation_on_the_papers_clusters(name, X, total, expect):
    K = len(X)
    assert total % K == 0
    b = oracle.static_allocate(X, total // K)
    assert b.tolist() == expect and b.sum() == total
    # throughput-proportional start is a fixed point of the controller when X is exact
    q = oracle.controller_targets(b, X, 1.0)
    assert np.abs(q - total * np.array(X) / sum(X)).max() < 1e-9


# ---------------------------------------------------------------- stabilised controller
def test_ewma_matches_pandas():
    import pandas as pd
    K, alpha = 3, 0.3
    st = oracle.ControllerState([32, 32, 32], kp=1.0, alpha=alpha, dmin=1e9)  # never readjust
    rng = np.random.default_rng(3)
    T = rng.uniform(0.5, 2.0, size=(10, K))
    for row in T:
        assert st.observe(row) is False
    want = pd.DataFrame(T).ewm(alpha=alpha, adjust=False).mean().to_numpy()[-1]
    assert np.allclose(st.ewma, want, rtol=1e-13)
    assert st.b.tolist() == [32, 32, 32]


def test_dead_band_holds_small_changes_and_passes_large_ones():
    """Threshold 0.05 (the paper's value): a 3 % imbalance is ignored, a 2x one is not."""
    st = oracle.ControllerState([100, 100], kp=1.0, alpha=1.0, dmin=0.05)
    assert st.observe([1.00, 1.03]) is False and st.b.tolist() == [100, 100]
    assert st.observe([1.0, 2.0]) is True
    assert st.b.tolist() == [133, 67] and int(st.n_since[0]) == 0


def test_dead_band_measures_the_largest_relative_move_against_the_current_batch():
    """Section 3.3.1, step 4: max_k |b'_k - b_k| / b_k > dmin, strictly, relative to the batch in use.
    (a) The largest relative move may be a decrease: b = (100, 10) -> (101, 9) is +1 % and -10 %.
    (b) b = (20, 20) -> (21, 19) moves both workers by exactly 1/20 = 0.05: not above 0.05, nothing
        changes (measured against the new batch 1/19 > 0.05 would readjust).
    (c) b = (20, 20) -> (19, 21) likewise; one more unit, (22, 18), is 10 % and readjusts."""
    # (a) times chosen so that the targets are q = (101, 9): X proportional to (101, 9)
    st = oracle.ControllerState([100, 10], kp=1.0, alpha=1.0, dmin=0.05)
    assert st.observe([100 / 101.0, 10 / 9.0]) is True and st.b.tolist() == [101, 9]
    # (b), (c)
    for X, moved in (((21.0, 19.0), [21, 19]), ((19.0, 21.0), [19, 21])):
        assert oracle.controller_step([20, 20], X, 1.0).tolist() == moved
        st = oracle.ControllerState([20, 20], kp=1.0, alpha=1.0, dmin=0.05)
        assert st.observe([20 / X[0], 20 / X[1]]) is False and st.b.tolist() == [20, 20]
    st = oracle.ControllerState([20, 20], kp=1.0, alpha=1.0, dmin=0.05)
    assert st.observe([20 / 22.0, 20 / 18.0]) is True and st.b.tolist() == [22, 18]


def test_dead_band_stops_oscillation_under_noise():
    """Fig. 4b: without a dead-band noisy times keep moving the batch sizes; with it they rest."""
    rng = np.random.default_rng(5)
    X = np.array([1.0, 2.0, 4.0])
    moves = {}
    for dmin in (0.0, 0.05):
        st = oracle.ControllerState([64, 64, 64], kp=1.0, alpha=0.5, dmin=dmin)
        rng = np.random.default_rng(5)
        n = 0
        for it in range(60):
            t = st.b / X * (1.0 + 0.01 * rng.standard_normal(3))
            n += st.observe(t) and it >= 5
        moves[dmin] = n
        assert st.b.sum() == 192
    assert moves[0.05] == 0 and moves[0.0] > 0


def test_adaptive_upper_bound_learns_from_a_throughput_drop():
    """Fig. 5 / "Batch size bounds": worker 0's throughput collapses above a batch of 100 (memory limit).
    Without learning the controller keeps pushing it over the cliff; with it the bound b_max = the last
    good batch is learnt and the batch stays at or below it."""
    def times(b):
        X0 = 10.0 if b[0] <= 100 else 4.0
        return [b[0] / X0, b[1] / 2.0]

    st = oracle.ControllerState([64, 64], kp=1.0, alpha=1.0, dmin=0.0, adaptive=True)
    history = []
    for _ in range(8):
        st.observe(times(st.b))
        history.append(int(st.b[0]))
    assert history[0] > 100                      # first adjustment overshoots the cliff (10:2 split of 128)
    assert int(st.learnt_max[0]) == 64           # the drop is seen: back to the last batch that ran well
    assert max(history[2:]) <= 64 and st.b.sum() == 128
    plain = oracle.ControllerState([64, 64], kp=1.0, alpha=1.0, dmin=0.0, adaptive=False)
    seen = []
    for _ in range(8):
        plain.observe(times(plain.b))
        seen.append(int(plain.b[0]))
    assert max(seen[2:]) > 100                   # without the learnt bound it keeps crossing the cliff


def _trace(st, rows):
    """Feed iteration times row by row; return (b, learnt_max) after each observation."""
    out = []
    for t in rows:
        st.observe(t)
        out.append((st.b.tolist(), st.learnt_max.tolist()))
    return out


def test_infeasible_learnt_bounds_fall_back_to_the_users_bounds():
    """Section 3.3.1, "Batch size bounds", worked by hand (kp = 1, alpha = 1, no dead-band, so every
    observation readjusts and b' = round(100 * X_k / sum X) within the bounds in force; X_k = b_k / t_k).

    obs 1  b = (40, 60), t = (8, 16)      X = (5, 3.75)  q = (57.14, 42.86)            -> (57, 43)
    obs 2  b = (57, 43), t = (19, 10.75)  X = (3, 4): worker 0 was raised 40 -> 57 and fell from 5 to 3,
           so its bound becomes 40.      q = (42.86, 57.14), capped at (40, 100)       -> (40, 60)
    obs 3  b = (40, 60), t = (8, 24)      X = (5, 2.5): worker 1 was raised 43 -> 60 and fell from 4 to
           2.5, so its bound becomes 43.  40 + 43 < 100: the learnt bounds cannot hold the global batch,
           the user's bounds (65, 100) alone apply.  q = (66.67, 33.33), capped at 65  -> (65, 35)
    """
    st = oracle.ControllerState([40, 60], kp=1.0, alpha=1.0, dmin=0.0, b_max=[65, 100], adaptive=True)
    got = _trace(st, [[8.0, 16.0], [19.0, 10.75], [8.0, 24.0]])
    assert got == [([57, 43], [0, 0]), ([40, 60], [40, 0]), ([65, 35], [40, 43])]


def test_a_second_drop_lowers_a_learnt_bound():
    """Same rules, five observations by hand: the bound learnt at 40 drops to 25 when a later raise
    from 25 also lowers the throughput, and a raise that does not lower it teaches nothing.

    obs 1  (40, 60), t = (8, 16)       X = (5, 3.75)                                   -> (57, 43)
    obs 2  (57, 43), t = (19, 10.75)   X = (3, 4)     bound_0 = 40; q_0 = 42.86 capped  -> (40, 60)
    obs 3  (40, 60), t = (20, 10)      X = (2, 6)     worker 1 raised, but 6 > 4: nothing learnt
                                                      q = (25, 75)                      -> (25, 75)
    obs 4  (25, 75), t = (6.25, 12.5)  X = (4, 6)     q = (40, 60)                      -> (40, 60)
    obs 5  (40, 60), t = (16, 12)      X = (2.5, 5)   worker 0 raised 25 -> 40, fell from 4 to 2.5:
                                                      bound_0 = 25; q_0 = 33.33 capped  -> (25, 75)
    """
    st = oracle.ControllerState([40, 60], kp=1.0, alpha=1.0, dmin=0.0, adaptive=True)
    got = _trace(st, [[8.0, 16.0], [19.0, 10.75], [20.0, 10.0], [6.25, 12.5], [16.0, 12.0]])
    assert got == [([57, 43], [0, 0]), ([40, 60], [40, 0]), ([25, 75], [40, 0]),
                   ([40, 60], [40, 0]), ([25, 75], [25, 0])]


def test_learnt_bound_compares_smoothed_throughput_at_every_observation():
    """alpha = 0.5, dead-band 0.35, by hand.  The comparison uses the smoothed time (a raw-time reading
    would learn one observation early) and is made at observations that do not readjust as well.

    obs 1  (40, 60), t = (8, 16): first sample, mu = t, X = (5, 3.75), b' = (57, 43); worker 1 moves
           by 17/60 but worker 0 by 17/40 > 0.35                                        -> readjust
    obs 2  t = (9, 10.75): first sample since, mu = (9, 10.75), X = (6.33, 4), b' = (61, 39),
           largest move 4/43                                                            -> keep
    obs 3  t = (13, 10.75): mu_0 = (13 + 9)/2 = 11, X_0 = 57/11 = 5.18 >= 5: nothing learnt
           (the raw 57/13 = 4.38 would have); b' = (56, 44)                             -> keep
    obs 4  t = (14, 10.75): mu_0 = (14 + 11)/2 = 12.5, X_0 = 4.56 < 5 after the raise 40 -> 57:
           bound_0 = 40; q_0 = 53.27 capped at 40, b' = (40, 60), moves 17/57 and 17/43 -> readjust
           (without the bound b' = (53, 47), inside the dead-band)
    """
    st = oracle.ControllerState([40, 60], kp=1.0, alpha=0.5, dmin=0.35, adaptive=True)
    assert st.observe([8.0, 16.0]) is True and st.b.tolist() == [57, 43]
    assert st.observe([9.0, 10.75]) is False and st.ewma.tolist() == [9.0, 10.75]
    assert st.observe([13.0, 10.75]) is False
    assert st.ewma.tolist() == [11.0, 10.75] and st.learnt_max.tolist() == [0, 0]
    assert st.b.tolist() == [57, 43]
    assert st.observe([14.0, 10.75]) is True
    assert st.learnt_max.tolist() == [40, 0] and st.b.tolist() == [40, 60]
