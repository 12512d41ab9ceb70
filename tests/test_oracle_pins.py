"""Pins for the CPU oracle: what the paper and the mathematics fix, checked without a GPU.

Each test compares `oracle/` with something that is not the oracle: a hand-worked
example, a literal replay of Algorithm 4's receive loop, exhaustive enumeration,
a library routine (numpy mean / argsort, torch's bf16 widening) or a closed form.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = vals
    return out


# ---------------------------------------------------------------- hand-worked example


def test_hand_worked_iteration():
    g = _read_golden("alg4_hand_example.txt")
    t, N, b = int(g["t"][0]), int(g["N"][0]), int(g["b"][0])
    W = N + b
    arrival = np.array(g["arrival"], dtype=np.float32)
    tags = np.array(g["tags"], dtype=np.int32)
    grad = np.array([g["grad%d" % w] for w in range(W)], dtype=np.float32)
    theta = np.array(g["theta"], dtype=np.float64)
    rc, mask, order, n_valid = oracle.select(arrival, tags, t, N, b)
    assert rc == oracle.OK
    assert n_valid == int(g["expect_n_valid"][0])
    assert mask.tolist() == [int(v) for v in g["expect_mask"]]
    assert order.tolist() == [int(v) for v in g["expect_order"]]
    mean = oracle.aggregate(grad, 2, order)
    assert mean.tolist() == [float(v) for v in g["expect_mean"]]
    rc, mask2, order2, _ = oracle.step(grad, 2, arrival, tags, t, N, b, theta, None, None,
                                       oracle.Opt(kind=oracle.SGD, lr=float(g["lr"][0])))
    assert rc == oracle.OK and order2.tolist() == order.tolist() and mask2.tolist() == mask.tolist()
    assert theta.tolist() == [float(v) for v in g["expect_theta"]]


# ---------------------------------------------------------------- selection


def _replay_algorithm4(arrival, tags, t, N):
    """Algorithm 4's loop, event by event: gradients reach the server one at a time in time order
    (equal times: lower id first); a gradient tagged t joins the set, any other is dropped; the
    server stops at |set| = N.  Returns the kept ids in the sequence they were received, or None."""
    W = len(arrival)
    pending = [w for w in range(W) if math.isfinite(float(arrival[w]))]
    kept = []
    while len(kept) < N:
        if not pending:
            return None  # the server would wait forever
        nxt = pending[0]
        for w in pending[1:]:
            if float(arrival[w]) < float(arrival[nxt]):  # strict: an equal time keeps the lower id
                nxt = w
        pending.remove(nxt)
        if int(tags[nxt]) == t:
            kept.append(nxt)
    return kept


def _random_case(rng, W, special=True):
    values = [0.25, 0.5, 0.5, 1.0, 1.5, 2.0, 7.0]
    if special:
        values += [float("inf"), float("nan"), -0.0, 0.0, -1.0, float("-inf")]
    arrival = np.array([values[i] for i in rng.integers(0, len(values), size=W)], dtype=np.float32)
    t = int(rng.integers(0, 5))
    tags = np.where(rng.random(W) < 0.25, t + rng.choice([-1, 1, -2], size=W), t).astype(np.int32)
    return arrival, tags, t


def test_select_matches_replay_of_algorithm4():
    rng = np.random.default_rng(1)
    seen_insufficient = seen_ok = 0
    for trial in range(3000):
        W = int(rng.integers(1, 9))
        N = int(rng.integers(1, W + 1))
        arrival, tags, t = _random_case(rng, W)
        rc, mask, order, n_valid = oracle.select(arrival, tags, t, N, W - N)
        kept = _replay_algorithm4(arrival, tags, t, N)
        valid = [w for w in range(W) if tags[w] == t and math.isfinite(float(arrival[w]))]
        assert n_valid == len(valid)
        if kept is None:
            assert rc == oracle.INSUFFICIENT
            seen_insufficient += 1
        else:
            assert rc == oracle.OK
            assert order.tolist() == kept
            assert mask.tolist() == [1 if w in kept else 0 for w in range(W)]
            seen_ok += 1
    assert seen_ok > 500 and seen_insufficient > 500


def test_select_is_the_unique_earliest_subset():
    """Enumerate every N-subset of the valid workers: exactly one has all its (time, id) keys below
    those of every valid worker left out, and it is the oracle's set."""
    rng = np.random.default_rng(2)
    for trial in range(400):
        W = int(rng.integers(2, 9))
        N = int(rng.integers(1, W + 1))
        arrival, tags, t = _random_case(rng, W, special=False)
        valid = [w for w in range(W) if tags[w] == t]
        rc, mask, order, _ = oracle.select(arrival, tags, t, N, W - N)
        if len(valid) < N:
            assert rc == oracle.INSUFFICIENT
            continue
        key = lambda w: (float(arrival[w]), w)
        winners = []
        for sub in itertools.combinations(valid, N):
            rest = [w for w in valid if w not in sub]
            if all(key(a) < key(r) for a in sub for r in rest):
                winners.append(sub)
        assert len(winners) == 1
        assert sorted(order.tolist()) == list(winners[0])
        assert order.tolist() == sorted(winners[0], key=key)


def test_select_special_cases():
    rng = np.random.default_rng(3)
    for W in (1, 2, 7, 33, 100, 208, 1024):
        arrival = rng.lognormal(0, 0.3, size=W).astype(np.float32)
        arrival[rng.integers(0, W, size=W // 3)] = 1.0  # ties
        tags = np.full(W, 4, dtype=np.int32)
        # b = 0, every tag current: all workers kept, in stable argsort order (library routine)
        rc, mask, order, n_valid = oracle.select(arrival, tags, 4, W, 0)
        assert rc == oracle.OK and n_valid == W and mask.all()
        assert order.tolist() == np.argsort(arrival, kind="stable").tolist()
        # N = 1: the single earliest valid gradient
        tags2 = tags.copy()
        tags2[np.argmin(arrival)] = 3  # the earliest one is stale
        rc, mask, order, _ = oracle.select(arrival, tags2, 4, 1, W - 1)
        if W == 1:
            assert rc == oracle.INSUFFICIENT
            continue
        cand = np.where(tags2 == 4)[0]
        best = cand[np.argmin(arrival[cand])]  # argmin returns the first (lowest id) minimum
        assert rc == oracle.OK and order.tolist() == [best] and mask.sum() == 1 and mask[best] == 1


def test_signed_zero_ties_and_never_arriving():
    arrival = np.array([0.0, -0.0, np.inf, np.nan, -np.inf, -3.0], dtype=np.float32)
    tags = np.zeros(6, dtype=np.int32)
    rc, mask, order, n_valid = oracle.select(arrival, tags, 0, 3, 3)
    assert rc == oracle.OK and n_valid == 3
    assert order.tolist() == [5, 0, 1]  # -3 first, then +0 and -0 compare equal: lower id first
    rc, *_ = oracle.select(arrival, tags, 0, 4, 2)
    assert rc == oracle.INSUFFICIENT


def test_stale_tag_removes_worker_and_admits_next():
    rng = np.random.default_rng(4)
    W, N, t = 12, 8, 3
    arrival = rng.permutation(W).astype(np.float32)
    tags = np.full(W, t, dtype=np.int32)
    _, mask, order, _ = oracle.select(arrival, tags, t, N, W - N)
    by_time = np.argsort(arrival, kind="stable").tolist()
    assert order.tolist() == by_time[:N]
    victim = order[2]
    for other in (t - 1, t + 1):  # a tag from the future is dropped like a stale one
        tags2 = tags.copy()
        tags2[victim] = other
        _, mask2, order2, n_valid = oracle.select(arrival, tags2, t, N, W - N)
        assert n_valid == W - 1 and mask2[victim] == 0
        assert order2.tolist() == [w for w in by_time if w != victim][:N]
    rc, mask3, order3, _ = oracle.select(arrival, np.full(W, t - 1, np.int32), t, N, W - N)
    assert rc == oracle.INSUFFICIENT and not mask3.any() and (order3 == -1).all()  # outputs untouched


# ---------------------------------------------------------------- aggregation


def test_b0_is_plain_minibatch_mean():
    """Section 3: with no backups the server averages every worker's gradient."""
    rng = np.random.default_rng(5)
    W, P = 17, 1003
    grad = rng.normal(size=(W, P)).astype(np.float32)
    arrival = rng.random(W).astype(np.float32)
    tags = np.zeros(W, np.int32)
    _, _, order, _ = oracle.select(arrival, tags, 0, W, 0)
    mean = oracle.aggregate(grad, P, order)
    ref = grad.astype(np.float64).mean(axis=0)
    np.testing.assert_allclose(mean, ref, rtol=0, atol=1e-15)


def test_constant_rows_give_mean_of_kept_constants():
    """Divisor is N (not N+b, not the number that arrived) and only kept rows count."""
    W, N, P = 9, 6, 50
    consts = np.array([1, 2, 4, 8, 16, 32, 64, 128, 256], dtype=np.float32)  # every subset has its own sum
    grad = np.repeat(consts[:, None], P, axis=1)
    arrival = np.array([5, 1, 9, 2, 8, 3, 7, 4, 6], dtype=np.float32)
    tags = np.array([0, 0, 0, 0, 0, -1, 0, 0, 0], dtype=np.int32)  # worker 5 is stale
    rc, mask, order, _ = oracle.select(arrival, tags, 0, N, W - N)
    assert order.tolist() == [1, 3, 7, 0, 8, 6]
    mean = oracle.aggregate(grad, P, order)
    expect = (2 + 8 + 128 + 1 + 256 + 64) / 6.0
    assert (mean == expect).all()


def test_leading_dimension_and_column_window():
    rng = np.random.default_rng(6)
    W, P, ld = 5, 37, 64
    grad = rng.normal(size=(W, ld)).astype(np.float32)
    order = np.array([3, 0, 4], dtype=np.int32)
    mean = oracle.aggregate(grad, P, order, ld=ld)
    ref = grad[[3, 0, 4], :P].astype(np.float64).mean(axis=0)
    np.testing.assert_allclose(mean, ref, rtol=0, atol=1e-15)


def test_bf16_widening_matches_torch_for_every_bit_pattern():
    bits = np.arange(65536, dtype=np.uint16).reshape(1, -1)
    mean = oracle.aggregate(bits, 65536, np.array([0], dtype=np.int32))
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()[0]
    same = (mean == ref) | (np.isnan(mean) & np.isnan(ref))
    assert same.all()
    nonzero = ~np.isnan(ref) & (ref != 0)  # the sum starts from +0, so -0 comes out as +0
    assert (np.signbit(mean) == np.signbit(ref))[nonzero].all()


def _poisoned_copy(grad, mask, rng, value):
    g = grad.copy()
    for w in np.where(mask == 0)[0]:
        g[w] = value if value is not None else rng.normal(size=g.shape[1]) * 1e6
    return g


@pytest.mark.parametrize("kind", [oracle.SGD, oracle.RMSPROP])
def test_dropped_rows_cannot_influence_theta(kind):
    """Section 3: late gradients are dropped when they arrive; Algorithm 4: so are wrongly tagged ones."""
    rng = np.random.default_rng(7)
    W, N, P, t = 10, 7, 200, 2
    grad = rng.normal(size=(W, P)).astype(np.float32)
    arrival = rng.random(W).astype(np.float32)
    tags = np.full(W, t, np.int32)
    tags[int(np.argmin(arrival))] = t - 1  # the earliest arrival is stale
    opt = oracle.Opt(kind=kind, lr=0.05, decay=0.9, momentum=0.9, eps=1.0)
    results = []
    for value in ("clean", None, np.nan, np.inf):
        th = np.linspace(-1, 1, P)
        s0, s1 = np.zeros(P), np.zeros(P)
        g = grad if value == "clean" else _poisoned_copy(grad, results[0][3], rng, value)
        rc, mask, order, _ = oracle.step(g, P, arrival, tags, t, N, W - N, th, s0, s1, opt)
        assert rc == oracle.OK and mask.sum() == N
        results.append((th, s0, s1, mask))
    for th, s0, s1, _ in results[1:]:
        assert th.tobytes() == results[0][0].tobytes()
        assert s0.tobytes() == results[0][1].tobytes() and s1.tobytes() == results[0][2].tobytes()


def test_insufficient_leaves_everything_untouched():
    W, N, P = 4, 3, 10
    grad = np.ones((W, P), np.float32)
    arrival = np.array([1, 2, np.inf, 3], np.float32)
    tags = np.array([0, 0, 0, 1], np.int32)
    th = np.arange(P, dtype=np.float64)
    s0 = np.full(P, 0.5)
    rc, mask, order, n_valid = oracle.step(grad, P, arrival, tags, 0, N, 1, th, s0, None,
                                           oracle.Opt(kind=oracle.MOMENTUM, lr=1.0, momentum=0.5))
    assert rc == oracle.INSUFFICIENT and n_valid == 2
    assert (th == np.arange(P)).all() and (s0 == 0.5).all()


# ---------------------------------------------------------------- optimizer rules (closed forms)


def _run_constant(kind, g, k, theta0=1.5, **hyper):
    P = len(g)
    th, s0, s1 = np.full(P, theta0), np.zeros(P), np.zeros(P)
    out = []
    for step in range(1, k + 1):
        oracle.update(th, s0, s1, g, oracle.Opt(kind=kind, step=step, **hyper))
        out.append(th.copy())
    return out


G_CONST = np.array([-3.0, -0.25, 0.0, 0.5, 2.0, 1e-3])


def test_sgd_multi_step_closed_form():
    """theta_T = theta_0 - lr * sum_t mean_t (Section 1.1), with selection and means from numpy."""
    rng = np.random.default_rng(8)
    W, N, P, T, lr = 6, 5, 300, 20, 0.1
    th = rng.normal(size=P)
    th0 = th.copy()
    total = np.zeros(P)
    for t in range(T):
        grad = rng.normal(size=(W, P)).astype(np.float32)
        arrival = rng.lognormal(0, 0.3, W).astype(np.float32)
        tags = np.full(W, t, np.int32)
        tags[rng.integers(0, W)] = t - 1
        rc, *_ = oracle.step(grad, P, arrival, tags, t, N, W - N, th, None, None, oracle.Opt(kind=oracle.SGD, lr=lr))
        assert rc == oracle.OK
        kept = _replay_algorithm4(arrival, tags, t, N)
        total += grad[kept].astype(np.float64).sum(axis=0) / N
    np.testing.assert_allclose(th, th0 - lr * total, rtol=0, atol=1e-12)


def test_momentum_closed_form():
    mu, lr, k = 0.9, 0.01, 12
    traj = _run_constant(oracle.MOMENTUM, G_CONST, k, lr=lr, momentum=mu)
    for j in range(1, k + 1):
        coeff = sum((1 - mu ** i) / (1 - mu) for i in range(1, j + 1))  # v_i = g (1-mu^i)/(1-mu)
        np.testing.assert_allclose(traj[j - 1], 1.5 - lr * G_CONST * coeff, rtol=1e-13, atol=1e-15)


def test_rmsprop_closed_form():
    rho, mu, lr, eps, k = 0.9, 0.9, 0.045, 1.0, 6
    traj = _run_constant(oracle.RMSPROP, G_CONST, k, lr=lr, decay=rho, momentum=mu, eps=eps)
    # first step from zero state: theta_1 = theta_0 - lr g / sqrt((1-rho) g^2 + eps)
    np.testing.assert_allclose(traj[0], 1.5 - lr * G_CONST / np.sqrt((1 - rho) * G_CONST ** 2 + eps), rtol=1e-14)
    # constant g: s_j = (1 - rho^j) g^2 ; m_j = sum_i mu^(j-i) lr g / sqrt(s_i + eps)
    theta = np.full_like(G_CONST, 1.5)
    for j in range(1, k + 1):
        m_j = sum(mu ** (j - i) * lr * G_CONST / np.sqrt((1 - rho ** i) * G_CONST ** 2 + eps) for i in range(1, j + 1))
        theta = theta - m_j
        np.testing.assert_allclose(traj[j - 1], theta, rtol=1e-13, atol=1e-15)


def test_rmsprop_eps_is_inside_the_root_and_state_is_callers():
    g = np.array([2.0])
    th, s, m = np.array([0.0]), np.array([1.0]), np.array([0.5])  # s_0 = 1, m_0 = 0.5
    oracle.update(th, s, m, g, oracle.Opt(kind=oracle.RMSPROP, lr=1.0, decay=0.5, momentum=0.5, eps=6.5))
    assert s[0] == 0.5 * 1.0 + 0.5 * 4.0  # 2.5
    assert m[0] == 0.25 + 2.0 / 3.0  # sqrt(2.5 + 6.5) = 3 ; outside the root it would be sqrt(2.5)+6.5
    assert th[0] == -m[0]


def test_rmsprop_learning_rate_enters_the_momentum_buffer():
    """With decay 0 and eps 0 the scaled gradient is sign(g); lr 1 then lr 4, momentum 0.5:
    m_1 = 1, m_2 = 0.5 * 1 + 4 = 4.5, theta_2 = theta_0 - 5.5 (lr applied outside the buffer would give -7)."""
    g = np.array([3.0, -2.0])
    th, s, m = np.array([10.0, 10.0]), np.zeros(2), np.zeros(2)
    oracle.update(th, s, m, g, oracle.Opt(kind=oracle.RMSPROP, lr=1.0, decay=0.0, momentum=0.5, eps=0.0))
    assert th.tolist() == [9.0, 11.0] and m.tolist() == [1.0, -1.0]
    oracle.update(th, s, m, g, oracle.Opt(kind=oracle.RMSPROP, lr=4.0, decay=0.0, momentum=0.5, eps=0.0))
    assert m.tolist() == [4.5, -4.5] and th.tolist() == [4.5, 15.5]


def test_adagrad_closed_form():
    """Constant g: s_k = k g^2, so with eps = 0 theta_k = theta_0 - lr sign(g) sum_{j<=k} 1/sqrt(j);
    with eps > 0 each term is |g| / (sqrt(j) |g| + eps)."""
    g = np.array([-3.0, -0.25, 0.5, 2.0])
    traj = _run_constant(oracle.ADAGRAD, g, 7, lr=0.1, eps=0.0)
    for k in range(1, 8):
        np.testing.assert_allclose(traj[k - 1], 1.5 - 0.1 * np.sign(g) * sum(1 / math.sqrt(j) for j in range(1, k + 1)), rtol=1e-13)
    traj = _run_constant(oracle.ADAGRAD, g, 5, lr=0.1, eps=0.5)
    for k in range(1, 6):
        step = sum(np.abs(g) / (math.sqrt(j) * np.abs(g) + 0.5) for j in range(1, k + 1))
        np.testing.assert_allclose(traj[k - 1], 1.5 - 0.1 * np.sign(g) * step, rtol=1e-13)
    th, acc = np.array([0.0]), np.array([5.0])  # the accumulator is the caller's: 5 + 2^2 = 9, root 3, eps 1 outside
    oracle.update(th, acc, None, np.array([2.0]), oracle.Opt(kind=oracle.ADAGRAD, lr=1.0, eps=1.0))
    assert acc[0] == 9.0 and th[0] == -0.5


def test_adam_closed_form_every_step():
    lr, eps, k = 1e-3, 1e-8, 9
    traj = _run_constant(oracle.ADAM, G_CONST, k, lr=lr, beta1=0.9, beta2=0.999, eps=eps)
    for j in range(1, k + 1):  # bias-corrected moments equal g and g^2 at every step
        np.testing.assert_allclose(traj[j - 1], 1.5 - j * lr * G_CONST / (np.abs(G_CONST) + eps), rtol=1e-12, atol=1e-15)


def test_adam_eps_is_outside_the_root():
    g = np.array([3.0])
    th, m, v = np.array([0.0]), np.array([0.0]), np.array([0.0])
    oracle.update(th, m, v, g, oracle.Opt(kind=oracle.ADAM, lr=1.0, beta1=0.5, beta2=0.5, eps=1.0, step=1))
    assert th[0] == pytest.approx(-3.0 / (3.0 + 1.0), rel=1e-15)  # inside the root: -3/sqrt(10)


# ---------------------------------------------------------------- arrival-by-arrival server


@pytest.mark.parametrize("kind,dtype", [(oracle.SGD, "f32"), (oracle.RMSPROP, "f32"), (oracle.ADAM, "bf16")])
def test_accumulate_on_arrival_equals_batched(kind, dtype):
    rng = np.random.default_rng(9)
    W, N, P, T = 9, 6, 120, 4
    opt_kw = dict(lr=0.05, decay=0.9, momentum=0.9, beta1=0.9, beta2=0.999, eps=0.1)
    th_a, s0_a, s1_a = rng.normal(size=P), np.zeros(P), np.zeros(P)
    th_b, s0_b, s1_b = th_a.copy(), np.zeros(P), np.zeros(P)
    acc, state = np.full(P, np.nan), oracle.new_server_state()  # acc needs no clearing by the caller
    leftovers = []  # (row, tag) that arrive after their iteration closed
    for t in range(T):
        grad = rng.normal(size=(W, P)).astype(np.float32)
        if dtype == "bf16":
            grad = torch.from_numpy(grad).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        arrival = rng.lognormal(0, 0.3, W).astype(np.float32)
        arrival[2] = arrival[5]  # a tie
        tags = np.full(W, t, np.int32)
        tags[int(rng.integers(0, W))] = t - 1
        opt = oracle.Opt(kind=kind, step=t + 1, **opt_kw)
        rc, mask, order, _ = oracle.step(grad, P, arrival, tags, t, N, W - N, th_b, s0_b, s1_b, opt)
        assert rc == oracle.OK
        outcomes = {}
        for row, tag in leftovers:  # stragglers of t-1 reach the server during t: dropped
            assert oracle.accumulate_arrival(row, tag, t, N, acc, state, th_a, s0_a, s1_a, opt) == 0
        leftovers = []
        fired = False
        for w in np.argsort(arrival, kind="stable"):
            res = oracle.accumulate_arrival(grad[w], int(tags[w]), t, N, acc, state, th_a, s0_a, s1_a, opt)
            outcomes[int(w)] = res
            if fired:
                assert res == 0  # Section 3: the slowest b are dropped when they arrive
            fired = fired or res == 2
        assert fired
        assert [w for w in np.argsort(arrival, kind="stable") if outcomes[int(w)] > 0] == order.tolist()
        assert state[0] == 0 and state[2] == t + 1
        np.testing.assert_allclose(th_a, th_b, rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(s0_a, s0_b, rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(s1_a, s1_b, rtol=1e-13, atol=1e-14)
        leftovers = [(grad[w], int(tags[w])) for w in range(W) if mask[w] == 0 and tags[w] == t][:1]


# ---------------------------------------------------------------- parameter average and learning-rate schedule


def test_ema_closed_form_under_sgd_with_constant_gradient():
    """theta(t) = theta0 - c t with c = lr g.  With avg(-1) = theta0 the recurrence
    avg(t) = alpha avg(t-1) + (1 - alpha) theta(t) solves to theta0 - c (t - alpha (1 - alpha^t) / (1 - alpha))."""
    W, N, P, lr, alpha = 4, 4, 3, 0.5, 0.75
    g = np.array([2.0, -1.0, 0.25])
    grad = np.repeat(g[None, :], W, axis=0).astype(np.float32)
    arrival, tags = np.arange(W, dtype=np.float32), None
    theta0 = np.array([1.0, 2.0, 3.0])
    theta, avg = theta0.copy(), theta0.copy()
    for t in range(12):
        tags = np.full(W, t, np.int32)
        rc, *_ = oracle.step_ema(grad, P, arrival, tags, t, N, 0, theta, None, None,
                                 oracle.Opt(kind=oracle.SGD, lr=lr), avg, alpha)
        assert rc == oracle.OK
        d = t - alpha * (1 - alpha ** t) / (1 - alpha)
        np.testing.assert_allclose(avg, theta0 - lr * g * d, rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(theta, theta0 - lr * g * (t + 1), rtol=1e-13)


def test_ema_sees_the_parameters_before_the_update_and_limits_of_alpha():
    grad = np.ones((2, 2), np.float32)
    arrival, tags = np.array([1, 2], np.float32), np.zeros(2, np.int32)
    opt = oracle.Opt(kind=oracle.SGD, lr=1.0)
    theta, avg = np.array([5.0, 7.0]), np.array([100.0, 100.0])
    oracle.step_ema(grad, 2, arrival, tags, 0, 2, 0, theta, None, None, opt, avg, 0.0)
    assert avg.tolist() == [5.0, 7.0] and theta.tolist() == [4.0, 6.0]  # alpha = 0: avg = theta(t), not theta(t+1)
    oracle.step_ema(grad, 2, arrival, tags, 0, 2, 0, theta, None, None, opt, avg, 1.0)
    assert avg.tolist() == [5.0, 7.0] and theta.tolist() == [3.0, 5.0]  # alpha = 1: avg frozen
    avg2 = np.array([8.0, 0.0])
    oracle.ema(avg2, np.array([0.0, 8.0]), 0.25)
    assert avg2.tolist() == [2.0, 6.0]
    # too few current gradients: nothing moves, the average included
    rc, *_ = oracle.step_ema(grad, 2, arrival, np.array([0, 9], np.int32), 0, 2, 0, theta, None, None, opt, avg, 0.0)
    assert rc == oracle.INSUFFICIENT and avg.tolist() == [5.0, 7.0] and theta.tolist() == [3.0, 5.0]


def test_learning_rate_schedule():
    """Appendix A: gamma0 * 0.94^(t N / (2 T)): one factor of beta every two passes over the data."""
    T = 40_000.0  # mini-batches per pass
    assert oracle.learning_rate(4.5, 0.94, 0, 100, T) == 4.5
    assert oracle.learning_rate(4.5, 0.94, 800, 100, T) == pytest.approx(4.5 * 0.94, rel=1e-14)  # t N = 2 T
    assert oracle.learning_rate(4.5, 0.94, 1600, 100, T) == pytest.approx(4.5 * 0.94 ** 2, rel=1e-14)
    assert oracle.learning_rate(0.045, 0.94, 80_000, 1, T) == pytest.approx(0.045 * 0.94, rel=1e-14)  # asynchronous rule
    assert oracle.learning_rate(1.0, 0.25, 100, 50, 5000.0) == pytest.approx(0.5, rel=1e-14)  # exponent 1/2


# ---------------------------------------------------------------- time-out instead of backup workers


def test_deadline_selection_matches_replay_until_the_time_out():
    """Replay: gradients reach the server in time order; at `deadline` it stops listening."""
    rng = np.random.default_rng(21)
    seen = set()
    for trial in range(2000):
        W = int(rng.integers(1, 9))
        arrival, tags, t = _random_case(rng, W)
        deadline = float(rng.choice([0.25, 0.5, 1.0, 1.25, 2.0, 7.0, 100.0, -0.5, np.inf]))
        n_min = int(rng.integers(1, 4))
        rc, mask, order, n = oracle.select_deadline(arrival, tags, t, deadline, n_min)
        kept = []
        for w in sorted((w for w in range(W) if math.isfinite(float(arrival[w]))), key=lambda w: (float(arrival[w]), w)):
            if float(arrival[w]) > deadline:
                break  # the server has stopped waiting
            if int(tags[w]) == t:
                kept.append(w)
        assert n == len(kept)
        if len(kept) < n_min:
            assert rc == oracle.INSUFFICIENT and not mask.any()
        else:
            assert rc == oracle.OK and order.tolist() == kept
            assert mask.tolist() == [1 if w in kept else 0 for w in range(W)]
        seen.add(rc)
    assert seen == {oracle.OK, oracle.INSUFFICIENT}


def test_deadline_rule_reduces_to_algorithm4_and_divides_by_the_number_kept():
    rng = np.random.default_rng(22)
    W, N, P, t = 9, 6, 40, 3
    arrival = rng.permutation(W).astype(np.float32) + 1.0  # distinct times 1..9
    tags = np.full(W, t, np.int32)
    grad = rng.normal(size=(W, P)).astype(np.float32)
    # a deadline at the N-th arrival keeps exactly Algorithm 4's first N
    rc, mask_n, order_n, _ = oracle.select(arrival, tags, t, N, W - N)
    rc2, mask_d, order_d, n = oracle.select_deadline(arrival, tags, t, float(N), 1)
    assert rc == rc2 == oracle.OK and n == N and order_d.tolist() == order_n.tolist() and mask_d.tolist() == mask_n.tolist()
    th_a, th_b = np.zeros(P), np.zeros(P)
    oracle.step(grad, P, arrival, tags, t, N, W - N, th_a, None, None, oracle.Opt(kind=oracle.SGD, lr=0.3))
    oracle.step_deadline(grad, P, arrival, tags, t, float(N), 1, th_b, None, None, oracle.Opt(kind=oracle.SGD, lr=0.3))
    assert th_a.tobytes() == th_b.tobytes()
    # no deadline: plain synchronous SGD over every current gradient (library mean)
    tags[4] = t - 1
    th = np.zeros(P)
    rc, mask, order, n = oracle.step_deadline(grad, P, arrival, tags, t, np.inf, 1, th, None, None,
                                              oracle.Opt(kind=oracle.SGD, lr=1.0))
    assert n == W - 1 and mask[4] == 0
    np.testing.assert_allclose(th, -np.delete(grad, 4, axis=0).astype(np.float64).mean(axis=0), rtol=0, atol=1e-15)
    # constant rows: the divisor is the number kept, whatever it is
    consts = (2.0 ** np.arange(W)).astype(np.float32)
    gc = np.repeat(consts[:, None], 3, axis=1)
    for deadline in (1.0, 3.0, 8.0):
        th = np.zeros(3)
        rc, mask, order, n = oracle.step_deadline(gc, 3, arrival, tags, t, deadline, 1, th, None, None,
                                                  oracle.Opt(kind=oracle.SGD, lr=1.0))
        kept = [w for w in range(W) if arrival[w] <= deadline and tags[w] == t]
        assert rc == oracle.OK and n == len(kept) and (th == -float(consts[kept].sum()) / len(kept)).all()
    th = np.ones(3)
    rc, *_ = oracle.step_deadline(gc, 3, arrival, tags, t, 0.5, 1, th, None, None, oracle.Opt(kind=oracle.SGD, lr=1.0))
    assert rc == oracle.INSUFFICIENT and (th == 1).all()


# ---------------------------------------------------------------- the asynchronous server (Algorithm 2)


def test_arrival_server_with_n_equal_one_is_algorithm2():
    """Algorithm 2 applies every arriving gradient at once: theta <- theta - gamma G.  The arrival-by-arrival
    server with N = 1 does exactly that; with SGD the result is theta0 - lr * (sum of all gradients)."""
    rng = np.random.default_rng(31)
    P, K, lr = 50, 17, 0.05
    rows = rng.normal(size=(K, P)).astype(np.float32)
    theta = rng.normal(size=P)
    theta0 = theta.copy()
    acc, state = np.zeros(P), oracle.new_server_state()
    for k in range(K):
        out = oracle.accumulate_arrival(rows[k], k, k, 1, acc, state, theta, None, None, oracle.Opt(kind=oracle.SGD, lr=lr))
        assert out == 2 and state.tolist() == [0, k + 1, k + 1]
    np.testing.assert_allclose(theta, theta0 - lr * rows.astype(np.float64).sum(axis=0), rtol=0, atol=1e-13)


def test_arrival_server_with_average_equals_batched_step_with_average():
    rng = np.random.default_rng(41)
    W, N, P, T, alpha = 7, 5, 60, 4, 0.8
    th_a = rng.normal(size=P)
    th_b, avg_a, avg_b = th_a.copy(), th_a.copy(), th_a.copy()
    acc, state = np.zeros(P), oracle.new_server_state()
    for t in range(T):
        grad = rng.normal(size=(W, P)).astype(np.float32)
        arrival = rng.lognormal(0, 0.3, W).astype(np.float32)
        tags = np.full(W, t, np.int32)
        tags[int(rng.integers(0, W))] = t - 1
        opt = oracle.Opt(kind=oracle.SGD, lr=0.1)
        rc, *_ = oracle.step_ema(grad, P, arrival, tags, t, N, W - N, th_b, None, None, opt, avg_b, alpha)
        assert rc == oracle.OK
        before = avg_a.copy()
        for i, w in enumerate(np.argsort(arrival, kind="stable")):
            out = oracle.accumulate_arrival_ema(grad[w], int(tags[w]), t, N, acc, state, th_a, None, None, opt, avg_a, alpha)
            if out != 2 and state[2] == t:
                assert (avg_a == before).all()  # the average only moves when the update fires
        np.testing.assert_allclose(th_a, th_b, rtol=1e-13, atol=1e-14)
        np.testing.assert_allclose(avg_a, avg_b, rtol=1e-13, atol=1e-14)


# ---------------------------------------------------------------- two-level aggregation (machines)


def test_two_level_hand_worked_iteration():
    g = _read_golden("two_level_hand_example.txt")
    t, M, N = int(g["t"][0]), int(g["M"][0]), int(g["N"][0])
    group = np.array(g["group"], dtype=np.int32)
    arrival = np.array(g["arrival"], dtype=np.float32)
    tags = np.array(g["tags"], dtype=np.int32)
    grad = np.array([g["grad%d" % w] for w in range(len(group))], dtype=np.float32)
    theta = np.array(g["theta"], dtype=np.float64)
    rc, mask, group_order, order, n_valid = oracle.step_grouped(grad, 2, arrival, tags, group, t, M, N, theta, None, None,
                                                                oracle.Opt(kind=oracle.SGD, lr=float(g["lr"][0])))
    assert rc == oracle.OK and n_valid == int(g["expect_n_valid"][0])
    assert mask.tolist() == [int(v) for v in g["expect_mask"]]
    assert group_order.tolist() == [int(v) for v in g["expect_group_order"]]
    assert order.tolist() == [int(v) for v in g["expect_order"]]
    assert theta.tolist() == [float(v) for v in g["expect_theta"]]


def _replay_machines(arrival, tags, group, t, M, N):
    """Event by event: workers finish in time order; a machine whose workers are all done sends one message,
    stamped with that moment; the server takes messages in (time, machine id) order and stops at N.  A machine
    with a worker that never finishes never sends; one with a worker that computed for another iteration sends
    a message the server drops.  Returns (kept machine ids in sequence, number of countable messages) or (None, n)."""
    W = len(arrival)
    members = {g: [w for w in range(W) if group[w] == g] for g in range(M)}
    outbox = []
    for g, ws in members.items():
        if not ws or not all(math.isfinite(float(arrival[w])) for w in ws):
            continue
        clock, done = None, 0
        for w in sorted(ws, key=lambda w: float(arrival[w])):  # the machine's own workers, one after another
            clock = float(arrival[w])
            done += 1
        assert done == len(ws)
        outbox.append((clock, g, all(int(tags[w]) == t for w in ws)))
    outbox.sort(key=lambda m: (m[0], m[1]))
    kept = []
    for _, g, current in outbox:
        if len(kept) == N:
            break
        if current:
            kept.append(g)
    n_countable = sum(1 for m in outbox if m[2])
    return (kept if len(kept) == N else None), n_countable


def _random_machines(rng, W, M):
    arrival, tags, t = _random_case(rng, W)
    group = rng.integers(0, M, size=W).astype(np.int32)
    return arrival, tags, group, t


def test_two_level_selection_matches_replay_of_machines():
    rng = np.random.default_rng(21)
    ok = short = 0
    for trial in range(3000):
        W, M = int(rng.integers(1, 10)), int(rng.integers(1, 6))
        N = int(rng.integers(1, M + 1))
        arrival, tags, group, t = _random_machines(rng, W, M)
        if trial % 3 == 0:
            tags[:] = t  # enough cases where most machines count
        rc, mask, group_order, order, n_valid = oracle.select_grouped(arrival, tags, group, t, M, N)
        kept, n_countable = _replay_machines(arrival, tags, group, t, M, N)
        assert n_valid == n_countable
        if kept is None:
            assert rc == oracle.INSUFFICIENT
            short += 1
            continue
        ok += 1
        assert rc == oracle.OK and group_order.tolist() == kept
        assert mask.tolist() == [1 if group[w] in kept else 0 for w in range(W)]
        want = []
        for g in kept:
            want += sorted([w for w in range(W) if group[w] == g], key=lambda w: (float(arrival[w]), w))
        assert order.tolist() == want
    assert ok > 500 and short > 500


def test_two_level_kept_machines_are_the_unique_earliest_subset():
    rng = np.random.default_rng(22)
    for trial in range(300):
        W, M = int(rng.integers(2, 10)), int(rng.integers(2, 6))
        N = int(rng.integers(1, M + 1))
        arrival, tags, t = _random_case(rng, W, special=False)
        group = rng.integers(0, M, size=W).astype(np.int32)
        sent = {}
        for g in range(M):
            ws = [w for w in range(W) if group[w] == g]
            if ws and all(tags[w] == t for w in ws):
                sent[g] = (max(float(arrival[w]) for w in ws), g)
        rc, _, group_order, _, n_valid = oracle.select_grouped(arrival, tags, group, t, M, N)
        assert n_valid == len(sent)
        if len(sent) < N:
            assert rc == oracle.INSUFFICIENT
            continue
        winners = [sub for sub in itertools.combinations(sorted(sent), N)
                   if all(sent[a] < sent[r] for a in sub for r in sent if r not in sub)]
        assert len(winners) == 1 and sorted(group_order.tolist()) == list(winners[0])
        assert group_order.tolist() == sorted(winners[0], key=lambda g: sent[g])


def test_two_level_with_one_worker_per_machine_is_algorithm4():
    """Machines of one worker each, machine id = worker id: nothing is left of the second level, and the result
    must be Algorithm 4's own, bit for bit, for every rule."""
    rng = np.random.default_rng(23)
    for kind in (oracle.SGD, oracle.MOMENTUM, oracle.RMSPROP, oracle.ADAM, oracle.ADAGRAD):
        for trial in range(20):
            W = int(rng.integers(1, 9))
            N = int(rng.integers(1, W + 1))
            P = 5
            arrival, tags, t = _random_case(rng, W)
            grad = rng.standard_normal((W, P)).astype(np.float32)
            opt = oracle.Opt(kind=kind, lr=0.1, momentum=0.9, decay=0.9, beta1=0.9, beta2=0.99, eps=0.5, step=3)
            a = [rng.standard_normal(P), np.abs(rng.standard_normal(P)), np.abs(rng.standard_normal(P))]
            b = [x.copy() for x in a]
            rc1, mask1, order1, n1 = oracle.step(grad, P, arrival, tags, t, N, W - N, *a, opt)
            rc2, mask2, gorder2, order2, n2 = oracle.step_grouped(grad, P, arrival, tags, np.arange(W, dtype=np.int32), t,
                                                                  W, N, *b, opt)
            assert rc1 == rc2 and n1 == n2
            for x, y in zip(a, b):
                assert np.array_equal(x, y)
            if rc1 == oracle.OK:
                assert mask1.tolist() == mask2.tolist() and order1.tolist() == order2.tolist() == gorder2.tolist()


def test_two_level_with_equal_machines_is_the_mean_over_their_workers():
    """Equal machine sizes: the mean of the machines' means is numpy's mean over all workers of the kept machines."""
    rng = np.random.default_rng(24)
    M, per, N, P = 6, 4, 4, 33
    W = M * per
    group = rng.permutation(np.repeat(np.arange(M), per)).astype(np.int32)  # workers of a machine need not be neighbours
    arrival = rng.lognormal(0.0, 0.3, W).astype(np.float32)
    tags = np.full(W, 2, np.int32)
    grad = rng.standard_normal((W, P)).astype(np.float32)
    theta = rng.standard_normal(P)
    theta0 = theta.copy()
    rc, mask, group_order, order, n_valid = oracle.step_grouped(grad, P, arrival, tags, group, 2, M, N, theta, None, None,
                                                                oracle.Opt(kind=oracle.SGD, lr=0.25))
    assert rc == oracle.OK and n_valid == M and int(mask.sum()) == N * per == len(order)
    sent = [max(arrival[group == g]) for g in range(M)]
    assert group_order.tolist() == list(np.argsort(np.array(sent, np.float32), kind="stable")[:N])
    want = theta0 - 0.25 * np.mean(grad[np.isin(group, group_order)].astype(np.float64), axis=0)
    assert np.allclose(theta, want, rtol=0, atol=1e-15)


def test_two_level_unequal_machines_weigh_messages_equally_and_wait_for_the_slowest():
    """Constant rows of powers of two: the mean of the kept machines' means is exact, and differs from the mean
    over workers, from a sum of machine sums and from what a send-at-first-worker rule would keep."""
    group = np.array([0, 0, 0, 0, 1, 2, 2], np.int32)
    arrival = np.array([0.1, 0.2, 0.3, 9.0, 1.0, 0.5, 2.0], np.float32)  # machine 0 has an early start and a late finish
    tags = np.zeros(7, np.int32)
    consts = np.array([1, 2, 4, 8, 16, 32, 64], np.float64)
    grad = np.repeat(consts[:, None], 3, axis=1).astype(np.float32)
    theta = np.zeros(3)
    rc, mask, group_order, order, _ = oracle.step_grouped(grad, 3, arrival, tags, group, 0, 3, 2, theta, None, None,
                                                          oracle.Opt(kind=oracle.SGD, lr=1.0))
    assert rc == oracle.OK and group_order.tolist() == [1, 2] and order.tolist() == [4, 5, 6]
    assert mask.tolist() == [0, 0, 0, 0, 1, 1, 1]
    assert theta.tolist() == [-(16 + (32 + 64) / 2) / 2] * 3  # = -32, not -(16+32+64)/3 and not -(16+96)


def test_two_level_a_stale_or_missing_worker_silences_its_machine():
    rng = np.random.default_rng(25)
    M, per, N, P = 5, 3, 3, 4
    W = M * per
    group = np.repeat(np.arange(M), per).astype(np.int32)
    arrival = (1.0 + np.arange(W) * 0.125).astype(np.float32)  # machine g sends before machine g + 1
    tags = np.full(W, 7, np.int32)
    grad = rng.standard_normal((W, P)).astype(np.float32)
    base = oracle.select_grouped(arrival, tags, group, 7, M, N)
    assert base[0] == oracle.OK and base[2].tolist() == [0, 1, 2] and base[4] == M
    for spoil in ("stale", "future", "nan", "inf"):
        a, tg = arrival.copy(), tags.copy()
        if spoil == "stale":
            tg[4] = 6
        elif spoil == "future":
            tg[4] = 8
        elif spoil == "nan":
            a[4] = np.nan
        else:
            a[4] = np.inf
        rc, mask, group_order, order, n_valid = oracle.select_grouped(a, tg, group, 7, M, N)
        assert rc == oracle.OK and n_valid == M - 1 and group_order.tolist() == [0, 2, 3]  # machine 1 is out, 3 moves up
        assert mask.tolist() == [1 if g in (0, 2, 3) else 0 for g in group]
    # rows of machines that are not used cannot influence the result
    theta_a, theta_b = np.ones(P), np.ones(P)
    poisoned = grad.copy()
    poisoned[group >= 3] = np.nan
    opt = oracle.Opt(kind=oracle.SGD, lr=0.5)
    assert oracle.step_grouped(grad, P, arrival, tags, group, 7, M, N, theta_a, None, None, opt)[0] == oracle.OK
    assert oracle.step_grouped(poisoned, P, arrival, tags, group, 7, M, N, theta_b, None, None, opt)[0] == oracle.OK
    assert np.array_equal(theta_a, theta_b) and np.isfinite(theta_a).all()
    # too few countable messages: nothing moves; a machine id out of range is refused
    tags[::per] = 6
    before = theta_a.copy()
    rc, *_ , n_valid = oracle.step_grouped(grad, P, arrival, tags, group, 7, M, N, theta_a, None, None, opt)
    assert rc == oracle.INSUFFICIENT and n_valid == 0 and np.array_equal(theta_a, before)
    bad = group.copy()
    bad[0] = M
    assert oracle.select_grouped(arrival, np.full(W, 7, np.int32), bad, 7, M, N)[0] == oracle.INVALID
    # a machine without workers sends nothing
    rc, _, group_order, _, n_valid = oracle.select_grouped(arrival[:6], np.full(6, 7, np.int32), np.array([0, 0, 0, 2, 2, 2], np.int32), 7, 3, 2)
    assert rc == oracle.OK and n_valid == 2 and group_order.tolist() == [0, 2]


# ---------------------------------------------------------------- time-out rule, one gradient at a time


@pytest.mark.parametrize("kind", [oracle.SGD, oracle.RMSPROP])
def test_arrival_server_with_deadline_equals_batched_deadline_step(kind):
    """Gradients delivered one by one in arrival sequence (stale ones, late ones and a straggler of the previous
    iteration included), then the close call: same set, same divisor, same bits as the batched time-out step, which
    is pinned on its own above.  Also in event order (late rows delivered after the close)."""
    rng = np.random.default_rng(41)
    P, W, T = 7, 9, 4
    for event_order in (False, True):
        theta_a, theta_b = np.linspace(-1, 1, P), np.linspace(-1, 1, P)
        avg_a, avg_b = theta_a.copy(), theta_b.copy()
        sa = [np.zeros(P), np.zeros(P)]
        sb = [np.zeros(P), np.zeros(P)]
        acc, state = np.full(P, np.nan), oracle.new_server_state()
        seen = 0
        prev = None
        for t in range(T):
            arrival = rng.lognormal(0.0, 0.5, W).astype(np.float32)
            arrival[rng.integers(0, W)] = np.inf
            tags = np.where(rng.random(W) < 0.2, t - 1, t).astype(np.int32)
            grad = rng.standard_normal((W, P)).astype(np.float32)
            deadline = float(np.float32(np.sort(arrival)[W // 2]))  # somewhere in the middle: an arrival exactly at it is kept
            opt = oracle.Opt(kind=kind, lr=0.05, decay=0.9, momentum=0.9, eps=1.0)
            rc_b, mask, order, n = oracle.step_deadline(grad, P, arrival, tags, t, deadline, 1, theta_b, sb[0], sb[1], opt)
            ids = [int(w) for w in np.argsort(arrival, kind="stable")]
            early = [w for w in ids if np.isfinite(arrival[w]) and arrival[w] <= np.float32(deadline)]
            late = [w for w in ids if np.isfinite(arrival[w]) and not arrival[w] <= np.float32(deadline)]
            outcomes = {}
            deliveries = early + ([] if event_order else late)
            if prev is not None:
                assert oracle.accumulate_arrival_deadline(prev, t - 1, 0.0, t, deadline, acc, state) == 0  # straggler of t - 1
                seen += 1
            for w in deliveries:
                outcomes[w] = oracle.accumulate_arrival_deadline(grad[w], int(tags[w]), float(arrival[w]), t, deadline, acc, state)
                seen += 1
            theta_t = theta_a.copy()
            rc_a, outcome = oracle.accumulate_close(t, 1, acc, state, theta_a, sa[0], sa[1], opt, avg_a, 0.9)
            assert rc_a == rc_b
            if rc_b == oracle.OK:
                assert outcome == 2 and state.tolist() == [0, seen, t + 1]
                assert sorted(w for w, o in outcomes.items() if o == 1) == sorted(order.tolist()) and n == len(order)
                assert np.array_equal(avg_a, 0.9 * avg_b + (1.0 - 0.9) * theta_t)
                avg_b = avg_a.copy()
            else:
                assert outcome == 0 and np.array_equal(theta_a, theta_t) and state[2] == t
                state[0] = 0  # the test moves on: forget the incomplete iteration
                state[2] = t + 1
            if event_order:
                for w in late:
                    assert oracle.accumulate_arrival_deadline(grad[w], int(tags[w]), float(arrival[w]), t, deadline, acc, state) == 0
                    seen += 1
            # closing again, or closing an older iteration, does nothing
            before = theta_a.copy()
            assert oracle.accumulate_close(t, 1, acc, state, theta_a, sa[0], sa[1], opt) == (oracle.OK, 0)
            assert np.array_equal(theta_a, before)
            assert np.array_equal(theta_a, theta_b) and np.array_equal(sa[0], sb[0]) and np.array_equal(sa[1], sb[1])
            prev = grad[0].copy()


def test_arrival_server_with_deadline_needs_n_min_and_divides_by_the_set():
    P = 3
    rows = np.array([[1, 2, 4], [3, 6, 12], [100, 100, 100]], np.float32)
    acc, state = np.zeros(P), oracle.new_server_state()
    theta = np.zeros(P)
    opt = oracle.Opt(kind=oracle.SGD, lr=1.0)
    assert oracle.accumulate_arrival_deadline(rows[0], 5, 1.0, 5, 2.0, acc, state) == 1
    assert oracle.accumulate_close(5, 2, acc, state, theta, None, None, opt) == (oracle.INSUFFICIENT, 0)
    assert theta.tolist() == [0, 0, 0] and state.tolist() == [1, 1, 0]  # the server may keep listening
    assert oracle.accumulate_arrival_deadline(rows[1], 5, 2.0, 5, 2.0, acc, state) == 1  # exactly at the deadline: kept
    assert oracle.accumulate_arrival_deadline(rows[2], 5, 2.5, 5, 2.0, acc, state) == 0  # after it: dropped
    assert oracle.accumulate_arrival_deadline(rows[2], 5, float("nan"), 5, 2.0, acc, state) == 0
    assert oracle.accumulate_close(5, 2, acc, state, theta, None, None, opt) == (oracle.OK, 2)
    assert theta.tolist() == [-2.0, -4.0, -8.0] and state.tolist() == [0, 4, 6]  # mean of two, not of three or four
