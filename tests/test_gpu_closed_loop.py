"""Closed loop (Section 3.2, Section 5): least-squares gradient descent whose gradient sum goes through
encode -> adversary -> decode every step, with a freshly drawn Byzantine set per step.  The iterates must equal
those of an attack-free run, and both must follow the oracle's float64 descent."""

import numpy as np
import pytest
import torch

from oracle import solon_oracle as so
from paper_2110_01595_b200 import binding, build, sgd

pytestmark = pytest.mark.gpu

P, S, M, R = 15, 2, 3, 7            # two groups (8 and 7 nodes), up to two attackers in each
D, ROWS, STEPS = 600, 64, 12


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def _problem():
    g = torch.Generator().manual_seed(2024)
    n = P * ROWS
    X = torch.randn(n, D, generator=g)
    w_star = torch.randn(D, generator=g)
    y = X @ w_star + 0.01 * torch.randn(n, generator=g)
    return X, y, torch.zeros(D), 0.4 / n


def _oracle_descent(X, y, w0, lr):
    X64, y64, w = X.numpy().astype(np.float64), y.numpy().astype(np.float64), w0.numpy().astype(np.float64)
    out = []
    for _ in range(STEPS):
        w = w - lr * so.plain_sum(so.lsq_grads(X64, y64, w, ROWS))
        out.append(w.copy())
    return out


def _run(per_group, attack, graph, early=1, optimistic=None):
    X, y, w0, lr = _problem()
    rng = np.random.default_rng(99)
    iterates, masks, sets = [], [], []
    with binding.Plan(P, S, M, R, D, seed=5) as plan:
        plan.set_early_locator(early)
        if optimistic is not None:
            plan.set_optimistic(optimistic)
        loop = sgd.ClosedLoop(plan, X.cuda(), y.cuda(), w0.cuda(), lr, ROWS, attackers_per_group=per_group, attack=attack)
        if graph:
            loop.set_attackers(sgd.draw_attackers(plan, np.random.default_rng(1), per_group))
            loop.capture()
        for _ in range(STEPS):
            nodes = sgd.draw_attackers(plan, rng, per_group)
            loop.set_attackers(nodes)
            loop.step()
            torch.cuda.synchronize()
            assert plan.decode_status() == 0
            iterates.append(loop.w.cpu().numpy().astype(np.float64))
            masks.append(loop.mask.cpu().numpy().nonzero()[0].tolist())
            sets.append(nodes)
    return iterates, masks, sets


@pytest.mark.parametrize("attack", sgd.ATTACKS)
def test_iterates_equal_the_attack_free_run(attack):
    clean, clean_masks, _ = _run(0, attack, graph=False)
    assert all(m == [] for m in clean_masks)
    attacked, masks, sets = _run(S, attack, graph=False)
    assert len({tuple(s) for s in sets}) > STEPS // 2          # the Byzantine set really changes
    assert masks == sets                                        # located exactly, every step
    X, y, w0, lr = _problem()
    ref = _oracle_descent(X, y, w0, lr)
    for k in range(STEPS):
        scale = np.abs(ref[k]).max()
        assert np.abs(attacked[k] - clean[k]).max() <= 2e-5 * scale, k
        assert np.abs(clean[k] - ref[k]).max() <= 5e-4 * scale, k
    # and the descent goes somewhere: the residual of the last iterate is far below that of the first
    assert np.linalg.norm(ref[-1] - ref[-2]) < 0.1 * np.linalg.norm(ref[0])


@pytest.mark.parametrize("early", [0, 2])
def test_graph_replay_equals_eager_steps(early):
    # bit for bit with the optimistic decode off: with it on, an aggregate may come from the previous decode's recovery
    # table (other trusted rows, the same sum up to rounding), and the captured run has one more decode behind it
    eager, masks_e, sets_e = _run(S, "alie", graph=False, optimistic=0)
    replay, masks_g, sets_g = _run(S, "alie", graph=True, early=early, optimistic=0)
    assert sets_e == sets_g and masks_e == masks_g == sets_e
    for a, b in zip(eager, replay):
        assert np.array_equal(a, b)
    # default mode: the same iterates up to that rounding
    replay_d, masks_d, sets_d = _run(S, "alie", graph=True, early=early)
    assert sets_d == sets_e and masks_d == sets_e
    for a, b in zip(eager, replay_d):
        assert np.abs(a - b).max() <= 2e-5 * np.abs(a).max()
