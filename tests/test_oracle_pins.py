"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each checks the oracle against
something other than itself: worked values (tests/golden), closed forms,
reductions to the baselines the method contains (Streaming DiLoCo, DiLoCo),
the torch CPU Nesterov optimizer, numpy's norm, and brute force over subsets.
"""

import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import reference as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rows(name):
    out = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                out.append([float(x) for x in line.split()])
    return out


def one_fragment(n):
    return [[(0, n)]]


def run_single(hp, w_now, w_snap, theta_g, mom, **kw):
    """Outer step over one fragment covering the whole vector."""
    n = theta_g.shape[0]
    res, last = orc.outer_step(one_fragment(n), hp, w_now, w_snap, theta_g, mom, [0],
                               kw.pop("t_p", 10), kw.pop("t_l", 12), [0], **kw)
    return res[0]


def rand_inputs(M, n, seed=0, drift=1e-3):
    rng = np.random.default_rng(seed)
    thg = (0.02 * rng.standard_normal(n)).astype(np.float32)
    snap = (thg + drift * rng.standard_normal((M, n))).astype(np.float32)
    now = (snap + drift * rng.standard_normal((M, n))).astype(np.float32)
    mom = (1e-3 * rng.standard_normal(n)).astype(np.float32)
    return now, snap, thg, mom


# ------------------------------------------------------------------ Eq. 8-9

@pytest.mark.parametrize("row", rows("schedule_sizing.txt"))
def test_sync_budget_golden(row):
    K, H, gamma, Tc, Ts, N, h = row
    assert orc.sync_budget(int(K), int(H), gamma, Tc, Ts) == (int(N), int(h))


def test_sync_budget_never_below_K():
    for K in (1, 4, 13):
        for ratio in (1e-6, 0.01, 0.3, 2.0):
            N, h = orc.sync_budget(K, 100, 0.4, ratio, 1.0)
            assert N >= K and h >= 1 and h * N <= max(100, N)


# ------------------------------------------------------------------ Eq. 1-2

def test_mean_is_identity_for_one_worker():
    now, snap, thg, mom = rand_inputs(1, 257, seed=1)
    hp = orc.Hyper(M=1)
    r = run_single(hp, now, snap, thg, mom)
    np.testing.assert_array_equal(r.delta_g, snap[0].astype(np.float64) - thg.astype(np.float64))


def test_identical_workers_and_permutation():
    now, snap, thg, mom = rand_inputs(4, 300, seed=2)
    same = np.repeat(snap[:1], 4, axis=0)
    r = run_single(orc.Hyper(M=4), now, same, thg, mom)
    np.testing.assert_allclose(r.delta_g, same[0].astype(np.float64) - thg, rtol=0, atol=1e-18)
    r1 = run_single(orc.Hyper(M=4), now, snap, thg, mom)
    perm = [2, 0, 3, 1]
    r2 = run_single(orc.Hyper(M=4), now[perm], snap[perm], thg, mom)
    np.testing.assert_allclose(r1.delta_g, r2.delta_g, rtol=1e-13)
    np.testing.assert_allclose(r1.theta_g, r2.theta_g, rtol=1e-13)
    np.testing.assert_allclose(r1.w_now[perm], r2.w_now, rtol=1e-13)


def test_plain_averaging_when_lr_one_no_momentum():
    """eta = 1, mu = 0: the new global state is the mean of the workers' parameters."""
    now, snap, thg, mom = rand_inputs(3, 500, seed=3)
    r = run_single(orc.Hyper(M=3, outer_lr=1.0, momentum=0.0), now, snap, thg, np.zeros_like(mom))
    np.testing.assert_allclose(r.theta_g, snap.astype(np.float64).mean(axis=0), rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(r.momentum, r.delta_g, rtol=0, atol=0)


def test_plain_sgd_when_no_momentum():
    now, snap, thg, mom = rand_inputs(2, 400, seed=4)
    r = run_single(orc.Hyper(M=2, outer_lr=0.3, momentum=0.0), now, snap, thg, mom)
    np.testing.assert_allclose(r.theta_g, thg + 0.3 * r.delta_g, rtol=1e-14)


@pytest.mark.parametrize("row", rows("nesterov_worked.txt"))
def test_nesterov_golden(row):
    thg, u, Delta, eta, mu, u_exp, G_exp = row
    thg32 = np.array([thg], dtype=np.float32)
    snap = (thg32.astype(np.float64) + Delta).astype(np.float32)[None, :]
    r = run_single(orc.Hyper(M=1, outer_lr=eta, momentum=mu), snap.copy(), snap, thg32,
                   np.array([u], dtype=np.float32))
    assert abs(r.momentum[0] - u_exp) < 2e-7
    assert abs(r.theta_g[0] - G_exp) < 3e-7


def test_outer_update_matches_torch_nesterov_sgd():
    """Three outer steps equal torch's CPU SGD(nesterov=True) fed the gradient -Delta (in float64)."""
    M, n, eta, mu = 4, 64, 0.7, 0.9
    rng = np.random.default_rng(5)
    thg = (0.02 * rng.standard_normal(n)).astype(np.float32)
    p = torch.tensor(thg.astype(np.float64), requires_grad=True)
    opt = torch.optim.SGD([p], lr=eta, momentum=mu, nesterov=True)
    mom = np.zeros(n, dtype=np.float32)
    hp = orc.Hyper(M=M, outer_lr=eta, momentum=mu)
    for step in range(3):
        snap = (thg + 1e-3 * rng.standard_normal((M, n))).astype(np.float32)
        r = run_single(hp, snap.copy(), snap, thg, mom)
        # torch side, from the float32 state the oracle was given
        with torch.no_grad():
            p.copy_(torch.tensor(thg.astype(np.float64)))
        if step > 0:
            opt.state[p]["momentum_buffer"] = torch.tensor(-mom.astype(np.float64))
        p.grad = torch.tensor(-(snap.astype(np.float64) - thg.astype(np.float64)).mean(axis=0))
        opt.step()
        np.testing.assert_allclose(r.theta_g, p.detach().numpy(), rtol=1e-13, atol=1e-16)
        np.testing.assert_allclose(r.momentum, -opt.state[p]["momentum_buffer"].numpy(), rtol=1e-13, atol=1e-18)
        thg = r.theta_g.astype(np.float32)
        mom = r.momentum.astype(np.float32)


# ------------------------------------------------------------------ Eq. 4-7 and Eq. 3

@pytest.mark.parametrize("row", rows("delay_compensation_worked.txt"))
def test_delay_compensation_golden(row):
    sign, G, b, a, tau, H, lam, expected = row
    hp = orc.Hyper(M=1, H=int(H), tau=int(tau), lam=lam, alpha=1.0, sign_mode=int(sign))
    out = orc.merge(one_fragment(1), hp, np.array([[a]], dtype=np.float32),
                    np.array([[b]], dtype=np.float32), np.array([G], dtype=np.float32), [0])
    assert abs(out[0][0, 0] - expected) < 1e-7


@pytest.mark.parametrize("sign", [orc.SIGN_FORWARD, orc.SIGN_PRINTED, orc.SIGN_DESCENT])
@pytest.mark.parametrize("lam,tau", [(0.0, 1), (0.5, 4), (1.0, 8)])
def test_zero_delay_gives_global_state(sign, lam, tau):
    """No local change during the overlap: the corrected target is the new global state."""
    now, snap, thg, mom = rand_inputs(3, 200, seed=6)
    hp = orc.Hyper(M=3, tau=tau, lam=lam, sign_mode=sign)
    r = run_single(hp, snap.copy(), snap, thg, mom)
    for m in range(3):
        np.testing.assert_array_equal(r.w_now[m], r.theta_g)


def test_lambda_zero_is_linear_in_local_change():
    now, snap, thg, mom = rand_inputs(2, 300, seed=7)
    d = now.astype(np.float64) - snap.astype(np.float64)
    for sign, c1 in ((orc.SIGN_FORWARD, 1.0), (orc.SIGN_PRINTED, -1.0), (orc.SIGN_DESCENT, 1.0)):
        r = run_single(orc.Hyper(M=2, tau=4, lam=0.0, sign_mode=sign), now, snap, thg, mom)
        np.testing.assert_allclose(r.w_now - r.theta_g[None, :], c1 * d, rtol=1e-9, atol=1e-18)


def test_compensation_term_scaling_laws():
    """The second-order term is linear in lambda, in 1/tau, in 1/H, quadratic in d, linear in D."""
    rng = np.random.default_rng(8)
    n = 128
    G = (0.02 * rng.standard_normal(n)).astype(np.float32)
    b = (np.round((G + 1e-3 * rng.standard_normal(n)) * 2.0 ** 14) / 2.0 ** 14).astype(np.float32)[None, :]
    d = (2.0 ** -3) * np.sign(rng.standard_normal(n)).astype(np.float32)
    a = (b + d).astype(np.float32)
    assert np.array_equal(a.astype(np.float64) - b, d[None, :].astype(np.float64))

    def term(lam, tau, H, a_=a, sign=orc.SIGN_FORWARD):
        hp = orc.Hyper(M=1, tau=tau, H=H, lam=lam, sign_mode=sign)
        out = orc.merge(one_fragment(n), hp, a_, b, G, [0])[0]
        lin = orc.merge(one_fragment(n), orc.Hyper(M=1, tau=tau, H=H, lam=0.0, sign_mode=sign), a_, b, G, [0])[0]
        return out - lin

    base = term(0.5, 2, 4)
    D = G.astype(np.float64) - b[0]
    np.testing.assert_allclose(base[0], 0.5 / (2 * 4) * d.astype(np.float64) ** 2 * D, rtol=1e-8, atol=1e-20)
    np.testing.assert_allclose(term(1.0, 2, 4), 2 * base, rtol=1e-8, atol=1e-20)
    np.testing.assert_allclose(term(0.5, 4, 4), base / 2, rtol=1e-8, atol=1e-20)
    np.testing.assert_allclose(term(0.5, 2, 2), 2 * base, rtol=1e-8, atol=1e-20)
    a2 = (b + 2 * d).astype(np.float32)
    np.testing.assert_allclose(term(0.5, 2, 4, a_=a2), 4 * base, rtol=1e-8, atol=1e-20)
    np.testing.assert_allclose(term(0.5, 2, 4, sign=orc.SIGN_PRINTED), base, rtol=1e-8, atol=1e-20)
    np.testing.assert_allclose(term(0.5, 2, 4, sign=orc.SIGN_DESCENT), -base, rtol=1e-8, atol=1e-20)


def test_self_sync_is_a_no_op_for_forward_and_descent():
    """One worker, eta = 1, mu = 0: syncing a worker with itself must leave it where it is."""
    now, snap, thg, mom = rand_inputs(1, 100, seed=9)
    for sign in (orc.SIGN_FORWARD, orc.SIGN_DESCENT):
        hp = orc.Hyper(M=1, outer_lr=1.0, momentum=0.0, tau=3, lam=0.5, sign_mode=sign)
        r = run_single(hp, now, snap, thg, np.zeros_like(mom))
        np.testing.assert_allclose(r.w_now[0], now[0].astype(np.float64), rtol=0, atol=1e-17)
    hp = orc.Hyper(M=1, outer_lr=1.0, momentum=0.0, tau=3, lam=0.5, sign_mode=orc.SIGN_PRINTED)
    r = run_single(hp, now, snap, thg, np.zeros_like(mom))
    np.testing.assert_allclose(r.w_now[0], 2.0 * snap[0].astype(np.float64) - now[0], rtol=0, atol=1e-17)


def test_alpha_zero_keeps_local_parameters():
    now, snap, thg, mom = rand_inputs(2, 100, seed=10)
    r = run_single(orc.Hyper(M=2, alpha=0.0), now, snap, thg, mom)
    np.testing.assert_array_equal(r.w_now, now.astype(np.float64))


def test_reduces_to_streaming_diloco():
    """No compensation: Eq. 1-3, with the outer update from torch's Nesterov SGD and Eq. 3 as torch.lerp."""
    M, n, eta, mu, alpha = 4, 96, 0.7, 0.9, 0.5
    now, snap, thg, mom = rand_inputs(M, n, seed=11)
    p = torch.tensor(thg.astype(np.float64), requires_grad=True)
    opt = torch.optim.SGD([p], lr=eta, momentum=mu, nesterov=True)
    opt.state[p]["momentum_buffer"] = torch.tensor(-mom.astype(np.float64))
    p.grad = -(torch.tensor(snap.astype(np.float64)) - torch.tensor(thg.astype(np.float64))).mean(0)
    opt.step()
    G = p.detach()
    blended = torch.lerp(torch.tensor(now.astype(np.float64)), G[None, :].expand(M, n), alpha).numpy()
    for kw in (dict(comp_mode=orc.COMP_NONE, tau=3, lam=0.5), dict(comp_mode=orc.COMP_NONE, tau=0, lam=0.0)):
        r = run_single(orc.Hyper(M=M, outer_lr=eta, momentum=mu, alpha=alpha, **kw), now, snap, thg, mom)
        np.testing.assert_allclose(r.theta_g, G.numpy(), rtol=1e-13, atol=1e-17)
        np.testing.assert_allclose(r.w_now, blended, rtol=1e-13, atol=1e-17)
    # zero compensation strength and zero local change during the delay: same thing with alpha = 1
    r = run_single(orc.Hyper(M=M, outer_lr=eta, momentum=mu, alpha=1.0, lam=0.0, tau=3), snap.copy(), snap, thg, mom)
    np.testing.assert_allclose(r.w_now, np.broadcast_to(G.numpy(), (M, n)), rtol=1e-13, atol=1e-17)


def test_reduces_to_diloco():
    """One fragment, blocking sync (snapshot = current), alpha = 1: all workers leave with OuterOptim's result."""
    M, n, eta, mu = 3, 80, 0.7, 0.9
    now, snap, thg, mom = rand_inputs(M, n, seed=12)
    p = torch.tensor(thg.astype(np.float64), requires_grad=True)
    opt = torch.optim.SGD([p], lr=eta, momentum=mu, nesterov=True)
    opt.state[p]["momentum_buffer"] = torch.tensor(-mom.astype(np.float64))
    p.grad = -(torch.tensor(now.astype(np.float64)).mean(0) - torch.tensor(thg.astype(np.float64)))
    opt.step()
    r = run_single(orc.Hyper(M=M, outer_lr=eta, momentum=mu, tau=0), now, now, thg, mom)
    for m in range(M):
        np.testing.assert_allclose(r.w_now[m], p.detach().numpy(), rtol=1e-12, atol=1e-16)


def test_unprocessed_fragments_are_not_reported_and_layouts_agree():
    """Multi-segment fragments and a packed snapshot pool give the same numbers as the plain layout."""
    rng = np.random.default_rng(13)
    N, M = 1000, 2
    frags = [[(3, 100), (700, 57)], [(103, 250)], [(400, 299)]]
    thg = (0.02 * rng.standard_normal(N)).astype(np.float32)
    snap = (thg + 1e-3 * rng.standard_normal((M, N))).astype(np.float32)
    now = (snap + 1e-3 * rng.standard_normal((M, N))).astype(np.float32)
    mom = (1e-3 * rng.standard_normal(N)).astype(np.float32)
    hp = orc.Hyper(M=M, tau=2)
    res, last = orc.outer_step(frags, hp, now, snap, thg, mom, [2, 0], 7, 9, [0, 0, 5])
    assert sorted(res) == [0, 2] and list(last) == [9, 0, 9]
    # the same through a packed pool
    pool = np.zeros((M, 600), dtype=np.float32)
    snap_offset = [301, -1, 0]
    pool[:, 0:299] = snap[:, 400:699]
    pool[:, 301:401] = snap[:, 3:103]
    pool[:, 401:458] = snap[:, 700:757]
    res2, _ = orc.outer_step(frags, hp, now, pool, thg, mom, [2, 0], 7, 9, [0, 0, 5], snap_offset=snap_offset)
    for p in (0, 2):
        np.testing.assert_array_equal(res[p].w_now, res2[p].w_now)
        np.testing.assert_array_equal(res[p].theta_g, res2[p].theta_g)
    # fragment 0 equals running its two segments as separate single-segment problems
    a, _ = orc.outer_step([[(3, 100)], [(700, 57)]], hp, now, snap, thg, mom, [0, 1], 7, 9, [0, 0])
    np.testing.assert_array_equal(res[0].theta_g, np.concatenate([a[0].theta_g, a[1].theta_g]))
    assert res[0].sumsq == pytest.approx(a[0].sumsq + a[1].sumsq, rel=1e-15)
    # Eq. 10: I_p = t_p - t_{p,b}
    assert res[2].score == pytest.approx(res[2].norm / (7 - 5), rel=1e-15)
    assert res[0].score == pytest.approx(res[0].norm / 7, rel=1e-15)
    # threads only split the element range
    res3, _ = orc.outer_step(frags, hp, now, snap, thg, mom, [2, 0], 7, 9, [0, 0, 5], threads=3)
    np.testing.assert_array_equal(res[2].w_now, res3[2].w_now)
    assert res[2].sumsq == pytest.approx(res3[2].sumsq, rel=1e-14)


# ------------------------------------------------------------------ Eq. 10

def test_norm_closed_forms():
    n = 12345
    x = np.full(n, -0.25, dtype=np.float32)
    norms, scores = orc.fragment_scores([[(0, n)]], x, [5])
    assert norms[0] == pytest.approx(0.25 * math.sqrt(n), rel=1e-14)
    assert scores[0] == pytest.approx(norms[0] / 5, rel=1e-15)
    rng = np.random.default_rng(14)
    y = rng.standard_normal(5000).astype(np.float32)
    frags = [[(0, 1000)], [(1000, 1500), (4000, 1000)], [(2500, 1500)]]
    norms, _ = orc.fragment_scores(frags, y)
    assert math.sqrt((norms ** 2).sum()) == pytest.approx(np.linalg.norm(y.astype(np.float64)), rel=1e-13)
    assert norms[2] == pytest.approx(np.linalg.norm(y[2500:4000].astype(np.float64)), rel=1e-13)
    norms4, _ = orc.fragment_scores(frags, (4 * y).astype(np.float32))
    np.testing.assert_allclose(norms4, 4 * norms, rtol=1e-14)
    # interval 0 is treated as 1
    _, s0 = orc.fragment_scores(frags, y, [0, 0, 0])
    np.testing.assert_array_equal(s0, norms)


def test_step_norm_is_norm_of_delta():
    now, snap, thg, mom = rand_inputs(4, 777, seed=15)
    r = run_single(orc.Hyper(M=4), now, snap, thg, mom)
    assert r.norm == pytest.approx(np.linalg.norm(r.delta_g), rel=1e-13)


# ------------------------------------------------------------------ Algorithm 2 / Eq. 11

def alg2_single(t_g, H, R, last):
    """Algorithm 2 as printed: first overdue fragment, else the arg max of R (lowest index on ties)."""
    for p in range(len(R)):
        if t_g - last[p] >= H:
            return p
    return int(np.argmax(np.asarray(R, dtype=np.float64)))


def test_budget_one_is_algorithm_2():
    rng = np.random.default_rng(16)
    for trial in range(200):
        K = int(rng.integers(1, 9))
        R = rng.choice([0.5, 1.0, 2.0, 3.0, np.inf], size=K).astype(np.float32)
        last = rng.integers(0, 150, size=K)
        t = int(rng.integers(100, 260))
        sizes = rng.integers(1, 50, size=K)
        for kind, budget in ((orc.BUDGET_COUNT, 1), (orc.BUDGET_PARAMS, 0)):
            mask, ids, n = orc.select_fragments(R, last, sizes, t, 100, kind, budget)
            assert n == 1 and ids[0] == alg2_single(t, 100, R, last) and mask.sum() == 1 and mask[ids[0]] == 1


def test_never_synced_fragments_go_first_in_index_order():
    """All scores start at infinity: successive single selections walk 0, 1, 2, ... (the fixed schedule)."""
    K = 5
    R = np.full(K, np.inf, dtype=np.float32)
    last = np.zeros(K, dtype=np.int64)
    seen = []
    for t in range(1, K + 1):
        _, ids, _ = orc.select_fragments(R, last, np.ones(K), t, 100, orc.BUDGET_COUNT, 1)
        seen.append(int(ids[0]))
        R[ids[0]] = 1.0 / t
        last[ids[0]] = t
    assert seen == list(range(K))


def test_count_budget_brute_force():
    rng = np.random.default_rng(17)
    for trial in range(60):
        K = int(rng.integers(2, 9))
        B = int(rng.integers(1, K + 1))
        R = rng.permutation(K).astype(np.float32) + 1.0
        last = np.where(rng.random(K) < 0.25, 0, 90)
        t = 100
        overdue = [p for p in range(K) if t - last[p] >= 100]
        mask, ids, n = orc.select_fragments(R, last, np.ones(K), t, 100, orc.BUDGET_COUNT, B)
        assert n == B
        if len(overdue) <= B:
            best = max(itertools.combinations(range(K), B),
                       key=lambda S: (len(set(S) & set(overdue)), sum(R[list(S)])))
            assert sorted(ids) == sorted(best)
        else:
            assert list(ids) == overdue[:B]
        # admission order: overdue by index, then by falling score
        k = sum(1 for p in ids if p in overdue)
        assert list(ids[:k]) == sorted(ids[:k]) and all(p in overdue for p in ids[:k])
        assert list(R[ids[k:]]) == sorted(R[ids[k:]], reverse=True)


def test_params_budget_brute_force():
    """The greedy walk equals the lexicographically largest feasible subset in priority order."""
    rng = np.random.default_rng(18)
    for trial in range(40):
        K = int(rng.integers(2, 11))
        sizes = rng.integers(1, 40, size=K)
        R = rng.permutation(K).astype(np.float32) + 1.0
        last = np.where(rng.random(K) < 0.2, 0, 95)
        inel = (rng.random(K) < 0.2).astype(np.uint8)
        if inel.all():
            inel[0] = 0
        budget = int(rng.integers(0, sizes.sum() + 1))
        t = 100
        mask, ids, n = orc.select_fragments(R, last, sizes, t, 100, orc.BUDGET_PARAMS, budget, inel)
        elig = [p for p in range(K) if not inel[p]]
        # priority order built independently with numpy's lexsort: overdue first (by index), then -R, then index
        over = np.array([t - last[p] >= 100 for p in elig])
        key_score = np.where(over, 0.0, -R[elig])
        order = [elig[j] for j in np.lexsort((np.array(elig), key_score, ~over))]
        head, rest = order[0], order[1:]
        room = budget - sizes[head]
        best = ()
        for bits in itertools.product((1, 0), repeat=len(rest)):      # lexicographically descending
            S = [p for p, bsel in zip(rest, bits) if bsel]
            if sizes[S].sum() <= room:
                best = tuple(S)
                break
        assert list(ids) == [head] + list(best)
        assert mask.sum() == n and all(mask[p] for p in ids) and not any(mask[p] for p in range(K) if inel[p])
        left = budget - sizes[list(ids)].sum()
        assert all(sizes[p] > left for p in elig if not mask[p])         # nothing skipped still fits


def test_exact_budget_matches_the_textbook_knapsack_table():
    """The subset search (an option outside the paper) against the 0/1-knapsack dynamic programme over
    capacities: integer scores, so every sum is exact and the optimum value is unique."""
    rng = np.random.default_rng(23)
    for trial in range(40):
        K = int(rng.integers(1, 11))
        sizes = rng.integers(1, 30, size=K)
        R = rng.integers(0, 50, size=K).astype(np.float32)
        budget = int(rng.integers(0, sizes.sum() + 1))
        last = np.full(K, 95)
        mask, ids, n = orc.select_fragments(R, last, sizes, 100, 100, orc.BUDGET_PARAMS_EXACT, budget)
        table = np.zeros(budget + 1)                                   # best value within capacity c
        for p in range(K):
            for c in range(budget, int(sizes[p]) - 1, -1):
                table[c] = max(table[c], table[c - int(sizes[p])] + float(R[p]))
        chosen = list(ids)
        assert mask.sum() == n == len(set(chosen)) and all(mask[p] for p in chosen)
        if sizes[chosen].sum() > budget:                                # only the always-admitted head may overdraw
            assert n == 1 and table[budget] == 0.0 and chosen[0] == int(np.lexsort((np.arange(K), -R))[0])
        else:
            assert R[chosen].sum() == table[budget] or (table[budget] == 0.0 and n == 1)
        g_mask, g_ids, _ = orc.select_fragments(R, last, sizes, 100, 100, orc.BUDGET_PARAMS, budget)
        if sizes[list(g_ids)].sum() <= budget and sizes[chosen].sum() <= budget:
            assert R[chosen].sum() >= R[list(g_ids)].sum()              # never worse than the greedy walk


def test_exact_budget_forced_fragments_ties_and_head():
    sizes = [10, 10, 10, 10, 10]
    # fragment 3 overdue, fragment 1 never synced: both forced first (overdue before +inf), as in the greedy walk
    R = np.array([5.0, np.inf, 7.0, 1.0, 6.0], dtype=np.float32)
    last = [95, 95, 95, 0, 95]
    mask, ids, n = orc.select_fragments(R, last, sizes, 100, 100, orc.BUDGET_PARAMS_EXACT, 40)
    assert list(ids) == [3, 1, 2, 4]                                   # forced, then the best pair by score order
    # equal scores and sizes, room for one: the fragment earlier in the order (lower index) wins
    mask, ids, n = orc.select_fragments([2.0, 2.0, 2.0], [95] * 3, [10, 10, 10], 100, 100, orc.BUDGET_PARAMS_EXACT, 15)
    assert list(ids) == [0]
    # one big fragment beats two small ones where the greedy walk (score order) would take the small ones
    R = [4.0, 3.0, 6.5]
    mask, ids, n = orc.select_fragments(R, [95] * 3, [5, 5, 10], 100, 100, orc.BUDGET_PARAMS_EXACT, 10)
    assert list(ids) == [0, 1]                                          # 7.0 > 6.5
    mask, ids, n = orc.select_fragments([4.0, 2.0, 6.5], [95] * 3, [5, 5, 10], 100, 100, orc.BUDGET_PARAMS_EXACT, 10)
    assert list(ids) == [2]                                             # 6.5 > 6.0
    # nothing fits: a decision still returns the head of the order
    mask, ids, n = orc.select_fragments([1.0, 9.0], [95] * 2, [50, 60], 100, 100, orc.BUDGET_PARAMS_EXACT, 10)
    assert list(ids) == [1]
    # ineligible fragments never enter
    mask, ids, n = orc.select_fragments([1.0, 9.0, 3.0], [95] * 3, [5, 5, 5], 100, 100, orc.BUDGET_PARAMS_EXACT, 10,
                                        [0, 1, 0])
    assert list(ids) == [2, 0]


def test_selection_is_deterministic_and_rejects_nan():
    R = np.array([1.0, 3.0, 3.0, np.inf], dtype=np.float32)
    a = orc.select_fragments(R, [0] * 4, [1] * 4, 10, 100, orc.BUDGET_COUNT, 3)
    b = orc.select_fragments(R.copy(), [0] * 4, [1] * 4, 10, 100, orc.BUDGET_COUNT, 3)
    assert list(a[1]) == list(b[1]) == [3, 1, 2]
    with pytest.raises(ValueError):
        orc.select_fragments([1.0, float("nan")], [0, 0], [1, 1], 1, 100, orc.BUDGET_COUNT, 1)
    mask, ids, n = orc.select_fragments([1.0, 2.0], [0, 0], [1, 1], 1, 100, orc.BUDGET_COUNT, 1, [1, 1])
    assert n == 0 and mask.sum() == 0


# ------------------------------------------------------------------ worker-per-device deployment (Section 2.1)

def test_received_sum_mode_equals_stacked_workers():
    """Two devices with two workers each, their pseudo-gradient sums all-reduced, reproduce the four stacked workers."""
    M, n = 4, 500
    now, snap, thg, mom = rand_inputs(M, n, seed=21)
    # quantise so that every partial sum is exact in fp32 and the comparison can be bit for bit
    q = lambda x: (np.round(x * 2.0 ** 16) / 2.0 ** 16).astype(np.float32)
    snap, thg = q(snap), q(thg)
    frs = one_fragment(n)
    parts = [orc.pseudo_gradient_sum(frs, 2, np.ascontiguousarray(snap[d * 2:d * 2 + 2]), thg, [0])[0] for d in range(2)]
    np.testing.assert_array_equal(parts[0], (snap[0].astype(np.float64) - thg) + (snap[1].astype(np.float64) - thg))
    total = (parts[0] + parts[1]).astype(np.float32)
    assert np.array_equal(total.astype(np.float64), parts[0] + parts[1])
    hp4 = orc.Hyper(M=4, tau=3)
    full = run_single(hp4, now, snap, thg, mom)
    for d in range(2):
        hp2 = orc.Hyper(M=2, tau=3)
        res, last = orc.outer_step(frs, hp2, np.ascontiguousarray(now[d * 2:d * 2 + 2]),
                                   np.ascontiguousarray(snap[d * 2:d * 2 + 2]), thg, mom, [0], 10, 12, [0],
                                   recv_sum=total, M_total=4)
        r = res[0]
        np.testing.assert_array_equal(r.theta_g, full.theta_g)
        np.testing.assert_array_equal(r.momentum, full.momentum)
        np.testing.assert_array_equal(r.w_now, full.w_now[d * 2:d * 2 + 2])
        assert r.norm == full.norm and list(last) == [12]
        # the same from the two devices' partial sums, left for the step to add up
        res2, _ = orc.outer_step(frs, hp2, np.ascontiguousarray(now[d * 2:d * 2 + 2]),
                                 np.ascontiguousarray(snap[d * 2:d * 2 + 2]), thg, mom, [0], 10, 12, [0],
                                 recv_sum=[parts[0].astype(np.float32), parts[1].astype(np.float32)], M_total=4)
        np.testing.assert_array_equal(res2[0].theta_g, full.theta_g)
        np.testing.assert_array_equal(res2[0].w_now, full.w_now[d * 2:d * 2 + 2])
    with pytest.raises(ValueError):
        orc.outer_step(frs, orc.Hyper(M=2), now[:2], snap[:2], thg, mom, [0], 10, 12, [0], recv_sum=total)
