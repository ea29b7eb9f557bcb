"""Pins for the CPU oracle: it is checked against things other than itself.

Hand-worked examples (tests/golden), torch.optim library routines for M = 1,
closed forms, invariants that follow from the algorithms' linearity, the
clipping bounds of Eqs. 5-6 and the communication ratios the paper prints.
"""
import json
import math
import os
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from oracle import ADAM, ADOPT, SGDM, SYNC_U, SYNC_V, SYNC_X

GOLD = os.path.join(os.path.dirname(__file__), "golden", "hand_examples.json")


def f32(a):
    return np.array(a, dtype=np.float32, order="C", copy=True)


def zeros(M, n):
    return np.zeros((M, n), dtype=np.float32)


def run_steps(cfg, T, lr, x, u, v, g_of_t, clip_bound=None):
    masks = []
    for t in range(T):
        cb = clip_bound(t) if clip_bound else 0.0
        lr_t = lr(t) if callable(lr) else lr
        masks.append(oracle.step(cfg, t, lr_t, x, u, v, f32(g_of_t(t)), clip_bound=cb))
    return masks


# --------------------------------------------------------------------------- hand examples
def test_hand_example_sgdm_exact_rationals():
    ex = json.load(open(GOLD))["sgdm"]
    cfg = oracle.make_cfg(2, SGDM, beta1=0.5, Kx=ex["Kx"], Ku=ex["Ku"], Kv=0)
    x = f32([[1.0], [1.0]])
    u = zeros(2, 1)
    for t, g in enumerate(ex["g"]):
        gt = f32([[float(Fraction(g[0]))], [float(Fraction(g[1]))]])
        mask = oracle.step(cfg, t, 0.1, x, u, None, gt)
        assert [int(bool(mask & SYNC_X)), int(bool(mask & SYNC_U))] == ex["masks_xu"][t]
        for m in range(2):
            # u is dyadic here (exact in fp32); x involves 1/10, rounded to fp32 each step
            assert float(u[m, 0]) == float(Fraction(ex["u"][t][m]))
            assert abs(float(x[m, 0]) - float(Fraction(ex["x"][t][m]))) < 2.5e-7
        assert abs(float(x.astype(np.float64).mean()) - float(Fraction(ex["mean_x"][t]))) < 2.5e-7


def test_hand_example_adam():
    ex = json.load(open(GOLD))["adam"]
    cfg = oracle.make_cfg(2, ADAM, beta1=0.5, beta2=0.5, eps=0.0, Kx=ex["Kx"], Ku=ex["Ku"],
                          Kv=ex["Kv"])
    x, u, v = f32([[1.0], [1.0]]), zeros(2, 1), zeros(2, 1)
    for t, g in enumerate(ex["g"]):
        mask = oracle.step(cfg, t, 0.1, x, u, v, f32([[g[0]], [g[1]]]))
        bits = [int(bool(mask & b)) for b in (SYNC_X, SYNC_U, SYNC_V)]
        assert bits == ex["masks_xuv"][t]
        for m in range(2):
            assert float(u[m, 0]) == ex["u"][t][m]
            assert float(v[m, 0]) == ex["v"][t][m]
            assert abs(float(x[m, 0]) - ex["x"][t][m]) < 3e-7


def test_hand_example_adopt():
    ex = json.load(open(GOLD))["adopt"]
    cfg = oracle.make_cfg(2, ADOPT, beta1=0.5, beta2=0.5, eps=ex["eps"], Kx=ex["Kx"],
                          Ku=ex["Km"], Kv=ex["Kv"])
    x, u, v = f32([[1.0], [1.0]]), zeros(2, 1), f32([[1.0], [1.0]])
    for t, g in enumerate(ex["g"]):
        mask = oracle.step(cfg, t, 0.1, x, u, v, f32([[g[0]], [g[1]]]))
        bits = [int(bool(mask & b)) for b in (SYNC_X, SYNC_U, SYNC_V)]
        assert bits == ex["masks_xuv"][t]
        for m in range(2):
            assert abs(float(u[m, 0]) - ex["m"][t][m]) < 4e-7
            assert float(v[m, 0]) == ex["v"][t][m]
            assert abs(float(x[m, 0]) - ex["x"][t][m]) < 4e-7


# --------------------------------------------------------------------------- M = 1 vs library
@pytest.mark.parametrize("K", [(1, 1, 1), (3, 5, 7), (0, 0, 0)])
@pytest.mark.parametrize("wd", [0.0, 0.1])
def test_m1_is_plain_adam(K, wd):
    """M = 1: averaging is the identity, so any schedule gives Adam (Eqs. 1-2 and Algorithm 2's
    direction).  With lambda = 0 and the bias correction folded into eta_t this is
    torch.optim.Adam / AdamW(eps=0) in fp64; AdamW's decoupled decay pins the weight-decay form."""
    rng = np.random.default_rng(1)
    n, T, lr, b1, b2 = 48, 40, 1e-2, 0.9, 0.99
    x0 = rng.normal(size=n)
    grads = rng.normal(size=(T, n)).astype(np.float32)
    p = torch.nn.Parameter(torch.tensor(x0.astype(np.float32), dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=0.0, weight_decay=wd)
    cfg = oracle.make_cfg(1, ADAM, beta1=b1, beta2=b2, eps=0.0, weight_decay=wd,
                          Kx=K[0], Ku=K[1], Kv=K[2])
    x, u, v = f32(x0[None]), zeros(1, n), zeros(1, n)
    for t in range(T):
        eta_t = lr * math.sqrt(1 - b2 ** (t + 1)) / (1 - b1 ** (t + 1))
        # torch decays with lr*wd; the oracle with eta_t*wd: rescale torch's group per step
        opt.param_groups[0]["weight_decay"] = wd * eta_t / lr
        p.grad = torch.tensor(grads[t], dtype=torch.float64)
        opt.step()
        oracle.step(cfg, t, eta_t, x, u, v, f32(grads[t][None]))
    ref = p.detach().numpy()
    assert np.max(np.abs(x[0] - ref)) < 5e-6          # fp32 storage of x ~ O(1) over 40 steps
    assert np.max(np.abs(x[0] - x0)) > 0.05           # the run moved far more than the tolerance


@pytest.mark.parametrize("K", [(1, 1, 0), (4, 2, 0)])
def test_m1_is_plain_sgdm(K):
    """M = 1 SGDM equals torch.optim.SGD(momentum=beta, dampening=beta), whose buffer update is
    buf = momentum*buf + (1-dampening)*g; that routine starts its buffer at the raw first
    gradient, i.e. u_{-1} = g_0."""
    rng = np.random.default_rng(2)
    n, T, lr, beta = 32, 30, 0.05, 0.9
    x0 = rng.normal(size=n).astype(np.float32)
    grads = rng.normal(size=(T, n)).astype(np.float32)
    p = torch.nn.Parameter(torch.tensor(x0, dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=lr, momentum=beta, dampening=beta)
    cfg = oracle.make_cfg(1, SGDM, beta1=beta, Kx=K[0], Ku=K[1], Kv=0)
    x, u = f32(x0[None]), f32(grads[0][None])
    for t in range(T):
        p.grad = torch.tensor(grads[t], dtype=torch.float64)
        opt.step()
        oracle.step(cfg, t, lr, x, u, None, f32(grads[t][None]))
    assert np.max(np.abs(x[0] - p.detach().numpy())) < 5e-6
    assert np.max(np.abs(u[0] - opt.state[p]["momentum_buffer"].numpy())) < 1e-6


# --------------------------------------------------------------------------- identical gradients
@pytest.mark.parametrize("opt,K", [(ADAM, (1, 1, 1)), (ADAM, (2, 3, 5)), (ADOPT, (3, 2, 4)),
                                   (SGDM, (2, 5, 0))])
@pytest.mark.parametrize("M", [2, 3, 4, 8])
def test_identical_gradients_match_single_worker(opt, K, M):
    """Same start and same gradients on every worker: the mean of equal values is that value,
    so every replica follows the M = 1 run bit for bit, whatever the schedule (K = 1 is the
    DDP-equivalent baseline of Section 5.1)."""
    rng = np.random.default_rng(3)
    n, T = 17, 24
    x0 = rng.normal(size=n).astype(np.float32)
    grads = rng.normal(size=(T, n)).astype(np.float32)
    kw = dict(beta1=0.9, beta2=0.99, eps=1e-6, clip_rho=1.5, Kx=K[0], Ku=K[1], Kv=K[2])
    xs, us, vs = f32(x0[None]), zeros(1, n), f32(np.full((1, n), 0.3))
    xm, um, vm = f32(np.tile(x0, (M, 1))), zeros(M, n), f32(np.full((M, n), 0.3))
    c1, cM = oracle.make_cfg(1, opt, **kw), oracle.make_cfg(M, opt, **kw)
    for t in range(T):
        oracle.step(c1, t, 1e-2, xs, us, None if opt == SGDM else vs, f32(grads[t][None]))
        oracle.step(cM, t, 1e-2, xm, um, None if opt == SGDM else vm,
                    f32(np.tile(grads[t], (M, 1))))
    for m in range(M):
        assert np.array_equal(xm[m], xs[0]) and np.array_equal(um[m], us[0])
        if opt != SGDM:
            assert np.array_equal(vm[m], vs[0])


def test_k1_with_different_gradients_is_not_single_worker_adam():
    """Averaging states is not averaging gradients: mean(g^2) != mean(g)^2, so K = 1 with
    different per-worker gradients must differ from Adam on the mean gradient."""
    n = 8
    g = f32([[1.0] * n, [3.0] * n])
    cfg = oracle.make_cfg(2, ADAM, beta1=0.5, beta2=0.5, eps=0.0)
    x, u, v = zeros(2, n), zeros(2, n), zeros(2, n)
    oracle.step(cfg, 0, 0.1, x, u, v, g)
    oracle.step(cfg, 1, 0.1, x, u, v, g)
    # t=1: v = 0.5*mean(0.5, 4.5) + 0.5*g^2 = (1.75, 5.75); Adam on mean g = 2 would hold 3.0
    assert np.allclose(v[:, 0], [1.75, 5.75]) and not np.allclose(v[:, 0], 3.0)


# --------------------------------------------------------------------------- mean preservation
def _mean(a):
    return a.astype(np.float64).mean(axis=0)


@pytest.mark.parametrize("M", [2, 4])
def test_state_means_do_not_depend_on_schedule_exact(M):
    """The moment recursions are linear in the state, so mean_m u_t and mean_m v_t are the same
    for every (K_u, K_v); for SGDM mean_m x_t is centralized SGDM on the mean gradient (Step 1 of
    the SGDM appendix).  beta = 1/2 and small integer gradients keep every value exact in fp32."""
    rng = np.random.default_rng(4)
    n, T = 9, 7
    grads = rng.integers(-4, 5, size=(T, M, n)).astype(np.float32)
    ref = None
    for K in [(1, 1, 1), (2, 3, 2), (0, 0, 0), (5, 2, 3)]:
        cfg = oracle.make_cfg(M, ADAM, beta1=0.5, beta2=0.5, eps=0.0, Kx=K[0], Ku=K[1], Kv=K[2])
        x, u, v = zeros(M, n), zeros(M, n), zeros(M, n)
        trace = []
        for t in range(T):
            oracle.step(cfg, t, 0.125, x, u, v, f32(grads[t]))
            trace.append((_mean(u).copy(), _mean(v).copy()))
        if ref is None:
            ref = trace
        for (a, b), (c, d) in zip(trace, ref):
            assert np.array_equal(a, c) and np.array_equal(b, d)
    # closed form of the mean: EMA of the mean gradient / mean squared gradient
    ubar = np.zeros(n)
    vbar = np.zeros(n)
    for t in range(T):
        ubar = 0.5 * ubar + 0.5 * grads[t].astype(np.float64).mean(axis=0)
        vbar = 0.5 * vbar + 0.5 * (grads[t].astype(np.float64) ** 2).mean(axis=0)
        assert np.array_equal(ref[t][0], ubar) and np.array_equal(ref[t][1], vbar)


@pytest.mark.parametrize("K", [(1, 1), (2, 3), (3, 2), (0, 4), (4, 0)])
def test_sgdm_mean_iterate_is_centralized_sgdm(K):
    M, n, T, beta, eta = 4, 6, 8, 0.5, 0.25
    rng = np.random.default_rng(5)
    grads = rng.integers(-3, 4, size=(T, M, n)).astype(np.float32)
    cfg = oracle.make_cfg(M, SGDM, beta1=beta, Kx=K[0], Ku=K[1], Kv=0)
    x0 = rng.integers(-2, 3, size=n).astype(np.float32)
    x, u = f32(np.tile(x0, (M, 1))), zeros(M, n)
    xc, uc = x0.astype(np.float64), np.zeros(n)
    for t in range(T):
        oracle.step(cfg, t, eta, x, u, None, f32(grads[t]))
        uc = beta * uc + (1 - beta) * grads[t].astype(np.float64).mean(axis=0)
        xc = xc - eta * uc
        assert np.array_equal(_mean(u), uc)
        assert np.array_equal(_mean(x), xc)


def test_averaging_step_preserves_the_mean_of_the_averaged_array():
    """One step with zero gradient and beta = 1 - 2^-k... simplest: g = 0, so u_t = beta * (mean or
    own u): the worker-mean of u_t is beta * mean(u_{t-1}) whether or not u is averaged."""
    M, n = 3, 5
    rng = np.random.default_rng(6)
    u0 = rng.integers(-8, 9, size=(M, n)).astype(np.float32) * 3  # multiples of 3: mean over 3 exact
    for Ku in (1, 0):
        cfg = oracle.make_cfg(M, SGDM, beta1=0.5, Kx=0, Ku=Ku, Kv=0)
        x, u = zeros(M, n), u0.copy()
        oracle.step(cfg, 0, 0.0, x, u, None, zeros(M, n))
        assert np.array_equal(_mean(u), 0.5 * _mean(u0))
        if Ku == 1:
            assert np.array_equal(u[0], u[1]) and np.array_equal(u[1], u[2])


# --------------------------------------------------------------------------- clipping
def test_coordinate_clip_definition():
    """clip(X, rho)_i = sgn(X_i) min(|X_i|, rho) (Section 3.1); rho <= 0 switches it off."""
    g = f32([[-5.0, -1.0, -0.25, 0.0, 0.25, 1.0, 5.0]])
    for rho, want in [(1.0, [-1, -1, -0.25, 0, 0.25, 1, 1]), (0.0, [-5, -1, -0.25, 0, 0.25, 1, 5]),
                      (-1.0, [-5, -1, -0.25, 0, 0.25, 1, 5]), (0.5, [-0.5, -0.5, -0.25, 0, 0.25, 0.5, 0.5])]:
        cfg = oracle.make_cfg(1, SGDM, beta1=0.0, clip_rho=rho, Kx=0, Ku=0, Kv=0)
        x, u = zeros(1, 7), zeros(1, 7)
        oracle.step(cfg, 0, 1.0, x, u, None, g)
        assert np.array_equal(u[0], f32(want))       # beta = 0: u = clipped g
        assert np.array_equal(x[0], -f32(want))      # x = 0 - 1 * u


@pytest.mark.parametrize("K", [(1, 1, 1), (3, 4, 6), (0, 0, 0)])
def test_bounds_under_clipping(K):
    """Eqs. 5-6 and the lemma of the max-change appendix: with |g_i| <= rho and zero seeds,
    |u_t| <= rho, v_t <= rho^2, |u_{t+K}-u_t| <= 2 rho (1-beta1^K), |v_{t+K}-v_t| <= 2 rho^2 (1-beta2^K).
    Averaging is a convex combination, so the bounds on |u|, v hold for every worker and schedule;
    the drift bounds are checked at M = 1."""
    rng = np.random.default_rng(7)
    rho, b1, b2, n, T = 0.75, 0.9, 0.97, 33, 60
    for M in (1, 4):
        cfg = oracle.make_cfg(M, ADAM, beta1=b1, beta2=b2, eps=1e-8, clip_rho=rho,
                              Kx=K[0], Ku=K[1], Kv=K[2])
        x, u, v = zeros(M, n), zeros(M, n), zeros(M, n)
        us, vs = [], []
        for t in range(T):
            g = rng.standard_cauchy(size=(M, n)).astype(np.float32) * 2  # heavy tails: clip active
            oracle.step(cfg, t, 1e-3, x, u, v, f32(g))
            assert np.max(np.abs(u)) <= rho * (1 + 1e-6)
            assert np.max(v) <= rho * rho * (1 + 1e-6) and np.min(v) >= 0
            us.append(u.astype(np.float64).copy())
            vs.append(v.astype(np.float64).copy())
        assert np.max(np.abs(us[-1])) > 0.2 * rho   # not vacuous
        if M == 1:
            for Kd in (1, 5, 17):
                for t in range(T - Kd):
                    assert np.max(np.abs(us[t + Kd] - us[t])) <= 2 * rho * (1 - b1 ** Kd) + 1e-6
                    assert np.max(np.abs(vs[t + Kd] - vs[t])) <= 2 * rho ** 2 * (1 - b2 ** Kd) + 1e-6


# --------------------------------------------------------------------------- schedule
def _counts(opt, K, T):
    c = [0, 0, 0]
    for t in range(T):
        m = oracle.sync_mask(opt, K[0], K[1], K[2], t)
        for b in range(3):
            c[b] += (m >> b) & 1
    return c


def test_schedule_matches_printed_communication_ratios():
    """Wall-clock appendix / Section 6 (RQ4): against DDP (one sync per step), periods
    (256, 768, 1536) cut communication 170x, Local Adam at K = 256 (three states) 85x, parameters
    only 256x; Section 6 (RQ3): K_u = 3 K_x, K_v = 6 K_x halves Local Adam's cost."""
    T = 1536 * 4
    ddp = T  # one payload per step
    assert round(ddp / sum(_counts(ADAM, (256, 768, 1536), T))) == 171  # 170.67: printed as 170x
    assert int(ddp / sum(_counts(ADAM, (256, 768, 1536), T))) == 170
    assert int(ddp / sum(_counts(ADAM, (256, 256, 256), T))) == 85
    assert ddp // sum(_counts(ADAM, (256, 0, 0), T)) == 256
    for Kx in (16, 256):
        T2 = 6 * Kx * 8
        local = sum(_counts(ADAM, (Kx, Kx, Kx), T2))
        des = sum(_counts(ADAM, (Kx, 3 * Kx, 6 * Kx), T2))
        assert local == 2 * des


def test_schedule_is_t_mod_k_from_zero():
    assert oracle.sync_mask(ADAM, 4, 8, 16, 0) == 7           # t = 0 syncs everything
    assert oracle.sync_mask(ADAM, 4, 8, 16, 4) == SYNC_X
    assert oracle.sync_mask(ADAM, 4, 8, 16, 8) == SYNC_X | SYNC_U
    assert oracle.sync_mask(ADAM, 4, 8, 16, 16) == 7
    assert oracle.sync_mask(ADAM, 4, 8, 16, 5) == 0
    assert oracle.sync_mask(ADAM, 0, 0, 0, 0) == 0            # K = infinity: never
    assert oracle.sync_mask(SGDM, 1, 1, 1, 0) == SYNC_X | SYNC_U  # SGDM has no second state
    for K in [(3, 5, 7), (2, 2, 2), (1, 4, 6)]:
        for T in (1, 10, 211):
            want = [-(-T // k) for k in K]                    # ceil(T / K) syncs in [0, T)
            assert _counts(ADAM, K, T) == want


def test_full_sync_at_multiples_of_lcm():
    """High-probability appendix: at multiples of lcm(K_x, K_u, K_v) all three arrays are averaged,
    so every worker enters that step with identical inputs; feeding one shared gradient at that
    step leaves all replicas bitwise equal."""
    M, n, K = 3, 11, (2, 3, 4)
    L = 12
    rng = np.random.default_rng(8)
    cfg = oracle.make_cfg(M, ADAM, beta1=0.9, beta2=0.99, eps=1e-8, Kx=K[0], Ku=K[1], Kv=K[2])
    x, u, v = f32(np.tile(rng.normal(size=n), (M, 1))), zeros(M, n), zeros(M, n)
    for t in range(2 * L + 1):
        if t % L == 0:
            g = np.tile(rng.normal(size=n), (M, 1))
        else:
            g = rng.normal(size=(M, n))
        mask = oracle.step(cfg, t, 1e-2, x, u, v, f32(g))
        if t % L == 0:
            assert mask == 7
            for a in (x, u, v):
                assert np.array_equal(a[0], a[1]) and np.array_equal(a[1], a[2])
        elif t % L == 1:
            assert not np.array_equal(x[0], x[1])             # they do diverge in between


# --------------------------------------------------------------------------- brute force
def _brute(opt, M, K, T, lr, b1, b2, eps, rho, wd, x0, u0, v0, grads, norm_clip=None, post=False):
    """Independent re-evaluation in 40-digit decimal arithmetic, worker-outer loop order,
    fp32 storage emulated by rounding through numpy.float32."""
    getcontext().prec = 40
    D = Decimal
    r32 = lambda a: D(float(np.float32(float(a))))
    n = len(x0[0])
    X = [[D(float(a)) for a in row] for row in x0]
    U = [[D(float(a)) for a in row] for row in u0]
    V = [[D(float(a)) for a in row] for row in v0]
    b1, b2, lr, wd, eps = D(b1), D(b2), D(lr), D(wd), D(eps)
    for t in range(T):
        sx = K[0] > 0 and t % K[0] == 0
        su = K[1] > 0 and t % K[1] == 0
        sv = opt != SGDM and K[2] > 0 and t % K[2] == 0
        mean = lambda A, i: sum(A[m][i] for m in range(M)) / D(M)
        Xb = [mean(X, i) for i in range(n)]
        Ub = [mean(U, i) for i in range(n)]
        Vb = [mean(V, i) for i in range(n)]
        nX = [[None] * n for _ in range(M)]
        nU = [[None] * n for _ in range(M)]
        nV = [[None] * n for _ in range(M)]
        for m in range(M):
            for i in range(n):
                g = D(float(grads[t][m][i]))
                if rho > 0:
                    g = max(min(g, D(rho)), -D(rho))
                up = Ub[i] if (su and not post) else U[m][i]
                vp = Vb[i] if (sv and not post) else V[m][i]
                if opt == ADAM:
                    nU[m][i] = b1 * up + (1 - b1) * g
                    nV[m][i] = b2 * vp + (1 - b2) * g * g
                elif opt == ADOPT:
                    nV[m][i] = b2 * vp + (1 - b2) * g * g
                    r = g / max(V[m][i].sqrt(), eps)
                    if norm_clip is not None:
                        c = D(norm_clip(t))
                        r = max(min(r, c), -c)
                    nU[m][i] = b1 * up + (1 - b1) * r
                else:
                    nU[m][i] = b1 * up + (1 - b1) * g
                    nV[m][i] = D(0)
        if post:
            for i in range(n):
                if su:
                    a = mean(nU, i)
                    for m in range(M):
                        nU[m][i] = a
                if sv:
                    a = mean(nV, i)
                    for m in range(M):
                        nV[m][i] = a
        for m in range(M):
            for i in range(n):
                xp = Xb[i] if (sx and not post) else X[m][i]
                if opt == ADAM:
                    d = lr * nU[m][i] / (nV[m][i] + eps * eps).sqrt()
                else:
                    d = lr * nU[m][i]
                nX[m][i] = xp * (1 - lr * wd) - d
        if post and sx:
            for i in range(n):
                a = mean(nX, i)
                for m in range(M):
                    nX[m][i] = a
        X = [[r32(a) for a in row] for row in nX]
        U = [[r32(a) for a in row] for row in nU]
        V = [[r32(a) for a in row] for row in nV]
    tof = lambda A: np.array([[float(a) for a in row] for row in A], dtype=np.float32)
    return tof(X), tof(U), tof(V)


def _close(a, b):
    """Agreement to about one fp32 rounding of the stored state: the oracle's own fp64 rounding can
    tip a value across an fp32 rounding boundary once in a while, and a one-ulp difference in a
    stored state then rides along (shrinking) in later steps."""
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    return bool(np.all(np.abs(a - b) <= 1.5e-7 * np.abs(b) + 2e-8))


@pytest.mark.parametrize("M", [1, 2, 3, 4, 8])
@pytest.mark.parametrize("opt", [ADAM, ADOPT, SGDM])
@pytest.mark.parametrize("post", [False, True])
def test_brute_force_small(M, opt, post):
    """N <= 8, T = 3 steps; periods (1, 2, 3) plus a second run with (2, 3, 1) reach all sync
    patterns; a slow decimal re-evaluation with another loop order must agree to about one fp32
    ulp of the stored state, and exactly on almost every element."""
    rng = np.random.default_rng(100 + 10 * M + opt)
    n, T = 7, 3
    for K in [(1, 2, 3), (2, 3, 1), (3, 1, 2)]:
        x0 = np.tile(rng.normal(size=n) * 0.5, (M, 1)).astype(np.float32)
        u0 = (rng.normal(size=(M, n)) * 0.1).astype(np.float32)
        v0 = (rng.uniform(0.05, 0.5, size=(M, n))).astype(np.float32)
        grads = rng.normal(size=(T, M, n)).astype(np.float32)
        # fp32-representable hyper-parameters, as they cross the library's ABI.  (A beta of
        # exactly 9/10 would put (9u+g)/10 on an fp32 rounding tie for one element in ten.)
        b1, b2, lr, wd = (float(np.float32(a)) for a in (0.9, 0.99, 0.03, 0.05))
        kw = dict(beta1=b1, beta2=b2, eps=1e-3, weight_decay=wd, clip_rho=1.25,
                  Kx=K[0], Ku=K[1], Kv=K[2])
        flags = (oracle.FLAG_POST_AVERAGE if post else 0) | (oracle.FLAG_ADOPT_NORM_CLIP if opt == ADOPT else 0)
        cfg = oracle.make_cfg(M, opt, flags=flags, **kw)
        nc = (lambda t: 0.5 + t) if opt == ADOPT else None
        x, u, v = x0.copy(), u0.copy(), v0.copy()
        for t in range(T):
            oracle.step(cfg, t, lr, x, u, None if opt == SGDM else v, f32(grads[t]),
                        clip_bound=(nc(t) if nc else 0.0))
        bx, bu, bv = _brute(opt, M, K, T, lr, b1, b2, 1e-3, 1.25, wd, x0, u0, v0, grads,
                            norm_clip=nc, post=post)
        assert _close(x, bx) and _close(u, bu)
        exact = [np.mean(x == bx), np.mean(u == bu)]
        if opt != SGDM:
            assert _close(v, bv)
            exact.append(np.mean(v == bv))
        assert min(exact) >= 0.98


# --------------------------------------------------------------------------- post-average ordering
def test_post_average_full_sync_makes_replicas_equal_and_k1_is_minibatch_sgdm():
    """Algorithm 4 with p_x = p_u = 1: every worker holds the average after each step, and the
    run is mini-batch SGDM on the mean gradient (the remark after Theorem 1)."""
    M, n, T, beta, eta = 4, 5, 6, 0.5, 0.25
    rng = np.random.default_rng(9)
    grads = rng.integers(-3, 4, size=(T, M, n)).astype(np.float32)
    cfg = oracle.make_cfg(M, SGDM, beta1=beta, Kx=1, Ku=1, Kv=0, flags=oracle.FLAG_POST_AVERAGE)
    x, u = zeros(M, n), zeros(M, n)
    xc, uc = np.zeros(n), np.zeros(n)
    for t in range(T):
        oracle.step(cfg, t, eta, x, u, None, f32(grads[t]))
        uc = beta * uc + (1 - beta) * grads[t].astype(np.float64).mean(axis=0)
        xc = xc - eta * uc
        for m in range(M):
            assert np.array_equal(x[m].astype(np.float64), xc)
            assert np.array_equal(u[m].astype(np.float64), uc)


@pytest.mark.parametrize("opt", [ADAM, SGDM])
def test_post_average_equals_pre_average_shifted_by_one_step(opt):
    """Averaging the previous state at the start of step t (Algorithms 1-3) is the same process
    as averaging the new state at the end of step t-1 (Algorithms 4-5) for everything that is
    linear in the state: the moments u, v of Adam, and u and x of SGDM.  With K = 1 on every
    array the post-average run after T steps equals the worker-mean of the pre-average run.
    (Adam's x is excluded: its direction u / sqrt(v) is not linear, so the two orderings differ.)"""
    M, n, T = 3, 6, 5
    rng = np.random.default_rng(10)
    grads = rng.normal(size=(T, M, n)).astype(np.float32)
    x0 = np.tile(rng.normal(size=n), (M, 1)).astype(np.float32)
    kw = dict(beta1=0.9, beta2=0.99, eps=1e-8, Kx=1, Ku=1, Kv=1)
    res = {}
    for post in (False, True):
        cfg = oracle.make_cfg(M, opt, flags=oracle.FLAG_POST_AVERAGE if post else 0, **kw)
        x, u, v = x0.copy(), zeros(M, n), zeros(M, n)
        for t in range(T):
            oracle.step(cfg, t, 1e-2, x, u, None if opt == SGDM else v, f32(grads[t]))
        res[post] = (x, u, v)
    which = (0, 1) if opt == SGDM else (1, 2)
    for j in which:
        a_pre, a_post = res[False][j], res[True][j]
        # the two runs round at different places (pre: per worker; post: after the mean)
        assert np.allclose(_mean(a_pre), a_post[0].astype(np.float64), rtol=3e-6, atol=1e-8)
        assert np.array_equal(a_post[0], a_post[1]) and np.array_equal(a_post[1], a_post[2])
    if opt == ADAM:
        assert not np.allclose(_mean(res[False][0]), res[True][0][0].astype(np.float64), rtol=1e-7, atol=0)


# --------------------------------------------------------------------------- norm-based clipping
def test_norm_scales_match_torch_clip_grad_norm():
    """Library routine: torch.nn.utils.clip_grad_norm_ scales by max_norm / (norm + 1e-6) (clamped
    to 1); the oracle by max_norm / norm.  They agree to that epsilon."""
    rng = np.random.default_rng(11)
    sizes = [7, 130, 1, 64]
    for scale, max_norm in [(1.0, 1.0), (1e-3, 1.0), (5.0, 0.25)]:
        tensors = [rng.normal(size=s).astype(np.float32) * scale for s in sizes]
        params = [torch.nn.Parameter(torch.zeros(s, dtype=torch.float64)) for s in sizes]
        for p, t in zip(params, tensors):
            p.grad = torch.tensor(t, dtype=torch.float64)
        total = float(torch.nn.utils.clip_grad_norm_(params, max_norm))
        flat = f32(np.concatenate(tensors)[None])
        norms, scales = oracle.norm_scales(flat, max_norm)
        assert abs(norms[0] - total) <= 1e-12 * total
        clipped = np.concatenate([p.grad.numpy() for p in params])
        assert np.allclose(flat[0].astype(np.float64) * scales[0], clipped, rtol=3e-6, atol=0)
        if total <= max_norm:
            assert scales[0] == 1.0


def test_norm_clip_closed_forms():
    g = f32([[3.0, 4.0, 0.0], [0.3, 0.4, 0.0], [0.0, 0.0, 0.0]])      # norms 5, 0.5, 0
    norms, scales = oracle.norm_scales(g, 1.0)
    assert np.allclose(norms, [5.0, 0.5, 0.0], rtol=1e-7)
    assert np.allclose(scales, [0.2, 1.0, 1.0], rtol=1e-7)
    # after scaling the norm is min(norm, max_norm)
    assert abs(np.linalg.norm(g[0].astype(np.float64) * scales[0]) - 1.0) < 1e-7
    # the scaled gradient feeds the coordinate clip and the update: SGDM, beta = 0 -> u = clip(s*g)
    cfg = oracle.make_cfg(3, SGDM, beta1=0.0, clip_rho=0.5, Kx=0, Ku=0, Kv=0)
    x, u = zeros(3, 3), zeros(3, 3)
    oracle.step(cfg, 0, 1.0, x, u, None, g, gscale=scales)
    assert np.allclose(u, [[0.5, 0.5, 0.0], [0.3, 0.4, 0.0], [0.0, 0.0, 0.0]], rtol=1e-6)


def test_rel_change_closed_forms():
    then = f32([[1.0, 2.0, 2.0], [3.0, 0.0, 4.0]])
    now = f32([[2.0, 4.0, 4.0], [3.0, 0.0, 4.0]])
    out = oracle.rel_change(now, then)
    assert np.allclose(out, [1.0, 0.0])
    now2 = f32([[1.0, 2.0, 5.0], [0.0, 0.0, 0.0]])      # diff (0,0,3)/3 ; (3,0,4)/5
    assert np.allclose(oracle.rel_change(now2, then), [1.0, 1.0])


# --------------------------------------------------------------------------- adding workers
def test_worker_mean_closed_forms_and_doubling_keeps_the_mean():
    s = f32([[1.0, -2.0, 0.5], [3.0, 2.0, 0.25], [2.0, 0.0, 0.0]])
    assert np.array_equal(oracle.worker_mean(s), f32([2.0, 0.0, 0.25]))
    # identical replicas: the mean is that replica, bit for bit, for any M
    rng = np.random.default_rng(12)
    row = rng.normal(size=33).astype(np.float32)
    for M in (2, 3, 5, 8):
        assert np.array_equal(oracle.worker_mean(f32(np.tile(row, (M, 1)))), row)
    # new workers that start from the mean leave the worker-mean unchanged (exact on dyadics)
    base = rng.integers(-8, 9, size=(4, 16)).astype(np.float32)
    mean = oracle.worker_mean(f32(base))
    doubled = f32(np.concatenate([base, np.tile(mean, (4, 1))]))
    assert np.array_equal(oracle.worker_mean(doubled), mean)


# --------------------------------------------------------------------------- closed forms, one step
def test_adam_stability_term_sits_inside_the_root():
    """Algorithm 2: d = eta / sqrt(v + lambda^2) * u.  One step from zero states with g = 3,
    beta1 = beta2 = 1/2, lambda = 4: u = 3/2, v = 9/2, x = x0 - eta * 1.5 / sqrt(4.5 + 16)."""
    cfg = oracle.make_cfg(1, ADAM, beta1=0.5, beta2=0.5, eps=4.0, Kx=0, Ku=0, Kv=0)
    x, u, v = f32([[1.0]]), zeros(1, 1), zeros(1, 1)
    oracle.step(cfg, 0, 0.5, x, u, v, f32([[3.0]]))
    assert float(u[0, 0]) == 1.5 and float(v[0, 0]) == 4.5
    want = 1.0 - 0.5 * 1.5 / math.sqrt(4.5 + 16.0)
    assert abs(float(x[0, 0]) - want) < 1e-7
    assert abs(float(x[0, 0]) - (1.0 - 0.5 * 1.5 / (math.sqrt(4.5) + 4.0))) > 1e-2   # not sqrt(v) + lambda


def test_adopt_normalised_gradient_clip_is_two_sided():
    """Optional ADOPT clip: g / max(sqrt(v_prev), eps) is clamped to [-c, c].  With v_prev = 1/4,
    g = (4, -4, 0.5): ratios (8, -8, 1) -> (2, -2, 1) for c = 2; m = (1 - beta1) * that."""
    cfg = oracle.make_cfg(1, ADOPT, beta1=0.5, beta2=0.5, eps=1e-6, Kx=0, Ku=0, Kv=0,
                          flags=oracle.FLAG_ADOPT_NORM_CLIP)
    x, u, v = zeros(1, 3), zeros(1, 3), f32([[0.25, 0.25, 0.25]])
    oracle.step(cfg, 0, 1.0, x, u, v, f32([[4.0, -4.0, 0.5]]), clip_bound=2.0)
    assert np.array_equal(u[0], f32([1.0, -1.0, 0.5]))
    assert np.array_equal(x[0], f32([-1.0, 1.0, -0.5]))
    assert np.array_equal(v[0], f32([0.125 + 8.0, 0.125 + 8.0, 0.125 + 0.125]))
    # c = 0 (the bound at step 0 of the t^(1/4) schedule) zeroes the direction, v still updates
    x, u, v = zeros(1, 3), zeros(1, 3), zeros(1, 3)
    oracle.step(cfg, 0, 1.0, x, u, v, f32([[4.0, -4.0, 0.5]]), clip_bound=0.0)
    assert np.array_equal(u[0], f32([0.0, 0.0, 0.0])) and np.all(v[0] > 0)


# --------------------------------------------------------------------------- update d_t and norms
def test_update_d_matches_hand_examples():
    """d_t from the oracle against the hand examples, two ways: as eta u_t / sqrt(v_t) (eta u_t
    for ADOPT and SGDM) evaluated from the golden states, and as the difference between the base
    the step starts from (the worker's own x_t, or the mean on an x-sync step) and the golden
    x_{t+1}."""
    gold = json.load(open(GOLD))
    cases = [
        ("adam", ADAM, dict(beta1=0.5, beta2=0.5, eps=0.0), "u", 0.0),
        ("adopt", ADOPT, dict(beta1=0.5, beta2=0.5, eps=1e-6), "m", 1.0),
        ("sgdm", SGDM, dict(beta1=0.5), "u", None),
    ]
    for key, opt, hp, uname, v_init in cases:
        ex = gold[key]
        Kv = ex.get("Kv", 0)
        cfg = oracle.make_cfg(2, opt, Kx=ex["Kx"], Ku=ex.get("Ku", ex.get("Km")), Kv=Kv, **hp)
        x, u = f32([[1.0], [1.0]]), zeros(2, 1)
        v = None if v_init is None else f32([[v_init], [v_init]])
        num = lambda s: float(Fraction(s)) if isinstance(s, str) else float(s)
        prev_x = [1.0, 1.0]
        for t, g in enumerate(ex["g"]):
            d = np.zeros((2, 1), dtype=np.float64)
            mask = oracle.step(cfg, t, 0.1, x, u, v, f32([[num(g[0])], [num(g[1])]]), d_out=d)
            base = [sum(prev_x) / 2.0] * 2 if mask & SYNC_X else prev_x
            for m in range(2):
                un = num(ex[uname][t][m])
                want = 0.1 * un / math.sqrt(num(ex["v"][t][m])) if opt == ADAM else 0.1 * un
                assert abs(d[m, 0] - want) < 2e-7, (key, t, m)
                assert abs(d[m, 0] - (base[m] - num(ex["x"][t][m]))) < 5e-7, (key, t, m)
            prev_x = [num(ex["x"][t][m]) for m in range(2)]


def test_update_d_is_the_parameter_change_of_torch_adamw_without_the_decay_term():
    """M = 1 against torch.optim.AdamW in fp64: with decay factor (1 - eta wd) applied to the
    parameter first, what remains of the library's parameter change is d_t."""
    rng = np.random.default_rng(5)
    n, T, lr, b1, b2, wd = 40, 12, 1e-2, 0.9, 0.99, 0.1
    x0 = rng.normal(size=n).astype(np.float32)
    grads = rng.normal(size=(T, n)).astype(np.float32)
    p = torch.nn.Parameter(torch.tensor(x0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=lr, betas=(b1, b2), eps=0.0, weight_decay=wd)
    cfg = oracle.make_cfg(1, ADAM, beta1=b1, beta2=b2, eps=0.0, weight_decay=wd, Kx=2, Ku=3, Kv=4)
    x, u, v = f32(x0[None]), zeros(1, n), zeros(1, n)
    for t in range(T):
        eta_t = lr * math.sqrt(1 - b2 ** (t + 1)) / (1 - b1 ** (t + 1))
        opt.param_groups[0]["weight_decay"] = wd * eta_t / lr
        p.grad = torch.tensor(grads[t], dtype=torch.float64)
        before = p.detach().clone()
        opt.step()
        d_lib = (before * (1.0 - eta_t * wd) - p.detach()).numpy()
        d = np.zeros((1, n), dtype=np.float64)
        oracle.step(cfg, t, eta_t, x, u, v, f32(grads[t][None]), d_out=d)
        # the oracle's u, v are re-read from fp32 storage every step: agreement to ~1e-6 relative
        assert np.max(np.abs(d[0] - d_lib)) < 2e-6 * np.max(np.abs(d_lib))
        assert np.max(np.abs(d_lib)) > 1e-3


def test_update_d_one_step_closed_forms():
    """From zero states one step gives u = (1-b1) g, v = (1-b2) g^2, so
    Adam d = eta (1-b1) g / sqrt((1-b2) g^2 + lambda^2), SGDM d = eta (1-b) g, and ADOPT (seeded
    v = 4, so the normaliser is 2) d = eta (1-b1) g / 2; weight decay does not enter d."""
    g = np.array([[3.0, -0.5, 0.25]], dtype=np.float32)
    g64 = g.astype(np.float64)
    for opt, want in (
        (ADAM, 0.1 * 0.25 * g64 / np.sqrt(0.5 * g64 ** 2 + 0.125 ** 2)),
        (SGDM, 0.1 * 0.25 * g64),
        (ADOPT, 0.1 * 0.25 * g64 / 2.0),
    ):
        cfg = oracle.make_cfg(1, opt, beta1=0.75, beta2=0.5, eps=0.125 if opt == ADAM else 1e-6,
                              weight_decay=0.3)
        x, u = f32([[1.0, 2.0, 3.0]]), zeros(1, 3)
        v = None if opt == SGDM else (f32([[4.0, 4.0, 4.0]]) if opt == ADOPT else zeros(1, 3))
        d = np.full((1, 3), np.nan)
        oracle.step(cfg, 0, 0.1, x, u, v, g.copy(), d_out=d)
        assert np.allclose(d, want, rtol=1e-13, atol=0)
        # and x moved by the decay plus d
        assert np.allclose(x, np.array([[1.0, 2.0, 3.0]]) * (1 - 0.1 * 0.3) - want, rtol=2e-7)


def test_tensor_norms_closed_forms_and_library():
    """3-4-5 and 5-12-13 triples in separate tensors with padding between them (padding holds
    garbage that must not be read), whole-model norm = sqrt of the sum of squares, and a random
    case against numpy.linalg.norm."""
    a = np.full((2, 12), 1e6, dtype=np.float32)
    offs, numel = [1, 4, 8], [2, 3, 1]
    a[0, 1:3] = [3, 4];  a[0, 4:7] = [0, -5, 12];  a[0, 8] = -2
    a[1, 1:3] = [0, 0];  a[1, 4:7] = [1, 2, 2];    a[1, 8] = 7
    per, tot = oracle.tensor_norms(a, offs, numel)
    assert np.array_equal(per, [[5.0, 13.0, 2.0], [0.0, 3.0, 7.0]])
    assert np.allclose(tot, [math.sqrt(25 + 169 + 4), math.sqrt(9 + 49)], rtol=1e-15)
    rng = np.random.default_rng(9)
    b = rng.normal(size=(3, 1000))
    offs, numel = [0, 10, 500, 999], [10, 400, 499, 1]
    per, tot = oracle.tensor_norms(b, offs, numel)
    for m in range(3):
        for k, (o, c) in enumerate(zip(offs, numel)):
            assert abs(per[m, k] - np.linalg.norm(b[m, o:o + c])) < 1e-12 * (1 + per[m, k])
        want = np.linalg.norm(np.concatenate([b[m, o:o + c] for o, c in zip(offs, numel)]))
        assert abs(tot[m] - want) < 1e-12 * want
    with pytest.raises(ValueError):
        oracle.tensor_norms(b, [990], [11])
