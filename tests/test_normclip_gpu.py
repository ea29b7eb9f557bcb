"""Norm-based gradient clipping in front of the step, and the relative rate-of-change
diagnostic, against the oracle."""
import numpy as np
import pytest
import torch

import desloc_inputs as di
import oracle
from _util import TOL, State, compare_per_tensor, f32r, oracle_cfg, rel_err
from test_parity_gpu import make_engine

pytestmark = pytest.mark.gpu


def _valid(st):
    return st.valid_mask()


@pytest.mark.parametrize("name,M", [("cfg2_adam_135m", 4), ("cfg3_adopt_360m", 8),
                                    ("cfg5_sgdm_desloc", 3), ("cfg2_adam_135m", 12),
                                    ("cfg2_adam_135m", 1)])
@pytest.mark.parametrize("align", [4, 1])
def test_normclip_step_matches_oracle(name, M, align):
    import paper_2505_22549_b200 as d
    w = di.mini(di.WORKLOADS[name], T=12).replace(M=M, K=(2, 3, 4))
    dev = torch.device("cuda:0")
    st = State(w, dev, align=align)
    eng = make_engine(d, w, st)
    ox, ou = st.to_numpy(st.x), st.to_numpy(st.u)
    ov = st.to_numpy(st.v) if st.v is not None else None
    ocfg = oracle_cfg(w)
    valid = _valid(st)
    # the mini model's gradient norm is ~1e-3 * sqrt(N) ~ 0.4: bounds on both sides of it
    bounds = [0.05, 10.0, 0.3, 0.01]
    for t in range(w.T):
        st.fill_grads(t)
        if t == 5:          # one worker far larger than the others
            st.g[0].mul_(50.0)
        mx = f32r(bounds[t % len(bounds)])
        lr, cb = f32r(w.lr), f32r(w.clip_bound(t))
        g_host = st.to_numpy(st.g)
        g_valid = np.ascontiguousarray(g_host[:, valid])
        norms, scales = oracle.norm_scales(g_valid, mx)
        mk = eng.step_normclip(t, lr, st.views(st.g), mx, clip_bound=cb)
        got_n, got_s = eng.grad_norms()
        assert np.allclose(got_n, norms, rtol=2e-6)
        assert np.allclose(got_s, scales, rtol=2e-6)
        if mx >= 10.0:
            assert all(s == 1.0 for s in got_s[1:])       # worker 0 is blown up at t = 5
            assert (got_s[0] == 1.0) == (t != 5)
        # the oracle steps with its OWN fp64 factors: nothing read back from the device enters it
        mo = oracle.step(ocfg, t, lr, ox, ou, ov, g_host, clip_bound=cb, gscale=scales)
        assert mk == mo
    torch.cuda.synchronize()
    compare_per_tensor(st, st.to_numpy(st.x), ox, "x")
    compare_per_tensor(st, st.to_numpy(st.u), ou, "u")
    if ov is not None:
        compare_per_tensor(st, st.to_numpy(st.v), ov, "v")
    assert eng.launches() == 3 * w.T     # two reductions + the step
    eng.close()


@pytest.mark.parametrize("M", [2, 8])
def test_normclip_with_fp32_gradients(M):
    """fp32 gradients take their own wide path in the sum-of-squares kernel: full chunks, ragged
    tails and misaligned tensors."""
    import paper_2505_22549_b200 as d
    numel = (4096 * 3, 4096 * 9 + 5, 17, 4096 * 8, 1000)
    w = di.Workload("nc_f32", "adam", M, numel, "f32", "normal1", lr=1e-2, K=(2, 3, 4), seed=21)
    dev = torch.device("cuda:0")
    for align in (4, 1):
        st = State(w, dev, align=align)
        eng = make_engine(d, w, st)
        ox, ou, ov = st.to_numpy(st.x), st.to_numpy(st.u), st.to_numpy(st.v)
        valid = _valid(st)
        for t in range(6):
            st.fill_grads(t)
            mx = f32r([50.0, 1e9, 5.0][t % 3])          # norm is about sqrt(N) = 290
            g_host = st.to_numpy(st.g)
            norms, scales = oracle.norm_scales(np.ascontiguousarray(g_host[:, valid]), mx)
            eng.step_normclip(t, f32r(w.lr), st.views(st.g), mx)
            got_n, got_s = eng.grad_norms()
            assert np.allclose(got_n, norms, rtol=2e-6) and np.allclose(got_s, scales, rtol=2e-6)
            oracle.step(oracle_cfg(w), t, f32r(w.lr), ox, ou, ov, g_host, gscale=scales)
        torch.cuda.synchronize()
        compare_per_tensor(st, st.to_numpy(st.x), ox, "x")
        compare_per_tensor(st, st.to_numpy(st.v), ov, "v")
        eng.close()


def test_normclip_workload4_recipe_with_decay():
    """Workload 4's recipe (weight decay 0.1) with a bound that clips every step."""
    import paper_2505_22549_b200 as d
    w = di.mini(di.WORKLOADS["cfg4_adam_1p7b"], T=10).replace(K=(2, 3, 4))
    dev = torch.device("cuda:0")
    st = State(w, dev)
    eng = make_engine(d, w, st)
    ox, ou, ov = st.to_numpy(st.x), st.to_numpy(st.u), st.to_numpy(st.v)
    ocfg = oracle_cfg(w)
    valid = _valid(st)
    for t in range(w.T):
        st.fill_grads(t)
        g_host = st.to_numpy(st.g)
        _, scales = oracle.norm_scales(np.ascontiguousarray(g_host[:, valid]), 0.1)
        eng.step_normclip(t, f32r(w.lr), st.views(st.g), 0.1)
        oracle.step(ocfg, t, f32r(w.lr), ox, ou, ov, g_host, gscale=scales)
    torch.cuda.synchronize()
    compare_per_tensor(st, st.to_numpy(st.x), ox, "x")
    compare_per_tensor(st, st.to_numpy(st.u), ou, "u")
    compare_per_tensor(st, st.to_numpy(st.v), ov, "v")
    eng.close()


def test_normclip_is_deterministic_and_rejects_bad_bounds():
    import paper_2505_22549_b200 as d
    w = di.mini(di.WORKLOADS["cfg2_adam_135m"], T=4)
    dev = torch.device("cuda:0")
    outs = []
    for _ in range(2):
        st = State(w, dev)
        eng = make_engine(d, w, st)
        for t in range(w.T):
            st.fill_grads(t)
            eng.step_normclip(t, f32r(w.lr), st.views(st.g), 0.2)
        torch.cuda.synchronize()
        outs.append((st.to_numpy(st.x), eng.grad_norms()))
        for bad in (0.0, -1.0, float("inf"), float("nan")):
            with pytest.raises(d.DeslocError) as e:
                eng.step_normclip(0, 1e-3, st.views(st.g), bad)
            assert e.value.status == d.DESLOC_E_RANGE
        eng.close()
    assert np.array_equal(outs[0][0], outs[1][0]) and outs[0][1] == outs[1][1]


@pytest.mark.parametrize("opt", ["adam", "sgdm"])
def test_rel_change_matches_oracle(opt):
    """||s_{t+K} - s_t|| / ||s_t|| over K = 5 steps for x, u (and v).  The oracle measures its own
    trajectory (same seeded inputs), never the device's buffers.  Both trajectories agree to
    1e-5 of each tensor's scale, which bounds the difference of the two ratios r by
    1e-5 (||now|| + ||then||) / ||then|| + 1e-5 r <= 2e-5 (1 + r); the assertion allows 3e-5 (1 + r)."""
    import paper_2505_22549_b200 as d
    w = di.mini(di.WORKLOADS[f"cfg5_{opt}_desloc"], T=8).replace(M=3, K=(2, 3, 4))
    dev = torch.device("cuda:0")
    for align in (4, 1):
        st = State(w, dev, align=align)
        eng = make_engine(d, w, st)
        valid = _valid(st)
        ox, ou = st.to_numpy(st.x), st.to_numpy(st.u)          # initial state, before any step
        ov = st.to_numpy(st.v) if st.v is not None else None
        ocfg = oracle_cfg(w)
        snaps = osnaps = None
        for t in range(w.T):
            if t == 3:
                snaps = [[b.clone() for b in bufs] if bufs is not None else None
                         for bufs in (st.x, st.u, st.v)]
                osnaps = [a.copy() if a is not None else None for a in (ox, ou, ov)]
            st.fill_grads(t)
            eng.step(t, f32r(w.lr), st.views(st.g))
            oracle.step(ocfg, t, f32r(w.lr), ox, ou, ov, st.to_numpy(st.g))
        torch.cuda.synchronize()
        arrays = [(0, ox), (1, ou)] + ([(2, ov)] if ov is not None else [])
        for idx, onow in arrays:
            got = np.asarray(eng.rel_change(idx, st.views(snaps[idx])), dtype=np.float64)
            want = oracle.rel_change(np.ascontiguousarray(onow[:, valid]),
                                     np.ascontiguousarray(osnaps[idx][:, valid]))
            assert np.all(np.abs(got - want) <= 3e-5 * (1.0 + want)), (idx, got, want)
            assert min(want) > 0
        if st.v is None:
            with pytest.raises(d.DeslocError):
                eng.rel_change(2, st.views(snaps[0]))
        eng.close()
