"""desloc_step_diag(): the step that also measures, per worker and per tensor, the L2 norms of
the gradient as read, of the new parameters and of the update d_t (the gradient, parameter and
update norms the paper plots for its runs).  Checked against the oracle, which reports d_t per
coordinate and computes the norms in fp64 from its own trajectory; and against the plain step,
whose state the diagnostics step must reproduce bit for bit."""
import numpy as np
import pytest
import torch

import desloc_inputs as di
import oracle
from _util import State, compare_per_tensor, f32r, oracle_cfg
from test_parity_gpu import make_engine

pytestmark = pytest.mark.gpu

# fp32 partial sums of at most 4096 squares per chunk (16 per thread, then a tree), fp64 above:
# relative error of a norm well below 1e-6; the states behind them agree to 1e-5 at worst.
RTOL = 2e-6


def _check_norms(st, got_per, got_tot, arrays, what):
    """arrays: three [M, nflat] float64 arrays (g, x_new, d) from the oracle side."""
    for kind, a in enumerate(arrays):
        per, tot = oracle.tensor_norms(a, st.offs, st.w.numel)
        gp = np.asarray(got_per[kind], dtype=np.float64)
        gt = np.asarray(got_tot[kind], dtype=np.float64)
        # tiny tensors (a few elements) can have norms near zero: floor at the worker's total
        floor = 1e-3 * tot[:, None]
        assert np.all(np.abs(gp - per) <= RTOL * np.maximum(per, floor)), (what, kind)
        assert np.all(np.abs(gt - tot) <= RTOL * tot), (what, kind, gt, tot)
        # (the update can be exactly zero: ADOPT's step 0 under the bound c_0 = 0)
        assert np.all(tot > 0) or kind == 2


@pytest.mark.parametrize("name,M", [("cfg2_adam_135m", 4), ("cfg3_adopt_360m", 8),
                                    ("cfg5_sgdm_desloc", 8), ("cfg4_adam_1p7b", 1),
                                    ("cfg5_adam_desloc", 5), ("cfg2_adam_135m", 12),
                                    ("cfg3_adopt_360m", 11), ("cfg5_sgdm_desloc", 2)])
@pytest.mark.parametrize("post", [False, True])
@pytest.mark.parametrize("align,g_shift", [(4, None), (1, None), (8, 4)])
def test_diag_step_norms_match_oracle_and_state_matches_plain_step(name, M, post, align, g_shift):
    import paper_2505_22549_b200 as d
    w = di.mini(di.WORKLOADS[name], T=9).replace(M=M, K=(2, 3, 4))
    dev = torch.device("cuda:0")
    # (g_shift: gradients 8 bytes off the state's layout -- the 128-bit path from global memory)
    a, b = State(w, dev, align=align, g_shift=g_shift), State(w, dev, align=align, g_shift=g_shift)    # diag / plain
    ea, eb = make_engine(d, w, a, post), make_engine(d, w, b, post)
    ox, ou = a.to_numpy(a.x), a.to_numpy(a.u)
    ov = a.to_numpy(a.v) if a.v is not None else None
    ocfg = oracle_cfg(w, oracle.FLAG_POST_AVERAGE if post else 0)
    with pytest.raises(d.DeslocError) as e:          # nothing measured yet
        ea.diag_norms()
    assert e.value.status == d.DESLOC_E_INVALID
    for t in range(w.T):
        a.fill_grads(t)
        for m in range(M):
            b.g[m].copy_(a.g[m])
        lr, cb = f32r(w.lr), f32r(w.clip_bound(t))
        g_host = a.to_numpy(a.g)
        dref = np.zeros(ox.shape, dtype=np.float64)
        mo = oracle.step(ocfg, t, lr, ox, ou, ov, g_host, clip_bound=cb, d_out=dref)
        assert ea.step_diag(t, lr, a.views(a.g), clip_bound=cb) == mo
        eb.step(t, lr, b.views(b.g), clip_bound=cb)
        got_per, got_tot = ea.diag_norms()
        _check_norms(a, got_per, got_tot, (g_host.astype(np.float64), ox.astype(np.float64), dref),
                     f"{name} M={M} post={post} t={t}")
    torch.cuda.synchronize()
    pairs = [(a.x, b.x), (a.u, b.u)] + ([(a.v, b.v)] if a.v is not None else [])
    for pa, pb in pairs:
        assert np.array_equal(a.to_numpy(pa), b.to_numpy(pb))      # same kernel arithmetic
    compare_per_tensor(a, a.to_numpy(a.x), ox, "x")
    ea.close(); eb.close()


@pytest.mark.parametrize("M", [3, 16])
def test_diag_with_norm_clipping_reports_the_unclipped_gradient(M):
    """Norm-based clipping in front of a diagnostics step: kind 0 stays the norm of the gradient
    as read (equal to what the clipping pass itself measured), the update shrinks."""
    import paper_2505_22549_b200 as d
    w = di.mini(di.WORKLOADS["cfg2_adam_135m"], T=4).replace(M=M, K=(2, 3, 4))
    dev = torch.device("cuda:0")
    st = State(w, dev)
    eng = make_engine(d, w, st)
    ox, ou, ov = st.to_numpy(st.x), st.to_numpy(st.u), st.to_numpy(st.v)
    valid = st.valid_mask()
    for t in range(w.T):
        st.fill_grads(t)
        g_host = st.to_numpy(st.g)
        _, scales = oracle.norm_scales(np.ascontiguousarray(g_host[:, valid]), 0.05)
        assert np.all(scales < 1.0)
        dref = np.zeros(ox.shape, dtype=np.float64)
        oracle.step(oracle_cfg(w), t, f32r(w.lr), ox, ou, ov, g_host, gscale=scales, d_out=dref)
        eng.step_diag(t, f32r(w.lr), st.views(st.g), max_norm=0.05)
        per, tot = eng.diag_norms()
        _check_norms(st, per, tot, (g_host.astype(np.float64), ox.astype(np.float64), dref), f"t={t}")
        clip_norms, _ = eng.grad_norms()
        assert np.allclose(tot[0], clip_norms, rtol=2e-6)
    eng.close()


def test_diag_is_deterministic_and_rejects_bad_arguments():
    import paper_2505_22549_b200 as d
    w = di.mini(di.WORKLOADS["cfg3_adopt_360m"], T=3).replace(K=(1, 2, 3))
    dev = torch.device("cuda:0")
    outs = []
    st = State(w, dev)
    for _ in range(2):
        st.reset()                      # the same buffers: the chunk plan follows their alignment
        eng = make_engine(d, w, st)
        for t in range(w.T):
            st.fill_grads(t)
            eng.step_diag(t, f32r(w.lr), st.views(st.g), clip_bound=f32r(w.clip_bound(t)))
        outs.append(eng.diag_norms())
        for bad in (-1.0, float("inf"), float("nan")):
            with pytest.raises(d.DeslocError) as e:
                eng.step_diag(0, 1e-3, st.views(st.g), max_norm=bad)
            assert e.value.status == d.DESLOC_E_RANGE
        eng.close()
    assert outs[0] == outs[1]


def test_diag_fullsize_totals_on_workload_2():
    """Workload 2 at full size (134.5 M parameters x 4 workers, 272 tensors) in the benchmark's
    launch configuration: norms that have a closed form or an independent route.  The gradient
    norm per worker and tensor against torch's own reduction of the same buffers, the parameter
    norm against torch's reduction of the updated parameters."""
    import paper_2505_22549_b200 as d
    w = di.WORKLOADS["cfg2_adam_135m"]
    dev = torch.device("cuda:0")
    st = State(w, dev, align=4)
    eng = make_engine(d, w, st)
    gv = st.views(st.g)
    for t in range(2):
        st.fill_grads(t)
        eng.step_diag(t, f32r(w.lr), gv)
    per, tot = eng.diag_norms()
    per = np.asarray(per)
    xv = st.views(st.x)
    for m in range(w.M):
        for k in (0, 1, 7, 100, len(w.numel) - 1):
            gref = float(torch.linalg.vector_norm(gv[m][k].double()))
            xref = float(torch.linalg.vector_norm(xv[m][k].double()))
            assert abs(per[0, m, k] - gref) <= RTOL * gref
            assert abs(per[1, m, k] - xref) <= RTOL * xref
        gtot = float(torch.sqrt(sum(torch.sum(g.double() ** 2) for g in gv[m])))
        assert abs(tot[0][m] - gtot) <= RTOL * gtot
    # the update of an Adam step from zero states is bounded by eta sqrt(1-b1)^2/(1-b2) per
    # coordinate; here just: positive, finite, far below the parameter norm
    assert np.all(per[2] > 0) and np.all(np.isfinite(per[2])) and np.all(per[2] < per[1])
    eng.close()
