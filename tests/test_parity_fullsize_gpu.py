"""Parity at the full sizes of the paper-shaped workloads, in the launch configuration the
benchmark times.  Every coordinate's trajectory depends only on that coordinate of the M
replicas, so running the oracle on a sampled index set (first/last 64 elements of every
tensor plus hashed positions) is exact for those coordinates, not statistical.  Gradients are
fresh at every step; the oracle receives the sampled gradient bits gathered from the device
buffers the kernel read."""
import numpy as np
import pytest
import torch

import desloc_inputs as di
import oracle
from _util import TOL, State, f32r, oracle_cfg, rel_err
from test_parity_gpu import make_engine

pytestmark = pytest.mark.gpu

CASES = [
    # (workload, steps, first step, hashed samples)
    ("cfg2_adam_135m", 40, 0, 1 << 17),
    ("cfg3_adopt_360m", 20, 0, 1 << 16),
    ("cfg4_adam_1p7b", 24, 56, 1 << 17),     # t = 56..79 crosses the x-sync at t = 64
    # workload 5: both optimizers under its three schedules (every step / every 16 / 16-64-256)
    ("cfg5_sgdm_ddp", 4, 0, 1 << 16),
    ("cfg5_sgdm_local", 18, 0, 1 << 16),
    ("cfg5_sgdm_desloc", 18, 0, 1 << 16),
    ("cfg5_adam_ddp", 6, 0, 1 << 16),
    ("cfg5_adam_local", 18, 0, 1 << 16),
    ("cfg5_adam_desloc", 18, 0, 1 << 16),
]

# The other orderings and kernels at full size: (workload, workers or None, post-average, steps)
VARIANTS = [
    ("cfg3_adopt_360m", None, True, 12),     # Algorithm 4-5 ordering, eight workers
    ("cfg2_adam_135m", None, True, 12),
    ("cfg2_adam_135m", 16, False, 12),       # more than eight workers: runtime-M kernel on sync steps
    ("cfg2_adam_135m", 16, True, 6),
    ("cfg5_sgdm_desloc", 3, False, 18),      # a worker count that is not a power of two
]


@pytest.mark.parametrize("name,T,t0,nsamp", CASES)
def test_fullsize_sampled_parity(name, T, t0, nsamp):
    _sampled_parity(di.WORKLOADS[name], name, T, t0, nsamp, post=False)


@pytest.mark.parametrize("name,M,post,T", VARIANTS)
def test_fullsize_sampled_parity_of_other_orderings_and_worker_counts(name, M, post, T):
    w = di.WORKLOADS[name]
    if M is not None:
        w = w.replace(M=M, K=(4, 8, 12))     # sync steps of every kind within a short run
    _sampled_parity(w, f"{name} M={w.M} post={post}", T, 0, 1 << 15, post=post)


def _sampled_parity(w, name, T, t0, nsamp, post):
    import paper_2505_22549_b200 as d
    dev = torch.device("cuda:0")
    free, _ = torch.cuda.mem_get_info()
    need = w.N * w.M * (14 if w.opt != "sgdm" else 10) + (6 << 30)
    if free < need:
        pytest.skip(f"needs {need >> 30} GiB of device memory, {free >> 30} GiB free")
    st = State(w, dev, align=4)
    # non-trivial moments at the first step: a run that starts mid-way, as a resumed job would
    if t0 > 0:
        for m in range(w.M):
            di.fill_grads_(w, 10_000 + m, m, st.g[m], align=4)
            st.u[m].copy_(st.g[m])
            st.v[m].copy_(st.g[m]).square_()
    eng = make_engine(d, w, st, post)
    idx_np = di.sample_indices(w.numel, nsamp, seed=1, align=4)
    idx = torch.from_numpy(idx_np).to(dev)
    ox, ou = st.to_numpy(st.x, idx), st.to_numpy(st.u, idx)
    ov = st.to_numpy(st.v, idx) if st.v is not None else None
    ocfg = oracle_cfg(w, oracle.FLAG_POST_AVERAGE if post else 0)
    gviews = st.views(st.g)
    for t in range(t0, t0 + T):
        st.fill_grads(t)
        lr, cb = f32r(w.lr), f32r(w.clip_bound(t))
        mk = eng.step(t, lr, gviews, clip_bound=cb)
        mo = oracle.step(ocfg, t, lr, ox, ou, ov, st.to_numpy(st.g, idx), clip_bound=cb)
        assert mk == mo
    torch.cuda.synchronize()
    pairs = [("x", st.x, ox), ("u", st.u, ou)] + ([("v", st.v, ov)] if ov is not None else [])
    for nm, bufs, ref in pairs:
        got = st.to_numpy(bufs, idx)
        for m in range(w.M):
            e = rel_err(got[m], ref[m])
            assert e <= TOL, f"{name} {nm} worker {m}: rel err {e:.3e}"
        frac_exact = float(np.mean(got == ref))
        print(f"{name} {nm}: max rel err {max(rel_err(got[m], ref[m]) for m in range(w.M)):.2e}, "
              f"bit-exact {100 * frac_exact:.2f}%")
    eng.close()
    del st, eng
    torch.cuda.empty_cache()


@pytest.mark.parametrize("name", ["cfg5_adam_ddp", "cfg5_sgdm_local"])
def test_fullsize_identical_gradients_keep_replicas_bitwise_equal(name):
    """Workload 5's identical-gradient run at full size (361.8 M parameters x 8 workers): with the
    same gradient on every worker the replicas must stay bitwise equal to one another under any
    schedule -- a property that holds at any size and needs no oracle -- and, on sampled
    coordinates, equal to the oracle's single-worker run."""
    import paper_2505_22549_b200 as d
    w = di.WORKLOADS[name]
    dev = torch.device("cuda:0")
    free, _ = torch.cuda.mem_get_info()
    if free < w.N * w.M * 14 + (6 << 30):
        pytest.skip("not enough device memory")
    st = State(w, dev, align=4)
    eng = make_engine(d, w, st)
    idx_np = di.sample_indices(w.numel, 1 << 14, seed=3, align=4)
    idx = torch.from_numpy(idx_np).to(dev)
    one = w.replace(M=1)
    ox, ou = st.to_numpy(st.x[:1], idx), st.to_numpy(st.u[:1], idx)
    ov = st.to_numpy(st.v[:1], idx) if st.v is not None else None
    gviews = st.views(st.g)
    for t in range(17):                          # crosses t = 16 for the K = 16 schedule
        di.fill_grads_(w, t, 0, st.g[0], align=4)
        for m in range(1, w.M):
            st.g[m].copy_(st.g[0])
        eng.step(t, f32r(w.lr), gviews)
        oracle.step(oracle_cfg(one), t, f32r(w.lr), ox, ou, ov, st.to_numpy(st.g[:1], idx))
    torch.cuda.synchronize()
    for bufs, ref in [(st.x, ox), (st.u, ou)] + ([(st.v, ov)] if ov is not None else []):
        for m in range(1, w.M):
            assert torch.equal(bufs[m], bufs[0]), f"replica {m} differs from replica 0"
        assert rel_err(st.to_numpy(bufs[:1], idx)[0], ref[0]) <= TOL
    eng.close()
    del st, eng
    torch.cuda.empty_cache()
