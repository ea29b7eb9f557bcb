"""The paper's toy-problem shape on the library: M = 256 workers, two parameters, periods
(192, 192, 692) -- the largest worker count a context accepts and the runtime-M kernel.  The
oracle is fed the very gradients the GPU run used, step by step."""
import numpy as np
import pytest
import torch

import oracle
from _util import TOL, f32r, rel_err

pytestmark = pytest.mark.gpu


def test_toy_shape_matches_oracle_over_a_full_v_period():
    from paper_2505_22549_b200 import toy
    M, T, K, lr = 256, 700, (192, 192, 692), f32r(2e-2)
    log = []

    def record(t, X, U, V, G):
        if t == 0:
            log.append((X.cpu().numpy().copy(), U.cpu().numpy().copy(), V.cpu().numpy().copy()))
        log.append(G.cpu().numpy().copy())

    dist = toy.run(K, T, lr, M=M, record=record)
    x0, u0, v0 = log[0]
    grads = log[1:]
    assert len(grads) == T
    cfg = oracle.make_cfg(M, oracle.ADAM, beta1=f32r(0.95), beta2=f32r(0.999), eps=f32r(1e-8),
                          Kx=K[0], Ku=K[1], Kv=K[2])
    ox, ou, ov = (np.ascontiguousarray(a, dtype=np.float32) for a in (x0, u0, v0))
    masks = []
    for t in range(T):
        masks.append(oracle.step(cfg, t, lr, ox, ou, ov, np.ascontiguousarray(grads[t], dtype=np.float32)))
    assert masks[0] == 7 and masks[192] == 3 and masks[692] == 4 and sum(m != 0 for m in masks) == 5
    # the oracle's worker-mean iterate gives the same distance the GPU run reported
    odist = float(np.linalg.norm(ox.astype(np.float64).mean(axis=0) - 1.0))
    assert abs(dist - odist) <= 1e-4 * max(1.0, odist)
    assert np.isfinite(dist)


def test_toy_state_parity_elementwise():
    """Same run, but keeping the GPU's end state for an element-by-element comparison."""
    import paper_2505_22549_b200 as d
    from paper_2505_22549_b200.toy import rosenbrock_grad
    M, T, K, lr = 256, 400, (192, 192, 692), f32r(2e-2)
    dev = torch.device("cuda:0")
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)
    X = torch.tensor([-1.0, 1.0], device=dev).repeat(M, 1).contiguous()
    U, V, G = torch.zeros_like(X), torch.zeros_like(X), torch.zeros_like(X)
    rows = lambda a: [[a[m]] for m in range(M)]
    eng = d.DesLoc(rows(X), rows(U), rows(V), opt="adam", grad_dtype="f32", beta1=0.95,
                   beta2=0.999, eps=1e-8, K=K)
    cfg = oracle.make_cfg(M, oracle.ADAM, beta1=f32r(0.95), beta2=f32r(0.999), eps=f32r(1e-8),
                          Kx=K[0], Ku=K[1], Kv=K[2])
    ox, ou, ov = X.cpu().numpy().copy(), U.cpu().numpy().copy(), V.cpu().numpy().copy()
    for t in range(T):
        G.copy_(rosenbrock_grad(X) + 1.5 * torch.randn(M, 2, generator=gen, device=dev))
        mk = eng.step(t, lr, rows(G))
        assert mk == oracle.step(cfg, t, lr, ox, ou, ov, G.cpu().numpy().copy())
    torch.cuda.synchronize()
    # two coordinates with very different scales: compare each column against its own RMS
    for got, ref in ((X, ox), (U, ou), (V, ov)):
        g = got.cpu().numpy()
        for c in range(2):
            assert rel_err(g[:, c], ref[:, c]) <= TOL
    eng.close()
