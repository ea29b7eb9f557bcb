"""The paper's toy-problem shape on the library: M = 256 workers, two parameters, periods
(192, 192, 692) -- the largest worker count a context accepts and the runtime-M kernel.

The toy problem is a closed loop (each worker's gradient is evaluated at its own iterate).  To
keep the oracle free of anything the device produced, the loop is closed on the HOST: the
oracle steps its own iterates, the noisy Rosenbrock gradients are evaluated there, and the
recorded gradient sequence is then replayed through the library.  Both sides see the same
gradient bits; the device's iterates never feed back into what the oracle reads."""
import numpy as np
import pytest
import torch

import desloc_inputs as di
import oracle
from _util import TOL, f32r, rel_err

pytestmark = pytest.mark.gpu


def _host_closed_loop(M, T, K, lr, seed):
    cfg = oracle.make_cfg(M, oracle.ADAM, beta1=f32r(0.95), beta2=f32r(0.999), eps=f32r(1e-8),
                          Kx=K[0], Ku=K[1], Kv=K[2])
    ox = np.ascontiguousarray(np.tile(np.array([-1.0, 1.0], dtype=np.float32), (M, 1)))
    ou, ov = np.zeros_like(ox), np.zeros_like(ox)
    grads, masks = [], []
    for t in range(T):
        g = di.toy_rosenbrock_grads(ox, t, sigma=1.5, seed=seed)
        grads.append(g)
        masks.append(oracle.step(cfg, t, lr, ox, ou, ov, g))
    return grads, masks, (ox, ou, ov)


def test_toy_shape_matches_oracle_over_a_full_v_period():
    import paper_2505_22549_b200 as d
    M, T, K, lr = 256, 700, (192, 192, 692), f32r(2e-2)
    grads, masks, (ox, ou, ov) = _host_closed_loop(M, T, K, lr, seed=1)
    assert masks[0] == 7 and masks[192] == 3 and masks[692] == 4 and sum(m != 0 for m in masks) == 5
    dev = torch.device("cuda:0")
    X = torch.tensor([-1.0, 1.0], device=dev).repeat(M, 1).contiguous()
    U, V, G = torch.zeros_like(X), torch.zeros_like(X), torch.zeros_like(X)
    rows = lambda a: [[a[m]] for m in range(M)]
    eng = d.DesLoc(rows(X), rows(U), rows(V), opt="adam", grad_dtype="f32", beta1=0.95,
                   beta2=0.999, eps=1e-8, K=K)
    grows = rows(G)
    for t in range(T):
        G.copy_(torch.from_numpy(grads[t]))
        assert eng.step(t, lr, grows) == masks[t]
    torch.cuda.synchronize()
    # two coordinates with very different scales: compare each column against its own RMS
    for got, ref in ((X, ox), (U, ou), (V, ov)):
        g = got.cpu().numpy()
        for c in range(2):
            assert rel_err(g[:, c], ref[:, c]) <= TOL
    eng.close()


def test_toy_module_runs_its_three_schedules():
    """The demonstration module itself (closed loop on the device): finite distances, and the
    same seed gives the same number twice."""
    from paper_2505_22549_b200 import toy
    for K in ((192, 192, 692), (192, 192, 192), (192, 0, 0)):
        a = toy.run(K, 250, 2e-2, M=256, seed=3)
        b = toy.run(K, 250, 2e-2, M=256, seed=3)
        assert np.isfinite(a) and a == b
