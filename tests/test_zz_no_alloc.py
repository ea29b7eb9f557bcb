"""desloc_step_static(): the entry point for callers that cannot allocate device memory (their
framework already owns all of HBM, or they cannot take cudaMalloc's device-wide
synchronisation).  It keeps its chunk and pointer tables in a fixed array inside the library
instead of cudaMalloc'ed memory.  Here it is driven through the C ABI next to the regular
desloc_create / desloc_step path on identical inputs: both run the same kernel, so the results
must agree bit for bit (the suite's tolerance of 1e-5 is asserted as well), on two calls in a
row -- the second call finds the previous call's tables in the array.

This file is named to be collected last."""
import numpy as np
import pytest
import torch

import desloc_inputs as di
from _util import TOL, State, f32r, rel_err

pytestmark = pytest.mark.gpu


def _flat_ptrs(st, bufs):
    return [t.data_ptr() for lst in st.views(bufs) for t in lst]


@pytest.mark.parametrize("name,K", [("cfg2_adam_135m", (1, 2, 1)), ("cfg3_adopt_360m", (2, 1, 2)),
                                    ("cfg5_sgdm_desloc", (2, 2, 0))])
def test_static_entry_point_matches_context_path_twice(name, K):
    import paper_2505_22549_b200 as d
    from test_parity_gpu import make_engine
    w = di.mini(di.WORKLOADS[name]).replace(K=K)
    dev = torch.device("cuda:0")
    a = State(w, dev)            # stepped through desloc_create / desloc_step
    b = State(w, dev)            # stepped through desloc_step_static
    eng = make_engine(d, w, a)
    flags = d.DESLOC_FLAG_ADOPT_NORM_CLIP if w.adopt_norm_clip else 0
    cfg = d.make_config(w.M, w.numel, w.opt, w.grad_dtype, w.beta1, w.beta2, w.eps,
                        w.weight_decay, w.clip_rho, K[0], K[1], K[2], flags)
    stream = torch.cuda.current_stream(dev).cuda_stream
    for t in range(2):           # two calls in a row; t = 1 reuses the array left by t = 0
        a.fill_grads(t)
        for m in range(w.M):
            b.g[m].copy_(a.g[m])
        lr, cb = f32r(w.lr), f32r(w.clip_bound(t) if t else 1.0)
        mk_a = eng.step(t, lr, a.views(a.g), clip_bound=cb)
        mk_b = d.desloc_step_static(cfg, _flat_ptrs(b, b.x), _flat_ptrs(b, b.u),
                                    _flat_ptrs(b, b.v) if b.v is not None else None,
                                    _flat_ptrs(b, b.g), t, lr, cb, 0, stream)
        assert mk_a == mk_b == d.desloc_sync_mask(cfg, t)
        torch.cuda.synchronize()
        pairs = [(a.x, b.x), (a.u, b.u)] + ([(a.v, b.v)] if a.v is not None else [])
        for pa, pb in pairs:
            ga, gb = a.to_numpy(pa), b.to_numpy(pb)
            assert rel_err(gb, ga) <= TOL
            assert np.array_equal(ga, gb)
    # the step did something
    assert not np.array_equal(a.to_numpy(a.x)[0], di.init_params(w, align=4).numpy())
    eng.close()


def test_static_entry_point_rejects_what_does_not_fit():
    import paper_2505_22549_b200 as d
    dev = torch.device("cuda:0")
    buf = torch.zeros(16, device=dev)
    p = buf.data_ptr()
    # too many chunks: one tensor of more than MAX_CHUNKS * chunk_elems parameters
    big = d.DESLOC_STATIC_MAX_CHUNKS * d.desloc_chunk_elems() + 1
    cfg = d.make_config(1, [big], "adam", "f32")
    with pytest.raises(d.DeslocError) as e:
        d.desloc_step_static(cfg, [p], [p], [p], [p], 0, 1e-3, 0.0, 0)
    assert e.value.status == d.DESLOC_E_TOO_LARGE
    # too many pointers
    nt = d.DESLOC_STATIC_MAX_POINTERS // 2 + 1
    cfg = d.make_config(2, [1] * nt, "adam", "f32")
    with pytest.raises(d.DeslocError) as e:
        d.desloc_step_static(cfg, [p] * (2 * nt), [p] * (2 * nt), [p] * (2 * nt), [p] * (2 * nt),
                             0, 1e-3, 0.0, 0)
    assert e.value.status == d.DESLOC_E_TOO_LARGE
    # nothing was written
    torch.cuda.synchronize()
    assert float(buf.abs().sum()) == 0.0
