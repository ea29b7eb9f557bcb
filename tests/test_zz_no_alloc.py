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
    big = d.DESLOC_STATIC_MAX_CHUNKS * 8192 + 1        # 8192 = a chunk of a large one-worker list
    cfg = d.make_config(1, [big], "adam", "f32")
    assert d.desloc_chunk_elems(cfg) == 8192
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


def _ctx_vs_static(d, w, K, steps, post=False, byte_shift=0, a=None, b=None):
    """Steps two identical states, one through a context, one through desloc_step_static(), and
    requires the same bits after every step."""
    from test_parity_gpu import make_engine
    dev = torch.device("cuda:0")
    w = w.replace(K=K)
    a = a or State(w, dev, byte_shift=byte_shift, v_init=0.25)
    b = b or State(w, dev, byte_shift=byte_shift, v_init=0.25)
    eng = make_engine(d, w, a, post)
    flags = (d.DESLOC_FLAG_ADOPT_NORM_CLIP if w.adopt_norm_clip else 0) | \
        (d.DESLOC_FLAG_POST_AVERAGE if post else 0)
    cfg = d.make_config(w.M, w.numel, w.opt, w.grad_dtype, w.beta1, w.beta2, w.eps,
                        w.weight_decay, w.clip_rho, K[0], K[1], K[2], flags)
    stream = torch.cuda.current_stream(dev).cuda_stream
    for t in range(steps):
        a.fill_grads(t)
        for m in range(w.M):
            b.g[m].copy_(a.g[m])
        lr, cb = f32r(w.lr), f32r(w.clip_bound(t) if t else 1.0)
        mk_a = eng.step(t, lr, a.views(a.g), clip_bound=cb)
        mk_b = d.desloc_step_static(cfg, _flat_ptrs(b, b.x), _flat_ptrs(b, b.u),
                                    _flat_ptrs(b, b.v) if b.v is not None else None,
                                    _flat_ptrs(b, b.g), t, lr, cb, 0, stream)
        assert mk_a == mk_b
        torch.cuda.synchronize()
        for pa, pb in [(a.x, b.x), (a.u, b.u)] + ([(a.v, b.v)] if a.v is not None else []):
            assert np.array_equal(a.to_numpy(pa), b.to_numpy(pb))
    eng.close()


def test_static_entry_point_with_one_worker_and_the_other_orderings():
    """M = 1 (the per-worker kernel), the post-average ordering, fp32 gradients and buffers that
    are not 16-byte aligned: each must give the context path's bits."""
    import paper_2505_22549_b200 as d
    base = di.mini(di.WORKLOADS["cfg2_adam_135m"])
    _ctx_vs_static(d, base.replace(M=1), (2, 3, 4), 3)
    _ctx_vs_static(d, base.replace(M=3), (1, 2, 3), 3, post=True)
    _ctx_vs_static(d, di.mini(di.WORKLOADS["cfg3_adopt_360m"]), (1, 1, 2), 3, post=True)
    _ctx_vs_static(d, base.replace(M=2, grad_dtype="f32", grad_kind="normal1", lr=1e-2), (2, 2, 2), 3,
                   byte_shift=1)


def test_static_entry_point_reuses_the_array_for_a_smaller_problem():
    """A large tensor list (many chunks, 8 workers) and then a small one (one tensor, 2 workers)
    on the same stream, then the large one again: each call must rewrite what it uses of the
    shared array, whatever the previous call left there.  Calls that repeat the previous call's
    buffers (nothing to upload) are in the sequence too."""
    import paper_2505_22549_b200 as d
    big = di.mini(di.WORKLOADS["cfg5_adam_desloc"])                        # M = 8, 21 tensors
    small = di.Workload("one_tensor", "adam", 2, (5000,), "bf16", "normal_offset", seed=5)
    for w, steps in ((big, 3), (small, 3), (big, 2), (small.replace(M=4), 2)):
        _ctx_vs_static(d, w, (2, 3, 2), steps)


def test_static_entry_point_refuses_a_capturing_stream():
    """The call uploads from host memory the library reuses, so it must not be recorded into a
    CUDA graph: on a capturing stream it returns DESLOC_E_INVALID and enqueues nothing."""
    import paper_2505_22549_b200 as d
    dev = torch.device("cuda:0")
    w = di.mini(di.WORKLOADS["cfg2_adam_135m"]).replace(M=2)
    st = State(w, dev)
    st.fill_grads(0)
    cfg = d.make_config(w.M, w.numel, w.opt, w.grad_dtype, w.beta1, w.beta2, w.eps)
    x_before = st.to_numpy(st.x)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream(dev))
    graph = torch.cuda.CUDAGraph()
    scratch = torch.zeros(8, device=dev)
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            scratch.add_(1.0)                     # the capture holds something of its own
            with pytest.raises(d.DeslocError) as e:
                d.desloc_step_static(cfg, _flat_ptrs(st, st.x), _flat_ptrs(st, st.u),
                                     _flat_ptrs(st, st.v), _flat_ptrs(st, st.g), 0, 1e-3, 0.0, 0,
                                     side.cuda_stream)
            assert e.value.status == d.DESLOC_E_INVALID
    graph.replay()
    torch.cuda.synchronize()
    assert float(scratch.sum()) == 8.0            # the capture survived and holds only its own op
    assert np.array_equal(st.to_numpy(st.x), x_before)
    # and the same call outside capture works
    d.desloc_step_static(cfg, _flat_ptrs(st, st.x), _flat_ptrs(st, st.u), _flat_ptrs(st, st.v),
                         _flat_ptrs(st, st.g), 0, 1e-3, 0.0, 0, torch.cuda.current_stream(dev).cuda_stream)
    torch.cuda.synchronize()
    assert not np.array_equal(st.to_numpy(st.x), x_before)
