"""Failure detection without a fault: every wait in the kernels is bounded.  A thread block that
does not see its tile arrive within the limit records that, lets the copies it requested land,
stores nothing and leaves; the host reports DESLOC_E_DEVICE_WAIT on the next call.  Here the
limit is set to zero polls through the test hook, so every block takes that path at once --
nothing hangs, nothing faults, and the context (and the GPU) stay usable."""
import numpy as np
import pytest
import torch

import desloc_inputs as di
from _util import State, f32r
from test_parity_gpu import make_engine

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["cfg2_adam_135m", "cfg3_adopt_360m", "cfg5_sgdm_desloc"])
def test_a_wait_that_runs_out_is_reported_and_nothing_is_stored(name):
    import paper_2505_22549_b200 as d
    w = di.mini(di.WORKLOADS[name], T=4).replace(K=(1, 1, 1))
    dev = torch.device("cuda:0")
    st = State(w, dev)
    eng = make_engine(d, w, st)
    st.fill_grads(0)
    eng.step(0, f32r(w.lr), st.views(st.g), clip_bound=1.0)
    torch.cuda.synchronize()
    before = [st.to_numpy(b) for b in (st.x, st.u) + ((st.v,) if st.v is not None else ())]

    d.desloc_testing_set_staging(eng.ctx, 0)                # stage even if the launch is small
    d.desloc_testing_set_wait_limit(eng.ctx, 0)             # every block gives up at once
    st.fill_grads(1)
    eng.step(1, f32r(w.lr), st.views(st.g), clip_bound=1.0)  # enqueues; the failure is on the device
    torch.cuda.synchronize()                                 # completes: no hang, no fault
    with pytest.raises(d.DeslocError) as e:
        eng.step(2, f32r(w.lr), st.views(st.g), clip_bound=1.0)
    assert e.value.status == d.DESLOC_E_DEVICE_WAIT
    with pytest.raises(d.DeslocError) as e:                  # and stays reported
        eng.step_masked(0, f32r(w.lr), st.views(st.g))
    assert e.value.status == d.DESLOC_E_DEVICE_WAIT
    after = [st.to_numpy(b) for b in (st.x, st.u) + ((st.v,) if st.v is not None else ())]
    # aligned full tiles stored nothing; the few ragged tiles (straight from global memory, no
    # wait involved) did their update: most of the state is untouched
    same = np.mean([np.mean(a == b) for a, b in zip(before, after)])
    assert same > 0.9

    d.desloc_testing_set_wait_limit(eng.ctx, -1)            # default limit, failure cleared
    ref = State(w, dev)
    eng2 = make_engine(d, w, ref)
    for b_dst, b_src in zip((ref.x, ref.u) + ((ref.v,) if ref.v is not None else ()),
                            (st.x, st.u) + ((st.v,) if st.v is not None else ())):
        for m in range(w.M):
            b_dst[m].copy_(b_src[m])
    for m in range(w.M):
        ref.g[m].copy_(st.g[m])
    eng.step(2, f32r(w.lr), st.views(st.g), clip_bound=1.0)      # the context works again
    eng2.step(2, f32r(w.lr), ref.views(ref.g), clip_bound=1.0)
    torch.cuda.synchronize()
    assert np.array_equal(st.to_numpy(st.x), ref.to_numpy(ref.x))
    assert not np.array_equal(st.to_numpy(st.x), after[0])
    eng.close(); eng2.close()
