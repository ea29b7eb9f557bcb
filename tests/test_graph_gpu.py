"""CUDA-graph replay of a window of lcm(K) steps for the small, launch-bound workload 1
(Adam, M = 2, N = 4096, K = (4, 8, 16), T = 64): four replays of a 16-step graph must equal
the oracle's 64 steps."""
import numpy as np
import pytest
import torch

import desloc_inputs as di
import oracle
from _util import State, compare_per_tensor, f32r, oracle_cfg
from test_parity_gpu import make_engine

pytestmark = pytest.mark.gpu


def test_graph_window_replay_matches_oracle():
    import paper_2505_22549_b200 as d
    w = di.WORKLOADS["cfg1_adam_n4096"]
    L = 16                                   # lcm(4, 8, 16)
    dev = torch.device("cuda:0")
    st = State(w, dev)
    eng = make_engine(d, w, st)
    ox, ou, ov = st.to_numpy(st.x), st.to_numpy(st.u), st.to_numpy(st.v)
    ocfg = oracle_cfg(w)
    # all 64 steps' gradients up front (2 MB); the window's 16 slots are refilled per replay
    allg = torch.empty(w.T, w.M, st.nflat, dtype=torch.float32, device=dev)
    for t in range(w.T):
        for m in range(w.M):
            di.fill_grads_(w, t, m, allg[t, m], align=4)
    win = torch.empty(L, w.M, st.nflat, dtype=torch.float32, device=dev)
    views = lambda j: [[win[j, m][o:o + n] for o, n in zip(st.offs, w.numel)] for m in range(w.M)]
    lr = f32r(w.lr)
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            masks = [eng.step(t, lr, views(t)) for t in range(L)]
    torch.cuda.current_stream().wait_stream(side)
    assert masks == [oracle.sync_mask(oracle.ADAM, 4, 8, 16, t) for t in range(L)]
    torch.cuda.synchronize()
    # capture itself ran nothing
    assert np.array_equal(st.to_numpy(st.x), ox)
    for r in range(w.T // L):
        win.copy_(allg[r * L:(r + 1) * L])
        graph.replay()
    torch.cuda.synchronize()
    for t in range(w.T):
        oracle.step(ocfg, t, lr, ox, ou, ov, np.ascontiguousarray(allg[t].cpu().numpy()))
    compare_per_tensor(st, st.to_numpy(st.x), ox, "x")
    compare_per_tensor(st, st.to_numpy(st.u), ou, "u")
    compare_per_tensor(st, st.to_numpy(st.v), ov, "v")
    assert eng.launches() == L               # captured once, replayed four times
    eng.close()


def test_capture_with_too_many_new_pointers_is_refused():
    import paper_2505_22549_b200 as d
    w = di.mini(di.WORKLOADS["cfg2_adam_135m"])       # 4 workers x 21 tensors = 84 pointers
    dev = torch.device("cuda:0")
    st = State(w, dev)
    eng = make_engine(d, w, st)
    st.fill_grads(0)
    other = [b.clone() for b in st.g]
    eng.step(0, 1e-3, st.views(st.g))                 # stages st.g's pointers
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        eng.step(1, 1e-3, st.views(st.g))             # same pointers on the capture stream
        with torch.cuda.graph(graph, stream=side):
            eng.step(2, 1e-3, st.views(st.g))         # resident table: allowed
            with pytest.raises(d.DeslocError) as e:
                eng.step(3, 1e-3, st.views(other))    # new pointers, too many to inline
            assert e.value.status == d.DESLOC_E_INVALID
    torch.cuda.current_stream().wait_stream(side)
    graph.replay()
    torch.cuda.synchronize()
    assert eng.counters()[0] == 3
    eng.close()
