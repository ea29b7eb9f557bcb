"""GPU parity: the CUDA library (through its C ABI binding) against the CPU oracle, element by
element on the same seeded inputs.  Bar: relative error <= 1e-5 on fp32 x, u, v after T steps
(denominator max(|ref|, rms(ref tensor))), sync masks and counters exact as integers."""
import numpy as np
import pytest
import torch

import desloc_inputs as di
import oracle
from _util import OPT_ID, TOL, State, compare_per_tensor, f32r, oracle_cfg, rel_err

pytestmark = pytest.mark.gpu


def _lib():
    import paper_2505_22549_b200 as d
    return d


def _flags(d, w, post=False):
    f = 0
    if w.adopt_norm_clip:
        f |= d.DESLOC_FLAG_ADOPT_NORM_CLIP
    if post:
        f |= d.DESLOC_FLAG_POST_AVERAGE
    return f


def make_engine(d, w, st, post=False):
    return d.DesLoc(st.views(st.x), st.views(st.u), st.views(st.v) if st.v is not None else None,
                    opt=w.opt, grad_dtype=w.grad_dtype, beta1=w.beta1, beta2=w.beta2, eps=w.eps,
                    weight_decay=w.weight_decay, clip_rho=w.clip_rho, K=w.K,
                    flags=_flags(d, w, post))


def run_both(w, T, align=4, byte_shift=0, post=False, v_init=0.0, identical=False,
             forced_masks=None, lr_of_t=None, max_blocks=0, g_shift=None, staging=None):
    """Runs T steps on the GPU and in the oracle on identical inputs; returns both end states."""
    d = _lib()
    dev = torch.device("cuda:0")
    st = State(w, dev, align=align, byte_shift=byte_shift, v_init=v_init, g_shift=g_shift)
    eng = make_engine(d, w, st, post)
    if max_blocks:
        d.desloc_testing_set_max_blocks(eng.ctx, max_blocks)   # blocks stride over the chunks
    if staging is not None:
        d.desloc_testing_set_staging(eng.ctx, staging)         # 0: always stage, 1: never
    ox, ou = st.to_numpy(st.x), st.to_numpy(st.u)
    ov = st.to_numpy(st.v) if st.v is not None else None
    ocfg = oracle_cfg(w, oracle.FLAG_POST_AVERAGE if post else 0)
    gviews = st.views(st.g)
    gpu_masks, ref_masks = [], []
    for t in range(T):
        st.fill_grads(t, identical=identical)
        lr = f32r(lr_of_t(t) if lr_of_t else w.lr)
        cb = f32r(w.clip_bound(t))
        g_host = st.to_numpy(st.g)
        if forced_masks is None:
            gpu_masks.append(eng.step(t, lr, gviews, clip_bound=cb))
            ref_masks.append(oracle.step(ocfg, t, lr, ox, ou, ov, g_host, clip_bound=cb))
        else:
            # force one sync pattern: the oracle gets periods that produce it at t = 0, else none
            mk = forced_masks[t]
            eng.step_masked(mk, lr, gviews, clip_bound=cb)
            c2 = oracle_cfg(w.replace(K=(mk & 1, (mk >> 1) & 1, (mk >> 2) & 1)),
                            oracle.FLAG_POST_AVERAGE if post else 0)
            got = oracle.step(c2, 0, lr, ox, ou, ov, g_host, clip_bound=cb)
            assert got == mk
    torch.cuda.synchronize()
    res = dict(st=st, gx=st.to_numpy(st.x), gu=st.to_numpy(st.u),
               gv=st.to_numpy(st.v) if st.v is not None else None, ox=ox, ou=ou, ov=ov,
               gpu_masks=gpu_masks, ref_masks=ref_masks, counters=eng.counters(),
               launches=eng.launches())
    eng.close()
    return res


def check(res, tol=TOL):
    st = res["st"]
    worst = {"x": compare_per_tensor(st, res["gx"], res["ox"], "x", tol),
             "u": compare_per_tensor(st, res["gu"], res["ou"], "u", tol)}
    if res["gv"] is not None:
        worst["v"] = compare_per_tensor(st, res["gv"], res["ov"], "v", tol)
    assert res["gpu_masks"] == res["ref_masks"]
    return worst


# ------------------------------------------------------------------ config 1, all elements
def test_cfg1_adam_n4096_full_run():
    w = di.WORKLOADS["cfg1_adam_n4096"]
    res = run_both(w, w.T)
    check(res)
    assert res["gpu_masks"][:9] == [7, 0, 0, 0, 1, 0, 0, 0, 3]
    assert res["counters"] == [64, 16, 8, 4]
    assert res["launches"] == 64            # one kernel per step
    # the run really moved the parameters (the check is not vacuous)
    x0 = di.init_params(w).numpy()
    assert np.max(np.abs(res["gx"][0] - x0)) > 1e-2


# ------------------------------------------------------------------ tiny and ragged shapes
@pytest.mark.parametrize("opt", ["adam", "adopt", "sgdm"])
@pytest.mark.parametrize("M", [1, 2, 3, 4, 5, 6, 7, 8])
@pytest.mark.parametrize("gd", ["f32", "bf16"])
@pytest.mark.parametrize("staging", [0, 1])
def test_every_mask_on_ragged_tensors(opt, M, gd, staging):
    """Tensors of 1..9 elements, one chunk + 1, odd sizes; all 8 sync patterns in turn, twice.
    A problem this small would skip the staging by itself: it is run staged (tiles through
    shared memory wherever alignment allows) and unstaged (everything straight from global
    memory)."""
    numel = (1, 2, 3, 4, 5, 7, 8, 9, 4095, 4096, 4097, 8191, 12289, 31)
    nmask = 4 if opt == "sgdm" else 8
    masks = list(range(nmask)) * 2
    w = di.Workload(f"tiny_{opt}", opt, M, numel, gd, "normal1", beta1=0.9, beta2=0.99,
                    eps=1e-3 if opt != "adopt" else 1e-2, lr=1e-2, weight_decay=0.05,
                    clip_rho=1.5, adopt_norm_clip=(opt == "adopt"), seed=M)
    for align in (4, 1):   # 4: vector path with tails; 1: packed, odd offsets -> scalar path
        res = run_both(w, len(masks), align=align, forced_masks=masks, v_init=0.25, staging=staging)
        check(res)


def test_small_launches_skip_the_staging_and_give_the_same_bits():
    """The library's own choice (no staging for a single wave of single-tile chunks) against
    both forced modes: the arithmetic per coordinate is the same, so are the bits."""
    w = di.Workload("small", "adam", 4, (4096, 1000, 37), "bf16", "normal1", lr=1e-2, K=(2, 3, 4), seed=5)
    runs = [run_both(w, 8, staging=mode) for mode in (None, 0, 1)]
    for r in runs:
        check(r)
    for r in runs[1:]:
        for k in ("gx", "gu", "gv"):
            assert np.array_equal(r[k], runs[0][k])


@pytest.mark.parametrize("opt", ["adam", "adopt", "sgdm"])
@pytest.mark.parametrize("M", [2, 3, 8])
def test_post_average_ordering(opt, M):
    numel = (5, 4096, 4099, 1000)
    nmask = 4 if opt == "sgdm" else 8
    masks = list(range(nmask)) + [nmask - 1]
    w = di.Workload(f"post_{opt}", opt, M, numel, "bf16", "normal1", beta1=0.9, beta2=0.99,
                    eps=1e-2, lr=1e-2, clip_rho=2.0, seed=7 + M)
    res = run_both(w, len(masks), forced_masks=masks, post=True, v_init=0.5)
    check(res)
    # after a step that averaged everything, replicas are bitwise equal
    for a in ("gx", "gu") + (("gv",) if opt != "sgdm" else ()):
        for m in range(1, M):
            assert np.array_equal(res[a][0], res[a][m])


@pytest.mark.parametrize("opt", ["adam", "adopt", "sgdm"])
@pytest.mark.parametrize("M,post", [(9, False), (16, False), (16, True), (33, True), (64, False), (256, False)])
def test_many_workers_runtime_m_path(opt, M, post):
    """More workers than the register-resident kernels hold (M > 8): runtime-M kernel on sync
    steps, per-worker items on local steps; up to the largest M a context accepts."""
    numel = (3, 4096, 4101, 777)
    nmask = 4 if opt == "sgdm" else 8
    masks = list(range(nmask)) + [nmask - 1, 0]
    w = di.Workload(f"many_{opt}", opt, M, numel, "bf16", "normal1", beta1=0.9, beta2=0.99,
                    eps=1e-2, lr=1e-2, weight_decay=0.01, clip_rho=2.0,
                    adopt_norm_clip=(opt == "adopt"), seed=11 + M)
    for align in (4, 1):
        res = run_both(w, len(masks), align=align, forced_masks=masks, post=post, v_init=0.5)
        check(res)


def test_identical_gradients_with_sixteen_workers_match_single_worker():
    base = di.mini(di.WORKLOADS["cfg5_adam_ddp"], T=8).replace(K=(1, 2, 3))
    many = run_both(base.replace(M=16), base.T, identical=True)
    one = run_both(base.replace(M=1), base.T, identical=True)
    check(many)
    for k in ("gx", "gu", "gv"):
        # the sixteen replicas stay bitwise equal to one another (their mean is exact: a batch of
        # equal values sums without rounding) ...
        for m in range(1, 16):
            assert np.array_equal(many[k][m], many[k][0])
        # ... and follow the single-worker run to within the bar, not bit for bit: the runtime-M
        # kernel takes the hardware reciprocal square root (2 ulp) where the others use IEEE
        # sqrt and division
        assert rel_err(many[k][0], one[k][0]) <= TOL


def test_misaligned_buffers_take_the_scalar_path():
    w = di.Workload("shift", "adam", 3, (4096 * 2 + 5, 17), "bf16", "normal1", lr=1e-2,
                    K=(2, 3, 4), seed=3)
    for shift in (1, 2, 3):
        res = run_both(w, 6, align=1, byte_shift=shift)
        check(res)


@pytest.mark.parametrize("M,opt", [(2, "adam"), (4, "adopt"), (8, "sgdm"), (12, "adam")])
@pytest.mark.parametrize("shift,g_shift", [(8, None), (24, None), (504, None), (8, 0), (8, 4), (40, 16),
                                           (4, None), (4, 0), (12, 2), (1, None), (3, 0)])
def test_first_chunks_cut_at_2kb_boundaries(M, opt, shift, g_shift):
    """State buffers that start 32 B ... 2016 B past a 2 KB boundary: the chunk plan cuts every
    tensor's first chunk at the next boundary (504, 488, 8 elements here, and others for the
    later tensors).  Gradients that share the state's offsets are then aligned as well; gradients
    laid out differently (g_shift) stay 16-byte aligned where they were (shift 0, 16 elements)
    or take the 128-bit path from global memory (bf16 shifted by 4 elements = 8 bytes)."""
    gd = "bf16" if opt != "sgdm" else "f32"
    w = di.Workload("heads", opt, M, (512 * 9 + 64, 40, 1024, 512 * 3 - 8, 7), gd, "normal1", lr=1e-2,
                    K=(2, 3, 4), seed=11, adopt_norm_clip=(opt == "adopt"))
    res = run_both(w, 7, align=8, byte_shift=shift, g_shift=g_shift)
    check(res)


# ------------------------------------------------------------------ scaled-down paper workloads
MINI = ["cfg2_adam_135m", "cfg3_adopt_360m", "cfg4_adam_1p7b", "cfg5_sgdm_ddp", "cfg5_sgdm_desloc",
        "cfg5_adam_local", "cfg5_adam_desloc"]


@pytest.mark.parametrize("name", MINI)
def test_mini_workloads_full_oracle(name):
    """Same recipe (optimizer, M, gradient distribution, hyper-parameters) on a 2-layer model
    of 21 tensors; periods shortened so that T = 40 steps see every sync pattern."""
    w = di.mini(di.WORKLOADS[name], T=40)
    if max(w.K) > 16:
        w = w.replace(K=tuple(max(1, k // 8) for k in w.K))
    res = run_both(w, w.T)
    worst = check(res)
    assert res["counters"][0] == w.T
    assert sum(res["counters"][1:]) == sum(bin(m).count("1") for m in res["ref_masks"])
    print(name, worst)


@pytest.mark.parametrize("name", ["cfg2_adam_135m", "cfg3_adopt_360m", "cfg5_adam_desloc",
                                  "cfg5_sgdm_desloc"])
def test_mini_workloads_full_horizon_and_periods(name):
    """The workloads' own step counts (T = 256 / 512) and periods (up to K_v = 256) on the mini
    model: the error bar must hold after the whole horizon, not only after a few steps."""
    w = di.mini(di.WORKLOADS[name])
    res = run_both(w, w.T)
    worst = check(res)
    want = [-(-w.T // k) for k in w.K[:2]] + ([-(-w.T // w.K[2])] if w.opt != "sgdm" else [0])
    assert res["counters"] == [w.T] + want
    print(name, w.T, worst)


@pytest.mark.parametrize("M", [1, 4, 8, 12])
def test_striding_grid_gives_identical_bits(M):
    """A grid smaller than the number of chunks (blocks stride over the rest) must give the same
    bits as one block per chunk: the step, local and diagnostics kernels all take the loop."""
    w = di.mini(di.WORKLOADS["cfg2_adam_135m"], T=12).replace(M=M, K=(2, 3, 4))
    a = run_both(w, w.T)
    b = run_both(w, w.T, max_blocks=3)
    for k in ("gx", "gu", "gv"):
        assert np.array_equal(a[k], b[k])


def test_two_runs_are_bitwise_equal():
    w = di.mini(di.WORKLOADS["cfg3_adopt_360m"], T=10).replace(K=(2, 3, 4))
    a = run_both(w, w.T)
    b = run_both(w, w.T)
    for k in ("gx", "gu", "gv"):
        assert np.array_equal(a[k], b[k])


@pytest.mark.parametrize("opt", ["adam", "sgdm"])
@pytest.mark.parametrize("M", [2, 4, 8])
def test_identical_gradients_match_single_worker_run(opt, M):
    """Same gradients on every worker: replicas stay bitwise equal to the M = 1 run for any
    schedule, (1,1,1) "DDP-equivalent" included (fp32 sums of M equal values and the division
    by M are exact for M a power of two)."""
    base = di.mini(di.WORKLOADS[f"cfg5_{opt}_ddp"], T=16)
    for K in [(1, 1, 1), (16, 16, 16), (2, 3, 5)]:
        many = run_both(base.replace(M=M, K=K), base.T, identical=True)
        one = run_both(base.replace(M=1, K=K), base.T, identical=True)
        for k in ("gx", "gu") + (("gv",) if opt != "sgdm" else ()):
            for m in range(M):
                assert np.array_equal(many[k][m], one[k][0]), (K, k, m)


def test_resume_is_bitwise_identical():
    """State is the caller's buffers plus the integer t: a fresh context continues a run."""
    d = _lib()
    w = di.mini(di.WORKLOADS["cfg2_adam_135m"], T=12).replace(K=(2, 3, 4))
    full = run_both(w, w.T)
    dev = torch.device("cuda:0")
    st = State(w, dev)
    gv = st.views(st.g)
    eng = make_engine(d, w, st)
    for t in range(w.T):
        if t == w.T // 2:
            eng.close()
            eng = make_engine(d, w, st)
        st.fill_grads(t)
        eng.step(t, f32r(w.lr), gv)
    torch.cuda.synchronize()
    assert np.array_equal(st.to_numpy(st.x), full["gx"])
    assert np.array_equal(st.to_numpy(st.v), full["gv"])
    eng.close()


# ------------------------------------------------------------------ API behaviour on a device
def test_gradient_pointers_may_change_every_step_and_lr_schedule():
    d = _lib()
    w = di.Workload("swap", "adam", 2, (5000, 33), "bf16", "normal1", lr=1e-2, K=(2, 2, 3), seed=5)
    dev = torch.device("cuda:0")
    st = State(w, dev)
    eng = make_engine(d, w, st)
    ox, ou, ov = st.to_numpy(st.x), st.to_numpy(st.u), st.to_numpy(st.v)
    ocfg = oracle_cfg(w)
    keep = []
    for t in range(20):                      # more table changes than staging slots
        st.fill_grads(t)
        fresh = [b.clone() for b in st.g]    # new addresses every step
        keep.append(fresh)
        lr = f32r(1e-2 / (1 + t))
        eng.step(t, lr, st.views(fresh))
        oracle.step(ocfg, t, lr, ox, ou, ov, st.to_numpy(fresh))
    torch.cuda.synchronize()
    assert rel_err(st.to_numpy(st.x), ox) <= TOL
    assert rel_err(st.to_numpy(st.v), ov) <= TOL
    eng.close()


@pytest.mark.parametrize("name", ["cfg2_adam_135m", "cfg3_adopt_360m"])
def test_step_host_equals_step_with_device_gradients(name):
    """Gradients handed over in pinned host memory: same bits as the device-gradient path, for
    packed buffers (merged copies) and for separately allocated tensors."""
    d = _lib()
    w = di.mini(di.WORKLOADS[name], T=6).replace(K=(2, 3, 4))
    dev = torch.device("cuda:0")
    a, b = State(w, dev), State(w, dev)
    ea, eb = make_engine(d, w, a), make_engine(d, w, b)
    hflat = [torch.empty(b.nflat, dtype=b.g[0].dtype).pin_memory() for _ in range(w.M)]
    hsep = [[torch.empty(n, dtype=b.g[0].dtype).pin_memory() for n in w.numel] for _ in range(w.M)]
    hview = [[h[o:o + n] for o, n in zip(b.offs, w.numel)] for h in hflat]
    for t in range(w.T):
        a.fill_grads(t)
        for m in range(w.M):
            hflat[m].copy_(a.g[m])
            for hs, src in zip(hsep[m], a.views(a.g)[m]):
                hs.copy_(src)
            b.g[m].zero_()
        torch.cuda.synchronize()
        lr, cb = f32r(w.lr), f32r(w.clip_bound(t))
        ma = ea.step(t, lr, a.views(a.g), clip_bound=cb)
        mb = eb.step_host(t, lr, hview if t % 2 == 0 else hsep, b.views(b.g), clip_bound=cb)
        assert ma == mb
    torch.cuda.synchronize()
    for pa, pb in [(a.x, b.x), (a.u, b.u), (a.v, b.v)]:
        assert np.array_equal(a.to_numpy(pa), b.to_numpy(pb))
    assert eb.launches() > ea.launches()      # one launch per tensor group
    ea.close(); eb.close()


def test_guard_bands_around_every_tensor_stay_untouched():
    """Each element is written by exactly one thread and nothing outside a tensor is touched:
    tensors are laid out with up to 15 elements of padding between them (and 32 in front and
    behind), filled with a sentinel that must survive every kind of step."""
    d = _lib()
    SENT = -12288.0        # exact in bf16 too
    for opt, M in [("adam", 4), ("adopt", 8), ("sgdm", 3), ("adam", 12), ("adam", 1)]:
        numel = (1, 5, 4096, 4097, 777, 8192 + 3, 64)
        w = di.Workload("guard", opt, M, numel, "bf16", "normal1", lr=1e-2, clip_rho=1.0, seed=9,
                        adopt_norm_clip=(opt == "adopt"))
        dev = torch.device("cuda:0")
        offs, pos = [], 32
        for n in numel:
            pos = -(-pos // 16) * 16 + (4 if n % 2 else 0)   # some starts 16-byte aligned, some not
            offs.append(pos)
            pos += n + 5
        total = pos + 32
        mk = lambda dt: torch.full((total,), SENT, dtype=dt, device=dev)
        X, U, V = [mk(torch.float32) for _ in range(M)], [mk(torch.float32) for _ in range(M)], \
            [mk(torch.float32) for _ in range(M)]
        G = [mk(torch.bfloat16) for _ in range(M)]
        views = lambda bufs: [[b[o:o + n] for o, n in zip(offs, numel)] for b in bufs]
        for bufs, val in ((X, 0.5), (U, 0.0), (V, 0.25), (G, 0.125)):
            for lst in views(bufs):
                for t in lst:
                    t.fill_(val)
        eng = d.DesLoc(views(X), views(U), views(V) if opt != "sgdm" else None, opt=opt,
                       grad_dtype="bf16", clip_rho=1.0, K=(2, 3, 4),
                       flags=d.DESLOC_FLAG_ADOPT_NORM_CLIP if opt == "adopt" else 0)
        inside = torch.zeros(total, dtype=torch.bool, device=dev)
        for o, n in zip(offs, numel):
            inside[o:o + n] = True
        for t in range(13):
            if t % 3 == 2:
                eng.step_normclip(t, 1e-2, views(G), 0.01, clip_bound=1.0)
            else:
                eng.step(t, 1e-2, views(G), clip_bound=1.0)
        torch.cuda.synchronize()
        for bufs in (X, U) + ((V,) if opt != "sgdm" else ()):
            for b in bufs:
                assert bool((b[~inside] == SENT).all()), f"{opt} M={M}: wrote outside a tensor"
                assert bool((b[inside] != SENT).all())
        assert bool((X[0][inside] != 0.5).all())          # every element was updated
        for b in G:
            assert bool((b[~inside].float() == SENT).all())
        eng.close()


def test_never_sync_periods_and_large_step_numbers():
    """K = 0 means never (the FedAvg-with-local-states baseline keeps K_u = K_v = 0); t far
    beyond 2^31 still schedules correctly."""
    d = _lib()
    w = di.Workload("never", "adam", 3, (100, 4096), "f32", "normal1", lr=1e-2, K=(4, 0, 0), seed=2)
    res = run_both(w, 9)
    check(res)
    assert res["gpu_masks"] == [1, 0, 0, 0, 1, 0, 0, 0, 1]
    assert res["counters"] == [9, 3, 0, 0]
    dev = torch.device("cuda:0")
    st = State(w.replace(K=(3, 5, 7)), dev)
    eng = make_engine(d, w.replace(K=(3, 5, 7)), st)
    st.fill_grads(0)
    big = 3 * 5 * 7 * (1 << 40)
    assert eng.step(big, 1e-3, st.views(st.g)) == 7
    assert eng.step(big + 3, 1e-3, st.views(st.g)) == 1
    assert eng.step(big + 35, 1e-3, st.views(st.g)) == 6
    torch.cuda.synchronize()
    eng.close()


def test_create_on_a_device_that_does_not_exist():
    d = _lib()
    x = torch.zeros(4, device="cuda:0")
    cfg = d.make_config(1, [4], "sgdm", "f32")
    with pytest.raises(d.DeslocError) as e:
        d.desloc_create(cfg, [x.data_ptr()], [x.data_ptr()], None, 4096)
    assert e.value.status == d.DESLOC_E_CUDA
    # the failed create left the runtime usable
    ctx = d.desloc_create(cfg, [x.data_ptr()], [torch.zeros(4, device="cuda:0").data_ptr()], None, 0)
    d.desloc_destroy(ctx)


def test_two_contexts_on_two_streams_and_stream_changes():
    """Independent contexts may run concurrently on different streams; one context may move from
    stream to stream (its gradient pointer table is re-staged on the new stream).  Results equal
    the plain single-stream runs bit for bit."""
    d = _lib()
    dev = torch.device("cuda:0")
    wa = di.mini(di.WORKLOADS["cfg2_adam_135m"], T=8).replace(K=(2, 3, 4))
    wb = di.mini(di.WORKLOADS["cfg5_sgdm_desloc"], T=8).replace(K=(3, 2, 0), seed=4)
    ref_a, ref_b = run_both(wa, wa.T), run_both(wb, wb.T)
    sa, sb = State(wa, dev), State(wb, dev)
    ea, eb = make_engine(d, wa, sa), make_engine(d, wb, sb)
    streams = [torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()]
    torch.cuda.synchronize()
    for t in range(8):
        sa.fill_grads(t)
        sb.fill_grads(t)
        torch.cuda.synchronize()                       # gradients ready before the side streams read them
        with torch.cuda.stream(streams[t % 2]):        # context a hops between two streams
            ea.step(t, f32r(wa.lr), sa.views(sa.g))
        with torch.cuda.stream(streams[2]):            # context b runs alongside on a third
            eb.step(t, f32r(wb.lr), sb.views(sb.g))
        for s_ in streams:                             # a's next step must see this one's result
            s_.synchronize()
    torch.cuda.synchronize()
    assert np.array_equal(sa.to_numpy(sa.x), ref_a["gx"]) and np.array_equal(sa.to_numpy(sa.v), ref_a["gv"])
    assert np.array_equal(sb.to_numpy(sb.x), ref_b["gx"]) and np.array_equal(sb.to_numpy(sb.u), ref_b["gu"])
    ea.close(); eb.close()


def test_steps_allocate_no_device_memory():
    """Everything a context needs is allocated by desloc_create(): free device memory (as the
    driver reports it, which also sees allocations made outside torch) is the same before and
    after many steps of every kind, with gradient pointers changing from step to step."""
    d = _lib()
    w = di.mini(di.WORKLOADS["cfg3_adopt_360m"], T=30).replace(K=(2, 3, 4))
    dev = torch.device("cuda:0")
    st = State(w, dev)
    eng = make_engine(d, w, st)
    alt = [b.clone() for b in st.g]
    hflat = [torch.empty(st.nflat, dtype=st.g[0].dtype).pin_memory() for _ in range(w.M)]
    hview = [[h[o:o + n] for o, n in zip(st.offs, w.numel)] for h in hflat]
    st.fill_grads(0)
    for kind in range(4):                       # first use of every entry point, then measure
        eng.step(kind, 1e-3, st.views(st.g), clip_bound=1.0)
    eng.step_normclip(4, 1e-3, st.views(alt), 0.5, clip_bound=1.0)
    eng.step_host(5, 1e-3, hview, st.views(st.g), clip_bound=1.0)
    cfg = d.make_config(w.M, w.numel, w.opt, w.grad_dtype, w.beta1, w.beta2, w.eps, 0.0, w.clip_rho,
                        2, 3, 4, d.DESLOC_FLAG_ADOPT_NORM_CLIP)
    flat = lambda bufs: [t.data_ptr() for lst in st.views(bufs) for t in lst]
    d.desloc_step_static(cfg, flat(st.x), flat(st.u), flat(st.v), flat(st.g), 6, 1e-3, 1.0, 0,
                         torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for t in range(7, 30):
        gsel = st.g if t % 2 else alt
        if t % 5 == 0:
            eng.step_normclip(t, 1e-3, st.views(gsel), 0.5, clip_bound=1.0)
        elif t % 7 == 0:
            eng.step_host(t, 1e-3, hview, st.views(st.g), clip_bound=1.0)
        elif t % 11 == 0:
            d.desloc_step_static(cfg, flat(st.x), flat(st.u), flat(st.v), flat(gsel), t, 1e-3, 1.0, 0,
                                 torch.cuda.current_stream().cuda_stream)
        else:
            eng.step(t, 1e-3, st.views(gsel), clip_bound=1.0)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    eng.close()


def test_errors_are_status_codes_and_context_survives():
    d = _lib()
    dev = torch.device("cuda:0")
    x = torch.zeros(8, device=dev)
    u = torch.zeros(8, device=dev)
    v = torch.zeros(8, device=dev)
    g = torch.ones(8, device=dev)
    cfg = d.make_config(1, [8], "adam", "f32")
    ctx = d.desloc_create(cfg, [x.data_ptr()], [u.data_ptr()], [v.data_ptr()], 0)
    with pytest.raises(d.DeslocError) as e:
        d.desloc_step(ctx, -1, 1e-3, 0.0, [g.data_ptr()])
    assert e.value.status == d.DESLOC_E_RANGE
    with pytest.raises(d.DeslocError) as e:
        d.desloc_step(ctx, 0, 1e-3, 0.0, [0])
    assert e.value.status == d.DESLOC_E_NULL
    with pytest.raises(d.DeslocError) as e:
        d.desloc_step_masked(ctx, 8, 1e-3, 0.0, [g.data_ptr()])
    assert e.value.status == d.DESLOC_E_INVALID
    with pytest.raises(d.DeslocError) as e:
        d.desloc_step(ctx, 0, float("nan"), 0.0, [g.data_ptr()])
    assert e.value.status == d.DESLOC_E_RANGE
    assert d.desloc_step(ctx, 0, 0.5, 0.0, [g.data_ptr()]) == 7
    torch.cuda.synchronize()
    assert d.desloc_get_counters(ctx) == [1, 1, 1, 1]
    # Adam, zero states, g = 1, default eps: u = 0.1, v = 0.001, x = -0.5*0.1/sqrt(0.001)
    assert torch.allclose(u, torch.full_like(u, 0.1), rtol=1e-6)
    assert torch.allclose(x, torch.full_like(x, -0.5 * 0.1 / 0.001 ** 0.5), rtol=1e-4)
    d.desloc_destroy(ctx)
    d.desloc_destroy(None)
