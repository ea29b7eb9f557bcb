"""World-size-2 checks on CPU (gloo): the parameter-range sharding used for more than one GPU
covers every element once, the ranks' timings reduce to max / their units to a sum, and --
because no coordinate depends on another -- stepping the shards separately reproduces the
unsharded run bit for bit (shown with the oracle; the CUDA path needs a device)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import desloc_inputs as di
        import oracle
        from paper_2505_22549_b200 import dist as dd

        w = di.mini(di.WORKLOADS["cfg2_adam_135m"], T=6).replace(K=(2, 3, 4))
        offs = di.offsets_of(w.numel)
        n = di.flat_size(w.numel)
        x0 = di.init_params(w).numpy()
        g = torch.empty(w.T, w.M, n, dtype=torch.bfloat16)
        for t in range(w.T):
            for m in range(w.M):
                di.fill_grads_(w, t, m, g[t, m])
        g = np.ascontiguousarray(g.float().numpy())
        f32 = lambda a: float(np.float32(a))
        cfg = oracle.make_cfg(w.M, oracle.ADAM, beta1=f32(w.beta1), beta2=f32(w.beta2),
                              eps=f32(w.eps), Kx=w.K[0], Ku=w.K[1], Kv=w.K[2])
        # this rank's slices, small alignment so that both ranks own something non-trivial
        mine = dd.shard_tensor_list(w.numel, rank, world, align=64)
        idx = np.concatenate([np.arange(offs[k] + s, offs[k] + s + c) for k, s, c in mine])
        x = np.ascontiguousarray(np.tile(x0[idx], (w.M, 1)))
        u, v = np.zeros_like(x), np.zeros_like(x)
        masks = oracle.run(cfg, 0, [f32(w.lr)] * w.T, x, u, v, np.ascontiguousarray(g[:, :, idx]))
        # gather every rank's result on rank 0
        gathered = [None] * world
        dist.all_gather_object(gathered, (idx, x, u, v, masks.tolist(), mine))
        rate = dd.whole_job_rate(units_per_rank=len(idx) * w.M, steps=w.T,
                                 local_ms=10.0 * (rank + 1))
        if rank == 0:
            xf = np.ascontiguousarray(np.tile(x0, (w.M, 1)))
            uf, vf = np.zeros_like(xf), np.zeros_like(xf)
            mfull = oracle.run(cfg, 0, [f32(w.lr)] * w.T, xf, uf, vf, g)
            cover = np.zeros(n, dtype=np.int64)
            ok = True
            for gi, gx, gu, gv, gm, _ in gathered:
                cover[gi] += 1
                ok &= np.array_equal(gx, xf[:, gi]) and np.array_equal(gu, uf[:, gi])
                ok &= np.array_equal(gv, vf[:, gi]) and gm == mfull.tolist()
            q.put(dict(ok=bool(ok), cover_ok=bool(np.all(cover == 1)), rate=rate,
                       want_rate=n * w.M * w.T / (10.0 * world * 1e-3),
                       sizes=[len(a[0]) for a in gathered]))
    finally:
        dist.destroy_process_group()


def test_two_ranks_shard_by_parameter_range_without_exchange():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = q.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert res["cover_ok"], "shards must cover every parameter exactly once"
    assert res["ok"], "sharded run must equal the unsharded run bit for bit"
    assert abs(res["rate"] - res["want_rate"]) / res["want_rate"] < 1e-12
    assert min(res["sizes"]) > 0.3 * max(res["sizes"])


def test_shard_tensor_list_properties():
    sys.path.insert(0, ROOT)
    from paper_2505_22549_b200 import dist as dd
    import desloc_inputs as di
    for numel in [[1], [5, 4096, 4097, 100000], list(di.WORKLOADS["cfg4_adam_1p7b"].numel)]:
        for world in (1, 2, 3, 8):
            seen = [0] * len(numel)
            sizes = []
            for r in range(world):
                sl = dd.shard_tensor_list(numel, r, world)
                sizes.append(sum(c for _, _, c in sl))
                for k, s, c in sl:
                    assert s % 4096 == 0 and c > 0 and s + c <= numel[k]
                    assert s == seen[k]          # contiguous, in order, no overlap
                    seen[k] += c
            assert seen == list(numel)
            if sum(numel) > 10 ** 8:
                assert (max(sizes) - min(sizes)) / max(sizes) < 1e-3
    with pytest.raises(ValueError):
        dd.shard_tensor_list([4], 2, 2)


def test_bench_gpus_n_starts_n_ranks(monkeypatch):
    """`python bench.py --gpus N` outside torchrun must become N ranks (one per GPU) through
    torch.distributed.run on 127.0.0.1; under torchrun (WORLD_SIZE set) it must not re-launch."""
    import importlib
    import os
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    sys.path.insert(0, root)
    bench = importlib.import_module("bench")
    cmd = bench.launcher_command(4, ["--gpus", "4", "--steps", "5", "--warmup", "3"], port=29555)
    assert cmd[:3] == [sys.executable, "-m", "torch.distributed.run"]
    assert "--nnodes=1" in cmd and "--nproc-per-node=4" in cmd
    assert cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    assert cmd[cmd.index("--master-port") + 1] == "29555"
    assert cmd[-7] == os.path.join(root, "bench.py") and cmd[-6:] == ["--gpus", "4", "--steps", "5", "--warmup", "3"]
    assert bench.launcher_command(2, [])[-1].endswith("bench.py")          # picks a free port itself

    calls = []
    monkeypatch.setattr(bench.subprocess, "call", lambda c: calls.append(c) or 0)
    monkeypatch.delenv("WORLD_SIZE", raising=False)
    assert bench.main(["--gpus", "2", "--steps", "3"]) == 0
    assert len(calls) == 1 and "--nproc-per-node=2" in calls[0] and calls[0][-4:] == ["--gpus", "2", "--steps", "3"]
    # as a rank of a torchrun job: no second launch (the reference arm returns at once off rank 0)
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setenv("RANK", "1")
    assert bench.main(["--gpus", "2", "--impl", "reference", "--steps", "1"]) == 0
    assert len(calls) == 1
