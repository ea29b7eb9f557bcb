"""Host-side checks that need no GPU: the shared library loads and exports every symbol the
header declares, the schedule and the chunk plan are right, and bad arguments are rejected
before any CUDA call."""
import os
import re

import numpy as np
import pytest

import desloc_inputs as di
import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def d():
    from paper_2505_22549_b200 import build
    build.build()
    import paper_2505_22549_b200 as lib
    return lib


def test_library_exports_every_declared_symbol(d):
    names = []
    for h in ("desloc.h", "desloc_testing.h"):
        header = open(os.path.join(ROOT, "include", h)).read()
        names += re.findall(r"DESLOC_API\s+[\w\s\*]+?\b(desloc_\w+)\s*\(", header)
    assert len(names) >= 19 and len(set(names)) == len(names)
    for must in ("desloc_create", "desloc_step", "desloc_destroy", "desloc_step_diag",
                 "desloc_get_diag_norms", "desloc_step_static", "desloc_testing_set_max_blocks"):
        assert must in names
    L = d.raw_lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in a header but not exported"


def test_header_is_plain_c_and_a_c_program_links(d, tmp_path):
    """include/desloc.h compiles as strict C99, and a C program linked against the shared
    library can call the host-only entry points."""
    import subprocess
    from paper_2505_22549_b200 import binding
    inc = os.path.join(ROOT, "include")
    src = os.path.join(ROOT, "tests", "c_abi", "abi_check.c")
    exe = str(tmp_path / "abi_check")
    libdir = os.path.dirname(binding.LIB_PATH)
    subprocess.check_call(["gcc", "-std=c99", "-pedantic", "-Wall", "-Wextra", "-Werror", "-I", inc,
                           src, "-o", exe, "-L", libdir, "-ldesloc", f"-Wl,-rpath,{libdir}"])
    r = subprocess.run([exe], capture_output=True, text=True)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "abi_check: ok" in r.stdout


def test_sync_mask_matches_oracle_schedule(d):
    for opt, oid in (("adam", oracle.ADAM), ("adopt", oracle.ADOPT), ("sgdm", oracle.SGDM)):
        for K in [(4, 8, 16), (1, 1, 1), (16, 64, 256), (0, 0, 0), (3, 0, 7), (256, 768, 1536)]:
            cfg = d.make_config(2, [8], opt, "bf16", Kx=K[0], Ku=K[1], Kv=K[2])
            for t in list(range(0, 70)) + [255, 256, 767, 768, 1536, 3072, 2 ** 40]:
                assert d.desloc_sync_mask(cfg, t) == oracle.sync_mask(oid, K[0], K[1], K[2], t)
    assert d.desloc_sync_mask(None, 0) == 0
    cfg = d.make_config(2, [8], "adam", "bf16")
    assert d.desloc_sync_mask(cfg, -1) == 0


def test_chunk_plan_covers_every_element_once(d):
    big = [1 << 24] * 4                       # plenty of tiles: the full run per chunk
    want = {1: 8192, 2: 8192, 3: 4096, 4: 4096, 5: 4096, 8: 4096, 9: 8192, 256: 8192}
    for M, ce_want in want.items():
        assert d.desloc_chunk_elems(d.make_config(M, big, "adam", "bf16")) == ce_want
    # a small problem gets single-tile chunks so that it still spreads over many blocks
    assert d.desloc_chunk_elems(d.make_config(2, [4096], "adam", "f32")) == 1024
    assert d.desloc_chunk_elems(d.make_config(4, [4096 * 100], "adam", "f32")) == 512
    for bad in (0, 257):
        with pytest.raises(d.DeslocError):
            d.desloc_chunk_elems(d.make_config(bad, [8], "adam", "f32"))
    ce = 4096
    for numel in [[1], [ce], [ce + 1], [3, ce * 2, 5, ce * 3 - 1], list(di.mini(di.WORKLOADS["cfg2_adam_135m"]).numel)]:
        total, chunks = d.desloc_plan_chunks(numel, ce)
        assert total == len(chunks) == sum(-(-n // ce) for n in numel)
        seen = [0] * len(numel)
        for k, s, c in chunks:
            assert s == seen[k] and 1 <= c <= ce
            assert c == ce or s + c == numel[k]      # only a tensor's last chunk is short
            seen[k] += c
        assert seen == list(numel)
    # capacity smaller than needed: still reports the full count
    total, chunks = d.desloc_plan_chunks([ce * 10], ce, cap=3)
    assert total == 10 and len(chunks) == 3
    # full-size list of the 1.7B workload
    w = di.WORKLOADS["cfg4_adam_1p7b"]
    total, _ = d.desloc_plan_chunks(w.numel, ce, cap=0)
    assert total == sum(-(-n // ce) for n in w.numel)
    with pytest.raises(d.DeslocError) as e:
        d.desloc_plan_chunks([5, 0], ce)
    assert e.value.status == d.DESLOC_E_RANGE


def test_chunk_plan_cuts_first_chunks_at_2kb_boundaries(d):
    """With the addresses of worker 0's x tensors the plan shortens a tensor's first chunk so
    that all later ones start on a 2 KB boundary -- unless the tensor ends in front of it."""
    ce = 4096
    base = 0x7f0000000000                     # 2 KB aligned
    numel = [10_000, 10_000, 10_000, 10_000, 300, 10_000, 3 * ce + 512 - 64, 10_000, 10_000]
    addr = [base, base + 4 * 64, base + 4 * 504, base + 4 * 4, base + 4 * 448, base + 2048,
            base + 4 * 64, base + 4 * 5, base + 4 * 510]
    total, chunks = d.desloc_plan_chunks(numel, ce, x0=addr)
    per = {k: [(s, c) for kk, s, c in chunks if kk == k] for k in range(len(numel))}
    assert per[0][0] == (0, ce)                            # on the boundary: nothing cut
    assert per[1][0] == (0, 448) and per[1][1] == (448, ce)
    assert per[2][0] == (0, 8) and per[2][1] == (8, ce)
    assert per[3][0] == (0, 508) and per[3][1] == (508, ce)   # an odd multiple of four elements
    assert per[7][0] == (0, 507) and per[7][1] == (507, ce)   # an odd offset of a packed buffer
    assert per[8][0] == (0, 2) and per[8][1] == (2, ce)
    assert per[4] == [(0, 64), (64, 236)]                  # short tensor that crosses the boundary
    assert per[5][0] == (0, ce)
    assert per[6] == [(0, 448), (448, ce), (448 + ce, ce), (448 + 2 * ce, ce)]
    for k, lst in per.items():
        pos = 0
        for s, c in lst:
            assert s == pos and c >= 1
            pos += c
            if s > 0:
                assert (addr[k] + 4 * s) % 2048 == 0
        assert pos == numel[k]
    assert total == len(chunks)
    # a tensor that ends in front of the boundary stays whole
    assert d.desloc_plan_chunks([60], ce, x0=[base + 4 * 448])[1] == [(0, 0, 60)]
    # no addresses: the plain plan
    assert d.desloc_plan_chunks(numel, ce)[1] == d.desloc_plan_chunks(numel, ce, x0=[base] * len(numel))[1]


def test_chunk_plan_at_random_addresses_covers_every_element_once(d):
    """Seeded sweep over tensor lists and addresses (any 4-byte alignment): every element of
    every tensor lies in exactly one chunk, chunks of a tensor are contiguous and in order, only
    the first and the last are short, and the later ones start on 2 KB boundaries."""
    rng = np.random.default_rng(2505)
    for trial in range(200):
        nt = int(rng.integers(1, 12))
        ce = int(rng.choice([512, 1024, 4096, 8192]))
        numel = [int(rng.choice([1, 7, 500, 511, 512, 513, 4096, 9000, 40_000])) + int(rng.integers(0, 3))
                 for _ in range(nt)]
        addr = [0x7f0000000000 + 4 * int(rng.integers(0, 4096)) for _ in range(nt)]
        total, chunks = d.desloc_plan_chunks(numel, ce, x0=addr)
        assert total == len(chunks)
        pos = [0] * nt
        first = [True] * nt
        last_k = -1
        for k, s0, c in chunks:
            assert k >= last_k                   # tensors in order
            last_k = k
            assert s0 == pos[k] and 1 <= c <= ce
            left = numel[k] - s0
            if first[k]:
                cut = (512 - (addr[k] // 4) % 512) % 512
                leaves_alone = cut == 0 or cut >= numel[k]
                assert c == (min(ce, left) if leaves_alone else cut)
            else:
                assert c == min(ce, left)
                assert (addr[k] + 4 * s0) % 2048 == 0
            first[k] = False
            pos[k] += c
        assert pos == numel


def test_workload_sizes_match_the_stated_totals():
    assert di.WORKLOADS["cfg2_adam_135m"].N == 134_515_008
    assert di.WORKLOADS["cfg3_adopt_360m"].N == 361_821_120
    assert di.WORKLOADS["cfg4_adam_1p7b"].N == 1_711_376_384
    assert len(di.WORKLOADS["cfg4_adam_1p7b"].numel) == 218


BAD = [
    (dict(M=0), "DESLOC_E_RANGE"), (dict(M=257), "DESLOC_E_RANGE"),
    (dict(Kx=-1), "DESLOC_E_RANGE"), (dict(beta1=1.0), "DESLOC_E_RANGE"),
    (dict(beta2=-0.1), "DESLOC_E_RANGE"), (dict(beta1=float("nan")), "DESLOC_E_RANGE"),
    (dict(eps=-1.0), "DESLOC_E_RANGE"), (dict(weight_decay=-1.0), "DESLOC_E_RANGE"),
    (dict(opt=3), "DESLOC_E_INVALID"), (dict(grad_dtype=2), "DESLOC_E_INVALID"),
    (dict(flags=4), "DESLOC_E_INVALID"), (dict(flags=1), "DESLOC_E_INVALID"),  # norm clip w/o ADOPT
    (dict(numel=[4, 0]), "DESLOC_E_RANGE"),
]


@pytest.mark.parametrize("kw,status", BAD)
def test_create_rejects_bad_config_before_touching_the_device(d, kw, status):
    args = dict(M=2, numel=[4, 4], opt="adam", grad_dtype="f32")
    args.update(kw)
    cfg = d.make_config(**args)
    n = max(1, cfg.M) * len(args["numel"])
    with pytest.raises(d.DeslocError) as e:
        d.desloc_create(cfg, [16] * n, [16] * n, [16] * n, 0)
    assert e.value.status == getattr(d, status)


def test_create_rejects_null_pointers(d):
    cfg = d.make_config(2, [4], "adam", "f32")
    for x, u, v in [([16, 0], [16, 16], [16, 16]), ([16, 16], None, [16, 16]),
                    ([16, 16], [16, 16], None), ([16, 16], [16, 16], [0, 16])]:
        with pytest.raises(d.DeslocError) as e:
            d.desloc_create(cfg, x, u, v, 0)
        assert e.value.status == d.DESLOC_E_NULL
    # SGDM needs no v
    cfg = d.make_config(2, [4], "sgdm", "f32")
    with pytest.raises(d.DeslocError) as e:
        d.desloc_create(cfg, [16, 16], [16, 16], None, -1)
    assert e.value.status == d.DESLOC_E_RANGE


def test_null_context_is_handled(d):
    L = d.raw_lib()
    assert L.desloc_destroy(None) == 0
    assert L.desloc_step(None, 0, 0.1, 0.0, None, None, None) == d.DESLOC_E_NULL
    assert L.desloc_get_counters(None, None) == d.DESLOC_E_NULL
    assert L.desloc_get_launch_count(None) == 0
    assert d.desloc_strerror(0) == "ok" and "unknown" in d.desloc_strerror(-99)


def test_no_cpu_fallback_without_a_device(d):
    """On a machine without a GPU a valid create must fail with a CUDA status, not fall back."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    cfg = d.make_config(1, [4], "adam", "f32")
    with pytest.raises(d.DeslocError) as e:
        d.desloc_create(cfg, [16], [16], [16], 0)
    assert e.value.status in (d.DESLOC_E_CUDA, d.DESLOC_E_NOMEM)


def test_diag_entry_points_reject_bad_arguments_without_a_device(d):
    L = d.raw_lib()
    assert L.desloc_step_diag(None, 0, 0.1, 0.0, 0.0, None, None, None) == d.DESLOC_E_NULL
    assert L.desloc_get_diag_norms(None, None, None, None) == d.DESLOC_E_NULL
    assert L.desloc_testing_set_max_blocks(None, 0) == d.DESLOC_E_NULL
    assert L.desloc_testing_set_staging(None, 0) == d.DESLOC_E_NULL


STATIC_BAD = [
    (dict(M=0), "DESLOC_E_RANGE"), (dict(M=9), "DESLOC_E_TOO_LARGE"), (dict(M=257), "DESLOC_E_RANGE"),
    (dict(beta1=1.0), "DESLOC_E_RANGE"), (dict(beta2=float("nan")), "DESLOC_E_RANGE"),
    (dict(eps=-1.0), "DESLOC_E_RANGE"), (dict(Kv=-2), "DESLOC_E_RANGE"),
    (dict(opt=7), "DESLOC_E_INVALID"), (dict(grad_dtype=5), "DESLOC_E_INVALID"),
    (dict(flags=8), "DESLOC_E_INVALID"), (dict(flags=1), "DESLOC_E_INVALID"),
    (dict(numel=[4, 0]), "DESLOC_E_RANGE"),
    (dict(numel=[1] * 1025), "DESLOC_E_TOO_LARGE"),                 # 2 x 1025 pointers
    (dict(M=1, numel=[32768 * 8192 + 1]), "DESLOC_E_TOO_LARGE"),    # one chunk too many
    (dict(M=4, numel=[32768 * 4096 + 1]), "DESLOC_E_TOO_LARGE"),
]


@pytest.mark.parametrize("kw,status", STATIC_BAD)
def test_static_entry_point_rejects_bad_arguments_before_any_cuda_call(d, kw, status):
    """desloc_step_static() validates everything first: these calls must return their status on
    a machine with no GPU at all (nothing may reach the CUDA runtime)."""
    args = dict(M=2, numel=[4, 4], opt="adam", grad_dtype="f32")
    args.update(kw)
    cfg = d.make_config(**args)
    n = max(1, cfg.M) * len(args["numel"])
    with pytest.raises(d.DeslocError) as e:
        d.desloc_step_static(cfg, [16] * n, [16] * n, [16] * n, [16] * n, 0, 1e-3, 0.0, 0)
    assert e.value.status == getattr(d, status)


def test_static_entry_point_rejects_nulls_and_bad_step_arguments(d):
    cfg = d.make_config(2, [4], "adam", "f32")
    ok = [16, 16]
    for x, u, v, g in [(None, ok, ok, ok), (ok, None, ok, ok), (ok, ok, None, ok), (ok, ok, ok, None),
                       ([16, 0], ok, ok, ok), (ok, ok, [0, 16], ok), (ok, ok, ok, [16, 0])]:
        with pytest.raises(d.DeslocError) as e:
            d.desloc_step_static(cfg, x, u, v, g, 0, 1e-3, 0.0, 0)
        assert e.value.status == d.DESLOC_E_NULL
    for t, lr, dev in [(-1, 1e-3, 0), (0, float("inf"), 0), (0, 1e-3, -1), (0, 1e-3, 64)]:
        with pytest.raises(d.DeslocError) as e:
            d.desloc_step_static(cfg, ok, ok, ok, ok, t, lr, 0.0, dev)
        assert e.value.status == d.DESLOC_E_RANGE
    assert d.raw_lib().desloc_step_static(None, None, None, None, None, 0, 0.1, 0.0, 0, None, None) \
        == d.DESLOC_E_NULL
    # the ADOPT bound must be a number >= 0 when its flag is set
    cfg = d.make_config(2, [4], "adopt", "f32", flags=d.DESLOC_FLAG_ADOPT_NORM_CLIP)
    with pytest.raises(d.DeslocError) as e:
        d.desloc_step_static(cfg, ok, ok, ok, ok, 0, 1e-3, float("nan"), 0)
    assert e.value.status == d.DESLOC_E_RANGE
