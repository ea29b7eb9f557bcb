"""Seeded synthetic inputs for DES-LOC: tensor lists, initial parameters, gradients.

This module serves both the CUDA library's tests/benchmark and the CPU oracle's
tests.  It holds data recipes only -- shapes, seeds, value distributions and
which elements to sample -- and none of the optimizer's arithmetic.

Workloads stand in for the paper's language-model training runs (GPT-style
models of 135M and 1.7B parameters, model table in the experimental-details
appendix): the training corpus and the trained weights are not available, so
parameters are drawn N(0, 0.02) and gradients from the distributions each
workload names.
"""
from __future__ import annotations

import dataclasses
from typing import List, Sequence, Tuple

import numpy as np
import torch

_MASK64 = (1 << 64) - 1


def _mix(*vals: int) -> int:
    """splitmix64-style integer hash of a tuple of ints -> 63-bit seed."""
    h = 0x9E3779B97F4A7C15
    for v in vals:
        h = (h ^ (int(v) & _MASK64)) & _MASK64
        h = (h * 0xBF58476D1CE4E5B9) & _MASK64
        h ^= h >> 31
        h = (h * 0x94D049BB133111EB) & _MASK64
        h ^= h >> 29
    return h & ((1 << 63) - 1)


def llama_tensor_list(layers: int, d: int, d_kv: int, ffn: int, vocab: int) -> List[int]:
    """Element counts of a Llama-style model, embedding first, tied output head.

    Per block: q[d,d] k[d,d_kv] v[d,d_kv] o[d,d] gate[ffn,d] up[ffn,d] down[d,ffn]
    and two norm vectors [d]; then one final norm [d].
    """
    out = [vocab * d]
    for _ in range(layers):
        out += [d * d, d * d_kv, d * d_kv, d * d, ffn * d, ffn * d, d * ffn, d, d]
    out.append(d)
    return out


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    opt: str                    # "adam" | "adopt" | "sgdm"
    M: int
    numel: Tuple[int, ...]
    grad_dtype: str             # "f32" | "bf16"
    grad_kind: str              # "normal1" | "normal_offset" | "student_t3"
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    lr: float = 1e-3
    weight_decay: float = 0.0
    clip_rho: float = 0.0
    K: Tuple[int, int, int] = (1, 1, 1)
    T: int = 1
    adopt_norm_clip: bool = False
    seed: int = 0

    @property
    def N(self) -> int:
        return int(sum(self.numel))

    def clip_bound(self, t: int) -> float:
        """Bound on ADOPT's normalised gradient at step t: t**0.25 (so 0 at t=0)."""
        return float(t) ** 0.25 if self.adopt_norm_clip else 0.0

    def replace(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _wl() -> dict:
    w = {}
    w["cfg1_adam_n4096"] = Workload(
        "cfg1_adam_n4096", "adam", 2, (4096,), "f32", "normal1", K=(4, 8, 16), T=64)
    w["cfg2_adam_135m"] = Workload(
        "cfg2_adam_135m", "adam", 4, tuple(llama_tensor_list(30, 576, 192, 1536, 49152)),
        "bf16", "normal_offset", K=(16, 32, 64), T=256)
    w["cfg3_adopt_360m"] = Workload(
        "cfg3_adopt_360m", "adopt", 8, tuple(llama_tensor_list(32, 960, 320, 2560, 49152)),
        "bf16", "student_t3", beta2=0.9999, eps=1e-6, clip_rho=1.0, K=(32, 64, 128), T=256,
        adopt_norm_clip=True)
    w["cfg4_adam_1p7b"] = Workload(
        "cfg4_adam_1p7b", "adam", 4, tuple(llama_tensor_list(24, 2048, 2048, 8192, 49152)),
        "bf16", "normal_offset", weight_decay=0.1, K=(64, 128, 256), T=128)
    base5 = Workload(
        "cfg5", "adam", 8, tuple(llama_tensor_list(32, 960, 320, 2560, 49152)),
        "bf16", "student_t3", T=512)
    for opt in ("sgdm", "adam"):
        for tag, K in (("ddp", (1, 1, 1)), ("local", (16, 16, 16)), ("desloc", (16, 64, 256))):
            name = f"cfg5_{opt}_{tag}"
            w[name] = base5.replace(name=name, opt=opt, K=K)
    # Small stand-ins of workloads 4 and 3 for profiler captures: same optimizer, M, dtypes and
    # gradient recipe on a 6-block model (44 M parameters; 2.5 / 4.9 GB resident, well above
    # the 126 MB L2, small enough for a multi-pass capture).
    prof = tuple(llama_tensor_list(6, 768, 256, 2048, 8192))
    w["prof_adam_m4_44m"] = w["cfg4_adam_1p7b"].replace(name="prof_adam_m4_44m", numel=prof,
                                                        K=(4, 8, 16), T=16)
    w["prof_adopt_m8_44m"] = w["cfg3_adopt_360m"].replace(name="prof_adopt_m8_44m", numel=prof,
                                                          K=(4, 8, 16), T=16)
    # Sixteen workers (the runtime-M kernel on sync steps) on a 3-block model: 25 M parameters,
    # 5.7 GB resident; every step syncs all three arrays.
    w["prof_adam_m16_25m"] = w["cfg2_adam_135m"].replace(
        name="prof_adam_m16_25m", M=16, numel=tuple(llama_tensor_list(3, 768, 256, 2048, 8192)),
        K=(1, 1, 1), T=16)
    return w


WORKLOADS = _wl()


def mini(w: Workload, layers: int = 2, d: int = 72, d_kv: int = 24, ffn: int = 200,
         vocab: int = 1031, T: int | None = None) -> Workload:
    """Same recipe on a model small enough for the oracle to run in full.

    The defaults give tensors from 72 to ~74 K elements, several of them not a
    multiple of 4 or of a kernel tile (ragged tails), 21 tensors in all.
    """
    numel = tuple(llama_tensor_list(layers, d, d_kv, ffn, vocab))
    return w.replace(name=w.name + "_mini", numel=numel, T=T if T is not None else w.T)


def offsets_of(numel: Sequence[int], align: int = 1) -> List[int]:
    """Start of each tensor inside one flat per-worker buffer (each start rounded up to `align`)."""
    offs, pos = [], 0
    for n in numel:
        pos = -(-pos // align) * align
        offs.append(pos)
        pos += int(n)
    return offs


def flat_size(numel: Sequence[int], align: int = 1) -> int:
    offs = offsets_of(numel, align)
    return offs[-1] + int(numel[-1]) if numel else 0


def init_params(w: Workload, device="cpu", align: int = 1) -> torch.Tensor:
    """x_0 ~ N(0, 0.02) as one flat fp32 buffer (identical for every worker)."""
    n = flat_size(w.numel, align)
    gen = torch.Generator(device=device)
    gen.manual_seed(_mix(w.seed, 0x5EED, 1))
    x0 = torch.empty(n, dtype=torch.float32, device=device)
    _blocked_normal_(x0, gen)
    x0.mul_(0.02)
    return x0


def _blocked_normal_(out: torch.Tensor, gen: torch.Generator, block: int = 1 << 26) -> None:
    for s in range(0, out.numel(), block):
        out[s:s + block].normal_(generator=gen)


def fill_grads_(w: Workload, t: int, m: int, out: torch.Tensor, align: int = 1,
                identical_workers: bool = False) -> None:
    """Write worker m's step-t gradient into the flat buffer `out` (fp32 or bf16).

    normal1        N(0, 1) from host_normals(): the same bits on every host and library version
    normal_offset  N(0, sd 1e-3) plus one constant per (worker, tensor) drawn N(0, sd 1e-4)
    student_t3     1e-3 * z / sqrt((z1^2 + z2^2 + z3^2) / 3)
    With identical_workers every worker receives worker 0's stream.
    """
    dev = out.device
    mm = 0 if identical_workers else m
    if w.grad_kind == "normal1":
        # the small fp32 workloads draw from the generator defined in this module, on the host
        z = host_normals(out.numel(), w.seed, 0x6AAD, t, mm).astype(np.float32)
        out.copy_(torch.from_numpy(z).to(out.dtype))
        return
    gen = torch.Generator(device=dev)
    gen.manual_seed(_mix(w.seed, 0x6AAD, t, mm))
    n = out.numel()
    block = 1 << 26
    if w.grad_kind == "normal_offset":
        cg = torch.Generator(device="cpu")
        cg.manual_seed(_mix(w.seed, 0x0FF5, mm))
        mu = (torch.randn(len(w.numel), generator=cg, dtype=torch.float32) * 1e-4).tolist()
        offs = offsets_of(w.numel, align)
    for s in range(0, n, block):
        e = min(n, s + block)
        z = torch.empty(e - s, dtype=torch.float32, device=dev)
        z.normal_(generator=gen)
        if w.grad_kind == "normal1":
            pass
        elif w.grad_kind == "normal_offset":
            z.mul_(1e-3)
            for k, (o, cnt) in enumerate(zip(offs, w.numel)):
                lo, hi = max(o, s), min(o + cnt, e)
                if lo < hi:
                    z[lo - s:hi - s].add_(mu[k])
        elif w.grad_kind == "student_t3":
            chi = torch.zeros_like(z)
            tmp = torch.empty_like(z)
            for _ in range(3):
                tmp.normal_(generator=gen)
                chi.addcmul_(tmp, tmp)
            chi.div_(3.0).sqrt_()
            z.div_(chi).mul_(1e-3)
            del chi, tmp
        else:
            raise ValueError(w.grad_kind)
        out[s:e].copy_(z)
        del z


def host_normals(n: int, *key: int) -> np.ndarray:
    """n standard normals in fp64 from a generator defined entirely here (independent of any
    library's random stream): splitmix64 of (key, counter) -> two 53-bit uniforms -> Box-Muller.
    The same key always gives the same bits on every host."""
    base = np.uint64(_mix(0xB0C5, *key))
    pairs = (n + 1) // 2
    with np.errstate(over="ignore"):
        ctr = base + np.arange(2 * pairs, dtype=np.uint64) * np.uint64(0x9E3779B97F4A7C15)
        z = ctr
        z = (z ^ (z >> np.uint64(30))) * np.uint64(0xBF58476D1CE4E5B9)
        z = (z ^ (z >> np.uint64(27))) * np.uint64(0x94D049BB133111EB)
        z = z ^ (z >> np.uint64(31))
    unit = (z >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))
    u1 = 1.0 - unit[0::2]            # (0, 1]: the logarithm stays finite
    u2 = unit[1::2]
    r = np.sqrt(-2.0 * np.log(u1))
    out = np.empty(2 * pairs, dtype=np.float64)
    out[0::2] = r * np.cos(2.0 * np.pi * u2)
    out[1::2] = r * np.sin(2.0 * np.pi * u2)
    return out[:n]


def toy_rosenbrock_grads(x: np.ndarray, t: int, sigma: float = 1.5, seed: int = 0) -> np.ndarray:
    """Noisy gradients of the toy problem f = (1 - x1)^2 + 100 (x2 - x1^2)^2 at the iterates
    x [M, 2] (fp32): the exact gradient in fp64 plus sigma * N(0, 1) per worker and coordinate,
    rounded to fp32.  A workload recipe: none of the optimizer's arithmetic is in here."""
    x1, x2 = x[:, 0].astype(np.float64), x[:, 1].astype(np.float64)
    g = np.stack([-2.0 * (1.0 - x1) - 400.0 * x1 * (x2 - x1 * x1), 200.0 * (x2 - x1 * x1)], axis=1)
    noise = host_normals(g.size, seed, 0x7070, t).reshape(g.shape)
    return np.ascontiguousarray(g + sigma * noise, dtype=np.float32)


def sample_indices(numel: Sequence[int], n_hashed: int, seed: int = 0, edge: int = 64,
                   align: int = 1) -> np.ndarray:
    """Flat-buffer indices to check at scale: the first and last `edge` elements of every
    tensor plus `n_hashed` pseudo-random positions spread over all tensors; sorted, unique."""
    offs = offsets_of(numel, align)
    parts = []
    for o, cnt in zip(offs, numel):
        k = min(edge, cnt)
        parts.append(np.arange(o, o + k, dtype=np.int64))
        parts.append(np.arange(o + cnt - k, o + cnt, dtype=np.int64))
    total = int(sum(numel))
    if n_hashed > 0 and total > 0:
        rng = np.random.Generator(np.random.PCG64(_mix(seed, 0x1D5)))
        r = rng.integers(0, total, size=n_hashed, dtype=np.int64)
        cum = np.concatenate([[0], np.cumsum(np.asarray(numel, dtype=np.int64))])
        k = np.searchsorted(cum, r, side="right") - 1
        parts.append(np.asarray(offs, dtype=np.int64)[k] + (r - cum[k]))
    return np.unique(np.concatenate(parts))
