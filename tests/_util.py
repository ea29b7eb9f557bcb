"""Shared helpers of the GPU parity tests: state allocation, the two runners, the error metric."""
from __future__ import annotations

import numpy as np
import torch

import desloc_inputs as di
import oracle

OPT_ID = {"adam": oracle.ADAM, "adopt": oracle.ADOPT, "sgdm": oracle.SGDM}
TOL = 1e-5  # the stated bar: max relative error on fp32 x, u, v after T steps


def f32r(a: float) -> float:
    """A hyper-parameter as the library sees it: rounded to fp32 when it crosses the C ABI."""
    return float(np.float32(a))


def oracle_cfg(w: di.Workload, flags: int = 0):
    fl = flags
    if w.adopt_norm_clip:
        fl |= oracle.FLAG_ADOPT_NORM_CLIP
    return oracle.make_cfg(w.M, OPT_ID[w.opt], beta1=f32r(w.beta1), beta2=f32r(w.beta2),
                           eps=f32r(w.eps), weight_decay=f32r(w.weight_decay),
                           clip_rho=f32r(w.clip_rho), Kx=w.K[0], Ku=w.K[1], Kv=w.K[2], flags=fl)


class State:
    """Per-worker flat fp32 buffers x, u, v and gradient buffer g on `device`, plus per-tensor views."""

    def __init__(self, w: di.Workload, device, align: int = 4, byte_shift: int = 0,
                 v_init: float = 0.0, g_shift: int | None = None):
        self.w, self.device, self.align = w, device, align
        self.offs = di.offsets_of(w.numel, align)
        self.nflat = di.flat_size(w.numel, align)
        gdt = torch.bfloat16 if w.grad_dtype == "bf16" else torch.float32
        x0 = di.init_params(w, device=device, align=align)
        # byte_shift (in elements) moves every buffer off its natural alignment (g_shift: the
        # gradient buffers by another amount than the state)
        sh = byte_shift
        mk = lambda dt: torch.zeros(self.nflat + sh, dtype=dt, device=device)[sh:]
        gsh = byte_shift if g_shift is None else g_shift
        mkg = lambda dt: torch.zeros(self.nflat + gsh, dtype=dt, device=device)[gsh:]
        self.x = [mk(torch.float32) for _ in range(w.M)]
        self.u = [mk(torch.float32) for _ in range(w.M)]
        self.v = [mk(torch.float32) for _ in range(w.M)] if w.opt != "sgdm" else None
        self.g = [mkg(gdt) for _ in range(w.M)]
        self.v_init = v_init
        self.valid = None
        self.reset(x0)

    def reset(self, x0=None):
        """Back to the initial state, in the same buffers."""
        if x0 is None:
            x0 = di.init_params(self.w, device=self.device, align=self.align)
        for m in range(self.w.M):
            self.x[m].copy_(x0)
            self.u[m].zero_()
            if self.v is not None:
                self.v[m].fill_(self.v_init)

    def views(self, bufs):
        return [[b[o:o + n] for o, n in zip(self.offs, self.w.numel)] for b in bufs]

    def fill_grads(self, t: int, identical: bool = False):
        for m in range(self.w.M):
            di.fill_grads_(self.w, t, m, self.g[m], align=self.align, identical_workers=identical)

    def valid_mask(self) -> np.ndarray:
        if self.valid is None:
            v = np.zeros(self.nflat, dtype=bool)
            for o, n in zip(self.offs, self.w.numel):
                v[o:o + n] = True
            self.valid = v
        return self.valid

    def to_numpy(self, bufs, idx: torch.Tensor | None = None) -> np.ndarray:
        """[M, n] float32 host copy (optionally only the flat positions idx)."""
        rows = []
        for b in bufs:
            t = b if idx is None else b[idx]
            rows.append(t.float().cpu().numpy())
        return np.ascontiguousarray(np.stack(rows, axis=0), dtype=np.float32)


def rel_err(gpu: np.ndarray, ref: np.ndarray, rms: float | None = None) -> float:
    """max_i |gpu_i - ref_i| / max(|ref_i|, rms(ref)): elementwise relative error with the
    tensor's RMS as floor for elements that pass near zero."""
    ref64 = ref.astype(np.float64)
    if rms is None:
        rms = float(np.sqrt(np.mean(ref64 * ref64))) if ref.size else 0.0
    den = np.maximum(np.abs(ref64), max(rms, 1e-30))
    if ref.size == 0:
        return 0.0
    return float(np.max(np.abs(gpu.astype(np.float64) - ref64) / den))


TINY = 64   # tensors with fewer elements have no meaningful RMS of their own


def compare_per_tensor(st: State, gpu: np.ndarray, ref: np.ndarray, what: str, tol: float = TOL):
    """gpu/ref are [M, nflat]; checks every (worker, tensor) block against `tol`.

    The error of an element is taken relative to max(|ref|, rms of its tensor): the floor is
    there because elements pass through zero while their absolute error stays at the scale of
    the tensor.  The RMS of a tensor of a handful of elements is no such scale (for one element
    it is the element itself), so tensors below TINY elements take the RMS of the worker's whole
    array as floor."""
    worst = 0.0
    for m in range(gpu.shape[0]):
        whole = np.concatenate([ref[m, o:o + n] for o, n in zip(st.offs, st.w.numel)]).astype(np.float64)
        rms_all = float(np.sqrt(np.mean(whole * whole))) if whole.size else 0.0
        for k, (o, n) in enumerate(zip(st.offs, st.w.numel)):
            e = rel_err(gpu[m, o:o + n], ref[m, o:o + n], rms=None if n >= TINY else rms_all)
            worst = max(worst, e)
            assert e <= tol, f"{what}: worker {m} tensor {k} (numel {n}) rel err {e:.3e} > {tol}"
    return worst
