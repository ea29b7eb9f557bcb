"""``DesLoc``: owns nothing but a context handle; holds references to the caller's tensors."""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as B


class BoundGrads:
    """Gradient tensors already checked and marshalled (see DesLoc.bind_grads)."""

    def __init__(self, array, keep):
        self.array, self._keep = array, keep


class DesLoc:
    """M worker replicas of a tensor list, stepped by the CUDA library.

    x, u, v: lists (one per worker) of lists of CUDA fp32 tensors (one per model tensor),
    updated in place by :meth:`step`.  v is None for SGDM.
    """

    def __init__(self, x: Sequence[Sequence[torch.Tensor]], u, v, *, opt, grad_dtype,
                 beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, clip_rho=0.0,
                 K=(1, 1, 1), flags=0):
        M = len(x)
        numel = [int(t.numel()) for t in x[0]]
        dev = x[0][0].device
        if dev.type != "cuda":
            raise ValueError("DesLoc needs CUDA tensors (there is no CPU path)")
        for arrs in (x, u) + ((v,) if v is not None else ()):
            if len(arrs) != M:
                raise ValueError("x, u, v need one tensor list per worker")
            for lst in arrs:
                if [int(t.numel()) for t in lst] != numel:
                    raise ValueError("every worker needs the same tensor list")
                for t in lst:
                    if t.dtype != torch.float32 or not t.is_contiguous() or t.device != dev:
                        raise ValueError("state tensors must be contiguous fp32 on one device")
        self._keep = (x, u, v)
        self.M, self.numel, self.device = M, numel, dev
        self.grad_dtype = B.DTYPE_BY_NAME.get(grad_dtype, grad_dtype)
        self.cfg = B.make_config(M, numel, opt, grad_dtype, beta1, beta2, eps, weight_decay,
                                 clip_rho, K[0], K[1], K[2], flags)
        flat = lambda a: [t.data_ptr() for lst in a for t in lst]
        self.ctx: Optional[int] = B.desloc_create(
            self.cfg, flat(x), flat(u), flat(v) if v is not None else None,
            dev.index if dev.index is not None else torch.cuda.current_device())
        self._gkey = None
        self._garr = None

    def bind_grads(self, grads: Sequence[Sequence[torch.Tensor]]):
        """Check a set of gradient tensors once and return a handle every step method accepts in
        place of the nested lists: a loop that reuses its gradient buffers then pays no
        per-step marshalling.  The handle keeps the tensors alive."""
        return BoundGrads(self._grad_array(grads), grads)

    def _grad_array(self, grads):
        if isinstance(grads, BoundGrads):
            return grads.array
        want = torch.bfloat16 if self.grad_dtype == B.DESLOC_BF16 else torch.float32
        ptrs: List[int] = []
        for lst in grads:
            for t, n in zip(lst, self.numel):
                if t.dtype != want or t.numel() != n or not t.is_contiguous():
                    raise ValueError("gradient tensor of wrong dtype, size or layout")
                ptrs.append(t.data_ptr())
        if len(ptrs) != self.M * len(self.numel):
            raise ValueError("need one gradient list per worker")
        key = tuple(ptrs)
        if key != self._gkey:
            self._gkey, self._garr = key, B.ptr_array(ptrs)
        return self._garr

    def step(self, t: int, lr: float, grads, clip_bound: float = 0.0) -> int:
        """Step t on torch's current stream; returns the sync mask."""
        stream = torch.cuda.current_stream(self.device).cuda_stream
        return B.desloc_step(self.ctx, t, lr, clip_bound, self._grad_array(grads), stream)

    def step_normclip(self, t: int, lr: float, grads, max_norm: float, clip_bound: float = 0.0) -> int:
        """Step t with norm-based gradient clipping (per worker, over the whole tensor list)."""
        stream = torch.cuda.current_stream(self.device).cuda_stream
        return B.desloc_step_normclip(self.ctx, t, lr, clip_bound, max_norm,
                                      self._grad_array(grads), stream)

    def step_diag(self, t: int, lr: float, grads, max_norm: float = 0.0, clip_bound: float = 0.0) -> int:
        """Step t that also accumulates the gradient, parameter and update norms (read them with
        diag_norms()); max_norm > 0 adds norm-based clipping in front."""
        stream = torch.cuda.current_stream(self.device).cuda_stream
        return B.desloc_step_diag(self.ctx, t, lr, clip_bound, max_norm, self._grad_array(grads),
                                  stream)

    def diag_norms(self):
        """(per_tensor [3][M][num_tensors], total [3][M]) of the latest step_diag; kind 0 =
        gradient as read, 1 = new parameters, 2 = update d_t.  Synchronises the current stream."""
        stream = torch.cuda.current_stream(self.device).cuda_stream
        return B.desloc_get_diag_norms(self.ctx, self.M, len(self.numel), stream)

    def grad_norms(self):
        """(norms, clip factors) of the latest step_normclip; synchronises the current stream."""
        stream = torch.cuda.current_stream(self.device).cuda_stream
        return B.desloc_get_grad_norms(self.ctx, self.M, stream)

    def rel_change(self, array: int, then: Sequence[Sequence[torch.Tensor]]):
        """Per-worker ||s - then|| / ||then|| against a snapshot (lists like x); synchronises."""
        ptrs = []
        for lst in then:
            for t, n in zip(lst, self.numel):
                if t.dtype != torch.float32 or t.numel() != n or not t.is_contiguous():
                    raise ValueError("snapshot tensor of wrong dtype, size or layout")
                ptrs.append(t.data_ptr())
        stream = torch.cuda.current_stream(self.device).cuda_stream
        return B.desloc_rel_change(self.ctx, array, ptrs, self.M, stream)

    def set_workers(self, x, u, v, first_new: int) -> None:
        """New worker set (lists like the constructor's); workers first_new.. start from the mean
        of the current workers.  Synchronises the current stream."""
        M = len(x)
        for arrs in (x, u) + ((v,) if v is not None else ()):
            if len(arrs) != M or any([int(t.numel()) for t in lst] != self.numel for lst in arrs):
                raise ValueError("every worker needs the same tensor list")
        flat = lambda a: [t.data_ptr() for lst in a for t in lst]
        stream = torch.cuda.current_stream(self.device).cuda_stream
        B.desloc_set_workers(self.ctx, M, first_new, flat(x), flat(u),
                             flat(v) if v is not None else None, stream)
        self._keep = (x, u, v)
        self.M = M
        self._gkey = self._garr = None

    def step_host(self, t: int, lr: float, host_grads, dev_grads, clip_bound: float = 0.0) -> int:
        """Step t with gradients in (pinned) host tensors; dev_grads are device staging tensors."""
        want = torch.bfloat16 if self.grad_dtype == B.DESLOC_BF16 else torch.float32
        hp = []
        for lst in host_grads:
            for t_, n in zip(lst, self.numel):
                if t_.dtype != want or t_.numel() != n or not t_.is_contiguous() or t_.is_cuda:
                    raise ValueError("host gradient tensor of wrong dtype, size, layout or device")
                hp.append(t_.data_ptr())
        stream = torch.cuda.current_stream(self.device).cuda_stream
        return B.desloc_step_host(self.ctx, t, lr, clip_bound, hp, self._grad_array(dev_grads),
                                  stream)

    def step_masked(self, mask: int, lr: float, grads, clip_bound: float = 0.0) -> None:
        stream = torch.cuda.current_stream(self.device).cuda_stream
        B.desloc_step_masked(self.ctx, mask, lr, clip_bound, self._grad_array(grads), stream)

    def counters(self):
        return B.desloc_get_counters(self.ctx)

    def launches(self) -> int:
        return B.desloc_get_launch_count(self.ctx)

    def close(self) -> None:
        if self.ctx is not None:
            B.desloc_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
