"""ctypes binding of libdesloc.so: the functions of include/desloc.h under the same names.

Argument marshalling only -- every step of the DES-LOC update runs in the CUDA kernels of
the library.  There is no fallback: if the library cannot be loaded, importing this module
raises.  Device pointers are plain integers (e.g. ``tensor.data_ptr()``); streams are the
integer ``cudaStream_t`` (e.g. ``torch.cuda.current_stream().cuda_stream``).
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libdesloc.so")

DESLOC_ADAM, DESLOC_ADOPT, DESLOC_SGDM = 0, 1, 2
DESLOC_F32, DESLOC_BF16 = 0, 1
DESLOC_SYNC_X, DESLOC_SYNC_U, DESLOC_SYNC_V = 1, 2, 4
DESLOC_FLAG_ADOPT_NORM_CLIP, DESLOC_FLAG_POST_AVERAGE = 1, 2
DESLOC_OK, DESLOC_E_NULL, DESLOC_E_RANGE, DESLOC_E_INVALID, DESLOC_E_NOMEM, DESLOC_E_CUDA = \
    0, -1, -2, -3, -4, -5
DESLOC_E_TOO_LARGE = -6
DESLOC_E_DEVICE_WAIT = -7
DESLOC_STATIC_MAX_POINTERS, DESLOC_STATIC_MAX_CHUNKS = 2048, 32768
DESLOC_MAX_M = 256

OPT_BY_NAME = {"adam": DESLOC_ADAM, "adopt": DESLOC_ADOPT, "sgdm": DESLOC_SGDM}
DTYPE_BY_NAME = {"f32": DESLOC_F32, "bf16": DESLOC_BF16}


class DeslocConfig(ctypes.Structure):
    """Mirror of ``desloc_config``."""
    _fields_ = [
        ("M", ctypes.c_int32),
        ("num_tensors", ctypes.c_int32),
        ("numel", ctypes.POINTER(ctypes.c_int64)),
        ("opt", ctypes.c_int32),
        ("grad_dtype", ctypes.c_int32),
        ("beta1", ctypes.c_float),
        ("beta2", ctypes.c_float),
        ("eps", ctypes.c_float),
        ("weight_decay", ctypes.c_float),
        ("clip_rho", ctypes.c_float),
        ("Kx", ctypes.c_int32),
        ("Ku", ctypes.c_int32),
        ("Kv", ctypes.c_int32),
        ("flags", ctypes.c_uint32),
    ]


class DeslocError(RuntimeError):
    def __init__(self, status: int, where: str, cuda_error: int = 0):
        self.status = status
        self.cuda_error = cuda_error
        msg = f"{where}: {desloc_strerror(status)} (status {status}"
        msg += f", cudaError {cuda_error})" if cuda_error else ")"
        super().__init__(msg)


if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2505_22549_b200.build` "
        "(there is no CPU or PyTorch fallback for the DES-LOC step)")
_lib = ctypes.CDLL(LIB_PATH)

_P = ctypes.c_void_p
_PP = ctypes.POINTER(ctypes.c_void_p)
_lib.desloc_sync_mask.restype = ctypes.c_uint32
_lib.desloc_sync_mask.argtypes = [ctypes.POINTER(DeslocConfig), ctypes.c_int64]
_lib.desloc_create.restype = ctypes.c_int
_lib.desloc_create.argtypes = [ctypes.POINTER(_P), ctypes.POINTER(DeslocConfig), _PP, _PP, _PP,
                               ctypes.c_int]
_lib.desloc_step.restype = ctypes.c_int
_lib.desloc_step.argtypes = [_P, ctypes.c_int64, ctypes.c_float, ctypes.c_float, _PP, _P,
                             ctypes.POINTER(ctypes.c_uint32)]
_lib.desloc_step_host.restype = ctypes.c_int
_lib.desloc_step_host.argtypes = [_P, ctypes.c_int64, ctypes.c_float, ctypes.c_float, _PP, _PP, _P,
                                  ctypes.POINTER(ctypes.c_uint32)]
_lib.desloc_step_masked.restype = ctypes.c_int
_lib.desloc_step_masked.argtypes = [_P, ctypes.c_uint32, ctypes.c_float, ctypes.c_float, _PP, _P]
_lib.desloc_destroy.restype = ctypes.c_int
_lib.desloc_destroy.argtypes = [_P]
_lib.desloc_set_workers.restype = ctypes.c_int
_lib.desloc_set_workers.argtypes = [_P, ctypes.c_int32, ctypes.c_int32, _PP, _PP, _PP, _P]
_lib.desloc_step_normclip.restype = ctypes.c_int
_lib.desloc_step_normclip.argtypes = [_P, ctypes.c_int64, ctypes.c_float, ctypes.c_float,
                                      ctypes.c_float, _PP, _P, ctypes.POINTER(ctypes.c_uint32)]
_lib.desloc_get_grad_norms.restype = ctypes.c_int
_lib.desloc_get_grad_norms.argtypes = [_P, ctypes.POINTER(ctypes.c_float),
                                       ctypes.POINTER(ctypes.c_float), _P]
_lib.desloc_rel_change.restype = ctypes.c_int
_lib.desloc_rel_change.argtypes = [_P, ctypes.c_int32, _PP, ctypes.POINTER(ctypes.c_float), _P]
_lib.desloc_step_static.restype = ctypes.c_int
_lib.desloc_step_static.argtypes = [ctypes.POINTER(DeslocConfig), _PP, _PP, _PP, _PP,
                                    ctypes.c_int64, ctypes.c_float, ctypes.c_float, ctypes.c_int,
                                    _P, ctypes.POINTER(ctypes.c_uint32)]
_lib.desloc_get_counters.restype = ctypes.c_int
_lib.desloc_get_counters.argtypes = [_P, ctypes.POINTER(ctypes.c_int64)]
_lib.desloc_get_launch_count.restype = ctypes.c_int64
_lib.desloc_get_launch_count.argtypes = [_P]
_lib.desloc_step_diag.restype = ctypes.c_int
_lib.desloc_step_diag.argtypes = [_P, ctypes.c_int64, ctypes.c_float, ctypes.c_float,
                                  ctypes.c_float, _PP, _P, ctypes.POINTER(ctypes.c_uint32)]
_lib.desloc_get_diag_norms.restype = ctypes.c_int
_lib.desloc_get_diag_norms.argtypes = [_P, ctypes.POINTER(ctypes.c_float),
                                       ctypes.POINTER(ctypes.c_float), _P]
_lib.desloc_testing_set_max_blocks.restype = ctypes.c_int
_lib.desloc_testing_set_max_blocks.argtypes = [_P, ctypes.c_int64]
_lib.desloc_testing_set_staging.restype = ctypes.c_int
_lib.desloc_testing_set_staging.argtypes = [_P, ctypes.c_int32]
_lib.desloc_testing_set_wait_limit.restype = ctypes.c_int
_lib.desloc_testing_set_wait_limit.argtypes = [_P, ctypes.c_int32]
_lib.desloc_plan_chunks.restype = ctypes.c_int64
_lib.desloc_plan_chunks.argtypes = [ctypes.POINTER(ctypes.c_int64), ctypes.c_int32,
                                    ctypes.c_int64, ctypes.POINTER(ctypes.c_int64),
                                    ctypes.c_int64]
_lib.desloc_plan_chunks_at.restype = ctypes.c_int64
_lib.desloc_plan_chunks_at.argtypes = [ctypes.POINTER(ctypes.c_int64), ctypes.c_int32,
                                       ctypes.c_int64, ctypes.POINTER(ctypes.c_void_p),
                                       ctypes.POINTER(ctypes.c_int64), ctypes.c_int64]
_lib.desloc_chunk_elems.restype = ctypes.c_int64
_lib.desloc_chunk_elems.argtypes = [ctypes.POINTER(DeslocConfig)]
_lib.desloc_strerror.restype = ctypes.c_char_p
_lib.desloc_strerror.argtypes = [ctypes.c_int]
_lib.desloc_last_cuda_error.restype = ctypes.c_int
_lib.desloc_last_cuda_error.argtypes = [_P]


def raw_lib() -> ctypes.CDLL:
    """The loaded shared library (for tests that check the exported symbols)."""
    return _lib


def make_config(M: int, numel: Sequence[int], opt, grad_dtype, beta1=0.9, beta2=0.999, eps=1e-8,
                weight_decay=0.0, clip_rho=0.0, Kx=1, Ku=1, Kv=1, flags=0) -> DeslocConfig:
    """Fill a ``desloc_config``.  The numel array is kept alive on the returned object."""
    opt = OPT_BY_NAME.get(opt, opt)
    grad_dtype = DTYPE_BY_NAME.get(grad_dtype, grad_dtype)
    arr = (ctypes.c_int64 * len(numel))(*[int(n) for n in numel])
    cfg = DeslocConfig(int(M), len(numel), ctypes.cast(arr, ctypes.POINTER(ctypes.c_int64)),
                       int(opt), int(grad_dtype), float(beta1), float(beta2), float(eps),
                       float(weight_decay), float(clip_rho), int(Kx), int(Ku), int(Kv), int(flags))
    cfg._numel_keepalive = arr
    return cfg


def _ptr_array(ptrs: Optional[Sequence[int]]):
    if ptrs is None:
        return None
    return (ctypes.c_void_p * len(ptrs))(*[int(p) if p else None for p in ptrs])


def desloc_strerror(status: int) -> str:
    return _lib.desloc_strerror(int(status)).decode()


def desloc_sync_mask(cfg: DeslocConfig, t: int) -> int:
    return int(_lib.desloc_sync_mask(ctypes.byref(cfg) if cfg is not None else None, int(t)))


def desloc_create(cfg: DeslocConfig, x: Sequence[int], u: Sequence[int],
                  v: Optional[Sequence[int]], cuda_device: int) -> int:
    """Returns the context handle (an integer); raises DeslocError on failure."""
    handle = ctypes.c_void_p()
    rc = _lib.desloc_create(ctypes.byref(handle), ctypes.byref(cfg) if cfg is not None else None,
                            _ptr_array(x), _ptr_array(u), _ptr_array(v), int(cuda_device))
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_create")
    return handle.value


def desloc_step(ctx: int, t: int, lr_t: float, clip_bound_t: float, grads, stream: int = 0) -> int:
    """One step; returns the sync mask applied.  `grads` is a sequence of device pointers or a
    ready ctypes pointer array (see ptr_array) to skip re-marshalling in a hot loop."""
    g = grads if isinstance(grads, ctypes.Array) else _ptr_array(grads)
    mask = ctypes.c_uint32(0)
    rc = _lib.desloc_step(ctx, int(t), float(lr_t), float(clip_bound_t), g, stream or None,
                          ctypes.byref(mask))
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_step", _lib.desloc_last_cuda_error(ctx))
    return int(mask.value)


def desloc_step_host(ctx: int, t: int, lr_t: float, clip_bound_t: float, host_grads, dev_grads,
                     stream: int = 0) -> int:
    """desloc_step() with gradients in host memory: copies them into the device staging buffers
    `dev_grads` group by group and pipelines the step behind the copies.  Returns the mask."""
    hg = host_grads if isinstance(host_grads, ctypes.Array) else _ptr_array(host_grads)
    dg = dev_grads if isinstance(dev_grads, ctypes.Array) else _ptr_array(dev_grads)
    mask = ctypes.c_uint32(0)
    rc = _lib.desloc_step_host(ctx, int(t), float(lr_t), float(clip_bound_t), hg, dg,
                               stream or None, ctypes.byref(mask))
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_step_host", _lib.desloc_last_cuda_error(ctx))
    return int(mask.value)


def desloc_step_masked(ctx: int, mask: int, lr_t: float, clip_bound_t: float, grads,
                       stream: int = 0) -> None:
    g = grads if isinstance(grads, ctypes.Array) else _ptr_array(grads)
    rc = _lib.desloc_step_masked(ctx, int(mask), float(lr_t), float(clip_bound_t), g,
                                 stream or None)
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_step_masked", _lib.desloc_last_cuda_error(ctx))


def desloc_step_static(cfg: DeslocConfig, x, u, v, grads, t: int, lr_t: float,
                       clip_bound_t: float, cuda_device: int, stream: int = 0) -> int:
    """One step with no context and no allocation (tables go to the library's fixed device
    array).  x, u, v, grads: sequences of device pointers, entry m*num_tensors + k.  Returns
    the sync mask; raises DeslocError (DESLOC_E_TOO_LARGE beyond the fixed capacity).  Calls
    that may overlap on the GPU must be serialised by the caller."""
    mask = ctypes.c_uint32(0)
    as_arr = lambda a: a if isinstance(a, ctypes.Array) else _ptr_array(a)
    rc = _lib.desloc_step_static(ctypes.byref(cfg) if cfg is not None else None, as_arr(x),
                                 as_arr(u), as_arr(v), as_arr(grads), int(t), float(lr_t),
                                 float(clip_bound_t), int(cuda_device), stream or None,
                                 ctypes.byref(mask))
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_step_static")
    return int(mask.value)


def desloc_step_normclip(ctx: int, t: int, lr_t: float, clip_bound_t: float, max_norm: float,
                         grads, stream: int = 0) -> int:
    """One step with norm-based gradient clipping in front; returns the sync mask."""
    g = grads if isinstance(grads, ctypes.Array) else _ptr_array(grads)
    mask = ctypes.c_uint32(0)
    rc = _lib.desloc_step_normclip(ctx, int(t), float(lr_t), float(clip_bound_t), float(max_norm),
                                   g, stream or None, ctypes.byref(mask))
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_step_normclip", _lib.desloc_last_cuda_error(ctx))
    return int(mask.value)


def desloc_step_diag(ctx: int, t: int, lr_t: float, clip_bound_t: float, max_norm: float,
                     grads, stream: int = 0) -> int:
    """One step that also accumulates the gradient / parameter / update norms (max_norm > 0 adds
    norm-based clipping in front, 0 = off); returns the sync mask."""
    g = grads if isinstance(grads, ctypes.Array) else _ptr_array(grads)
    mask = ctypes.c_uint32(0)
    rc = _lib.desloc_step_diag(ctx, int(t), float(lr_t), float(clip_bound_t), float(max_norm), g,
                               stream or None, ctypes.byref(mask))
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_step_diag", _lib.desloc_last_cuda_error(ctx))
    return int(mask.value)


def desloc_get_diag_norms(ctx: int, M: int, num_tensors: int, stream: int = 0):
    """Norms of the latest desloc_step_diag: (per_tensor, total) as nested lists indexed
    [kind][worker][tensor] and [kind][worker]; kind 0 = gradient, 1 = parameters, 2 = update."""
    per = (ctypes.c_float * (3 * M * num_tensors))()
    tot = (ctypes.c_float * (3 * M))()
    rc = _lib.desloc_get_diag_norms(ctx, per, tot, stream or None)
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_get_diag_norms", _lib.desloc_last_cuda_error(ctx))
    per_l = [[[per[(k * M + m) * num_tensors + j] for j in range(num_tensors)] for m in range(M)]
             for k in range(3)]
    tot_l = [[tot[k * M + m] for m in range(M)] for k in range(3)]
    return per_l, tot_l


def desloc_get_grad_norms(ctx: int, M: int, stream: int = 0):
    """(norms, clip factors) of the latest desloc_step_normclip as two lists of M floats."""
    norms, scales = (ctypes.c_float * M)(), (ctypes.c_float * M)()
    rc = _lib.desloc_get_grad_norms(ctx, norms, scales, stream or None)
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_get_grad_norms", _lib.desloc_last_cuda_error(ctx))
    return list(norms), list(scales)


def desloc_rel_change(ctx: int, array: int, then: Sequence[int], M: int, stream: int = 0):
    """Per-worker ||s - then|| / ||then|| for array 0 = x, 1 = u, 2 = v; `then` are device pointers."""
    out = (ctypes.c_float * M)()
    rc = _lib.desloc_rel_change(ctx, int(array), _ptr_array(then), out, stream or None)
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_rel_change", _lib.desloc_last_cuda_error(ctx))
    return list(out)


def desloc_set_workers(ctx: int, M_new: int, first_new: int, x, u, v, stream: int = 0) -> None:
    """Replace the worker set; workers first_new.. are filled with the mean of the old workers."""
    rc = _lib.desloc_set_workers(ctx, int(M_new), int(first_new), _ptr_array(x), _ptr_array(u),
                                 _ptr_array(v), stream or None)
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_set_workers", _lib.desloc_last_cuda_error(ctx))


def desloc_destroy(ctx: Optional[int]) -> None:
    rc = _lib.desloc_destroy(ctx)
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_destroy")


def desloc_get_counters(ctx: int):
    out = (ctypes.c_int64 * 4)()
    rc = _lib.desloc_get_counters(ctx, out)
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_get_counters")
    return [int(a) for a in out]


def desloc_get_launch_count(ctx: int) -> int:
    return int(_lib.desloc_get_launch_count(ctx))


def desloc_testing_set_max_blocks(ctx: int, max_blocks: int) -> None:
    """Test hook (include/desloc_testing.h): cap the step kernels' grid so that blocks stride."""
    rc = _lib.desloc_testing_set_max_blocks(ctx, int(max_blocks))
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_testing_set_max_blocks")


def desloc_chunk_elems(cfg: DeslocConfig) -> int:
    """Elements per chunk (the run of tiles one thread block streams) of a context made from cfg."""
    n = int(_lib.desloc_chunk_elems(ctypes.byref(cfg) if cfg is not None else None))
    if n < 0:
        raise DeslocError(n, "desloc_chunk_elems")
    return n


def desloc_testing_set_staging(ctx: int, mode: int) -> None:
    """Test hook (include/desloc_testing.h): -1 the library decides, 0 always stage, 1 never."""
    rc = _lib.desloc_testing_set_staging(ctx, int(mode))
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_testing_set_staging")


def desloc_testing_set_wait_limit(ctx: int, polls: int) -> None:
    """Test hook (include/desloc_testing.h): bound on a block's wait for its tile; negative =
    default, and clears a recorded failure."""
    rc = _lib.desloc_testing_set_wait_limit(ctx, int(polls))
    if rc != DESLOC_OK:
        raise DeslocError(rc, "desloc_testing_set_wait_limit")


def desloc_plan_chunks(numel: Sequence[int], chunk_elems: int, cap: Optional[int] = None,
                       x0: Optional[Sequence[int]] = None):
    """Returns (total_chunks, [(tensor, start, count), ...] up to cap).  x0: the addresses of
    worker 0's x tensors (desloc_plan_chunks_at: first chunks cut at 2 KB boundaries) or None."""
    arr = (ctypes.c_int64 * max(1, len(numel)))(*[int(n) for n in numel])
    xs = None
    if x0 is not None:
        if len(x0) != len(numel):
            raise ValueError("x0 must hold one address per tensor")
        xs = (ctypes.c_void_p * max(1, len(x0)))(*[int(p) for p in x0])
    total = _lib.desloc_plan_chunks_at(arr, len(numel), int(chunk_elems), xs, None, 0)
    if total < 0:
        raise DeslocError(int(total), "desloc_plan_chunks")
    cap = total if cap is None else min(cap, total)
    out = (ctypes.c_int64 * max(1, 3 * cap))()
    if x0 is None:
        total2 = _lib.desloc_plan_chunks(arr, len(numel), int(chunk_elems), out, cap)
    else:
        total2 = _lib.desloc_plan_chunks_at(arr, len(numel), int(chunk_elems), xs, out, cap)
    assert total2 == total
    return int(total), [(int(out[3 * i]), int(out[3 * i + 1]), int(out[3 * i + 2]))
                        for i in range(cap)]


def ptr_array(ptrs: Sequence[int]):
    """A reusable ctypes array of device pointers for desloc_step()."""
    return _ptr_array(ptrs)


def desloc_last_cuda_error(ctx: int) -> int:
    return int(_lib.desloc_last_cuda_error(ctx))
