"""ctypes binding of libagzo.so: same names as include/agzo.h, argument marshalling only.

torch is used for device memory and streams; every step of the path runs in the library's
kernels.  There is no fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libagzo.so")

AGZO_OK = 0
AGZO_ERR_INVALID_ARG = 1
AGZO_ERR_UNSUPPORTED = 2
AGZO_ERR_CUDA = 3
AGZO_ERR_WORKSPACE = 4
AGZO_ERR_STATE = 5
AGZO_ERR_TIMEOUT = 6
AGZO_ERR_CALLBACK = 7
AGZO_WARN_RANK_DEFICIENT = 100
AGZO_BF16, AGZO_F32 = 0, 1
AGZO_MAX_RANK = 64

EXPORTS = [
    "agzo_workspace_bytes", "agzo_create", "agzo_destroy", "agzo_set_option", "agzo_poll",
    "agzo_status_string", "agzo_last_cuda_error", "agzo_extract_subspace", "agzo_perturb",
    "agzo_restore", "agzo_update", "agzo_ghat", "agzo_restore_update", "agzo_step",
    "agzo_perturb_dense", "agzo_debug_philox", "agzo_debug_gaussian", "agzo_read_counters",
    "agzo_extract_subspace_static", "agzo_fill_gaussian_basis", "agzo_set_allreduce",
    "agzo_debug_wait_timeout", "agzo_query_fused", "agzo_query_cluster_capacity", "agzo_debug_fused_split",
]
KC_RMW, KC_XT_T, KC_X_Q, KC_PANEL_QR, KC_TC_XT_T, KC_TC_X_Q, KC_OMEGA, KC_RMW_TC, KC_FUSED_POWER = 1, 2, 3, 4, 5, 6, 7, 8, 9


class agzo_layer(C.Structure):
    _fields_ = [
        ("W", C.c_void_p), ("ldw", C.c_int64),
        ("W16", C.c_void_p), ("ldw16", C.c_int64),
        ("X", C.c_void_p), ("ldx", C.c_int64),
        ("V", C.c_void_p), ("ldv", C.c_int64),
        ("w_dtype", C.c_int32), ("x_dtype", C.c_int32),
        ("d_out", C.c_int32), ("d_in", C.c_int32),
        ("m", C.c_int32), ("r", C.c_int32),
        ("layer_id", C.c_uint32), ("reserved", C.c_uint32),
    ]


class agzo_params(C.Structure):
    _fields_ = [("seed", C.c_uint64), ("eps", C.c_float), ("lr", C.c_float),
                ("K", C.c_int32), ("mode", C.c_int32)]


LOSS_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p)
ALLREDUCE_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_size_t)

_lib = None


class AgzoError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: status {status} ({status_string(status)})")
        self.status = status


def lib() -> C.CDLL:
    """Loads libagzo.so; raises if it has not been built (no fallback path exists)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2601_17261_b200.build`; "
            "the AGZO path has no CPU or PyTorch fallback")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, u32, u64, f32 = C.c_void_p, C.c_int, C.c_int64, C.c_uint32, C.c_uint64, C.c_float
    LP = C.POINTER(agzo_layer)
    sig = {
        "agzo_workspace_bytes": (i32, [LP, i32, C.POINTER(C.c_size_t)]),
        "agzo_create": (i32, [C.POINTER(vp), i32, vp, C.c_size_t]),
        "agzo_destroy": (i32, [vp]),
        "agzo_set_option": (i32, [vp, C.c_char_p, i64]),
        "agzo_poll": (i32, [vp, vp]),
        "agzo_status_string": (C.c_char_p, [i32]),
        "agzo_last_cuda_error": (i32, [vp]),
        "agzo_extract_subspace": (i32, [vp, LP, i32, u64, i32, vp]),
        "agzo_perturb": (i32, [vp, LP, i32, u64, f32, vp]),
        "agzo_fill_gaussian_basis": (i32, [vp, LP, i32, u64, vp]),
        "agzo_restore": (i32, [vp, LP, i32, u64, f32, vp]),
        "agzo_update": (i32, [vp, LP, i32, u64, f32, vp, vp]),
        "agzo_ghat": (i32, [vp, vp, vp, f32, i32, vp, vp]),
        "agzo_restore_update": (i32, [vp, LP, i32, u64, f32, f32, i32, vp, vp]),
        "agzo_step": (i32, [vp, LP, i32, C.POINTER(agzo_params), LOSS_FN, vp, vp, vp, vp]),
        "agzo_perturb_dense": (i32, [vp, vp, i64, i32, u64, u32, f32, vp, vp]),
        "agzo_debug_philox": (i32, [vp, u64, u32, u32, u64, u64, vp, vp]),
        "agzo_debug_gaussian": (i32, [vp, u64, u32, u32, u64, u64, vp, vp]),
        "agzo_read_counters": (i32, [vp, C.POINTER(C.c_double), C.POINTER(i64), C.POINTER(i64)]),
        "agzo_set_allreduce": (i32, [vp, ALLREDUCE_FN, vp, i64]),
        "agzo_debug_wait_timeout": (i32, [vp, vp]),
        "agzo_query_fused": (i32, [vp, LP, i32, C.POINTER(C.c_int32), vp]),
        "agzo_query_cluster_capacity": (i32, [vp, C.POINTER(C.c_int32)]),
        "agzo_debug_fused_split": (i32, [C.POINTER(C.c_int32), i32, i32, C.POINTER(C.c_int32), C.POINTER(C.c_int32),
                                         C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int32)]),
        "agzo_extract_subspace_static": (i32, [vp, i64, C.c_int32, C.c_int32, C.c_int32, C.c_int32,
                                               C.c_int32, u64, u32, vp, i64, vp, vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(L, name)
        fn.restype = res
        fn.argtypes = args
    _lib = L
    return L


def status_string(status: int) -> str:
    return lib().agzo_status_string(int(status)).decode()


def _check(status: int, what: str, allow: Sequence[int] = ()) -> int:
    if status != AGZO_OK and status not in allow:
        raise AgzoError(status, what)
    return status


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return AGZO_BF16
    if t.dtype == torch.float32:
        return AGZO_F32
    raise TypeError(f"unsupported dtype {t.dtype}")


def _stream_ptr(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def make_layer(*, V: torch.Tensor, r: int, layer_id: int, W: Optional[torch.Tensor] = None,
               X: Optional[torch.Tensor] = None, W16: Optional[torch.Tensor] = None,
               d_in: Optional[int] = None) -> agzo_layer:
    """Descriptor from 2-D torch tensors (last dimension contiguous); keeps no reference."""
    L = agzo_layer()
    if V.dim() != 2 or V.stride(1) != 1 or V.dtype != torch.float32:
        raise ValueError("V must be [r][ldv] fp32 with unit inner stride")
    L.V, L.ldv, L.r, L.layer_id, L.reserved = V.data_ptr(), V.stride(0), int(r), int(layer_id), 0
    if d_in is None:
        d_in = W.shape[1] if W is not None else X.shape[1]
    L.d_in = int(d_in)
    if W is not None:
        if W.dim() != 2 or W.stride(1) != 1:
            raise ValueError("W must be 2-D with unit inner stride")
        L.W, L.ldw, L.w_dtype, L.d_out = W.data_ptr(), W.stride(0), _dtype_code(W), W.shape[0]
    if W16 is not None:
        if W16.dtype != torch.bfloat16 or W16.stride(1) != 1:
            raise ValueError("W16 must be bf16 with unit inner stride")
        L.W16, L.ldw16 = W16.data_ptr(), W16.stride(0)
    if X is not None:
        if X.dim() != 2 or X.stride(1) != 1:
            raise ValueError("X must be 2-D with unit inner stride")
        L.X, L.ldx, L.x_dtype, L.m = X.data_ptr(), X.stride(0), _dtype_code(X), X.shape[0]
    return L


def layer_array(layers: Sequence[agzo_layer]):
    arr = (agzo_layer * max(1, len(layers)))()
    for i, l in enumerate(layers):
        arr[i] = l
    return arr


# ---------------------------------------------------------------- thin wrappers, same names
def agzo_workspace_bytes(layers: Sequence[agzo_layer]) -> int:
    out = C.c_size_t(0)
    _check(lib().agzo_workspace_bytes(layer_array(layers), len(layers), C.byref(out)),
           "agzo_workspace_bytes")
    return int(out.value)


class Context:
    """Owns the opaque agzo_ctx and the torch tensor that backs its workspace."""

    def __init__(self, device: int, workspace_bytes: int):
        self.device = int(device)
        self.workspace = torch.empty(max(int(workspace_bytes), 4096), dtype=torch.uint8,
                                     device=f"cuda:{self.device}")
        h = C.c_void_p()
        _check(lib().agzo_create(C.byref(h), self.device, self.workspace.data_ptr(),
                                 self.workspace.numel()), "agzo_create")
        self.handle = h

    def close(self):
        if self.handle is not None and self.handle.value:
            lib().agzo_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def agzo_create(layers: Sequence[agzo_layer], device: int = 0, extra_bytes: int = 0) -> Context:
    return Context(device, agzo_workspace_bytes(layers) + extra_bytes)


def agzo_destroy(ctx: Context) -> None:
    ctx.close()


def agzo_set_option(ctx: Context, name: str, value: int) -> None:
    _check(lib().agzo_set_option(ctx.handle, name.encode(), int(value)), "agzo_set_option")


def agzo_read_counters(ctx: Context):
    """(summed ms of the timed kernel class, its launches, launches of every class)."""
    ms, nt, na = C.c_double(0), C.c_int64(0), C.c_int64(0)
    _check(lib().agzo_read_counters(ctx.handle, C.byref(ms), C.byref(nt), C.byref(na)),
           "agzo_read_counters")
    return ms.value, nt.value, na.value


def agzo_query_fused(ctx: Context, layers, stream=None, arr=None):
    """Per layer: the cluster size of the fused power-step kernel, 0 = two-sweep kernels."""
    arr = arr if arr is not None else layer_array(layers)
    out = (C.c_int32 * len(layers))()
    _check(lib().agzo_query_fused(ctx.handle, arr, len(layers), out, _stream_ptr(stream)), "agzo_query_fused")
    return list(out)


def agzo_debug_fused_split(tiles, clusters: int):
    """(tile0, first, parts, share_begin) of the fused power step's work split; host arithmetic only."""
    n = len(tiles)
    t = (C.c_int32 * max(n, 1))(*tiles)
    tile0, first, parts = (C.c_int32 * max(n, 1))(), (C.c_int32 * max(n, 1))(), (C.c_int32 * max(n, 1))()
    begin = (C.c_int32 * (clusters + 1))()
    shares = C.c_int32(0)
    _check(lib().agzo_debug_fused_split(t, n, clusters, tile0, first, parts, begin, C.byref(shares)),
           "agzo_debug_fused_split")
    return list(tile0)[:n], list(first)[:n], list(parts)[:n], list(begin)[:shares.value + 1]


def agzo_query_cluster_capacity(ctx: Context):
    """[0, clusters of 1 CTA, of 2 CTAs, ..., of 16 CTAs] of the fused kernel resident at once."""
    out = (C.c_int32 * 17)()
    _check(lib().agzo_query_cluster_capacity(ctx.handle, out), "agzo_query_cluster_capacity")
    return list(out)


def agzo_poll(ctx: Context, stream=None) -> int:
    return lib().agzo_poll(ctx.handle, _stream_ptr(stream))


def agzo_extract_subspace(ctx: Context, layers, seed: int, K: int, stream=None, arr=None) -> None:
    arr = arr if arr is not None else layer_array(layers)
    _check(lib().agzo_extract_subspace(ctx.handle, arr, len(layers), seed, K, _stream_ptr(stream)),
           "agzo_extract_subspace")


def agzo_extract_subspace_static(X: torch.Tensor, V: torch.Tensor, r: int, K: int, seed: int,
                                 layer_id: int, d_rank_deficient: Optional[torch.Tensor] = None,
                                 stream=None) -> None:
    """Algorithm 1 for one layer with the library's built-in scratch: for callers that cannot
    allocate a workspace (see include/agzo.h).  No context; allocates nothing; uses the current
    device; calls that can overlap on the GPU must be ordered by the caller."""
    if X.dim() != 2 or X.stride(1) != 1 or V.dim() != 2 or V.stride(1) != 1 or V.dtype != torch.float32:
        raise ValueError("X [m][ldx] and V [r][ldv] (fp32) need unit inner strides")
    flag = d_rank_deficient.data_ptr() if d_rank_deficient is not None else None
    _check(lib().agzo_extract_subspace_static(X.data_ptr(), X.stride(0), _dtype_code(X), X.shape[0],
                                              X.shape[1], r, K, seed, layer_id, V.data_ptr(),
                                              V.stride(0), flag, _stream_ptr(stream)),
           "agzo_extract_subspace_static")


def agzo_fill_gaussian_basis(ctx: Context, layers, seed: int, stream=None, arr=None) -> None:
    arr = arr if arr is not None else layer_array(layers)
    _check(lib().agzo_fill_gaussian_basis(ctx.handle, arr, len(layers), seed, _stream_ptr(stream)),
           "agzo_fill_gaussian_basis")


def agzo_perturb(ctx: Context, layers, seed: int, scale: float, stream=None, arr=None) -> None:
    arr = arr if arr is not None else layer_array(layers)
    _check(lib().agzo_perturb(ctx.handle, arr, len(layers), seed, scale, _stream_ptr(stream)),
           "agzo_perturb")


def agzo_restore(ctx: Context, layers, seed: int, scale: float, stream=None, arr=None) -> None:
    arr = arr if arr is not None else layer_array(layers)
    _check(lib().agzo_restore(ctx.handle, arr, len(layers), seed, scale, _stream_ptr(stream)),
           "agzo_restore")


def agzo_update(ctx: Context, layers, seed: int, lr: float, d_ghat: torch.Tensor, stream=None,
                arr=None) -> None:
    arr = arr if arr is not None else layer_array(layers)
    _check(lib().agzo_update(ctx.handle, arr, len(layers), seed, lr, d_ghat.data_ptr(),
                             _stream_ptr(stream)), "agzo_update")


def agzo_ghat(ctx: Context, d_f_plus: torch.Tensor, d_f_other: torch.Tensor, eps: float, mode: int,
              d_ghat: torch.Tensor, stream=None) -> None:
    if d_f_plus.dtype != torch.float64 or d_f_other.dtype != torch.float64:
        raise TypeError("losses are float64 device scalars")
    _check(lib().agzo_ghat(ctx.handle, d_f_plus.data_ptr(), d_f_other.data_ptr(), eps, mode,
                           d_ghat.data_ptr(), _stream_ptr(stream)), "agzo_ghat")


def agzo_restore_update(ctx: Context, layers, seed: int, eps: float, lr: float, mode: int,
                        d_ghat: torch.Tensor, stream=None, arr=None) -> None:
    arr = arr if arr is not None else layer_array(layers)
    _check(lib().agzo_restore_update(ctx.handle, arr, len(layers), seed, eps, lr, mode,
                                     d_ghat.data_ptr(), _stream_ptr(stream)), "agzo_restore_update")


def agzo_step(ctx: Context, layers, *, seed: int, eps: float, lr: float, K: int, mode: int,
              loss_fn, d_losses2: torch.Tensor, d_ghat: torch.Tensor, stream=None,
              arr=None) -> None:
    """loss_fn(phase:int, slot:int, stream_ptr:int) -> None leaves the float64 loss in
    d_losses2[slot] on the stream; exceptions become AGZO_ERR_CALLBACK."""
    if d_losses2.dtype != torch.float64 or d_losses2.numel() < 2 or d_ghat.dtype != torch.float32:
        raise TypeError("d_losses2 is 2 float64, d_ghat 1 float32 (device)")
    base = d_losses2.data_ptr()
    arr = arr if arr is not None else layer_array(layers)
    p = agzo_params(seed, eps, lr, K, mode)
    err: List[BaseException] = []

    def tramp(user, stream_ptr, phase, d_loss):
        try:
            loss_fn(int(phase), (int(d_loss) - base) // 8, int(stream_ptr or 0))
            return 0
        except BaseException as e:  # noqa: BLE001 - must not unwind through C
            err.append(e)
            return 1

    cb = LOSS_FN(tramp)
    st = lib().agzo_step(ctx.handle, arr, len(layers), C.byref(p), cb, None, d_losses2.data_ptr(),
                         d_ghat.data_ptr(), _stream_ptr(stream))
    if st == AGZO_ERR_CALLBACK and err:
        raise AgzoError(st, f"agzo_step (callback raised {err[0]!r})")
    _check(st, "agzo_step")


class _DeviceFloats:
    """A float32 device buffer given by address, for torch.as_tensor (no copy)."""

    def __init__(self, ptr: int, count: int):
        self.__cuda_array_interface__ = {"shape": (count,), "typestr": "<f4", "data": (ptr, False),
                                         "version": 2}


def device_floats(ptr: int, count: int, device: int) -> torch.Tensor:
    """View of `count` floats at device address `ptr` (memory owned by someone else)."""
    return torch.as_tensor(_DeviceFloats(ptr, count), device=f"cuda:{device}")


def agzo_set_allreduce(ctx: Context, fn, token_offset: int = 0) -> None:
    """fn(buf: torch.Tensor, stream_ptr: int) -> None sums the float32 device view `buf` over
    all ranks in place, enqueued on the stream; None (with token_offset 0) switches
    token-sharded extraction off.  The context keeps the callback alive."""
    if fn is None:
        _check(lib().agzo_set_allreduce(ctx.handle, ALLREDUCE_FN(), None, 0), "agzo_set_allreduce")
        ctx._allreduce_cb = None
        return
    errors: List[BaseException] = []

    def tramp(user, stream_ptr, d_buf, count):
        try:
            fn(device_floats(int(d_buf), int(count), ctx.device), int(stream_ptr or 0))
            return 0
        except BaseException as e:  # noqa: BLE001 - must not unwind through C
            errors.append(e)
            return 1

    cb = ALLREDUCE_FN(tramp)
    _check(lib().agzo_set_allreduce(ctx.handle, cb, None, int(token_offset)), "agzo_set_allreduce")
    ctx._allreduce_cb = cb
    ctx._allreduce_errors = errors


def torch_allreduce(group=None):
    """An `fn` for agzo_set_allreduce that sums with torch.distributed (NCCL for device
    buffers) on the stream the library passes."""
    import torch.distributed as dist

    def fn(buf: torch.Tensor, stream_ptr: int) -> None:
        if buf.is_cuda:
            with torch.cuda.stream(torch.cuda.ExternalStream(stream_ptr, device=buf.device)):
                dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)
        else:
            dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)

    return fn


def agzo_perturb_dense(ctx: Context, w: torch.Tensor, seed: int, layer_id: int, scale: float,
                       d_scale: Optional[torch.Tensor] = None, stream=None) -> None:
    if not w.is_contiguous():
        raise ValueError("w must be contiguous")
    _check(lib().agzo_perturb_dense(ctx.handle, w.data_ptr(), w.numel(), _dtype_code(w), seed,
                                    layer_id, scale,
                                    d_scale.data_ptr() if d_scale is not None else None,
                                    _stream_ptr(stream)), "agzo_perturb_dense")


def agzo_debug_wait_timeout(ctx: Context, stream=None) -> None:
    _check(lib().agzo_debug_wait_timeout(ctx.handle, _stream_ptr(stream)), "agzo_debug_wait_timeout")


def agzo_debug_philox(ctx: Context, seed: int, layer_id: int, tag: int, first: int, n: int,
                      stream=None) -> torch.Tensor:
    out = torch.empty(max(n, 1), dtype=torch.int32, device=f"cuda:{ctx.device}")
    _check(lib().agzo_debug_philox(ctx.handle, seed, layer_id, tag, first, n, out.data_ptr(),
                                   _stream_ptr(stream)), "agzo_debug_philox")
    return out[:n]


def agzo_debug_gaussian(ctx: Context, seed: int, layer_id: int, tag: int, first: int, n: int,
                        stream=None) -> torch.Tensor:
    out = torch.empty(max(n, 1), dtype=torch.float32, device=f"cuda:{ctx.device}")
    _check(lib().agzo_debug_gaussian(ctx.handle, seed, layer_id, tag, first, n, out.data_ptr(),
                                     _stream_ptr(stream)), "agzo_debug_gaussian")
    return out[:n]
