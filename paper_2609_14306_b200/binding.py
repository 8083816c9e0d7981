"""ctypes binding of libvpce.so: argument marshalling only, same names as the C entry points.

Tensors are torch CUDA tensors (torch supplies device memory and streams); the binding
checks dtype/shape/contiguity, passes raw device pointers and the current stream, and turns
non-zero status codes into ``VpceError``.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

_LIB: Optional[ctypes.CDLL] = None
_LIB_NAME = "libvpce.so"


class VpceError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"vp_ce status {code}: {msg}")
        self.code = code


def library_path() -> str:
    return os.path.join(os.path.dirname(os.path.abspath(__file__)), _LIB_NAME)


def load_library() -> ctypes.CDLL:
    """Load the in-tree CUDA library; raises if it has not been built (no fallback exists)."""
    global _LIB
    if _LIB is not None:
        return _LIB
    path = library_path()
    if not os.path.exists(path):
        # Not built yet: compile it in-tree now (nvcc, sm_100a).  There is no other implementation to fall
        # back to, so a failed build is fatal.
        try:
            from .build import build_library
            build_library()
        except Exception as exc:
            raise RuntimeError(
                f"{path} is missing and could not be built ({exc}); build it with "
                "`python -m paper_2609_14306_b200.build`; this package has no CPU fallback") from exc
    lib = ctypes.CDLL(path)
    i64, i32, vp, sz = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_size_t
    lib.vp_ce_workspace_bytes.restype = sz
    lib.vp_ce_workspace_bytes.argtypes = [i64, i64, i64]
    lib.vp_ce_forward.restype = ctypes.c_int
    lib.vp_ce_forward.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, vp, vp, i64, i64, vp, sz, vp]
    lib.vp_ce_backward.restype = ctypes.c_int
    lib.vp_ce_backward.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, i32, i64, i64,
                                   ctypes.c_int, vp, sz, vp]
    lib.vp_ce_mean_loss.restype = ctypes.c_int
    lib.vp_ce_mean_loss.argtypes = [vp, vp, i64, i64, i32, vp, vp, vp]
    lib.vp_ce_meeting_workspace_bytes.restype = sz
    lib.vp_ce_meeting_workspace_bytes.argtypes = [i64, i64, i64]
    lib.vp_ce_meeting_forward.restype = ctypes.c_int
    lib.vp_ce_meeting_forward.argtypes = [vp, vp, vp, i64, i64, i64, i64, i64, i32, vp, ctypes.c_int, ctypes.c_int,
                                          vp, vp, vp, sz, vp]
    lib.vp_ce_meeting_backward.restype = ctypes.c_int
    lib.vp_ce_meeting_backward.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i64, i64, i32, ctypes.c_int, vp,
                                           ctypes.c_int, ctypes.c_int, vp, vp, ctypes.c_int, vp, sz, vp]
    lib.vp_ce_mean_loss_grad.restype = ctypes.c_int
    lib.vp_ce_mean_loss_grad.argtypes = [vp, i64, i64, i32, vp, vp, vp, vp]
    lib.vp_ce_device_status.restype = ctypes.c_int
    lib.vp_ce_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int32), vp]
    lib.vp_ce_status_string.restype = ctypes.c_char_p
    lib.vp_ce_status_string.argtypes = [ctypes.c_int]
    lib.vp_ce_launch_count.restype = i64
    lib.vp_ce_launch_count.argtypes = []
    lib.vp_ce_fwd_bwd_host.restype = ctypes.c_int
    lib.vp_ce_fwd_bwd_host.argtypes = [vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, i32, i64, i64, ctypes.c_int,
                                       vp, vp, vp, vp, vp, vp, sz, vp]
    lib.vp_ce_forward_static.restype = ctypes.c_int
    lib.vp_ce_forward_static.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, vp, vp, i64, i64, vp, vp]
    lib.vp_ce_workspace_bytes_f32.restype = sz
    lib.vp_ce_workspace_bytes_f32.argtypes = [i64, i64, i64]
    lib.vp_ce_forward_f32.restype = ctypes.c_int
    lib.vp_ce_forward_f32.argtypes = [vp, vp, vp, i64, i64, i64, i64, i32, vp, vp, i64, i64, vp, sz, vp]
    lib.vp_ce_backward_f32.restype = ctypes.c_int
    lib.vp_ce_backward_f32.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i64, i32, i64, i64,
                                       ctypes.c_int, vp, sz, vp]
    lib.vp_ce_set_wait_limit_ns.restype = i64
    lib.vp_ce_set_wait_limit_ns.argtypes = [i64]
    lib.vp_ce_set_tail_parts.restype = ctypes.c_int
    lib.vp_ce_set_tail_parts.argtypes = [ctypes.c_int]
    lib.vp_ce_tail_choice.restype = ctypes.c_int
    lib.vp_ce_tail_choice.argtypes = [ctypes.c_int] * 6 + [ctypes.POINTER(ctypes.c_int)] * 3
    lib.vp_ce_debug_drop_copy.restype = ctypes.c_int
    lib.vp_ce_debug_drop_copy.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int]
    f32 = ctypes.c_float
    lib.osadamw_staging_bytes.restype = sz
    lib.osadamw_staging_bytes.argtypes = [i64, ctypes.c_int]
    lib.osadamw_create.restype = ctypes.c_int
    lib.osadamw_create.argtypes = [ctypes.POINTER(vp), i64, ctypes.c_int, vp, sz]
    lib.osadamw_destroy.restype = ctypes.c_int
    lib.osadamw_destroy.argtypes = [vp]
    lib.osadamw_step.restype = ctypes.c_int
    lib.osadamw_step.argtypes = [vp, vp, vp, vp, vp, vp, i64, vp, i64, f32, f32, f32, f32, f32, i64, vp]
    lib.osadamw_wait.restype = ctypes.c_int
    lib.osadamw_wait.argtypes = [vp]
    lib.osadamw_update_device.restype = ctypes.c_int
    lib.osadamw_update_device.argtypes = [vp, vp, vp, vp, vp, i64, f32, f32, f32, f32, f32, i64, vp]
    lib.vp_ce_profile_enable.restype = None
    lib.vp_ce_profile_enable.argtypes = [ctypes.c_int]
    lib.vp_ce_profile_collect.restype = ctypes.c_int
    lib.vp_ce_profile_collect.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
    _LIB = lib
    return lib


def _check(code: int) -> None:
    if code != 0:
        raise VpceError(code, vp_ce_status_string(code))


def vp_ce_status_string(code: int) -> str:
    return load_library().vp_ce_status_string(int(code)).decode()


def vp_ce_launch_count() -> int:
    return int(load_library().vp_ce_launch_count())


def vp_ce_workspace_bytes(T_chunk: int, d: int, block_v: int) -> int:
    return int(load_library().vp_ce_workspace_bytes(int(T_chunk), int(d), int(block_v)))


def _stream_ptr(stream, like=None) -> int:
    """Raw cudaStream_t: the given stream, else the current stream of the device that holds `like`."""
    import torch
    if stream is not None:
        return int(stream.cuda_stream)
    dev = like.device if like is not None else None
    return int(torch.cuda.current_stream(dev).cuda_stream)


class _on_device:
    """Makes the device that holds the operands current for the duration of a call (the library launches
    on the current device)."""

    def __init__(self, t):
        import torch
        self._guard = torch.cuda.device(t.device)

    def __enter__(self):
        return self._guard.__enter__()

    def __exit__(self, *a):
        return self._guard.__exit__(*a)


def _ptr(t, dtype, name: str, numel: Optional[int] = None) -> int:
    import torch
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype:
        raise TypeError(f"{name} must have dtype {dtype}, got {t.dtype}")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if numel is not None and t.numel() != numel:
        raise ValueError(f"{name} has {t.numel()} elements, expected {numel}")
    return int(t.data_ptr())


def _shapes(H, W) -> Tuple[int, int, int]:
    if H.dim() != 2 or W.dim() != 2 or H.shape[1] != W.shape[1]:
        raise ValueError("H must be [T, d] and W [V, d]")
    return int(H.shape[0]), int(H.shape[1]), int(W.shape[0])


def vp_ce_forward(H, W, labels, block_v: int, ignore_index: int, loss, lse, T_chunk: int,
                  chunk_index_base: int, workspace, stream=None) -> None:
    """loss[n], lse[n] for every token (Algorithm 3); see include/vp_ce.h for the contract."""
    import torch
    lib = load_library()
    T, d, V = _shapes(H, W)
    with _on_device(H):
        _check(lib.vp_ce_forward(
            _ptr(H, torch.bfloat16, "H"), _ptr(W, torch.bfloat16, "W"), _ptr(labels, torch.int32, "labels", T),
            T, d, V, int(block_v), int(ignore_index),
            _ptr(loss, torch.float32, "loss", T), _ptr(lse, torch.float32, "lse", T),
            int(T_chunk), int(chunk_index_base),
            _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream, H)))


def vp_ce_backward(H, W, labels, lse, dloss, dH, dW, block_v: int, ignore_index: int, T_chunk: int,
                   chunk_index_base: int, accumulate_dW: bool, workspace, stream=None) -> None:
    """dH (bf16, overwritten) and dW (fp32, overwritten or accumulated); dloss may be None; one of dH, dW may be
    None (that gradient is skipped)."""
    import torch
    lib = load_library()
    T, d, V = _shapes(H, W)
    with _on_device(H):
        _check(lib.vp_ce_backward(
            _ptr(H, torch.bfloat16, "H"), _ptr(W, torch.bfloat16, "W"), _ptr(labels, torch.int32, "labels", T),
            _ptr(lse, torch.float32, "lse", T),
            None if dloss is None else _ptr(dloss, torch.float32, "dloss", T),
            None if dH is None else _ptr(dH, torch.bfloat16, "dH", T * d),
            None if dW is None else _ptr(dW, torch.float32, "dW", V * d),
            T, d, V, int(block_v), int(ignore_index), int(T_chunk), int(chunk_index_base),
            1 if accumulate_dW else 0,
            _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream, H)))


PHASE_RESIDUAL, PHASE_INPUT_GRAD, PHASE_WEIGHT_GRAD = 1, 2, 4


def vp_ce_meeting_workspace_bytes(N: int, d: int, shard_rows: int) -> int:
    return int(load_library().vp_ce_meeting_workspace_bytes(int(N), int(d), int(shard_rows)))


def vp_ce_meeting_forward(X, W_shard, targets, v_lo: int, V: int, ignore_index: int, state, first: bool, last: bool,
                          loss, lse, workspace, stream=None) -> None:
    """One forward meeting of batch X [N, d] with shard W_shard (vocabulary ids v_lo ...): folds the strip into
    state [3, N] = (m, z, y_t); with last=True also writes lse and loss."""
    import torch
    lib = load_library()
    N, d, S = _shapes(X, W_shard)
    with _on_device(X):
        _check(lib.vp_ce_meeting_forward(
            _ptr(X, torch.bfloat16, "X"), _ptr(W_shard, torch.bfloat16, "W_shard"),
            _ptr(targets, torch.int32, "targets", N), N, d, S, int(v_lo), int(V), int(ignore_index),
            _ptr(state, torch.float32, "state", 3 * N), 1 if first else 0, 1 if last else 0,
            None if loss is None else _ptr(loss, torch.float32, "loss", N),
            None if lse is None else _ptr(lse, torch.float32, "lse", N),
            _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream, X)))


def vp_ce_meeting_backward(X, W_shard, targets, lse, dloss, v_lo: int, V: int, ignore_index: int, phases: int,
                           dX_acc, first: bool, last: bool, dX, dW_shard, accumulate_dW: bool, workspace,
                           stream=None) -> None:
    """One backward meeting (phases: bit mask of PHASE_*); see include/vp_ce.h."""
    import torch
    lib = load_library()
    N, d, S = _shapes(X, W_shard)
    with _on_device(X):
        _check(lib.vp_ce_meeting_backward(
            _ptr(X, torch.bfloat16, "X"), _ptr(W_shard, torch.bfloat16, "W_shard"),
            _ptr(targets, torch.int32, "targets", N), _ptr(lse, torch.float32, "lse", N),
            _ptr(dloss, torch.float32, "dloss", N), N, d, S, int(v_lo), int(V), int(ignore_index), int(phases),
            None if dX_acc is None else _ptr(dX_acc, torch.float32, "dX_acc", N * d),
            1 if first else 0, 1 if last else 0,
            None if dX is None else _ptr(dX, torch.bfloat16, "dX", N * d),
            None if dW_shard is None else _ptr(dW_shard, torch.float32, "dW_shard", S * d),
            1 if accumulate_dW else 0,
            _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream, X)))


def vp_ce_mean_loss_grad(labels, V: int, ignore_index: int, n_valid, upstream, dloss_out, stream=None) -> None:
    """dloss_out[n] = upstream / n_valid on valid tokens, 0 elsewhere (upstream may be None = 1)."""
    import torch
    lib = load_library()
    T = labels.numel()
    with _on_device(labels):
        _check(lib.vp_ce_mean_loss_grad(
            _ptr(labels, torch.int32, "labels"), T, int(V), int(ignore_index),
            _ptr(n_valid, torch.int32, "n_valid", 1),
            None if upstream is None else _ptr(upstream, torch.float32, "upstream", 1),
            _ptr(dloss_out, torch.float32, "dloss_out", T), _stream_ptr(stream, labels)))


def vp_ce_mean_loss(loss, labels, V: int, ignore_index: int, mean_out, n_valid_out, stream=None) -> None:
    import torch
    lib = load_library()
    T = loss.numel()
    with _on_device(loss):
        _check(lib.vp_ce_mean_loss(
            _ptr(loss, torch.float32, "loss"), _ptr(labels, torch.int32, "labels", T), T, int(V), int(ignore_index),
            _ptr(mean_out, torch.float32, "mean_out", 1), _ptr(n_valid_out, torch.int32, "n_valid_out", 1),
            _stream_ptr(stream, loss)))


def vp_ce_device_status(workspace, stream=None) -> int:
    import torch
    lib = load_library()
    out = ctypes.c_int32(-1)
    with _on_device(workspace):
        _check(lib.vp_ce_device_status(_ptr(workspace, torch.uint8, "workspace"), ctypes.byref(out),
                                       _stream_ptr(stream, workspace)))
    return int(out.value)


def _host_ptr(t, dtype, name: str, numel: int) -> int:
    import torch
    if not isinstance(t, torch.Tensor) or t.is_cuda:
        raise TypeError(f"{name} must be a CPU tensor")
    if t.dtype != dtype or not t.is_contiguous() or t.numel() != numel:
        raise ValueError(f"{name}: expected contiguous {dtype} with {numel} elements")
    return int(t.data_ptr())


def vp_ce_fwd_bwd_host(H_host, labels_host, W, loss_host, dH_host, dW, block_v: int, ignore_index: int,
                       T_chunk: int, chunk_index_base: int, accumulate_dW: bool,
                       H_dev, labels_dev, loss_dev, lse_dev, dH_dev, workspace, stream=None) -> None:
    """Forward + backward with activations in host memory (copies inside the call); W/dW on device."""
    import torch
    lib = load_library()
    T, d = int(H_host.shape[0]), int(H_host.shape[1])
    V = int(W.shape[0])
    with _on_device(W):
        _check(lib.vp_ce_fwd_bwd_host(
            _host_ptr(H_host, torch.bfloat16, "H_host", T * d), _host_ptr(labels_host, torch.int32, "labels_host", T),
            _ptr(W, torch.bfloat16, "W", V * d), _host_ptr(loss_host, torch.float32, "loss_host", T),
            _host_ptr(dH_host, torch.bfloat16, "dH_host", T * d), _ptr(dW, torch.float32, "dW", V * d),
            T, d, V, int(block_v), int(ignore_index), int(T_chunk), int(chunk_index_base), 1 if accumulate_dW else 0,
            _ptr(H_dev, torch.bfloat16, "H_dev", T * d), _ptr(labels_dev, torch.int32, "labels_dev", T),
            _ptr(loss_dev, torch.float32, "loss_dev", T), _ptr(lse_dev, torch.float32, "lse_dev", T),
            _ptr(dH_dev, torch.bfloat16, "dH_dev", T * d),
            _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream, W)))


def vp_ce_set_wait_limit_ns(ns: int) -> int:
    """Sets the limit of every wait inside the kernels (ns <= 0: query only); returns the previous limit."""
    return int(load_library().vp_ce_set_wait_limit_ns(int(ns)))


def vp_ce_set_tail_parts(parts: int) -> int:
    """Overrides how the remainder tiles of the gradient GEMMs are split along K (-1 library's choice, 0 never,
    2..8 that many parts); returns the previous setting."""
    return int(load_library().vp_ce_set_tail_parts(int(parts)))


def vp_ce_tail_choice(row_tiles: int, col_tiles: int, group_cols: int, last_width: int, k_blocks: int, pairs: int):
    """(tiles split, parts, stagger) the library picks for a gradient GEMM of that launch geometry (host only)."""
    n, k, s = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    _check(load_library().vp_ce_tail_choice(int(row_tiles), int(col_tiles), int(group_cols), int(last_width),
                                            int(k_blocks), int(pairs), ctypes.byref(n), ctypes.byref(k), ctypes.byref(s)))
    return n.value, k.value, s.value


def vp_ce_debug_drop_copy(kernel_kind: int, k_block: int = 0, cta_ranks: int = 1) -> None:
    """Test hook: the next launch of that kernel kind loses the copies of one k-block (see include/vp_ce.h)."""
    _check(load_library().vp_ce_debug_drop_copy(int(kernel_kind), int(k_block), int(cta_ranks)))


KERNEL_KINDS = ("fwd_strip_fold", "bwd_strip_residual", "dH_gemm", "dW_gemm")


def vp_ce_profile_enable(on: bool) -> None:
    load_library().vp_ce_profile_enable(1 if on else 0)


def vp_ce_profile_collect():
    """Returns {kind: (total_ms, launches)} for the launches recorded since profiling was enabled."""
    lib = load_library()
    ms = (ctypes.c_double * 4)()
    n = (ctypes.c_int64 * 4)()
    _check(lib.vp_ce_profile_collect(ms, n))
    return {k: (float(ms[i]), int(n[i])) for i, k in enumerate(KERNEL_KINDS)}


def vp_ce_forward_static(H, W, labels, block_v: int, ignore_index: int, loss, lse, T_chunk: int,
                         chunk_index_base: int, device_status_out=None, stream=None) -> None:
    """vp_ce_forward for callers that cannot allocate or pass a workspace: the scratch is a fixed
    array inside the library (see include/vp_ce.h for its size limit and the sharing rules)."""
    import torch
    lib = load_library()
    T, d, V = _shapes(H, W)
    with _on_device(H):
        _check(lib.vp_ce_forward_static(
            _ptr(H, torch.bfloat16, "H"), _ptr(W, torch.bfloat16, "W"), _ptr(labels, torch.int32, "labels", T),
            T, d, V, int(block_v), int(ignore_index),
            _ptr(loss, torch.float32, "loss", T), _ptr(lse, torch.float32, "lse", T),
            int(T_chunk), int(chunk_index_base),
            None if device_status_out is None else _ptr(device_status_out, torch.int32, "device_status_out", 1),
            _stream_ptr(stream, H)))


def vp_ce_workspace_bytes_f32(T_chunk: int, d: int, block_v: int) -> int:
    return int(load_library().vp_ce_workspace_bytes_f32(int(T_chunk), int(d), int(block_v)))


def vp_ce_forward_f32(H, W, labels, block_v: int, ignore_index: int, loss, lse, T_chunk: int,
                      chunk_index_base: int, workspace, stream=None) -> None:
    """vp_ce_forward for float32 H and W (TF32 tensor cores)."""
    import torch
    lib = load_library()
    T, d, V = _shapes(H, W)
    with _on_device(H):
        _check(lib.vp_ce_forward_f32(
            _ptr(H, torch.float32, "H"), _ptr(W, torch.float32, "W"), _ptr(labels, torch.int32, "labels", T),
            T, d, V, int(block_v), int(ignore_index),
            _ptr(loss, torch.float32, "loss", T), _ptr(lse, torch.float32, "lse", T),
            int(T_chunk), int(chunk_index_base),
            _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream, H)))


def vp_ce_backward_f32(H, W, labels, lse, dloss, dH, dW, block_v: int, ignore_index: int, T_chunk: int,
                       chunk_index_base: int, accumulate_dW: bool, workspace, stream=None) -> None:
    """vp_ce_backward for float32 H and W; dH is float32."""
    import torch
    lib = load_library()
    T, d, V = _shapes(H, W)
    with _on_device(H):
        _check(lib.vp_ce_backward_f32(
            _ptr(H, torch.float32, "H"), _ptr(W, torch.float32, "W"), _ptr(labels, torch.int32, "labels", T),
            _ptr(lse, torch.float32, "lse", T),
            None if dloss is None else _ptr(dloss, torch.float32, "dloss", T),
            _ptr(dH, torch.float32, "dH", T * d), _ptr(dW, torch.float32, "dW", V * d),
            T, d, V, int(block_v), int(ignore_index), int(T_chunk), int(chunk_index_base),
            1 if accumulate_dW else 0,
            _ptr(workspace, torch.uint8, "workspace"), workspace.numel(), _stream_ptr(stream, H)))


# --------------------------------------------------------------------------- bucket-streamed AdamW (stream_adamw.h)
def osadamw_staging_bytes(bucket_params: int, slots: int) -> int:
    return int(load_library().osadamw_staging_bytes(int(bucket_params), int(slots)))


def osadamw_create(bucket_params: int, slots: int, staging) -> int:
    """Creates a pipeline over the caller's device staging buffer (uint8 CUDA tensor); returns the handle."""
    import torch
    lib = load_library()
    handle = ctypes.c_void_p()
    with _on_device(staging):
        _check(lib.osadamw_create(ctypes.byref(handle), int(bucket_params), int(slots),
                                  _ptr(staging, torch.uint8, "staging"), staging.numel()))
    return int(handle.value)


def osadamw_destroy(handle: int) -> None:
    _check(load_library().osadamw_destroy(ctypes.c_void_p(handle)))


def osadamw_step(handle: int, master, m, v, grad, w_bf16, lr: float, beta1: float, beta2: float, eps: float,
                 weight_decay: float, step: int, bucket_offsets=None, stream=None) -> None:
    """One optimizer step over HOST fp32 state (CPU tensors, ideally pinned) and the DEVICE bf16 working weight;
    asynchronous, see osadamw_wait."""
    import torch
    lib = load_library()
    n = master.numel()
    offs, nb = None, 0
    if bucket_offsets is not None:
        offs = (ctypes.c_int64 * len(bucket_offsets))(*[int(o) for o in bucket_offsets])
        nb = len(bucket_offsets) - 1
    with _on_device(w_bf16):
        _check(lib.osadamw_step(
            ctypes.c_void_p(handle), _host_ptr(master, torch.float32, "master", n), _host_ptr(m, torch.float32, "m", n),
            _host_ptr(v, torch.float32, "v", n), _host_ptr(grad, torch.float32, "grad", n),
            _ptr(w_bf16, torch.bfloat16, "w_bf16", n), n, offs, nb,
            float(lr), float(beta1), float(beta2), float(eps), float(weight_decay), int(step),
            _stream_ptr(stream, w_bf16)))


def osadamw_wait(handle: int) -> None:
    _check(load_library().osadamw_wait(ctypes.c_void_p(handle)))


def osadamw_update_device(p, m, v, g, w_bf16, lr: float, beta1: float, beta2: float, eps: float, weight_decay: float,
                          step: int, stream=None) -> None:
    """The fused AdamW update + bf16 refresh on device-resident fp32 state (in place)."""
    import torch
    lib = load_library()
    n = p.numel()
    with _on_device(p):
        _check(lib.osadamw_update_device(
            _ptr(p, torch.float32, "p"), _ptr(m, torch.float32, "m", n), _ptr(v, torch.float32, "v", n),
            _ptr(g, torch.float32, "g", n), _ptr(w_bf16, torch.bfloat16, "w_bf16", n), n,
            float(lr), float(beta1), float(beta2), float(eps), float(weight_decay), int(step), _stream_ptr(stream, p)))
