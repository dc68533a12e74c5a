"""Thin ctypes binding over libselectinfer.so: argument marshalling only.

Every function here has the name and argument order of its C entry point
(include/selectinfer.h; the si_debug_* diagnostics: include/selectinfer_debug.h) and takes torch CUDA tensors where the C side takes device
pointers.  torch is used for device memory and the current stream, nothing else: no
step of the path runs in Python or on the CPU.  If the CUDA library cannot be loaded
the import of this module fails -- there is no fallback.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch  # noqa: F401  (also makes libcudart resolvable for the library)

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libselectinfer.so")

SI_F16, SI_BF16, SI_F32 = 1, 2, 3
SI_OK = 0
SI_ERR_INVALID_ARG, SI_ERR_OUT_OF_RANGE, SI_ERR_DUPLICATE, SI_ERR_ALIGNMENT = -1, -2, -3, -4
SI_ERR_NOMEM, SI_ERR_CUDA, SI_ERR_TIMEOUT, SI_ERR_UNSUPPORTED = -5, -6, -7, -8
SI_ERR_TOO_LARGE = -9
SI_FLAG_CHECK, SI_FLAG_RESIDUAL, SI_FLAG_UNION_UNMASKED, SI_FLAG_SCORE_ABS = 1, 2, 4, 8
SI_FLAG_SHARED_LIST = 16
SI_FLAG_UNION_PATH = 32
SI_FLAG_LIST_PER_LAYER = 64
SI_FLAG_STEPS_ANY_ORDER = 128
SI_FLAG_SIMPLE_KERNELS = 256
SI_FLAG_PRENORM = 512
SI_SELECT_TOPK, SI_SELECT_THRESHOLD = 0, 1

EXPORTS = [
    "si_strerror", "si_last_cuda_error", "si_build_info", "si_store_bytes", "si_store_create", "si_store_free",
    "si_load_neurons", "si_store_slot_to_global", "si_store_global_to_slot", "si_store_records",
    "si_workspace_bytes", "si_select_workspace_bytes", "si_select", "si_ffn_forward",
    "si_layer_forward", "si_decode_stack_forward", "si_decode_chain_forward", "si_decode_prefix_forward", "si_ffn_forward_noalloc", "si_union",
    "si_debug_decode_stack_forward", "si_debug_decode_chain_forward", "si_debug_union_masks", "si_debug_ffn_forward_waits",
    "si_debug_read_bandwidth", "si_prefill_vote_workspace_bytes", "si_prefill_vote", "si_prefill_forward", "si_layer_range", "si_profile_accumulate", "si_profile_merge", "si_profile_rank",
    "si_loadset", "si_shard_count", "si_shard_lists", "si_shard_reduce", "si_ffn_forward_sharded",
    "si_debug_ffn_forward_sharded_group", "si_debug_pair_plan",
]


class SelectInferError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = f": {_lib.si_last_cuda_error().decode()}" if status == SI_ERR_CUDA else ""
        super().__init__(f"{where}: {strerror(status)} ({status}){detail}")


def _load_library() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2607_18081_b200.build` "
            "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cu, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint, ctypes.c_size_t
    psz = ctypes.POINTER(ctypes.c_size_t)
    lib.si_strerror.argtypes = [ci]; lib.si_strerror.restype = ctypes.c_char_p
    lib.si_build_info.argtypes = []; lib.si_build_info.restype = ctypes.c_char_p
    lib.si_last_cuda_error.argtypes = []; lib.si_last_cuda_error.restype = ctypes.c_char_p
    lib.si_store_bytes.argtypes = [ci, ci, ci, vp, ci, psz]
    lib.si_store_create.argtypes = [ctypes.POINTER(vp), vp, sz, ci, ci, ci, vp, ci]
    lib.si_store_free.argtypes = [vp]
    lib.si_load_neurons.argtypes = [vp, ci, vp, vp, vp, vp, ci, ci, vp]
    lib.si_store_slot_to_global.argtypes = [vp, ci, ctypes.POINTER(vp), ctypes.POINTER(ci), ctypes.POINTER(ci)]
    lib.si_store_global_to_slot.argtypes = [vp, ci, ctypes.POINTER(vp)]
    lib.si_store_records.argtypes = [vp, ci, ctypes.POINTER(vp), psz]
    lib.si_workspace_bytes.argtypes = [vp, ci, ci, ci, psz]
    lib.si_select_workspace_bytes.argtypes = [ci, psz]
    lib.si_select.argtypes = [vp, ci, ci, ci, ctypes.c_float, cu, vp, ci, vp, vp, sz, vp]
    lib.si_ffn_forward.argtypes = [vp, ci, vp, ci, vp, vp, ci, vp, ci, cu, vp, sz, vp, vp]
    lib.si_layer_forward.argtypes = [vp, ci, vp, ci, vp, ci, vp, vp, vp, ci, cu, vp, sz, vp, vp]
    lib.si_decode_stack_forward.argtypes = [vp, ci, vp, vp, vp, vp, ci, vp, ci, cu, vp, sz, vp, vp]
    lib.si_union.argtypes = [vp, ci, ci, vp, vp, ci, vp, vp, vp, sz, vp]
    lib.si_ffn_forward_noalloc.argtypes = [vp, ci, vp, vp, ci, vp, ci, cu, vp, vp]
    lib.si_decode_chain_forward.argtypes = [vp, ci, vp, ci, vp, vp, vp, ci, vp, vp, ctypes.c_float, cu, vp, sz, vp, vp]
    lib.si_decode_prefix_forward.argtypes = [vp, ci, vp, ci, ci, vp, vp, vp, ci, vp, ci, vp, ctypes.c_float, cu, vp, sz, vp, vp]
    lib.si_debug_decode_stack_forward.argtypes = lib.si_decode_stack_forward.argtypes + [vp]
    lib.si_debug_decode_chain_forward.argtypes = lib.si_decode_chain_forward.argtypes + [vp]
    lib.si_debug_union_masks.argtypes = [vp, ci, ci, vp, vp, ci, vp, vp, vp, vp, sz, vp]
    lib.si_debug_ffn_forward_waits.argtypes = lib.si_ffn_forward.argtypes + [ctypes.c_longlong, ci]
    lib.si_debug_read_bandwidth.argtypes = [vp, ctypes.c_size_t, vp, vp]
    lib.si_debug_pair_plan.argtypes = [ci, ci, ci, ci, ctypes.POINTER(ctypes.c_int)]
    lib.si_prefill_vote_workspace_bytes.argtypes = [ci, ci, ci, psz]
    lib.si_prefill_vote.argtypes = [vp, ci, ci, ci, ci, ci, ci, ci, cu, vp, ci, vp, vp, vp, sz, vp]
    lib.si_profile_accumulate.argtypes = [vp, ci, ci, ci, vp, vp]
    lib.si_profile_merge.argtypes = [vp, vp, ctypes.c_longlong, ci, vp]
    lib.si_profile_rank.argtypes = [vp, ci, vp, vp]
    lib.si_loadset.argtypes = [vp, vp, ci, ci, ci, vp, vp, sz, vp, vp]
    lib.si_layer_range.argtypes = [ci, ci, ci, ctypes.POINTER(ci), ctypes.POINTER(ci)]
    lib.si_shard_count.argtypes = [ci, ci, ci, ctypes.POINTER(ci)]
    lib.si_shard_lists.argtypes = [vp, vp, ci, ci, ci, ci, vp, vp, vp, sz, vp, vp]
    lib.si_shard_reduce.argtypes = [vp, ci, vp, ci, ci, ci, vp, ci, cu, vp]
    lib.si_ffn_forward_sharded.argtypes = [vp, ci, vp, vp, ci, vp, ci, cu, ci, ci, vp, vp, cu, vp, sz, vp, vp]
    lib.si_debug_ffn_forward_sharded_group.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp, vp, ci, cu, vp, vp, cu, vp, sz,
                                                       ctypes.c_longlong, vp, vp]
    lib.si_prefill_forward.argtypes = [vp, ci, vp, ci, vp, ci, ci, ci, ci, ci, cu, vp, ci, vp, vp, vp, sz, vp, sz, vp, vp]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("si_strerror", "si_build_info", "si_last_cuda_error"):
            fn.restype = ci
    return lib


_lib = _load_library()


def lib() -> ctypes.CDLL:
    return _lib


def strerror(status: int) -> str:
    return _lib.si_strerror(status).decode()


def build_info() -> str:
    return _lib.si_build_info().decode()


def _check(status: int, where: str) -> None:
    if status != SI_OK:
        raise SelectInferError(status, where)


def _dp(t) -> ctypes.c_void_p:
    """Device pointer of a torch tensor (None -> NULL)."""
    if t is None:
        return ctypes.c_void_p(0)
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None) -> ctypes.c_void_p:
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def dtype_code(dtype) -> int:
    if dtype in (torch.float16, "f16", SI_F16):
        return SI_F16
    if dtype in (torch.bfloat16, "bf16", SI_BF16):
        return SI_BF16
    if dtype in (torch.float32, "f32", SI_F32):
        return SI_F32
    raise ValueError(f"unsupported dtype {dtype}")


def torch_dtype(code) -> torch.dtype:
    return {SI_F16: torch.float16, SI_BF16: torch.bfloat16, SI_F32: torch.float32}[dtype_code(code)]


def _host_i32(a):
    if a is None:
        return None, ctypes.c_void_p(0)
    arr = np.ascontiguousarray(a, dtype=np.int32)
    return arr, arr.ctypes.data_as(ctypes.c_void_p)


# ------------------------------------------------------------------------- C entry points

def si_store_bytes(n_layers: int, d_model: int, d_ff: int, n_loaded, dtype) -> int:
    keep, p = _host_i32(n_loaded)
    out = ctypes.c_size_t(0)
    _check(_lib.si_store_bytes(n_layers, d_model, d_ff, p, dtype_code(dtype), ctypes.byref(out)), "si_store_bytes")
    return out.value


def si_store_create(store_mem: torch.Tensor, n_layers: int, d_model: int, d_ff: int, n_loaded, dtype):
    keep, p = _host_i32(n_loaded)
    handle = ctypes.c_void_p(0)
    _check(_lib.si_store_create(ctypes.byref(handle), _dp(store_mem), store_mem.numel() * store_mem.element_size(),
                                n_layers, d_model, d_ff, p, dtype_code(dtype)), "si_store_create")
    return handle


def si_store_free(handle) -> None:
    _check(_lib.si_store_free(handle), "si_store_free")


def si_load_neurons(handle, layer: int, w_gate, w_up, w_down, neuron_ids, n_base: int, stream=None) -> None:
    keep, p = _host_i32(neuron_ids)
    _check(_lib.si_load_neurons(handle, layer, _dp(w_gate), _dp(w_up), _dp(w_down), p, len(keep), n_base,
                                _stream(stream)), "si_load_neurons")


def si_workspace_bytes(handle, T_max: int, k_max: int, max_steps: int = 1) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib.si_workspace_bytes(handle, T_max, k_max, max_steps, ctypes.byref(out)), "si_workspace_bytes")
    return out.value


def si_select_workspace_bytes(n: int) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib.si_select_workspace_bytes(n, ctypes.byref(out)), "si_select_workspace_bytes")
    return out.value


def si_select(scores, mode: int, k: int, tau: float, flags: int, idx_out, n_out, workspace, stream=None) -> None:
    _check(_lib.si_select(_dp(scores), scores.numel(), mode, k, tau, flags, _dp(idx_out), idx_out.numel(),
                          _dp(n_out), _dp(workspace),
                          0 if workspace is None else workspace.numel() * workspace.element_size(),
                          _stream(stream)), "si_select")


def si_profile_accumulate(acts, scores, stream=None) -> None:
    T, n = acts.shape
    _check(_lib.si_profile_accumulate(_dp(acts), T, n, acts.stride(0), _dp(scores), _stream(stream)), "si_profile_accumulate")


def si_profile_merge(merged, scores, tokens: int, stream=None) -> None:
    _check(_lib.si_profile_merge(_dp(merged), _dp(scores), tokens, scores.numel(), _stream(stream)), "si_profile_merge")


def si_profile_rank(scores, ranking, stream=None) -> None:
    _check(_lib.si_profile_rank(_dp(scores), scores.numel(), _dp(ranking), _stream(stream)), "si_profile_rank")


def si_loadset(task_rank, model_rank, n_base: int, ids_out, workspace, status=None, stream=None) -> None:
    _check(_lib.si_loadset(_dp(task_rank), _dp(model_rank), task_rank.numel(), n_base, ids_out.numel(), _dp(ids_out),
                           _dp(workspace), workspace.numel() * workspace.element_size(), _dp(status), _stream(stream)),
           "si_loadset")


def si_layer_range(n_layers: int, first: int = 5, last: int = -2):
    """Selective layers of Table 1's policy as a half-open range (first, end)."""
    lo, hi = ctypes.c_int(0), ctypes.c_int(0)
    _check(_lib.si_layer_range(n_layers, first, last, ctypes.byref(lo), ctypes.byref(hi)), "si_layer_range")
    return lo.value, hi.value


def si_prefill_vote_workspace_bytes(T: int, n: int, alpha: int) -> int:
    out = ctypes.c_size_t(0)
    _check(_lib.si_prefill_vote_workspace_bytes(T, n, alpha, ctypes.byref(out)), "si_prefill_vote_workspace_bytes")
    return out.value


def si_prefill_vote(acts, alpha: int, beta: int, n_static: int, phi_count: int, flags: int, idx_out, n_out,
                    counts_out, workspace, stream=None) -> None:
    T, n = acts.shape
    _check(_lib.si_prefill_vote(_dp(acts), T, n, acts.stride(0), alpha, beta, n_static, phi_count, flags, _dp(idx_out),
                                idx_out.numel(), _dp(n_out), _dp(counts_out), _dp(workspace),
                                workspace.numel() * workspace.element_size(), _stream(stream)), "si_prefill_vote")


def si_prefill_forward(handle, layer: int, x, T: int, y, alpha: int, beta: int, n_static: int, phi_count: int,
                       flags: int, idx_out, n_out, acts_out, workspace, vote_workspace, status=None, stream=None) -> None:
    _check(_lib.si_prefill_forward(handle, layer, _dp(x), T, _dp(y), dtype_code(y.dtype), alpha, beta, n_static,
                                   phi_count, flags, _dp(idx_out), idx_out.numel(), _dp(n_out), _dp(acts_out),
                                   _dp(workspace), workspace.numel() * workspace.element_size(), _dp(vote_workspace),
                                   vote_workspace.numel() * vote_workspace.element_size(), _dp(status),
                                   _stream(stream)), "si_prefill_forward")


def si_ffn_forward(handle, layer: int, x, T: int, idx, idx_offsets, k_fixed: int, y, flags: int, workspace,
                   status=None, stream=None) -> None:
    _check(_lib.si_ffn_forward(handle, layer, _dp(x), T, _dp(idx), _dp(idx_offsets), k_fixed, _dp(y),
                               dtype_code(y.dtype), flags, _dp(workspace),
                               workspace.numel() * workspace.element_size(), _dp(status), _stream(stream)),
           "si_ffn_forward")


def si_layer_forward(handle, layer: int, x, T: int, scores, k: int, idx, idx_offsets, y, flags: int, workspace,
                     status=None, stream=None) -> None:
    _check(_lib.si_layer_forward(handle, layer, _dp(x), T, _dp(scores), k, _dp(idx), _dp(idx_offsets), _dp(y),
                                 dtype_code(y.dtype), flags, _dp(workspace),
                                 workspace.numel() * workspace.element_size(), _dp(status), _stream(stream)),
           "si_layer_forward")


def si_decode_stack_forward(handle, n_steps: int, layers, x, idx, idx_offsets, k_fixed: int, y, flags: int,
                            workspace, status=None, stream=None) -> None:
    keep, p = _host_i32(layers)
    _check(_lib.si_decode_stack_forward(handle, n_steps, p, _dp(x), _dp(idx), _dp(idx_offsets), k_fixed, _dp(y),
                                        dtype_code(y.dtype), flags, _dp(workspace),
                                        workspace.numel() * workspace.element_size(), _dp(status),
                                        _stream(stream)), "si_decode_stack_forward")


def si_shard_count(n: int, rank: int, world: int) -> int:
    out = ctypes.c_int(0)
    _check(_lib.si_shard_count(n, rank, world, ctypes.byref(out)), "si_shard_count")
    return out.value


def si_shard_lists(idx, idx_offsets, k_fixed: int, n_lists: int, rank: int, world: int, idx_out, offsets_out,
                   workspace, status=None, stream=None) -> None:
    _check(_lib.si_shard_lists(_dp(idx), _dp(idx_offsets), k_fixed, n_lists, rank, world, _dp(idx_out), _dp(offsets_out),
                               _dp(workspace), workspace.numel() * workspace.element_size(), _dp(status),
                               _stream(stream)), "si_shard_lists")


def si_shard_reduce(parts_dev, world: int, x, T: int, d_model: int, y, flags: int, x_dtype=None, stream=None) -> None:
    """parts_dev: int64 CUDA tensor holding `world` device addresses of fp32 [T, d_model] buffers."""
    xd = dtype_code(x.dtype) if x is not None else dtype_code(torch.bfloat16 if x_dtype is None else x_dtype)
    _check(_lib.si_shard_reduce(_dp(parts_dev), world, _dp(x), xd, T, d_model, _dp(y), dtype_code(y.dtype), flags,
                                _stream(stream)), "si_shard_reduce")


def _ptr_array(tensors_or_handles):
    vals = [t.value if isinstance(t, ctypes.c_void_p) else (0 if t is None else t.data_ptr()) for t in tensors_or_handles]
    return (ctypes.c_void_p * len(vals))(*vals)


def si_ffn_forward_sharded(handle, layer: int, x, idx, k: int, y, flags: int, rank: int, world: int, recv, marks, epoch: int,
                           workspace, status=None, stream=None) -> None:
    """recv, marks: lists of `world` tensors (every device's receive area / delivery marks as this device sees them)."""
    _check(_lib.si_ffn_forward_sharded(handle, layer, _dp(x), _dp(idx), k, _dp(y), dtype_code(y.dtype), flags, rank, world,
                                       _ptr_array(recv), _ptr_array(marks), epoch, _dp(workspace),
                                       workspace.numel() * workspace.element_size(), _dp(status), _stream(stream)),
           "si_ffn_forward_sharded")


def si_debug_ffn_forward_sharded_group(handles, rank_base: int, world: int, layer: int, xs, idxs, ks, ys, flags: int, recv,
                                       marks, epoch: int, workspaces, status=None, wait_cycles: int = 0, stream=None) -> None:
    n = len(handles)
    karr = (ctypes.c_int * n)(*[int(v) for v in ks])
    ws_bytes = min(w.numel() * w.element_size() for w in workspaces)
    _check(_lib.si_debug_ffn_forward_sharded_group(_ptr_array(handles), n, rank_base, world, layer, _ptr_array(xs), _ptr_array(idxs),
                                                   karr, _ptr_array(ys), dtype_code(ys[0].dtype), flags, _ptr_array(recv),
                                                   _ptr_array(marks), epoch, _ptr_array(workspaces), ws_bytes, wait_cycles,
                                                   _dp(status), _stream(stream)), "si_debug_ffn_forward_sharded_group")


def si_ffn_forward_noalloc(handle, layer: int, x, idx, k: int, y, flags: int, status=None, stream=None) -> None:
    """Batch-1 selective FFN through the entry point that allocates nothing: its scratch is a
    fixed array inside the library, so only inputs and outputs are passed."""
    _check(_lib.si_ffn_forward_noalloc(handle, layer, _dp(x), _dp(idx), k, _dp(y), dtype_code(y.dtype), flags,
                                       _dp(status), _stream(stream)), "si_ffn_forward_noalloc")


def si_union(handle, layer: int, T: int, idx, idx_offsets, k_fixed: int, union_out, n_union_out, workspace,
             stream=None) -> None:
    _check(_lib.si_union(handle, layer, T, _dp(idx), _dp(idx_offsets), k_fixed, _dp(union_out), _dp(n_union_out),
                         _dp(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "si_union")


def si_debug_read_bandwidth(mem, nbytes: int, checksum, stream=None) -> None:
    _check(_lib.si_debug_read_bandwidth(_dp(mem), nbytes, _dp(checksum), _stream(stream)), "si_debug_read_bandwidth")


class DecodeOpts(ctypes.Structure):
    """si_debug_decode_opts_t: per-call diagnostics of a persistent decode launch (all zero = none)."""
    _fields_ = [("skip_mask", ctypes.c_int), ("ring_stages", ctypes.c_int), ("step_groups", ctypes.c_int),
                ("withhold", ctypes.c_int), ("chain_form", ctypes.c_int), ("wait_cycles", ctypes.c_longlong),
                ("profile", ctypes.c_void_p)]


def _opts(skip_mask=0, ring_stages=0, step_groups=0, withhold=0, chain_form=0, wait_cycles=0, profile=None) -> DecodeOpts:
    return DecodeOpts(skip_mask, ring_stages, step_groups, withhold, chain_form, wait_cycles,
                      None if profile is None else profile.data_ptr())


def si_debug_decode_stack_forward(handle, n_steps: int, layers, x, idx, idx_offsets, k_fixed: int, y, flags: int,
                                  workspace, status=None, stream=None, **opts) -> None:
    keep, p = _host_i32(layers)
    o = _opts(**opts)
    _check(_lib.si_debug_decode_stack_forward(handle, n_steps, p, _dp(x), _dp(idx), _dp(idx_offsets), k_fixed, _dp(y),
                                              dtype_code(y.dtype), flags, _dp(workspace),
                                              workspace.numel() * workspace.element_size(), _dp(status),
                                              _stream(stream), ctypes.byref(o)), "si_debug_decode_stack_forward")


def si_decode_chain_forward(handle, n_steps: int, layers, chain_len: int, x, idx, idx_offsets, k_fixed: int, y,
                            xn_out, norm_eps: float, flags: int, workspace, status=None, stream=None) -> None:
    keep, p = _host_i32(layers)
    _check(_lib.si_decode_chain_forward(handle, n_steps, p, chain_len, _dp(x), _dp(idx), _dp(idx_offsets), k_fixed,
                                        _dp(y), _dp(xn_out), norm_eps, flags, _dp(workspace),
                                        workspace.numel() * workspace.element_size(), _dp(status), _stream(stream)),
           "si_decode_chain_forward")


def si_decode_prefix_forward(handle, n_steps: int, layers, n_static: int, chain_len: int, x, idx, idx_offsets, k_fixed: int, y,
                             xn_out, norm_eps: float, flags: int, workspace, status=None, stream=None) -> None:
    keep, p = _host_i32(layers)
    _check(_lib.si_decode_prefix_forward(handle, n_steps, p, n_static, chain_len, _dp(x), _dp(idx), _dp(idx_offsets), k_fixed,
                                         _dp(y), dtype_code(y.dtype), _dp(xn_out), norm_eps, flags, _dp(workspace),
                                         workspace.numel() * workspace.element_size(), _dp(status), _stream(stream)),
           "si_decode_prefix_forward")


def si_debug_decode_chain_forward(handle, n_steps: int, layers, chain_len: int, x, idx, idx_offsets, k_fixed: int, y,
                                  xn_out, norm_eps: float, flags: int, workspace, status=None, stream=None,
                                  **opts) -> None:
    keep, p = _host_i32(layers)
    o = _opts(**opts)
    _check(_lib.si_debug_decode_chain_forward(handle, n_steps, p, chain_len, _dp(x), _dp(idx), _dp(idx_offsets),
                                              k_fixed, _dp(y), _dp(xn_out), norm_eps, flags, _dp(workspace),
                                              workspace.numel() * workspace.element_size(), _dp(status),
                                              _stream(stream), ctypes.byref(o)), "si_debug_decode_chain_forward")


def si_debug_union_masks(handle, layer: int, T: int, idx, idx_offsets, k_fixed: int, union_out, n_union_out,
                         masks_out, workspace, stream=None) -> None:
    _check(_lib.si_debug_union_masks(handle, layer, T, _dp(idx), _dp(idx_offsets), k_fixed, _dp(union_out),
                                     _dp(n_union_out), _dp(masks_out), _dp(workspace),
                                     workspace.numel() * workspace.element_size(), _stream(stream)),
           "si_debug_union_masks")


def si_debug_pair_plan(d_model: int, union_cap: int, T: int, num_sms: int) -> dict:
    """Kernel shapes of a call with more than 128 tokens (host logic only, no device needed)."""
    out = (ctypes.c_int * 6)()
    _check(_lib.si_debug_pair_plan(d_model, union_cap, T, num_sms, out), "si_debug_pair_plan")
    return {"gateup_w": out[0], "gateup_sub": out[1], "gateup_pairs": out[2], "down_n": out[3], "down_ksplit": out[4],
            "down_ctas": out[5]}


def si_debug_ffn_forward_waits(handle, layer: int, x, T: int, idx, idx_offsets, k_fixed: int, y, flags: int,
                               workspace, status, spin_limit: int, withhold: int, stream=None) -> None:
    _check(_lib.si_debug_ffn_forward_waits(handle, layer, _dp(x), T, _dp(idx), _dp(idx_offsets), k_fixed, _dp(y),
                                           dtype_code(y.dtype), flags, _dp(workspace),
                                           workspace.numel() * workspace.element_size(), _dp(status),
                                           _stream(stream), spin_limit, withhold), "si_debug_ffn_forward_waits")


# ------------------------------------------------------------------------- owner object

class NeuronStore:
    """Owns the device memory of a store and its handle (allocation and lifetime only)."""

    def __init__(self, n_layers: int, d_model: int, d_ff: int, n_loaded, dtype, device="cuda:0"):
        self.n_layers, self.d_model, self.d_ff = n_layers, d_model, d_ff
        self.n_loaded = [int(v) for v in n_loaded]
        self.dtype = torch_dtype(dtype)
        self.device = torch.device(device)
        nbytes = si_store_bytes(n_layers, d_model, d_ff, self.n_loaded, self.dtype)
        self.mem = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        off = (-self.mem.data_ptr()) % 256
        self.mem_aligned = self.mem[off:off + nbytes]
        with torch.cuda.device(self.device):
            self.handle = si_store_create(self.mem_aligned, n_layers, d_model, d_ff, self.n_loaded, self.dtype)
        self.nbytes = nbytes

    def load(self, layer: int, w_gate, w_up, w_down, neuron_ids, n_base: int = 0) -> None:
        si_load_neurons(self.handle, layer, w_gate, w_up, w_down, neuron_ids, n_base)

    def workspace(self, T_max: int, k_max: int, max_steps: int = 1) -> torch.Tensor:
        nbytes = si_workspace_bytes(self.handle, T_max, k_max, max_steps)
        buf = torch.zeros(nbytes + 256, dtype=torch.uint8, device=self.device)
        off = (-buf.data_ptr()) % 256
        return buf[off:off + nbytes]

    def records(self, layer: int) -> torch.Tensor:
        """[n_loaded, 3, d_model] view of the layer's records (same memory, no copy)."""
        ptr, rb = ctypes.c_void_p(0), ctypes.c_size_t(0)
        _check(_lib.si_store_records(self.handle, layer, ctypes.byref(ptr), ctypes.byref(rb)), "si_store_records")
        off = ptr.value - self.mem_aligned.data_ptr()
        n = self.n_loaded[layer]
        return self.mem_aligned[off:off + n * rb.value].view(self.dtype).view(n, 3, self.d_model)

    def slot_maps(self, layer: int):
        """(slot_to_global int32 [n_loaded], global_to_slot int32 [d_ff]) views."""
        p1, p2 = ctypes.c_void_p(0), ctypes.c_void_p(0)
        n, nb = ctypes.c_int(0), ctypes.c_int(0)
        _check(_lib.si_store_slot_to_global(self.handle, layer, ctypes.byref(p1), ctypes.byref(n), ctypes.byref(nb)),
               "si_store_slot_to_global")
        _check(_lib.si_store_global_to_slot(self.handle, layer, ctypes.byref(p2)), "si_store_global_to_slot")
        base = self.mem_aligned.data_ptr()
        s2g = self.mem_aligned[p1.value - base:p1.value - base + 4 * n.value].view(torch.int32)
        g2s = self.mem_aligned[p2.value - base:p2.value - base + 4 * self.d_ff].view(torch.int32)
        return s2g, g2s

    def close(self) -> None:
        if self.handle is not None:
            si_store_free(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
