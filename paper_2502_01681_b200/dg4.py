"""Thin Python binding of libdg4.so: same names as the C ABI, argument marshalling only.

Every function here forwards to the CUDA library; there is no Python or CPU implementation of any step.
Importing works without a GPU (so that symbols can be checked); calling a compute entry point without the
library or without a CUDA device raises.

Tensors are torch CUDA tensors (used for memory and streams only); index arrays handed to
``dg4_graph_create`` are host numpy int32 arrays.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import numpy as np

from . import build as _build

DG4_OK = 0
DG4_ERR_INVALID_ARG = -1
DG4_ERR_NOT_SORTED = -2
DG4_ERR_BAD_DEGREE = -3
DG4_ERR_BAD_LEVEL = -4
DG4_ERR_UNSUPPORTED = -5
DG4_ERR_ALLOC = -6
DG4_ERR_CUDA = -7
DG4_ERR_TIMEOUT = -8

DG4_F32, DG4_BF16 = 0, 1
DG4_FLAG_RESIDUAL = 1
DG4_FLAG_LEVEL_LAUNCHES = 2
DG4_FLAG_FUSED_LAYER = 4

(DG4_ARR_NBR_PTR, DG4_ARR_NBR_IDX, DG4_ARR_LEVEL_PTR, DG4_ARR_LEVEL_NODES, DG4_ARR_PERM, DG4_ARR_CLASS_PTR,
 DG4_ARR_LEVEL_PERM, DG4_ARR_LEVEL_CLASS_PTR, DG4_ARR_NBR_PAD) = range(9)

EXPORTS = [
    "dg4_status_string", "dg4_last_error", "dg4_launch_count", "dg4_graph_create", "dg4_graph_rebuild", "dg4_graph_destroy",
    "dg4_graph_info", "dg4_graph_export", "dg4_graph_poll_status", "dg4_graph_device_array", "dg4_qkv_project", "dg4_sparse_attn_fwd",
    "dg4_out_project", "dg4_layer_workspace_bytes", "dg4_layer_fwd_parallel", "dg4_layer_fwd_levelised",
    "dg4_layer_fwd_parallel_static", "dg4_static_max_nodes", "dg4_layers_workspace_bytes", "dg4_layers_fwd_levelised",
    "dg4_selftest_bounded_wait", "dg4_sparse_attn_additive_fwd", "dg4_graph_partition",
    "dg4_layernorm_fwd", "dg4_ffn_fwd", "dg4_block_fwd_parallel", "dg4_graph_destroy_async", "dg4_memory_trim",
    "dg4_debug_set_poll_limit", "dg4_debug_override_current_device",
    "dg4_cone_update_workspace_bytes", "dg4_cone_update_fwd", "dg4_block_fwd_levelised",
    "dg4_blocks_workspace_bytes", "dg4_blocks_fwd_levelised",
]


class Dg4Error(RuntimeError):
    def __init__(self, status: int, detail: str):
        super().__init__(f"dg4 status {status}: {detail}")
        self.status = status
        self.detail = detail


class dg4_desc(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("heads", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("flags", ctypes.c_int32), ("scale", ctypes.c_float)]


class dg4_graph_info_t(ctypes.Structure):
    _fields_ = [("n_nodes", ctypes.c_int64), ("n_edges", ctypes.c_int64), ("n_nbr", ctypes.c_int64),
                ("n_levels", ctypes.c_int32), ("max_class", ctypes.c_int32), ("hops", ctypes.c_int32),
                ("perm_chunk", ctypes.c_int32), ("n_chunks", ctypes.c_int32), ("device", ctypes.c_int32)]


_lib = None


def library_path() -> str:
    return _build.LIB


def load():
    """Loads libdg4.so (building it with nvcc if it is missing or stale).  Raises if that is impossible."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.LIB
    if _build.needs_build():
        path = _build.build()
    if not os.path.exists(path):
        raise RuntimeError("libdg4.so is missing and could not be built; there is no fallback path")
    lib = ctypes.CDLL(path)
    vp, i32p, i64 = ctypes.c_void_p, ctypes.POINTER(ctypes.c_int32), ctypes.c_int64
    dp = ctypes.POINTER(dg4_desc)
    lib.dg4_status_string.restype = ctypes.c_char_p
    lib.dg4_status_string.argtypes = [ctypes.c_int]
    lib.dg4_last_error.restype = ctypes.c_char_p
    lib.dg4_last_error.argtypes = []
    lib.dg4_launch_count.restype = ctypes.c_int64
    lib.dg4_launch_count.argtypes = []
    lib.dg4_graph_create.restype = ctypes.c_int
    lib.dg4_graph_create.argtypes = [ctypes.c_int32, i32p, i32p, i32p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                     ctypes.POINTER(vp)]
    lib.dg4_graph_rebuild.restype = ctypes.c_int
    lib.dg4_graph_rebuild.argtypes = [vp, vp]
    lib.dg4_graph_destroy.restype = ctypes.c_int
    lib.dg4_graph_destroy.argtypes = [vp]
    lib.dg4_graph_destroy_async.restype = ctypes.c_int
    lib.dg4_graph_destroy_async.argtypes = [vp, vp]
    lib.dg4_memory_trim.restype = ctypes.c_int
    lib.dg4_memory_trim.argtypes = [ctypes.c_int32]
    lib.dg4_graph_info.restype = ctypes.c_int
    lib.dg4_graph_info.argtypes = [vp, ctypes.POINTER(dg4_graph_info_t)]
    lib.dg4_graph_export.restype = ctypes.c_int
    lib.dg4_graph_export.argtypes = [vp, ctypes.c_int, i32p, i64, ctypes.POINTER(i64)]
    lib.dg4_graph_partition.restype = ctypes.c_int
    lib.dg4_graph_partition.argtypes = [vp, ctypes.c_int32, vp, vp, ctypes.POINTER(i64)]
    lib.dg4_graph_poll_status.restype = ctypes.c_int
    lib.dg4_graph_poll_status.argtypes = [vp, i32p]
    lib.dg4_graph_device_array.restype = vp
    lib.dg4_graph_device_array.argtypes = [vp, ctypes.c_int]
    lib.dg4_qkv_project.restype = ctypes.c_int
    lib.dg4_qkv_project.argtypes = [vp, dp, vp, i64, vp, vp, i64, vp, i64, vp, i64, vp]
    lib.dg4_sparse_attn_fwd.restype = ctypes.c_int
    lib.dg4_sparse_attn_fwd.argtypes = [vp, dp, vp, i64, vp, i64, vp, i64, vp, i64, vp]
    lib.dg4_sparse_attn_additive_fwd.restype = ctypes.c_int
    lib.dg4_sparse_attn_additive_fwd.argtypes = [vp, dp, vp, vp, ctypes.c_float, vp, i64, vp, i64, vp]
    lib.dg4_out_project.restype = ctypes.c_int
    lib.dg4_out_project.argtypes = [vp, dp, vp, i64, vp, vp, i64, vp, i64, vp]
    lib.dg4_layer_workspace_bytes.restype = ctypes.c_size_t
    lib.dg4_layer_workspace_bytes.argtypes = [vp, dp]
    lib.dg4_layer_fwd_parallel.restype = ctypes.c_int
    lib.dg4_layer_fwd_parallel.argtypes = [vp, dp, vp, i64, vp, vp, vp, i64, vp, ctypes.c_size_t, vp]
    lib.dg4_layer_fwd_levelised.restype = ctypes.c_int
    lib.dg4_layer_fwd_levelised.argtypes = [vp, dp, vp, i64, vp, vp, vp, ctypes.c_size_t, vp, vp]
    lib.dg4_layers_workspace_bytes.restype = ctypes.c_size_t
    lib.dg4_layers_workspace_bytes.argtypes = [vp, dp, ctypes.c_int32]
    lib.dg4_layers_fwd_levelised.restype = ctypes.c_int
    lib.dg4_layers_fwd_levelised.argtypes = [vp, dp, vp, i64, ctypes.c_int32, ctypes.POINTER(vp), ctypes.POINTER(vp), vp,
                                             ctypes.c_size_t, vp, vp]
    lib.dg4_selftest_bounded_wait.restype = ctypes.c_int
    lib.dg4_selftest_bounded_wait.argtypes = [vp, vp]
    lib.dg4_layer_fwd_parallel_static.restype = ctypes.c_int
    lib.dg4_layer_fwd_parallel_static.argtypes = [vp, dp, vp, i64, vp, vp, vp, i64, vp]
    lib.dg4_static_max_nodes.restype = ctypes.c_int64
    lib.dg4_static_max_nodes.argtypes = []
    cf = ctypes.c_float
    lib.dg4_layernorm_fwd.restype = ctypes.c_int
    lib.dg4_layernorm_fwd.argtypes = [vp, dp, vp, i64, vp, vp, cf, vp, i64, vp]
    lib.dg4_ffn_fwd.restype = ctypes.c_int
    lib.dg4_ffn_fwd.argtypes = [vp, dp, vp, i64, vp, vp, vp, vp, vp, vp, cf, ctypes.c_int32, vp, i64, vp]
    lib.dg4_block_fwd_parallel.restype = ctypes.c_int
    lib.dg4_block_fwd_parallel.argtypes = [vp, dp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, cf, ctypes.c_int32,
                                           vp, i64, vp, ctypes.c_size_t, vp]
    lib.dg4_block_fwd_levelised.restype = ctypes.c_int
    lib.dg4_block_fwd_levelised.argtypes = [vp, dp, vp, i64, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, cf, ctypes.c_int32,
                                            vp, ctypes.c_size_t, vp]
    lib.dg4_blocks_workspace_bytes.restype = ctypes.c_size_t
    lib.dg4_blocks_workspace_bytes.argtypes = [vp, dp, ctypes.c_int32]
    pvp = ctypes.POINTER(vp)
    lib.dg4_blocks_fwd_levelised.restype = ctypes.c_int
    lib.dg4_blocks_fwd_levelised.argtypes = [vp, dp, vp, i64, ctypes.c_int32, pvp, pvp, pvp, pvp, pvp, pvp, pvp, pvp, pvp, pvp,
                                             cf, ctypes.c_int32, vp, ctypes.c_size_t, vp]
    lib.dg4_cone_update_workspace_bytes.restype = ctypes.c_size_t
    lib.dg4_cone_update_workspace_bytes.argtypes = [vp, dp, ctypes.c_int32]
    lib.dg4_cone_update_fwd.restype = ctypes.c_int
    lib.dg4_cone_update_fwd.argtypes = [vp, dp, vp, i64, ctypes.c_int32, ctypes.POINTER(vp), ctypes.POINTER(vp),
                                        ctypes.c_int32, ctypes.c_int32, vp, ctypes.c_size_t, vp, ctypes.POINTER(i64), vp]
    lib.dg4_debug_set_poll_limit.restype = None
    lib.dg4_debug_set_poll_limit.argtypes = [ctypes.c_uint32]
    lib.dg4_debug_override_current_device.restype = None
    lib.dg4_debug_override_current_device.argtypes = [ctypes.c_int32]
    _lib = lib
    return lib


def _check(status: int):
    if status != DG4_OK:
        raise Dg4Error(status, load().dg4_last_error().decode())


def _i32(a):
    a = np.ascontiguousarray(a, np.int32)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _stream(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    return ctypes.c_void_p(int(getattr(stream, "cuda_stream", stream)))     # a raw handle or a torch stream


def _ptr(t):
    return ctypes.c_void_p(t.data_ptr()) if t is not None else None


def _ld(t):
    assert t.dim() == 2 and t.stride(1) == 1, "tensors are [rows, d] with unit inner stride"
    return int(t.stride(0))


def desc(heads: int, dtype: int, scale: float, residual: bool = False, d: int = 128,
         level_launches: bool = False, fused_layer: bool = False) -> dg4_desc:
    flags = ((DG4_FLAG_RESIDUAL if residual else 0) | (DG4_FLAG_LEVEL_LAUNCHES if level_launches else 0)
             | (DG4_FLAG_FUSED_LAYER if fused_layer else 0))
    return dg4_desc(d, heads, dtype, flags, float(scale))


@dataclass
class Graph:
    """Owner of a dg4_graph handle (destroyed with the object)."""
    handle: ctypes.c_void_p
    info: dg4_graph_info_t

    def __del__(self):
        try:
            if self.handle:
                load().dg4_graph_destroy(self.handle)
                self.handle = None
        except Exception:
            pass

    @property
    def n(self) -> int:
        return int(self.info.n_nodes)


def dg4_launch_count() -> int:
    return int(load().dg4_launch_count())


def dg4_graph_create(row_ptr, col_idx, level, hops: int, perm_chunk: int = 0, device: int = 0) -> Graph:
    lib = load()
    rp, rpp = _i32(row_ptr)
    ci, cip = _i32(col_idx)
    lv, lvp = _i32(level)
    h = ctypes.c_void_p()
    _check(lib.dg4_graph_create(rp.shape[0] - 1, rpp, cip, lvp, hops, perm_chunk, device, ctypes.byref(h)))
    info = dg4_graph_info_t()
    _check(lib.dg4_graph_info(h, ctypes.byref(info)))
    return Graph(h, info)


def dg4_graph_rebuild(g: Graph, stream=None):
    _check(load().dg4_graph_rebuild(g.handle, _stream(stream)))


def dg4_graph_destroy(g: Graph):
    if g.handle:
        _check(load().dg4_graph_destroy(g.handle))
        g.handle = None


def dg4_graph_destroy_async(g: Graph, stream=None):
    """Frees the handle in the order of `stream` (work enqueued there before may still use it); does not wait."""
    if g.handle:
        _check(load().dg4_graph_destroy_async(g.handle, _stream(stream)))
        g.handle = None


def dg4_memory_trim(device: int = 0):
    _check(load().dg4_memory_trim(device))


def dg4_graph_info(g: Graph) -> dg4_graph_info_t:
    info = dg4_graph_info_t()
    _check(load().dg4_graph_info(g.handle, ctypes.byref(info)))
    return info


def dg4_graph_export(g: Graph, which: int) -> np.ndarray:
    lib = load()
    n = ctypes.c_int64()
    _check(lib.dg4_graph_export(g.handle, which, None, 0, ctypes.byref(n)))
    out = np.zeros(max(int(n.value), 1), np.int32)
    _check(lib.dg4_graph_export(g.handle, which, out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), out.shape[0],
                                ctypes.byref(n)))
    return out[:n.value]


def dg4_graph_poll_status(g: Graph) -> int:
    out = ctypes.c_int32(0)
    _check(load().dg4_graph_poll_status(g.handle, ctypes.byref(out)))
    return int(out.value)


def dg4_graph_device_array(g: Graph, which: int) -> int:
    return int(load().dg4_graph_device_array(g.handle, which) or 0)


def dg4_qkv_project(g: Graph, dsc: dg4_desc, X, W_qkv, Q, K, V, stream=None):
    _check(load().dg4_qkv_project(g.handle, ctypes.byref(dsc), _ptr(X), _ld(X), _ptr(W_qkv), _ptr(Q), _ld(Q),
                                  _ptr(K), _ld(K), _ptr(V), _ld(V), _stream(stream)))


def dg4_sparse_attn_fwd(g: Graph, dsc: dg4_desc, Q, K, V, O, stream=None):
    _check(load().dg4_sparse_attn_fwd(g.handle, ctypes.byref(dsc), _ptr(Q), _ld(Q), _ptr(K), _ld(K), _ptr(V), _ld(V),
                                      _ptr(O), _ld(O), _stream(stream)))


def dg4_out_project(g: Graph, dsc: dg4_desc, O, W_o, H_res, H_out, stream=None):
    _check(load().dg4_out_project(g.handle, ctypes.byref(dsc), _ptr(O), _ld(O), _ptr(W_o), _ptr(H_res),
                                  _ld(H_res) if H_res is not None else 0, _ptr(H_out), _ld(H_out), _stream(stream)))


def dg4_layer_workspace_bytes(g: Graph, dsc: dg4_desc) -> int:
    return int(load().dg4_layer_workspace_bytes(g.handle, ctypes.byref(dsc)))


def dg4_layer_fwd_parallel(g: Graph, dsc: dg4_desc, H_in, W_qkv, W_o, H_out, workspace, stream=None):
    _check(load().dg4_layer_fwd_parallel(g.handle, ctypes.byref(dsc), _ptr(H_in), _ld(H_in), _ptr(W_qkv), _ptr(W_o),
                                         _ptr(H_out), _ld(H_out), _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)))


def dg4_layer_fwd_levelised(g: Graph, dsc: dg4_desc, H, W_qkv, W_o, workspace, device_status=None, stream=None):
    _check(load().dg4_layer_fwd_levelised(g.handle, ctypes.byref(dsc), _ptr(H), _ld(H), _ptr(W_qkv), _ptr(W_o),
                                          _ptr(workspace), workspace.numel() * workspace.element_size(),
                                          _ptr(device_status), _stream(stream)))


def dg4_static_max_nodes() -> int:
    return int(load().dg4_static_max_nodes())


def dg4_layer_fwd_parallel_static(g: Graph, dsc: dg4_desc, H_in, W_qkv, W_o, H_out, stream=None):
    """The parallel layer without a workspace argument: its scratch is a fixed array inside the library, for
    callers that cannot allocate device memory.  Graphs above dg4_static_max_nodes() are rejected; calls must
    not overlap on the GPU."""
    _check(load().dg4_layer_fwd_parallel_static(g.handle, ctypes.byref(dsc), _ptr(H_in), _ld(H_in), _ptr(W_qkv),
                                                _ptr(W_o), _ptr(H_out), _ld(H_out), _stream(stream)))


def dg4_layers_workspace_bytes(g: Graph, dsc: dg4_desc, n_layers: int) -> int:
    return int(load().dg4_layers_workspace_bytes(g.handle, ctypes.byref(dsc), n_layers))


def dg4_layers_fwd_levelised(g: Graph, dsc: dg4_desc, H, W_qkv_list, W_o_list, workspace, device_status=None,
                             stream=None):
    """Several levelised layers in one call (same result as one dg4_layer_fwd_levelised call per layer)."""
    n = len(W_qkv_list)
    assert n == len(W_o_list)
    arr = ctypes.c_void_p * n
    wq = arr(*[t.data_ptr() for t in W_qkv_list])
    wo = arr(*[t.data_ptr() for t in W_o_list])
    _check(load().dg4_layers_fwd_levelised(g.handle, ctypes.byref(dsc), _ptr(H), _ld(H), n, wq, wo, _ptr(workspace),
                                           workspace.numel() * workspace.element_size(), _ptr(device_status),
                                           _stream(stream)))


def dg4_selftest_bounded_wait(device_status, stream=None):
    _check(load().dg4_selftest_bounded_wait(_ptr(device_status), _stream(stream)))


def dg4_cone_update_workspace_bytes(g: Graph, dsc: dg4_desc, batch: int) -> int:
    return int(load().dg4_cone_update_workspace_bytes(g.handle, ctypes.byref(dsc), int(batch)))


def dg4_cone_update_fwd(g: Graph, dsc: dg4_desc, H, W_qkv_list, W_o_list, delta: int, batch: int, workspace,
                        stored=None, stream=None) -> int:
    """Sec. 3.4's updating strategy over Algorithm 1's partition (cone mini-batches against the table H, updated in
    place).  Returns the number of mini-batches."""
    n = len(W_qkv_list)
    assert n == len(W_o_list)
    arr = ctypes.c_void_p * n
    wq = arr(*[t.data_ptr() for t in W_qkv_list])
    wo = arr(*[t.data_ptr() for t in W_o_list])
    nb = ctypes.c_int64(0)
    _check(load().dg4_cone_update_fwd(g.handle, ctypes.byref(dsc), _ptr(H), _ld(H), n, wq, wo, int(delta), int(batch),
                                      _ptr(workspace), workspace.numel() * workspace.element_size(), _ptr(stored),
                                      ctypes.byref(nb), _stream(stream)))
    return int(nb.value)


def dg4_debug_set_poll_limit(polls: int):
    """Poll limit of the device-side waits for the launches that follow (0 = default); see dg4.h."""
    load().dg4_debug_set_poll_limit(int(polls))


def dg4_debug_override_current_device(device: int):
    """Makes the forward calls' device check on this thread behave as if `device` were current (-1 = off)."""
    load().dg4_debug_override_current_device(int(device))


def dg4_sparse_attn_additive_fwd(g: Graph, dsc: dg4_desc, S_dst, S_src, negative_slope, V, O, stream=None):
    assert S_dst.is_contiguous() and S_src.is_contiguous()
    _check(load().dg4_sparse_attn_additive_fwd(g.handle, ctypes.byref(dsc), _ptr(S_dst), _ptr(S_src),
                                               float(negative_slope), _ptr(V), _ld(V), _ptr(O), _ld(O), _stream(stream)))


def dg4_layernorm_fwd(g: Graph, dsc: dg4_desc, X, gamma, beta, eps, Y, stream=None):
    _check(load().dg4_layernorm_fwd(g.handle, ctypes.byref(dsc), _ptr(X), _ld(X), _ptr(gamma), _ptr(beta),
                                    ctypes.c_float(eps), _ptr(Y), _ld(Y), _stream(stream)))


def dg4_ffn_fwd(g: Graph, dsc: dg4_desc, X, W1, b1, W2, b2, gamma, beta, eps, Y, stream=None):
    """Y = LayerNorm(X + max(0, X W1^T + b1) W2^T + b2); W1 [512, 128] and W2 [128, 512] bf16, vectors fp32."""
    _check(load().dg4_ffn_fwd(g.handle, ctypes.byref(dsc), _ptr(X), _ld(X), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2),
                              _ptr(gamma), _ptr(beta), ctypes.c_float(eps), int(W1.shape[0]), _ptr(Y), _ld(Y),
                              _stream(stream)))


def dg4_block_fwd_parallel(g: Graph, dsc: dg4_desc, H_in, W_qkv, W_o, ln1_gamma, ln1_beta, W1, b1, W2, b2, ln2_gamma,
                           ln2_beta, eps, H_out, workspace, stream=None):
    """One whole block (attention sub-layer, LayerNorm, feed-forward sub-layer, LayerNorm) on all nodes at once."""
    _check(load().dg4_block_fwd_parallel(g.handle, ctypes.byref(dsc), _ptr(H_in), _ld(H_in), _ptr(W_qkv), _ptr(W_o),
                                         _ptr(ln1_gamma), _ptr(ln1_beta), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2),
                                         _ptr(ln2_gamma), _ptr(ln2_beta), ctypes.c_float(eps), int(W1.shape[0]),
                                         _ptr(H_out), _ld(H_out), _ptr(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)))


def dg4_block_fwd_levelised(g: Graph, dsc: dg4_desc, H, W_qkv, W_o, ln1_gamma, ln1_beta, W1, b1, W2, b2, ln2_gamma,
                            ln2_beta, eps, workspace, stream=None):
    """One whole block in level-by-level order, in place on H (one group of launches per level)."""
    _check(load().dg4_block_fwd_levelised(g.handle, ctypes.byref(dsc), _ptr(H), _ld(H), _ptr(W_qkv), _ptr(W_o),
                                          _ptr(ln1_gamma), _ptr(ln1_beta), _ptr(W1), _ptr(b1), _ptr(W2), _ptr(b2),
                                          _ptr(ln2_gamma), _ptr(ln2_beta), ctypes.c_float(eps), int(W1.shape[0]),
                                          _ptr(workspace), workspace.numel() * workspace.element_size(),
                                          _stream(stream)))


def dg4_blocks_workspace_bytes(g: Graph, dsc: dg4_desc, n_blocks: int) -> int:
    return int(load().dg4_blocks_workspace_bytes(g.handle, ctypes.byref(dsc), n_blocks))


def dg4_blocks_fwd_levelised(g: Graph, dsc: dg4_desc, H, blocks, eps, workspace, stream=None):
    """Several whole blocks level by level as one wavefront, in place on H.  `blocks`: one tuple per block,
    (W_qkv, W_o, ln1_gamma, ln1_beta, W1, b1, W2, b2, ln2_gamma, ln2_beta), device tensors."""
    n = len(blocks)
    arr = ctypes.c_void_p * n
    cols = [arr(*[blk[i].data_ptr() for blk in blocks]) for i in range(10)]
    _check(load().dg4_blocks_fwd_levelised(g.handle, ctypes.byref(dsc), _ptr(H), _ld(H), n, *cols, ctypes.c_float(eps),
                                           int(blocks[0][4].shape[0]), _ptr(workspace),
                                           workspace.numel() * workspace.element_size(), _stream(stream)))


def dg4_graph_partition(g: Graph, delta: int):
    """Algorithm 1: returns (roots, group_ptr) as CUDA int32 tensors (roots trimmed to their number)."""
    import torch
    roots = torch.empty(g.n, dtype=torch.int32, device="cuda")
    group_ptr = torch.empty(int(g.info.n_levels) + 1, dtype=torch.int32, device="cuda")
    m = ctypes.c_int64(0)
    _check(load().dg4_graph_partition(g.handle, int(delta), _ptr(roots), _ptr(group_ptr), ctypes.byref(m)))
    return roots[: m.value], group_ptr
