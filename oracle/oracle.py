"""ctypes front-end of the CPU checker (``dg4_oracle.cpp``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the benchmark's CPU-baseline
leg.  The CUDA library and its Python binding never import this module.

All tensors are numpy float64, row-major; index arrays are int32.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dg4_oracle.cpp")
_LIB = os.path.join(_HERE, "_dg4oracle.so")
_lib = None

_f64p = ctypes.POINTER(ctypes.c_double)
_i32p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["g++", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", _LIB, _SRC])
    return _LIB


def _load():
    global _lib
    if _lib is None:
        # DG4_ORACLE_LIB: used only by tests/test_oracle_mutants.py, which checks that the pins reject deliberately
        # broken builds of the checker
        lib = ctypes.CDLL(os.environ.get("DG4_ORACLE_LIB") or build())
        c_int, c_dbl = ctypes.c_int, ctypes.c_double
        lib.orc_round_bf16.restype = c_dbl
        lib.orc_round_bf16.argtypes = [c_dbl]
        lib.orc_round_bf16_array.restype = None
        lib.orc_round_bf16_array.argtypes = [_f64p, _f64p, ctypes.c_int64]
        lib.orc_levels.restype = c_int
        lib.orc_levels.argtypes = [c_int, _i32p, _i32p, _i32p]
        lib.orc_neighbourhood.restype = ctypes.c_int64
        lib.orc_neighbourhood.argtypes = [c_int, _i32p, _i32p, c_int, _i32p, _i32p]
        lib.orc_level_buckets.restype = c_int
        lib.orc_level_buckets.argtypes = [c_int, _i32p, c_int, _i32p, _i32p]
        lib.orc_class_order.restype = c_int
        lib.orc_class_order.argtypes = [c_int, _i32p, c_int, _i32p, _i32p, c_int, _i32p, _i32p]
        lib.orc_partition_roots.restype = c_int
        lib.orc_partition_roots.argtypes = [c_int, _i32p, _i32p, _i32p, c_int, c_int, c_int, _i32p, _i32p]
        lib.orc_attention.restype = None
        lib.orc_attention.argtypes = [c_int, c_int, c_int, c_dbl, _f64p, _f64p, _f64p, _i32p, _i32p, _f64p, _f64p]
        lib.orc_attention_additive.restype = None
        lib.orc_attention_additive.argtypes = [c_int, c_int, c_int, c_dbl, _f64p, _f64p, _f64p, _i32p, _i32p, _f64p, _f64p]
        lib.orc_project.restype = None
        lib.orc_project.argtypes = [c_int, c_int, c_int, _f64p, _f64p, _f64p, _f64p]
        lib.orc_layernorm.restype = None
        lib.orc_layernorm.argtypes = [c_int, c_int, _f64p, _f64p, _f64p, c_dbl, _f64p]
        lib.orc_ffn.restype = None
        lib.orc_ffn.argtypes = [c_int, c_int, c_int, _f64p, _f64p, _f64p, _f64p, _f64p, _f64p, _f64p, c_dbl, c_int, _f64p]
        lib.orc_layer_parallel.restype = None
        lib.orc_layer_parallel.argtypes = [c_int, c_int, c_int, c_dbl, _f64p, _f64p, _f64p, c_int, _i32p, _i32p,
                                           c_int, _f64p]
        lib.orc_layer_levelised.restype = None
        lib.orc_layer_levelised.argtypes = [c_int, c_int, c_int, c_dbl, _f64p, _f64p, _f64p, c_int, _i32p, _i32p,
                                            c_int, _i32p, _i32p, c_int]
        lib.orc_block_levelised.restype = None
        lib.orc_block_levelised.argtypes = [c_int, c_int, c_int, c_dbl, _f64p, _f64p, _f64p, _f64p, _f64p, c_int, _f64p, _f64p,
                                            _f64p, _f64p, _f64p, _f64p, c_dbl, _i32p, _i32p, c_int, _i32p, _i32p, c_int]
        lib.orc_cone_update.restype = c_int
        lib.orc_cone_update.argtypes = [c_int, c_int, c_int, c_dbl, c_int, _f64p, _f64p, _f64p, c_int, _i32p, _i32p, _i32p,
                                        c_int, c_int, c_int, c_int, c_int, _f64p, _i32p]
        lib.orc_num_threads.restype = c_int
        _lib = lib
    return _lib


def _d(a):
    return a.ctypes.data_as(_f64p) if a is not None else None


def _i(a):
    return a.ctypes.data_as(_i32p) if a is not None else None


def _f64(a):
    return np.ascontiguousarray(a, np.float64)


def _i32(a):
    return np.ascontiguousarray(a, np.int32)


ROUND = {"none": 0, None: 0, "bf16": 1, "f32": 2}


def num_threads() -> int:
    return int(_load().orc_num_threads())


def round_bf16(x):
    """Nearest bfloat16 (ties to even) of each fp64 value, as fp64."""
    a = _f64(x)
    out = np.empty_like(a)
    _load().orc_round_bf16_array(_d(a), _d(out), a.size)
    return out


def levels(row_ptr, col_idx):
    """Eq. 1: logic level of every node."""
    row_ptr, col_idx = _i32(row_ptr), _i32(col_idx)
    n = row_ptr.shape[0] - 1
    out = np.zeros(n, np.int32)
    if _load().orc_levels(n, _i(row_ptr), _i(col_idx), _i(out)) != 0:
        raise ValueError("node ids are not a topological order")
    return out


def neighbourhood(row_ptr, col_idx, hops):
    """cone_k(v) lists: self first, then ascending id.  Returns (nbr_ptr, nbr_idx)."""
    row_ptr, col_idx = _i32(row_ptr), _i32(col_idx)
    n = row_ptr.shape[0] - 1
    nbr_ptr = np.zeros(n + 1, np.int32)
    total = _load().orc_neighbourhood(n, _i(row_ptr), _i(col_idx), hops, _i(nbr_ptr), None)
    nbr_idx = np.zeros(max(int(total), 1), np.int32)
    _load().orc_neighbourhood(n, _i(row_ptr), _i(col_idx), hops, _i(nbr_ptr), _i(nbr_idx))
    return nbr_ptr, nbr_idx[:total]


def level_buckets(level):
    """Nodes ordered by (level, id).  Returns (level_ptr[n_levels+1], level_nodes[n])."""
    level = _i32(level)
    n = level.shape[0]
    n_levels = int(level.max()) + 1 if n else 0
    level_ptr = np.zeros(n_levels + 1, np.int32)
    level_nodes = np.zeros(n, np.int32)
    _load().orc_level_buckets(n, _i(level), n_levels, _i(level_ptr), _i(level_nodes))
    return level_ptr, level_nodes


def class_order(seq, seg_ptr, nbr_ptr, max_class):
    """Reorder each segment of ``seq`` by (|neighbourhood|, id).  Returns (perm, class_ptr[n_seg, max_class+1])."""
    seq, seg_ptr, nbr_ptr = _i32(seq), _i32(seg_ptr), _i32(nbr_ptr)
    n, n_seg = seq.shape[0], seg_ptr.shape[0] - 1
    perm = np.zeros(n, np.int32)
    class_ptr = np.zeros((n_seg, max_class + 1), np.int32)
    _load().orc_class_order(n, _i(seq), n_seg, _i(seg_ptr), _i(nbr_ptr), max_class, _i(perm), _i(class_ptr))
    return perm, class_ptr


def partition_roots(row_ptr, col_idx, level, k, delta):
    """Algorithm 1: roots of the partition's cones, grouped by level.  Returns (roots, group_ptr[n_levels+1])."""
    row_ptr, col_idx, level = _i32(row_ptr), _i32(col_idx), _i32(level)
    n = level.shape[0]
    n_levels = int(level.max()) + 1
    roots = np.zeros(n, np.int32)
    group_ptr = np.zeros(n_levels + 1, np.int32)
    m = _load().orc_partition_roots(n, _i(row_ptr), _i(col_idx), _i(level), n_levels, int(k), int(delta), _i(roots),
                                    _i(group_ptr))
    return roots[:m].copy(), group_ptr


def chunk_ptr(n, chunk):
    """Segment boundaries of consecutive id chunks (chunk <= 0: one segment)."""
    if chunk <= 0 or chunk >= n:
        return np.array([0, n], np.int32)
    b = list(range(0, n, chunk)) + [n]
    return np.array(b, np.int32)


def attention(Q, K, V, nbr_ptr, nbr_idx, heads, scale, return_alpha=False):
    """Q: [n, d]; K, V: [n_kv, d]; neighbour ids index K / V rows."""
    Q, K, V = _f64(Q), _f64(K), _f64(V)
    nbr_ptr, nbr_idx = _i32(nbr_ptr), _i32(nbr_idx)
    n, d = Q.shape
    assert nbr_ptr.shape[0] == n + 1 and (nbr_idx.size == 0 or nbr_idx.max() < K.shape[0])
    O = np.zeros((n, d), np.float64)
    alpha = np.zeros((nbr_idx.shape[0], heads), np.float64) if return_alpha else None
    _load().orc_attention(n, d, heads, float(scale), _d(Q), _d(K), _d(V), _i(nbr_ptr), _i(nbr_idx), _d(O), _d(alpha))
    return (O, alpha) if return_alpha else O


def attention_additive(S_dst, S_src, V, nbr_ptr, nbr_idx, slope=0.2, return_alpha=False):
    """GAT-style additive scores: e = LeakyReLU(S_src[u,h] + S_dst[v,h]).  S_dst: [n, heads]; S_src: [n_kv, heads];
    V: [n_kv, d]."""
    S_dst, S_src, V = _f64(S_dst), _f64(S_src), _f64(V)
    nbr_ptr, nbr_idx = _i32(nbr_ptr), _i32(nbr_idx)
    n, heads = S_dst.shape
    d = V.shape[1]
    assert nbr_ptr.shape[0] == n + 1 and S_src.shape == (V.shape[0], heads)
    O = np.zeros((n, d), np.float64)
    alpha = np.zeros((nbr_idx.shape[0], heads), np.float64) if return_alpha else None
    _load().orc_attention_additive(n, d, heads, float(slope), _d(S_dst), _d(S_src), _d(V), _i(nbr_ptr), _i(nbr_idx),
                                   _d(O), _d(alpha))
    return (O, alpha) if return_alpha else O


def project(X, W, R=None):
    X, W = _f64(X), _f64(W)
    R = _f64(R) if R is not None else None
    n, d_in = X.shape
    d_out = W.shape[0]
    Y = np.zeros((n, d_out), np.float64)
    _load().orc_project(n, d_in, d_out, _d(X), _d(W), _d(R), _d(Y))
    return Y


def layernorm(X, gamma, beta, eps=1e-5):
    """Row-wise layer normalisation (biased variance over the features of a row)."""
    X, gamma, beta = _f64(X), _f64(gamma), _f64(beta)
    n, d = X.shape
    Y = np.zeros((n, d), np.float64)
    _load().orc_layernorm(n, d, _d(X), _d(gamma), _d(beta), float(eps), _d(Y))
    return Y


def ffn(X, W1, b1, W2, b2, gamma, beta, eps=1e-5, rounding=None):
    """LayerNorm(X + max(0, X W1^T + b1) W2^T + b2); W1 [d_ff, d], W2 [d, d_ff]."""
    X, W1, b1, W2, b2, gamma, beta = (_f64(a) for a in (X, W1, b1, W2, b2, gamma, beta))
    n, d = X.shape
    d_ff = W1.shape[0]
    assert W1.shape == (d_ff, d) and W2.shape == (d, d_ff) and b1.shape == (d_ff,) and b2.shape == (d,)
    Y = np.zeros((n, d), np.float64)
    _load().orc_ffn(n, d, d_ff, _d(X), _d(W1), _d(b1), _d(W2), _d(b2), _d(gamma), _d(beta), float(eps),
                    ROUND[rounding], _d(Y))
    return Y


def layer_parallel(X, W_qkv, W_o, nbr_ptr, nbr_idx, heads, scale, residual=True, rounding=None):
    X, W_qkv, W_o = _f64(X), _f64(W_qkv), _f64(W_o)
    nbr_ptr, nbr_idx = _i32(nbr_ptr), _i32(nbr_idx)
    n, d = X.shape
    H = np.zeros((n, d), np.float64)
    _load().orc_layer_parallel(n, d, heads, float(scale), _d(X), _d(W_qkv), _d(W_o), int(bool(residual)),
                               _i(nbr_ptr), _i(nbr_idx), ROUND[rounding], _d(H))
    return H


def layer_levelised(H, W_qkv, W_o, nbr_ptr, nbr_idx, level_ptr, level_nodes, heads, scale, residual=True,
                    rounding=None):
    H = _f64(H).copy()
    W_qkv, W_o = _f64(W_qkv), _f64(W_o)
    nbr_ptr, nbr_idx, level_ptr, level_nodes = _i32(nbr_ptr), _i32(nbr_idx), _i32(level_ptr), _i32(level_nodes)
    n, d = H.shape
    _load().orc_layer_levelised(n, d, heads, float(scale), _d(H), _d(W_qkv), _d(W_o), int(bool(residual)),
                                _i(nbr_ptr), _i(nbr_idx), level_ptr.shape[0] - 1, _i(level_ptr), _i(level_nodes),
                                ROUND[rounding])
    return H


def block_levelised(H, W_qkv, W_o, ln1_gamma, ln1_beta, W1, b1, W2, b2, ln2_gamma, ln2_beta, nbr_ptr, nbr_idx, level_ptr,
                    level_nodes, heads, scale, eps=1e-5, rounding=None):
    """The whole block (attention sub-layer + LayerNorm, feed-forward sub-layer + LayerNorm) level by level."""
    H = _f64(H).copy()
    W_qkv, W_o, W1, W2 = _f64(W_qkv), _f64(W_o), _f64(W1), _f64(W2)
    g1, be1, b1, b2, g2, be2 = (_f64(a) for a in (ln1_gamma, ln1_beta, b1, b2, ln2_gamma, ln2_beta))
    nbr_ptr, nbr_idx, level_ptr, level_nodes = _i32(nbr_ptr), _i32(nbr_idx), _i32(level_ptr), _i32(level_nodes)
    n, d = H.shape
    _load().orc_block_levelised(n, d, heads, float(scale), _d(H), _d(W_qkv), _d(W_o), _d(g1), _d(be1), W1.shape[0],
                                _d(W1), _d(b1), _d(W2), _d(b2), _d(g2), _d(be2), float(eps), _i(nbr_ptr), _i(nbr_idx),
                                level_ptr.shape[0] - 1, _i(level_ptr), _i(level_nodes), ROUND[rounding])
    return H


def cone_update(X, W_qkv_list, W_o_list, row_ptr, col_idx, level, k, delta, batch, heads, scale, residual=True,
                rounding=None):
    """Sec. 3.4's updating strategy over Algorithm 1's partition (cone mini-batches against a table of historical
    embeddings) for a stack of layers.  Returns (table [n, d], stored [n] = times each row was stored, n_batches)."""
    X = _f64(X)
    Wq = _f64(np.stack([_f64(w) for w in W_qkv_list]))
    Wo = _f64(np.stack([_f64(w) for w in W_o_list]))
    row_ptr, col_idx, level = _i32(row_ptr), _i32(col_idx), _i32(level)
    n, d = X.shape
    hist = np.zeros((n, d), np.float64)
    stored = np.zeros(n, np.int32)
    nb = _load().orc_cone_update(n, d, heads, float(scale), Wq.shape[0], _d(X), _d(Wq), _d(Wo), int(bool(residual)),
                                 _i(row_ptr), _i(col_idx), _i(level), int(level.max()) + 1, int(k), int(delta),
                                 int(batch), ROUND[rounding], _d(hist), _i(stored))
    return hist, stored, int(nb)
