"""Small graph builders and comparison helpers shared by the tests (no layer arithmetic here)."""
import numpy as np


def csr_from_fanins(fanins):
    """fanins: list over nodes of lists of source ids -> (row_ptr, col_idx) int32, sources ascending."""
    row_ptr = [0]
    col = []
    for f in fanins:
        col.extend(sorted(f))
        row_ptr.append(len(col))
    return np.array(row_ptr, np.int32), np.array(col, np.int32)


def binary_in_tree(depth):
    """Complete binary in-tree: leaves are primary inputs, root is the last node; ids are topological.
    Returns (fanins, root, levels)."""
    counts = [2 ** (depth - l) for l in range(depth + 1)]
    start = np.concatenate([[0], np.cumsum(counts)])
    fanins, levels = [], []
    for l, c in enumerate(counts):
        for i in range(c):
            if l == 0:
                fanins.append([])
            else:
                fanins.append([int(start[l - 1] + 2 * i), int(start[l - 1] + 2 * i + 1)])
            levels.append(l)
    return fanins, len(fanins) - 1, np.array(levels, np.int32)


def random_dag(rng, n_pi, n_gates, window=8, not_ratio=0.3):
    """Tiny random AIG-like DAG built with numpy's RNG (independent of the C generator).  An AND may
    draw the same source twice (both inputs tied to one node)."""
    fanins = [[] for _ in range(n_pi)]
    for i in range(n_pi, n_pi + n_gates):
        lo = max(0, i - window)
        if rng.random() < not_ratio:
            fanins.append([int(rng.integers(lo, i))])
        else:
            fanins.append([int(rng.integers(lo, i)), int(rng.integers(lo, i))])
    return fanins


def levels_of(fanins):
    lv = []
    for f in fanins:
        lv.append(0 if not f else 1 + max(lv[u] for u in f))
    return np.array(lv, np.int32)


def rel_row_err(got, want):
    """Per-row ||got - want||_2 / ||want||_2 (rows with tiny norm compared absolutely)."""
    got = np.asarray(got, np.float64)
    want = np.asarray(want, np.float64)
    num = np.linalg.norm(got - want, axis=1)
    den = np.linalg.norm(want, axis=1)
    return num / np.maximum(den, 1e-30)
