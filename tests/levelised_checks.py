"""Checks of a levelised layer's result that the checker can afford at any size (used by the full-size GPU tests;
exercised on the CPU, with the checker's own result standing in for the GPU's, by tests/test_levelised_checks_cpu.py)."""
import numpy as np

from oracle import oracle as orc
from tests.gpu_util import f64_of_bits
from tests.helpers import rel_row_err


def every_step_check(ptr, idx, rows, in_bits, out_bits, wq, wo, heads, scale, chunk=400_000):
    """One levelised layer, checked STEP BY STEP on the given rows: the checker recomputes each node's new row
    from the layer's input row of the node itself (its query and its own key / value) and from the GPU's final
    rows of the other members of its neighbourhood (all on lower levels, hence final when the node is computed).
    Every node is thereby checked against exactly the inputs the levelised order prescribes, so a stale read on
    any level is a mismatch; what this does NOT measure is how rounding differences add up over many levels
    (the end-to-end comparisons do that).  Returns the per-row relative errors."""
    rows = np.asarray(rows, np.int64)
    errs = np.zeros(rows.shape[0])
    for lo in range(0, rows.shape[0], chunk):
        part = rows[lo:lo + chunk]
        starts, sizes = ptr[part].astype(np.int64), (ptr[part + 1] - ptr[part]).astype(np.int64)
        lptr = np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)
        take = np.repeat(starts - lptr[:-1], sizes) + np.arange(lptr[-1])
        members = idx[take]                                  # the lists of these rows, back to back (self first)
        is_self = np.zeros(members.shape[0], bool)
        is_self[lptr[:-1]] = True
        others = np.unique(members[~is_self])
        lidx = np.where(is_self, np.repeat(np.arange(part.shape[0]), sizes),
                        part.shape[0] + np.searchsorted(others, members)).astype(np.int32)
        x_self = f64_of_bits(in_bits[part])
        qkv_self = orc.round_bf16(orc.project(x_self, wq))                                  # from the layer's input
        kv_other = orc.round_bf16(orc.project(f64_of_bits(out_bits[others]), wq[128:]))     # from the final rows
        k_tab = np.concatenate([qkv_self[:, 128:256], kv_other[:, :128]])
        v_tab = np.concatenate([qkv_self[:, 256:], kv_other[:, 128:]])
        o = orc.round_bf16(orc.attention(qkv_self[:, :128], k_tab, v_tab, lptr, lidx, heads, scale))
        want = orc.round_bf16(orc.project(o, wo, x_self))
        errs[lo:lo + chunk] = rel_row_err(f64_of_bits(out_bits[part]), want)
    return errs


def drift_by_level_decile(level, err):
    """Largest row error in each tenth of the level range."""
    top = int(level.max()) + 1
    edges = [top * i // 10 for i in range(11)]
    return [float(err[(level >= a) & (level < b)].max()) if ((level >= a) & (level < b)).any() else 0.0
            for a, b in zip(edges[:-1], edges[1:])]
