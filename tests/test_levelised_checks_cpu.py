"""The step-by-step check of a levelised layer (tests/levelised_checks.py), run on the CPU with the checker's own
levelised result in the place of the GPU's: it must accept that result exactly, and it must reject a result in
which one node was computed from a neighbour's row as it was BEFORE that neighbour's level had been processed."""
import numpy as np

from oracle import oracle as orc
from paper_2502_01681_b200 import synth
from tests.gpu_util import bf16_weights, f64_of_bits
from tests.levelised_checks import drift_by_level_decile, every_step_check


def _problem():
    w = synth.workload(5, 400)
    g = w.graph()
    ptr, idx = orc.neighbourhood(g.row_ptr, g.col_idx, w.hops)
    lptr, lnodes = orc.level_buckets(g.level)
    xb = w.x_bf16_bits()
    _, wq = bf16_weights(w.w_qkv_f32(0))
    _, wo = bf16_weights(w.w_o_f32(0))
    out = orc.layer_levelised(f64_of_bits(xb), wq, wo, ptr, idx, lptr, lnodes, w.heads, w.scale, residual=True,
                              rounding="bf16")
    out_bits = synth.f32_to_bf16_bits(out.astype(np.float32))
    assert (f64_of_bits(out_bits) == out).all()            # the checker's rounded rows are exact bf16 values
    return w, g, ptr, idx, xb, wq, wo, out_bits


def test_step_check_accepts_the_checkers_own_levelised_result():
    w, g, ptr, idx, xb, wq, wo, out_bits = _problem()
    for chunk in (1000, 400_000):                          # several chunks with a ragged tail, and one chunk
        err = every_step_check(ptr, idx, np.arange(g.n), xb, out_bits, wq, wo, w.heads, w.scale, chunk=chunk)
        assert err.max() == 0.0
    rows = np.array([0, g.n_pi, g.n - 1, g.n // 2])
    assert every_step_check(ptr, idx, rows, xb, out_bits, wq, wo, w.heads, w.scale).max() == 0.0


def test_step_check_rejects_a_stale_read():
    w, g, ptr, idx, xb, wq, wo, out_bits = _problem()
    sizes = np.diff(ptr)
    v = int(np.nonzero(sizes == 7)[0][-1])                 # a gate with a full two-hop cone
    u = int(idx[ptr[v] + 1])                               # one of its fan-in-side members
    stale_in = out_bits.copy()
    stale_in[u] = xb[u]                                    # as if u's level had not been written yet
    one = every_step_check(ptr, idx, np.array([v]), xb, stale_in, wq, wo, w.heads, w.scale)
    recomputed = every_step_check(ptr, idx, np.array([v]), xb, out_bits, wq, wo, w.heads, w.scale)
    assert recomputed[0] == 0.0 and one[0] > 1e-4


def test_drift_table_bins_levels_into_tenths():
    level = np.arange(100)
    err = np.arange(100) / 100.0
    assert np.allclose(drift_by_level_decile(level, err), [0.09 + 0.1 * i for i in range(10)])
