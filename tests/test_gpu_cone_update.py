"""GPU parity of the cone-by-cone updating (Sec. 3.4 over Algorithm 1's partition): dg4_cone_update_fwd through the
C ABI against the CPU checker's orc.cone_update on the same seeded circuits and tensors."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2502_01681_b200 import dg4, synth
from tests.gpu_util import bf16_weights, dev_bf16, f64_of_bits, host_f64_of_bf16
from tests.helpers import binary_in_tree, csr_from_fanins, levels_of, random_dag, rel_row_err

pytestmark = pytest.mark.gpu
BF16_ROW_TOL = 2e-2


def _run_both(rp, ci, level, xb, weights, k, delta, batch, heads, scale, residual=True):
    gr = dg4.dg4_graph_create(rp, ci, level, k, 0)
    dsc = dg4.desc(heads, dg4.DG4_BF16, scale, residual=residual)
    ws = torch.empty(dg4.dg4_cone_update_workspace_bytes(gr, dsc, batch), dtype=torch.uint8, device="cuda")
    h = dev_bf16(xb).clone()
    stored = torch.full((len(level),), -1, dtype=torch.int32, device="cuda")
    nb = dg4.dg4_cone_update_fwd(gr, dsc, h, [dev_bf16(w[0]) for w in weights], [dev_bf16(w[2]) for w in weights],
                                 delta, batch, ws, stored)
    torch.cuda.synchronize()
    assert dg4.dg4_graph_poll_status(gr) == 0
    want, want_stored, want_nb = orc.cone_update(f64_of_bits(xb), [w[1] for w in weights], [w[3] for w in weights],
                                                 rp, ci, level, k, delta, batch, heads, scale, residual=residual,
                                                 rounding="bf16")
    return host_f64_of_bf16(h), stored.cpu().numpy(), nb, want, want_stored, want_nb


@pytest.mark.parametrize("cfg,shrink,k,delta,batch,layers", [(2, 10, 2, 1, 128, 3), (5, 400, 2, 1, 128, 3),
                                                             (2, 10, 8, 6, 128, 2), (5, 400, 8, 6, 128, 3),
                                                             (5, 400, 8, 6, 7, 1), (4, 20, 1, 1, 64, 2),
                                                             (5, 400, 4, 3, 1000, 2)])
def test_cone_update_matches_checker_on_workloads(cfg, shrink, k, delta, batch, layers):
    w = synth.workload(cfg, shrink)
    g = w.graph()
    xb = w.x_bf16_bits()
    weights = [bf16_weights(w.w_qkv_f32(l)) + bf16_weights(w.w_o_f32(l)) for l in range(layers)]
    got, stored, nb, want, want_stored, want_nb = _run_both(g.row_ptr, g.col_idx, g.level, xb, weights, k, delta, batch,
                                                            w.heads, w.scale)
    assert nb == want_nb and (stored == want_stored).all()
    err = rel_row_err(got, want)
    assert err.max() <= BF16_ROW_TOL, (err.max(), int(err.argmax()))
    untouched = want_stored == 0                                   # gates no cone covers keep their input row, bit for bit
    assert (got[untouched] == f64_of_bits(xb)[untouched]).all()


def test_cone_update_small_shapes_and_larger_weights():
    rng = np.random.default_rng(5)
    shapes = [[[]], [[] for _ in range(9)], [[]] + [[i - 1] for i in range(1, 40)], binary_in_tree(6)[0],
              [[], [], [0, 0], [2, 2], [1, 3], [3, 4]], random_dag(rng, 12, 900, window=25)]
    for fanins in shapes:
        rp, ci = csr_from_fanins(fanins)
        level = levels_of(fanins)
        n = len(fanins)
        xb = synth.normal_bf16_bits(31, 1, (n, 128), 1.0)
        weights = [bf16_weights(synth.normal_f32(31, 10 + l, (384, 128), 0.05)) +
                   bf16_weights(synth.normal_f32(31, 20 + l, (128, 128), 0.05)) for l in range(2)]
        for k, delta, batch, heads, residual in ((3, 2, 5, 8, True), (2, 1, 1, 4, False)):
            got, stored, nb, want, want_stored, want_nb = _run_both(rp, ci, level, xb, weights, k, delta, batch, heads,
                                                                    1.0 / np.sqrt(128 // heads), residual)
            assert nb == want_nb and (stored == want_stored).all(), n
            assert rel_row_err(got, want).max() <= BF16_ROW_TOL, n


def test_cone_update_rejects_bad_arguments():
    fanins = random_dag(np.random.default_rng(1), 4, 60, window=8)
    rp, ci = csr_from_fanins(fanins)
    gr = dg4.dg4_graph_create(rp, ci, levels_of(fanins), 2, 0)
    dsc = dg4.desc(8, dg4.DG4_BF16, 0.25, residual=True)
    n = len(fanins)
    h = torch.zeros(n, 128, dtype=torch.bfloat16, device="cuda")
    wq = torch.zeros(384, 128, dtype=torch.bfloat16, device="cuda")
    wo = torch.zeros(128, 128, dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(dg4.dg4_cone_update_workspace_bytes(gr, dsc, 4), dtype=torch.uint8, device="cuda")
    for kwargs, status in ((dict(delta=0, batch=4), dg4.DG4_ERR_INVALID_ARG), (dict(delta=1, batch=0), dg4.DG4_ERR_INVALID_ARG),
                           (dict(delta=1, batch=4096), dg4.DG4_ERR_INVALID_ARG)):        # the last: workspace too small
        with pytest.raises(dg4.Dg4Error) as e:
            dg4.dg4_cone_update_fwd(gr, dsc, h, [wq], [wo], kwargs["delta"], kwargs["batch"], ws)
        assert e.value.status == status, kwargs
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_cone_update_fwd(gr, dg4.desc(8, dg4.DG4_F32, 0.25), h, [wq], [wo], 1, 4, ws)
    assert e.value.status == dg4.DG4_ERR_UNSUPPORTED
    torch.cuda.synchronize()
