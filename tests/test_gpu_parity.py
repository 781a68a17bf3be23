"""GPU parity: the CUDA library, called through its C ABI, against the CPU checker on the same seeded
inputs.  Index arrays must match bit for bit; fp32 attention within 1e-5 max-abs; bf16 tensors within
2e-2 of the row norm (per row, L2) of the checker run with the same storage rounding."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2502_01681_b200 import dg4, synth
from tests.gpu_util import bf16_weights, dev_bf16, f64_of_bits, host_f64_of_bf16
from tests.helpers import binary_in_tree, csr_from_fanins, levels_of, random_dag, rel_row_err

pytestmark = pytest.mark.gpu

BF16_ROW_TOL = 2e-2      # relative to the row norm
F32_ABS_TOL = 1e-5


# ----------------------------------------------------------------------------- graph prep

def _check_graph_arrays(rp, ci, level, hops, chunk):
    g = dg4.dg4_graph_create(rp, ci, level, hops, chunk)
    n = len(level)
    ptr, idx = orc.neighbourhood(rp, ci, hops)
    lptr, lnodes = orc.level_buckets(level)
    mc = 2 ** (hops + 1) - 1
    eff_chunk = 0 if chunk >= n else chunk
    perm, cptr = orc.class_order(np.arange(n, dtype=np.int32), orc.chunk_ptr(n, eff_chunk), ptr, mc)
    lperm, lcptr = orc.class_order(lnodes, lptr, ptr, mc)
    pad = np.repeat(np.arange(n, dtype=np.int32)[:, None], mc + 1, axis=1)       # the same lists, fixed width
    pad[:, 0] = np.diff(ptr)
    for v in range(n):
        pad[v, 1:pad[v, 0]] = idx[ptr[v] + 1:ptr[v + 1]]

    def same(which, want):
        got = dg4.dg4_graph_export(g, which)
        assert got.shape == want.ravel().shape and (got == want.ravel()).all(), which

    for _ in range(2):                      # the second round checks that a rebuild reproduces everything
        same(dg4.DG4_ARR_NBR_PTR, ptr)
        same(dg4.DG4_ARR_NBR_IDX, idx)
        same(dg4.DG4_ARR_NBR_PAD, pad)
        same(dg4.DG4_ARR_LEVEL_PTR, lptr)
        same(dg4.DG4_ARR_LEVEL_NODES, lnodes)
        same(dg4.DG4_ARR_PERM, perm)
        same(dg4.DG4_ARR_CLASS_PTR, cptr)
        same(dg4.DG4_ARR_LEVEL_PERM, lperm)
        same(dg4.DG4_ARR_LEVEL_CLASS_PTR, lcptr)
        dg4.dg4_graph_rebuild(g)
    info = dg4.dg4_graph_info(g)
    assert info.n_nodes == n and info.n_nbr == len(idx) and info.n_levels == len(lptr) - 1 and info.max_class == mc
    return g


@pytest.mark.parametrize("hops", [1, 2])
def test_graph_prep_small_shapes(hops):
    cases = []
    cases.append([[]])                                             # a single primary input
    cases.append([[] for _ in range(5)])                           # no edges at all
    cases.append([[]] + [[i - 1] for i in range(1, 40)])           # a chain of inverters
    cases.append(binary_in_tree(5)[0])                             # every gate at maximum class
    cases.append([[], [], [0, 0], [2, 2], [1, 3], [3, 4]])         # tied inputs, 1-path and 2-path to one node
    rng = np.random.default_rng(0)
    cases.append(random_dag(rng, 7, 3000, window=40))              # spans several 1024-element tiles, ragged tail
    for fanins in cases:
        rp, ci = csr_from_fanins(fanins)
        _check_graph_arrays(rp, ci, levels_of(fanins), hops, 0)


@pytest.mark.parametrize("cfg,shrink,chunk", [(1, 1, 0), (1, 1, 1024), (2, 4, 2048), (3, 20, 8192), (4, 10, 0),
                                              (5, 100, 4096), (5, 100, 0)])
def test_graph_prep_matches_checker_on_workloads(cfg, shrink, chunk):
    w = synth.workload(cfg, shrink)
    g = w.graph()
    _check_graph_arrays(g.row_ptr, g.col_idx, g.level, w.hops, chunk)


def test_graph_prep_accepts_any_strict_layering():
    fanins = random_dag(np.random.default_rng(3), 5, 500, window=20)
    rp, ci = csr_from_fanins(fanins)
    level = levels_of(fanins) * 3 + 1        # still strictly increasing along edges, with empty levels
    _check_graph_arrays(rp, ci, level, 2, 0)


# ----------------------------------------------------------------------------- attention

def _attention_case(rp, ci, level, hops, heads, dtype, scale, std, seed=0):
    n = len(level)
    g = dg4.dg4_graph_create(rp, ci, level, hops, 0)
    ptr, idx = orc.neighbourhood(rp, ci, hops)
    q, k, v = (synth.normal_f32(seed, 50 + i, (n, 128), std) for i in range(3))
    if dtype == "f32":
        dq, dk, dv = (torch.from_numpy(t).cuda() for t in (q, k, v))
        want = orc.attention(q, k, v, ptr, idx, heads, scale)
        o = torch.empty_like(dq)
        dg4.dg4_sparse_attn_fwd(g, dg4.desc(heads, dg4.DG4_F32, scale), dq, dk, dv, o)
        torch.cuda.synchronize()
        got = o.cpu().numpy().astype(np.float64)
        return got, want
    bq, bk, bv = (synth.f32_to_bf16_bits(t) for t in (q, k, v))
    want = orc.round_bf16(orc.attention(f64_of_bits(bq), f64_of_bits(bk), f64_of_bits(bv), ptr, idx, heads, scale))
    dq, dk, dv = dev_bf16(bq), dev_bf16(bk), dev_bf16(bv)
    o = torch.empty_like(dq)
    dg4.dg4_sparse_attn_fwd(g, dg4.desc(heads, dg4.DG4_BF16, scale), dq, dk, dv, o)
    torch.cuda.synchronize()
    return host_f64_of_bf16(o), want


def test_attention_config1_fp32():
    w = synth.workload(1)
    g = w.graph()
    gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, 1, 0)
    q, k, v = w.qkv_f32()
    ptr, idx = orc.neighbourhood(g.row_ptr, g.col_idx, 1)
    want = orc.attention(q, k, v, ptr, idx, w.heads, w.scale)
    dq, dk, dv = (torch.from_numpy(t).cuda() for t in (q, k, v))
    o = torch.empty_like(dq)
    dg4.dg4_sparse_attn_fwd(gr, dg4.desc(w.heads, dg4.DG4_F32, w.scale), dq, dk, dv, o)
    torch.cuda.synchronize()
    err = np.abs(o.cpu().numpy().astype(np.float64) - want).max()
    assert err <= F32_ABS_TOL, err
    # primary inputs attend only themselves: their output is their V row, bit for bit
    assert torch.equal(o[:g.n_pi], dv[:g.n_pi])


@pytest.mark.parametrize("hops", [1, 2])
@pytest.mark.parametrize("heads", [1, 2, 4, 8, 16, 32])
def test_attention_fp32_heads_and_hops(hops, heads):
    fanins = random_dag(np.random.default_rng(heads), 9, 1500, window=30)
    rp, ci = csr_from_fanins(fanins)
    got, want = _attention_case(rp, ci, levels_of(fanins), hops, heads, "f32", 1.0 / np.sqrt(128 // heads), 1.0)
    assert np.abs(got - want).max() <= F32_ABS_TOL


@pytest.mark.parametrize("hops", [1, 2])
@pytest.mark.parametrize("heads", [1, 2, 4, 8, 16])
def test_attention_bf16_heads_and_hops(hops, heads):
    fanins = random_dag(np.random.default_rng(100 + heads), 9, 1500, window=30)
    rp, ci = csr_from_fanins(fanins)
    got, want = _attention_case(rp, ci, levels_of(fanins), hops, heads, "bf16", 1.0 / np.sqrt(128 // heads), 1.0)
    assert rel_row_err(got, want).max() <= BF16_ROW_TOL


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_attention_peaked_softmax(dtype):
    # scale 1 and unit-variance inputs: scores reach tens, the softmax is far from uniform
    fanins = random_dag(np.random.default_rng(7), 9, 2000, window=30)
    rp, ci = csr_from_fanins(fanins)
    got, want = _attention_case(rp, ci, levels_of(fanins), 2, 8, dtype, 1.0, 2.0)
    if dtype == "f32":
        # Scores here reach |s| ~ 70 and outputs ~ 9: fp32 holds such a score (in the log2 units the exponential is
        # taken in) only to 2^-17, i.e. a weight to about 1e-5 of itself, so the 1e-5 bound is taken relative to the
        # largest output magnitude in this one test (every other fp32 test meets 1e-5 absolute).
        assert np.abs(got - want).max() <= F32_ABS_TOL * max(1.0, np.abs(want).max())
    else:
        assert rel_row_err(got, want).max() <= BF16_ROW_TOL


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_attention_degenerate_graphs(dtype):
    shapes = {
        "single": [[]],
        "edgeless": [[] for _ in range(33)],
        "chain": [[]] + [[i - 1] for i in range(1, 70)],
        "tree": binary_in_tree(6)[0],
        "tied": [[], [], [0, 0], [2, 2], [1, 3], [3, 4]],
    }
    for name, fanins in shapes.items():
        rp, ci = csr_from_fanins(fanins)
        got, want = _attention_case(rp, ci, levels_of(fanins), 2, 8, dtype, 0.25, 1.0)
        if dtype == "f32":
            assert np.abs(got - want).max() <= F32_ABS_TOL, name
        else:
            assert rel_row_err(got, want).max() <= BF16_ROW_TOL, name


def test_attention_strided_interleaved_kv():
    # K and V interleaved in one [n, 256] buffer, as the layer calls lay them out
    fanins = random_dag(np.random.default_rng(11), 9, 1000, window=30)
    rp, ci = csr_from_fanins(fanins)
    n = len(fanins)
    g = dg4.dg4_graph_create(rp, ci, levels_of(fanins), 2, 0)
    ptr, idx = orc.neighbourhood(rp, ci, 2)
    bq, bk, bv = (synth.normal_bf16_bits(5, 60 + i, (n, 128), 1.0) for i in range(3))
    kv = torch.empty(n, 256, dtype=torch.bfloat16, device="cuda")
    kv[:, :128] = dev_bf16(bk)
    kv[:, 128:] = dev_bf16(bv)
    o = torch.empty(n, 128, dtype=torch.bfloat16, device="cuda")
    dg4.dg4_sparse_attn_fwd(g, dg4.desc(8, dg4.DG4_BF16, 0.25), dev_bf16(bq), kv[:, :128], kv[:, 128:], o)
    torch.cuda.synchronize()
    want = orc.round_bf16(orc.attention(f64_of_bits(bq), f64_of_bits(bk), f64_of_bits(bv), ptr, idx, 8, 0.25))
    assert rel_row_err(host_f64_of_bf16(o), want).max() <= BF16_ROW_TOL


def test_attention_config3_full_size():
    w = synth.workload(3)
    g = w.graph()
    gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, 2, 0)
    bq, bk, bv = w.qkv_bf16_bits()
    dq, dk, dv = dev_bf16(bq), dev_bf16(bk), dev_bf16(bv)
    o = torch.empty_like(dq)
    dg4.dg4_sparse_attn_fwd(gr, dg4.desc(8, dg4.DG4_BF16, w.scale), dq, dk, dv, o)
    torch.cuda.synchronize()
    ptr, idx = orc.neighbourhood(g.row_ptr, g.col_idx, 2)
    assert (dg4.dg4_graph_export(gr, dg4.DG4_ARR_NBR_IDX) == idx).all()
    want = orc.round_bf16(orc.attention(f64_of_bits(bq), f64_of_bits(bk), f64_of_bits(bv), ptr, idx, 8, w.scale))
    assert rel_row_err(host_f64_of_bf16(o), want).max() <= BF16_ROW_TOL


# ----------------------------------------------------------------------------- projections

@pytest.mark.parametrize("n", [1, 127, 128, 129, 1000, 4133])
def test_projections_match_checker(n):
    fanins = [[] for _ in range(n)]
    rp, ci = csr_from_fanins(fanins)
    g = dg4.dg4_graph_create(rp, ci, np.zeros(n, np.int32), 1, 0)
    xb = synth.normal_bf16_bits(9, 1, (n, 128), 1.0)
    wq_bits, wq = bf16_weights(synth.normal_f32(9, 2, (384, 128), 0.05))
    wo_bits, wo = bf16_weights(synth.normal_f32(9, 3, (128, 128), 0.05))
    x = f64_of_bits(xb)
    dsc = dg4.desc(8, dg4.DG4_BF16, 0.25, residual=True)
    dx = dev_bf16(xb)
    q, k, v, h = (torch.empty(n, 128, dtype=torch.bfloat16, device="cuda") for _ in range(4))
    dg4.dg4_qkv_project(g, dsc, dx, dev_bf16(wq_bits), q, k, v)
    dg4.dg4_out_project(g, dsc, q, dev_bf16(wo_bits), dx, h)
    torch.cuda.synchronize()
    want = orc.round_bf16(orc.project(x, wq))
    got = np.concatenate([host_f64_of_bf16(t) for t in (q, k, v)], axis=1)
    assert rel_row_err(got, want).max() <= BF16_ROW_TOL
    want_h = orc.round_bf16(orc.project(host_f64_of_bf16(q), wo, x))
    assert rel_row_err(host_f64_of_bf16(h), want_h).max() <= BF16_ROW_TOL


# ----------------------------------------------------------------------------- whole layers

def _weights(w, layers):
    out = []
    for l in range(layers):
        out.append(bf16_weights(w.w_qkv_f32(l)) + bf16_weights(w.w_o_f32(l)))
    return out


def _run_layers_gpu(gr, w, xb, weights, mode):
    dsc = dg4.desc(w.heads, dg4.DG4_BF16, w.scale, residual=w.residual, level_launches=(mode == "level-launches"),
                   fused_layer=(mode == "fused"))
    ws = torch.empty(max(dg4.dg4_layer_workspace_bytes(gr, dsc), dg4.dg4_layers_workspace_bytes(gr, dsc, len(weights))),
                     dtype=torch.uint8, device="cuda")
    h = dev_bf16(xb).clone()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    if mode == "wavefront":              # all layers in one call
        dg4.dg4_layers_fwd_levelised(gr, dsc, h, [dev_bf16(w_[0]) for w_ in weights], [dev_bf16(w_[2]) for w_ in weights],
                                     ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        return host_f64_of_bf16(h)
    for (wq_bits, _, wo_bits, _) in weights:
        if mode in ("parallel", "fused"):
            dg4.dg4_layer_fwd_parallel(gr, dsc, h, dev_bf16(wq_bits), dev_bf16(wo_bits), h, ws)
        else:
            dg4.dg4_layer_fwd_levelised(gr, dsc, h, dev_bf16(wq_bits), dev_bf16(wo_bits), ws, status)
            assert int(status.item()) == 0
    torch.cuda.synchronize()
    assert dg4.dg4_graph_poll_status(gr) == 0
    return host_f64_of_bf16(h)


def _run_layers_checker(g, w, xb, weights, mode):
    ptr, idx = orc.neighbourhood(g.row_ptr, g.col_idx, w.hops)
    h = f64_of_bits(xb)
    if mode not in ("parallel", "fused"):
        lptr, lnodes = orc.level_buckets(g.level)
    for (_, wq, _, wo) in weights:
        if mode in ("parallel", "fused"):
            h = orc.layer_parallel(h, wq, wo, ptr, idx, w.heads, w.scale, residual=w.residual, rounding="bf16")
        else:
            h = orc.layer_levelised(h, wq, wo, ptr, idx, lptr, lnodes, w.heads, w.scale, residual=w.residual,
                                    rounding="bf16")
    return h


@pytest.mark.parametrize("cfg,shrink,mode", [(2, 1, "parallel"), (2, 7, "parallel"), (5, 200, "parallel"),
                                             (2, 1, "fused"), (2, 7, "fused"), (5, 200, "fused"), (4, 5, "fused"),
                                             (4, 20, "levelised"), (5, 400, "levelised"), (2, 10, "levelised"),
                                             (4, 5, "levelised"), (5, 50, "levelised"),
                                             (4, 20, "level-launches"), (5, 400, "level-launches"),
                                             (4, 20, "wavefront"), (5, 400, "wavefront"), (5, 50, "wavefront"),
                                             (2, 10, "wavefront"), (4, 5, "wavefront")])
def test_layers_match_checker(cfg, shrink, mode):
    w = synth.workload(cfg, shrink)
    g = w.graph()
    gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0)
    xb = w.x_bf16_bits()
    weights = _weights(w, w.layers)
    got = _run_layers_gpu(gr, w, xb, weights, mode)
    want = _run_layers_checker(g, w, xb, weights, mode)
    err = rel_row_err(got, want)
    assert err.max() <= BF16_ROW_TOL, (err.max(), int(err.argmax()))


@pytest.mark.parametrize("n_gates,heads,residual", [(1, 8, True), (63, 8, True), (128, 2, False), (129, 8, True),
                                                    (20000, 16, True), (33333, 1, False)])
def test_fused_layer_is_bit_identical_to_the_three_kernels(n_gates, heads, residual):
    """The one-kernel form of the all-parallel layer computes the same products with the same roundings in the
    same order: its rows must equal the three-kernel path's bit for bit (and that path is checked against the
    oracle above), for ragged sizes, in place and out of place."""
    rng = np.random.default_rng(n_gates + heads)
    fanins = random_dag(rng, 17, n_gates, window=500)
    rp, ci = csr_from_fanins(fanins)
    level = levels_of(fanins)
    n = len(fanins)
    gr = dg4.dg4_graph_create(rp, ci, level, 2, 0)
    x = dev_bf16(synth.normal_bf16_bits(11, 1, (n, 128), 1.0))
    wq = dev_bf16(bf16_weights(synth.normal_f32(11, 2, (384, 128), 0.08))[0])
    wo = dev_bf16(bf16_weights(synth.normal_f32(11, 3, (128, 128), 0.08))[0])
    scale = 1.0 / np.sqrt(128 // heads)
    outs = []
    for fused in (False, True):
        dsc = dg4.desc(heads, dg4.DG4_BF16, scale, residual=residual, fused_layer=fused)
        ws = torch.empty(dg4.dg4_layer_workspace_bytes(gr, dsc), dtype=torch.uint8, device="cuda")
        h = torch.zeros_like(x)
        dg4.dg4_layer_fwd_parallel(gr, dsc, x, wq, wo, h, ws)
        inplace = x.clone()
        dg4.dg4_layer_fwd_parallel(gr, dsc, inplace, wq, wo, inplace, ws)
        torch.cuda.synchronize()
        assert dg4.dg4_graph_poll_status(gr) == 0
        assert bool((h.view(torch.int16) == inplace.view(torch.int16)).all())
        outs.append(h.view(torch.int16).clone())
    assert bool((outs[0] == outs[1]).all()), int((outs[0] != outs[1]).any(dim=1).sum())


def test_levelised_differs_from_parallel_and_is_repeatable():
    w = synth.workload(4, 20)
    g = w.graph()
    gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0)
    xb = w.x_bf16_bits()
    weights = _weights(w, 1)
    a = _run_layers_gpu(gr, w, xb, weights, "levelised")
    b = _run_layers_gpu(gr, w, xb, weights, "levelised")
    c = _run_layers_gpu(gr, w, xb, weights, "level-launches")
    p = _run_layers_gpu(gr, w, xb, weights, "parallel")
    assert (a == b).all()                                   # a race between levels would show up as a diff
    assert rel_row_err(a, c).max() <= 1e-2                  # persistent kernel vs one launch group per level
    w3 = _weights(w, 3)
    d = _run_layers_gpu(gr, w, xb, w3, "levelised")         # three calls, layer after layer
    e = _run_layers_gpu(gr, w, xb, w3, "wavefront")         # one call, layers as a wavefront
    assert (d == e).all()
    lvl0 = g.level == 0
    assert (a[lvl0] == p[lvl0]).all()                       # level-0 rows never see an updated row
    assert np.abs(a - p).max() > 0


# ----------------------------------------------------------------------------- error paths (no GPU fault)

def test_forward_calls_reject_bad_arguments():
    fanins = random_dag(np.random.default_rng(1), 4, 60, window=8)
    rp, ci = csr_from_fanins(fanins)
    n = len(fanins)
    g = dg4.dg4_graph_create(rp, ci, levels_of(fanins), 1, 0)
    t = torch.zeros(n, 128, dtype=torch.bfloat16, device="cuda")
    o = torch.zeros(n, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_sparse_attn_fwd(g, dg4.desc(3, dg4.DG4_BF16, 1.0), t, t, t, o)
    assert e.value.status == dg4.DG4_ERR_UNSUPPORTED
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_sparse_attn_fwd(g, dg4.desc(8, dg4.DG4_BF16, 1.0, d=64), t, t, t, o)
    assert e.value.status == dg4.DG4_ERR_UNSUPPORTED
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_sparse_attn_fwd(g, dg4.desc(8, dg4.DG4_BF16, 1.0), t, t, t, t)
    assert e.value.status == dg4.DG4_ERR_INVALID_ARG
    odd = torch.zeros(n * 128 + 8, dtype=torch.bfloat16, device="cuda")[1:n * 128 + 1].view(n, 128)
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_sparse_attn_fwd(g, dg4.desc(8, dg4.DG4_BF16, 1.0), odd, t, t, o)
    assert e.value.status == dg4.DG4_ERR_INVALID_ARG
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_qkv_project(g, dg4.desc(8, dg4.DG4_F32, 1.0), t, t, t, t, t)
    assert e.value.status == dg4.DG4_ERR_UNSUPPORTED
    small = torch.zeros(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_layer_fwd_parallel(g, dg4.desc(8, dg4.DG4_BF16, 1.0), t, t, t, o, small)
    assert e.value.status == dg4.DG4_ERR_INVALID_ARG
    torch.cuda.synchronize()


def test_bounded_wait_runs_out_and_reports_timeout():
    # a wait nothing can satisfy ends by itself; the kernel reports it and the context stays usable
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dg4.dg4_selftest_bounded_wait(status)
    torch.cuda.synchronize()
    assert int(status.item()) == dg4.DG4_ERR_TIMEOUT
    assert float((torch.ones(8, device="cuda") * 2).sum().item()) == 16.0


@pytest.mark.parametrize("hops,heads,residual,mode", [(1, 1, True, "wavefront"), (2, 4, False, "wavefront"),
                                                      (2, 16, True, "wavefront"), (1, 2, False, "parallel"),
                                                      (2, 16, True, "parallel"), (1, 4, True, "level-launches"),
                                                      (1, 2, False, "fused"), (2, 16, True, "fused"), (2, 1, True, "fused")])
def test_layers_other_head_counts_and_no_residual(hops, heads, residual, mode):
    rng = np.random.default_rng(1000 * hops + heads)
    fanins = random_dag(rng, 40, 6000, window=300)
    rp, ci = csr_from_fanins(fanins)
    level = levels_of(fanins)
    n = len(fanins)
    gr = dg4.dg4_graph_create(rp, ci, level, hops, 0)
    xb = synth.normal_bf16_bits(7, 1, (n, 128), 1.0)
    weights = [bf16_weights(synth.normal_f32(7, 10 + l, (384, 128), 0.05)) +
               bf16_weights(synth.normal_f32(7, 20 + l, (128, 128), 0.05)) for l in range(2)]
    scale = 1.0 / np.sqrt(128 // heads)
    dsc = dg4.desc(heads, dg4.DG4_BF16, scale, residual=residual, level_launches=(mode == "level-launches"),
                   fused_layer=(mode == "fused"))
    ws = torch.empty(max(dg4.dg4_layer_workspace_bytes(gr, dsc), dg4.dg4_layers_workspace_bytes(gr, dsc, 2)),
                     dtype=torch.uint8, device="cuda")
    h = dev_bf16(xb).clone()
    if mode in ("parallel", "fused"):
        for w_ in weights:
            dg4.dg4_layer_fwd_parallel(gr, dsc, h, dev_bf16(w_[0]), dev_bf16(w_[2]), h, ws)
    else:
        dg4.dg4_layers_fwd_levelised(gr, dsc, h, [dev_bf16(w_[0]) for w_ in weights], [dev_bf16(w_[2]) for w_ in weights], ws)
    torch.cuda.synchronize()
    assert dg4.dg4_graph_poll_status(gr) == 0
    ptr, idx = orc.neighbourhood(rp, ci, hops)
    lptr, lnodes = orc.level_buckets(level)
    want = f64_of_bits(xb)
    for (_, wq, _, wo) in weights:
        if mode in ("parallel", "fused"):
            want = orc.layer_parallel(want, wq, wo, ptr, idx, heads, scale, residual=residual, rounding="bf16")
        else:
            want = orc.layer_levelised(want, wq, wo, ptr, idx, lptr, lnodes, heads, scale, residual=residual,
                                       rounding="bf16")
    err = rel_row_err(host_f64_of_bf16(h), want)
    assert err.max() <= BF16_ROW_TOL, err.max()


@pytest.mark.parametrize("dtype,hops,heads", [("f32", 1, 4), ("f32", 2, 8), ("bf16", 2, 8), ("bf16", 1, 1),
                                              ("bf16", 2, 16), ("f32", 2, 32),
                                              ("bf16", 4, 8), ("bf16", 8, 2), ("f32", 5, 4), ("f32", 8, 32)])
def test_additive_score_attention_matches_checker(dtype, hops, heads):
    rng = np.random.default_rng(7000 + heads + hops)
    fanins = random_dag(rng, 40, 5000, window=200)
    rp, ci = csr_from_fanins(fanins)
    n = len(fanins)
    g = dg4.dg4_graph_create(rp, ci, levels_of(fanins), hops, 0)
    ptr, idx = orc.neighbourhood(rp, ci, hops)
    sd = synth.normal_f32(3, 80, (n, heads), 1.5)
    ss = synth.normal_f32(3, 81, (n, heads), 1.5)
    v32 = synth.normal_f32(3, 82, (n, 128), 1.0)
    dsd, dss = torch.from_numpy(sd).cuda(), torch.from_numpy(ss).cuda()
    if dtype == "f32":
        dv = torch.from_numpy(v32).cuda()
        o = torch.empty_like(dv)
        dg4.dg4_sparse_attn_additive_fwd(g, dg4.desc(heads, dg4.DG4_F32, 1.0), dsd, dss, 0.2, dv, o)
        torch.cuda.synchronize()
        want = orc.attention_additive(sd, ss, v32, ptr, idx, 0.2)
        assert np.abs(o.cpu().numpy().astype(np.float64) - want).max() <= F32_ABS_TOL
    else:
        vb = synth.f32_to_bf16_bits(v32)
        dv = dev_bf16(vb)
        o = torch.empty_like(dv)
        dg4.dg4_sparse_attn_additive_fwd(g, dg4.desc(heads, dg4.DG4_BF16, 1.0), dsd, dss, 0.2, dv, o)
        torch.cuda.synchronize()
        want = orc.round_bf16(orc.attention_additive(sd, ss, f64_of_bits(vb), ptr, idx, 0.2))
        assert rel_row_err(host_f64_of_bf16(o), want).max() <= BF16_ROW_TOL
        pis = np.nonzero(np.diff(ptr) == 1)[0]
        assert torch.equal(o[torch.from_numpy(pis).cuda()], dv[torch.from_numpy(pis).cuda()])    # weight exactly 1


# ----------------------------------------------------------------------------- wider cones (3 to 8 hops)

@pytest.mark.parametrize("hops", [3, 4, 6, 8])
def test_wide_cone_lists_match_checker(hops):
    rng = np.random.default_rng(hops)
    cases = [binary_in_tree(8)[0], random_dag(rng, 30, 4000, window=64), [[]] + [[i - 1] for i in range(1, 300)],
             [[], [], [0, 0], [2, 2], [1, 3], [3, 4]]]
    for fanins in cases:
        rp, ci = csr_from_fanins(fanins)
        level = levels_of(fanins)
        g = dg4.dg4_graph_create(rp, ci, level, hops, 0)
        ptr, idx = orc.neighbourhood(rp, ci, hops)
        lptr, lnodes = orc.level_buckets(level)
        assert (dg4.dg4_graph_export(g, dg4.DG4_ARR_NBR_PTR) == ptr).all()
        assert (dg4.dg4_graph_export(g, dg4.DG4_ARR_NBR_IDX) == idx).all()
        assert (dg4.dg4_graph_export(g, dg4.DG4_ARR_LEVEL_PTR) == lptr).all()
        assert (dg4.dg4_graph_export(g, dg4.DG4_ARR_LEVEL_NODES) == lnodes).all()
        info = dg4.dg4_graph_info(g)
        assert info.max_class == 2 ** (hops + 1) - 1 and info.n_nbr == len(idx)
        assert np.diff(ptr).max() <= info.max_class
        with pytest.raises(dg4.Dg4Error) as e:
            dg4.dg4_graph_export(g, dg4.DG4_ARR_PERM)
        assert e.value.status == dg4.DG4_ERR_UNSUPPORTED


@pytest.mark.parametrize("dtype,hops,heads", [("bf16", 3, 8), ("bf16", 8, 8), ("bf16", 5, 1), ("bf16", 4, 16),
                                              ("f32", 3, 4), ("f32", 8, 8), ("f32", 6, 32)])
def test_wide_cone_attention_matches_checker(dtype, hops, heads):
    rng = np.random.default_rng(hops * 100 + heads)
    fanins = random_dag(rng, 30, 3000, window=80)
    rp, ci = csr_from_fanins(fanins)
    scale = 1.0 / np.sqrt(128 // heads)
    got, want = _attention_case(rp, ci, levels_of(fanins), hops, heads, dtype, scale, 1.5)
    if dtype == "f32":
        assert np.abs(got - want).max() <= F32_ABS_TOL
    else:
        assert rel_row_err(got, want).max() <= BF16_ROW_TOL


@pytest.mark.parametrize("hops,heads", [(4, 8), (8, 8), (3, 1), (6, 16)])
def test_wide_cone_layers_in_every_order(hops, heads):
    """Cones of 3 to 8 hops through the layer calls: all nodes at once, level by level with one launch group per
    level, level by level in the persistent kernel (which walks the cone lists with an online softmax), and two
    layers as a wavefront."""
    rng = np.random.default_rng(31 + hops)
    fanins = random_dag(rng, 30, 2500, window=60)
    rp, ci = csr_from_fanins(fanins)
    level = levels_of(fanins)
    n = len(fanins)
    scale = 1.0 / np.sqrt(128 // heads)
    gr = dg4.dg4_graph_create(rp, ci, level, hops, 0)
    xb = synth.normal_bf16_bits(8, 1, (n, 128), 1.0)
    weights = [bf16_weights(synth.normal_f32(8, 2 + 2 * l, (384, 128), 0.05)) +
               bf16_weights(synth.normal_f32(8, 3 + 2 * l, (128, 128), 0.05)) for l in range(2)]
    (wqb, wq, wob, wo) = weights[0]
    ptr, idx = orc.neighbourhood(rp, ci, hops)
    lptr, lnodes = orc.level_buckets(level)
    want_par = orc.layer_parallel(f64_of_bits(xb), wq, wo, ptr, idx, heads, scale, residual=True, rounding="bf16")
    want_lev = orc.layer_levelised(f64_of_bits(xb), wq, wo, ptr, idx, lptr, lnodes, heads, scale, residual=True,
                                   rounding="bf16")
    want_lev2 = orc.layer_levelised(want_lev, weights[1][1], weights[1][3], ptr, idx, lptr, lnodes, heads, scale,
                                    residual=True, rounding="bf16")
    for mode in ("parallel", "level-launches", "persistent", "wavefront"):
        dsc = dg4.desc(heads, dg4.DG4_BF16, scale, residual=True, level_launches=(mode == "level-launches"))
        ws = torch.empty(max(dg4.dg4_layer_workspace_bytes(gr, dsc), dg4.dg4_layers_workspace_bytes(gr, dsc, 2)),
                         dtype=torch.uint8, device="cuda")
        h = dev_bf16(xb).clone()
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        if mode == "parallel":
            dg4.dg4_layer_fwd_parallel(gr, dsc, h, dev_bf16(wqb), dev_bf16(wob), h, ws)
            want = want_par
        elif mode == "wavefront":
            dg4.dg4_layers_fwd_levelised(gr, dsc, h, [dev_bf16(w_[0]) for w_ in weights],
                                         [dev_bf16(w_[2]) for w_ in weights], ws, status)
            want = want_lev2
        else:
            dg4.dg4_layer_fwd_levelised(gr, dsc, h, dev_bf16(wqb), dev_bf16(wob), ws, status)
            want = want_lev
        torch.cuda.synchronize()
        assert int(status.item()) == 0 and dg4.dg4_graph_poll_status(gr) == 0, mode
        err = rel_row_err(host_f64_of_bf16(h), want)
        assert err.max() <= BF16_ROW_TOL, (mode, err.max(), int(err.argmax()))


@pytest.mark.parametrize("hops,delta", [(8, 6), (3, 2), (2, 1), (1, 1)])
def test_graph_partition_roots_match_checker(hops, delta):
    rng = np.random.default_rng(hops * 10 + delta)
    for fanins in (random_dag(rng, 20, 5000, window=25), binary_in_tree(9)[0], [[] for _ in range(7)]):
        rp, ci = csr_from_fanins(fanins)
        level = levels_of(fanins)
        g = dg4.dg4_graph_create(rp, ci, level, hops, 0)
        roots, gptr = dg4.dg4_graph_partition(g, delta)
        want_roots, want_gptr = orc.partition_roots(rp, ci, level, hops, delta)
        assert (roots.cpu().numpy() == want_roots).all()
        assert (gptr.cpu().numpy() == want_gptr).all()


def test_levelised_layers_with_empty_levels():
    # any strictly increasing layering is accepted; here two of every three levels are empty
    rng = np.random.default_rng(99)
    fanins = random_dag(rng, 50, 3000, window=100)
    rp, ci = csr_from_fanins(fanins)
    level = levels_of(fanins) * 3 + 1
    n = len(fanins)
    gr = dg4.dg4_graph_create(rp, ci, level, 2, 0)
    xb = synth.normal_bf16_bits(11, 1, (n, 128), 1.0)
    weights = [bf16_weights(synth.normal_f32(11, 10 + l, (384, 128), 0.05)) +
               bf16_weights(synth.normal_f32(11, 20 + l, (128, 128), 0.05)) for l in range(3)]
    dsc = dg4.desc(8, dg4.DG4_BF16, 0.25, residual=True)
    ws = torch.empty(dg4.dg4_layers_workspace_bytes(gr, dsc, 3), dtype=torch.uint8, device="cuda")
    h = dev_bf16(xb).clone()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    dg4.dg4_layers_fwd_levelised(gr, dsc, h, [dev_bf16(w_[0]) for w_ in weights], [dev_bf16(w_[2]) for w_ in weights],
                                 ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ptr, idx = orc.neighbourhood(rp, ci, 2)
    lptr, lnodes = orc.level_buckets(level)
    want = f64_of_bits(xb)
    for (_, wq, _, wo) in weights:
        want = orc.layer_levelised(want, wq, wo, ptr, idx, lptr, lnodes, 8, 0.25, residual=True, rounding="bf16")
    assert rel_row_err(host_f64_of_bf16(h), want).max() <= BF16_ROW_TOL


def test_stream_ordered_destroy_and_pooled_create():
    """A handle freed in stream order right after its kernels were enqueued: the kernels still see intact arrays,
    and handles created afterwards (served from the library's pool) give the same results."""
    w = synth.workload(5, 400)
    g = w.graph()
    xb = w.x_bf16_bits()
    wq_bits, _ = bf16_weights(w.w_qkv_f32(0))
    wo_bits, _ = bf16_weights(w.w_o_f32(0))
    dsc = dg4.desc(w.heads, dg4.DG4_BF16, w.scale, residual=True)
    outs = []
    for rep in range(4):
        gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0)
        ws = torch.empty(dg4.dg4_layer_workspace_bytes(gr, dsc), dtype=torch.uint8, device="cuda")
        h = dev_bf16(xb).clone()
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        dg4.dg4_layer_fwd_parallel(gr, dsc, h, dev_bf16(wq_bits), dev_bf16(wo_bits), h, ws)
        dg4.dg4_layer_fwd_levelised(gr, dsc, h, dev_bf16(wq_bits), dev_bf16(wo_bits), ws, st)
        dg4.dg4_graph_destroy_async(gr)                    # no wait: the two layers are still queued or running
        assert gr.handle is None
        outs.append((h, st))
    torch.cuda.synchronize()
    for h, st in outs:
        assert int(st.item()) == 0
        assert torch.equal(h, outs[0][0])
    dg4.dg4_memory_trim(0)                                 # the pool gives its free memory back; later creates still work
    gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0)
    assert (dg4.dg4_graph_export(gr, dg4.DG4_ARR_NBR_PTR) == orc.neighbourhood(g.row_ptr, g.col_idx, w.hops)[0]).all()
    dg4.dg4_graph_destroy(gr)


def test_graph_create_from_several_host_threads_under_a_read_back():
    """Graph creation fetches its small results through one staging buffer taken in turn: handles created from
    four host threads at once, of different sizes, while a large device-to-host copy is in flight on another
    stream, all hold the oracle's lists and level buckets, and the host's copy of the level offsets is whole."""
    import threading
    cases = [(2, 40), (3, 40), (2, 7), (4, 40)]
    graphs = [synth.workload(c, s).graph() for c, s in cases]
    big = torch.empty(64 << 20, dtype=torch.int32, device="cuda")
    host = torch.empty(64 << 20, dtype=torch.int32).pin_memory()
    side = torch.cuda.Stream()
    made, errors = [None] * len(cases), []

    def create(i):
        try:
            made[i] = dg4.dg4_graph_create(graphs[i].row_ptr, graphs[i].col_idx, graphs[i].level, 2, 0)
        except Exception as e:                                 # reported by the main thread
            errors.append(e)

    for rep in range(2):
        with torch.cuda.stream(side):
            host.copy_(big, non_blocking=True)
        threads = [threading.Thread(target=create, args=(i,)) for i in range(len(cases))]
        for t in threads:
            t.start()
        for t in threads:
            t.join()
        torch.cuda.synchronize()
        assert not errors
        for i, g in enumerate(graphs):
            ptr, idx = orc.neighbourhood(g.row_ptr, g.col_idx, 2)
            lptr, lnodes = orc.level_buckets(g.level)
            assert made[i].info.n_nbr == len(idx) and made[i].info.n_levels == len(lptr) - 1
            assert (dg4.dg4_graph_export(made[i], dg4.DG4_ARR_NBR_PTR) == ptr).all()
            assert (dg4.dg4_graph_export(made[i], dg4.DG4_ARR_LEVEL_PTR) == lptr).all()
            assert (dg4.dg4_graph_export(made[i], dg4.DG4_ARR_LEVEL_NODES) == lnodes).all()
            # the host's copy of the level offsets drives the one-launch-group-per-level order: same bits as the
            # persistent kernel's order only if every offset arrived
            dsc = dg4.desc(8, dg4.DG4_BF16, 0.25, residual=True)
            by_level = dg4.desc(8, dg4.DG4_BF16, 0.25, residual=True, level_launches=True)
            ws = torch.empty(dg4.dg4_layer_workspace_bytes(made[i], dsc), dtype=torch.uint8, device="cuda")
            xb = synth.normal_bf16_bits(31, i, (g.n, 128), 1.0)
            wq_bits, wq = bf16_weights(synth.normal_f32(31, 50, (384, 128), 0.08))
            wo_bits, wo = bf16_weights(synth.normal_f32(31, 51, (128, 128), 0.08))
            h_a, h_b = dev_bf16(xb).clone(), dev_bf16(xb).clone()
            dg4.dg4_layer_fwd_levelised(made[i], dsc, h_a, dev_bf16(wq_bits), dev_bf16(wo_bits), ws)
            dg4.dg4_layer_fwd_levelised(made[i], by_level, h_b, dev_bf16(wq_bits), dev_bf16(wo_bits), ws)
            torch.cuda.synchronize()
            assert dg4.dg4_graph_poll_status(made[i]) == 0
            assert rel_row_err(host_f64_of_bf16(h_a), host_f64_of_bf16(h_b)).max() <= BF16_ROW_TOL
            if i == 0 and rep == 0:
                want = orc.layer_levelised(f64_of_bits(xb), wq, wo, ptr, idx, lptr, lnodes, 8, 0.25, residual=True,
                                           rounding="bf16")
                assert rel_row_err(host_f64_of_bf16(h_b), want).max() <= BF16_ROW_TOL
            dg4.dg4_graph_destroy(made[i])


@pytest.mark.parametrize("mode", ["parallel", "levelised"])
def test_forward_calls_can_be_captured_in_a_cuda_graph(mode):
    """The forward calls only enqueue work on the caller's stream (no allocation, no synchronisation), so a stack
    of layers can be captured once and replayed: the launch-bound small circuits need that."""
    w = synth.workload(2, 10)
    g = w.graph()
    gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0)
    weights = _weights(w, 3)
    dsc = dg4.desc(w.heads, dg4.DG4_BF16, w.scale, residual=True)
    ws = torch.empty(max(dg4.dg4_layer_workspace_bytes(gr, dsc), dg4.dg4_layers_workspace_bytes(gr, dsc, 3)),
                     dtype=torch.uint8, device="cuda")
    x = dev_bf16(w.x_bf16_bits())
    wq = [dev_bf16(t[0]) for t in weights]
    wo = [dev_bf16(t[2]) for t in weights]
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    h = torch.empty_like(x)

    def run():
        h.copy_(x)
        if mode == "parallel":
            for l in range(3):
                dg4.dg4_layer_fwd_parallel(gr, dsc, h, wq[l], wo[l], h, ws)
        else:
            dg4.dg4_layers_fwd_levelised(gr, dsc, h, wq, wo, ws, status)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run()                                              # first calls outside the capture (one-off function attributes)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    eager = h.clone()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        run()
    for _ in range(2):
        h.zero_()
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(h, eager)
    assert int(status.item()) == 0
