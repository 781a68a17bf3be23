"""Error paths of the forward calls on a GPU, exercised without anything faulting, trapping or hanging:
a call made with the wrong device current is refused on the host, and device-side waits that run out (forced by
a poll limit of one, not by anything being stuck) make each pipelined kernel wind down, report DG4_ERR_TIMEOUT and
leave the context usable for a normal call right after."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2502_01681_b200 import dg4, synth
from tests.gpu_util import bf16_weights, dev_bf16, f64_of_bits, host_f64_of_bf16
from tests.helpers import rel_row_err

pytestmark = pytest.mark.gpu
BF16_ROW_TOL = 2e-2


def _small_problem():
    w = synth.workload(5, 400)                 # ~25k nodes, 2-hop cones: a few tiles per SM, dozens of levels
    g = w.graph()
    xb = w.x_bf16_bits()
    wq_bits, wq = bf16_weights(w.w_qkv_f32(0))
    wo_bits, wo = bf16_weights(w.w_o_f32(0))
    return w, g, xb, (wq_bits, wq), (wo_bits, wo)


def test_forward_calls_refuse_a_foreign_device():
    w, g, xb, (wq_bits, _), (wo_bits, _) = _small_problem()
    gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0)
    dsc = dg4.desc(w.heads, dg4.DG4_BF16, w.scale, residual=True)
    n = g.n
    x, dwq, dwo = dev_bf16(xb), dev_bf16(wq_bits), dev_bf16(wo_bits)
    q, k, v, o = (torch.zeros(n, 128, dtype=torch.bfloat16, device="cuda") for _ in range(4))
    ws = torch.empty(max(dg4.dg4_layer_workspace_bytes(gr, dsc), dg4.dg4_layers_workspace_bytes(gr, dsc, 2)),
                     dtype=torch.uint8, device="cuda")
    sd = torch.zeros(n, w.heads, device="cuda")
    vec = torch.ones(128, device="cuda")
    b1 = torch.zeros(512, device="cuda")
    w1 = torch.zeros(512, 128, dtype=torch.bfloat16, device="cuda")
    w2 = torch.zeros(128, 512, dtype=torch.bfloat16, device="cuda")
    calls = {
        "qkv": lambda: dg4.dg4_qkv_project(gr, dsc, x, dwq, q, k, v),
        "attn": lambda: dg4.dg4_sparse_attn_fwd(gr, dsc, q, k, v, o),
        "additive": lambda: dg4.dg4_sparse_attn_additive_fwd(gr, dsc, sd, sd, 0.2, v, o),
        "out": lambda: dg4.dg4_out_project(gr, dsc, o, dwo, x, q),
        "layer": lambda: dg4.dg4_layer_fwd_parallel(gr, dsc, x, dwq, dwo, o, ws),
        "levelised": lambda: dg4.dg4_layer_fwd_levelised(gr, dsc, q, dwq, dwo, ws),
        "layers": lambda: dg4.dg4_layers_fwd_levelised(gr, dsc, q, [dwq, dwq], [dwo, dwo], ws),
        "static": lambda: dg4.dg4_layer_fwd_parallel_static(gr, dsc, x, dwq, dwo, o),
        "layernorm": lambda: dg4.dg4_layernorm_fwd(gr, dsc, x, vec, vec, 1e-5, o),
        "ffn": lambda: dg4.dg4_ffn_fwd(gr, dsc, x, w1, b1, w2, vec, vec, vec, 1e-5, o),
        "block": lambda: dg4.dg4_block_fwd_parallel(gr, dsc, x, dwq, dwo, vec, vec, w1, b1, w2, vec, vec, vec, 1e-5, o, ws),
        "rebuild": lambda: dg4.dg4_graph_rebuild(gr),
    }
    launches = dg4.dg4_launch_count()
    dg4.dg4_debug_override_current_device(1)           # as if another GPU were current on this thread
    try:
        for name, call in calls.items():
            with pytest.raises(dg4.Dg4Error) as e:
                call()
            assert e.value.status == dg4.DG4_ERR_INVALID_ARG, name
            assert "device" in e.value.detail, name
    finally:
        dg4.dg4_debug_override_current_device(-1)
    assert dg4.dg4_launch_count() == launches           # refused on the host: nothing was launched
    calls["layer"]()                                    # and accepted again with the check back to normal
    torch.cuda.synchronize()
    assert dg4.dg4_graph_poll_status(gr) == 0


def test_waits_that_run_out_wind_the_kernels_down_and_report_timeout():
    w, g, xb, (wq_bits, wq), (wo_bits, wo) = _small_problem()
    n = g.n
    dsc = dg4.desc(w.heads, dg4.DG4_BF16, w.scale, residual=True)
    x, dwq, dwo = dev_bf16(xb), dev_bf16(wq_bits), dev_bf16(wo_bits)
    w1 = (torch.randn(512, 128, device="cuda") * 0.05).to(torch.bfloat16)
    w2 = (torch.randn(128, 512, device="cuda") * 0.05).to(torch.bfloat16)
    b1, vec = torch.zeros(512, device="cuda"), torch.ones(128, device="cuda")
    q, k, v, y = (torch.zeros(n, 128, dtype=torch.bfloat16, device="cuda") for _ in range(4))

    def fresh():
        gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0)
        ws = torch.empty(dg4.dg4_layers_workspace_bytes(gr, dsc, 3), dtype=torch.uint8, device="cuda")
        return gr, ws

    dg4.dg4_debug_set_poll_limit(1)
    try:
        gr, ws = fresh()                                # projection kernel
        dg4.dg4_qkv_project(gr, dsc, x, dwq, q, k, v)
        assert dg4.dg4_graph_poll_status(gr) == dg4.DG4_ERR_TIMEOUT
        gr, ws = fresh()                                # feed-forward kernel
        dg4.dg4_ffn_fwd(gr, dsc, x, w1, b1, w2, vec, vec, vec, 1e-5, y)
        assert dg4.dg4_graph_poll_status(gr) == dg4.DG4_ERR_TIMEOUT
        gr, ws = fresh()                                # one-kernel form of the parallel layer (behind its K|V projection)
        h = x.clone()
        dg4.dg4_layer_fwd_parallel(gr, dg4.desc(w.heads, dg4.DG4_BF16, w.scale, residual=True, fused_layer=True),
                                   h, dwq, dwo, h, ws)
        assert dg4.dg4_graph_poll_status(gr) == dg4.DG4_ERR_TIMEOUT
        gr, ws = fresh()                                # the block level by level as one persistent kernel
        h = x.clone()
        dg4.dg4_block_fwd_levelised(gr, dsc, h, dwq, dwo, vec, vec * 0, w1, b1, w2, vec * 0, vec, vec * 0, 1e-5, ws)
        torch.cuda.synchronize()
        assert dg4.dg4_graph_poll_status(gr) == dg4.DG4_ERR_TIMEOUT
        gr, ws = fresh()                                # persistent levelised kernel (its table-filling projection too)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        h = x.clone()
        dg4.dg4_layers_fwd_levelised(gr, dsc, h, [dwq] * 3, [dwo] * 3, ws, status)
        torch.cuda.synchronize()
        assert int(status.item()) == dg4.DG4_ERR_TIMEOUT
    finally:
        dg4.dg4_debug_set_poll_limit(0)
    # the context is intact and the same calls, with the default limit, give the right answer
    assert float((torch.ones(8, device="cuda") * 2).sum().item()) == 16.0
    gr, ws = fresh()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    h = x.clone()
    dg4.dg4_layers_fwd_levelised(gr, dsc, h, [dwq] * 3, [dwo] * 3, ws, status)
    dg4.dg4_qkv_project(gr, dsc, x, dwq, q, k, v)
    hf = x.clone()
    dg4.dg4_layer_fwd_parallel(gr, dg4.desc(w.heads, dg4.DG4_BF16, w.scale, residual=True, fused_layer=True),
                               hf, dwq, dwo, hf, ws)
    torch.cuda.synchronize()
    assert int(status.item()) == 0 and dg4.dg4_graph_poll_status(gr) == 0
    want_par = orc.layer_parallel(f64_of_bits(xb), wq, wo, *orc.neighbourhood(g.row_ptr, g.col_idx, w.hops), w.heads,
                                  w.scale, residual=True, rounding="bf16")
    assert rel_row_err(host_f64_of_bf16(hf), want_par).max() <= BF16_ROW_TOL
    ptr, idx = orc.neighbourhood(g.row_ptr, g.col_idx, w.hops)
    lptr, lnodes = orc.level_buckets(g.level)
    want = f64_of_bits(xb)
    for _ in range(3):
        want = orc.layer_levelised(want, wq, wo, ptr, idx, lptr, lnodes, w.heads, w.scale, residual=True, rounding="bf16")
    assert rel_row_err(host_f64_of_bf16(h), want).max() <= BF16_ROW_TOL
    want_qkv = orc.round_bf16(orc.project(f64_of_bits(xb), wq))
    got_qkv = np.concatenate([host_f64_of_bf16(t) for t in (q, k, v)], axis=1)
    assert rel_row_err(got_qkv, want_qkv).max() <= BF16_ROW_TOL
