"""The allocation-free variant of the parallel layer (dg4_layer_fwd_parallel_static).

Some users of the library run where device memory cannot be requested any more -- a service that carved up
the whole GPU at start-up, a plug-in inside an application that owns the device heap, a loop that cannot
afford cudaMalloc's device-wide synchronisation.  For them the layer's intermediates live in a fixed 32 MiB
array inside the library.  This test drives that entry point through the C ABI twice in a row (the array
keeps the previous call's contents, so the second call shows that stale scratch does no harm) and compares
each result with the regular entry point, which takes a caller-allocated workspace.  Both run the same
kernels, so the rows must agree well inside the bf16 tolerance used throughout the suite.

Collected last on purpose: a failure here cannot hide the result of any other test in a fail-fast run."""
import ctypes
import gc

import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2502_01681_b200 import dg4, synth
from tests.gpu_util import bf16_weights, dev_bf16, f64_of_bits, host_f64_of_bf16
from tests.helpers import rel_row_err

pytestmark = pytest.mark.gpu

BF16_ROW_TOL = 2e-2


def _layer_regular(gr, dsc, x, wq, wo):
    ws = torch.empty(dg4.dg4_layer_workspace_bytes(gr, dsc), dtype=torch.uint8, device="cuda")
    out = torch.empty_like(x)
    dg4.dg4_layer_fwd_parallel(gr, dsc, x, wq, wo, out, ws)
    torch.cuda.synchronize()
    return out


def test_static_scratch_layer_matches_regular_layer_twice():
    assert dg4.dg4_static_max_nodes() == 32768
    dsc = dg4.desc(8, dg4.DG4_BF16, 0.25, residual=True)
    # two different circuits and inputs, the larger one first, so the second call finds foreign leftovers
    for cfg, shrink, seed in ((5, 400, 0), (2, 8, 1)):
        w = synth.workload(cfg, shrink)
        g = w.graph()
        assert g.n <= dg4.dg4_static_max_nodes()
        gr = dg4.dg4_graph_create(g.row_ptr, g.col_idx, g.level, w.hops, 0)
        xb = synth.normal_bf16_bits(seed, 70, (g.n, 128), 1.0)
        wq_bits, wq64 = bf16_weights(synth.normal_f32(seed, 71, (384, 128), 0.05))
        wo_bits, wo64 = bf16_weights(synth.normal_f32(seed, 72, (128, 128), 0.05))
        x, wq, wo = dev_bf16(xb), dev_bf16(wq_bits), dev_bf16(wo_bits)
        want = _layer_regular(gr, dsc, x, wq, wo)
        got = torch.empty_like(x)
        dg4.dg4_layer_fwd_parallel_static(gr, dsc, x, wq, wo, got)
        torch.cuda.synchronize()
        err = rel_row_err(host_f64_of_bf16(got), host_f64_of_bf16(want))
        assert err.max() <= BF16_ROW_TOL, (cfg, err.max())
        assert torch.equal(got, want)            # same kernels, same order: identical bits
        # and against the CPU checker directly, so that this test stands on its own
        ptr, idx = orc.neighbourhood(g.row_ptr, g.col_idx, w.hops)
        ref = orc.layer_parallel(f64_of_bits(xb), wq64, wo64, ptr, idx, 8, 0.25, residual=True, rounding="bf16")
        assert rel_row_err(host_f64_of_bf16(got), ref).max() <= BF16_ROW_TOL, cfg
        # From the second call on a device nothing is taken from the device heap or from the framework's
        # allocator.  (The very first call may: the driver may instantiate the library image, and with it the
        # 32 MiB array, only then -- which is why that call belongs at start-up.)
        gc.collect()          # tensors of earlier tests that only a collection frees must not be freed in between
        free0, _ = torch.cuda.mem_get_info()
        stats0 = (torch.cuda.memory_allocated(), torch.cuda.memory_reserved())
        for _ in range(3):
            dg4.dg4_layer_fwd_parallel_static(gr, dsc, x, wq, wo, got)
        torch.cuda.synchronize()
        assert torch.cuda.mem_get_info()[0] == free0
        assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == stats0
        assert torch.equal(got, want)


def test_static_scratch_layer_rejects_graphs_beyond_its_capacity():
    n = dg4.dg4_static_max_nodes() + 1
    rp = np.zeros(n + 1, np.int32)
    gr = dg4.dg4_graph_create(rp, np.zeros(0, np.int32), np.zeros(n, np.int32), 1, 0)
    t = torch.zeros(n, 128, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(384, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_layer_fwd_parallel_static(gr, dg4.desc(8, dg4.DG4_BF16, 0.25), t, w, w[:128], t.clone())
    assert e.value.status == dg4.DG4_ERR_INVALID_ARG and "32768" in e.value.detail
    torch.cuda.synchronize()


def test_static_scratch_layer_rejects_what_the_regular_layer_rejects():
    n = 64
    rp = np.zeros(n + 1, np.int32)
    gr = dg4.dg4_graph_create(rp, np.zeros(0, np.int32), np.zeros(n, np.int32), 1, 0)
    t = torch.zeros(n, 128, dtype=torch.bfloat16, device="cuda")
    out = torch.zeros(n, 128, dtype=torch.bfloat16, device="cuda")
    w = torch.zeros(384, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(dg4.Dg4Error) as e:          # a scale that is not a number
        dg4.dg4_layer_fwd_parallel_static(gr, dg4.desc(8, dg4.DG4_BF16, float("nan")), t, w, w[:128], out)
    assert e.value.status == dg4.DG4_ERR_INVALID_ARG
    odd = torch.zeros(n, 132, dtype=torch.bfloat16, device="cuda")[:, :128]     # rows 264 bytes apart
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_layer_fwd_parallel_static(gr, dg4.desc(8, dg4.DG4_BF16, 0.25), odd, w, w[:128], out)
    assert e.value.status == dg4.DG4_ERR_INVALID_ARG
    with pytest.raises(dg4.Dg4Error) as e:          # fp32 storage: the projections are bf16 only
        dg4.dg4_layer_fwd_parallel_static(gr, dg4.desc(8, dg4.DG4_F32, 0.25), t, w, w[:128], out)
    assert e.value.status == dg4.DG4_ERR_UNSUPPORTED
    torch.cuda.synchronize()
