"""GPU parity for the rest of the Transformer block (layer normalisation, feed-forward sub-layer, whole block)
against the CPU checker on the same seeded inputs: bf16 rows within 2e-2 of the row norm of the checker run with
the same storage rounding."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc
from paper_2502_01681_b200 import dg4, synth
from tests.gpu_util import bf16_weights, dev_bf16, f64_of_bits, host_f64_of_bf16
from tests.helpers import csr_from_fanins, random_dag, rel_row_err, levels_of

pytestmark = pytest.mark.gpu

BF16_ROW_TOL = 2e-2
EPS = 1e-5


def _edgeless(n):
    rp, ci = csr_from_fanins([[] for _ in range(n)])
    return dg4.dg4_graph_create(rp, ci, np.zeros(n, np.int32), 1, 0)


def _vec(seed, stream, n, std, mean=0.0):
    v = synth.normal_f32(seed, stream, (n,), std) + np.float32(mean)
    return v.astype(np.float32), torch.from_numpy(v.astype(np.float32)).cuda()


def _ffn_params(seed, w_std=0.08):
    w1_bits, w1 = bf16_weights(synth.normal_f32(seed, 31, (512, 128), w_std))
    w2_bits, w2 = bf16_weights(synth.normal_f32(seed, 32, (128, 512), w_std))
    b1, db1 = _vec(seed, 33, 512, 0.3)
    b2, db2 = _vec(seed, 34, 128, 0.3)
    gam, dgam = _vec(seed, 35, 128, 0.2, 1.0)
    bet, dbet = _vec(seed, 36, 128, 0.2)
    host = (w1, b1.astype(np.float64), w2, b2.astype(np.float64), gam.astype(np.float64), bet.astype(np.float64))
    dev = (dev_bf16(w1_bits), db1, dev_bf16(w2_bits), db2, dgam, dbet)
    return host, dev


@pytest.mark.parametrize("n", [1, 31, 128, 129, 1000])
def test_layernorm_matches_checker(n):
    g = _edgeless(n)
    dsc = dg4.desc(8, dg4.DG4_BF16, 0.25)
    xb = synth.normal_bf16_bits(21, 1, (n, 128), 2.0)
    xb[n // 2] = synth.f32_to_bf16_bits(np.full(128, 3.0, np.float32))       # a constant row: beta comes out
    gam, dgam = _vec(21, 2, 128, 0.5, 1.0)
    bet, dbet = _vec(21, 3, 128, 0.5)
    x = dev_bf16(xb)
    y = torch.empty_like(x)
    dg4.dg4_layernorm_fwd(g, dsc, x, dgam, dbet, EPS, y)
    torch.cuda.synchronize()
    want = orc.round_bf16(orc.layernorm(f64_of_bits(xb), gam, bet, EPS))
    assert rel_row_err(host_f64_of_bf16(y), want).max() <= BF16_ROW_TOL
    dg4.dg4_layernorm_fwd(g, dsc, x, dgam, dbet, EPS, x)                      # in place
    torch.cuda.synchronize()
    assert torch.equal(x, y)


@pytest.mark.parametrize("n", [1, 127, 128, 129, 1000, 20000])
def test_ffn_matches_checker(n):
    g = _edgeless(n)
    dsc = dg4.desc(8, dg4.DG4_BF16, 0.25)
    xb = synth.normal_bf16_bits(22, 1, (n, 128), 1.0)
    host, dev = _ffn_params(22)
    x = dev_bf16(xb)
    y = torch.empty_like(x)
    dg4.dg4_ffn_fwd(g, dsc, x, *dev, EPS, y)
    torch.cuda.synchronize()
    assert dg4.dg4_graph_poll_status(g) == 0
    want = orc.ffn(f64_of_bits(xb), *host, eps=EPS, rounding="bf16")
    assert rel_row_err(host_f64_of_bf16(y), want).max() <= BF16_ROW_TOL
    # the unrounded result is close too (the drift of 16-bit storage stays well inside the tolerance)
    exact = orc.ffn(f64_of_bits(xb), *host, eps=EPS)
    assert rel_row_err(host_f64_of_bf16(y), exact).max() <= BF16_ROW_TOL
    dg4.dg4_ffn_fwd(g, dsc, x, *dev, EPS, x)                                  # in place, and repeatable bit for bit
    torch.cuda.synchronize()
    assert torch.equal(x, y)


def test_ffn_strided_rows_and_switched_off_units():
    n = 300
    g = _edgeless(n)
    dsc = dg4.desc(8, dg4.DG4_BF16, 0.25)
    xb = synth.normal_bf16_bits(23, 1, (n, 128), 1.0)
    host, dev = _ffn_params(23)
    host, dev = list(host), list(dev)
    host[1] = np.full(512, -1e4)                                              # every hidden unit off: LayerNorm(x + b2)
    dev[1] = torch.full((512,), -1e4, device="cuda")
    wide_in = torch.zeros(n, 256, dtype=torch.bfloat16, device="cuda")
    wide_out = torch.full((n, 384), 7.0, dtype=torch.bfloat16, device="cuda")
    wide_in[:, 128:] = dev_bf16(xb)
    dg4.dg4_ffn_fwd(g, dsc, wide_in[:, 128:], *dev, EPS, wide_out[:, 128:256])
    torch.cuda.synchronize()
    want = orc.round_bf16(orc.layernorm(f64_of_bits(xb) + host[3], host[4], host[5], EPS))
    assert rel_row_err(host_f64_of_bf16(wide_out[:, 128:256]), want).max() <= BF16_ROW_TOL
    assert (wide_out[:, :128] == 7.0).all() and (wide_out[:, 256:] == 7.0).all()      # nothing outside the rows


@pytest.mark.parametrize("hops,heads,n", [(1, 8, 700), (2, 4, 2500)])
def test_block_matches_checker(hops, heads, n):
    fanins = random_dag(np.random.default_rng(11 + hops), 20, n - 20, window=64)
    rp, ci = csr_from_fanins(fanins)
    level = levels_of(fanins)
    g = dg4.dg4_graph_create(rp, ci, level, hops, 0)
    scale = 1.0 / np.sqrt(128 // heads)
    dsc = dg4.desc(heads, dg4.DG4_BF16, scale)
    xb = synth.normal_bf16_bits(24, 1, (n, 128), 1.0)
    wq_bits, wq = bf16_weights(synth.normal_f32(24, 2, (384, 128), 0.08))
    wo_bits, wo = bf16_weights(synth.normal_f32(24, 3, (128, 128), 0.08))
    g1, dg1 = _vec(24, 4, 128, 0.2, 1.0)
    be1, dbe1 = _vec(24, 5, 128, 0.2)
    host, dev = _ffn_params(24)
    ws = torch.empty(dg4.dg4_layer_workspace_bytes(g, dsc), dtype=torch.uint8, device="cuda")
    x = dev_bf16(xb)
    out = torch.empty_like(x)
    dg4.dg4_block_fwd_parallel(g, dsc, x, dev_bf16(wq_bits), dev_bf16(wo_bits), dg1, dbe1, *dev, EPS, out, ws)
    torch.cuda.synchronize()
    assert dg4.dg4_graph_poll_status(g) == 0
    ptr, idx = orc.neighbourhood(rp, ci, hops)
    h1 = orc.layer_parallel(f64_of_bits(xb), wq, wo, ptr, idx, heads, scale, residual=True, rounding="bf16")
    h1 = orc.round_bf16(orc.layernorm(h1, g1, be1, EPS))
    want = orc.ffn(h1, *host, eps=EPS, rounding="bf16")
    assert rel_row_err(host_f64_of_bf16(out), want).max() <= BF16_ROW_TOL


@pytest.mark.parametrize("driver", ["persistent", "level-launches"])
@pytest.mark.parametrize("hops,heads,n,window", [(1, 8, 900, 40), (2, 4, 3000, 64), (4, 8, 1500, 50), (2, 16, 20000, 3000),
                                                 (1, 1, 31, 4), (8, 2, 2500, 300)])
def test_block_in_level_order_matches_checker(hops, heads, n, window, driver):
    """The whole block level by level (dg4_block_fwd_levelised): higher levels read the block outputs of lower ones.
    Two drivers: one persistent kernel whose attention-stage and feed-forward-stage CTAs hand the levels to one
    another (cones of at most two hops), and one group of launches per level."""
    fanins = random_dag(np.random.default_rng(31 + hops), 30, n - 30, window=window)
    rp, ci = csr_from_fanins(fanins)
    level = levels_of(fanins)
    g = dg4.dg4_graph_create(rp, ci, level, hops, 0)
    scale = 1.0 / np.sqrt(128 // heads)
    dsc = dg4.desc(heads, dg4.DG4_BF16, scale, level_launches=(driver == "level-launches"))
    xb = synth.normal_bf16_bits(26, 1, (n, 128), 1.0)
    wq_bits, wq = bf16_weights(synth.normal_f32(26, 2, (384, 128), 0.08))
    wo_bits, wo = bf16_weights(synth.normal_f32(26, 3, (128, 128), 0.08))
    g1, dg1 = _vec(26, 4, 128, 0.2, 1.0)
    be1, dbe1 = _vec(26, 5, 128, 0.2)
    host, dev = _ffn_params(26)
    ws = torch.empty(dg4.dg4_layer_workspace_bytes(g, dsc), dtype=torch.uint8, device="cuda")
    h = dev_bf16(xb).clone()
    launches = dg4.dg4_launch_count()
    dg4.dg4_block_fwd_levelised(g, dsc, h, dev_bf16(wq_bits), dev_bf16(wo_bits), dg1, dbe1, *dev, EPS, ws)
    torch.cuda.synchronize()
    assert dg4.dg4_graph_poll_status(g) == 0
    if driver == "persistent":
        assert dg4.dg4_launch_count() - launches == 1       # one kernel for the whole block
    ptr, idx = orc.neighbourhood(rp, ci, hops)
    lptr, lnodes = orc.level_buckets(level)
    w1, b1, w2, b2, g2, be2 = host
    want = orc.block_levelised(f64_of_bits(xb), wq, wo, g1, be1, w1, b1, w2, b2, g2, be2, ptr, idx, lptr, lnodes, heads,
                               scale, eps=EPS, rounding="bf16")
    got = host_f64_of_bf16(h)
    assert rel_row_err(got, want).max() <= BF16_ROW_TOL
    # level 0 sees no updated row: there the level order and the all-at-once block agree bit for bit
    out = torch.empty_like(h)
    dg4.dg4_block_fwd_parallel(g, dsc, dev_bf16(xb), dev_bf16(wq_bits), dev_bf16(wo_bits), dg1, dbe1, *dev, EPS, out, ws)
    torch.cuda.synchronize()
    lvl0 = torch.from_numpy(np.nonzero(level == 0)[0]).cuda()
    assert torch.equal(h[lvl0], out[lvl0]) and not torch.equal(h, out)


def test_block_in_level_order_with_empty_levels_and_many_tiles_per_level():
    """A layering with gaps (every level number tripled) and levels wider than the feed-forward stage's CTAs x 16
    nodes: both drivers give the same rows bit for bit (same arithmetic, same order), and they match the oracle."""
    fanins = random_dag(np.random.default_rng(77), 3000, 9000, window=6000)
    rp, ci = csr_from_fanins(fanins)
    level = (levels_of(fanins) * 3).astype(np.int32)
    n = len(fanins)
    g = dg4.dg4_graph_create(rp, ci, level, 2, 0)
    assert np.bincount(level).max() > 75 * 16
    heads, scale = 8, 0.25
    xb = synth.normal_bf16_bits(27, 1, (n, 128), 1.0)
    wq_bits, wq = bf16_weights(synth.normal_f32(27, 2, (384, 128), 0.08))
    wo_bits, wo = bf16_weights(synth.normal_f32(27, 3, (128, 128), 0.08))
    g1, dg1 = _vec(27, 4, 128, 0.2, 1.0)
    be1, dbe1 = _vec(27, 5, 128, 0.2)
    host, dev = _ffn_params(27)
    outs = []
    for launches in (False, True):
        dsc = dg4.desc(heads, dg4.DG4_BF16, scale, level_launches=launches)
        ws = torch.empty(dg4.dg4_layer_workspace_bytes(g, dsc), dtype=torch.uint8, device="cuda")
        h = dev_bf16(xb).clone()
        dg4.dg4_block_fwd_levelised(g, dsc, h, dev_bf16(wq_bits), dev_bf16(wo_bits), dg1, dbe1, *dev, EPS, ws)
        torch.cuda.synchronize()
        assert dg4.dg4_graph_poll_status(g) == 0
        outs.append(h)
    ptr, idx = orc.neighbourhood(rp, ci, 2)
    lptr, lnodes = orc.level_buckets(level)
    w1, b1, w2, b2, g2, be2 = host
    want = orc.block_levelised(f64_of_bits(xb), wq, wo, g1, be1, w1, b1, w2, b2, g2, be2, ptr, idx, lptr, lnodes, heads,
                               scale, eps=EPS, rounding="bf16")
    for h in outs:
        assert rel_row_err(host_f64_of_bf16(h), want).max() <= BF16_ROW_TOL


@pytest.mark.parametrize("hops,n_blocks", [(2, 3), (1, 2), (4, 2)])
def test_blocks_as_one_wavefront_equal_successive_blocks(hops, n_blocks):
    """dg4_blocks_fwd_levelised: the stages of all blocks as one wavefront give, bit for bit, what one
    dg4_block_fwd_levelised call per block gives; and that matches the oracle applied block after block."""
    fanins = random_dag(np.random.default_rng(91 + hops), 60, 6000, window=150)
    rp, ci = csr_from_fanins(fanins)
    level = levels_of(fanins)
    n = len(fanins)
    g = dg4.dg4_graph_create(rp, ci, level, hops, 0)
    heads, scale = 8, 0.25
    dsc = dg4.desc(heads, dg4.DG4_BF16, scale)
    xb = synth.normal_bf16_bits(28, 1, (n, 128), 1.0)
    host_blocks, dev_blocks = [], []
    for k in range(n_blocks):
        wq_bits, wq = bf16_weights(synth.normal_f32(28, 10 * k + 2, (384, 128), 0.08))
        wo_bits, wo = bf16_weights(synth.normal_f32(28, 10 * k + 3, (128, 128), 0.08))
        g1, dg1 = _vec(28, 10 * k + 4, 128, 0.2, 1.0)
        be1, dbe1 = _vec(28, 10 * k + 5, 128, 0.2)
        host, dev = _ffn_params(28 + k)
        host_blocks.append((wq, wo, g1, be1) + tuple(host))
        dev_blocks.append((dev_bf16(wq_bits), dev_bf16(wo_bits), dg1, dbe1) + tuple(dev))
    ws = torch.empty(max(dg4.dg4_blocks_workspace_bytes(g, dsc, n_blocks), dg4.dg4_layer_workspace_bytes(g, dsc)),
                     dtype=torch.uint8, device="cuda")
    h = dev_bf16(xb).clone()
    launches = dg4.dg4_launch_count()
    dg4.dg4_blocks_fwd_levelised(g, dsc, h, dev_blocks, EPS, ws)
    torch.cuda.synchronize()
    assert dg4.dg4_graph_poll_status(g) == 0 and dg4.dg4_launch_count() - launches == 1
    h2 = dev_bf16(xb).clone()
    for blk in dev_blocks:
        dg4.dg4_block_fwd_levelised(g, dsc, h2, *blk, EPS, ws)
    torch.cuda.synchronize()
    assert dg4.dg4_graph_poll_status(g) == 0
    assert torch.equal(h.view(torch.int16), h2.view(torch.int16))
    ptr, idx = orc.neighbourhood(rp, ci, hops)
    lptr, lnodes = orc.level_buckets(level)
    want = f64_of_bits(xb)
    for (wq, wo, g1, be1, w1, b1, w2, b2, g2, be2) in host_blocks:
        want = orc.block_levelised(want, wq, wo, g1, be1, w1, b1, w2, b2, g2, be2, ptr, idx, lptr, lnodes, heads, scale,
                                   eps=EPS, rounding="bf16")
    assert rel_row_err(host_f64_of_bf16(h), want).max() <= BF16_ROW_TOL


def test_blocks_wavefront_can_be_captured_in_a_cuda_graph():
    """The persistent block kernel (a cooperative launch in clusters of two) only enqueues on the caller's stream:
    captured once, its replays give the bits of the eager call."""
    fanins = random_dag(np.random.default_rng(97), 40, 3000, window=120)
    rp, ci = csr_from_fanins(fanins)
    n = len(fanins)
    g = dg4.dg4_graph_create(rp, ci, levels_of(fanins), 2, 0)
    dsc = dg4.desc(8, dg4.DG4_BF16, 0.25)
    x = dev_bf16(synth.normal_bf16_bits(29, 1, (n, 128), 1.0))
    blocks = []
    for k in range(2):
        wq_bits, _ = bf16_weights(synth.normal_f32(29, 10 * k + 2, (384, 128), 0.08))
        wo_bits, _ = bf16_weights(synth.normal_f32(29, 10 * k + 3, (128, 128), 0.08))
        blocks.append((dev_bf16(wq_bits), dev_bf16(wo_bits), _vec(29, 10 * k + 4, 128, 0.2, 1.0)[1],
                       _vec(29, 10 * k + 5, 128, 0.2)[1]) + tuple(_ffn_params(29 + k)[1]))
    ws = torch.empty(dg4.dg4_blocks_workspace_bytes(g, dsc, 2), dtype=torch.uint8, device="cuda")
    h = torch.empty_like(x)
    side = torch.cuda.Stream()

    def run():
        h.copy_(x)
        dg4.dg4_blocks_fwd_levelised(g, dsc, h, blocks, EPS, ws)

    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        run()
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
        assert torch.equal(h.view(torch.int16), eager.view(torch.int16))
    assert dg4.dg4_graph_poll_status(g) == 0
    dg4.dg4_graph_destroy(g)


def test_block_calls_reject_bad_arguments():
    n = 64
    g = _edgeless(n)
    dsc = dg4.desc(8, dg4.DG4_BF16, 0.25)
    host, dev = _ffn_params(25)
    x = torch.zeros(n, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_ffn_fwd(g, dsc, x, dev[0][:256], *dev[1:], EPS, x)            # d_ff = 256
    assert e.value.status == dg4.DG4_ERR_UNSUPPORTED
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_ffn_fwd(g, dsc, x, *dev, -1.0, x)
    assert e.value.status == dg4.DG4_ERR_INVALID_ARG
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_layernorm_fwd(g, dsc, x, dev[4][1:], dev[5], EPS, x)          # misaligned gamma
    assert e.value.status == dg4.DG4_ERR_INVALID_ARG
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_ffn_fwd(g, dg4.desc(4, dg4.DG4_F32, 0.25), x, *dev, EPS, x)
    assert e.value.status == dg4.DG4_ERR_UNSUPPORTED
    # several blocks in one call: block count and workspace size are checked on the host, nothing is launched
    blk = (torch.zeros(384, 128, dtype=torch.bfloat16, device="cuda"), torch.zeros(128, 128, dtype=torch.bfloat16, device="cuda"),
           dev[4], dev[5]) + tuple(dev)
    ws = torch.empty(dg4.dg4_blocks_workspace_bytes(g, dsc, 2), dtype=torch.uint8, device="cuda")
    launches = dg4.dg4_launch_count()
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_blocks_fwd_levelised(g, dsc, x, [blk] * 9, EPS, ws)
    assert e.value.status == dg4.DG4_ERR_UNSUPPORTED
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_blocks_fwd_levelised(g, dsc, x, [blk] * 3, EPS, ws)           # workspace sized for two blocks
    assert e.value.status == dg4.DG4_ERR_INVALID_ARG
    with pytest.raises(dg4.Dg4Error) as e:
        dg4.dg4_blocks_fwd_levelised(g, dsc, x, [blk[:6] + (dev[2][:, :256],) + blk[7:]] * 2, EPS, ws[1:])   # misaligned workspace
    assert e.value.status == dg4.DG4_ERR_INVALID_ARG
    assert dg4.dg4_launch_count() == launches
    assert dg4.dg4_blocks_workspace_bytes(g, dsc, 0) == 0 and dg4.dg4_blocks_workspace_bytes(g, dsc, 9) == 0
