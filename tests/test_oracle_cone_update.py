"""Pins for the CPU checker's cone-by-cone updating (Sec. 3.4 over Algorithm 1's partition, `orc.cone_update`):
a hand-worked schedule, an independent dense restatement (reachability by boolean matrix powers, masked attention
by torch) on small random circuits, cases that reduce to routines pinned elsewhere, and invariants.  CPU only."""
import os

import numpy as np
import torch

from oracle import oracle as orc
from tests.helpers import binary_in_tree, csr_from_fanins, levels_of, random_dag

GOLDEN_AIG = os.path.join(os.path.dirname(__file__), "golden", "tiny_aig.txt")
GOLDEN_RUN = os.path.join(os.path.dirname(__file__), "golden", "cone_update_tiny.txt")
D, HEADS = 16, 4


def _weights(rng, layers, d=D, std=0.15):
    return ([rng.normal(0, std, (3 * d, d)) for _ in range(layers)], [rng.normal(0, std, (d, d)) for _ in range(layers)])


def _dense_layer(x, wq, wo, mask, heads, scale, residual):
    """One attention layer with a dense boolean mask (mask[i, j]: i attends to j), by torch's dense algebra."""
    x = torch.from_numpy(x)
    m, d = x.shape
    dh = d // heads
    qkv = x @ torch.from_numpy(wq).T
    q, k, v = (t.reshape(m, heads, dh).permute(1, 0, 2) for t in (qkv[:, :d], qkv[:, d:2 * d], qkv[:, 2 * d:]))
    s = scale * (q @ k.transpose(1, 2))
    s = s.masked_fill(~torch.from_numpy(mask)[None], float("-inf"))
    o = (torch.softmax(s, dim=-1) @ v).permute(1, 0, 2).reshape(m, d)
    y = o @ torch.from_numpy(wo).T
    return (y + x if residual else y).numpy()


def _reach_within(fanins, k):
    """R[u, v]: a path u -> v of length <= k exists (u == v included), by boolean matrix powers."""
    n = len(fanins)
    A = np.zeros((n, n), bool)
    for v, f in enumerate(fanins):
        for u in f:
            A[u, v] = True
    R = np.eye(n, dtype=bool)
    P = np.eye(n, dtype=bool)
    for _ in range(k):
        P = (P.astype(np.int64) @ A.astype(np.int64)) > 0
        R |= P
    return R


def _groups_by_walking_levels(fanins, level, k, delta):
    n = len(fanins)
    fed = {u for f in fanins for u in f}
    groups, l = {}, k
    while l <= int(level.max()):
        groups[l] = {v for v in range(n) if level[v] == l}
        l += delta
    for v in range(n):
        if v not in fed:
            groups.setdefault(int(level[v]), set()).add(v)
    return groups


def _dense_cone_update(fanins, level, X, wq_list, wo_list, k, delta, batch, heads, scale, residual, schedule=None):
    """The updating strategy restated with dense masks; `schedule` (optional) receives, per mini-batch, the
    sub-graph, the frozen gates, the attention sets and the stored gates."""
    R = _reach_within(fanins, k)
    groups = _groups_by_walking_levels(fanins, level, k, delta)
    hist, updated, stored, n_batches = X.copy(), set(), np.zeros(len(fanins), np.int32), 0
    for l in sorted(groups):
        roots = sorted(groups[l])
        for b in range(0, len(roots), batch):
            S = sorted({int(u) for r in roots[b:b + batch] for u in np.nonzero(R[:, r])[0]})
            frozen = [v for v in S if v in updated]
            mask = np.array([[(i == j) or (S[i] not in updated and R[S[j], S[i]]) for j in range(len(S))]
                             for i in range(len(S))])
            x = hist[S]
            for wq, wo in zip(wq_list, wo_list):
                x = _dense_layer(x, wq, wo, mask, heads, scale, residual)
            keep = [i for i, v in enumerate(S) if v not in updated]
            for i in keep:
                hist[S[i]] = x[i]
                stored[S[i]] += 1
            if schedule is not None:
                schedule.append((S, frozen, {S[i]: [S[j] for j in np.nonzero(mask[i])[0]] for i in range(len(S))},
                                 [S[i] for i in keep]))
            updated |= set(S)
            n_batches += 1
    return hist, stored, n_batches


def _tiny_circuit():
    fanins = []
    for line in open(GOLDEN_AIG):
        line = line.strip()
        if line and not line.startswith("#"):
            f = [p.strip() for p in line.split("|")]
            fanins.append([] if f[1] == "-" else [int(t) for t in f[1].split()])
    return fanins


def _read_hand_worked_schedule():
    out = []
    for line in open(GOLDEN_RUN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        f = [p.strip() for p in line.split("|")]
        ints = lambda t: [] if t == "-" else [int(x) for x in t.split()]
        att = {}
        for item in f[3].split(";"):
            gate, lst = item.split(":")
            att[int(gate)] = sorted(ints(lst.strip()))
        out.append((ints(f[1]), ints(f[2]), att, ints(f[4])))
    return out


def test_hand_worked_schedule_on_the_tiny_circuit():
    """The dense restatement reproduces the hand-worked mini-batches, frozen sets, attention sets and stored gates;
    the checker then agrees with the restatement's numbers, so both are tied to the hand-worked run."""
    fanins = _tiny_circuit()
    level = levels_of(fanins)
    rp, ci = csr_from_fanins(fanins)
    rng = np.random.default_rng(3)
    X = rng.normal(0, 1, (len(fanins), D))
    wq, wo = _weights(rng, 2)
    schedule = []
    want, stored, nb = _dense_cone_update(fanins, level, X, wq, wo, 2, 1, 1, HEADS, 0.5, True, schedule)
    hand = _read_hand_worked_schedule()
    assert len(schedule) == len(hand) == nb == 4
    for (S, frozen, att, kept), (hS, hfrozen, hatt, hkept) in zip(schedule, hand):
        assert S == hS and frozen == hfrozen and kept == hkept
        assert {g: sorted(a) for g, a in att.items()} == hatt
    got, got_stored, got_nb = orc.cone_update(X, wq, wo, rp, ci, level, 2, 1, 1, HEADS, 0.5)
    assert got_nb == 4 and (got_stored == 1).all() and (stored == 1).all()
    assert np.abs(got - want).max() <= 1e-12
    # the fixture's remark: with these cones, mini-batches of two give the same embeddings, in three mini-batches
    got2, _, nb2 = orc.cone_update(X, wq, wo, rp, ci, level, 2, 1, 2, HEADS, 0.5)
    assert nb2 == 3 and np.abs(got2 - got).max() <= 1e-12


def test_dense_restatement_on_random_circuits():
    rng = np.random.default_rng(11)
    for trial, (k, delta, batch, layers, residual) in enumerate([(2, 1, 1, 1, True), (2, 1, 3, 2, True),
                                                                 (3, 2, 4, 2, False), (4, 3, 2, 3, True),
                                                                 (8, 6, 5, 1, True), (3, 1, 100, 2, True)]):
        fanins = random_dag(rng, 5, 60, window=7)
        level = levels_of(fanins)
        rp, ci = csr_from_fanins(fanins)
        X = rng.normal(0, 1, (len(fanins), D))
        wq, wo = _weights(rng, layers)
        want, stored, nb = _dense_cone_update(fanins, level, X, wq, wo, k, delta, batch, HEADS, 0.5, residual)
        got, got_stored, got_nb = orc.cone_update(X, wq, wo, rp, ci, level, k, delta, batch, HEADS, 0.5, residual=residual)
        assert got_nb == nb and (got_stored == stored).all(), trial
        assert np.abs(got - want).max() <= 1e-12 * max(1.0, np.abs(want).max()), trial


def test_one_cone_covering_the_circuit_is_the_parallel_layer_stack():
    # complete binary in-tree of depth 3 with k = 3: the only root is the tree's root and its cone is everything
    fanins, root, level = binary_in_tree(3)
    rp, ci = csr_from_fanins(fanins)
    rng = np.random.default_rng(5)
    X = rng.normal(0, 1, (len(fanins), D))
    wq, wo = _weights(rng, 2)
    got, stored, nb = orc.cone_update(X, wq, wo, rp, ci, level, 3, 2, 128, HEADS, 0.5)
    ptr, idx = orc.neighbourhood(rp, ci, 3)
    want = X
    for a, b in zip(wq, wo):
        want = orc.layer_parallel(want, a, b, ptr, idx, HEADS, 0.5, residual=True)
    assert nb == 1 and (stored == 1).all() and np.abs(got - want).max() <= 1e-12


def test_chain_reduces_to_the_levelised_layer():
    """A chain of inverters, k = 2, delta = 1, one cone per mini-batch, one layer: the first cone {0, 1, 2} is encoded
    at once (all three from their input rows), every later gate from the stored rows of its two predecessors --
    the levelised layer with the buckets {0, 1, 2}, {3}, {4}, ..."""
    n = 12
    fanins = [[]] + [[i - 1] for i in range(1, n)]
    rp, ci = csr_from_fanins(fanins)
    level = levels_of(fanins)
    rng = np.random.default_rng(8)
    X = rng.normal(0, 1, (n, D))
    wq, wo = _weights(rng, 1)
    got, stored, nb = orc.cone_update(X, wq, wo, rp, ci, level, 2, 1, 1, HEADS, 0.5)
    ptr, idx = orc.neighbourhood(rp, ci, 2)
    bucket_ptr = np.array([0, 3] + list(range(4, n + 1)), np.int32)
    want = orc.layer_levelised(X, wq[0], wo[0], ptr, idx, bucket_ptr, np.arange(n, dtype=np.int32), HEADS, 0.5)
    assert nb == n - 2 and (stored == 1).all() and np.abs(got - want).max() <= 1e-12


def test_disjoint_circuits_do_not_depend_on_the_mini_batch_size():
    # several separate chains: their cones never meet, so how many share a mini-batch cannot matter
    fanins, length, copies = [], 7, 5
    for c in range(copies):
        base = len(fanins)
        fanins += [[]] + [[base + i - 1] for i in range(1, length)]
    rp, ci = csr_from_fanins(fanins)
    level = levels_of(fanins)
    rng = np.random.default_rng(9)
    X = rng.normal(0, 1, (len(fanins), D))
    wq, wo = _weights(rng, 2)
    ref, _, nb1 = orc.cone_update(X, wq, wo, rp, ci, level, 3, 2, 1, HEADS, 0.5)
    for batch in (2, 5, 1000):
        got, stored, nb = orc.cone_update(X, wq, wo, rp, ci, level, 3, 2, batch, HEADS, 0.5)
        assert np.abs(got - ref).max() <= 1e-12 and nb <= nb1 and (stored == 1).all()


def test_counts_and_coverage():
    rng = np.random.default_rng(21)
    fanins = random_dag(rng, 8, 300, window=12)
    level = levels_of(fanins)
    rp, ci = csr_from_fanins(fanins)
    n = len(fanins)
    X = rng.normal(0, 1, (n, D))
    wq, wo = _weights(rng, 1)
    for k, delta, batch in ((2, 1, 7), (8, 6, 128), (4, 3, 1)):
        got, stored, nb = orc.cone_update(X, wq, wo, rp, ci, level, k, delta, batch, HEADS, 0.5)
        roots, gptr = orc.partition_roots(rp, ci, level, k, delta)
        ptr, idx = orc.neighbourhood(rp, ci, k)
        covered = np.zeros(n, bool)
        for r in roots:
            covered[idx[ptr[r]:ptr[r + 1]]] = True
        assert ((stored == 1) == covered).all() and stored.max() <= 1        # each covered gate stored exactly once
        assert (got[~covered] == X[~covered]).all()                          # the others keep their input row
        assert nb == sum(-(-int(c) // batch) for c in np.diff(gptr))         # ceil(cones of a level / batch), summed
    # 16-bit storage: every row of the table is a bfloat16 value
    got, _, _ = orc.cone_update(X, wq, wo, rp, ci, level, 4, 3, 5, HEADS, 0.5, rounding="bf16")
    assert (orc.round_bf16(got) == got).all()
