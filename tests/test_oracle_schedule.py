"""Pins for the asynchronous pipeline schedule of Sec. III-C: the prose example of the paper (three devices,
batches 0 to 6 on stage 0), invariants of the 1F1B order, and the float64 simulation against closed forms."""
import numpy as np
import pytest

import oracle
import synth
from oracle import schedule as S


def test_one_f_one_b_order_of_the_papers_example():
    """Three stages, stage 0: three batches are fed first; "the backwarding of batch 1 follows immediately after
    the forwarding of batch 3"."""
    order = S.stage_order(3, 0, 7)
    assert order[:9] == [("F", 0), ("F", 1), ("F", 2), ("B", 0), ("F", 3), ("B", 1), ("F", 4), ("B", 2), ("F", 5)]
    assert order.index(("B", 1)) == order.index(("F", 3)) + 1


@pytest.mark.parametrize("n,nb", [(1, 5), (2, 3), (3, 7), (4, 9), (5, 2)])
def test_one_f_one_b_invariants(n, nb):
    for s in range(n):
        order = S.stage_order(n, s, nb)
        assert sorted(order) == sorted([("F", b) for b in range(nb)] + [("B", b) for b in range(nb)])
        in_flight, most = 0, 0
        for kind, b in order:
            if kind == "B":
                assert ("F", b) in order[:order.index(("B", b))]
            in_flight += 1 if kind == "F" else -1
            most = max(most, in_flight)
        assert most == min(n - s, nb)                       # n - i batches in flight on stage i: n - i weight versions
        assert [b for k, b in order if k == "F"] == list(range(nb)) and [b for k, b in order if k == "B"] == list(range(nb))


def test_version_numbers_of_the_papers_example():
    """3_f^1, 4_f^2, 5_f^3; batch 1 is backwarded with version 0; the aggregation of the three versions turns version 3
    into 4, the backward pass of batch 3 makes 5, and batch 6 is forwarded with version 5."""
    fwd, after_bwd, agg = S.version_trace(3, 0, 8)
    assert fwd[:7] == [0, 0, 0, 1, 2, 3, 5]
    assert after_bwd[:4] == [1, 2, 3, 5]
    assert agg[0] == 5                                       # the aggregation follows the forward pass of batch 5
    # the last of three stages has one version: a forward, then its backward, nothing to aggregate
    fwd2, after2, agg2 = S.version_trace(3, 2, 4)
    assert fwd2 == [0, 1, 2, 3] and after2 == [1, 2, 3, 4] and agg2 == []


def _pipeline(points, nb, k=1, momentum=0.9):
    ls, cfg = synth.tiny_mbv2(momentum=momentum)
    ap = S.AsyncPipeline(ls, cfg, synth.init_params(5, ls), synth.init_state(ls), points, k)
    batches = [synth.make_batch(5, cfg, t) for t in range(nb)]
    return ls, cfg, ap, batches


def test_simulation_follows_the_example_on_stage_zero_and_vertical_sync_on_the_last_stage():
    ls, cfg, ap, batches = _pipeline([0, 2, 5, 7], 8)
    ap.run(batches, 0.01)
    s0 = [e for e in ap.log if e[1] == 0]
    assert s0[:12] == [("F", 0, 0, 0), ("F", 0, 1, 0), ("F", 0, 2, 0), ("B", 0, 0, 0, 1), ("F", 0, 3, 1), ("B", 0, 1, 0, 2), ("F", 0, 4, 2),
                       ("B", 0, 2, 0, 3), ("F", 0, 5, 3), ("A", 0, [3, 4, 5], 4), ("B", 0, 3, 1, 5), ("F", 0, 6, 5)]
    s2 = [e for e in ap.log if e[1] == 2]
    # "it forwards batch 1 with weight version 0 even though the weight version is updated to 1 when backwarding batch 0 in stage 2"
    assert s2[:3] == [("F", 2, 0, 0), ("B", 2, 0, 0, 1), ("F", 2, 1, 0)]
    assert not [e for e in s2 if e[0] == "A"]


def test_a_single_stage_is_plain_sequential_training():
    """One stage: forward, backward, update, one batch at a time, no stale weights, nothing to aggregate: the simulation
    must reproduce OracleModel.step batch by batch."""
    ls, cfg, ap, batches = _pipeline([0, 7], 4)
    losses = ap.run(batches, 0.01)
    om = oracle.OracleModel(ls, cfg, synth.init_params(5, ls), synth.init_state(ls), storage="none")
    ref = [om.step([0, om.L], x, y, 0.01) for x, y in batches]
    assert losses == ref
    for u in range(om.L):
        assert np.array_equal(ap.master.unit_params(u), om.unit_params(u)) and np.array_equal(ap.master.unit_state(u), om.unit_state(u))


def test_aggregation_is_the_mean_of_the_stashed_versions():
    """Two stages, plain SGD (no momentum): on stage 0 the second update is followed by F3 and the aggregation of the two
    stashed versions v1 (batch 2) and v2 (batch 3).  With w_1 = w_0 - lr g_0 and w_2 = w_1 - lr g_1 the aggregate is
    w_0 - lr g_0 - lr g_1 / 2, whatever the gradients are; checked on the stem's weights."""
    ls, cfg, ap, batches = _pipeline([0, 3, 7], 4, momentum=0.0)
    w0 = ap.master.unit_params(0).copy()
    seen = {}
    orig = ap.master.sgd

    def spy(a, b, lr=None):                                   # the gradients the updates of stage 0 used, in order
        if a == 0:
            seen[len(seen)] = ap.master.unit_grads(0).copy() + cfg["weight_decay"] * ap.master.unit_params(0)
        orig(a, b, lr)
    ap.master.sgd = spy
    ap.run(batches, 0.01)
    agg = [e for e in ap.log if e[0] == "A" and e[1] == 0]
    assert agg and agg[0] == ("A", 0, [2, 3], 3)
    want = w0 - 0.01 * seen[0] - 0.01 * seen[1] / 2
    assert np.allclose(ap.history[0][3][0][0][0].reshape(-1), want[:ap.history[0][3][0][0][0].size], rtol=0, atol=1e-15)
