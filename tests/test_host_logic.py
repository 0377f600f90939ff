"""CPU tests of the library's host side: exported symbols, the scheduling arithmetic against the
oracle (bit-exact), model validation and workspace planning.  No kernel is launched."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import synth

F = pytest.importorskip("paper_2110_02781_b200")
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", fn)).read()
        names |= set(re.findall(r"\b(ftp_[a-z0-9_]+)\s*\(", text))
    assert len(names) >= 25
    lib = ctypes.CDLL(F.LIB_PATH)
    for n in sorted(names):
        assert hasattr(lib, n), f"{n} is declared but not exported"


def test_choose_partition_bit_exact_with_oracle():
    rng = np.random.default_rng(5)
    for trial in range(300):
        L = int(rng.integers(1, 21))
        N = int(rng.integers(1, min(L, 5) + 1))
        t = rng.uniform(1e-5, 3e-3, L).tolist()
        c = rng.uniform(1.0, 10.0, N).tolist()
        comm = trial % 3 == 0 and N > 1
        d = rng.integers(1 << 10, 1 << 26, L).astype(float).tolist() if comm else None
        bw = rng.uniform(1e8, 1e11, N - 1).tolist() if comm else None
        got_p, got_b = F.ftp_choose_partition(t, c, d, bw)
        ref_p, ref_b = oracle.choose_partition(t, c, d, bw)
        assert got_p == ref_p and got_b == ref_b            # == on floats: bit-exact
    # ties everywhere: identical layers
    assert F.ftp_choose_partition([1.0] * 12, [1.0] * 4)[0] == oracle.choose_partition([1.0] * 12, [1.0] * 4)[0]
    with pytest.raises(F.FtpError):
        F.ftp_choose_partition([1.0, 2.0], [1.0, 1.0, 1.0])
    with pytest.raises(F.FtpError):
        F.ftp_choose_partition([1.0, 2.0], [1.0, 1.0], [1.0, 1.0], None)


def test_estimate_capacity_bit_exact_with_oracle():
    rng = np.random.default_rng(6)
    for _ in range(100):
        L = int(rng.integers(2, 21))
        N = int(rng.integers(1, min(L, 5) + 1))
        t = rng.uniform(1e-5, 3e-3, L).tolist()
        pts = [0] + sorted(rng.choice(np.arange(1, L), N - 1, replace=False).tolist()) + [L]
        st = rng.uniform(1e-4, 1e-1, N).tolist()
        assert F.ftp_estimate_capacity(t, pts, st) == oracle.estimate_capacity(t, pts, st)
    with pytest.raises(F.FtpError):
        F.ftp_estimate_capacity([1.0, 1.0], [0, 2, 1], [1.0, 1.0])


@pytest.mark.parametrize("i_fail", [-1, 0, 1, 2, 3])
def test_redistribution_plan_equals_oracle(i_fail):
    rng = np.random.default_rng(8)
    L = 9
    for _ in range(150):
        n_cur = 4
        n_new = n_cur if i_fail < 0 else n_cur - 1
        p_cur = [0] + sorted(rng.choice(np.arange(1, L), n_cur - 1, replace=False).tolist()) + [L]
        p_new = [0] + sorted(rng.choice(np.arange(1, L), n_new - 1, replace=False).tolist()) + [L]
        survivors = [w for w in range(n_cur) if w != i_fail]
        for i_new, i_cur in enumerate(survivors):
            owners, n_local = F.ftp_redistribution_plan(p_new, p_cur, i_cur, i_new, i_fail)
            need, local = oracle.redistribution_plan(p_new, p_cur, i_cur, i_new, i_fail)
            ref = [-1] * (p_new[i_new + 1] - p_new[i_new])
            for owner, units in need.items():
                for u in units:
                    ref[u - p_new[i_new]] = owner
            assert owners == ref and n_local == len(local)


def test_workspace_and_validation_without_gpu():
    for net in (synth.har_cnn(), synth.tiny_mbv2(), synth.tiny_vgg(), synth.mobilenetv2(128, 32, 10, 0, True)):
        dev, pin = F.ftp_workspace_bytes(*net)
        assert dev > 0 and dev % 256 == 0 and pin > 0
    ls, cfg = synth.tiny_mbv2()
    bad = list(ls)
    bad[2] = bad[2]._replace(cin=bad[2].cin + 1)                      # shapes no longer chain
    with pytest.raises(F.FtpError):
        F.ftp_workspace_bytes(bad, cfg)
    bad = list(ls)[:-1]                                               # no loss at the end
    with pytest.raises(F.FtpError):
        F.ftp_workspace_bytes(bad, cfg)
    bad = [l._replace(unit=l.unit + (2 if i > 3 else 0)) for i, l in enumerate(ls)]   # a gap in the unit ids
    with pytest.raises(F.FtpError):
        F.ftp_workspace_bytes(bad, cfg)
    add = next(i for i, l in enumerate(ls) if l.kind == synth.KIND["ADD_RESIDUAL"])
    bad = list(ls)
    bad[add] = bad[add]._replace(residual_src=0)                      # residual reaching across a unit edge
    with pytest.raises(F.FtpError):
        F.ftp_workspace_bytes(bad, cfg)
    with pytest.raises(F.FtpError):
        F.ftp_workspace_bytes(ls, dict(cfg, batch=0))


def test_recovery_plan_equals_oracle():
    """ftp_recovery_plan (Sec. III-F) against the oracle's plan, unit by unit, over random partitions and every set
    of up to three failed workers out of five; bad failure lists are refused."""
    import itertools
    rng = np.random.default_rng(9)
    L, n_cur = 11, 5
    code = {"local": F.SRC_LOCAL, "stage": F.SRC_STAGE, "replica": F.SRC_REPLICA, "central": F.SRC_CENTRAL}
    for _ in range(40):
        p_cur = [0] + sorted(rng.choice(np.arange(1, L), n_cur - 1, replace=False).tolist()) + [L]
        for k in (1, 2, 3):
            for failed in itertools.combinations(range(1, n_cur), k):
                n_new = n_cur - k
                p_new = [0] + sorted(rng.choice(np.arange(1, L), n_new - 1, replace=False).tolist()) + [L]
                kind, index = F.ftp_recovery_plan(p_cur, list(failed), p_new)
                for j, items in enumerate(oracle.recovery_sources(p_cur, list(failed), p_new)):
                    for u, src in items:
                        assert kind[u] == code[src[0]], (p_cur, failed, p_new, u)
                        want = j if src[0] == "local" else (src[1] if len(src) > 1 else 0)
                        assert index[u] == want, (p_cur, failed, p_new, u)
    for bad in ([0], [5], [2, 2]):
        with pytest.raises(F.FtpError):
            F.ftp_recovery_plan([0, 2, 4, 6, 8, 11], bad, [0, 3, 6, 11] if len(bad) == 2 else [0, 3, 6, 8, 11])
    with pytest.raises(F.FtpError):
        F.ftp_recovery_plan([0, 2, 4, 6, 8, 11], [1], [0, 3, 6, 11])          # one failure leaves four stages, not three



def test_train_state_and_probe_match_the_oracle():
    """The Table I state and the fault handler's decisions (Sec. III-F), library against oracle on random event
    sequences and on every response pattern of up to five workers."""
    import itertools
    from oracle import recovery as R
    rng = np.random.default_rng(11)
    for trial in range(50):
        lr, ep, nb = float(rng.uniform(0.001, 1.0)), int(rng.integers(1, 400)), int(rng.integers(1, 2000))
        o, g = R.TrainState(lr, ep, nb), F.ftp_state_init(lr, ep, nb)
        same = lambda: (o.committed_forward_id, o.committed_backward_id, o.status, ep, nb) == \
            (g.committed_forward_id, g.committed_backward_id, g.status, g.epoch_number, g.batch_number)
        assert same() and g.committed_forward_id == -1 and g.status == 0 and abs(g.learning_rate - lr) < 1e-6
        for _ in range(60):
            ev, b = int(rng.integers(0, 5)), int(rng.integers(0, 300))
            if ev == 0:
                o.forward_done(b); F.ftp_state_forward_done(g, b)
            elif ev == 1:
                o.backward_done(b); F.ftp_state_backward_done(g, b)
            elif ev == 2:
                assert o.timer_expired(b) == F.ftp_state_timer_expired(g, b)
            elif ev == 3:
                assert o.reset(b) == F.ftp_state_reset(g, b)
            assert o.may_forward(b) == F.ftp_state_may_forward(g, b) and same()
    for n in range(1, 6):
        for rest in itertools.product((0, 1, 2), repeat=n - 1):
            resp = [0] + list(rest)
            assert F.ftp_classify_probe(resp) == R.classify_probe(resp)
    with pytest.raises(F.FtpError):
        F.ftp_classify_probe([2, 0])                      # the central node does not fail


def test_schedule_helpers_match_the_oracle():
    for it in range(-2, 1300):
        assert F.ftp_is_repartition_iter(it) == oracle.is_repartition_iter(it) if it >= 0 else not F.ftp_is_repartition_iter(it)
        for period in (20, 50, 100):
            assert F.ftp_is_replication_iter(it, period) == (oracle.is_replication_iter(it, period) if it >= 0 else False)
    assert [it + 1 for it in range(450) if F.ftp_is_repartition_iter(it)] == [10, 100, 200, 300, 400]
    assert F.ftp_is_repartition_iter(6, 7, 5) and F.ftp_is_repartition_iter(9, 7, 5) and not F.ftp_is_repartition_iter(7, 7, 5)
