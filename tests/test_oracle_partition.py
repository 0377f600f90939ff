"""Pins for capacity estimate (Eq. 1-3), partition optimiser (Eq. 4-7), Algorithm 1 and schedules."""
import itertools

import numpy as np
import pytest

import oracle

RNG = np.random.default_rng(11)


def exact_inputs(L, N, comm):
    """Integer times and dyadic capacities: every sum and product is exact in float64."""
    t = [float(v) for v in RNG.integers(1, 40, size=L)]
    c = [float(v) for v in RNG.choice([0.5, 1.0, 2.0, 4.0, 8.0, 1.5], size=N)]
    if not comm:
        return t, c, None, None
    d = [float(v) for v in RNG.integers(1, 64, size=L)]
    bw = [float(v) for v in RNG.choice([1.0, 2.0, 4.0], size=N - 1)]
    return t, c, d, bw


@pytest.mark.parametrize("comm", [False, True])
def test_dp_equals_brute_force_every_cell(comm):
    for L, N in [(1, 1), (2, 2), (5, 1), (6, 3), (7, 4), (9, 5), (8, 8)]:
        for _ in range(6):
            t, c, d, bw = exact_inputs(L, N, comm)
            A, cut = oracle.partition_table(t, c, d, bw)
            for n in range(1, N + 1):
                for j in range(n - 1, L):       # every prefix problem
                    _, best = oracle.brute_force_partition(t[:j + 1], c[:n], None if d is None else d[:j + 1],
                                                           None if bw is None else bw[:n - 1])
                    assert A[n][j] == best
            pts, bott = oracle.choose_partition(t, c, d, bw)
            _, best = oracle.brute_force_partition(t, c, d, bw)
            assert bott == best == oracle.stage_cost(pts, t, c, d, bw)
            assert pts[0] == 0 and pts[-1] == L and all(a < b for a, b in zip(pts, pts[1:]))
            # canonical tie rule: last cut = smallest l reaching the optimum, recursively
            j, n = L - 1, N
            for p in reversed(pts[1:-1]):
                cands = [l for l in range(n - 2, j)
                         if max(A[n - 1][l], 0.0 if d is None else 2.0 * (d[l] / bw[n - 2]),
                                c[n - 1] * (sum(t[:j + 1]) - sum(t[:l + 1]))) == A[n][j]]
                assert p - 1 == min(cands)
                j, n = p - 1, n - 1


def test_dp_special_cases():
    assert oracle.choose_partition([3.0, 1.0, 2.0], [1.0]) == ([0, 3], 6.0)
    assert oracle.choose_partition([1.0] * 12, [1.0] * 4) == ([0, 3, 6, 9, 12], 3.0)
    t = [float(v) for v in RNG.integers(1, 9, size=10)]
    c = [1.0, 2.0, 4.0]
    p1, b1 = oracle.choose_partition(t, c)
    p2, b2 = oracle.choose_partition(t, [4.0 * v for v in c])      # common scale: same points
    assert p1 == p2 and b2 == 4.0 * b1
    # a 10x slower last stage gets fewer units than a fast one
    fast, _ = oracle.choose_partition([1.0] * 20, [1.0, 1.0, 1.0])
    slow, _ = oracle.choose_partition([1.0] * 20, [1.0, 1.0, 10.0])
    assert slow[-1] - slow[-2] < fast[-1] - fast[-2]
    # an expensive link moves the cut to the small boundary
    pts, _ = oracle.choose_partition([1.0] * 4, [1.0, 1.0], [100.0, 100.0, 1.0, 100.0], [10.0])
    assert pts == [0, 3, 4]
    with pytest.raises(ValueError):
        oracle.choose_partition([1.0, 1.0], [1.0, 1.0, 1.0])


def test_capacity_estimate_recovers_slowdown_factors():
    t = [float(v) for v in RNG.integers(1, 9, size=9)]
    pts = [0, 2, 5, 9]
    f = [1.0, 2.5, 10.0]
    stage = [f[i] * sum(t[a:b]) for i, (a, b) in enumerate(zip(pts, pts[1:]))]
    assert np.allclose(oracle.estimate_capacity(t, pts, stage), f)
    stage[0] *= 3.0                                   # C_0 is 1.0 by definition whatever stage 0 reports
    assert oracle.estimate_capacity(t, pts, stage)[0] == 1.0


def all_partitions(L, N):
    for cuts in itertools.combinations(range(1, L), N - 1):
        yield [0] + list(cuts) + [L]


def test_redistribution_without_failure_invariants():
    L, N = 7, 3
    for p_cur in all_partitions(L, N):
        for p_new in all_partitions(L, N):
            for i in range(N):
                need, local = oracle.redistribution_plan(p_new, p_cur, i, i)
                got = sorted(local + [l for v in need.values() for l in v])
                assert got == list(range(p_new[i], p_new[i + 1]))           # covers the new range once
                assert all(p_cur[i] <= l < p_cur[i + 1] for l in local)     # local = already held
                for owner, units in need.items():
                    assert owner != i
                    assert all(p_cur[owner] <= l < p_cur[owner + 1] for l in units)
                if p_new == p_cur:
                    assert need == {} and local == list(range(p_cur[i], p_cur[i + 1]))


def test_redistribution_failure_rules_from_the_prose():
    # Sec. III-F: 4 workers, worker 1 fails; survivors 0,2,3 become 0,1,2.
    p_cur, p_new = [0, 2, 4, 6, 8], [0, 3, 6, 8]
    assert oracle.renew_worker_list([0, 1, 2, 3], [1]) == [0, 2, 3]
    # old worker 2 (new index 1) needs units 3..5: unit 3 was the failed worker's -> its replica sits
    # on failed+1, whose new index equals the failed index (target unchanged); 4,5 are its own.
    need, local = oracle.redistribution_plan(p_new, p_cur, 2, 1, i_fail=1)
    assert local == [4, 5] and need == {1: [3]}
    # old worker 0 needs unit 2 (failed worker's) -> index 1 as well
    need, local = oracle.redistribution_plan(p_new, p_cur, 0, 0, i_fail=1)
    assert local == [0, 1] and need == {1: [2]}
    # old worker 3 (new 2): target above the failed index moves down by one
    need, local = oracle.redistribution_plan([0, 2, 5, 8], p_cur, 3, 2, i_fail=1)
    assert local == [6, 7] and need == {1: [5]}      # unit 5 lived on old worker 2 -> new index 1
    # last stage fails: its replica is on the central node, index 0
    need, local = oracle.redistribution_plan([0, 3, 6, 8], p_cur, 2, 2, i_fail=3)
    assert local == [] or all(4 <= l < 6 for l in local)
    assert need.get(0) == [6, 7]


def _compositions(L, n):
    import itertools
    for cuts in itertools.combinations(range(1, L), n - 1):
        yield [0, *cuts, L]


def test_recovery_sources_single_failure_equals_algorithm_1():
    """With one failed worker the prose of Sec. III-F and the printed Algorithm 1 must name the same
    place for every unit: the plan built from the prose is compared with Algorithm 1 run for every
    surviving worker, over every pair of partitions of 6 units on 4 -> 3 workers."""
    L, n = 6, 4
    for p_cur in _compositions(L, n):
        for p_new in _compositions(L, n - 1):
            for f in range(1, n):
                alive = oracle.renew_worker_list(list(range(n)), [f])
                plan = oracle.recovery_sources(p_cur, [f], p_new)
                for j, old in enumerate(alive):
                    need, local = oracle.redistribution_plan(p_new, p_cur, old, j, i_fail=f)
                    want = {}
                    for u, src in plan[j]:
                        if src[0] == "local":
                            assert u in local
                        else:
                            assert src[0] in ("stage", "replica")       # one failure never needs the global replica
                            want.setdefault(src[1], []).append(u)
                    assert want == need, (p_cur, p_new, f, j)


def test_recovery_sources_every_source_really_holds_the_unit():
    """A small world: worker i holds its units; worker i+1 keeps the chain replica of worker i, the
    central node (0) that of the last worker and the global replica of everything.  After any set of
    failures every unit of every new stage must come from a place that survived and has it, the new
    ranges must cover all units exactly once, and the global replica is used only when a failed
    worker's neighbour failed too."""
    import itertools
    L, n = 7, 5
    for p_cur in list(_compositions(L, n))[::3]:
        for k in (1, 2, 3):
            for failed in itertools.combinations(range(1, n), k):
                alive = oracle.renew_worker_list(list(range(n)), list(failed))
                p_new = next(_compositions(L, len(alive)))
                plan = oracle.recovery_sources(p_cur, list(failed), p_new)
                seen = []
                for j, items in enumerate(plan):
                    for u, src in items:
                        seen.append(u)
                        holder = next(i for i in range(n) if p_cur[i] <= u < p_cur[i + 1])
                        if src[0] == "local":
                            assert holder == alive[j]
                        elif src[0] == "stage":
                            assert alive[src[1]] == holder and holder not in failed
                        elif src[0] == "replica":
                            keeper = 0 if holder == n - 1 else holder + 1
                            assert holder in failed and alive[src[1]] == keeper and keeper not in failed
                        else:
                            assert holder in failed and holder != n - 1 and holder + 1 in failed
                assert seen == list(range(L))


def test_schedules_match_the_paper(golden_dir):
    facts = {}
    for line in open(golden_dir + "/schedule_ticks.txt"):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            facts[k] = int(v)
    first, period = facts["repartition_first_batches"], facts["repartition_period"]
    hits = [it + 1 for it in range(450) if oracle.is_repartition_iter(it)]
    assert hits == [first, period, 2 * period, 3 * period, 4 * period]
    chain = [it + 1 for it in range(210) if oracle.is_replication_iter(it, facts["chain_period"])]
    glob = [it + 1 for it in range(210) if oracle.is_replication_iter(it, facts["global_period"])]
    assert chain == [50, 100, 150, 200] and glob == [100, 200]
    assert facts["both_replications_after_batch"] in chain and facts["both_replications_after_batch"] in glob


def _facts(golden_dir):
    facts = {}
    for line in open(golden_dir + "/schedule_ticks.txt"):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            facts[k] = int(v)
    return facts


def test_state_variables_start_as_table_one_says(golden_dir):
    """Sec. III-B, Table I: both committed ids are initialised as -1 and the status as 0."""
    from oracle import recovery as R
    facts = _facts(golden_dir)
    st = R.TrainState(0.1, 300, 196)
    assert st.committed_forward_id == facts["committed_id_init"] and st.committed_backward_id == facts["committed_id_init"]
    assert st.status == facts["status_init"]
    assert (st.learning_rate, st.epoch_number, st.batch_number) == (0.1, 300, 196)


def test_fault_handler_state_follows_section_three_f():
    """The worked case of Sec. IV-E in the words of Sec. III-F: the worker dies when batch 205 starts its backward
    pass.  Batches up to 204 have gone all the way round, 205..207 have been forwarded into the pipeline.  The
    timer of 205 triggers the handler once (status 1), later timers do not; batches beyond the committed forward
    id are held back; the reset sets both ids to 205, the status to 0, and training resumes by forwarding 205."""
    from oracle import recovery as R
    st = R.TrainState(0.1, 1, 1000)
    for b in range(208):
        st.forward_done(b)
        if b - 3 >= 0:
            st.backward_done(b - 3)
    assert (st.committed_forward_id, st.committed_backward_id, st.status) == (207, 204, 0)
    assert st.may_forward(208)
    assert st.timer_expired(205) is True and st.status == 1
    assert st.timer_expired(206) is False and st.timer_expired(207) is False and st.status == 1
    assert not st.may_forward(208) and st.may_forward(207)
    assert st.reset(205) == 205
    assert (st.committed_forward_id, st.committed_backward_id, st.status) == (205, 205, 0)
    assert st.may_forward(206)


def test_probe_outcomes_are_the_three_cases_of_the_paper():
    from oracle import recovery as R
    N, S, X = R.NORMAL, R.RESTARTED, R.SILENT
    assert R.classify_probe([N, N, N, N]) == (R.RESTART_BATCH, [], None)              # all respond normally
    assert R.classify_probe([N, N, S, N]) == (R.RESEND_STATE, [], 2)                  # one restarted at once
    assert R.classify_probe([N, X, N, X]) == (R.REDISTRIBUTE, [1, 3], None)           # multiple workers silent
    assert R.classify_probe([N, N, X, N]) == (R.REDISTRIBUTE, [2], None)              # one silent: Algorithm 1 with its index
    assert R.classify_probe([N, S, X, N]) == (R.REDISTRIBUTE, [1, 2], None)           # a restart beside a failure: both lost their weights
    # the failed list is what the recovery plan takes: survivors keep their order
    action, failed, _ = R.classify_probe([N, X, N, X, N])
    assert oracle.renew_worker_list([0, 1, 2, 3, 4], failed) == [0, 2, 4]
    plan = oracle.recovery_sources([0, 2, 4, 6, 8, 10], failed, [0, 4, 7, 10])
    assert [u for items in plan for u, _ in items] == list(range(10))
