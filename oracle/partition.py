"""Capacity estimate, partition optimiser, brute-force partition, weight-redistribution plan
and the periodic schedules, as the paper states them (test infrastructure only).

Units are 0-indexed; a partition is N+1 boundaries 0 = p_0 < p_1 < ... < p_N = L and stage i
runs units [p_i, p_{i+1}).
"""
import itertools

__all__ = ["estimate_capacity", "choose_partition", "partition_table", "brute_force_partition",
           "stage_cost", "redistribution_plan", "is_repartition_iter", "is_replication_iter",
           "renew_worker_list", "recovery_sources"]


def estimate_capacity(layer_times, points, stage_times):
    """Eq. 1-3: C_i = measured mean batch time of stage i / sum of the central node's per-layer
    times over that stage's layers; C_0 is 1.0 by definition."""
    caps = []
    for i, (a, b) in enumerate(zip(points[:-1], points[1:])):
        t0 = 0.0
        for j in range(a, b):
            t0 = t0 + layer_times[j]
        caps.append(stage_times[i] / t0)
    caps[0] = 1.0
    return caps


def _prefix(layer_times):
    s = [0.0]
    for t in layer_times:
        s.append(s[-1] + t)
    return s


def _comm(l, n, out_bytes, bandwidth):
    """2 * T_c of Eq. 4-5: activation forward plus gradient backward over the link between
    stage n-2 and stage n-1, for a cut after unit l."""
    if out_bytes is None or bandwidth is None:
        return 0.0
    return 2.0 * (out_bytes[l] / bandwidth[n - 2])


def partition_table(layer_times, capacities, out_bytes=None, bandwidth=None):
    """Eq. 4-7.  A[n][j] = least possible slowest-part time for units 0..j on the first n stages.
    A(j,1) = T^0(0,j);  A(j,n) = min_l max{ A(l,n-1), 2*T_c(l, n-2), T^{n-1}(l+1, j) } over cuts l
    that leave every stage non-empty.  Returns (A, cut) with cut[n][j] the smallest minimising l."""
    L, N = len(layer_times), len(capacities)
    S = _prefix(layer_times)
    INF = float("inf")
    A = [[INF] * L for _ in range(N + 1)]
    cut = [[-1] * L for _ in range(N + 1)]
    for j in range(L):
        A[1][j] = capacities[0] * (S[j + 1] - S[0])
    for n in range(2, N + 1):
        for j in range(n - 1, L):
            best, arg = INF, -1
            for l in range(n - 2, j):
                last = capacities[n - 1] * (S[j + 1] - S[l + 1])
                v = max(A[n - 1][l], _comm(l, n, out_bytes, bandwidth), last)
                if v < best:
                    best, arg = v, l
            A[n][j], cut[n][j] = best, arg
    return A, cut


def choose_partition(layer_times, capacities, out_bytes=None, bandwidth=None):
    """Partition points of the optimal pipeline and its bottleneck time A(L-1, N)."""
    L, N = len(layer_times), len(capacities)
    if N < 1 or N > L:
        raise ValueError("need 1 <= N <= L")
    A, cut = partition_table(layer_times, capacities, out_bytes, bandwidth)
    points = [L]
    j = L - 1
    for n in range(N, 1, -1):
        l = cut[n][j]
        points.append(l + 1)
        j = l
    points.append(0)
    return points[::-1], A[N][L - 1]


def stage_cost(points, layer_times, capacities, out_bytes=None, bandwidth=None):
    """Slowest part of a given partition, evaluated directly (not through the recurrence)."""
    S = _prefix(layer_times)
    worst = 0.0
    for i, (a, b) in enumerate(zip(points[:-1], points[1:])):
        worst = max(worst, capacities[i] * (S[b] - S[a]))
        if i >= 1:
            worst = max(worst, _comm(a - 1, i + 1, out_bytes, bandwidth))
    return worst


def brute_force_partition(layer_times, capacities, out_bytes=None, bandwidth=None):
    """Enumerate every way to cut L units into N non-empty contiguous stages."""
    L, N = len(layer_times), len(capacities)
    best, arg = float("inf"), None
    for cuts in itertools.combinations(range(1, L), N - 1):
        pts = [0] + list(cuts) + [L]
        v = stage_cost(pts, layer_times, capacities, out_bytes, bandwidth)
        if v < best:
            best, arg = v, pts
    return arg, best


def redistribution_plan(p_new, p_cur, i_cur, i_new, i_fail=-1, n_nodes=None):
    """Algorithm 1.  For the worker that was index i_cur and becomes index i_new: which units of
    its new range it already holds (L_local) and, per owner index, which it must fetch (M_need).
    p_cur is indexed by the OLD worker list; owners are reported in the NEW list's indices.
    Without a failure (i_fail < 0) no index correction applies (Sec. III-D)."""
    if i_cur is None or i_cur < 0:
        held = range(0)
    else:
        held = range(p_cur[i_cur], p_cur[i_cur + 1])
    needed = range(p_new[i_new], p_new[i_new + 1])
    missing = [l for l in needed if l not in held]
    l_local = [l for l in needed if l not in missing]
    m_need = {}
    last_old = (len(p_cur) - 2) if n_nodes is None else n_nodes
    for l in missing:
        target = next(i for i in range(len(p_cur) - 1) if p_cur[i] <= l < p_cur[i + 1])
        if i_fail >= 0:
            if target > i_fail:
                target -= 1
            elif target == i_fail and i_fail == last_old:
                target = 0
        m_need.setdefault(target, []).append(l)
    return m_need, l_local


def renew_worker_list(workers, failed):
    """Sec. III-F: drop the failed workers; the survivors keep their order, so every index above
    a failed one moves down."""
    return [w for w in workers if w not in failed]


def recovery_sources(p_cur, failed, p_new):
    """Sec. III-F, recovery after one or several workers failed.  p_cur is indexed by the old worker
    list, p_new by the renewed one (survivors in order).  For every new stage j the units of its new
    range with where their weights come from:
      ("local",)        the worker holds the unit already;
      ("stage", i)      the live weights of surviving worker i (new index);
      ("replica", i)    the chain replica of a failed worker, kept by the worker after it in the old
                        list (new index i), or by the central node (i = 0) when the last worker failed;
      ("central",)      the global replica on the central node: the failed worker's neighbour failed too.
    Worker 0 is the central node and does not fail (Sec. III-E)."""
    n_cur = len(p_cur) - 1
    failed = sorted(set(failed))
    assert failed and all(0 < f < n_cur for f in failed), "failed workers must be among 1 .. n_cur-1"
    alive = renew_worker_list(list(range(n_cur)), failed)
    assert len(p_new) - 1 == len(alive), "the new partition must have one stage per survivor"
    plan = []
    for j, old in enumerate(alive):
        items = []
        for u in range(p_new[j], p_new[j + 1]):
            holder = next(i for i in range(n_cur) if p_cur[i] <= u < p_cur[i + 1])
            if holder == old:
                src = ("local",)
            elif holder not in failed:
                src = ("stage", alive.index(holder))
            elif holder == n_cur - 1:
                src = ("replica", 0)
            elif holder + 1 not in failed:
                src = ("replica", alive.index(holder + 1))
            else:
                src = ("central",)
            items.append((u, src))
        plan.append(items)
    return plan


def is_repartition_iter(it, first=10, period=100):
    """Sec. III-D: repartition after the first 10 batches, then every 100 batches.
    `it` is the 0-indexed batch that has just finished."""
    done = it + 1
    return done == first or (done > first and done % period == 0)


def is_replication_iter(it, period):
    """Sec. IV-B / IV-E: replication runs when a batch whose 1-indexed count is a multiple of
    the period has finished (chain every 50, global every 100: both when batch 200 finishes)."""
    return (it + 1) % period == 0
