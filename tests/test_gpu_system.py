"""GPU tests of the scheduling side of the path: profile -> capacity -> partition, re-homing of
weights (Algorithm 1 + commit), snapshots (bit-exact), the fused SGD+snapshot, error returns."""
import numpy as np
import pytest

import oracle
import synth
from helpers import clear_batch, gpu_step_split, make_gpu, make_oracle, perturb, rel_err, to_dev, TOL_FP32

pytestmark = pytest.mark.gpu
F = pytest.importorskip("paper_2110_02781_b200")


def test_profile_then_partition_matches_oracle_choice():
    import torch
    ls, cfg = synth.mobilenetv2(16, 32, 10, 0, True)
    gm = make_gpu(ls, cfg, 30)
    x, y = synth.make_batch(30, cfg)
    state0 = [gm.ftp_get_tensor(F.T_STATE, u) for u in range(gm.L)]
    w0 = [gm.ftp_get_tensor(F.T_WEIGHTS, u) for u in range(gm.L)]
    f, b, ob = gm.ftp_profile_layers(10, to_dev(x), to_dev(y))           # ten runs averaged (Sec. III-B)
    assert np.all(f > 0) and np.all(b > 0)
    for u in range(gm.L):                                                # profiling trains nothing
        assert np.array_equal(state0[u], gm.ftp_get_tensor(F.T_STATE, u))
        assert np.array_equal(w0[u], gm.ftp_get_tensor(F.T_WEIGHTS, u))
        shp, nbytes = gm.ftp_unit_output_shape(u)
        assert ob[u] == nbytes == (4 if u == gm.L - 1 else int(np.prod(shp)) * 4)
    t = (f + b).tolist()
    for caps in ([1.0, 1.0, 1.0], [1.0, 2.0, 5.0, 10.0]):
        pts, bott = F.ftp_choose_partition(t, caps)
        assert (pts, bott) == oracle.choose_partition(t, caps)           # same times in -> same points, exactly
        # simulated devices: stage time = measured layer time x slowdown; Eq. 1-3 recovers the factors
        stage = [caps[i] * sum(t[a:bb]) for i, (a, bb) in enumerate(zip(pts, pts[1:]))]
        est = F.ftp_estimate_capacity(t, pts, stage)
        assert est == oracle.estimate_capacity(t, pts, stage)
        assert np.allclose(est[1:], caps[1:], rtol=1e-12)
    gm.close()


def test_repartition_moves_weights_and_training_continues_identically():
    ls, cfg = synth.mobilenetv2(4, 16, 10, 0, True)
    a, b = make_gpu(ls, cfg, 31), make_gpu(ls, cfg, 31)
    x, y = synth.make_batch(31, cfg)
    xd, yd = to_dev(x), to_dev(y)
    b.ftp_set_partition([0, 5, 12, 20])
    for m in (a, b):
        m.ftp_train_step(xd, yd, 0.01)
    cur, new = [0, 5, 12, 20], [0, 2, 15, 18, 20]
    moved = b.ftp_set_partition(new)
    # Algorithm 1: units whose owner changes = union of every stage's missing set
    expect = 0
    for i in range(len(new) - 1):
        need, _ = oracle.redistribution_plan(new, cur, i if i < len(cur) - 1 else None, i)
        expect += sum(len(v) for v in need.values())
    assert moved == expect and b.ftp_get_partition() == new
    for m in (a, b):
        m.ftp_train_step(xd, yd, 0.01)
    for u in range(a.L):
        for which in (F.T_WEIGHTS, F.T_MOMENTUM, F.T_STATE):
            assert np.array_equal(a.ftp_get_tensor(which, u), b.ftp_get_tensor(which, u))


def test_snapshots_are_bit_exact_and_laid_out_like_the_oracle():
    import torch
    ls, cfg = synth.tiny_mbv2()
    gm, om = make_gpu(ls, cfg, 32), make_oracle(ls, cfg, 32)
    pts = [0, 2, 5, gm.L]
    gm.ftp_set_partition(pts)
    x, y = synth.make_batch(32, cfg)
    gm.ftp_train_step(to_dev(x), to_dev(y), 0.01)
    om.step(pts, x, y)
    total = sum(gm.ftp_unit_param_span(u)[1] + gm.ftp_unit_state_span(u)[1] for u in range(gm.L))
    central = torch.zeros(total, dtype=torch.float32).pin_memory()          # global replication target
    off = 0
    for s in range(3):
        a, b = pts[s], pts[s + 1]
        n = sum(gm.ftp_unit_param_span(u)[1] + gm.ftp_unit_state_span(u)[1] for u in range(a, b))
        replica = torch.full((n + 8,), -7.0, device="cuda")                  # chain replication target
        assert gm.ftp_snapshot_weights(s, replica) == 4 * n
        assert gm.ftp_snapshot_weights(s, central[off:off + n]) == 4 * n
        torch.cuda.synchronize()
        live = np.concatenate([np.concatenate([gm.ftp_get_tensor(F.T_WEIGHTS, u), gm.ftp_get_tensor(F.T_STATE, u)])
                               for u in range(a, b)])
        got = replica.cpu().numpy()
        assert np.array_equal(got[:n], live) and np.all(got[n:] == -7.0)     # bytes equal, nothing past the end
        assert np.array_equal(central[off:off + n].numpy(), live)
        assert rel_err(got[:n], om.snapshot(a, b)) <= TOL_FP32               # same layout as the oracle's replica
        off += n
    with pytest.raises(F.FtpError):
        gm.ftp_snapshot_weights(0, torch.zeros(3, device="cuda"))            # too small: refused, nothing written
    with pytest.raises(F.FtpError):
        gm.ftp_snapshot_weights(3, central)


def test_fused_sgd_snapshot_equals_separate_copy():
    import torch
    ls, cfg = synth.tiny_mbv2()
    a, b = make_gpu(ls, cfg, 33), make_gpu(ls, cfg, 33)
    x, y = synth.make_batch(33, cfg)
    xd, yd = to_dev(x), to_dev(y)
    L = a.L
    n = sum(a.ftp_unit_param_span(u)[1] for u in range(L))
    snap_dev = torch.zeros(n, device="cuda")
    snap_host = torch.zeros(n).pin_memory()
    for m in (a, b):
        loss = torch.zeros(1, device="cuda")
        m.ftp_run_stage_forward(0, L, xd, None, yd, loss)
        m.ftp_run_stage_backward(0, L)
    a.ftp_sgd_step(0, L, 0.01)
    b.ftp_sgd_step(0, L, 0.01, snap_dev, snap_host)
    torch.cuda.synchronize()
    live = np.concatenate([a.ftp_get_tensor(F.T_WEIGHTS, u) for u in range(L)])
    assert np.array_equal(live, np.concatenate([b.ftp_get_tensor(F.T_WEIGHTS, u) for u in range(L)]))
    assert np.array_equal(snap_dev.cpu().numpy(), live) and np.array_equal(snap_host.numpy(), live)


def test_errors_are_returned_before_any_launch():
    import torch
    ls, cfg = synth.tiny_mbv2()
    gm = make_gpu(ls, cfg, 34)
    x, y = synth.make_batch(34, cfg)
    xd, yd = to_dev(x), to_dev(y)
    loss = torch.zeros(1, device="cuda")
    before = gm.ftp_launch_count()
    for call in (lambda: gm.ftp_run_stage_forward(3, 3, xd, None, yd, loss),            # empty range
                 lambda: gm.ftp_run_stage_forward(0, gm.L + 1, xd, None, yd, loss),
                 lambda: gm.ftp_run_stage_forward(0, gm.L, xd, None, None, loss),       # labels missing
                 lambda: gm.ftp_run_stage_forward(0, 2, xd, None),                      # act_out missing
                 lambda: gm.ftp_run_stage_backward(0, gm.L),                            # backward before forward
                 lambda: gm.ftp_set_partition([0, 3, 3, gm.L]),                         # empty stage
                 lambda: gm.ftp_set_partition(list(range(gm.L + 1)) ),                  # more stages than max_stages
                 lambda: gm.ftp_set_tensor(F.T_WEIGHTS, 0, np.zeros(3, np.float32)),    # wrong size
                 lambda: gm.ftp_get_tensor(F.T_WEIGHTS, gm.L)):
        with pytest.raises(F.FtpError):
            call()
    assert gm.ftp_launch_count() == before
    gm.ftp_run_stage_forward(0, gm.L, xd, None, yd, loss)                               # and the model still works
    gm.ftp_run_stage_backward(0, gm.L)
    torch.cuda.synchronize()
    assert np.isfinite(loss.item())


def test_trace_records_every_launch_with_its_algorithmic_work():
    ls, cfg = synth.tiny_mbv2()
    gm = make_gpu(ls, cfg, 35)
    x, y = synth.make_batch(35, cfg)
    gm.ftp_trace_enable(True)
    n0 = gm.ftp_launch_count()
    gm.ftp_train_step(to_dev(x), to_dev(y), 0.01)
    recs = gm.ftp_trace_read()
    gm.ftp_trace_enable(False)
    assert len(recs) > 50 and all(r["ms"] > 0 for r in recs if r["kernel"] != "copy")
    names = {r["kernel"] for r in recs}
    assert {"conv_fwd_f32", "conv_dgrad_f32", "conv_wgrad_f32", "bn_stats", "bn_apply", "bn_bwd_reduce", "bn_bwd_apply",
            "dw_fwd", "dw_dgrad", "gap_fwd", "softmax_ce", "sgd"} <= names       # dw_dgrad: one pass gives both depthwise gradients
    assert gm.ftp_launch_count() - n0 >= len(recs)


def _replicas(gm, sizes):
    """Chain and global replicas as the paper keeps them: stage i's weights with stage i+1 (device), the last
    stage's and everybody's with the central node (pinned host)."""
    import torch
    pts = gm.ftp_get_partition()
    n = len(pts) - 1
    total = sum(sizes)
    chain = {}
    central = torch.empty(total, dtype=torch.float32).pin_memory()
    off = 0
    for s in range(n):
        cnt = sum(sizes[pts[s]:pts[s + 1]])
        chain[s] = torch.empty(cnt, dtype=torch.float32, device="cuda") if s + 1 < n else torch.empty(cnt, dtype=torch.float32).pin_memory()
        gm.ftp_snapshot_weights(s, chain[s])
        gm.ftp_snapshot_weights(s, central[off:off + cnt])
        off += cnt
    torch.cuda.synchronize()
    return chain, central


@pytest.mark.parametrize("failed", [[2], [3], [1, 2], [1, 3]], ids=lambda f: "fail" + "_".join(map(str, f)))
def test_recovery_after_stage_failures(failed):
    """Sec. III-F on one GPU: train, replicate, train on (so the replicas are stale), then lose some stages.  After
    ftp_recover every unit of a surviving stage must hold its live weights bit for bit, every unit of a failed stage
    the bytes of the replica the plan names, and training must go on exactly as the oracle does from that state
    (momentum of the reloaded units restarted)."""
    import torch
    ls, cfg = synth.tiny_mbv2(momentum=0.9)
    cfg = dict(cfg, max_stages=4)
    params, state = perturb(ls, 81), synth.init_state(ls)
    om = oracle.OracleModel(ls, cfg, params, state)
    gm = F.Model(ls, cfg)
    gm.load_params(params, state)
    L = gm.L
    p_cur = [0, 2, 4, 5, L]
    gm.ftp_set_partition(p_cur)
    x, y, _ = clear_batch(om, 81, cfg)
    xd, yd = to_dev(x), to_dev(y)
    lr = cfg["lr"]
    sizes = [gm.ftp_unit_param_span(u)[1] + gm.ftp_unit_state_span(u)[1] for u in range(L)]
    for _ in range(2):
        gm.ftp_train_step(xd, yd, lr)
        om.step(p_cur, x, y)
    chain, central = _replicas(gm, sizes)
    snap_w = [om.unit_params(u).copy() for u in range(L)]
    snap_s = [om.unit_state(u).copy() for u in range(L)]
    gm.ftp_train_step(xd, yd, lr)                       # the replicas are one step old when the failure happens
    om.step(p_cur, x, y)
    live = [np.concatenate([gm.ftp_get_tensor(F.T_WEIGHTS, u), gm.ftp_get_tensor(F.T_STATE, u)]) for u in range(L)]
    n_new = len(p_cur) - 1 - len(failed)
    p_new = {3: [0, 3, 5, L], 2: [0, 4, L]}[n_new]
    plan = oracle.recovery_sources(p_cur, failed, p_new)
    # the chain replica of a failed stage is usable only if its keeper (the next stage) survived
    counts = gm.ftp_recover({f: chain[f] for f in failed}, p_new, central)
    torch.cuda.synchronize()
    assert gm.ftp_get_partition() == p_new
    want = [sum(1 for items in plan for _, s in items if s[0] == k) for k in ("stage", "replica", "central")]
    assert list(counts) == want
    offs = np.concatenate([[0], np.cumsum(sizes)])
    central_np = central.numpy()
    for items in plan:
        for u, src in items:
            got = np.concatenate([gm.ftp_get_tensor(F.T_WEIGHTS, u), gm.ftp_get_tensor(F.T_STATE, u)])
            if src[0] in ("local", "stage"):
                assert np.array_equal(got, live[u]), f"unit {u} ({src}) lost its live weights"
            else:
                assert np.array_equal(got, central_np[offs[u]:offs[u + 1]]), f"unit {u} ({src}) is not the replicated copy"
                om.set_unit(u, snap_w[u], snap_s[u], reset_momentum=True)
    # training continues identically on both sides
    for _ in range(2):
        loss = gm.ftp_train_step(xd, yd, lr)
        ref = om.step(p_new, x, y)
        assert abs(loss - ref) <= TOL_FP32 * max(abs(ref), 1.0)
    for u in range(L):
        assert rel_err(gm.ftp_get_tensor(F.T_WEIGHTS, u), om.unit_params(u)) <= TOL_FP32
    # a stage can rejoin: four stages again, on whichever arenas are idle
    gm.ftp_set_partition(p_cur)
    loss = gm.ftp_train_step(xd, yd, lr)
    ref = om.step(p_cur, x, y)
    assert abs(loss - ref) <= TOL_FP32 * max(abs(ref), 1.0)
    gm.close()


def test_recover_refuses_what_it_cannot_restore():
    import torch
    ls, cfg = synth.tiny_mbv2()
    cfg = dict(cfg, max_stages=4)
    gm = F.Model(ls, cfg)
    gm.load_params(synth.init_params(82, ls), synth.init_state(ls))
    L = gm.L
    gm.ftp_set_partition([0, 2, 4, L])
    before = gm.ftp_get_partition()
    with pytest.raises(F.FtpError):
        gm.ftp_recover({0: None}, [0, 3, L])                        # the central node does not fail
    with pytest.raises(F.FtpError):
        gm.ftp_recover({1: None}, [0, 3, L])                        # no replica of any kind
    with pytest.raises(F.FtpError):
        gm.ftp_recover({1: torch.empty(5, device="cuda")}, [0, 3, L])   # replica of the wrong size
    with pytest.raises(F.FtpError):
        gm.ftp_recover({1: None}, [0, 2, 4, L])                     # one failure leaves two stages
    assert gm.ftp_get_partition() == before
    gm.close()


def test_stage_times_feed_the_capacity_estimate():
    """Sec. III-B / Eq. 1-3 in a closed loop: the per-stage times that ftp_train_step reports, scaled by simulated
    slowdown factors, must give back those factors (relative to the central node) through ftp_estimate_capacity and
    the profiled layer times, to within the noise of timing short kernels."""
    import torch
    ls, cfg = synth.mobilenetv2(32, 32, 10, 0, True)
    gm = make_gpu(ls, dict(cfg, max_stages=4), 83)
    x, y = synth.make_batch(83, cfg)
    xd, yd = to_dev(x), to_dev(y)
    pts = [0, 5, 10, 15, gm.L]
    gm.ftp_set_partition(pts)
    with pytest.raises(F.FtpError):
        gm.ftp_stage_times()                                  # timing is off
    fwd, bwd, _ = gm.ftp_profile_layers(5, xd, yd)
    layer_times = (fwd + bwd).tolist()
    gm.ftp_stage_timing_enable(True)
    with pytest.raises(F.FtpError):
        gm.ftp_stage_times()                                  # no step timed yet
    for _ in range(3):
        gm.ftp_train_step(xd, yd, 0.01, want_loss=False)
    reports = []
    for _ in range(5):
        gm.ftp_train_step(xd, yd, 0.01, want_loss=False)
        reports.append(gm.ftp_stage_times())
    assert all(len(r) == 4 and min(r) > 0 for r in reports)
    mean = np.mean(reports, axis=0)
    factors = [2.0, 1.0, 8.0, 4.0]
    caps = F.ftp_estimate_capacity([t * factors[0] for t in layer_times], pts, [m_ * f for m_, f in zip(mean, factors)])
    assert caps[0] == 1.0
    for c, f in zip(caps[1:], factors[1:]):
        assert 0.5 * f / factors[0] <= c <= 2.0 * f / factors[0], (caps, factors)
    gm.ftp_stage_timing_enable(False)
    with pytest.raises(F.FtpError):
        gm.ftp_stage_times()
    gm.close()



def test_device_status_word_is_reported_and_cleared():
    """The status word that a tensor-core kernel sets when a bounded wait runs out, set here from the host
    (no kernel is altered, no wait is made to expire, and no tensor-core kernel runs while it is set): the
    synchronising routes return FTP_ETIMEOUT and clear it; an asynchronous call carries it to the host and
    every later call refuses before launching; after the check training matches the oracle again."""
    import torch
    ls, cfg = synth.tiny_mbv2()
    gm, om = make_gpu(ls, cfg, 36), make_oracle(ls, cfg, 36)
    x, y = synth.make_batch(36, cfg)
    xd, yd = to_dev(x), to_dev(y)
    gm.ftp_check_device_status()                                            # clean model: no error
    # synchronising routes read the word itself
    for call in (lambda: gm.ftp_check_device_status(), lambda: gm.ftp_get_tensor(F.T_WEIGHTS, 0)):
        gm.ftp_debug_set_device_status(12)
        with pytest.raises(F.FtpError) as e:
            call()
        assert e.value.status == 6 and "12" in str(e.value)
        gm.ftp_check_device_status()                                        # the failed call cleared it
    # asynchronous route: the optimiser step (streaming kernels only) queues a copy of the word behind its launches
    gm.ftp_debug_set_device_status(13)
    loss = torch.zeros(1, device="cuda")
    gm.ftp_sgd_step(0, 1, 0.0)
    torch.cuda.synchronize()
    before = gm.ftp_launch_count()
    for call in (lambda: gm.ftp_run_stage_forward(0, gm.L, xd, None, yd, loss), lambda: gm.ftp_run_stage_backward(0, gm.L),
                 lambda: gm.ftp_sgd_step(0, gm.L, 0.0), lambda: gm.ftp_train_step(xd, yd, 0.0, want_loss=False),
                 lambda: gm.ftp_train_step(xd, yd, 0.0), lambda: gm.ftp_profile_layers(1, xd, yd)):
        with pytest.raises(F.FtpError) as e:
            call()
        assert e.value.status == 6 and "13" in str(e.value)
    assert gm.ftp_launch_count() == before                                   # refused before any launch
    with pytest.raises(F.FtpError):
        gm.ftp_check_device_status()                                        # reports once more and clears
    gm.ftp_check_device_status()
    got = gm.ftp_train_step(xd, yd, cfg["lr"])
    ref = om.step([0, om.L], x, y)
    assert abs(got - ref) <= TOL_FP32 * abs(ref)
    gm.close()


def test_measured_link_bandwidth_feeds_the_partition_choice():
    """Sec. III-B / Eq. 4-5: the bandwidth between a worker and the next is measured (here: a device-to-device copy and
    the path to pinned host memory, timed with CUDA events), and the partition optimiser takes D_j / B with those
    numbers exactly as the oracle does."""
    import torch
    ls, cfg = synth.mobilenetv2(16, 32, 10, 0, True)
    gm = make_gpu(ls, cfg, 37)
    x, y = synth.make_batch(37, cfg)
    f, b, ob = gm.ftp_profile_layers(3, to_dev(x), to_dev(y))
    host = torch.empty(8 << 20, dtype=torch.uint8).pin_memory()
    d2d, d2h = gm.ftp_measure_bandwidth(host, 8 << 20, 3)
    assert 5e10 < d2d < 2e13 and 1e9 < d2h < 2e11, (d2d, d2h)          # device memory: tens of GB/s to TB/s; host link: GB/s
    assert gm.ftp_measure_bandwidth(None, 1 << 20, 2)[1] == 0.0
    with pytest.raises(F.FtpError):
        gm.ftp_measure_bandwidth(host, 16, 1)
    t = (f + b).tolist()
    caps = [1.0, 2.0, 5.0, 10.0]
    for bw in (d2d, d2h, 1e6):                                         # the last: a link slow enough that the term decides the cut
        got = F.ftp_choose_partition(t, caps, ob.tolist(), [bw] * 3)
        assert got == oracle.choose_partition(t, caps, [float(v) for v in ob], [bw] * 3)
    slow, _ = F.ftp_choose_partition(t, caps, ob.tolist(), [1e6] * 3)
    fast, _ = F.ftp_choose_partition(t, caps)
    assert slow != fast
    gm.close()


def test_guard_zones_stay_intact_on_ragged_shapes_and_catch_a_planted_overwrite():
    """Every buffer of the workspace ends in a guard zone.  After training steps on shapes with ragged tails (row counts
    off the 128-row tiles, channel counts off the vector widths, odd maps) in both precisions every zone still holds its
    pattern; a byte changed from the host inside one zone (no kernel misbehaves) is found and located."""
    import torch
    L, K, A = synth.Layer, synth.KIND, synth.ACT
    odd = [L(0, K["CONV2D"], 3, 6, 3, 1, 1, 0, 0, -1), L(0, K["BN"], 6, 6, 0, 1, 0, A["RELU6"], 0, -1),
           L(1, K["DWCONV3x3"], 6, 6, 3, 2, 1, 0, 0, -1), L(1, K["BN"], 6, 6, 0, 1, 0, A["RELU"], 0, -1),
           L(1, K["CONV2D"], 6, 10, 1, 1, 0, A["RELU"], 1, -1), L(2, K["MAXPOOL2"], 10, 10, 2, 2, 0, 0, 0, -1),
           L(2, K["GAP"], 10, 10, 0, 1, 0, 0, 0, -1), L(2, K["FC"], 10, 7, 1, 1, 0, 0, 1, -1), L(2, K["SOFTMAX_CE"], 7, 7, 0, 1, 0, 0, 0, -1)]
    nets = [synth.mobilenetv2(3, 10, 7, 0, True, table=[(1, 16, 1, 1), (6, 24, 2, 1), (6, 40, 1, 2)], stem_c=32, last_c=64),
            synth.mobilenetv2(3, 10, 7, 1, True, table=[(1, 16, 1, 1), (6, 24, 2, 1), (6, 40, 1, 2)], stem_c=32, last_c=64),
            synth.mobilenetv2(5, 9, 5, 0, False, table=[(1, 8, 1, 1), (6, 16, 1, 2)], stem_c=32, last_c=32),
            synth.tiny_vgg(batch=6, hw=4, precision=1), synth.har_cnn(5, 9, 131, 20, 6), (odd, synth.config(3, 3, 5, 5, 7, momentum=0.9))]
    for ls, cfg in nets:
        gm = make_gpu(ls, cfg, 38)
        x, y = synth.make_batch(38, cfg)
        xd = to_dev(x, torch.bfloat16 if cfg["precision"] == 1 else None)
        yd = to_dev(y)
        if gm.L >= 3:
            gm.ftp_set_partition([0, 1, gm.L])
        for _ in range(2):
            gm.ftp_train_step(xd, yd, 0.01)
        gm.ftp_profile_layers(1, xd, yd)
        assert gm.ftp_check_guards() > 20
        gm.close()
    ls, cfg = synth.tiny_mbv2()
    gm = make_gpu(ls, cfg, 38)
    n = gm.ftp_check_guards()
    base = (gm.dev_ws.data_ptr() + 255) // 256 * 256 - gm.dev_ws.data_ptr()
    # find a guard zone from the host: the first 256-byte run of the pattern after the first buffer
    ws = gm.dev_ws[base:base + (1 << 20)].cpu().numpy()
    runs = np.flatnonzero((ws.reshape(-1, 256) == 0xA5).all(axis=1))
    assert runs.size > 0
    off = int(runs[0]) * 256 + 17
    gm.dev_ws[base + off] = 0                                            # planted from the host
    with pytest.raises(F.FtpError) as e:
        gm.ftp_check_guards()
    assert e.value.status == 5 and e.value.bad_offset == off
    gm.dev_ws[base + off] = 0xA5
    assert gm.ftp_check_guards() == n
    gm.close()


def test_train_step_captured_into_a_graph_with_host_inputs_equals_eager_calls():
    """A step recorded into a CUDA graph with pinned host inputs and a pinned loss (the copies are nodes of the graph):
    three replays with the host buffers refilled in between give bit for bit the losses and weights of three eager calls."""
    import torch
    ls, cfg = synth.tiny_mbv2()
    batches = [synth.make_batch(70 + k, cfg) for k in range(3)]
    first = synth.make_batch(69, cfg)
    ref = make_gpu(ls, cfg, 70)
    gm = make_gpu(ls, cfg, 70)
    # one eager step on both before recording: whether a momentum buffer is initialised (a unit's first update) or
    # accumulated is decided when the step is recorded, so a graph is recorded after the first update
    for mdl in (ref, gm):
        mdl.ftp_train_step(torch.from_numpy(first[0]).pin_memory(), torch.from_numpy(first[1]).pin_memory(), 0.01, inputs_on_host=True)
    ref_losses = [ref.ftp_train_step(torch.from_numpy(x).pin_memory(), torch.from_numpy(y).pin_memory(), 0.01, inputs_on_host=True)
                  for x, y in batches]
    xh, yh = torch.from_numpy(batches[0][0].copy()).pin_memory(), torch.from_numpy(batches[0][1].copy()).pin_memory()
    loss_pin = torch.zeros(1, dtype=torch.float32).pin_memory()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    state = [gm.ftp_get_tensor(F.T_WEIGHTS, u) for u in range(gm.L)]        # capture runs nothing: the weights stay as loaded
    with torch.cuda.graph(g, stream=side):
        gm.ftp_train_step(xh, yh, 0.01, inputs_on_host=True, loss_pinned=loss_pin)
    for u in range(gm.L):
        assert np.array_equal(gm.ftp_get_tensor(F.T_WEIGHTS, u), state[u])
    losses = []
    for x, y in batches:
        xh.copy_(torch.from_numpy(x)); yh.copy_(torch.from_numpy(y))
        g.replay()
        torch.cuda.synchronize()
        losses.append(float(loss_pin[0]))
    assert losses == [float(np.float32(v)) for v in ref_losses]
    for u in range(gm.L):
        assert np.array_equal(gm.ftp_get_tensor(F.T_WEIGHTS, u), ref.ftp_get_tensor(F.T_WEIGHTS, u))
    with pytest.raises(ValueError):
        gm.ftp_train_step(xh, yh, 0.01, inputs_on_host=True, loss_pinned=torch.zeros(1))      # not pinned
    gm.close(); ref.close()


def _three_steps(net, idx, points, env):
    """Weights and losses after three training steps of a model built under the given environment switches."""
    import os
    import torch
    ls, cfg = net
    old = {k: os.environ.get(k) for k in env}
    os.environ.update(env)
    try:
        m = make_gpu(ls, cfg, idx)            # the switches are read when the model is built
    finally:
        for k, v in old.items():
            if v is None:
                os.environ.pop(k, None)
            else:
                os.environ[k] = v
    m.ftp_set_partition(points)
    bf16 = cfg["precision"] == 1
    losses = []
    for it in range(3):
        x, y = synth.make_batch(idx, cfg, it)
        xt = torch.from_numpy(x).to(torch.bfloat16) if bf16 else torch.from_numpy(x)
        losses.append(m.ftp_train_step(xt.cuda(), torch.from_numpy(y).cuda(), 0.01))
    w = [m.ftp_get_tensor(F.T_WEIGHTS, u) for u in range(m.L)]
    m.close()
    return losses, w


def test_one_join_before_the_update_changes_no_bit():
    """Networks without depthwise convolutions let the weight-gradient stream run on across the stages of a training
    step and join it once, before the update; with the join after every stage the same step gives the same bits
    (bf16 VGG groups at their real widths, three stages, 64-channel layers on the paired-tap weight gradient)."""
    net = synth.vgg16(32, 8, 10, 1, plan=[64, 64, "M", 128, 128, "M", 128, "M"])
    a = _three_steps(net, 63, [0, 2, 4, 6], {"FTP_DEFER_JOIN": "1"})
    b = _three_steps(net, 63, [0, 2, 4, 6], {"FTP_DEFER_JOIN": "0"})
    assert a[0] == b[0]
    assert all(np.array_equal(p, q) for p, q in zip(a[1], b[1]))


@pytest.mark.parametrize("precision", [0, 1])
def test_depthwise_partial_sums_on_the_second_stream_change_no_bit(precision):
    """The kernel that adds the per-block weight-gradient partials of the fused depthwise backward kernels runs on the
    second stream from buffers handed out in turn; on the main stream it gives the same bits (and so does the join taken
    once before the update, which these networks do not use by default)."""
    ls, cfg = synth.tiny_mbv2(precision=precision)
    pts = [0, 2, 4, synth.num_units(ls)]
    a = _three_steps((ls, cfg), 71, pts, {"FTP_DW_FIN_SIDE": "1"})
    b = _three_steps((ls, cfg), 71, pts, {"FTP_DW_FIN_SIDE": "0"})
    c = _three_steps((ls, cfg), 71, pts, {"FTP_DW_FIN_SIDE": "1", "FTP_DEFER_JOIN": "1"})
    assert a[0] == b[0] == c[0]
    assert all(np.array_equal(p, q) and np.array_equal(p, r) for p, q, r in zip(a[1], b[1], c[1]))
