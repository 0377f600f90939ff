"""GPU test of the asynchronous pipeline of Sec. III-C (1F1B, weight stashing, vertical sync, weight aggregation):
the library's calls, strung together by the package's driver, against the oracle's float64 simulation of the same
schedule on the same seeded batches; and the host-side schedule functions against the oracle's."""
import numpy as np
import pytest

import synth
from helpers import TOL_FP32, rel_err, safe_params, to_dev
from oracle import schedule as S

pytestmark = pytest.mark.gpu
F = pytest.importorskip("paper_2110_02781_b200")


def test_schedule_functions_match_the_oracle():
    for n in range(1, 6):
        for s in range(n):
            for nb in (0, 1, 2, 5, 11):
                assert F.ftp_async_stage_order(n, s, nb) == S.stage_order(n, s, nb)
                for k in (1, 2):
                    assert F.ftp_async_version_trace(n, s, nb, k) == tuple(S.version_trace(n, s, nb, k))
    fwd, after, agg = F.ftp_async_version_trace(3, 0, 8)
    assert fwd[:7] == [0, 0, 0, 1, 2, 3, 5] and agg[0] == 5          # the paper's example: 3_f^1 4_f^2 5_f^3, then batch 6 with version 5


def test_aggregate_is_the_mean_and_sync_copies_exactly():
    ls, cfg = synth.tiny_mbv2()
    ms = []
    for k in range(3):
        m = F.Model(ls, cfg)
        m.load_params(safe_params(ls, 80 + k), synth.init_state(ls))
        ms.append(m)
    dst = F.Model(ls, cfg)
    dst.load_params(synth.init_params(80, ls), synth.init_state(ls))
    before = [dst.ftp_get_tensor(F.T_WEIGHTS, u) for u in range(dst.L)]
    F.ftp_aggregate_weights(dst, ms, 1, 4)
    for u in range(dst.L):
        got = dst.ftp_get_tensor(F.T_WEIGHTS, u)
        if 1 <= u < 4:
            want = np.mean([m.ftp_get_tensor(F.T_WEIGHTS, u).astype(np.float64) for m in ms], axis=0)
            assert rel_err(got, want) <= 1e-6
        else:
            assert np.array_equal(got, before[u])
    F.ftp_sync_units(dst, ms[1], 0, dst.L, F.SYNC_WEIGHTS | F.SYNC_STATE)
    for u in range(dst.L):
        assert np.array_equal(dst.ftp_get_tensor(F.T_WEIGHTS, u), ms[1].ftp_get_tensor(F.T_WEIGHTS, u))
    with pytest.raises(F.FtpError):
        F.ftp_aggregate_weights(dst, ms * 3, 0, 1)                     # nine versions: more than the call takes
    for m in ms + [dst]:
        m.close()


@pytest.mark.parametrize("points,nb,k", [([0, 2, 5, 7], 8, 1), ([0, 3, 7], 7, 1), ([0, 7], 3, 1), ([0, 1, 3, 5, 7], 9, 1)])
def test_async_pipeline_matches_the_oracle_simulation(points, nb, k):
    from paper_2110_02781_b200.async_pipeline import AsyncPipeline
    ls, cfg = synth.tiny_mbv2()
    params, state = safe_params(ls, 81), synth.init_state(ls)      # BN outputs inside the linear range of ReLU6: no ambiguous decisions
    op = S.AsyncPipeline(ls, cfg, params, state, points, k)
    batches = [synth.make_batch(81, cfg, t) for t in range(nb)]
    ref = op.run(batches, cfg["lr"])
    gp = AsyncPipeline(ls, cfg, points, params, state, k)
    got = gp.run([(to_dev(x), to_dev(y)) for x, y in batches], cfg["lr"])
    assert gp.log == op.log                                          # same passes with the same version ids, same aggregations
    for b in range(nb):
        assert abs(got[b] - ref[b]) <= 5 * TOL_FP32 * abs(ref[b]), b
    for u in range(gp.L):                                            # several updates of drift, not one
        assert rel_err(gp.master.ftp_get_tensor(F.T_WEIGHTS, u), op.master.unit_params(u)) <= 1e-3, u
        assert rel_err(gp.master.ftp_get_tensor(F.T_STATE, u), op.master.unit_state(u)) <= 1e-3, u
    gp.close()
