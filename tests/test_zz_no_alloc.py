"""The allocation-free weight-gradient entry point against the model API (collected last on purpose).

Some users of the library sit where device memory cannot be requested: inside a stream-ordered
section that an allocation would stall, or under a host that hands out buffers and keeps the
allocator to itself.  ftp_conv_wgrad_static serves them with scratch built into the library.
Here its result is compared with the weight gradient that ftp_run_stage_backward leaves in the
gradient arena for the same convolution and with the oracle's, on two calls in a row (the second
after a call of a different shape has dirtied the shared scratch)."""
import numpy as np
import pytest

import oracle.ops
import synth
from helpers import TOL_FP32, rel_err, to_dev

pytestmark = pytest.mark.gpu
F = pytest.importorskip("paper_2110_02781_b200")


def _model_wgrad(cin, cout, k, stride, pad, x, gout):
    """dW of a lone convolution through the existing entry points."""
    import torch
    L, K = synth.Layer, synth.KIND
    n, h = x.shape[0], x.shape[1]
    ls = [L(0, K["CONV2D"], cin, cout, k, stride, pad, 0, 0, -1), L(1, K["GAP"], cout, cout, 0, 1, 0, 0, 0, -1),
          L(1, K["FC"], cout, 3, 1, 1, 0, 0, 1, -1), L(1, K["SOFTMAX_CE"], 3, 3, 0, 1, 0, 0, 0, -1)]
    cfg = synth.config(n, cin, h, h, 3)
    m = F.Model(ls, cfg)
    m.load_params(synth.init_params(50, ls), synth.init_state(ls))
    y = torch.empty(gout.shape, device="cuda")
    dx = torch.empty(x.shape, device="cuda")
    m.ftp_run_stage_forward(0, 1, x, y)
    m.ftp_run_stage_backward(0, 1, gout, dx)
    torch.cuda.synchronize()
    out = m.ftp_get_tensor(F.T_GRADS, 0)
    m.close()
    return out


@pytest.mark.parametrize("n,h,cin,cout,k,stride,pad", [(16, 32, 24, 144, 1, 1, 0), (8, 16, 32, 64, 3, 1, 1)])
def test_static_scratch_wgrad_matches_model_api_twice(n, h, cin, cout, k, stride, pad):
    import torch
    g = synth.rng_stream(50, "misc")
    ho = (h + 2 * pad - k) // stride + 1
    x = to_dev(g.standard_normal((n, h, h, cin)).astype(np.float32))
    gout = to_dev(g.standard_normal((n, ho, ho, cout)).astype(np.float32))
    ref = _model_wgrad(cin, cout, k, stride, pad, x, gout)
    dw = torch.full((k, k, cin, cout), float("nan"), device="cuda")
    F.ftp_conv_wgrad_static(x, gout, dw, k, stride, pad)
    torch.cuda.synchronize()
    first = dw.cpu().numpy().reshape(-1)
    assert rel_err(first, ref) <= TOL_FP32
    _, want_dw, _ = oracle.ops.conv_bwd(x.cpu().numpy().astype(np.float64), np.zeros((k, k, cin, cout)), gout.cpu().numpy().astype(np.float64),
                                        stride, pad, pad, False)
    assert rel_err(first, want_dw.reshape(-1)) <= TOL_FP32
    # a call of another shape leaves its partial sums in the shared scratch
    x2, g2 = torch.randn(4, 8, 8, 16, device="cuda"), torch.randn(4, 8, 8, 8, device="cuda")
    dw2 = torch.empty(1, 1, 16, 8, device="cuda")
    F.ftp_conv_wgrad_static(x2, g2, dw2, 1, 1, 0)
    dw.fill_(float("nan"))
    F.ftp_conv_wgrad_static(x, gout, dw, k, stride, pad)
    torch.cuda.synchronize()
    second = dw.cpu().numpy().reshape(-1)
    assert rel_err(second, ref) <= TOL_FP32 and np.array_equal(first, second)
    want = (x2.reshape(-1, 16).double().T @ g2.reshape(-1, 8).double()).cpu().numpy().reshape(-1)
    assert rel_err(dw2.cpu().numpy().reshape(-1), want) <= TOL_FP32


def test_static_scratch_refuses_shapes_beyond_its_size():
    import torch
    x = torch.zeros(1, 8, 8, 1024, device="cuda")
    dy = torch.zeros(1, 8, 8, 4096, device="cuda")
    dw = torch.zeros(1, 1, 1024, 4096, device="cuda")
    # one tile column per 64 outputs -> no split, no scratch: accepted
    F.ftp_conv_wgrad_static(x, dy, dw, 1, 1, 0)
    xs = torch.zeros(64, 32, 32, 256, device="cuda")
    dys = torch.zeros(64, 32, 32, 256, device="cuda")
    dws = torch.zeros(3, 3, 256, 256, device="cuda")
    with pytest.raises(F.FtpError) as e:
        F.ftp_conv_wgrad_static(xs, dys, dws, 3, 1, 1)        # 9*256*256 floats x several splits > 8 MiB
    assert "scratch" in str(e.value)


def test_static_scratch_wrapper_refuses_wrong_shapes_and_types():
    import torch
    x = torch.zeros(2, 8, 8, 16, device="cuda")
    dy = torch.zeros(2, 8, 8, 8, device="cuda")
    dw = torch.zeros(1, 1, 16, 8, device="cuda")
    F.ftp_conv_wgrad_static(x, dy, dw, 1, 1, 0)
    for bad in ((x, dy[:, :4], dw), (x, dy, dw[:, :, :8]), (x.double(), dy, dw), (x, dy.cpu(), dw), (x, dy.permute(0, 2, 1, 3)[:, ::2], dw)):
        with pytest.raises(F.FtpError):
            F.ftp_conv_wgrad_static(*bad, 1, 1, 0)
    with pytest.raises(F.FtpError):
        F.ftp_conv_wgrad_static(x, dy, dw, 3, 1, 0)           # dy would have to be 6 x 6
