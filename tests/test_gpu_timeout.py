"""The give-up path of the bounded device-side waits, without faulting or hanging anything: the per-token INT8
exchange is told (host-side test hook) to expect one more unit per row strip than the layer has, with the wait limit
set to one millisecond.  Nothing ever publishes that unit's row maxima, so every CTA's wait runs out; the kernel must
then record a status code, tear down normally and return, qwt_qlinear_check_status must report QWT_ERR_TIMEOUT, and
the next ordinary call on the same workspace must be clean and correct."""
import numpy as np
import pytest
import torch

from oracle import qwt_oracle as O
from tolerances import assert_codes_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


def test_exchange_wait_runs_out_and_the_next_call_is_clean():
    from paper_2505_20932_b200 import binding as B
    M, N, K = 256, 512, 128                      # two row strips x two 256-wide tiles: four CTAs
    g = torch.Generator(device=DEV)
    g.manual_seed(1)
    Xq = torch.randint(-127, 128, (M, K), generator=g, device=DEV, dtype=torch.int8)
    Wq = torch.randint(-127, 128, (N, K), generator=g, device=DEV, dtype=torch.int8)
    xs = torch.rand(M, generator=g, device=DEV) * 0.04 + 0.01
    fs = torch.rand(N, generator=g, device=DEV) * 2e-4 + 1e-4
    fb = torch.randn(N, generator=g, device=DEV) * 0.01
    Y = torch.zeros((M, N), dtype=torch.int8, device=DEV)
    ys = torch.zeros(M, dtype=torch.float32, device=DEV)
    mode, wf = B.QWT_OUT_INT8_PER_TOKEN, B.QWT_W_INT8
    try:
        B.qwt_test_set_phantom_units(1)
        B.qwt_test_set_wait_limit_ns(1_000_000)
        wsb = B.qwt_qlinear_workspace_bytes(M, N, K, wf, mode)      # sized for the extra unit
        ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device=DEV)
        t0 = torch.cuda.Event(enable_timing=True)
        t1 = torch.cuda.Event(enable_timing=True)
        t0.record()
        assert B.qwt_qlinear_cwac_forward(Xq, xs, Wq, wf, fs, fb, M, N, K, mode, Y, ys, ws, wsb, check=False) == B.QWT_OK
        t1.record()
        s = B.qwt_qlinear_check_status(ws, check=False)            # waits for the stream
    finally:
        B.qwt_test_set_phantom_units(0)
        B.qwt_test_set_wait_limit_ns(0)
    assert s == B.QWT_ERR_TIMEOUT
    assert "timed out" in B.qwt_status_string(s)
    assert 0.5 < t0.elapsed_time(t1) < 500.0                        # the kernel returned after about the limit (ms)
    assert wsb >= B.qwt_qlinear_workspace_bytes(M, N, K, wf, mode)  # the ordinary plan fits the same workspace
    # the device and the workspace are usable: an ordinary call is clean and matches the oracle
    B.qwt_qlinear_cwac_forward(Xq, xs, Wq, wf, fs, fb, M, N, K, mode, Y, ys, ws, wsb)
    assert B.qwt_qlinear_check_status(ws, check=False) == B.QWT_OK
    z = O.forward_folded(O.int_matmul(Xq.cpu().numpy(), Wq.cpu().numpy()), xs.cpu().numpy(), fs.cpu().numpy(),
                         fb.cpu().numpy())
    c_ref, ys_ref = O.requant_per_token(z)
    assert np.allclose(ys.cpu().numpy(), ys_ref, rtol=1e-5)
    assert_codes_close(Y.cpu().numpy(), c_ref)
