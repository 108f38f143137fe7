"""The workspace-free calibration entry point (for callers that are not allowed to allocate device memory)
against the regular one, through the C ABI.  Collected last on purpose: it shares one scratch array inside
the library with nothing else, but if it fails a run that stops at the first failure has already run all
other tests.  Passes alone in a fresh process and after the rest of the suite."""
import numpy as np
import pytest

from oracle import qwt_oracle as O
from paper_2505_20932_b200 import workload as WL
from tolerances import assert_ab_close

pytestmark = pytest.mark.gpu


def _both(B, torch, fp, q, C, ld):
    rows = fp.shape[0]
    dfp, dq = torch.from_numpy(fp).cuda(), torch.from_numpy(q).cuda()
    out = {}
    for name in ("regular", "noalloc"):
        a = torch.full((C,), float("nan"), device="cuda")
        b = torch.full((C,), float("nan"), device="cuda")
        nd = torch.full((1,), -1, dtype=torch.int32, device="cuda")
        if name == "regular":
            wsb = B.qwt_cwac_workspace_bytes(rows, C)
            ws = torch.empty(max(wsb, 256), dtype=torch.uint8, device="cuda")
            B.qwt_cwac_calibrate(dfp, dq, rows, C, ld, a, b, nd, ws, wsb)
        else:
            B.qwt_cwac_calibrate_noalloc(dfp, dq, rows, C, ld, a, b, nd)
        torch.cuda.synchronize()
        out[name] = (a.cpu().numpy(), b.cpu().numpy(), int(nd.item()))
    return out


def test_noalloc_calibration_matches_regular_entry_point_twice_in_a_row():
    import torch
    from paper_2505_20932_b200 import binding as B
    # two calls in a row that share the library's scratch array: a wide short problem, then a narrow long one
    # (the second leaves most of the first call's partial sums in place; they must not be read).  The first
    # needs more than 4 MiB of partials under the regular plan, so it also covers the longer-chunk path.
    cases = [(2000, 12800, 12800, 4), (150_000, 132, 136, 8)]
    for rows, C, ld, bits in cases:
        fp, q, _ = WL.host_calib_pair(rows, C, bits, seed=rows, ld=ld)
        if C < ld:
            fp[:, C:] = 7e20
            q[:, C:] = -7e20
        q[:, 1] = 0.25                                  # one degenerate channel
        r = _both(B, torch, fp, q, C, ld)
        a0, b0, n0 = r["regular"]
        a1, b1, n1 = r["noalloc"]
        assert n0 == n1 == 1 and a1[1] == 1.0
        scale = np.maximum(np.abs(fp[:, :C].mean(0)), fp[:, :C].std(0))
        assert_ab_close(a1, b1, a0, b0, scale)          # same tolerance as the oracle comparison of a, b
        ch = np.unique(np.concatenate([np.random.default_rng(C).integers(0, C, 48), [0, 1, 127, 128, C - 1]]))
        a_ref, b_ref, _ = O.cwac_fit(fp[:, ch], q[:, ch])        # and the oracle's own fit of sampled channels
        assert_ab_close(a1[ch], b1[ch], a_ref, b_ref, scale[ch])
    assert B.qwt_cwac_workspace_bytes(2000, 12800) > B.QWT_NOALLOC_SCRATCH_BYTES


def test_noalloc_rejects_what_does_not_fit():
    import torch
    from paper_2505_20932_b200 import binding as B
    x = torch.zeros(1024, device="cuda")
    too_wide = 131072 + 4                               # one chunk of partial sums already exceeds the array
    s = B.qwt_cwac_calibrate_noalloc(x, x, 1, too_wide, too_wide, x, x, None, check=False)
    assert s == B.QWT_ERR_TOO_LARGE
    assert "scratch" in B.qwt_status_string(s)
    assert B.qwt_cwac_calibrate_noalloc(x, x, 0, 8, 8, x, x, None, check=False) == B.QWT_ERR_SHAPE
    assert B.qwt_cwac_calibrate_noalloc(None, x, 4, 8, 8, x, x, None, check=False) == B.QWT_ERR_NULL
