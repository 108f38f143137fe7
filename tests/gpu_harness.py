"""Helpers for the GPU parity tests: move numpy inputs to the device, call the C ABI through the
binding, bring results back.  No arithmetic of the method happens here."""
import numpy as np
import torch

from paper_2505_20932_b200 import binding as B

DEV = "cuda"


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def empty_bytes(n):
    return torch.empty(max(int(n), 256), dtype=torch.uint8, device=DEV)


def gpu_quantize_rows(X, qmax=127, ld=None):
    X = np.ascontiguousarray(X, dtype=np.float32)
    rows, cols = X.shape
    dX = dev(X)
    Xq = torch.empty((rows, cols), dtype=torch.int8, device=DEV)
    sc = torch.empty(rows, dtype=torch.float32, device=DEV)
    B.qwt_quantize_rows_i8(dX, rows, cols, cols if ld is None else ld, qmax, Xq, sc)
    torch.cuda.synchronize()
    return Xq.cpu().numpy(), sc.cpu().numpy()


def gpu_pack_int4(codes):
    rows, cols = codes.shape
    d = dev(codes.astype(np.int8))
    out = torch.empty((rows, cols // 2), dtype=torch.uint8, device=DEV)
    B.qwt_pack_int4(d, rows, cols, out)
    torch.cuda.synchronize()
    return out.cpu().numpy()


def gpu_calibrate(fp, q, channels=None):
    """fp, q: float32 [rows, ld] arrays; channels <= ld."""
    rows, ld = fp.shape
    C = ld if channels is None else channels
    dfp, dq = dev(fp), dev(q)
    a = torch.empty(C, dtype=torch.float32, device=DEV)
    b = torch.empty(C, dtype=torch.float32, device=DEV)
    nd = torch.full((1,), -1, dtype=torch.int32, device=DEV)
    wsb = B.qwt_cwac_workspace_bytes(rows, C)
    ws = empty_bytes(wsb)
    B.qwt_cwac_calibrate(dfp, dq, rows, C, ld, a, b, nd, ws, wsb)
    torch.cuda.synchronize()
    return a.cpu().numpy(), b.cpu().numpy(), int(nd.item())


def gpu_calibrate_streamed(fp, q, batches):
    rows, C = fp.shape
    stats = torch.zeros(5 * C, dtype=torch.float64, device=DEV)
    dfp, dq = dev(fp), dev(q)
    edges = np.linspace(0, rows, batches + 1).astype(int)
    for r0, r1 in zip(edges[:-1], edges[1:]):
        if r1 == r0:
            continue
        wsb = B.qwt_cwac_workspace_bytes(int(r1 - r0), C)
        ws = empty_bytes(wsb)
        B.qwt_cwac_stats_accumulate(dfp[r0:r1], dq[r0:r1], int(r1 - r0), C, C, stats, ws, wsb)
    a = torch.empty(C, dtype=torch.float32, device=DEV)
    b = torch.empty(C, dtype=torch.float32, device=DEV)
    nd = torch.zeros(1, dtype=torch.int32, device=DEV)
    B.qwt_cwac_solve(stats, C, a, b, nd)
    torch.cuda.synchronize()
    return a.cpu().numpy(), b.cpu().numpy(), int(nd.item()), stats.cpu().numpy().reshape(5, C)


def gpu_fold(ws_, bias, a, b):
    n = ws_.shape[0]
    fs = torch.empty(n, dtype=torch.float32, device=DEV)
    fb = torch.empty(n, dtype=torch.float32, device=DEV)
    B.qwt_cwac_fold(dev(ws_), None if bias is None else dev(bias), None if a is None else dev(a),
                    None if b is None else dev(b), n, fs, fb)
    torch.cuda.synchronize()
    return fs.cpu().numpy(), fb.cpu().numpy()


_OUT_DTYPE = {B.QWT_OUT_INT8_PER_TOKEN: torch.int8, B.QWT_OUT_BF16: torch.bfloat16,
              B.QWT_OUT_FP32: torch.float32, B.QWT_OUT_INT32_ACC: torch.int32, B.QWT_OUT_INT8_STATIC: torch.int8}


def gpu_fold_static(ws_, bias, a, b, S_x, S_r):
    n = ws_.shape[0]
    mult = torch.empty(n, dtype=torch.float32, device=DEV)
    off = torch.empty(n, dtype=torch.int32, device=DEV)
    B.qwt_cwac_fold_static(dev(ws_), None if bias is None else dev(bias), None if a is None else dev(a),
                           None if b is None else dev(b), n, float(S_x), float(S_r), mult, off)
    torch.cuda.synchronize()
    return mult.cpu().numpy(), off.cpu().numpy()


def gpu_forward(Xq, xs, W, fs, fb, out_mode, wfmt=B.QWT_W_INT8, K=None, check_guard=True):
    """Returns (Y numpy, y_scale numpy or None).  BF16 output is returned as uint16 bit patterns.
    Output buffers carry guard bands that must stay untouched."""
    M = Xq.shape[0]
    K = Xq.shape[1] if K is None else K
    N = W.shape[0]
    dX, dW = dev(Xq), dev(W)
    dxs = None if xs is None else dev(xs.astype(np.float32))
    dfs = None if fs is None else dev(fs.astype(np.float32))
    # static INT8 mode: the "fbias" pointer carries the INT32 accumulator offsets
    dfb = None if fb is None else dev(fb.astype(np.int32) if out_mode == B.QWT_OUT_INT8_STATIC else fb.astype(np.float32))
    dt = _OUT_DTYPE[out_mode]
    guard = 64
    Ybuf = torch.zeros(M * N + 2 * guard, dtype=dt, device=DEV)
    Ybuf_i = Ybuf.view(torch.int8 if dt == torch.int8 else (torch.int16 if dt == torch.bfloat16 else torch.int32))
    Ybuf_i.fill_(0x5A)
    Y = Ybuf[guard:guard + M * N]
    ysbuf = torch.full((M + 2 * guard,), -7.0, dtype=torch.float32, device=DEV)
    ys = ysbuf[guard:guard + M] if out_mode == B.QWT_OUT_INT8_PER_TOKEN else None
    wsb = B.qwt_qlinear_workspace_bytes(M, N, K, wfmt, out_mode)
    ws = empty_bytes(wsb)
    ws.fill_(0xFF)                      # the call must initialise its own scratch
    B.qwt_qlinear_cwac_forward(dX, dxs, dW, wfmt, dfs, dfb, M, N, K, out_mode, Y, ys, ws, wsb)
    B.qwt_qlinear_check_status(ws)
    if check_guard:
        gi = Ybuf_i.cpu().numpy()
        assert (gi[:guard] == 0x5A).all() and (gi[guard + M * N:] == 0x5A).all(), "output guard band overwritten"
        if ys is not None:
            g = ysbuf.cpu().numpy()
            assert (g[:guard] == -7.0).all() and (g[guard + M:] == -7.0).all(), "y_scale guard band overwritten"
    if dt == torch.bfloat16:
        Yh = Y.view(torch.int16).cpu().numpy().view(np.uint16).reshape(M, N)
    else:
        Yh = Y.cpu().numpy().reshape(M, N)
    return Yh, (None if ys is None else ys.cpu().numpy())


def gpu_calibrate_fused(Xq, xs, W, w_scale, bias, fp, wfmt=B.QWT_W_INT8, K=None, stats=None, solve=True):
    """Calibration inside the layer's epilogue: returns (a, b, n_degenerate, stats [5, N] or None).
    fp: float32 [M, ld] with ld >= N.  stats: running statistics (numpy [5, N]) to continue from, or None."""
    M = Xq.shape[0]
    K = Xq.shape[1] if K is None else K
    N = W.shape[0]
    ld = fp.shape[1]
    dX, dW, dxs, dws, dfp = dev(Xq), dev(W), dev(xs.astype(np.float32)), dev(w_scale.astype(np.float32)), dev(fp)
    dbias = None if bias is None else dev(bias.astype(np.float32))
    dstats = None if stats is None else dev(np.ascontiguousarray(stats, dtype=np.float64).reshape(-1))
    a = torch.full((N,), 7.0, dtype=torch.float32, device=DEV) if solve else None
    b = torch.full((N,), 7.0, dtype=torch.float32, device=DEV) if solve else None
    nd = torch.full((1,), -1, dtype=torch.int32, device=DEV) if solve else None
    wsb = B.qwt_qlinear_cwac_calibrate_workspace_bytes(M, N, K, wfmt)
    ws = empty_bytes(wsb)
    ws.fill_(0xFF)
    B.qwt_qlinear_cwac_calibrate(dX, dxs, dW, wfmt, dws, dbias, dfp, ld, M, N, K, dstats, a, b, nd, ws, wsb)
    B.qwt_qlinear_check_status(ws)
    return (None if a is None else a.cpu().numpy(), None if b is None else b.cpu().numpy(),
            None if nd is None else int(nd.item()), None if dstats is None else dstats.cpu().numpy().reshape(5, N))
