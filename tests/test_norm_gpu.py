"""Residual connection + RMS normalisation (paper Section 3.6, second fusion example) against the CPU oracle."""
import numpy as np
import pytest

from oracle import qlinear_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def P(_built_library):
    import paper_2505_00232_b200 as P
    return P


@pytest.fixture(scope="module")
def torch():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch


def inputs(seed, M, K, spread=4.0):
    rng = np.random.default_rng(seed)
    x = (rng.standard_normal((M, K)) * rng.uniform(0.1, spread, size=(M, 1))).astype(np.float16)
    r = (rng.standard_normal((M, K)) * rng.uniform(0.1, 4 * spread, size=(M, 1))).astype(np.float16)
    g = (rng.standard_normal(K) / 4).astype(np.float16)
    return x, r, g


def check(h_gpu, y_gpu, x, r, g, eps, off):
    K = x.shape[1]
    h64, h16, y64, _ = O.residual_rmsnorm(x, r, g, eps, off)
    bh, by = O.residual_rmsnorm_bound(h64, y64, K)
    if h_gpu is not None:
        assert (h_gpu.view(np.uint16) == h16.view(np.uint16)).all()      # the sum of two fp16 values, rounded once: unique
        assert (np.abs(h_gpu.astype(np.float64) - h64) <= bh).all()
    d = np.abs(y_gpu.astype(np.float64) - y64)
    assert (d <= by).all(), f"worst |dy| / bound = {(d / by).max():.3e}"


# every vector tail (K = 8 .. one vector per thread and beyond), the paper's models' widths, ragged row counts
@pytest.mark.parametrize("M,K", [(1, 8), (3, 40), (5, 2048), (1, 2304), (4, 4096), (7, 14336), (300, 2304), (2048, 4096), (33, 9216)])
@pytest.mark.parametrize("off", [0.0, 1.0])
def test_parity(P, torch, M, K, off):
    x, r, g = inputs(100 + M + K, M, K)
    eps = 1e-6 if off == 1.0 else 1e-5
    h, y = P.qlinear_residual_rmsnorm(torch.from_numpy(x).cuda(), torch.from_numpy(r).cuda(), torch.from_numpy(g).cuda(), eps, off)
    torch.cuda.synchronize()
    check(h.cpu().numpy(), y.cpu().numpy(), x, r, g, eps, off)


def test_no_residual_no_h_and_in_place(P, torch):
    M, K = 64, 4096
    x, r, g = inputs(9, M, K)
    xd, rd, gd = (torch.from_numpy(a).cuda() for a in (x, r, g))
    h, y = P.qlinear_residual_rmsnorm(xd, None, gd, 1e-5, 0.0, want_h=False)
    assert h is None
    check(None, y.cpu().numpy(), x, None, g, 1e-5, 0.0)
    # in place: the residual stream is updated where it lives, the normalised values overwrite x
    h2, y2 = P.qlinear_residual_rmsnorm(xd, rd, gd, 1e-5, 1.0, h_out=rd, y_out=xd)
    torch.cuda.synchronize()
    assert h2.data_ptr() == rd.data_ptr() and y2.data_ptr() == xd.data_ptr()
    check(rd.cpu().numpy(), xd.cpu().numpy(), x, r, g, 1e-5, 1.0)


def test_extremes_and_guard_band(P, torch):
    M, K = 9, 1024
    x = np.zeros((M, K), np.float16)
    r = np.zeros((M, K), np.float16)
    x[1, :] = 65504.0                                                    # largest fp16: the squares need fp32
    x[2, 0] = 6e-8                                                       # one subnormal, everything else zero
    x[3, :], r[3, :] = 40000.0, 40000.0                                  # the sum leaves the fp16 range: h is +inf in fp16, y is finite
    x[4, ::2], r[4, 1::2] = -7.0, 5.0
    g = np.ones(K, np.float16)
    pad = 512
    buf = torch.full((pad + M * K + pad,), -3.0, dtype=torch.float16, device="cuda")
    hbuf = torch.full((pad + M * K + pad,), -3.0, dtype=torch.float16, device="cuda")
    y = buf[pad:pad + M * K].view(M, K)
    h = hbuf[pad:pad + M * K].view(M, K)
    P.qlinear_residual_rmsnorm(torch.from_numpy(x).cuda(), torch.from_numpy(r).cuda(), torch.from_numpy(g).cuda(), 1e-6, 0.0, h_out=h, y_out=y)
    torch.cuda.synchronize()
    for b in (buf, hbuf):
        c = b.cpu().numpy()
        assert (c[:pad] == -3.0).all() and (c[pad + M * K:] == -3.0).all()
    yh, hh = y.cpu().numpy(), h.cpu().numpy()
    assert (yh[0] == 0).all() and np.isfinite(yh).all()
    assert np.isinf(hh[3]).all() and np.allclose(yh[3].astype(np.float64), 1.0, rtol=2e-3)
    check(None, yh, x, r, g, 1e-6, 0.0)


def test_bad_arguments(P, torch):
    x = torch.zeros((4, 64), dtype=torch.float16, device="cuda")
    g = torch.ones((64,), dtype=torch.float16, device="cuda")
    with pytest.raises(P.QLinearError):
        P.qlinear_residual_rmsnorm(x[:, :60], None, g[:60], 1e-5)       # K not a multiple of 8 / not contiguous
    with pytest.raises(P.QLinearError):
        P.qlinear_residual_rmsnorm(x, None, g, 1e-5, h_out=x, y_out=x)   # the two outputs must differ
    with pytest.raises(P.QLinearError):
        P.qlinear_residual_rmsnorm(x, None, g, -1.0)


def test_chain_with_linear_layers_needs_no_synchronisation(P, torch):
    """norm -> linear -> norm -> linear on one stream, decode and prefill sizes, buffers reused: every kernel releases its
    successor early (programmatic dependent launch), so the unsynchronised chain must give the bits of the synchronised one."""
    from workloads import configs as C
    K = 2048
    spec = C.LayerSpec("t", K, K, 4, 32, -8, 7)
    lins = []
    for i in range(2):
        q, s = C.layer_weights(70 + i, spec)
        lins.append(P.QLinear.from_weights(q, (s.astype(np.float32) / 8).astype(np.float16), 4, 32, device="cuda:0"))
    g = torch.from_numpy(inputs(1, 1, K)[2]).cuda()
    for M in (1, 4, 300):
        x0 = torch.from_numpy(inputs(2 + M, M, K)[0]).cuda()
        res = torch.zeros((M, K), dtype=torch.float16, device="cuda")
        a = torch.empty_like(res)
        b = torch.empty_like(res)

        def chain(sync):
            res.zero_()
            cur = x0
            for lin in lins:
                P.qlinear_residual_rmsnorm(cur, res, g, 1e-5, 1.0, h_out=res, y_out=a)
                if sync:
                    torch.cuda.synchronize()
                lin.forward_raw(a.data_ptr(), b.data_ptr(), M)
                if sync:
                    torch.cuda.synchronize()
                cur = b
            torch.cuda.synchronize()
            return res.clone(), b.clone()

        ref = chain(True)
        for _ in range(4):
            got = chain(False)
            assert all(torch.equal(r.view(torch.int16), o.view(torch.int16)) for r, o in zip(ref, got))
