"""Decode kernel (M <= 8) against the CPU oracle, through the C-ABI, on a B200."""
import numpy as np
import pytest

from oracle import qlinear_oracle as O
from workloads import configs as C

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


def run_layer(P, torch, q, s, bits, group, x):
    lin = P.QLinear.from_weights(q, s, bits, group, device="cuda:0")
    assert lin.path_for(x.shape[0]) == P.QL_PATH_GEMV
    xd = torch.from_numpy(x).cuda()
    y = lin.forward(xd)
    torch.cuda.synchronize()
    st, detail = lin.device_status()
    assert st == 0, f"device status {st} detail {detail:#x}"
    return lin, y.cpu().numpy()


def assert_parity(y_gpu, x, q, s, group):
    y64, A, _ = O.linear(x, q, s, group)
    ok, rel, worst = O.check_against(y_gpu, y64, A)
    assert ok, f"rel_l2={rel:.3e} (tol {O.REL_L2_TOL}) worst |dy|/A={worst:.3e} (tol {O.ELEM_TOL})"
    return rel, worst


def rand_case(seed, M, N, K, bits, group):
    layer = C.LayerSpec("t", N, K, bits, group, *((-8, 7) if bits == 4 else (-128, 127)))
    q, s = C.layer_weights(seed, layer)
    x = C.layer_activations(seed, layer, M)
    return q, s, x


SMALL = [
    # (M, N, K, bits, group): several row-blocks / chunks, ragged N and K tails, every scheme
    (1, 8, 32, 8, 0), (1, 8, 32, 4, 32), (3, 24, 96, 4, 32), (8, 136, 160, 8, 0), (5, 200, 352, 4, 32),
    (2, 264, 2304, 4, 32), (7, 520, 1056, 8, 0), (4, 40, 256, 4, 64), (6, 16, 384, 4, 128), (1, 1000, 64, 8, 0),
    (8, 384, 4096, 4, 0), (1, 2304, 2304, 8, 0), (2, 128, 14336, 4, 32), (8, 128, 14336, 4, 32), (8, 64, 9216, 8, 0),
]


@pytest.mark.parametrize("M,N,K,bits,group", SMALL)
def test_parity_small_and_ragged(P, torch, M, N, K, bits, group):
    q, s, x = rand_case(1000 + N + K, M, N, K, bits, group)
    _, y = run_layer(P, torch, q, s, bits, group, x)
    assert_parity(y, x, q, s, group)


@pytest.mark.parametrize("M,N,K,bits,group", [(1, 136, 160, 8, 0), (4, 200, 352, 4, 32), (8, 40, 256, 4, 64),
                                              (3, 2304, 2304, 8, 0), (2, 384, 4096, 4, 0)])
def test_device_unpack_is_bit_exact(P, torch, M, N, K, bits, group):
    q, s, x = rand_case(7, M, N, K, bits, group)
    lo, hi = (-8, 7) if bits == 4 else (-128, 127)
    q[0, 0], q[-1, -1], q[N // 2, K // 2] = lo, hi, lo
    lin = P.QLinear.from_weights(q, s, bits, group, device="cuda:0")
    qd = lin.debug_unpack().cpu().numpy()
    assert (qd == q).all()


@pytest.mark.parametrize("N,K,bits,group", [(136, 160, 8, 0), (200, 352, 4, 32), (264, 2304, 4, 32), (128, 4096, 4, 0)])
def test_one_hot_returns_rounded_weight_column_bit_exact(P, torch, N, K, bits, group):
    q, s, _ = rand_case(11, 1, N, K, bits, group)
    lo, hi = (-8, 7) if bits == 4 else (-128, 127)
    q[:, 5] = lo
    q[:, 6] = hi
    G = K if group == 0 else group
    lin = P.QLinear.from_weights(q, s, bits, group, device="cuda:0")
    ks = [0, 5, 6, 31, 32, 63, 64 % K, K - 1, K // 2 + 1]
    for m_tokens in (1, 8):
        x = np.zeros((m_tokens, K), np.float16)
        for m in range(m_tokens):
            x[m, ks[m % len(ks)] if m_tokens > 1 else 0] = 1.0
        for k0 in (ks if m_tokens == 1 else [None]):
            if k0 is not None:
                x[:] = 0
                x[0, k0] = 1.0
            y = lin.forward(torch.from_numpy(x).cuda()).cpu().numpy()
            for m in range(m_tokens):
                kk = int(np.argmax(x[m]))
                want = (s[:, kk // G].astype(np.float64) * q[:, kk].astype(np.float64)).astype(np.float16)
                assert (y[m].view(np.uint16) == want.view(np.uint16)).all(), (m_tokens, kk)


def test_zero_input_gives_positive_zero(P, torch):
    q, s, x = rand_case(13, 8, 200, 352, 4, 32)
    _, y = run_layer(P, torch, q, s, 4, 32, np.zeros_like(x))
    assert (y.view(np.uint16) == 0).all()


def test_forward_does_not_write_outside_y(P, torch):
    q, s, x = rand_case(17, 3, 200, 352, 4, 32)
    lin = P.QLinear.from_weights(q, s, 4, 32, device="cuda:0")
    guard = 1024
    buf = torch.full((3 * 200 + 2 * guard,), -7.0, dtype=torch.float16, device="cuda")
    y = buf[guard:guard + 600].view(3, 200)
    lin.forward(torch.from_numpy(x).cuda(), out=y)
    torch.cuda.synchronize()
    assert (buf[:guard] == -7.0).all() and (buf[-guard:] == -7.0).all()
    assert_parity(y.cpu().numpy(), x, q, s, 32)


def test_run_to_run_deterministic(P, torch):
    q, s, x = rand_case(19, 4, 1024, 4096, 8, 0)
    lin = P.QLinear.from_weights(q, s, 8, 0, device="cuda:0")
    xd = torch.from_numpy(x).cuda()
    a = lin.forward(xd).clone()
    for _ in range(5):
        assert torch.equal(a, lin.forward(xd))


def test_forward_argument_errors(P, torch):
    q, s, x = rand_case(23, 1, 16, 64, 8, 0)
    lin = P.QLinear.from_weights(q, s, 8, 0, device="cuda:0")
    xd = torch.from_numpy(x).cuda()
    y = torch.empty((1, 16), dtype=torch.float16, device="cuda")
    import ctypes
    f = P.lib.qlinear_forward
    assert f(lin._h, None, ctypes.c_void_p(y.data_ptr()), 1, None) == 1
    assert f(lin._h, ctypes.c_void_p(xd.data_ptr()), None, 1, None) == 1
    assert f(lin._h, ctypes.c_void_p(xd.data_ptr()), ctypes.c_void_p(y.data_ptr()), 0, None) == 1
    assert f(lin._h, ctypes.c_void_p(xd.data_ptr() + 2), ctypes.c_void_p(y.data_ptr()), 1, None) == 1
    with pytest.raises(P.QLinearError):
        lin.forward(xd.float())


def _config_cases():
    out = []
    for w in (C.CONFIGS[0], C.CONFIGS[1], C.CONFIGS[2]):
        for li, layer in enumerate(w.layers):
            for M in w.Ms:
                out.append(pytest.param(w, li, M, id=f"{w.name}-{layer.name}-M{M}"))
    return out


@pytest.mark.parametrize("w,li,M", _config_cases())
def test_parity_decode_configs_full_size(P, torch, w, li, M):
    """Configs 1-3 at their full shapes (the oracle's fp64 matmul handles M <= 8 in seconds)."""
    layer = w.layers[li]
    q, s = C.layer_weights(w.seed, layer, li)
    x = C.layer_activations(w.seed, layer, M, li)
    lin, y = run_layer(P, torch, q, s, layer.bits, layer.group, x)
    assert_parity(y, x, q, s, layer.group)
    # device-side integers, sampled rows (full compare for the small layers)
    qd = lin.debug_unpack().cpu().numpy()
    assert (qd == q).all()


@pytest.mark.parametrize("M,N,K,bits,group", [(1, 2304, 2304, 8, 0), (3, 264, 2304, 4, 32), (8, 1024, 4096, 4, 32),
                                              (2, 4096, 4096, 8, 0), (5, 384, 4096, 4, 0), (1, 520, 1056, 8, 0)])
def test_streaming_kernel_parity(P, torch, monkeypatch, M, N, K, bits, group):
    """The optional persistent streaming decode kernel (selected at handle creation) meets the same bar."""
    monkeypatch.setenv("QLINEAR_GEMV_KERNEL", "stream")
    q, s, x = rand_case(3000 + N + K, M, N, K, bits, group)
    lin, y = run_layer(P, torch, q, s, bits, group, x)
    assert_parity(y, x, q, s, group)
    xd = torch.from_numpy(x).cuda()
    a = lin.forward(xd).clone()
    for _ in range(3):
        assert torch.equal(a, lin.forward(xd))           # counters reset themselves between launches
    xo = np.zeros_like(x)
    xo[:, 7] = 1.0
    G = K if group == 0 else group
    want = (s[:, 7 // G].astype(np.float64) * q[:, 7].astype(np.float64)).astype(np.float16)
    yo = lin.forward(torch.from_numpy(xo).cuda()).cpu().numpy()
    assert (yo.view(np.uint16) == want.view(np.uint16)[None, :]).all()


GROUPS = [
    # (M, K, bits, group, [N_i]): q/k/v-like and gate/up-like groups, ragged N, N not a multiple of 16, K tail
    (1, 4096, 8, 0, [4096, 1024, 1024]), (4, 2304, 8, 0, [2048, 1024, 1024]), (1, 4096, 4, 32, [2048, 2048]),
    (8, 2304, 4, 32, [1160, 520]), (3, 352, 4, 32, [200, 8, 24, 136]), (2, 160, 8, 0, [136, 8]), (5, 384, 4, 0, [40, 264]),
]


@pytest.mark.parametrize("M,K,bits,group,Ns", GROUPS)
def test_forward_group_parity(P, torch, M, K, bits, group, Ns):
    """Layers that share x in one launch: every layer's output meets the single-layer bar."""
    cases = [rand_case(5000 + 17 * i + N + K, M, N, K, bits, group) for i, N in enumerate(Ns)]
    x = cases[0][2]
    lins = [P.QLinear.from_weights(q, s, bits, group, device="cuda:0") for q, s, _ in cases]
    xd = torch.from_numpy(x).cuda()
    ys = P.qlinear_forward_group(lins, xd)
    torch.cuda.synchronize()
    assert lins[0].device_status()[0] == 0
    for (q, s, _), y in zip(cases, ys):
        assert_parity(y.cpu().numpy(), x, q, s, group)
    again = P.qlinear_forward_group(lins, xd)
    for a, b in zip(ys, again):
        assert torch.equal(a, b)                         # run-to-run identical
    # a one-hot x gives the correctly rounded single product in every layer, bit for bit
    xo = np.zeros_like(x)
    xo[:, 5] = 1.0
    G = K if group == 0 else group
    yo = P.qlinear_forward_group(lins, torch.from_numpy(xo).cuda())
    for (q, s, _), y in zip(cases, yo):
        want = (s.reshape(q.shape[0], -1)[:, 5 // G].astype(np.float64) * q[:, 5].astype(np.float64)).astype(np.float16)
        assert (y.cpu().numpy().view(np.uint16) == want.view(np.uint16)[None, :]).all()


def test_forward_group_prefill_and_errors(P, torch):
    """M > 8 with layers the CTA-pair prefill kernel does not take (M <= 128) runs them one after the other (same
    results as single calls); mismatched layers are refused."""
    M, K = 24, 256
    cases = [rand_case(6000 + N, M, N, K, 4, 32) for N in (128, 264)]
    x = cases[0][2]
    lins = [P.QLinear.from_weights(q, s, 4, 32, device="cuda:0") for q, s, _ in cases]
    xd = torch.from_numpy(x).cuda()
    ys = P.qlinear_forward_group(lins, xd)
    for lin, y in zip(lins, ys):
        assert torch.equal(y, lin.forward(xd))
    q8, s8, _ = rand_case(6100, M, 128, K, 8, 0)
    other = P.QLinear.from_weights(q8, s8, 8, 0, device="cuda:0")
    with pytest.raises(P.QLinearError):
        P.qlinear_forward_group([lins[0], other], xd)
    with pytest.raises(P.QLinearError):
        P.qlinear_forward_group(lins * 3, xd)            # more than four layers


@pytest.mark.parametrize("wi,names,M", [(2, ("q", "k", "v"), 1), (2, ("gate", "up"), 1), (2, ("gate", "up"), 4),
                                        (1, ("q", "k", "v"), 1), (1, ("gate", "up"), 1)])
def test_forward_group_configs_full_size(P, torch, wi, names, M):
    """The grouped launches bench.py times (configs 2 and 3 at full size) against the oracle, layer by layer."""
    w = C.CONFIGS[wi]
    ids = [i for i, l in enumerate(w.layers) if l.name in names]
    ws = [C.layer_weights(w.seed, w.layers[i], i) for i in ids]
    x = C.layer_activations(w.seed, w.layers[ids[0]], M, ids[0])
    lins = [P.QLinear.from_weights(q, s, w.layers[i].bits, w.layers[i].group, device="cuda:0") for i, (q, s) in zip(ids, ws)]
    ys = P.qlinear_forward_group(lins, torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    assert lins[0].device_status()[0] == 0
    for i, (q, s), y in zip(ids, ws, ys):
        assert_parity(y.cpu().numpy(), x, q, s, w.layers[i].group)
