"""Prefill kernel (M > 8, tcgen05) against the CPU oracle, through the C-ABI, on a B200."""
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


def forward(P, torch, lin, x):
    assert lin.path_for(x.shape[0]) == P.QL_PATH_GEMM
    y = lin.forward(torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    st, detail = lin.device_status()
    assert st == 0, f"device status {st} detail {detail:#x}"
    return y.cpu().numpy()


def assert_parity(y_gpu, x, q, s, group):
    y64, A, _ = O.linear(x, q, s, group)
    ok, rel, worst = O.check_against(y_gpu, y64, A)
    assert ok, f"rel_l2={rel:.3e} (tol {O.REL_L2_TOL}) worst |dy|/A={worst:.3e} (tol {O.ELEM_TOL})"


def assert_parity_whole_output(y_gpu, x, q, s, group, rows=2048):
    """Every element of the M x N output against the oracle, walking N in blocks of `rows` output channels
    (bounds the oracle's fp64 working set).  The relative L2 error is taken over the whole output: squared
    norms are accumulated across the blocks; the per-element ratio is the maximum over all of them."""
    N = q.shape[0]
    d2 = y2 = 0.0
    worst = 0.0
    for r0 in range(0, N, rows):
        r1 = min(N, r0 + rows)
        y64, A, _ = O.linear(x, q[r0:r1], s[r0:r1], group)
        d = y_gpu[:, r0:r1].astype(np.float64) - y64
        d2 += float((d * d).sum())
        y2 += float((y64 * y64).sum())
        with np.errstate(divide="ignore", invalid="ignore"):
            ratio = np.where(A > 0, np.abs(d) / A, np.where(d == 0, 0.0, np.inf))
        worst = max(worst, float(ratio.max(initial=0.0)))
    rel = (d2 / y2) ** 0.5 if y2 > 0 else d2 ** 0.5
    assert rel <= O.REL_L2_TOL and worst <= O.ELEM_TOL, \
        f"rel_l2={rel:.3e} (tol {O.REL_L2_TOL}) worst |dy|/A={worst:.3e} (tol {O.ELEM_TOL})"
    assert np.isfinite(y_gpu.astype(np.float32)).all()


def rand_case(seed, M, N, K, bits, group):
    layer = C.LayerSpec("t", N, K, bits, group, *((-8, 7) if bits == 4 else (-128, 127)))
    q, s = C.layer_weights(seed, layer)
    return q, s, C.layer_activations(seed, layer, M)


SMALL = [
    # (M, N, K, bits, group): every tile width, ragged M / N / K tails, every scheme
    (9, 8, 32, 8, 0), (16, 128, 64, 4, 32), (17, 136, 160, 8, 0), (33, 200, 352, 4, 32), (64, 256, 512, 4, 0),
    (127, 264, 2304, 4, 32), (128, 128, 1056, 8, 0), (129, 384, 1024, 4, 32), (300, 520, 1056, 8, 0),
    (256, 40, 256, 4, 64), (257, 16, 384, 4, 128), (512, 1000, 96, 8, 0), (1024, 256, 2304, 4, 32),
    (700, 384, 4096, 8, 0), (2048, 128, 14336, 4, 32),
    # few tiles: the CTA-pair kernel splits K across clusters and adds the parts through scratch
    (600, 512, 2048, 8, 0), (300, 256, 4096, 4, 32), (1024, 1024, 1024, 4, 0),
]


@pytest.mark.parametrize("M,N,K,bits,group", SMALL)
def test_parity_small_and_ragged(P, torch, M, N, K, bits, group):
    q, s, x = rand_case(2000 + N + K + M, M, N, K, bits, group)
    lin = P.QLinear.from_weights(q, s, bits, group, device="cuda:0")
    assert_parity(forward(P, torch, lin, x), x, q, s, group)


@pytest.mark.parametrize("N,K,bits,group", [(136, 160, 8, 0), (200, 352, 4, 32), (264, 2304, 4, 32), (128, 1024, 4, 0)])
@pytest.mark.parametrize("M", [16, 200])
def test_one_hot_rows_return_rounded_weight_columns_bit_exact(P, torch, N, K, bits, group, M):
    q, s, _ = rand_case(31, 1, N, K, bits, group)
    lo, hi = (-8, 7) if bits == 4 else (-128, 127)
    q[:, 5], q[:, 6] = lo, hi
    G = K if group == 0 else group
    lin = P.QLinear.from_weights(q, s, bits, group, device="cuda:0")
    rng = np.random.default_rng(M)
    ks = np.concatenate([[0, 5, 6, 31, 32 % K, 63 % K, K - 1], rng.integers(0, K, size=M - 7)])
    x = np.zeros((M, K), np.float16)
    x[np.arange(M), ks] = 1.0
    y = forward(P, torch, lin, x)
    want = (s[:, ks // G].astype(np.float64) * q[:, ks].astype(np.float64)).astype(np.float16).T   # [M, N]
    assert (y.view(np.uint16) == want.view(np.uint16)).all()


def test_split_k_is_deterministic_and_counters_reset(P, torch):
    q, s, x = rand_case(47, 600, 512, 2048, 8, 0)
    lin = P.QLinear.from_weights(q, s, 8, 0, device="cuda:0")
    xd = torch.from_numpy(x).cuda()
    a = lin.forward(xd).clone()
    for _ in range(4):
        assert torch.equal(a, lin.forward(xd))
    assert_parity(a.cpu().numpy(), x, q, s, 0)


def test_zero_input_gives_positive_zero(P, torch):
    q, s, x = rand_case(37, 100, 200, 352, 4, 32)
    lin = P.QLinear.from_weights(q, s, 4, 32, device="cuda:0")
    y = forward(P, torch, lin, np.zeros_like(x))
    assert (y.view(np.uint16) == 0).all()


def test_forward_does_not_write_outside_y(P, torch):
    M, N, K = 77, 200, 352
    q, s, x = rand_case(41, M, N, K, 4, 32)
    lin = P.QLinear.from_weights(q, s, 4, 32, device="cuda:0")
    guard = 4096
    buf = torch.full((M * N + 2 * guard,), -7.0, dtype=torch.float16, device="cuda")
    y = buf[guard:guard + M * N].view(M, N)
    lin.forward(torch.from_numpy(x).cuda(), out=y)
    torch.cuda.synchronize()
    assert (buf[:guard] == -7.0).all() and (buf[-guard:] == -7.0).all()
    assert_parity(y.cpu().numpy(), x, q, s, 32)


def test_run_to_run_deterministic_and_stage_boundary(P, torch):
    q, s, x = rand_case(43, 9, 256, 1024, 8, 0)
    lin = P.QLinear.from_weights(q, s, 8, 0, device="cuda:0")
    xd = torch.from_numpy(x).cuda()
    a = lin.forward(xd).clone()
    for _ in range(3):
        assert torch.equal(a, lin.forward(xd))
    # M = 8 takes the decode kernel, M = 9 the prefill kernel: both within tolerance of the oracle
    assert lin.path_for(8) == P.QL_PATH_GEMV and lin.path_for(9) == P.QL_PATH_GEMM
    y8 = lin.forward(xd[:8].contiguous()).cpu().numpy()
    assert_parity(y8, x[:8], q, s, 0)
    assert_parity(a.cpu().numpy(), x, q, s, 0)


@pytest.mark.parametrize("li", range(3), ids=["gate", "up", "down"])
def test_parity_config4_gemma_prefill_full(P, torch, li):
    """Config 4 at full size, every output element against the oracle (fp64 matmul, ~seconds)."""
    w = C.CONFIGS[3]
    layer, M = w.layers[li], w.Ms[0]
    q, s = C.layer_weights(w.seed, layer, li)
    x = C.layer_activations(w.seed, layer, M, li)
    lin = P.QLinear.from_weights(q, s, layer.bits, layer.group, device="cuda:0")
    assert_parity(forward(P, torch, lin, x), x, q, s, layer.group)
    assert (lin.debug_unpack().cpu().numpy() == q).all()


@pytest.mark.parametrize("li", range(7), ids=[l.name for l in C.LLAMA31_8B])
def test_parity_config5_llama_prefill_full(P, torch, li):
    """Config 5 at full size (M = 2048), in the launch configuration the bench times: every one of the
    2048 x N outputs of every layer against the oracle."""
    w = C.CONFIGS[4]
    layer, M = w.layers[li], w.Ms[0]
    q, s = C.layer_weights(w.seed, layer, li)
    x = C.layer_activations(w.seed, layer, M, li)
    lin = P.QLinear.from_weights(q, s, layer.bits, layer.group, device="cuda:0")
    y = forward(P, torch, lin, x)
    assert_parity_whole_output(y, x, q, s, layer.group)


def test_lm_head_decode_config5b(P, torch):
    """The int4 LM head (128256 x 4096) at M = 1: all outputs against the oracle."""
    w = C.CONFIG_5B
    layer = w.layers[0]
    q, s = C.layer_weights(w.seed, layer, 7)
    x = C.layer_activations(w.seed, layer, 1, 7)
    lin = P.QLinear.from_weights(q, s, layer.bits, layer.group, device="cuda:0")
    y = lin.forward(torch.from_numpy(x).cuda()).cpu().numpy()
    y64 = np.empty((1, layer.N))
    A = np.empty((1, layer.N))
    for r0 in range(0, layer.N, 16384):                      # bounds the oracle's fp64 working set
        r1 = min(layer.N, r0 + 16384)
        y64[:, r0:r1], A[:, r0:r1], _ = O.linear(x, q[r0:r1], s[r0:r1], layer.group)
    ok, rel, worst = O.check_against(y, y64, A)
    assert ok, (rel, worst)


GROUPS = [
    # (M, K, bits, group, [N_i]): one launch of the CTA-pair kernel for layers that share x
    (300, 512, 8, 0, [512, 256, 256]),           # q/k/v-like; few tiles: split along K
    (200, 1024, 4, 32, [200, 256]),              # ragged N, ragged M
    (1024, 256, 8, 0, [2560, 1280, 1024]),       # enough tiles for 512-token tiles
    (640, 384, 4, 0, [512, 768]),                # int4 per channel
]


@pytest.mark.parametrize("M,K,bits,group,Ns", GROUPS)
def test_forward_group_prefill_parity(P, torch, M, K, bits, group, Ns):
    cases = [rand_case(8000 + 13 * i + N + K, M, N, K, bits, group) for i, N in enumerate(Ns)]
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
        assert torch.equal(a, b)


@pytest.mark.parametrize("names", [("q", "k", "v"), ("gate", "up")], ids=["qkv", "gate_up"])
def test_forward_group_config5_llama_prefill_full(P, torch, names):
    """The grouped prefill launches bench.py times (config 5, M = 2048): every output element of every
    layer of the group against the oracle."""
    w = C.CONFIGS[4]
    M = w.Ms[0]
    ids = [i for i, l in enumerate(w.layers) if l.name in names]
    ws = [C.layer_weights(w.seed, w.layers[i], i) for i in ids]
    x = C.layer_activations(w.seed, w.layers[ids[0]], M, ids[0])
    lins = [P.QLinear.from_weights(q, s, w.layers[i].bits, w.layers[i].group, device="cuda:0") for i, (q, s) in zip(ids, ws)]
    ys = P.qlinear_forward_group(lins, torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    assert lins[0].device_status()[0] == 0
    for i, (q, s), y in zip(ids, ws, ys):
        assert_parity_whole_output(y.cpu().numpy(), x, q, s, w.layers[i].group)
