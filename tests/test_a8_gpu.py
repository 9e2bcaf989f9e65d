"""The linear layer with int8 activations (paper Section 3.7) against the step-by-step CPU oracle, through the
C-ABI, on a B200: the quantisation kernel bit-exact, the fused decode kernel exact in its integer part."""
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


def rand_case(seed, M, N, K, bits, group):
    layer = C.LayerSpec("t", N, K, bits, group, *((-8, 7) if bits == 4 else (-128, 127)))
    q, s = C.layer_weights(seed, layer)
    return q, s, C.layer_activations(seed, layer, M)


def assert_a8(y_gpu, x, q, s, group):
    """Integer part exact, so only the fp32 dequantisation and the fp16 rounding separate the two:
    |y - y64| <= 2^-10 |y64| + 1e-5 * scale_x * sum_g |s * acc_g| + 2^-25 (the last term: half the spacing of the fp16
    subnormals, the rounding error of an output below 2^-14, where it no longer shrinks with |y|)."""
    y64, acc, xq, sx, _ = O.linear_int8_activations(x, q, s, group)
    N, K = q.shape
    G = K if group == 0 else group
    mag = sx.astype(np.float64)[:, None] * np.einsum("mng,ng->mn", np.abs(acc).astype(np.float64), np.abs(s.reshape(N, K // G).astype(np.float64)))
    d = np.abs(y_gpu.astype(np.float64) - y64)
    bound = 2.0 ** -10 * np.abs(y64) + 1e-5 * mag + 2.0 ** -25
    assert (d <= bound).all(), f"worst |dy|/bound = {(d / bound).max():.3e}"


@pytest.mark.parametrize("M,K", [(1, 32), (3, 352), (8, 4096), (5, 14336)])
def test_quantisation_kernel_is_bit_exact(P, torch, M, K):
    x = C.layer_activations(70 + M, C.LayerSpec("t", 8, K, 8, 0, 0, 0), M)
    x[0, :] *= np.float16(37.0)                       # different magnitudes per token
    if M > 2:
        x[2, :] = 0                                   # a row of zeros: scale 1, zeros
    xq, sx = P.qlinear_quantize_activations(torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    xq_ref, sx_ref = O.quantize_activations(x)
    assert (xq.cpu().numpy() == xq_ref).all()
    assert (sx.cpu().numpy().view(np.uint32) == sx_ref.view(np.uint32)).all()


CASES = [
    # (M, N, K, bits, group): every scheme, ragged N, K slices inside a CTA and across a cluster
    (1, 2304, 2304, 8, 0), (4, 264, 2304, 4, 32), (8, 1024, 4096, 4, 32), (2, 4096, 4096, 8, 0), (5, 384, 4096, 4, 0),
    (1, 520, 1056, 8, 0), (3, 200, 352, 4, 32), (7, 136, 160, 8, 0), (1, 4096, 14336, 4, 32), (8, 512, 14336, 4, 32), (4, 4096, 14336, 8, 0),
    (1, 8, 32, 8, 0), (2, 16, 64, 4, 64),
]


@pytest.mark.parametrize("M,N,K,bits,group", CASES)
def test_a8_decode_parity(P, torch, M, N, K, bits, group):
    q, s, x = rand_case(7000 + N + K + M, M, N, K, bits, group)
    lin = P.QLinear.from_weights(q, s, bits, group, device="cuda:0")
    xd = torch.from_numpy(x).cuda()
    y = lin.forward_a8(xd)
    torch.cuda.synchronize()
    assert lin.device_status() == (0, 0)
    assert_a8(y.cpu().numpy(), x, q, s, group)
    assert torch.equal(y, lin.forward_a8(xd))         # run-to-run identical


@pytest.mark.parametrize("bits,group", [(8, 0), (4, 32), (4, 0)])
def test_a8_integer_path_is_bit_exact_when_no_rounding_is_left(P, torch, bits, group):
    """Power-of-two scales and x on the int8 grid: every fp32 operation of the dequantisation is exact, so the
    fp16 result must equal the oracle's bit for bit -- which it can only do if every integer dot product is exact
    (weight extremes -8 / -128 and activation extremes +-127 included)."""
    M, N, K = 4, 200, 1024
    rng = np.random.default_rng(3)
    lo, hi = (-8, 7) if bits == 4 else (-128, 127)
    q = rng.integers(lo, hi + 1, size=(N, K)).astype(np.int8)
    q[:, 0], q[:, 1] = lo, hi
    G = K if group == 0 else group
    s = (2.0 ** rng.integers(-12, -8, size=(N, K // G))).astype(np.float16)
    ints = rng.integers(-127, 128, size=(M, K))
    ints[:, 0], ints[:, 1] = 127, -127
    x = (ints * np.array([[2.0 ** -6], [2.0 ** -3], [1.0], [2.0 ** -5]])).astype(np.float16)
    lin = P.QLinear.from_weights(q, s, bits, group, device="cuda:0")
    y = lin.forward_a8(torch.from_numpy(x).cuda()).cpu().numpy()
    y64, acc, xq, sx, y16 = O.linear_int8_activations(x, q, s, group)
    assert (xq == ints).all()
    assert (y.view(np.uint16) == y16.view(np.uint16)).all()


PREFILL = [
    # (M, N, K, bits): per-channel schemes on the integer tensor-core path (K a multiple of 128, 256-channel tiles)
    (129, 256, 128, 8), (300, 512, 1024, 8), (256, 256, 2304, 4), (700, 768, 1152, 4), (1024, 1024, 4096, 4), (2048, 256, 14336, 8),
    (257, 1000, 512, 8),
    # enough tiles for the kernel that keeps the weight bytes in tensor memory (more than a quarter of the SM count):
    # ragged M, both bit widths, a single k-step, ragged N
    (520, 4864, 384, 4), (1000, 2560, 640, 8), (300, 9728, 128, 4), (777, 5112, 1280, 8),
]


@pytest.mark.parametrize("M,N,K,bits", PREFILL)
def test_a8_prefill_parity(P, torch, M, N, K, bits):
    """Prefill stage: quantisation kernel + kind::i8 matmul + output dequantisation against the same oracle."""
    q, s, x = rand_case(7300 + N + K + M, M, N, K, bits, 0)
    lin = P.QLinear.from_weights(q, s, bits, 0, device="cuda:0")
    xd = torch.from_numpy(x).cuda()
    y = lin.forward_a8(xd)
    torch.cuda.synchronize()
    assert lin.device_status() == (0, 0)
    assert_a8(y.cpu().numpy(), x, q, s, 0)
    assert torch.equal(y, lin.forward_a8(xd))


@pytest.mark.parametrize("bits,N", [(8, 256), (4, 256), (8, 9728), (4, 9728)])
def test_a8_prefill_integer_path_is_bit_exact_when_no_rounding_is_left(P, torch, bits, N):
    M, K = 300, 512
    rng = np.random.default_rng(4)
    lo, hi = (-8, 7) if bits == 4 else (-128, 127)
    q = rng.integers(lo, hi + 1, size=(N, K)).astype(np.int8)
    q[:, 0], q[:, 1] = lo, hi
    s = (2.0 ** rng.integers(-12, -8, size=(N, 1))).astype(np.float16)
    ints = rng.integers(-127, 128, size=(M, K))
    ints[:, 0], ints[:, 1] = 127, -127
    x = (ints * (2.0 ** -rng.integers(0, 6, size=(M, 1)))).astype(np.float16)
    lin = P.QLinear.from_weights(q, s, bits, 0, device="cuda:0")
    y = lin.forward_a8(torch.from_numpy(x).cuda()).cpu().numpy()
    _, _, xq, _, y16 = O.linear_int8_activations(x, q, s, 0)
    assert (xq == ints).all()
    assert (y.view(np.uint16) == y16.view(np.uint16)).all()


@pytest.mark.parametrize("name,bits", [("q", 8), ("gate", 4), ("down", 4)])
def test_a8_prefill_llama_shapes_full_size(P, torch, name, bits):
    """The Llama3.1-8B shapes at M = 2048 in the paper's own schemes (q8 attention, per-channel int4 feed-forward)."""
    layer = [l for l in C.LLAMA31_8B if l.name == name][0]
    spec = C.LayerSpec(name, layer.N, layer.K, bits, 0, *((-8, 7) if bits == 4 else (-128, 127)))
    q, s = C.layer_weights(7400, spec)
    x = C.layer_activations(7400, spec, 2048)
    lin = P.QLinear.from_weights(q, s, bits, 0, device="cuda:0")
    y = lin.forward_a8(torch.from_numpy(x).cuda()).cpu().numpy()
    for r0 in range(0, layer.N, 2048):                  # bounds the oracle's working set
        assert_a8(y[:, r0:r0 + 2048], x, q[r0:r0 + 2048], s[r0:r0 + 2048], 0)


@pytest.mark.parametrize("bits", [8, 4])
def test_a8_prefill_back_to_back_launches_keep_their_bits(P, torch, bits):
    """Several thousand integer-form launches in a row from two handles, without host synchronisation in between: no
    bounded wait expires and every sampled output has the bits of the first one.  (The weight ring of the int8 form is
    not a multiple of the three dequantise turns long; a warp that takes a stage's previous phase for its own reads stale
    bytes and leaves the ring one arrival short, which shows up only under particular load timings.)"""
    N, K, M = 4096, 4096, 2048
    q, s, x = rand_case(7500 + bits, M, N, K, bits, 0)
    lins = [P.QLinear.from_weights(q, s, bits, 0, device="cuda:0") for _ in range(2)]
    xd = torch.from_numpy(x).cuda()
    y = torch.empty((M, N), dtype=torch.float16, device="cuda:0")
    first = lins[0].forward_a8(xd).clone()
    for rnd in range(6):
        for i in range(500):
            lins[i & 1].forward_a8_raw(xd.data_ptr(), y.data_ptr(), M)
        assert torch.equal(y, first), f"round {rnd}"
    torch.cuda.synchronize()
    assert lins[0].device_status() == (0, 0)


def test_a8_zero_input_and_guard_bands(P, torch):
    q, s, x = rand_case(7100, 3, 200, 352, 4, 32)
    lin = P.QLinear.from_weights(q, s, 4, 32, device="cuda:0")
    guard = 1024
    buf = torch.full((3 * 200 + 2 * guard,), -7.0, dtype=torch.float16, device="cuda")
    y = buf[guard:guard + 600].view(3, 200)
    lin.forward_a8(torch.zeros((3, 352), dtype=torch.float16, device="cuda"), out=y)
    torch.cuda.synchronize()
    assert (buf[:guard] == -7.0).all() and (buf[-guard:] == -7.0).all()
    assert (y == 0).all()
    with pytest.raises(P.QLinearError) as err:        # prefill stage: per-channel schemes only
        lin.forward_a8(torch.zeros((300, 352), dtype=torch.float16, device="cuda"))
    assert err.value.status == P.QL_ERR_UNSUPPORTED


@pytest.mark.parametrize("li", range(7), ids=[l.name for l in C.LLAMA31_8B])
def test_a8_config3_llama_decode_full_size(P, torch, li):
    w = C.CONFIGS[2]
    layer = w.layers[li]
    q, s = C.layer_weights(w.seed, layer, li)
    for M in w.Ms:
        x = C.layer_activations(w.seed, layer, M, li)
        lin = P.QLinear.from_weights(q, s, layer.bits, layer.group, device="cuda:0")
        y = lin.forward_a8(torch.from_numpy(x).cuda()).cpu().numpy()
        assert_a8(y, x, q, s, layer.group)
