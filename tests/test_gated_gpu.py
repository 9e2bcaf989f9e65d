"""Fused gating y = act(gate) * up (paper Section 3.6) against the CPU oracle, through the C-ABI, on a B200."""
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


def make(seed, N, K, bits, group):
    layer = C.LayerSpec("t", N, K, bits, group, *((-8, 7) if bits == 4 else (-128, 127)))
    return C.layer_weights(seed, layer), C.layer_weights(seed + 1, layer)


def run(P, torch, gate_w, up_w, bits, group, x, act):
    lg = P.QLinear.from_weights(*gate_w, bits, group, device="cuda:0")
    lu = P.QLinear.from_weights(*up_w, bits, group, device="cuda:0")
    y = P.qlinear_forward_gated(lg, lu, torch.from_numpy(x).cuda(), act)
    torch.cuda.synchronize()
    assert lg.device_status() == (0, 0)
    return lg, lu, y


def assert_gated(y, x, gate_w, up_w, group, act, rows=2048):
    """Every element against the oracle, walking N in blocks; rel-L2 over the whole output."""
    N = gate_w[0].shape[0]
    d2 = y2 = worst = 0.0
    for r0 in range(0, N, rows):
        r1 = min(N, r0 + rows)
        y64, bound, _ = O.gated_linear(x, gate_w[0][r0:r1], gate_w[1][r0:r1], up_w[0][r0:r1], up_w[1][r0:r1], group, act)
        d = y[:, r0:r1].astype(np.float64) - y64
        d2 += float((d * d).sum())
        y2 += float((y64 * y64).sum())
        with np.errstate(divide="ignore", invalid="ignore"):
            ratio = np.where(bound > 0, np.abs(d) / bound, np.where(d == 0, 0.0, np.inf))
        worst = max(worst, float(ratio.max(initial=0.0)))
    rel = (d2 / y2) ** 0.5 if y2 > 0 else d2 ** 0.5
    assert rel <= O.REL_L2_TOL and worst <= 1.0, f"rel_l2={rel:.3e} worst |dy|/bound={worst:.3e}"


CASES = [
    # (M, N, K, bits, group, act): decode (fused in one launch), prefill (fused in the CTA-pair kernel: M > 128 and
    # a multiple of 256 channels after padding), and shapes that take the unfused route
    (1, 2048, 4096, 4, 32, "silu"), (4, 1160, 2304, 4, 32, "gelu_tanh"), (8, 520, 1024, 8, 0, "silu"), (3, 264, 512, 4, 0, "identity"),
    (2, 200, 352, 4, 32, "silu"),                                        # K not a whole number of int4 chunks: unfused
    (300, 512, 1024, 4, 32, "silu"), (1024, 256, 2304, 4, 32, "gelu_tanh"), (257, 1000, 512, 8, 0, "silu"), (700, 768, 384, 4, 0, "identity"),
    (24, 264, 256, 4, 32, "silu"), (128, 384, 512, 8, 0, "gelu_tanh"), (200, 384, 512, 4, 32, "silu"),   # unfused: M <= 128, odd tile count
]


@pytest.mark.parametrize("M,N,K,bits,group,act", CASES)
def test_gated_parity(P, torch, M, N, K, bits, group, act):
    gate_w, up_w = make(9000 + M + N + K, N, K, bits, group)
    x = C.layer_activations(9000 + M, C.LayerSpec("t", N, K, bits, group, 0, 0), M)
    lg, lu, y = run(P, torch, gate_w, up_w, bits, group, x, act)
    assert_gated(y.cpu().numpy(), x, gate_w, up_w, group, act)
    again = P.qlinear_forward_gated(lg, lu, torch.from_numpy(x).cuda(), act)
    assert torch.equal(y, again)                                          # run-to-run identical


def test_gated_does_not_write_outside_y_and_zero_input_gives_zero(P, torch):
    for M in (3, 300):
        N, K = 512, 1024
        gate_w, up_w = make(9100 + M, N, K, 4, 32)
        lg = P.QLinear.from_weights(*gate_w, 4, 32, device="cuda:0")
        lu = P.QLinear.from_weights(*up_w, 4, 32, device="cuda:0")
        guard = 4096
        buf = torch.full((M * N + 2 * guard,), -7.0, dtype=torch.float16, device="cuda")
        y = buf[guard:guard + M * N].view(M, N)
        P.qlinear_forward_gated(lg, lu, torch.zeros((M, K), dtype=torch.float16, device="cuda"), "silu", out=y)
        torch.cuda.synchronize()
        assert (buf[:guard] == -7.0).all() and (buf[-guard:] == -7.0).all()
        assert (y == 0).all()


def test_gated_refuses_layers_that_do_not_agree(P, torch):
    (qa, sa), _ = make(9200, 256, 512, 4, 32)
    (qb, sb), _ = make(9201, 128, 512, 4, 32)
    a = P.QLinear.from_weights(qa, sa, 4, 32, device="cuda:0")
    b = P.QLinear.from_weights(qb, sb, 4, 32, device="cuda:0")
    x = torch.zeros((2, 512), dtype=torch.float16, device="cuda")
    with pytest.raises(P.QLinearError):
        P.qlinear_forward_gated(a, b, x, "silu")
    import ctypes
    y = torch.zeros((2, 256), dtype=torch.float16, device="cuda")
    assert P.lib.qlinear_forward_gated(a._h, a._h, ctypes.c_void_p(x.data_ptr()), ctypes.c_void_p(y.data_ptr()), 2, 7, None) == 1


@pytest.mark.parametrize("wi,M,act", [(2, 1, "silu"), (2, 4, "silu"), (1, 1, "gelu_tanh"), (3, 1024, "gelu_tanh"), (4, 2048, "silu")],
                         ids=["llama-decode-M1", "llama-decode-M4", "gemma-decode-M1", "gemma-prefill-M1024", "llama-prefill-M2048"])
def test_gated_configs_full_size(P, torch, wi, M, act):
    """The gate / up layers of configs 2-5 at full size, every output element against the oracle."""
    w = C.CONFIGS[wi]
    ig = [i for i, l in enumerate(w.layers) if l.name == "gate"][0]
    iu = [i for i, l in enumerate(w.layers) if l.name == "up"][0]
    layer = w.layers[ig]
    gate_w, up_w = C.layer_weights(w.seed, layer, ig), C.layer_weights(w.seed, w.layers[iu], iu)
    x = C.layer_activations(w.seed, layer, M, ig)
    _, _, y = run(P, torch, gate_w, up_w, layer.bits, layer.group, x, act)
    assert_gated(y.cpu().numpy(), x, gate_w, up_w, layer.group, act)
