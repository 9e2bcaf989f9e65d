"""qlinear_forward_batch: layers with different inputs in one decode launch (the KV-head case of paper Section 3.8)."""
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


def layer(seed, N, K, bits, group):
    spec = C.LayerSpec("t", N, K, bits, group, *((-8, 7) if bits == 4 else (-128, 127)))
    return C.layer_weights(seed, spec), spec


@pytest.mark.parametrize("M", [1, 3, 8])
@pytest.mark.parametrize("Ns,K,bits,group", [((1280, 1280, 1280, 1280), 128, 8, 0), ((256, 136, 4096), 1024, 4, 32), ((512, 512), 2304, 4, 0),
                                              ((1000,), 512, 8, 0)])
def test_parity_every_layer_with_its_own_input(P, torch, M, Ns, K, bits, group):
    lins, ws, xs = [], [], []
    for i, N in enumerate(Ns):
        (q, s), spec = layer(300 + i + N, N, K, bits, group)
        lins.append(P.QLinear.from_weights(q, s, bits, group, device="cuda:0"))
        ws.append((q, s))
        xs.append(C.layer_activations(500 + i, spec, M))
    ys = P.qlinear_forward_batch(lins, [torch.from_numpy(x).cuda() for x in xs])
    torch.cuda.synchronize()
    assert lins[0].device_status() == (0, 0)
    for (q, s), x, y in zip(ws, xs, ys):
        y64, A, _ = O.linear(x, q, s, group)
        ok, rel, worst = O.check_against(y.cpu().numpy(), y64, A)
        assert ok, f"rel_l2={rel:.3e} worst={worst:.3e}"


def test_inputs_are_not_mixed_up(P, torch):
    """One-hot inputs: layer i gets e_(i+1), so output i must be column i + 1 of ITS weights (times its scale), exactly."""
    K, N, M = 128, 256, 1
    lins, cols, xs = [], [], []
    for i in range(4):
        (q, s), _ = layer(40 + i, N, K, 8, 0)
        lins.append(P.QLinear.from_weights(q, s, 8, 0, device="cuda:0"))
        x = np.zeros((M, K), np.float16)
        x[0, i + 1] = 1.0
        xs.append(torch.from_numpy(x).cuda())
        cols.append((q[:, i + 1].astype(np.float64) * s[:, 0].astype(np.float64)).astype(np.float16))
    ys = P.qlinear_forward_batch(lins, xs)
    for y, c in zip(ys, cols):
        assert (y.cpu().numpy()[0].view(np.uint16) == c.view(np.uint16)).all()


def test_kv_heads_in_one_launch(P, torch):
    d_h, size, heads, R = 128, 1280, 4, 4
    rng = np.random.default_rng(12)
    caches, refs, rows = [], [], []
    for h in range(heads):
        c = P.KVCache(size, d_h, device="cuda:0")
        k = rng.standard_normal((300 + 10 * h, d_h)).astype(np.float16)
        c.append(torch.from_numpy(k).cuda(), torch.from_numpy(k).cuda())
        r = torch.from_numpy(rng.standard_normal((R, d_h)).astype(np.float16)).cuda()
        caches.append(c)
        rows.append(r)
        refs.append(c.scores(r))
    got = P.kv_scores_batch(caches, rows)
    torch.cuda.synchronize()
    for g, r in zip(got, refs):
        assert torch.allclose(g.float(), r.float(), rtol=2e-3, atol=2e-3)


def test_falls_back_for_prefill_sizes_and_checks_arguments(P, torch):
    (q, s), spec = layer(7, 256, 256, 8, 0)
    lins = [P.QLinear.from_weights(q, s, 8, 0, device="cuda:0") for _ in range(2)]
    xs = [torch.from_numpy(C.layer_activations(9 + i, spec, 40)).cuda() for i in range(2)]
    ys = P.qlinear_forward_batch(lins, xs)                               # M = 40: two prefill calls
    for x, y in zip(xs, ys):
        y64, A, _ = O.linear(x.cpu().numpy(), q, s, 0)
        assert O.check_against(y.cpu().numpy(), y64, A)[0]
    with pytest.raises(P.QLinearError):
        P.qlinear_forward_batch(lins, xs[:1])
    with pytest.raises(P.QLinearError):
        P.qlinear_forward_batch(lins * 5, xs * 5)                        # more than 8 layers
