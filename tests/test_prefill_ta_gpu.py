"""Prefill kernel that keeps the dequantised weights in tensor memory (launches with at least one 256 x 256 tile per
CTA pair): against the CPU oracle on ragged shapes of every scheme, and bit for bit against the shared-memory form of
the same product, which a child process computes with the kernel switched off (the switch is read once per process).
Both forms feed the tensor cores the same fp16 weights in the same k order, so their outputs must be identical."""
import os
import subprocess
import sys

import numpy as np
import pytest

from oracle import qlinear_oracle as O
from workloads import configs as C

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def P(_built_library):
    import paper_2505_00232_b200 as P
    return P


@pytest.fixture(scope="module")
def torch():
    import torch
    assert torch.cuda.is_available(), "these tests need a CUDA device"
    return torch


# (M, N, K, bits, group): >= 74 tiles of 256 channels x 256 tokens each; ragged M, N and K tails; an odd number of
# int8 chunks; a single k-step pair; grouped and per-channel int4; group sizes the packer expands to 32
CASES = [
    (1000, 4856, 1056, 4, 32), (777, 6400, 352, 8, 0), (2048, 2560, 2304, 4, 0), (520, 9728, 640, 4, 128),
    (4096, 1280, 1024, 8, 0), (300, 19456, 128, 4, 64), (2047, 2816, 4096, 4, 32),
]


def case(seed, M, N, K, bits, group):
    layer = C.LayerSpec("t", N, K, bits, group, *((-8, 7) if bits == 4 else (-128, 127)))
    q, s = C.layer_weights(seed, layer)
    return q, s, C.layer_activations(seed, layer, M)


def run(P, torch, M, N, K, bits, group, seed):
    q, s, x = case(seed, M, N, K, bits, group)
    desc = P.Desc(N, K, bits, group)
    lin = P.QLinear(desc, torch.from_numpy(P.qlinear_pack(desc, q, s)).cuda())
    y = lin.forward(torch.from_numpy(x).cuda())
    torch.cuda.synchronize()
    st, detail = lin.device_status()
    assert st == 0, f"device status {st} detail {detail:#x}"
    return q, s, x, y.cpu().numpy()


@pytest.mark.parametrize("M,N,K,bits,group", CASES)
def test_parity_against_oracle(P, torch, M, N, K, bits, group):
    q, s, x, y = run(P, torch, M, N, K, bits, group, 7000 + M + N)
    assert np.isfinite(y.astype(np.float32)).all()
    rows = 2048
    d2 = y2 = worst = 0.0
    for r0 in range(0, N, rows):
        y64, A, _ = O.linear(x, q[r0:r0 + rows], s[r0:r0 + rows], group)
        d = y[:, r0:r0 + rows].astype(np.float64) - y64
        d2 += float((d * d).sum())
        y2 += float((y64 * y64).sum())
        with np.errstate(divide="ignore", invalid="ignore"):
            worst = max(worst, float(np.where(A > 0, np.abs(d) / A, np.where(d == 0, 0.0, np.inf)).max()))
    assert (d2 / y2) ** 0.5 <= O.REL_L2_TOL and worst <= O.ELEM_TOL, f"rel_l2={(d2 / y2) ** 0.5:.3e} worst={worst:.3e}"


CHILD = """
import sys, numpy as np, torch
sys.path.insert(0, {root!r})
import paper_2505_00232_b200 as P
from tests.test_prefill_ta_gpu import CASES, run
np.savez({out!r}, **{{str(i): run(P, torch, *c, 7000 + c[0] + c[1])[3] for i, c in enumerate(CASES)}})
"""


def test_bit_identical_to_the_shared_memory_form(P, torch, tmp_path):
    out = str(tmp_path / "shared_memory_form.npz")
    env = dict(os.environ, QLINEAR_GEMM_TA="0")
    subprocess.run([sys.executable, "-c", CHILD.format(root=ROOT, out=out)], check=True, env=env, cwd=ROOT, timeout=600)
    ref = np.load(out)
    for i, c in enumerate(CASES):
        y = run(P, torch, *c, 7000 + c[0] + c[1])[3]
        assert np.array_equal(y.view(np.uint16), ref[str(i)].view(np.uint16)), f"case {c}"


def test_guard_band_around_y(P, torch):
    """The output tile leaves through bulk copies of whole 256-byte rows: nothing outside [M, N] may be written."""
    M, N, K, bits, group = 300, 19448, 128, 4, 32                        # ragged last row super-block (120 channels)
    q, s, x = case(11, M, N, K, bits, group)
    desc = P.Desc(N, K, bits, group)
    lin = P.QLinear(desc, torch.from_numpy(P.qlinear_pack(desc, q, s)).cuda())
    pad = 4096
    buf = torch.full((pad + M * N + pad,), -7.0, dtype=torch.float16, device="cuda")
    xd = torch.from_numpy(x).cuda()
    lin.forward_raw(xd.data_ptr(), buf.data_ptr() + 2 * pad, M)
    torch.cuda.synchronize()
    h = buf.cpu().numpy()
    assert (h[:pad] == -7.0).all() and (h[pad + M * N:] == -7.0).all()
    y = h[pad:pad + M * N].reshape(M, N)
    y64, A, _ = O.linear(x, q, s, group)
    ok, rel, worst = O.check_against(y, y64, A)
    assert ok, f"rel_l2={rel:.3e} worst={worst:.3e}"


def test_dependent_launches_back_to_back(P, torch):
    """A chain y1 = L1(x), y2 = L2(y1), y3 = L3(y2) launched without any host synchronisation (each kernel releases the
    next one early and the next one may already run its set-up): same bits as the chain with a synchronise after every
    launch, on every repetition, with the buffers reused."""
    M, D = 1500, 4864                                                    # 19 row-super-block pairs x 6 token blocks = 114 tiles
    lins = []
    for i, (bits, group) in enumerate([(4, 32), (8, 0), (4, 0)]):
        q, s, _ = case(900 + i, 8, D, D, bits, group)
        desc = P.Desc(D, D, bits, group)
        lins.append(P.QLinear(desc, torch.from_numpy(P.qlinear_pack(desc, q, (s.astype(np.float32) / 16).astype(np.float16))).cuda()))
    x = torch.from_numpy(case(77, M, D, D, 4, 32)[2]).cuda()
    bufs = [torch.empty((M, D), dtype=torch.float16, device="cuda") for _ in range(3)]

    def chain(sync):
        src = x
        for lin, dst in zip(lins, bufs):
            lin.forward_raw(src.data_ptr(), dst.data_ptr(), M)
            if sync:
                torch.cuda.synchronize()
            src = dst
        torch.cuda.synchronize()
        return [b.clone() for b in bufs]

    ref = chain(True)
    assert all(torch.isfinite(r.float()).all() for r in ref)
    for _ in range(5):
        for b in bufs:
            b.fill_(float("nan"))
        got = chain(False)
        for r, g in zip(ref, got):
            assert torch.equal(r.view(torch.int16), g.view(torch.int16))
    assert lins[0].device_status() == (0, 0)


# (M, N, K, bits, group): whole tiles round-robin (two ring lengths), a K split of 4 and of 2 parts through the scratch,
# a launch of at most 128 tokens
STRESS = [(2048, 4096, 4096, 4, 32), (2048, 4096, 4096, 8, 0), (1024, 2304, 9216, 4, 32), (512, 4864, 2048, 8, 0), (64, 4096, 14336, 4, 0)]


@pytest.mark.parametrize("M,N,K,bits,group", STRESS)
def test_back_to_back_launches_keep_their_bits(P, torch, M, N, K, bits, group):
    """A few thousand launches in a row from two handles without host synchronisation (the pipelines of consecutive
    launches overlap, loads land in whatever order the memory system returns them): no bounded wait expires and every
    sampled output has the bits of the first one."""
    q, s, x = case(31 + M + K, M, N, K, bits, group)
    desc = P.Desc(N, K, bits, group)
    blob = torch.from_numpy(P.qlinear_pack(desc, q, s)).cuda()
    lins = [P.QLinear(desc, blob), P.QLinear(desc, blob.clone())]
    xd = torch.from_numpy(x).cuda()
    y = torch.empty((M, N), dtype=torch.float16, device="cuda")
    first = lins[0].forward(xd).clone()
    for rnd in range(6):
        for i in range(400):
            lins[i & 1].forward_raw(xd.data_ptr(), y.data_ptr(), M)
        assert torch.equal(y.view(torch.int16), first.view(torch.int16)), f"round {rnd}"
    torch.cuda.synchronize()
    assert lins[0].device_status() == (0, 0)


@pytest.mark.parametrize("form", ["gated", "grouped", "gated_fallback"])
def test_back_to_back_multi_layer_launches_keep_their_bits(P, torch, form):
    """The same for the launches that serve two layers: the fused gating (gate tile and up tile of a position back to
    back in one cluster), the grouped launch, and the gating of a shape the fused kernel does not take (both
    projections into the device scratch, then the element-wise kernel)."""
    M, N, K = (2048, 9728, 1024) if form != "gated_fallback" else (96, 2304, 2048)
    lins, xs = [], None
    for i in range(2):
        q, s, x = case(53 + i, M, N, K, 4, 32)
        desc = P.Desc(N, K, 4, 32)
        lins.append(P.QLinear(desc, torch.from_numpy(P.qlinear_pack(desc, q, s)).cuda()))
        xs = x
    xd = torch.from_numpy(xs).cuda()
    ys = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _ in range(2)]

    def launch():
        if form == "grouped":
            P.qlinear_forward_group_raw(lins, xd.data_ptr(), [y.data_ptr() for y in ys], M)
        else:
            P.qlinear_forward_gated_raw(lins[0], lins[1], xd.data_ptr(), ys[0].data_ptr(), M, "silu")
    launch()
    first = [y.clone() for y in ys]
    n_out = 2 if form == "grouped" else 1
    for rnd in range(5):
        for _ in range(300):
            launch()
        for y, f in zip(ys[:n_out], first[:n_out]):
            assert torch.equal(y.view(torch.int16), f.view(torch.int16)), f"round {rnd}"
    torch.cuda.synchronize()
    assert lins[0].device_status() == (0, 0)
