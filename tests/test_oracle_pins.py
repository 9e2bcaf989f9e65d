"""Pins for the CPU oracle: everything here is fixed by the definition or by
hand arithmetic, never by the oracle's own output or by the CUDA path."""
import numpy as np
import pytest

from oracle import qlinear_oracle as O

IMPLS = [pytest.param(O.linear, id="numpy"), pytest.param(O.linear_loops, id="c_loops")]


# ---------------------------------------------------------------- worked examples (tests/golden)
@pytest.mark.parametrize("linear", IMPLS)
def test_example_A_int8_per_channel(golden, linear):
    g = golden["A_int8_per_channel"]
    y64, A, y16 = linear(np.array(g["x"], np.float16), np.array(g["q"], np.int8),
                         np.array(g["s"], np.float16), g["group"])
    assert y64.tolist() == g["y64"]
    assert A.tolist() == g["A"]
    assert y16.astype(np.float64).tolist() == g["y64"]   # both values are fp16-representable


@pytest.mark.parametrize("linear", IMPLS)
def test_example_B_int4_group32(golden, linear):
    g = golden["B_int4_group32"]
    q = np.array([[(k % 16) - 8 for k in range(64)]], np.int8)
    s = np.array(g["s"], np.float16)
    xs = [np.ones((1, 64), np.float16),
          np.concatenate([np.ones(32), -np.ones(32)]).astype(np.float16)[None, :]]
    for x, case in zip(xs, g["cases"]):
        y64, A, _ = linear(x, q, s, 32)
        assert y64[0, 0] == case["y64"] and A[0, 0] == case["A"]
        # the same through the canonical nibble-byte interchange form
        y64b, _, _ = O.linear_from_nibbles(x, O.pack_nibbles(q), s, 32)
        assert y64b[0, 0] == case["y64"]


def test_example_C_nibble_bytes(golden):
    g = golden["C_nibble_bytes"]
    pairs = np.array(g["pairs"], np.int8)
    want = np.array([int(b, 16) for b in g["bytes"]], np.uint8)
    assert O.pack_nibbles(pairs).ravel().tolist() == want.tolist()
    assert O.unpack_nibbles(want[:, None]).tolist() == pairs.tolist()
    assert O.unpack_nibbles_loops(want[:, None]).tolist() == pairs.tolist()


@pytest.mark.parametrize("linear", IMPLS)
def test_examples_D_E_extremes_and_single_rounding(golden, linear):
    d, e = golden["D_extremes"], golden["E_single_rounding"]
    y64, _, y16 = linear(np.array([[d["x"]]], np.float16), np.array([[d["q"]]], np.int8),
                         np.array([[d["s"]]], np.float16), 0)
    assert y64[0, 0] == d["y64"] and float(y16[0, 0]) == d["y64"]
    s = np.array([[e["s_decimal"]]], np.float16)
    assert float(s[0, 0]) == e["s_fp16"]
    y64, _, y16 = linear(np.array([[e["x"]]], np.float16), np.array([[e["q"]]], np.int8), s, 0)
    assert y64[0, 0] == e["y64"] and float(y16[0, 0]) == e["y16"]


# ---------------------------------------------------------------- brute force on tiny inputs
def test_all_byte_values_unpack_by_definition():
    b = np.arange(256, dtype=np.uint8)[:, None]
    want = [[(v & 15) if (v & 15) < 8 else (v & 15) - 16, (v >> 4) if (v >> 4) < 8 else (v >> 4) - 16]
            for v in range(256)]
    assert O.unpack_nibbles(b).tolist() == want
    assert O.unpack_nibbles_loops(b).tolist() == want
    assert O.pack_nibbles(np.array(want, np.int8)).ravel().tolist() == list(range(256))


def test_pack_rejects_out_of_range():
    with pytest.raises(ValueError):
        O.pack_nibbles(np.array([[8, 0]], np.int8))
    with pytest.raises(ValueError):
        O.pack_nibbles(np.array([[-9, 0]], np.int8))


@pytest.mark.parametrize("linear", IMPLS)
def test_every_q_and_scale_exponent_single_term(linear):
    # N = 1, K = 32, only k0 carries weight: y must equal s * q * x[k0] computed by scalar Python.
    xs = np.zeros((1, 32), np.float16)
    xs[0, 5] = 1.5
    for e in range(-14, 4):
        s = np.array([[2.0 ** e * 1.25]], np.float16)
        for qv in range(-128, 128):
            q = np.zeros((1, 32), np.int8)
            q[0, 5] = qv
            y64, A, _ = linear(xs, q, s, 0)
            assert y64[0, 0] == float(s[0, 0]) * qv * 1.5
            assert A[0, 0] == abs(float(s[0, 0]) * qv * 1.5)


# ---------------------------------------------------------------- invariants
def _rand_case(rng, M, N, K, bits, group):
    lo, hi = (-8, 7) if bits == 4 else (-128, 127)
    q = rng.integers(lo, hi + 1, size=(N, K)).astype(np.int8)
    ng = 1 if group == 0 else K // group
    s = rng.uniform(1e-3, 1e-2, size=(N, ng)).astype(np.float16)
    x = rng.standard_normal((M, K)).astype(np.float16)
    return x, q, s


CASES = [(3, 8, 64, 4, 32), (2, 24, 96, 8, 0), (1, 16, 128, 4, 0), (5, 40, 160, 4, 32)]


@pytest.mark.parametrize("linear", IMPLS)
@pytest.mark.parametrize("M,N,K,bits,group", CASES)
def test_zero_input_gives_positive_zero(linear, M, N, K, bits, group):
    x, q, s = _rand_case(np.random.default_rng(1), M, N, K, bits, group)
    y64, A, y16 = linear(np.zeros_like(x), q, s, group)
    assert not y64.any() and not A.any()
    assert (y16.view(np.uint16) == 0).all()          # +0, not -0


@pytest.mark.parametrize("linear", IMPLS)
@pytest.mark.parametrize("M,N,K,bits,group", CASES)
def test_one_hot_returns_rounded_weight_column(linear, M, N, K, bits, group):
    rng = np.random.default_rng(2)
    _, q, s = _rand_case(rng, M, N, K, bits, group)
    G = K if group == 0 else group
    for k0 in (0, 1, G - 1, G % K, K - 1, int(rng.integers(K))):
        x = np.zeros((1, K), np.float16)
        x[0, k0] = 1.0
        y64, _, y16 = linear(x, q, s, group)
        col = s[:, k0 // G].astype(np.float64) * q[:, k0].astype(np.float64)   # one exact product
        assert (y64[0] == col).all()
        assert (y16[0].view(np.uint16) == col.astype(np.float16).view(np.uint16)).all()


@pytest.mark.parametrize("linear", IMPLS)
@pytest.mark.parametrize("M,N,K,bits,group", CASES)
def test_power_of_two_scaling_and_negation_are_exact(linear, M, N, K, bits, group):
    x, q, s = _rand_case(np.random.default_rng(3), M, N, K, bits, group)
    q = np.clip(q, -7 if bits == 4 else -127, None)
    y64, A, _ = linear(x, q, s, group)
    y2, A2, _ = linear((x.astype(np.float32) * 4).astype(np.float16), q, s, group)
    assert (y2 == 4 * y64).all() and (A2 == 4 * A).all()
    y3, _, _ = linear(x, q, (s.astype(np.float32) * 0.5).astype(np.float16), group)
    assert (y3 == 0.5 * y64).all()
    y4, A4, _ = linear(x, -q, s, group)
    assert (y4 == -y64).all() and (A4 == A).all()


@pytest.mark.parametrize("linear", IMPLS)
def test_all_ones_weights_closed_form(linear):
    rng = np.random.default_rng(4)
    K, N = 96, 8
    x = rng.integers(-8, 9, size=(2, K)).astype(np.float16)       # small integers: sums exact
    s = (2.0 ** rng.integers(-8, -2, size=(N, 1))).astype(np.float16)
    y64, _, _ = linear(x, np.ones((N, K), np.int8), s, 0)
    want = x.astype(np.float64).sum(axis=1)[:, None] * s.astype(np.float64).T
    assert (y64 == want).all()


@pytest.mark.parametrize("linear", IMPLS)
def test_group_boundaries_matter(linear):
    # scale of group g must apply to k in [32g, 32g+32) and to no other k
    K = 96
    q = np.ones((1, K), np.int8)
    s = np.array([[1.0, 2.0, 4.0]], np.float16)
    for k0 in range(K):
        x = np.zeros((1, K), np.float16)
        x[0, k0] = 1
        assert linear(x, q, s, 32)[0][0, 0] == [1.0, 2.0, 4.0][k0 // 32]


@pytest.mark.parametrize("linear", IMPLS)
def test_orientation_rows_are_output_channels(linear):
    # W is N x K: a non-square, asymmetric case where a transposed operand cannot pass
    q = np.array([[1, 2, 3, 4, 5, 6, 7, 8] * 4, [-1] * 32], np.int8)        # N=2, K=32
    s = np.array([[1.0], [0.5]], np.float16)
    x = np.zeros((3, 32), np.float16)
    x[0, 0] = 1; x[1, 1] = 1; x[2, :] = 1
    y64, _, _ = linear(x, q, s, 0)
    assert y64.shape == (3, 2)
    assert y64.tolist() == [[1.0, -0.5], [2.0, -0.5], [144.0, -16.0]]


@pytest.mark.parametrize("M,N,K,bits,group", CASES)
def test_permuting_k_within_groups_keeps_result(M, N, K, bits, group):
    rng = np.random.default_rng(5)
    x, q, s = _rand_case(rng, M, N, K, bits, group)
    G = K if group == 0 else group
    perm = np.concatenate([g * G + rng.permutation(G) for g in range(K // G)])
    y, A, _ = O.linear_loops(x, q, s, group)
    yp, Ap, _ = O.linear_loops(x[:, perm], q[:, perm], s, group)
    assert np.abs(yp - y).max() <= 1e-13 * A.max()


# ---------------------------------------------------------------- reduction to library routines
@pytest.mark.parametrize("M,N,K,bits,group", CASES + [(4, 48, 2304, 8, 0), (2, 32, 1024, 4, 32)])
def test_loops_agree_with_library_matmul(M, N, K, bits, group):
    import torch
    x, q, s = _rand_case(np.random.default_rng(6), M, N, K, bits, group)
    y_np, A_np, y16_np = O.linear(x, q, s, group)
    y_c, A_c, y16_c = O.linear_loops(x, q, s, group)
    assert np.abs(y_np - y_c).max() <= 1e-12 * A_c.max()
    assert np.abs(A_np - A_c).max() <= 1e-12 * A_c.max()
    w = O.dequantize(q, s, group)
    assert (w == O.dequantize_loops(q, s, group)).all()                    # products are exact
    y_t = (torch.from_numpy(x.astype(np.float64)) @ torch.from_numpy(w).T).numpy()
    assert np.abs(y_t - y_c).max() <= 1e-12 * A_c.max()
    # the two fp16 roundings may differ only where y64 differs, i.e. almost never
    assert (y16_np.view(np.uint16) != y16_c.view(np.uint16)).mean() < 0.01


# ---------------------------------------------------------------- fp16 conversions of the C oracle
def test_c_fp16_decode_all_patterns():
    L = O.c_lib()
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    want = bits.view(np.float16).astype(np.float64)
    got = np.array([L.oracle_fp16_to_double(int(b)) for b in bits])
    finite = np.isfinite(want)
    assert (got[finite] == want[finite]).all()
    assert (np.isnan(got) == np.isnan(want)).all() and (np.isinf(got) == np.isinf(want)).all()
    assert (np.signbit(got) == np.signbit(want))[~np.isnan(want)].all()


def test_c_fp16_encode_exact_values_midpoints_and_double_rounding_trap():
    L = O.c_lib()
    enc = lambda v: int(L.oracle_double_to_fp16(float(v)))
    bits = np.arange(0x7C00, dtype=np.uint16)               # all finite non-negative fp16
    vals = bits.view(np.float16).astype(np.float64)
    for b, v in zip(bits[::7], vals[::7]):                  # exact values map to themselves
        assert enc(v) == int(b) and enc(-v) == (int(b) | 0x8000)
    for i in range(0, len(vals) - 1, 11):                   # midpoints go to the even neighbour
        mid = 0.5 * (vals[i] + vals[i + 1])
        assert enc(mid) == (int(bits[i]) if bits[i] % 2 == 0 else int(bits[i + 1]))
        assert enc(np.nextafter(mid, np.inf)) == int(bits[i + 1])
        assert enc(np.nextafter(mid, -np.inf)) == int(bits[i])
    assert enc(65519.999) == 0x7BFF and enc(65520.0) == 0x7C00 and enc(1e9) == 0x7C00
    assert enc(2.0 ** -25) == 0 and enc(np.nextafter(2.0 ** -25, 1)) == 1   # tie to even at half the least subnormal
    # rounding through fp32 first would give 1.0 here (fp32 lands on the tie); one rounding gives 1 + 2^-10
    trap = 1.0 + 2.0 ** -11 + 2.0 ** -30
    assert enc(trap) == 0x3C01
    assert np.float64(trap).astype(np.float16).view(np.uint16) == 0x3C01    # numpy path too
    rng = np.random.default_rng(7)
    r = rng.standard_normal(4000) * 10.0 ** rng.integers(-6, 5, size=4000)
    assert [enc(v) for v in r] == r.astype(np.float16).view(np.uint16).tolist()


# ---------------------------------------------------------------- the tolerance itself
def test_fp32_accumulation_sits_inside_the_error_bound():
    # fp16-rounded dequantised weights, fp32 accumulation, fp16 output: the arithmetic the GPU
    # path is allowed.  Its error must sit inside K*2^-24 + 2*2^-11 relative to A, which in turn
    # is inside the 5e-3 acceptance bound for every K of the workloads.
    rng = np.random.default_rng(8)
    for K, bits, group in [(14336, 4, 32), (9216, 4, 32), (4096, 8, 0)]:
        x, q, s = _rand_case(rng, 2, 24, K, bits, group)
        y64, A, _ = O.linear(x, q, s, group)
        w16 = O.dequantize(q, s, group).astype(np.float16).astype(np.float32)
        acc = np.zeros((2, 24), np.float32)
        xf = x.astype(np.float32)
        for k in range(K):
            acc += xf[:, k:k + 1] * w16[None, :, k]
        y = acc.astype(np.float16)
        bound = K * 2.0 ** -24 + 2 * 2.0 ** -11
        assert bound < O.ELEM_TOL
        ok, rel, worst = O.check_against(y, y64, A)
        assert ok and worst <= bound and rel <= O.REL_L2_TOL


def test_check_against_flags_errors():
    y64 = np.array([[1.0, -2.0]])
    A = np.array([[1.0, 2.0]])
    assert O.check_against(y64.astype(np.float16), y64, A)[0]
    assert not O.check_against(np.array([[1.01, -2.0]]), y64, A)[0]     # 1e-2 * A
    assert not O.check_against(np.array([[1.0, 2.0]]), y64, A)[0]       # sign flip
