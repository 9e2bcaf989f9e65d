"""Pins of the oracle's three extensions: fused gating (paper Section 3.6), int8 activation quantisation
(Section 3.7) and the KV cache held as weights (Section 3.8).  CPU only.  Each pin checks the oracle against
something other than itself: hand-computed examples (tests/golden), closed forms and identities of the
activations, a library routine, brute force in plain Python integers, or the special case in which the
extension must fall back onto the plain linear layer."""
import math

import numpy as np
import pytest

from oracle import qlinear_oracle as O
from workloads import configs as C


def rand_layer(seed, N, K, bits, group):
    layer = C.LayerSpec("t", N, K, bits, group, *((-8, 7) if bits == 4 else (-128, 127)))
    return C.layer_weights(seed, layer)


# ----------------------------------------------------------------------------- fused gating
def test_example_F_gated_silu(golden):
    e = golden["F_gated_silu"]
    x = np.array(e["x"], np.float16)
    y64, bound, y16 = O.gated_linear(x, np.array(e["q_gate"], np.int8), np.array(e["s_gate"], np.float16),
                                     np.array(e["q_up"], np.int8), np.array(e["s_up"], np.float16), e["group"], "silu")
    np.testing.assert_allclose(y64, np.array(e["y64"]), rtol=1e-15, atol=0)
    assert (bound > 0).all()
    assert (y16 == y64.astype(np.float16)).all()


@pytest.mark.parametrize("act", ["silu", "gelu_tanh"])
def test_activation_identities_and_closed_values(act):
    g = np.linspace(-12, 12, 4801)
    a = O.activation(g, act)
    np.testing.assert_allclose(a - O.activation(-g, act), g, rtol=0, atol=1e-14)     # act(g) - act(-g) = g for both
    assert O.activation(np.array([0.0]), act)[0] == 0.0
    assert abs(O.activation(np.array([30.0]), act)[0] - 30.0) < 1e-10               # identity far to the right
    assert abs(O.activation(np.array([-30.0]), act)[0]) < 1e-10                     # zero far to the left
    if act == "silu":
        assert abs(O.activation(np.array([math.log(3.0)]), act)[0] - 0.75 * math.log(3.0)) < 1e-15   # sigmoid(ln 3) = 3/4
    # the slope bound used in the acceptance bound is the true maximum slope, to three digits
    slope = np.abs(np.diff(O.activation(np.linspace(-8, 8, 1_600_001), act)) / 1e-5)
    assert O.ACT_LIPSCHITZ[act] - 2e-3 < slope.max() <= O.ACT_LIPSCHITZ[act]


def test_activations_agree_with_library_routines():
    torch = pytest.importorskip("torch")
    g = np.linspace(-9, 9, 2001)
    t = torch.from_numpy(g)
    np.testing.assert_allclose(O.activation(g, "silu"), torch.nn.functional.silu(t).numpy(), rtol=1e-14, atol=1e-16)
    np.testing.assert_allclose(O.activation(g, "gelu_tanh"), torch.nn.functional.gelu(t, approximate="tanh").numpy(), rtol=1e-13, atol=2e-15)   # 1 + tanh cancels far to the left


@pytest.mark.parametrize("bits,group", [(8, 0), (4, 32), (4, 0)])
def test_gated_identity_is_the_product_of_two_linear_calls_and_branches_are_not_swapped(bits, group):
    qg, sg = rand_layer(11, 24, 128, bits, group)
    qu, su = rand_layer(12, 24, 128, bits, group)
    x = C.layer_activations(13, C.LayerSpec("t", 24, 128, bits, group, 0, 0), 3)
    g64, _, _ = O.linear(x, qg, sg, group)
    u64, _, _ = O.linear(x, qu, su, group)
    y64, _, _ = O.gated_linear(x, qg, sg, qu, su, group, "identity")
    assert (y64 == g64 * u64).all()
    ys, _, _ = O.gated_linear(x, qg, sg, qu, su, group, "silu")
    yt, _, _ = O.gated_linear(x, qu, su, qg, sg, group, "silu")                   # branches swapped: a different function
    np.testing.assert_allclose(ys, g64 / (1 + np.exp(-g64)) * u64, rtol=1e-15)
    np.testing.assert_allclose(yt, u64 / (1 + np.exp(-u64)) * g64, rtol=1e-15)
    assert np.abs(ys - yt).max() > 1e-3


def test_gated_bound_holds_for_an_fp32_emulation_of_the_fused_kernel():
    """fp16-rounded grouped weights, fp32 accumulation of both branches, fp32 activation, one fp16 rounding."""
    K, N, M = 4096, 48, 4
    qg, sg = rand_layer(21, N, K, 4, 32)
    qu, su = rand_layer(22, N, K, 4, 32)
    x = C.layer_activations(23, C.LayerSpec("t", N, K, 4, 32, 0, 0), M)
    def branch32(q, s):
        w16 = (np.repeat(s.astype(np.float32), 32, axis=1) * q.astype(np.float32)).astype(np.float16).astype(np.float32)
        acc = np.zeros((M, N), np.float32)
        for k0 in range(0, K, 64):
            acc = (acc + x[:, k0:k0 + 64].astype(np.float32) @ w16[:, k0:k0 + 64].T).astype(np.float32)
        return acc
    g32, u32 = branch32(qg, sg), branch32(qu, su)
    y = ((g32 / (np.float32(1) + np.exp(-g32))) * u32).astype(np.float16)
    y64, bound, _ = O.gated_linear(x, qg, sg, qu, su, 32, "silu")
    ok, rel, worst = O.check_gated(y, y64, bound)
    assert ok and rel < 6e-4 and worst < 0.5, (rel, worst)
    bad = y.copy()
    bad[1, 5] = np.float16(float(bad[1, 5]) + 3 * float(bound[1, 5]) + 1e-3)
    assert not O.check_gated(bad, y64, bound)[0]


# ----------------------------------------------------------------------------- activation quantisation
def test_example_G_activation_quantisation(golden):
    e = golden["G_act_quant"]
    x = np.array(e["x"], np.float16)
    xq, sx = O.quantize_activations(x)
    assert xq.tolist() == e["xq"] and sx.tolist() == e["scale_x"]
    y64, acc, _, _, _ = O.linear_int8_activations(x, np.array(e["q"], np.int8), np.array(e["s"], np.float16), 0)
    assert acc.tolist() == e["acc"] and y64.tolist() == e["y64"]


def test_quantisation_rounds_half_to_even_clamps_and_handles_zero_rows():
    # amax = 127 * 2^-3 makes r = 8 exactly: x * 8 is exact, ties are real ties
    x = np.array([[127 / 8, 0.5 / 8, 1.5 / 8, 2.5 / 8, -0.5 / 8, -1.5 / 8, -126.5 / 8, 63.5 / 8],
                  [0, 0, 0, 0, 0, 0, 0, 0],
                  [-3.0, 1.0, 0.0, 3.0, 2.9, -2.9, 0.01, -0.01]], np.float16)
    assert all(float(v) * 8 == round(float(v) * 8 * 2) / 2 for v in x[0])           # the fixture is exact in fp16
    xq, sx = O.quantize_activations(x)
    assert xq[0].tolist() == [127, 0, 2, 2, 0, -2, -126, 64]
    assert sx[0] == np.float32(1 / 8) and sx[1] == np.float32(1.0) and not xq[1].any()
    assert xq[2, 0] == -127 and xq[2, 3] == 127 and np.abs(xq).max() == 127         # the largest magnitude maps to +-127
    # reconstruction error is at most half a step (plus fp32 round-off of the two operations)
    err = np.abs(x.astype(np.float64) - sx.astype(np.float64)[:, None] * xq)
    assert (err <= 0.5 * sx.astype(np.float64)[:, None] * (1 + 1e-6)).all()


@pytest.mark.parametrize("bits,group", [(8, 0), (4, 32), (4, 0), (4, 64)])
def test_activations_on_the_int8_grid_give_the_fp16_activation_result_exactly(bits, group):
    """If x is already scale * integer with |integer| <= 127 and the largest equal to 127, quantisation loses
    nothing: the integer path must equal the plain linear layer's fp64 result exactly."""
    N, K, M = 40, 256, 3
    q, s = rand_layer(31, N, K, bits, group)
    rng = np.random.default_rng(5)
    ints = rng.integers(-127, 128, size=(M, K))
    ints[:, 0] = 127
    x = (ints * np.array([[2.0 ** -4], [2.0 ** -7], [2.0 ** 0]])).astype(np.float16)
    y64, acc, xq, sx, _ = O.linear_int8_activations(x, q, s, group)
    assert (xq == ints).all()
    assert sx.tolist() == [2.0 ** -4, 2.0 ** -7, 1.0]
    y_ref, _, _ = O.linear(x, q, s, group)
    np.testing.assert_allclose(y64, y_ref, rtol=1e-13, atol=0)                      # same real number, fp64 summation order differs


def test_integer_dot_products_are_exact_against_python_integers():
    N, K, M, G = 5, 64, 2, 32
    q, s = rand_layer(41, N, K, 4, G)
    x = C.layer_activations(42, C.LayerSpec("t", N, K, 4, G, 0, 0), M)
    y64, acc, xq, sx, _ = O.linear_int8_activations(x, q, s, G)
    for m in range(M):
        for n in range(N):
            total = 0.0
            for g in range(K // G):
                a = sum(int(xq[m, k]) * int(q[n, k]) for k in range(g * G, (g + 1) * G))
                assert a == int(acc[m, n, g])
                total += float(s[n, g]) * a
            assert abs(y64[m, n] - float(sx[m]) * total) <= 1e-12 * abs(y64[m, n]) + 1e-300


def test_quantised_result_stays_close_to_the_unquantised_layer():
    """A sign error, a dropped scale or a wrong group index would move the result by far more than int8 noise."""
    N, K, M = 64, 2048, 4
    q, s = rand_layer(51, N, K, 4, 32)
    x = C.layer_activations(52, C.LayerSpec("t", N, K, 4, 32, 0, 0), M)
    y64, _, _, _, _ = O.linear_int8_activations(x, q, s, 32)
    y_ref, _, _ = O.linear(x, q, s, 32)
    rel = np.linalg.norm(y64 - y_ref) / np.linalg.norm(y_ref)
    assert 1e-4 < rel < 3e-2, rel


# ----------------------------------------------------------------------------- KV cache as weights
def test_example_H_kv_cache_orientation(golden):
    e = golden["H_kv_cache"]
    sc, _, _ = O.kv_scores(np.array(e["qry"], np.float16), np.array(e["k_q"], np.int8), np.array(e["k_s"], np.float16))
    assert sc.tolist() == e["scores64"]
    out, _, _ = O.kv_output(np.array(e["prob"], np.float16), np.array(e["v_q"], np.int8), np.array(e["v_s"], np.float16))
    assert out.tolist() == e["out64"]


def test_kv_products_against_plain_loops():
    rng = np.random.default_rng(9)
    T, d, R = 37, 16, 3
    k_q = rng.integers(-128, 128, size=(T, d)).astype(np.int8)
    k_s = rng.uniform(1e-3, 1e-2, size=T).astype(np.float16)
    v_q = rng.integers(-128, 128, size=(d, T)).astype(np.int8)
    v_s = rng.uniform(1e-3, 1e-2, size=d).astype(np.float16)
    qry = rng.standard_normal((R, d)).astype(np.float16)
    prob = rng.uniform(0, 1, size=(R, T)).astype(np.float16)
    sc, _, _ = O.kv_scores(qry, k_q, k_s)
    out, _, _ = O.kv_output(prob, v_q, v_s)
    for r in range(R):
        for t in range(T):                                   # one score per cached key: O = cache positions
            want = sum(float(qry[r, j]) * float(k_s[t]) * int(k_q[t, j]) for j in range(d))
            assert abs(sc[r, t] - want) <= 1e-12 * max(1.0, abs(want))
        for j in range(d):                                   # one output per head dimension: O = d_h, I = cache positions
            want = sum(float(prob[r, t]) * float(v_s[j]) * int(v_q[j, t]) for t in range(T))
            assert abs(out[r, j] - want) <= 1e-12 * max(1.0, abs(want))


def test_kv_row_quantisation_hand_cases():
    # row 0: amax = 127 / 64 exactly, so s = 1/64 and every quotient is exact; -0.5/64 * 64 = -0.5 is a tie (to even: -0)
    # row 1: all zeros -> zeros with scale 1
    # row 2: amax = 1: s = fp16(1/127) = 0.00787353515625 (rounded DOWN), 1 / s = 127.0078 -> 127
    # row 3: a scale in fp16's subnormal range: 1.4 * 2^-24 rounds to 2^-24, the quotient 177.8 is clamped to 127
    rows = np.zeros((4, 4), np.float64)
    rows[0] = [127 / 64, -63.5 / 64, 0.5 / 64, 2.5 / 64]
    rows[2] = [1.0, -0.5, 0.25, 0.004]
    rows[3] = [127 * 1.4 * 2.0 ** -24, 2.0 ** -24, 0, 0]
    a = rows.astype(np.float16)
    q, s = O.kv_quantize_rows(a)
    assert s[0] == np.float16(1 / 64) and q[0].tolist() == [127, -64, 0, 2]
    assert s[1] == np.float16(1.0) and not q[1].any()
    assert float(s[2]) == 0.00787353515625 and q[2].tolist() == [127, -64, 32, 1]
    assert float(s[3]) == 2.0 ** -24 and q[3, 0] == 127 and q[3, 1] == 1
    assert np.abs(q).max() <= 127


def test_kv_attention_matches_a_plain_float_attention_closely_and_exactly_on_the_grid():
    rng = np.random.default_rng(17)
    T, d, R = 96, 32, 4
    k = rng.standard_normal((T, d)).astype(np.float16)
    v = rng.standard_normal((T, d)).astype(np.float16)
    qry = rng.standard_normal((R, d)).astype(np.float16)
    prob = rng.uniform(0, 1, size=(R, T)).astype(np.float16)
    sc64, _, out64, _ = O.kv_attention(qry, k, v, prob)
    sc_ref = qry.astype(np.float64) @ k.astype(np.float64).T
    out_ref = prob.astype(np.float64) @ v.astype(np.float64)
    assert np.linalg.norm(sc64 - sc_ref) / np.linalg.norm(sc_ref) < 1e-2          # int8 noise, nothing structural
    assert np.linalg.norm(out64 - out_ref) / np.linalg.norm(out_ref) < 1e-2
    # keys and values already on an int8 grid with power-of-two scales, probabilities that are powers of two:
    # every step is exact, so the result equals plain fp64 attention
    ki = rng.integers(-127, 128, size=(T, d)); ki[:, 0] = 127
    vi = rng.integers(-127, 128, size=(T, d)); vi[:, 0] = -127
    kg = (ki * 2.0 ** -5).astype(np.float16)
    vg = (vi * 2.0 ** -6).astype(np.float16)
    pg = (2.0 ** -rng.integers(1, 6, size=(R, T))).astype(np.float16)
    sc64, _, out64, _ = O.kv_attention(qry, kg, vg, pg)
    np.testing.assert_allclose(sc64, qry.astype(np.float64) @ kg.astype(np.float64).T, rtol=1e-13, atol=1e-12)
    np.testing.assert_allclose(out64, pg.astype(np.float64) @ vg.astype(np.float64), rtol=1e-13, atol=1e-12)


# ----------------------------------------------------------------------------- residual + RMS normalisation
def test_example_I_residual_rmsnorm(golden):
    e = golden["I_residual_rmsnorm"]
    h64, h16, y64, y16 = O.residual_rmsnorm(np.array(e["x"], np.float16), np.array(e["r"], np.float16),
                                            np.array(e["g"], np.float16), e["eps"], e["offset"])
    assert (h64 == np.array(e["h64"])).all() and (y64 == np.array(e["y64"])).all()       # exact: powers of two throughout
    assert (h16 == h64).all() and (y16 == y64).all()


def test_rmsnorm_against_plain_loops_and_the_library_routine():
    import torch
    rng = np.random.default_rng(5)
    M, K = 7, 96
    x = rng.standard_normal((M, K)).astype(np.float16)
    r = (3 * rng.standard_normal((M, K))).astype(np.float16)
    g = rng.standard_normal(K).astype(np.float16)
    eps, off = 1e-5, 1.0
    h64, _, y64, _ = O.residual_rmsnorm(x, r, g, eps, off)
    for m in range(M):                                                   # the definition written out with Python floats
        h = [float(x[m, k]) + float(r[m, k]) for k in range(K)]
        ms = math.fsum(v * v for v in h) / K
        for k in range(K):
            assert h64[m, k] == h[k]
            assert y64[m, k] == pytest.approx(h[k] / math.sqrt(ms + eps) * (off + float(g[k])), rel=1e-14, abs=0)
    # special case the library has: no residual, offset 0
    _, _, y0, _ = O.residual_rmsnorm(x, None, g, eps, 0.0)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x.astype(np.float64)), (K,), torch.from_numpy(g.astype(np.float64)), eps)
    np.testing.assert_allclose(y0, ref.numpy(), rtol=1e-13, atol=0)


def test_rmsnorm_invariants():
    rng = np.random.default_rng(6)
    M, K = 5, 64
    x = rng.standard_normal((M, K)).astype(np.float16)
    r = rng.standard_normal((M, K)).astype(np.float16)
    g = (1 + rng.standard_normal(K) / 4).astype(np.float16)
    # without eps the output does not change when the input is scaled (power of two: exact); the sign follows
    _, _, y1, _ = O.residual_rmsnorm(x, r, g, 0.0)
    _, _, y2, _ = O.residual_rmsnorm((x * np.float16(-4)).astype(np.float16), (r * np.float16(-4)).astype(np.float16), g, 0.0)
    np.testing.assert_allclose(y2, -y1, rtol=1e-15, atol=0)
    # mean of (y / scale)^2 is ms / (ms + eps)
    eps = 0.37
    h64, _, y, _ = O.residual_rmsnorm(x, r, g, eps)
    ms = (h64 ** 2).mean(axis=1)
    np.testing.assert_allclose(((y / g.astype(np.float64)) ** 2).mean(axis=1), ms / (ms + eps), rtol=1e-13)
    # the residual branch is a plain sum: the two inputs commute, and no residual is a residual of zeros
    a = O.residual_rmsnorm(x, r, g, eps, 1.0)
    b = O.residual_rmsnorm(r, x, g, eps, 1.0)
    assert all((u == v).all() for u, v in zip(a, b))
    c = O.residual_rmsnorm(x, None, g, eps)
    d = O.residual_rmsnorm(x, np.zeros_like(x), g, eps)
    assert all((u == v).all() for u, v in zip(c, d))
    # a constant row comes out as +-scale (eps = 0), whatever the constant
    _, _, yc, _ = O.residual_rmsnorm(np.full((1, K), -3.0, np.float16), None, g, 0.0)
    np.testing.assert_allclose(yc[0], -g.astype(np.float64), rtol=1e-15)


def test_rmsnorm_bound_holds_for_an_fp32_emulation():
    rng = np.random.default_rng(8)
    M, K = 16, 4096
    x = (2 * rng.standard_normal((M, K))).astype(np.float16)
    r = (8 * rng.standard_normal((M, K))).astype(np.float16)
    g = rng.standard_normal(K).astype(np.float16)
    eps = 1e-6
    h64, _, y64, _ = O.residual_rmsnorm(x, r, g, eps, 0.0)
    bh, by = O.residual_rmsnorm_bound(h64, y64, K)
    h32 = x.astype(np.float32) + r.astype(np.float32)
    part = np.zeros((M, 128), np.float32)                                # 128 partial sums, then pairwise
    for k0 in range(0, K, 128):
        part = (part + h32[:, k0:k0 + 128] * h32[:, k0:k0 + 128]).astype(np.float32)
    while part.shape[1] > 1:
        part = (part[:, 0::2] + part[:, 1::2]).astype(np.float32)
    ss = part[:, 0]
    rstd = (np.float32(1) / np.sqrt((ss / np.float32(K) + np.float32(eps)).astype(np.float32))).astype(np.float32)
    y32 = ((h32 * rstd[:, None]).astype(np.float32) * g.astype(np.float32)[None, :]).astype(np.float32)
    assert (np.abs(h32.astype(np.float16).astype(np.float64) - h64) <= bh).all()
    assert (np.abs(y32.astype(np.float16).astype(np.float64) - y64) <= by).all()
    # and a wrong divisor (mean over K - 1) is caught where 1 / (2 K) exceeds an fp16 rounding
    K2 = 64
    h2, _, y2, _ = O.residual_rmsnorm(x[:, :K2], r[:, :K2], g[:K2], eps, 0.0)
    _, by2 = O.residual_rmsnorm_bound(h2, y2, K2)
    assert (np.abs(y2 * np.sqrt(K2 / (K2 - 1.0)) - y2) > by2).any()


# ----------------------------------------------------------------------------- rotary embedding + QKV layout
def test_example_J_rope_qkv(golden):
    e = golden["J_rope_qkv"]
    qo, ko, vo, _, _ = O.rope_qkv(np.array(e["q"], np.float16), np.array(e["k"], np.float16), np.array(e["v"], np.float16),
                                  np.array(e["pos"]), np.array(e["cos"], np.float32), np.array(e["sin"], np.float32),
                                  e["B"], e["S"], e["h_q"], e["h_kv"], e["d_h"])
    assert (qo == np.array(e["q_out"])).all() and (ko == np.array(e["k_out"])).all() and (vo == np.array(e["v_out"])).all()


def _rope_case(seed, B, S, h_q, h_kv, d_h, n_pos=64):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((B * S, h_q * d_h)).astype(np.float16)
    k = rng.standard_normal((B * S, h_kv * d_h)).astype(np.float16)
    v = rng.standard_normal((B * S, h_kv * d_h)).astype(np.float16)
    pos = rng.integers(0, n_pos, size=B * S)
    inv = 10000.0 ** (-np.arange(d_h // 2) * 2.0 / d_h)
    ang = np.arange(n_pos)[:, None] * inv[None, :]
    return q, k, v, pos, np.cos(ang).astype(np.float32), np.sin(ang).astype(np.float32)


def test_rope_layout_is_the_stated_index_map_and_v_is_only_moved():
    B, S, h_q, h_kv, d_h = 2, 3, 6, 2, 4
    g = h_q // h_kv
    q, k, v, pos, cos, sin = _rope_case(1, B, S, h_q, h_kv, d_h)
    one, zero = np.ones_like(cos), np.zeros_like(sin)                    # angle 0 everywhere: the pure layout transform
    qo, ko, vo, _, _ = O.rope_qkv(q, k, v, pos, one, zero, B, S, h_q, h_kv, d_h)
    for b in range(B):
        for s in range(S):
            for hk in range(h_kv):
                assert (ko[b * h_kv + hk, s] == k[b * S + s, hk * d_h:(hk + 1) * d_h]).all()
                assert (vo[b * h_kv + hk, s] == v[b * S + s, hk * d_h:(hk + 1) * d_h]).all()
                for j in range(g):
                    hq = hk * g + j
                    assert (qo[b * h_kv + hk, s * g + j] == q[b * S + s, hq * d_h:(hq + 1) * d_h]).all()
    _, _, vo2, _, _ = O.rope_qkv(q, k, v, pos, cos, sin, B, S, h_q, h_kv, d_h)
    assert (vo2 == vo).all()                                             # V is never rotated


def test_rope_is_the_complex_product_and_plain_loops():
    B, S, h_q, h_kv, d_h = 1, 5, 4, 2, 8
    half = d_h // 2
    q, k, v, pos, cos, sin = _rope_case(2, B, S, h_q, h_kv, d_h)
    qo, ko, _, aq, _ = O.rope_qkv(q, k, v, pos, cos, sin, B, S, h_q, h_kv, d_h)
    g = h_q // h_kv
    for s in range(S):
        c, sn = cos[pos[s]].astype(np.float64), sin[pos[s]].astype(np.float64)
        for hq in range(h_q):
            x = q[s, hq * d_h:(hq + 1) * d_h].astype(np.float64)
            z = (x[:half] + 1j * x[half:]) * (c + 1j * sn)               # the library's complex multiplication
            row = qo[hq // g, s * g + hq % g]
            np.testing.assert_allclose(row[:half], z.real, rtol=1e-15, atol=1e-300)
            np.testing.assert_allclose(row[half:], z.imag, rtol=1e-15, atol=1e-300)
            for i in range(half):                                        # and written out element by element
                assert row[i] == x[i] * c[i] - x[i + half] * sn[i]
                assert row[i + half] == x[i + half] * c[i] + x[i] * sn[i]
                assert aq[hq // g, s * g + hq % g, i] == abs(x[i]) + abs(x[i + half])


def test_rope_invariants():
    B, S, h_q, h_kv, d_h = 1, 4, 2, 2, 16
    half = d_h // 2
    q, k, v, pos, cos, sin = _rope_case(3, B, S, h_q, h_kv, d_h)
    qo, ko, _, _, _ = O.rope_qkv(q, k, v, pos, cos, sin, B, S, h_q, h_kv, d_h)
    # a rotation keeps the length of every (i, i + d/2) pair (up to the rounding of the fp32 tables)
    x = k.astype(np.float64).reshape(S, h_kv, d_h).transpose(1, 0, 2)
    np.testing.assert_allclose(ko[:, :, :half] ** 2 + ko[:, :, half:] ** 2, x[:, :, :half] ** 2 + x[:, :, half:] ** 2, rtol=1e-6)
    # the score of a query and a key depends on the DIFFERENCE of their positions only: shift all positions by 7
    qo2, ko2, _, _, _ = O.rope_qkv(q, k, v, pos + 7, *_rope_case(3, B, S, h_q, h_kv, d_h, 80)[4:], B, S, h_q, h_kv, d_h)
    np.testing.assert_allclose(np.einsum("hsd,htd->hst", qo2, ko2), np.einsum("hsd,htd->hst", qo, ko), rtol=0, atol=2e-5)
    # the opposite sign of the sine table undoes the rotation
    back = O.rope_qkv(np.zeros_like(q), ko.transpose(1, 0, 2).reshape(S, h_kv * d_h).astype(np.float16), v, pos, cos, -sin, B, S, h_q, h_kv, d_h)[1]
    np.testing.assert_allclose(back.transpose(1, 0, 2).reshape(S, h_kv * d_h), k.astype(np.float64), rtol=0, atol=4e-3)
