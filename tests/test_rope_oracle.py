"""CPU pins of the rotary-prologue oracle: each test fixes it to something other than its own
formula (textbook constants, closed forms, RoFormer's relative-position property that Appendix B
builds on, layout one-hots, the adjoint identity for the backward)."""
import numpy as np
import pytest

from oracle import rope_oracle as ro

COS1, SIN1 = 0.5403023058681398, 0.8414709848078965  # cos(1), sin(1)


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape)


def test_position_zero_is_identity_and_v_is_copied():
    T, Hq, Hkv, D = 5, 4, 2, 8
    qkv = _rand((T, (Hq + 2 * Hkv) * D), 1)
    Q, K, V = ro.rope_qkv_fwd(qkv, np.zeros(T, int), np.zeros(T, int), Hq, Hkv, D, 500000.0)
    assert np.array_equal(Q.reshape(T, -1), qkv[:, : Hq * D])
    assert np.array_equal(K.reshape(T, -1), qkv[:, Hq * D : (Hq + Hkv) * D])
    assert np.array_equal(V.reshape(T, -1), qkv[:, (Hq + Hkv) * D :])


def test_two_dimensional_head_is_a_plane_rotation_by_p_radians():
    # D = 2: one pair, base ** 0 = 1, so the angle is p itself
    qkv = np.array([[1.0, 0.0, 0.0, 1.0, 7.0, 9.0]])  # q = e0, k = e1, v
    Q, K, V = ro.rope_qkv_fwd(qkv, [1], [0], 1, 1, 2, 12345.0)
    np.testing.assert_allclose(Q[0, 0], [COS1, SIN1], atol=1e-15)
    np.testing.assert_allclose(K[0, 0], [-SIN1, COS1], atol=1e-15)
    np.testing.assert_array_equal(V[0, 0], [7.0, 9.0])


def test_frequency_of_the_second_pair():
    # D = 4, base 10000: pair 1 turns at base ** (-2/4) = 0.01 rad per position; at p = 100, 1 rad
    x = np.zeros((1, 4 * 3))
    x[0, 1] = 1.0  # q, element 1 (pairs with element 3)
    Q, _, _ = ro.rope_qkv_fwd(x, [60], [40], 1, 1, 4, 10000.0)
    np.testing.assert_allclose(Q[0, 0], [0.0, COS1, 0.0, SIN1], atol=1e-13)


def test_pairing_is_half_split_not_interleaved():
    x = np.zeros((1, 8 * 3))
    x[0, 0] = 1.0
    Q, _, _ = ro.rope_qkv_fwd(x, [3], [0], 1, 1, 8, 500000.0)
    assert Q[0, 0, 0] != 0.0 and Q[0, 0, 4] != 0.0
    assert np.count_nonzero(Q[0, 0]) == 2


def test_position_is_anchor_plus_depth():
    T, Hq, Hkv, D = 2, 2, 1, 16
    row = _rand((1, (Hq + 2 * Hkv) * D), 2)
    qkv = np.repeat(row, 2, axis=0)
    Q, K, _ = ro.rope_qkv_fwd(qkv, [3, 5], [2, 0], Hq, Hkv, D, 500000.0)
    np.testing.assert_array_equal(Q[0], Q[1])
    np.testing.assert_array_equal(K[0], K[1])


def test_rotation_preserves_pair_norms():
    T, Hq, Hkv, D = 7, 3, 1, 32
    qkv = _rand((T, (Hq + 2 * Hkv) * D), 3)
    a = np.arange(T) * 1000
    Q, _, _ = ro.rope_qkv_fwd(qkv, a, np.arange(T) % 4, Hq, Hkv, D, 500000.0)
    q0 = qkv[:, : Hq * D].reshape(T, Hq, D)
    n0 = q0[..., : D // 2] ** 2 + q0[..., D // 2 :] ** 2
    n1 = Q[..., : D // 2] ** 2 + Q[..., D // 2 :] ** 2
    np.testing.assert_allclose(n1, n0, rtol=1e-12)


def test_score_depends_on_the_position_difference_only():
    # <R_p q, R_p' k> = <R_{p - p'} q, k>: the property Appendix B starts from
    D, base = 64, 500000.0
    q, k = _rand((1, 1, D), 4), _rand((1, 1, D), 5)
    for p, pk in ((17, 5), (4096, 4000), (20000, 19999)):
        lhs = np.sum(ro.rotate(q, ro.rope_angles([p], D, base)) * ro.rotate(k, ro.rope_angles([pk], D, base)))
        rhs = np.sum(ro.rotate(q, ro.rope_angles([p - pk], D, base)) * k)
        shifted = np.sum(ro.rotate(q, ro.rope_angles([p + 123], D, base)) *
                         ro.rotate(k, ro.rope_angles([pk + 123], D, base)))
        assert lhs == pytest.approx(rhs, rel=1e-9, abs=1e-9)
        assert lhs == pytest.approx(shifted, rel=1e-9, abs=1e-9)


def test_rotations_compose_additively():
    D, base = 16, 500000.0
    x = _rand((1, 2, D), 6)
    twice = ro.rotate(ro.rotate(x, ro.rope_angles([30], D, base)), ro.rope_angles([12], D, base))
    once = ro.rotate(x, ro.rope_angles([42], D, base))
    np.testing.assert_allclose(twice, once, atol=1e-12)


def test_layout_of_the_fused_row():
    T, Hq, Hkv, D = 1, 3, 2, 4
    width = (Hq + 2 * Hkv) * D
    for col in range(width):
        x = np.zeros((T, width))
        x[0, col] = 1.0
        Q, K, V = ro.rope_qkv_fwd(x, [0], [0], Hq, Hkv, D, 500000.0)
        flat = np.concatenate([Q.reshape(-1), K.reshape(-1), V.reshape(-1)])
        assert flat[col] == 1.0 and np.count_nonzero(flat) == 1


def test_backward_is_the_adjoint_of_the_forward():
    T, Hq, Hkv, D, base = 6, 4, 2, 16, 500000.0
    a, d = np.arange(T) * 37, np.arange(T) % 3
    x = _rand((T, (Hq + 2 * Hkv) * D), 7)
    gQ, gK, gV = _rand((T, Hq, D), 8), _rand((T, Hkv, D), 9), _rand((T, Hkv, D), 10)
    Q, K, V = ro.rope_qkv_fwd(x, a, d, Hq, Hkv, D, base)
    gx = ro.rope_qkv_bwd(gQ, gK, gV, a, d, Hq, Hkv, D, base)
    lhs = np.sum(Q * gQ) + np.sum(K * gK) + np.sum(V * gV)
    assert lhs == pytest.approx(np.sum(x * gx), rel=1e-12)
    # and the gradient of an unrotated part passes through unchanged
    np.testing.assert_array_equal(gx[:, (Hq + Hkv) * D :], gV.reshape(T, -1))
