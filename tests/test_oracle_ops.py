"""Pins for the oracle's single operations: fp64 restatements in dense/matrix form, closed
forms and special cases.  None of these call the CUDA path."""
import math

import numpy as np
import pytest

from oracle import sdv_oracle as O
from sdv_inputs import bf16_bits_to_f32, f32_to_bf16_bits

RNG = np.random.default_rng(1234)


def _bf16(x):
    return f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


@pytest.mark.parametrize("M,N,K", [(1, 5, 7), (9, 33, 64), (17, 20, 130), (70, 19, 96), (256, 8, 40)])
def test_matmul_against_fp64_einsum(M, N, K):
    x = RNG.standard_normal((M, K)).astype(np.float32)
    wb = _bf16(RNG.standard_normal((N, K)))
    bias = RNG.standard_normal(N).astype(np.float32)
    ref = np.einsum("mk,nk->mn", x.astype(np.float64), bf16_bits_to_f32(wb).astype(np.float64)) + bias
    got = O.matmul(x, wb, bias)
    assert got.shape == (M, N)
    np.testing.assert_allclose(got, ref, rtol=0, atol=2e-5 * math.sqrt(K))
    # a transposed or mis-strided operand cannot pass: single-entry probes
    e = np.zeros((M, K), dtype=np.float32)
    e[M - 1, K - 2] = 1.0
    np.testing.assert_array_equal(O.matmul(e, wb)[M - 1], bf16_bits_to_f32(wb)[:, K - 2])


@pytest.mark.parametrize("M,N,K", [(1, 5, 7), (9, 33, 64), (17, 21, 130), (33, 7, 96), (70, 19, 50), (3, 130, 257)])
def test_fast_matmul_equals_the_plain_triple_loop_bit_for_bit(M, N, K):
    """orc_matmul (blocked, transposed, threaded) against orc_matmul_plain (the definition as three
    nested loops): the same sums in the same order, so not one bit may differ, bias included."""
    x = (RNG.standard_normal((M, K)) * 3).astype(np.float32)
    wb = _bf16(RNG.standard_normal((N, K)))
    bias = RNG.standard_normal(N).astype(np.float32)
    np.testing.assert_array_equal(O.matmul(x, wb, bias), O.matmul_plain(x, wb, bias))
    np.testing.assert_array_equal(O.matmul(x, wb), O.matmul_plain(x, wb))


def test_plain_matmul_against_hand_values():
    # y[m][n] = sum_k x[m][k] w[n][k] + b[n], worked by hand
    x = np.array([[1, 2, 3], [0, -1, 4]], dtype=np.float32)
    w = np.array([[1, 0, 2], [0.5, 0.5, 0.5], [-1, 1, 0], [0, 0, 1]], dtype=np.float32)
    b = np.array([10, 0, 0, -1], dtype=np.float32)
    want = np.array([[17, 3, 1, 2], [18, 1.5, -1, 3]], dtype=np.float32)
    np.testing.assert_array_equal(O.matmul_plain(x, _bf16(w), b), want)
    np.testing.assert_array_equal(O.matmul(x, _bf16(w), b), want)


def test_top2_margin_and_runner_up():
    """The margin decides which flipped greedy tokens the parity tests forgive, the runner-up which
    token they may flip to."""
    # exact tie: margin 0, greedy = the lower id, runner-up = the other tied id
    assert O.top2(np.array([1.0, 5.0, 5.0, 2.0], dtype=np.float32)) == (1, 2, 0.0)
    # known gap, maximum at either end
    assert O.top2(np.array([9.0, 1.0, 2.0, 8.5], dtype=np.float32)) == (0, 3, 0.5)
    assert O.top2(np.array([-3.0, -7.0, -2.25, -2.0], dtype=np.float32)) == (3, 2, 0.25)
    # three-way tie: the two lowest ids
    assert O.top2(np.array([4.0, 4.0, 4.0], dtype=np.float32)) == (0, 1, 0.0)
    assert O.top2_margin(np.array([0.0, 1.5], dtype=np.float32)) == 1.5
    for _ in range(200):
        n = int(RNG.integers(2, 300))
        row = RNG.standard_normal(n).astype(np.float32)
        if RNG.random() < 0.3:      # plant ties
            row[RNG.integers(0, n, size=3)] = row.max()
        best, second, margin = O.top2(row)
        srt = sorted(row.tolist())
        assert margin == np.float32(srt[-1]) - np.float32(srt[-2])
        order = sorted(range(n), key=lambda i: (-row[i], i))     # value descending, id ascending
        assert (best, second) == (order[0], order[1])
        assert best == O.argmax(row)


def test_matmul_rows_do_not_depend_on_batch():
    x = RNG.standard_normal((70, 96)).astype(np.float32)
    wb = _bf16(RNG.standard_normal((24, 96)))
    full = O.matmul(x, wb)
    for m in (0, 16, 69):
        np.testing.assert_array_equal(O.matmul(x[m:m + 1], wb)[0], full[m])


def test_rmsnorm():
    d = 96
    x = RNG.standard_normal(d).astype(np.float32) * 3
    w = RNG.standard_normal(d).astype(np.float32)
    x64 = x.astype(np.float64)
    ref = x64 / np.sqrt(np.mean(x64 ** 2) + 1e-6) * w
    np.testing.assert_allclose(O.rmsnorm(x, w, 1e-6), ref, atol=1e-5)
    # a constant row normalises to sign(c) * w
    np.testing.assert_allclose(O.rmsnorm(np.full(d, -7.0), w, 1e-9), -w, atol=1e-5)
    # eps matters for tiny rows: x = 1e-3 -> x / sqrt(1e-6 + eps)
    np.testing.assert_allclose(O.rmsnorm(np.full(d, 1e-3), np.ones(d), 3e-6), np.full(d, 1e-3 / math.sqrt(4e-6)),
                               rtol=1e-5)


def test_rope_closed_forms():
    # hd = 4: pairs (0,2) and (1,3); frequencies theta^0 = 1 and theta^(-1/2)
    th = 10000.0
    np.testing.assert_allclose(O.rope([1, 0, 0, 0], 1, th), [math.cos(1), 0, math.sin(1), 0], atol=1e-7)
    np.testing.assert_allclose(O.rope([0, 1, 0, 0], 3, th), [0, math.cos(0.03), 0, math.sin(0.03)], atol=1e-7)
    np.testing.assert_allclose(O.rope([0, 0, 1, 0], 1, th), [-math.sin(1), 0, math.cos(1), 0], atol=1e-7)
    v = RNG.standard_normal(64).astype(np.float32)
    np.testing.assert_array_equal(O.rope(v, 0, 1e6), v)                       # position 0 is the identity
    np.testing.assert_allclose(np.linalg.norm(O.rope(v, 777, 1e6)), np.linalg.norm(v), rtol=1e-6)


def test_rope_scores_depend_on_relative_position_only():
    q = RNG.standard_normal(128).astype(np.float32)
    k = RNG.standard_normal(128).astype(np.float32)
    base = float(O.rope(q, 40, 5e5) @ O.rope(k, 33, 5e5))
    for shift in (1, 100, 4000):
        assert abs(float(O.rope(q, 40 + shift, 5e5) @ O.rope(k, 33 + shift, 5e5)) - base) < 2e-4
    assert abs(float(O.rope(q, 41, 5e5) @ O.rope(k, 33, 5e5)) - base) > 1e-3


def test_rope_large_position_against_fp64():
    hd, pos, th = 128, 8447, 1e6
    v = RNG.standard_normal(hd)
    i = np.arange(hd // 2)
    ang = pos * th ** (-2.0 * i / hd)
    ref = np.concatenate([v[:64] * np.cos(ang) - v[64:] * np.sin(ang), v[64:] * np.cos(ang) + v[:64] * np.sin(ang)])
    np.testing.assert_allclose(O.rope(v, pos, th), ref, atol=1e-6)


@pytest.mark.parametrize("n,hd", [(1, 64), (7, 64), (300, 128)])
def test_attention_row_against_dense_fp64(n, hd):
    q = RNG.standard_normal(hd) * 1.5
    k = RNG.standard_normal((n, hd))
    v = RNG.standard_normal((n, hd))
    s = (k @ q) / math.sqrt(hd)
    p = np.exp(s - s.max())
    p /= p.sum()
    np.testing.assert_allclose(O.attention_row(q, k, v), p @ v, atol=2e-5)


def test_attention_special_cases():
    hd = 64
    q = RNG.standard_normal(hd)
    v = RNG.standard_normal((5, hd)).astype(np.float32)
    np.testing.assert_allclose(O.attention_row(q, RNG.standard_normal((1, hd)), v[:1]), v[0], atol=1e-7)
    same = np.tile(RNG.standard_normal(hd), (5, 1))                      # equal keys -> mean of v
    np.testing.assert_allclose(O.attention_row(q, same, v), v.mean(0), atol=1e-6)
    k = np.zeros((5, hd)); k[3] = q * 100                                 # one dominant key -> its v
    np.testing.assert_allclose(O.attention_row(q, k, v), v[3], atol=1e-6)
    big = np.tile(q * 1e3, (5, 1))                                        # huge equal scores stay finite
    assert np.all(np.isfinite(O.attention_row(q, big, v)))


def test_swiglu():
    g = np.array([0.0, 1.0, -1.0, 30.0, -30.0, 2.5])
    u = np.array([3.0, 2.0, 2.0, 0.5, 4.0, -1.0])
    ref = g / (1 + np.exp(-g)) * u
    np.testing.assert_allclose(O.swiglu(g, u), ref, atol=1e-6)
    assert O.swiglu([0.0], [5.0])[0] == 0.0


def test_argmax_ties_and_nan():
    assert O.argmax([1.0, 3.0, 3.0, 2.0]) == 1                 # lowest index among equal maxima
    assert O.argmax([5.0, 5.0, 5.0]) == 0
    assert O.argmax([float("nan"), 1.0, float("nan"), 1.0]) == 1  # NaN never wins
    assert O.argmax([-np.inf, -1e30]) == 1
    x = RNG.standard_normal(5000).astype(np.float32)
    assert O.argmax(x) == int(np.argmax(x))
