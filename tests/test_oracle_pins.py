"""Pins for the fp64 oracle of y = y_base + s_i * (x . A_i) . B_i (CPU only).

Each test checks the oracle against something other than itself: a closed form,
an algebraic identity evaluated with a different association by a library
routine, exact integer arithmetic, or a hand-worked example.
"""
import numpy as np
import pytest

from conftest import read_golden
from oracle import lora_oracle as orc
from paper_2602_24044_b200 import workloads as W


def _rand_problem(rng, T=9, d_in=11, d_out=7, ranks=(1, 2, 3, 5)):
    N = len(ranks)
    x = rng.standard_normal((T, d_in))
    yb = rng.standard_normal((T, d_out))
    A = [rng.standard_normal((d_in, r)) for r in ranks]
    B = [rng.standard_normal((r, d_out)) for r in ranks]
    s = rng.uniform(0.1, 3.0, N)
    idx = rng.integers(0, N, T).astype(np.int32)
    return x, yb, A, B, np.array(ranks, np.int32), s, idx


def test_hand_worked_example():
    g = read_golden("lora_forward_hand.txt")
    d_in, d_out = int(g["d_in"][0]), int(g["d_out"][0])
    rank = np.array(g["rank"], np.int32)
    x = np.array(g["x"]).reshape(-1, d_in)
    yb = np.array(g["y_base"]).reshape(-1, d_out)
    A = [np.array(g["A%d" % i]).reshape(d_in, rank[i]) for i in range(2)]
    B = [np.array(g["B%d" % i]).reshape(rank[i], d_out) for i in range(2)]
    y, n_inv = orc.apply(x, yb, np.array(g["slot_idx"], np.int32), A, B, rank,
                         np.array(g["scale"]), np.ones(2, np.int32))
    assert n_inv == 0
    assert np.array_equal(y, np.array(g["y"]).reshape(-1, d_out))


def test_merged_weight_equivalence():
    """x.(W + s.A.B) with y_base = x.W, merged in a different association by numpy."""
    rng = np.random.default_rng(1)
    x, _, A, B, rank, s, idx = _rand_problem(rng)
    Wm = rng.standard_normal((x.shape[1], B[0].shape[1]))
    yb = x @ Wm
    y, _ = orc.apply(x, yb, idx, A, B, rank, s, np.ones(len(A), np.int32))
    for t in range(x.shape[0]):
        i = idx[t]
        merged = Wm + s[i] * (A[i] @ B[i])
        want = x[t] @ merged
        mag = np.abs(x[t]) @ (np.abs(Wm) + s[i] * (np.abs(A[i]) @ np.abs(B[i])))
        assert np.all(np.abs(y[t] - want) <= 1e-12 * mag)


def test_zero_B_returns_base_exactly():
    rng = np.random.default_rng(2)
    x, yb, A, B, rank, s, idx = _rand_problem(rng)
    B = [np.zeros_like(b) for b in B]
    y, _ = orc.apply(x, yb, idx, A, B, rank, s, np.ones(len(A), np.int32))
    assert np.array_equal(y, yb)


def test_rank1_closed_form_exact():
    """x = 1, a = 2^-m, small-integer b: y = y_base + s * d_in * 2^-m * b_j exactly."""
    T, d_in, d_out, m = 4, 64, 10, 3
    x = np.ones((T, d_in))
    a = np.full((d_in, 1), 2.0 ** -m)
    b = np.arange(-5, 5, dtype=np.float64).reshape(1, d_out)
    yb = np.arange(T * d_out, dtype=np.float64).reshape(T, d_out)
    s = np.array([3.0])
    y, _ = orc.apply(x, yb, np.zeros(T, np.int32), [a], [b], np.array([1], np.int32), s,
                     np.ones(1, np.int32))
    want = yb + 3.0 * (d_in * 2.0 ** -m) * b
    assert np.array_equal(y, want)


def test_rank1_closed_form_general():
    rng = np.random.default_rng(3)
    T, d_in, d_out = 6, 13, 5
    x = rng.standard_normal((T, d_in))
    a = rng.standard_normal((d_in, 1))
    b = rng.standard_normal((1, d_out))
    yb = rng.standard_normal((T, d_out))
    y, _ = orc.apply(x, yb, np.zeros(T, np.int32), [a], [b], np.array([1], np.int32),
                     np.array([0.7]), np.ones(1, np.int32))
    for t in range(T):
        for j in range(d_out):
            want = yb[t, j] + 0.7 * float(x[t] @ a[:, 0]) * b[0, j]
            assert abs(y[t, j] - want) <= 1e-13 * (abs(yb[t, j]) + abs(want) + 1)


def test_batch_permutation_invariance_bitwise():
    rng = np.random.default_rng(4)
    x, yb, A, B, rank, s, idx = _rand_problem(rng, T=23)
    ld = np.ones(len(A), np.int32)
    y, _ = orc.apply(x, yb, idx, A, B, rank, s, ld)
    p = rng.permutation(x.shape[0])
    yp, _ = orc.apply(x[p], yb[p], idx[p], A, B, rank, s, ld)
    assert np.array_equal(yp, y[p])


def test_linearity_in_scale_and_rank_additivity():
    rng = np.random.default_rng(5)
    T, d_in, d_out, r = 7, 12, 9, 4
    x = rng.standard_normal((T, d_in))
    A = rng.standard_normal((d_in, r))
    B = rng.standard_normal((r, d_out))
    z = np.zeros((T, d_out))
    idx = np.zeros(T, np.int32)
    one = np.ones(1, np.int32)
    full, _ = orc.apply(x, z, idx, [A], [B], np.array([r], np.int32), np.array([1.0]), one)
    twice, _ = orc.apply(x, z, idx, [A], [B], np.array([r], np.int32), np.array([2.0]), one)
    assert np.array_equal(twice, 2.0 * full)          # power-of-two scaling is exact
    third, _ = orc.apply(x, z, idx, [A], [B], np.array([r], np.int32), np.array([0.3]), one)
    assert np.allclose(third, 0.3 * full, rtol=1e-14, atol=0)
    parts = np.zeros_like(full)
    for k in range(r):
        pk, _ = orc.apply(x, z, idx, [A[:, k:k + 1]], [B[k:k + 1, :]], np.array([1], np.int32),
                          np.array([1.0]), one)
        parts += pk
    mag = (np.abs(x) @ np.abs(A)) @ np.abs(B)
    assert np.all(np.abs(parts - full) <= 1e-13 * mag)


def test_single_adapter_equals_two_library_matmuls():
    rng = np.random.default_rng(6)
    T, d_in, d_out, r = 33, 40, 24, 8
    x = rng.standard_normal((T, d_in))
    yb = rng.standard_normal((T, d_out))
    A = rng.standard_normal((d_in, r))
    B = rng.standard_normal((r, d_out))
    y, _ = orc.apply(x, yb, np.zeros(T, np.int32), [A], [B], np.array([r], np.int32),
                     np.array([1.7]), np.ones(1, np.int32))
    want = yb + 1.7 * ((x @ A) @ B)
    mag = np.abs(yb) + 1.7 * ((np.abs(x) @ np.abs(A)) @ np.abs(B))
    assert np.all(np.abs(y - want) <= 1e-12 * mag)


def test_exact_integer_case_matches_int64_arithmetic():
    """Small-integer inputs: fp64 is exact, so the oracle must equal integer arithmetic."""
    wl = W.make_custom(37, 64, 48, 5, [1, 3, 8, 16, 5], scale=2.0, weight_mode="int",
                       act_mode="int", frac_none=0.2)
    y, _ = orc.apply_workload(wl)
    x_h, yb_h = wl.activations(0)
    xi = W.bf16_to_f64(x_h).astype(np.int64)
    ybi = W.bf16_to_f64(yb_h).astype(np.int64)
    want = ybi.copy()
    for t in range(wl.T):
        i = wl.slot_idx[t]
        if i < 0:
            continue
        a_h, b_h = wl.adapter_weights(int(i), 0)
        Ai = W.bf16_to_f64(a_h).astype(np.int64)
        Bi = W.bf16_to_f64(b_h).astype(np.int64)
        want[t] = ybi[t] + 2 * ((xi[t] @ Ai) @ Bi)
    assert np.array_equal(y, want.astype(np.float64))
    assert np.any(want != ybi)


def test_inactive_tokens_get_base_and_are_counted():
    rng = np.random.default_rng(8)
    x, yb, A, B, rank, s, idx = _rand_problem(rng, T=12)
    idx[:] = [0, -1, 1, 7, 2, -5, 3, 3, -1, 2, 4, 0]      # 7, 4 out of range; -5 invalid
    loaded = np.array([1, 1, 0, 1], np.int32)              # slot 2 empty -> tokens 4, 9 invalid
    y, n_inv = orc.apply(x, yb, idx, A, B, rank, s, loaded)
    assert n_inv == 5
    for t in (1, 3, 4, 5, 8, 9, 10):
        assert np.array_equal(y[t], yb[t])
    for t in (0, 2, 6, 7, 11):
        assert not np.array_equal(y[t], yb[t])


def test_transposed_operand_would_fail():
    """Square case d_in == r == d_out with asymmetric matrices: A and B orientation is pinned."""
    rng = np.random.default_rng(9)
    n = 4
    x = rng.standard_normal((3, n))
    A = rng.standard_normal((n, n))
    B = rng.standard_normal((n, n))
    z = np.zeros((3, n))
    y, _ = orc.apply(x, z, np.zeros(3, np.int32), [A], [B], np.array([n], np.int32),
                     np.array([1.0]), np.ones(1, np.int32))
    assert np.allclose(y, x @ A @ B, rtol=1e-12)
    assert not np.allclose(y, x @ A.T @ B, rtol=1e-3)
    assert not np.allclose(y, x @ A @ B.T, rtol=1e-3)
    assert not np.allclose(y, x @ B @ A, rtol=1e-3)


def test_threads_do_not_change_result():
    wl = W.make_custom(50, 128, 96, 6, [4, 8, 16], scale=[0.3, 1.5], frac_none=0.1)
    y1, _ = orc.apply_workload(wl, threads=1)
    y4, _ = orc.apply_workload(wl, threads=4)
    assert np.array_equal(y1, y4)


def test_row_subset_matches_full():
    wl = W.make_config(0)
    y, _ = orc.apply_workload(wl)
    rows = np.array([3, 9, 15])
    ys, _ = orc.apply_workload(wl, rows=rows)
    assert np.array_equal(ys, y[rows])


@pytest.mark.parametrize("cfg", [0, 1])
def test_config_delta_statistics(cfg):
    """The configured distributions give the delta size the tolerance analysis assumes."""
    wl = W.make_config(cfg)
    y, _ = orc.apply_workload(wl, threads=4)
    _, yb_h = wl.activations(0)
    delta = y - W.bf16_to_f64(yb_h)
    r = int(wl.ranks[0])
    expect = 2.0 * np.sqrt(r / 3.0) * 0.02     # s * sqrt(r * Var(v) * Var(B)), Var(v) = 1/3
    assert 0.8 * expect < delta.std() < 1.2 * expect
