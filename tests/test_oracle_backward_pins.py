"""Pins for the oracle's backward pass (the gradients that the training task of Sections 2.2 and 4.1 takes through the
mixed-adapter linear layer).  Nothing here calls the CUDA path.

* The forward oracle is linear in x, in A and in B, so a central difference of the scalar
  L = sum(dy * y) in any direction equals the directional derivative exactly up to rounding:
  dL/dx, dL/dA, dL/dB from the backward oracle are checked against differences of the FORWARD oracle
  (an independent routine) on inputs whose perturbed values are still exact in bf16.
* Closed forms: one token, rank 1, hand-computed numbers.
* Structure: entries no token is bound to get zero gradients; unbound rows get dx = dy.W0; perm
  only renames rows; two segments with the same entry add up.
"""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

pytestmark = pytest.mark.filterwarnings("ignore")


def bits(a):
    return wl.f32_to_bf16_bits(np.asarray(a, np.float32))


def small_ints(rng, shape, lo=-3, hi=4):
    return rng.integers(lo, hi, size=shape).astype(np.float32)   # exact in bf16, and so are +-1 steps


def problem(seed, T=5, K=6, N=4, ranks=(2, 3), perm=False):
    rng = np.random.default_rng(seed)
    x, W0, dy = small_ints(rng, (T, K)), small_ints(rng, (N, K)), small_ints(rng, (T, N))
    entries = [wl.AdapterEntry(i, 1, r, float(s), bits(small_ints(rng, (r, K))), bits(small_ints(rng, (N, r))))
               for i, (r, s) in enumerate(zip(ranks, (0.5, 2.0, 1.0)))]
    so = np.array([0, 2, 3, T], np.int32)
    se = np.array([1, -1, 0], np.int32)
    pm = rng.permutation(T).astype(np.int32) if perm else None
    return x, W0, dy, entries, so, se, pm


def loss(x, W0, dy, entries, so, se, pm):
    y, _ = oracle.forward(bits(x), bits(W0), entries, so, se, pm)
    return float((dy * y).sum())


@pytest.mark.parametrize("perm", [False, True])
def test_dx_is_the_derivative_of_the_forward_oracle(perm):
    x, W0, dy, entries, so, se, pm = problem(1, perm=perm)
    dx, _, _, flags = oracle.backward(bits(x), bits(dy), bits(W0), entries, so, se, pm)
    assert flags == 0
    for t in range(x.shape[0]):
        for k in range(x.shape[1]):
            xp, xm = x.copy(), x.copy()
            xp[t, k] += 1.0
            xm[t, k] -= 1.0
            fd = (loss(xp, W0, dy, entries, so, se, pm) - loss(xm, W0, dy, entries, so, se, pm)) / 2.0
            assert dx[t, k] == pytest.approx(fd, abs=1e-9), (t, k)


@pytest.mark.parametrize("perm", [False, True])
def test_dA_and_dB_are_the_derivatives_of_the_forward_oracle(perm):
    x, W0, dy, entries, so, se, pm = problem(2, perm=perm)
    _, dA, dB, _ = oracle.backward(bits(x), bits(dy), bits(W0), entries, so, se, pm)
    import dataclasses
    for e, ent in enumerate(entries):
        A = wl.bf16_bits_to_f64(ent.A).astype(np.float32)
        B = wl.bf16_bits_to_f64(ent.B).astype(np.float32)
        for which, M, grad in (("A", A, dA[e]), ("B", B, dB[e])):
            for idx in np.ndindex(M.shape):
                vals = []
                for sign in (+1.0, -1.0):
                    Mp = M.copy()
                    Mp[idx] += sign
                    ent2 = dataclasses.replace(ent, **{which: bits(Mp)})
                    es = list(entries)
                    es[e] = ent2
                    vals.append(loss(x, W0, dy, es, so, se, pm))
                assert grad[idx] == pytest.approx((vals[0] - vals[1]) / 2.0, abs=1e-9), (e, which, idx)


def test_hand_worked_single_token_rank_one():
    # x = [1, 2], W0 = [[3, 4]], A = [[5, 6]], B = [[7]], s = 2, dy = [10]
    # y = 1*3 + 2*4 + 2 * (1*5 + 2*6) * 7 = 11 + 238
    # dx = 10*[3, 4] + 2 * (10*7) * [5, 6] = [30 + 700, 40 + 840]
    # dA = 2 * (10*7) * [1, 2] = [140, 280];   dB = 2 * 10 * (1*5 + 2*6) = 340
    e = wl.AdapterEntry(0, 1, 1, 2.0, bits([[5, 6]]), bits([[7]]))
    dx, dA, dB, flags = oracle.backward(bits([[1, 2]]), bits([[10]]), bits([[3, 4]]), [e], [0, 1], [0])
    assert flags == 0
    assert dx.tolist() == [[730.0, 880.0]] and dA[0].tolist() == [[140.0, 280.0]] and dB[0].tolist() == [[340.0]]


def test_matches_the_matrix_identities_in_numpy():
    rng = np.random.default_rng(7)
    T, K, N, r = 9, 16, 12, 4
    xb, Wb, dyb = wl.normal_bf16(7, 1, (T, K), 1.0), wl.normal_bf16(7, 2, (N, K), 0.3), wl.normal_bf16(7, 3, (T, N), 1.0)
    ent = wl.AdapterEntry(0, 1, r, 1.5, wl.normal_bf16(7, 4, (r, K), 0.3), wl.normal_bf16(7, 5, (N, r), 0.3))
    dx, dA, dB, _ = oracle.backward(xb, dyb, Wb, [ent], [0, T], [0])
    x, W, dy = (wl.bf16_bits_to_f64(v) for v in (xb, Wb, dyb))
    A, B = wl.bf16_bits_to_f64(ent.A), wl.bf16_bits_to_f64(ent.B)
    assert np.allclose(dx, dy @ W + 1.5 * (dy @ B) @ A, rtol=1e-12, atol=1e-12)
    assert np.allclose(dA[0], 1.5 * (dy @ B).T @ x, rtol=1e-12, atol=1e-12)
    assert np.allclose(dB[0], 1.5 * dy.T @ (x @ A.T), rtol=1e-12, atol=1e-12)


def test_structure_unbound_rows_unused_entries_repeated_entries():
    x, W0, dy, entries, so, se, pm = problem(3, T=6, ranks=(2, 3, 1))
    so = np.array([0, 2, 3, 5, 6], np.int32)
    se = np.array([1, -1, 1, -1], np.int32)       # entry 1 twice, entries 0 and 2 never
    dx, dA, dB, flags = oracle.backward(bits(x), bits(dy), bits(W0), entries, so, se)
    assert flags == 0
    assert not dA[0].any() and not dB[0].any() and not dA[2].any() and not dB[2].any()
    xw = dy.astype(np.float64) @ W0.astype(np.float64)
    for t in (2, 5):
        assert np.array_equal(dx[t], xw[t])
    # the two segments of entry 1 add up: same as one call per segment
    parts = []
    for lo, hi in ((0, 2), (3, 5)):
        so1 = np.array([0, lo, hi, 6], np.int32)
        parts.append(oracle.backward(bits(x), bits(dy), bits(W0), entries, so1, np.array([-1, 1, -1], np.int32)))
    assert np.array_equal(dA[1], parts[0][1][1] + parts[1][1][1])
    assert np.array_equal(dB[1], parts[0][2][1] + parts[1][2][1])


def test_dead_entry_is_flagged_and_contributes_nothing():
    x, W0, dy, entries, so, se, pm = problem(4)
    dx, dA, dB, flags = oracle.backward(bits(x), bits(dy), bits(W0), entries, so, se, live=[1, 0])
    assert flags & 1
    assert not dA[1].any() and not dB[1].any()
    assert np.array_equal(dx[0], (dy.astype(np.float64) @ W0.astype(np.float64))[0])
