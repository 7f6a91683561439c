"""Pins for the checker's NTT: brute force, closed forms, round trips."""
import numpy as np
import pytest

from oracle.ckks_oracle import Oracle
from paper_2609_12378_b200 import inputs
from tests.harness import brev, negacyclic_schoolbook, params


def _smallest_root_bruteforce(q, N):
    for x in range(2, q):
        if pow(x, N, q) == q - 1:
            return x


@pytest.mark.parametrize("q,log_n", [(17, 3), (97, 4), (257, 7), (7681, 8), (12289, 10)])
def test_root_is_smallest_primitive_2n_th_root(q, log_n):
    o = Oracle(log_n, [q], [], 1)
    assert o.root(0) == _smallest_root_bruteforce(q, 1 << log_n)


def test_root_50_bit():
    P = params(16, 24, 8, 3)
    for t in (0, 23, 24, 31):
        m, psi = P.oracle.mod[t], P.oracle.root(t)
        assert pow(psi, P.N, m) == m - 1
    # values recomputed independently when the parameter rule was written down
    assert (P.oracle.root(0), P.oracle.root(23), P.oracle.root(24)) == (756806287, 9962773766, 938640682)


def test_worked_example_q17_n8():
    """q = 17, N = 8, psi = 3, a = 1..8, all by hand-sized brute force."""
    q, N, psi = 17, 8, 3
    a = list(range(1, 9))
    nat = [sum(a[j] * pow(psi, (2 * k + 1) * j, q) for j in range(N)) % q for k in range(N)]
    assert nat == [5, 9, 13, 5, 0, 11, 8, 8]
    stored = [nat[brev(p, 3)] for p in range(N)]
    o = Oracle(3, [q], [], 1)
    arr = np.array(a, dtype=np.uint64)
    assert o.ntt_definition(arr, 0).tolist() == stored == [5, 0, 13, 8, 9, 11, 5, 8]
    assert o.ntt(arr.reshape(1, N))[0].tolist() == stored
    sq = o.ntt(arr.reshape(1, N))[0].astype(object) ** 2 % q
    conv = o.intt(np.array(sq.tolist(), dtype=np.uint64).reshape(1, N))[0].tolist()
    assert conv == negacyclic_schoolbook(a, a, q) == [7, 10, 10, 9, 9, 12, 3, 1]


@pytest.mark.parametrize("q,log_n", [(17, 3), (97, 4), (193, 5), (int(inputs.ntt_primes(6, 1)[0]), 6)])
def test_convolution_theorem_vs_schoolbook(q, log_n):
    N = 1 << log_n
    o = Oracle(log_n, [q], [], 1)
    g = inputs.rng(11, log_n)
    a = inputs.uniform_residues(g, [q], N)[0]
    b = inputs.uniform_residues(g, [q], N)[0]
    fa, fb = o.ntt(a)[0], o.ntt(b)[0]
    prod = np.array([int(x) * int(y) % q for x, y in zip(fa, fb)], dtype=np.uint64)
    assert o.intt(prod.reshape(1, N))[0].tolist() == negacyclic_schoolbook(a[0], b[0], q)
    # the O(N^2) definitions agree with the fast transforms and invert each other
    assert np.array_equal(o.ntt_definition(a[0], 0), fa)
    assert np.array_equal(o.intt_definition(fa, 0), a[0])


def test_fast_vs_definition_n1024():
    P = params(10, 2, 1, 2)
    g = inputs.rng(12)
    for t in range(3):
        a = inputs.uniform_residues(g, [P.oracle.mod[t]], P.N)[0]
        f = P.oracle.ntt(a, first=t)[0]
        assert np.array_equal(P.oracle.ntt_definition(a[0], t), f)
        assert np.array_equal(P.oracle.intt_definition(f, t), a[0])
        assert np.array_equal(P.oracle.intt(f.reshape(1, -1), first=t)[0], a[0])


@pytest.mark.parametrize("log_n", [4, 10, 16])
def test_closed_forms_and_horner(log_n):
    P = params(log_n, 3, 1, 3) if log_n != 16 else params(16, 24, 8, 3)
    o, N = P.oracle, P.N
    for t in (0, P.L - 1, P.L):                      # first q, last q, first p
        m, psi = o.mod[t], o.root(t)
        one = np.zeros((1, N), dtype=np.uint64); one[0, 0] = 1
        assert (o.ntt(one, first=t) == 1).all()
        x = np.zeros((1, N), dtype=np.uint64); x[0, 1] = 1
        fx = o.ntt(x, first=t)[0]
        ps = [0, 1, 2, 3, N // 2, N - 1] + [int(v) for v in inputs.rng(13, t).integers(0, N, 8)]
        for p in ps:
            assert int(fx[p]) == pow(psi, 2 * brev(p, log_n) + 1, m)
        a = inputs.uniform_residues(inputs.rng(14, t), [m], N)[0]
        fa = o.ntt(a, first=t)[0]
        for p in ps:                                  # Horner evaluation at psi^(2 brev(p) + 1)
            pt, acc = pow(psi, 2 * brev(p, log_n) + 1, m), 0
            for c in a[0][::-1].tolist():
                acc = (acc * pt + c) % m
            assert int(fa[p]) == acc
        assert np.array_equal(o.intt(fa.reshape(1, N), first=t)[0], a[0])


def test_batched_layout():
    """[batch][limbs][N]: limb i of every batch entry goes under prime first+i."""
    P = params(10, 3, 1, 3)
    o = P.oracle
    g = inputs.rng(15)
    x = inputs.uniform_residues(g, o.mod[1:4], P.N, batch=3)
    y = o.ntt(x, first=1)
    for b in range(3):
        for i in range(3):
            assert np.array_equal(y[b, i], o.ntt_definition(x[b, i], 1 + i))
    assert np.array_equal(o.intt(y, first=1), x)
