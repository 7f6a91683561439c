"""Pins for the checker's encode / decode / encrypt / decrypt."""
import cmath
import math

import numpy as np
import pytest

from oracle.ckks_oracle import Oracle
from paper_2609_12378_b200 import inputs
from tests.harness import Client, negacyclic_schoolbook, params


def _embedding_coeffs(z, N, scale):
    """m_k = (scale/n) Re sum_j z_j zeta^(-5^j k), straight from the definition."""
    n, M = N // 2, 2 * N
    out = []
    for k in range(N):
        acc = 0
        for j in range(n):
            acc += z[j] * cmath.exp(-2j * math.pi * (pow(5, j, M) * k % M) / M)
        out.append(acc.real * scale / n)
    return out


def test_worked_example_n8():
    """N = 8, Delta = 2^10, z = (1,2,3,4); then X -> X^5 is a left rotation by one slot."""
    o = Oracle(3, [inputs.ntt_primes(3, 1)[0]], [], 1)
    z = [1.0, 2.0, 3.0, 4.0]
    want = [round(v) for v in _embedding_coeffs(z, 8, 2.0 ** 10)]
    assert want == [2560, -277, -362, -669, 0, 669, 362, 277]
    m = o.encode_coeffs(np.array(z), 2.0 ** 10)
    assert m.tolist() == want
    rot = o.automorphism_small(m, 5)
    assert rot.tolist() == [2560, -669, 362, 277, 0, -277, -362, 669]
    back = o.decode(rot.astype(np.longdouble), 2.0 ** 10)
    assert np.abs(back - np.array([2, 3, 4, 1])).max() < 2e-3
    assert np.abs(o.decode(m.astype(np.longdouble), 2.0 ** 10, direct=True) - np.array(z)).max() < 2e-3


@pytest.mark.parametrize("log_n", [4, 7, 10])
def test_encode_matches_definition_sum(log_n):
    P = params(log_n, 2, 1, 2)
    g = inputs.rng(21, log_n)
    z = g.uniform(-1, 1, P.n) + 1j * g.uniform(-1, 1, P.n)
    scale = 2.0 ** 40
    m = P.oracle.encode_coeffs(z, scale)
    want = _embedding_coeffs(z.tolist(), P.N, scale)
    diff = np.array([int(a) - b for a, b in zip(m.tolist(), want)])
    assert np.abs(diff).max() <= 0.5 + 1e-2       # rounding of the exact value, fp64 slack of the python sum


def test_decode_direct_equals_fast():
    P = params(8, 2, 1, 2)
    m = inputs.rng(22).integers(-2 ** 45, 2 ** 45, P.N).astype(np.longdouble)
    a, b = P.oracle.decode(m, 2.0 ** 40), P.oracle.decode(m, 2.0 ** 40, direct=True)
    assert np.abs(a - b).max() < 1e-9


@pytest.mark.parametrize("log_n", [10, 13, 16])
def test_decode_encode_roundtrip_bound(log_n):
    P = params(log_n, 2, 1, 2)
    g = inputs.rng(23, log_n)
    z = g.uniform(-1, 1, P.n) + 1j * g.uniform(-1, 1, P.n)
    scale = 2.0 ** 40
    m = P.oracle.encode_coeffs(z, scale)
    back = P.oracle.decode(m.astype(np.longdouble), scale)
    err = np.abs(back - z).max()
    assert err <= P.N / (2 * scale)               # worst case: every coefficient off by 1/2
    assert err < 2.0 ** -30


def test_constant_and_cosine_closed_forms():
    P = params(10, 2, 1, 2)
    o, N, n, M = P.oracle, P.N, P.n, 2 * P.N
    scale = 2.0 ** 40
    c = 0.7316
    m = o.encode_coeffs(np.full(n, c), scale)
    assert m[0] == round(c * scale) and np.abs(m[1:]).max() <= 1
    for k in (1, 5, 77, n - 1, n + 3):
        z = np.array([math.cos(2 * math.pi * (pow(5, j, M) * k % M) / M) for j in range(n)])
        m = o.encode_coeffs(z, scale)                 # (Delta/2)(X^k - X^(N-k))
        want = np.zeros(N); want[k] = scale / 2; want[N - k] = -scale / 2
        assert np.abs(m - want).max() <= 64          # fp64 twiddle error at 2^40, far below Delta


def test_slotwise_product_homomorphism():
    """encode(z) * encode(w) in the ring decodes to z .* w at scale Delta^2."""
    log_n = 5
    q = inputs.ntt_primes(log_n, 1)[0]
    o = Oracle(log_n, [q], [], 1)
    g = inputs.rng(24)
    z, w = g.uniform(-1, 1, 16), g.uniform(-1, 1, 16)
    scale = 2.0 ** 20
    a, b = o.encode_coeffs(z, scale), o.encode_coeffs(w, scale)
    big = 1 << 100
    prod = negacyclic_schoolbook([int(x) % big for x in a], [int(x) % big for x in b], big)
    prod = np.array([x - big if x > big // 2 else x for x in prod], dtype=np.longdouble)
    assert np.abs(o.decode(prod, scale * scale) - z * w).max() < 1e-4


def test_encode_limbs_are_ntt_of_reduced_coeffs():
    P = params(10, 3, 1, 3)
    o = P.oracle
    z = inputs.rng(25).uniform(-1, 1, P.n)
    m = o.encode_coeffs(z, 2.0 ** 40)
    limbs = o.encode(z, 2.0 ** 40, 3)
    for i in range(3):
        red = np.array([int(v) % o.mod[i] for v in m.tolist()], dtype=np.uint64)
        assert np.array_equal(limbs[i], o.ntt_definition(red, i))
    assert np.array_equal(o.small_to_limbs(m, 0, 3), limbs)


def test_encode_range_error():
    P = params(10, 2, 1, 2)
    with pytest.raises(OverflowError):
        P.oracle.encode_coeffs(np.full(P.n, 1.0), 2.0 ** 63)


def test_encrypt_decrypt_exact():
    """decrypt(encrypt(m)) = m + e exactly, as integers."""
    P = params(10, 3, 1, 3)
    o = P.oracle
    cl = Client(P, 31)
    z = inputs.rng(26).uniform(-1, 1, P.n)
    pt = o.encode(z, 2.0 ** 40, 3)
    g = inputs.rng(27)
    a = inputs.uniform_residues(g, P.q[:3], P.N)[0]
    e = inputs.rounded_gaussian(g, P.N)
    ct = o.encrypt(pt, a, e, cl.s)
    assert np.array_equal(ct[1], a)
    got = o.decrypt(ct, cl.s, exact=True)
    want = (o.encode_coeffs(z, 2.0 ** 40) + e).tolist()
    assert got == want
    # single-limb decrypt path
    assert o.decrypt(ct[:, :1], cl.s, exact=True) == want
    assert np.abs(cl.decrypt_slots(ct, 2.0 ** 40) - z).max() < 2.0 ** -25


def test_decrypt_three_components():
    """c0 + c1 s + c2 s^2 of a tensor product equals the ring product of the two plaintexts."""
    P = params(5, 3, 1, 3)
    o = P.oracle
    cl = Client(P, 32)
    g = inputs.rng(28)
    z, w = g.uniform(-1, 1, P.n), g.uniform(-1, 1, P.n)
    scale = 2.0 ** 30
    ca, cb = cl.encrypt_slots(z, scale, 3), cl.encrypt_slots(w, scale, 3)
    ma, mb = o.decrypt(ca, cl.s, exact=True), o.decrypt(cb, cl.s, exact=True)
    big = 1 << 120
    want = negacyclic_schoolbook([x % big for x in ma], [x % big for x in mb], big)
    want = [x - big if x > big // 2 else x for x in want]
    assert o.decrypt(o.tensor(ca, cb), cl.s, exact=True) == want
