"""Client-side harness for the tests: parameter sets, secret/key/ciphertext
generation through the CPU checker, big-integer helpers.  The library under
test never sees a secret key; everything secret lives here."""
from __future__ import annotations

from functools import lru_cache

import numpy as np

from oracle.ckks_oracle import Oracle
from paper_2609_12378_b200 import inputs


class Params:
    def __init__(self, log_n, num_q, num_p, dnum, bits=50):
        self.log_n, self.L, self.K, self.dnum = log_n, num_q, num_p, dnum
        self.N, self.n = 1 << log_n, 1 << (log_n - 1)
        self.q, self.p = inputs.prime_chain(log_n, num_q, num_p, bits)
        self.oracle = Oracle(log_n, self.q, self.p, dnum)


@lru_cache(maxsize=None)
def params(log_n, num_q, num_p, dnum, bits=50) -> Params:
    return Params(log_n, num_q, num_p, dnum, bits)


class Client:
    """Holds the secret; makes ciphertexts and switching keys with seeded draws."""

    def __init__(self, P: Params, seed: int):
        self.P, self.o, self.seed = P, P.oracle, seed
        self.s = inputs.ternary(inputs.rng(seed, 0), P.N)
        self._stream = 1

    def _g(self):
        self._stream += 1
        return inputs.rng(self.seed, self._stream)

    def encrypt_slots(self, z, scale, level):
        P = self.P
        pt = self.o.encode(z, scale, level)
        g = self._g()
        a = inputs.uniform_residues(g, P.q[:level], P.N)[0]
        e = inputs.rounded_gaussian(g, P.N)
        return self.o.encrypt(pt, a, e, self.s)

    def _key_draws(self):
        P = self.P
        g = self._g()
        a = inputs.uniform_residues(g, list(P.q) + list(P.p), P.N, batch=P.dnum)
        e = inputs.rounded_gaussian(g, (P.dnum, P.N))
        return a, e

    def rotation_key(self, galois):
        a, e = self._key_draws()
        return self.o.rotation_key(self.s, galois, a, e)

    def relin_key(self):
        a, e = self._key_draws()
        return self.o.relin_key(self.s, a, e)

    def decrypt_slots(self, ct, scale):
        return self.o.decrypt_decode(ct, self.s, scale)


# ------------------------------------------------------------ big-integer side

def crt(residues, moduli):
    """The integer in [0, prod moduli) with the given residues (Python ints)."""
    x, m = 0, 1
    for r, q in zip(residues, moduli):
        r, q = int(r), int(q)
        t = (r - x) * pow(m, -1, q) % q
        x += m * t
        m *= q
    return x, m


def centred(x, m):
    x %= m
    return x - m if x > m // 2 else x


def negacyclic_schoolbook(a, b, q):
    n = len(a)
    c = [0] * n
    for i in range(n):
        for j in range(n):
            k = i + j
            if k < n:
                c[k] = (c[k] + int(a[i]) * int(b[j])) % q
            else:
                c[k - n] = (c[k - n] - int(a[i]) * int(b[j])) % q
    return c


def brev(x, bits):
    return int(format(x, "0%db" % bits)[::-1], 2) if bits else 0


# ------------------------------------------------------------ Softmax by doubling (Algorithm 1), synthetic case

def softmax_case(P: Params, seed: int, row_len: int = 16, rounds: int = 2, degree: int = 4, spread: float = 11.0):
    """Scores in [shift - spread, shift] laid out row by row with stride n / row_len, polynomial fits of exp on
    [-spread / 2^rounds, 0] and of 1 / sqrt on the measured range of every round's row sums (times a safety factor),
    and the same pipeline evaluated in the clear.  Returns (slots, shift, exp_coeffs_in_z, rsqrt_coeffs, clear_result,
    true_softmax), all per slot."""
    n, stride = P.n, P.n // row_len
    g = inputs.rng(seed, 7)
    shift = 3.0
    rows = shift - spread * g.uniform(0.0, 1.0, (stride, row_len)) ** 2      # row r, element i
    rows[:, 0] = shift - 0.25                                                # one score near the top of every row
    x = np.empty(n)
    for i in range(row_len):
        x[i * stride:(i + 1) * stride] = rows[:, i]

    def fit(f, lo, hi, deg):
        t = np.cos(np.pi * (np.arange(64) + 0.5) / 64) * (hi - lo) / 2 + (hi + lo) / 2
        return np.polynomial.polynomial.polyfit(t, f(t), deg)

    ce = fit(np.exp, -spread / 2 ** rounds, 0.0, degree)
    exp_in_z = ce / (2.0 ** rounds) ** np.arange(degree + 1)                 # p_exp(z / 2^k) as a polynomial in z
    pv = np.polynomial.polynomial.polyval
    u = pv(rows - shift, exp_in_z)
    rs = []
    for _ in range(rounds):
        s = (u * u).sum(1)
        c = fit(lambda t: 1.0 / np.sqrt(t), s.min() / 1.3, s.max() * 1.3, degree)
        rs.append(c)
        u = (pv(s, c)[:, None] * u) ** 2
    clear = np.empty(n)
    for i in range(row_len):
        clear[i * stride:(i + 1) * stride] = u[:, i]
    e = np.exp(rows - rows.max(1, keepdims=True))
    true = e / e.sum(1, keepdims=True)
    truth = np.empty(n)
    for i in range(row_len):
        truth[i * stride:(i + 1) * stride] = true[:, i]
    return x, shift, exp_in_z, np.stack(rs), clear, truth


# ------------------------------------------------------------ attention in the diagonal-block layout, synthetic case

def attention_case(seed: int, tokens: int, heads: int, dim: int, dim_v: int, rounds: int = 1, degree: int = 4, spread: float = 4.0):
    """Seeded Q, K [tokens][heads][dim] and V [tokens][heads][dim_v] whose scores Q K^T fall in [shift - spread, shift],
    polynomial fits as in softmax_case, the pipeline of Algorithm 1 evaluated in the clear on the full score matrix
    (out_clear [tokens][heads][dim_v]) and plain Softmax attention (out_true).  Returns a dict."""
    g = inputs.rng(seed, 11)
    Q = g.uniform(-1.0, 1.0, (tokens, heads, dim))
    K = g.uniform(-1.0, 1.0, (tokens, heads, dim))
    V = g.uniform(-1.0, 1.0, (tokens, heads, dim_v))
    S = np.einsum("ihd,jhd->hij", Q, K)                       # [heads][query][key]
    Q = Q * (0.5 * spread / np.abs(S).max())                  # scores within +- spread / 2
    return attention_case_from(Q, K, V, rounds, degree, spread)


def attention_case_from(Q, K, V, rounds: int = 1, degree: int = 4, spread: float = 4.0):
    """The same dict for given Q, K [tokens][heads][dim], V [tokens][heads][dim_v] whose scores lie within +- spread / 2."""
    S = np.einsum("ihd,jhd->hij", Q, K)
    assert np.abs(S).max() <= 0.5 * spread * (1 + 1e-9)
    shift = 0.5 * spread

    def fit(f, lo, hi, deg):
        t = np.cos(np.pi * (np.arange(64) + 0.5) / 64) * (hi - lo) / 2 + (hi + lo) / 2
        return np.polynomial.polynomial.polyfit(t, f(t), deg)

    ce = fit(np.exp, -spread / 2 ** rounds, 0.0, degree)
    exp_in_z = ce / (2.0 ** rounds) ** np.arange(degree + 1)
    pv = np.polynomial.polynomial.polyval
    u = pv(S - shift, exp_in_z)
    rs = []
    for _ in range(rounds):
        s = (u * u).sum(2)
        c = fit(lambda t: 1.0 / np.sqrt(t), s.min() / 1.3, s.max() * 1.3, degree)
        rs.append(c)
        u = (pv(s, c)[:, :, None] * u) ** 2
    out_clear = np.einsum("hij,jhd->ihd", u, V)
    e = np.exp(S - S.max(2, keepdims=True))
    out_true = np.einsum("hij,jhd->ihd", e / e.sum(2, keepdims=True), V)
    return dict(Q=Q, K=K, V=V, S=S, shift=shift, exp_coeffs=exp_in_z, rsqrt_coeffs=np.stack(rs), probs_clear=u, out_clear=out_clear,
                out_true=out_true)
