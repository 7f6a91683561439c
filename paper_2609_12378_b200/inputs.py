"""Seeded synthetic input generators shared by the tests and the benchmark.

This module holds none of the scheme's arithmetic: it only produces the
*inputs* that both the CUDA library and the CPU checker are given -- the prime
chain (a parameter of the scheme, chosen by a stated rule), uniform residues,
activations, weights, and the raw random draws (ternary secrets, rounded
Gaussian errors, uniform masks) that key generation and encryption consume.

It imports neither the CUDA binding nor the CPU checker.
"""
from __future__ import annotations

import numpy as np

# ---------------------------------------------------------------------------
# Prime chain: the L+K largest primes below 2^50 that are 1 mod 2N.  The K
# largest are the special primes p_0 > p_1 > ...; the rest, in descending
# order, are the ciphertext primes q_0 > q_1 > ...
# ---------------------------------------------------------------------------

_MR_BASES = (2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37)  # deterministic below 3.3e24


def is_prime(n: int) -> bool:
    """Deterministic Miller-Rabin for n < 3.3e24."""
    if n < 2:
        return False
    for b in _MR_BASES:
        if n % b == 0:
            return n == b
    d, s = n - 1, 0
    while d % 2 == 0:
        d //= 2
        s += 1
    for a in _MR_BASES:
        x = pow(a, d, n)
        if x in (1, n - 1):
            continue
        for _ in range(s - 1):
            x = x * x % n
            if x == n - 1:
                break
        else:
            return False
    return True


def ntt_primes(log_n: int, count: int, bits: int = 50) -> list[int]:
    """The `count` largest primes r < 2^bits with r = 1 (mod 2N), descending."""
    m = 2 << log_n
    r = ((1 << bits) - 1) // m * m + 1
    if r >= (1 << bits):
        r -= m
    out: list[int] = []
    while len(out) < count:
        if is_prime(r):
            out.append(r)
        r -= m
        if r <= (1 << (bits - 1)):
            raise ValueError("ran out of primes")
    return out


def prime_chain(log_n: int, num_q: int, num_p: int, bits: int = 50):
    """(q, p) as uint64 arrays: p = the num_p largest primes, q = the next num_q."""
    r = ntt_primes(log_n, num_q + num_p, bits)
    p = np.array(r[:num_p], dtype=np.uint64)
    q = np.array(r[num_p:], dtype=np.uint64)
    return q, p


# ---------------------------------------------------------------------------
# Random draws
# ---------------------------------------------------------------------------

def rng(seed: int, stream: int = 0) -> np.random.Generator:
    """Independent seeded stream (Philox counter-based generator)."""
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def uniform_residues(g: np.random.Generator, primes, n: int, batch: int = 1) -> np.ndarray:
    """[batch][len(primes)][n] uint64, limb i uniform in [0, primes[i])."""
    primes = [int(x) for x in primes]
    out = np.empty((batch, len(primes), n), dtype=np.uint64)
    for i, q in enumerate(primes):
        out[:, i, :] = g.integers(0, q, size=(batch, n), dtype=np.uint64)
    return out


def ternary(g: np.random.Generator, n: int) -> np.ndarray:
    """iid uniform {-1,0,1} as int64."""
    return g.integers(-1, 2, size=n, dtype=np.int64)


def rounded_gaussian(g: np.random.Generator, shape, sigma: float = 3.2, bound: int = 19) -> np.ndarray:
    """rint(N(0, sigma^2)), resampled while |e| > bound, as int64."""
    e = np.rint(g.normal(0.0, sigma, size=shape)).astype(np.int64)
    bad = np.abs(e) > bound
    while bad.any():
        e[bad] = np.rint(g.normal(0.0, sigma, size=int(bad.sum()))).astype(np.int64)
        bad = np.abs(e) > bound
    return e


def activations_uniform(g: np.random.Generator, tokens: int, features: int) -> np.ndarray:
    """[tokens][features] fp64 iid U[-1,1]."""
    return g.uniform(-1.0, 1.0, size=(tokens, features))


def activations_normal(g: np.random.Generator, tokens: int, features: int) -> np.ndarray:
    """[tokens][features] fp64 iid N(0,1)."""
    return g.normal(0.0, 1.0, size=(tokens, features))


def weights_normal(g: np.random.Generator, d_in: int, d_out: int, std: float = 0.02) -> np.ndarray:
    """[d_in][d_out] fp64 iid N(0, std^2), row-major."""
    return g.normal(0.0, std, size=(d_in, d_out))


def pack_feature_major(x: np.ndarray, tokens_per_shard: int, slots: int) -> np.ndarray:
    """Lay activations x[tokens][features] out as token-shard slot vectors.

    Shard c holds tokens c*T .. c*T+T-1; slot index = f*T + t (feature major,
    token minor).  When features*T < slots the block is repeated to fill the
    slot vector, so that a slot rotation by k*T is a cyclic feature rotation.
    Returns [nshards][slots] fp64.  Pure data movement.
    """
    tokens, feats = x.shape
    T = tokens_per_shard
    assert tokens % T == 0 and slots % (feats * T) == 0
    ns = tokens // T
    out = np.empty((ns, slots), dtype=np.float64)
    for c in range(ns):
        blk = x[c * T:(c + 1) * T, :].T.reshape(-1)          # [f][t] flattened
        out[c] = np.tile(blk, slots // (feats * T))
    return out


def attention_slot_index(tokens: int, heads: int, diag_block: int, slots: int, token_inner: int = 1):
    """Index arrays (e, i, h) of every slot of the attention operand layout:
        slot = ((((e * P + pos) * heads + h) * token_inner + t) * R + r,   token i = pos * token_inner + t,
    P = tokens / token_inner positions per block, R = slots / (diag_block * tokens * heads) trailing copies.  token_inner = 1
    puts a token's heads side by side; token_inner = T keeps T consecutive tokens innermost, as the projections' token-shard
    layout does.  Pure index arithmetic."""
    E, Tk, H, Ti = diag_block, tokens, heads, token_inner
    assert slots % (E * Tk * H) == 0 and Tk % E == 0 and E % Ti == 0 and Tk % Ti == 0
    R = slots // (E * Tk * H)
    s = np.arange(slots) // R
    t = s % Ti; s = s // Ti
    h = s % H; s = s // H
    P = Tk // Ti
    return s // P, (s % P) * Ti + t, h


def pack_attention_operands(Q: np.ndarray, K: np.ndarray, V: np.ndarray, diag_block: int, slots: int, token_inner: int = 1):
    """Lay Q, K [tokens][heads][dim] and V [tokens][heads][dim_v] out as one slot vector per channel in the attention
    operand layout (slot index as in attention_slot_index): the query operand repeats Q[i, h, d] in every block e, the
    key and value operands hold token (i + e) mod tokens in block e, so that block e of a product lines query i up with
    key i + e.  Returns (Qs [dim][slots], Ks [dim][slots], Vs [dim_v][slots]).  Pure data movement."""
    tokens, heads, _ = Q.shape
    e, i, h = attention_slot_index(tokens, heads, diag_block, slots, token_inner)
    Qs = np.ascontiguousarray(Q[i, h, :].T)
    Ks = np.ascontiguousarray(K[(i + e) % tokens, h, :].T)
    Vs = np.ascontiguousarray(V[(i + e) % tokens, h, :].T)
    return Qs, Ks, Vs


def pack_channel_major_shards(X: np.ndarray, tokens_per_shard: int, slots: int) -> np.ndarray:
    """Lay X [tokens][heads][dim] out as token-shard slot vectors with the features in channel-major order:
    shard c holds tokens c*T .. c*T+T-1, slot = (d * heads + h) * T + t, which must fill the slots exactly.
    Returns [tokens / T][slots].  Pure data movement (pack_feature_major with feature index d * heads + h)."""
    tokens, heads, dim = X.shape
    assert dim * heads * tokens_per_shard == slots
    return pack_feature_major(np.ascontiguousarray(X.transpose(0, 2, 1)).reshape(tokens, dim * heads), tokens_per_shard, slots)
