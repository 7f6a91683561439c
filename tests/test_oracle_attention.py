"""Pins for the checker's attention in the diagonal-block layout: the layout's index structure in the clear (every
query meets every key exactly once; rotations as array rolls), the score ciphertexts against Q K^T, and the whole block
(scores, Softmax by doubling over rows spread across ciphertexts, probability x value) against the same pipeline in the
clear (tight) and against plain Softmax attention (as good as the synthetic polynomials)."""
import numpy as np
import pytest

from oracle.ckks_oracle import AttnDesc
from paper_2609_12378_b200 import inputs
from tests.harness import Client, attention_case, attention_case_from, params


def _key_of(desc, n, g):
    """Key token met by slot (e, i) of score group g, from the layout's definition: the key operand holds token i + e in
    block e and is rotated left by g * diag_block token positions of the flattened (e, i) index."""
    E, Tk, Ti = desc.diag_block, desc.tokens, desc.token_inner
    e, i, h = inputs.attention_slot_index(Tk, desc.heads, E, n, Ti)
    P = Tk // Ti                                       # positions per block, token_inner tokens each
    u = (e * P + i // Ti + g * (E // Ti)) % (E * P)    # the rotation moves whole positions
    return ((u % P) * Ti + i % Ti + u // P) % Tk, i, h


@pytest.mark.parametrize("tokens,heads,E,n,Ti", [(8, 1, 4, 512, 1), (16, 2, 4, 512, 1), (8, 1, 8, 512, 1), (128, 32, 8, 32768, 1), (16, 4, 1, 64, 1),
                                                 (16, 8, 4, 512, 4), (16, 8, 4, 512, 2), (128, 32, 8, 32768, 8)])
def test_layout_meets_every_key_once_and_rolls_agree(tokens, heads, E, n, Ti):
    desc = AttnDesc(tokens, heads, E, 1, Ti)
    g0 = inputs.rng(5, tokens)
    Q = g0.integers(1, 50, (tokens, heads, 2)).astype(np.float64)
    K = g0.integers(1, 50, (tokens, heads, 2)).astype(np.float64)
    Qs, Ks, _ = inputs.pack_attention_operands(Q, K, K, E, n, Ti)
    R = n // (E * tokens * heads)
    seen = np.zeros((tokens, heads, tokens), dtype=np.int64)
    for g in range(desc.groups()):
        key, i, h = _key_of(desc, n, g)
        # the rotation as an array roll: left by g * E tokens = g * E * heads * R slots
        prod = (Qs * np.roll(Ks, -g * E * heads * R, axis=1)).sum(0)
        want = (Q[i, h, :] * K[key, h, :]).sum(1)
        assert np.array_equal(prod, want)
        np.add.at(seen, (i[::R], h[::R], key[::R]), 1)
    assert (seen == 1).all()          # the score row of (query i, head h) holds every key exactly once


def _keys(cl, o, desc):
    tok, lad = o.attention_rotations(desc)
    return {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in tok + lad}


def _unpack_rows(desc, n, vals_by_group):
    """[groups][n] slot values -> [tokens][heads][tokens (key)] using the layout's definition."""
    out = np.full((desc.tokens, desc.heads, desc.tokens), np.nan)
    for g, vals in enumerate(vals_by_group):
        key, i, h = _key_of(desc, n, g)
        out[i, h, key] = vals
    return out


@pytest.mark.parametrize("tokens,heads,E,dim,seed", [(8, 1, 4, 8, 81), (16, 2, 4, 4, 82)])
def test_attention_against_clear_pipeline_and_softmax_attention(tokens, heads, E, dim, seed):
    P = params(10, 13, 4, 4)
    o = P.oracle
    cl = Client(P, seed)
    desc = AttnDesc(tokens, heads, E)
    level, scale, rounds = 13, 2.0 ** 50, 1
    c = attention_case(seed, tokens, heads, dim, dim, rounds)
    Qs, Ks, Vs = inputs.pack_attention_operands(c["Q"], c["K"], c["V"], E, P.n)
    q = np.stack([cl.encrypt_slots(z, scale, level) for z in Qs])
    k = np.stack([cl.encrypt_slots(z, scale, level) for z in Ks])
    v = np.stack([cl.encrypt_slots(z, scale, level) for z in Vs])
    rlk, keys = cl.relin_key(), _keys(cl, o, desc)
    # scores: slot (e, i, h) of group g is Q[i, h] . K[key, h]
    S = o.attention_scores(desc, q, k, rlk, keys)
    ss = scale * scale / float(P.q[level - 1])
    rows = _unpack_rows(desc, P.n, [cl.decrypt_slots(S[g], ss).real for g in range(desc.groups())])
    assert np.abs(rows - c["S"].transpose(1, 0, 2)).max() < 2.0 ** -20
    # Softmax over rows spread across the groups
    Pr, sp = o.softmax_rows(desc, S, ss, c["shift"], rounds, c["exp_coeffs"], c["rsqrt_coeffs"], rlk, keys)
    assert Pr.shape[2] == level - 1 - 3 - rounds * 6
    probs = _unpack_rows(desc, P.n, [cl.decrypt_slots(Pr[g], sp).real for g in range(desc.groups())])
    assert np.abs(probs - c["probs_clear"].transpose(1, 0, 2)).max() < 2.0 ** -20
    assert np.abs(probs.sum(2) - 1.0).max() < 0.1
    # probability x value, and the three steps in one call give the same integers
    out = o.attention_values(desc, Pr, v, rlk, keys)
    whole, so = o.attention(desc, q, k, v, scale, scale, c["shift"], rounds, c["exp_coeffs"], c["rsqrt_coeffs"], rlk, keys)
    assert np.array_equal(out, whole) and out.shape[2] == Pr.shape[2] - 1
    e, i, h = inputs.attention_slot_index(tokens, heads, E, P.n)
    for d in range(dim):
        got = cl.decrypt_slots(out[d], so).real
        assert np.abs(got - c["out_clear"][i, h, d]).max() < 2.0 ** -19       # every block e holds the output (query layout)
        assert np.abs(got - c["out_true"][i, h, d]).max() < 0.05


def test_single_group_needs_no_token_rotation_and_one_block_no_ladder():
    P = params(10, 4, 2, 2)
    o = P.oracle
    assert o.attention_rotations(AttnDesc(8, 1, 8)) == ([], [8 * 1 * 8 * k for k in (1, 2, 4)])
    assert o.attention_rotations(AttnDesc(16, 4, 1)) == ([g * 4 * 8 for g in range(1, 16)], [])
    with pytest.raises(ValueError):
        o.attention_rotations(AttnDesc(8, 1, 3))


@pytest.mark.parametrize("tokens,heads,E,dim,Gb,seed", [(16, 2, 4, 4, 2, 83), (16, 1, 2, 4, 4, 84), (16, 2, 4, 4, 4, 85)])
def test_scores_with_split_groups_hold_the_same_slots(tokens, heads, E, dim, Gb, seed):
    """The baby-step / giant-step split of the score groups: the same slot values as Q K^T and as the unsplit schedule
    (other integers), the rotation set it asks for, and the query operand's right rotation being a query operand again."""
    P = params(10, 6, 2, 3)
    o = P.oracle
    cl = Client(P, seed)
    plain, split = AttnDesc(tokens, heads, E), AttnDesc(tokens, heads, E, Gb)
    tok, lad = o.attention_rotations(split)
    assert (tok, lad) == o.attention_rotations(plain)
    G, R = split.groups(), P.n // (E * tokens * heads)
    neg = o.attention_query_rotations(split)
    assert neg == [-g1 * Gb * E * heads * R for g1 in range(1, G // Gb)] and o.attention_query_rotations(plain) == []
    level, scale = 6, 2.0 ** 50
    c = attention_case(seed, tokens, heads, dim, dim, 1)
    Qs, Ks, _ = inputs.pack_attention_operands(c["Q"], c["K"], c["V"], E, P.n)
    # in the clear: rolling a query operand to the right by s group steps gives the query operand of the tokens shifted by s E
    for g1 in range(1, G // Gb):
        Qshift = np.roll(c["Q"], g1 * Gb * E, axis=0)
        Qs2, _, _ = inputs.pack_attention_operands(Qshift, c["K"], c["V"], E, P.n)
        assert np.array_equal(np.roll(Qs, -neg[g1 - 1], axis=1), Qs2)
    q = np.stack([cl.encrypt_slots(z, scale, level) for z in Qs])
    k = np.stack([cl.encrypt_slots(z, scale, level) for z in Ks])
    rlk = cl.relin_key()
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in tok + neg}
    S = o.attention_scores(split, q, k, rlk, keys)
    S0 = o.attention_scores(plain, q, k, rlk, keys)
    assert S.shape == S0.shape
    for g in range(Gb):
        assert np.array_equal(S[g], S0[g])                 # groups without a giant step are the unsplit schedule's
    if G > Gb:
        assert not np.array_equal(S[Gb], S0[Gb])
    else:
        assert np.array_equal(S, S0)                      # a single giant step: nothing is rotated back
    ss = scale * scale / float(P.q[level - 1])
    rows = _unpack_rows(split, P.n, [cl.decrypt_slots(S[g], ss).real for g in range(G)])
    assert np.abs(rows - c["S"].transpose(1, 0, 2)).max() < 2.0 ** -20
    rows0 = _unpack_rows(plain, P.n, [cl.decrypt_slots(S0[g], ss).real for g in range(G)])
    assert np.abs(rows - rows0).max() < 2.0 ** -22
    with pytest.raises(ValueError):
        o.attention_query_rotations(AttnDesc(tokens, heads, E, 3))


@pytest.mark.parametrize("tokens,heads,E,Ti,dim,seed", [(16, 8, 4, 4, 3, 91), (16, 8, 4, 2, 2, 92), (16, 8, 4, 1, 2, 93), (32, 16, 1, 1, 2, 94)])
def test_pack_and_unpack_against_the_clear_layouts(tokens, heads, E, Ti, dim, seed):
    """Token-shard ciphertexts in channel-major feature order -> attention operands -> back: every operand decrypts to the
    clear packing of the same tokens (query: every block alike; key: token i + e in block e), the way back to the shards'
    slots, and the rotation sets are the block moves and token shifts the layout's index arithmetic gives."""
    P = params(10, 6, 2, 3)
    o = P.oracle
    cl = Client(P, seed)
    desc = AttnDesc(tokens, heads, E, 1, Ti)
    D = P.n // (heads * Ti)                                  # channels a shard ciphertext holds
    g0 = inputs.rng(seed, 3)
    X = g0.uniform(-1.0, 1.0, (tokens, heads, D))
    shards = inputs.pack_channel_major_shards(X, Ti, P.n)
    level, scale = 6, 2.0 ** 40
    cts = np.stack([cl.encrypt_slots(z, scale, level) for z in shards])
    Qs, Ks, _ = inputs.pack_attention_operands(X[:, :, :dim], X[:, :, :dim], X[:, :, :dim], E, P.n, Ti)
    B, Pp = heads * Ti, tokens // Ti
    move, lad = o.attention_pack_rotations(desc, 0, dim)
    assert move == [-c * B for c in range(1, Pp)] + [d * B for d in range(1, dim)] and lad == o.attention_rotations(desc)[1]
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in move + lad}
    q = o.attention_pack(desc, 0, cts, dim, keys)
    assert q.shape == (dim, 2, level - 1, P.N)
    for d in range(dim):
        assert np.abs(cl.decrypt_slots(q[d], scale).real - Qs[d]).max() < 2.0 ** -20
    move1, dbl, shift = o.attention_pack_rotations(desc, 1, dim)
    assert move1 == move and dbl == ([-Pp * B] if E > 1 else []) and len(shift) == E and shift[0] == (0, None)
    more = [r for pair in shift for r in pair if r] + dbl
    keys.update({o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in more})
    k = o.attention_pack(desc, 1, cts, dim, keys)
    assert k.shape == (dim, 2, level - (2 if E > 1 else 1), P.N)
    for d in range(dim):
        assert np.abs(cl.decrypt_slots(k[d], scale).real - Ks[d]).max() < 2.0 ** -20
    # back: the query layout is the attention output's
    back = o.attention_unpack_rotations(desc, dim)
    assert back == [-d * B for d in range(1, dim)] + [c * B for c in range(1, Pp)]
    keys.update({o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in back})
    Y = o.attention_unpack(desc, q, keys)
    assert Y.shape == (Pp, 2, level - 2, P.N)
    keep = np.arange(P.n) < dim * B                           # the channels that were carried along
    for c in range(Pp):
        got = cl.decrypt_slots(Y[c], scale).real
        assert np.abs(got - shards[c] * keep).max() < 2.0 ** -20
    with pytest.raises(ValueError):
        o.attention_pack_rotations(AttnDesc(tokens, heads // 2, E, 1, Ti), 0, dim)     # trailing copies: not supported


def test_attention_from_packed_shards_is_softmax_attention():
    """Projection-layout shards of Q, K, V -> operands -> scores, Softmax over the rows, values -> shards again: the decrypted
    result is the clear pipeline's attention output in the shards' slots."""
    tokens, heads, E, Ti, dim, seed = 16, 8, 4, 4, 2, 95
    P = params(10, 16, 4, 4)
    o = P.oracle
    cl = Client(P, seed)
    desc = AttnDesc(tokens, heads, E, 1, Ti)
    D = P.n // (heads * Ti)
    c = attention_case(seed, tokens, heads, dim, dim, 1)
    level, scale = 16, 2.0 ** 50
    def shards_of(A):
        full = np.zeros((tokens, heads, D)); full[:, :, :dim] = A
        return np.stack([cl.encrypt_slots(z, scale, level) for z in inputs.pack_channel_major_shards(full, Ti, P.n)])
    rots = set(o.attention_rotations(desc)[0] + o.attention_rotations(desc)[1] + o.attention_pack_rotations(desc, 0, dim)[0] + o.attention_unpack_rotations(desc, dim))
    _, dbl, shift = o.attention_pack_rotations(desc, 1, dim)
    rots |= set(dbl) | {r for pair in shift for r in pair if r}
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in rots}
    rlk = cl.relin_key()
    q = o.attention_pack(desc, 0, shards_of(c["Q"]), dim, keys)[:, :, :level - 2]         # down to the key operands' level
    k = o.attention_pack(desc, 1, shards_of(c["K"]), dim, keys)
    v = o.attention_pack(desc, 1, shards_of(c["V"]), dim, keys)
    out, so = o.attention(desc, np.ascontiguousarray(q), k, v, scale, scale, c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], rlk, keys)
    Y = o.attention_unpack(desc, out, keys)
    want = np.zeros((tokens, heads, D)); want[:, :, :dim] = c["out_clear"]
    want = inputs.pack_channel_major_shards(want, Ti, P.n)
    for cc in range(tokens // Ti):
        assert np.abs(cl.decrypt_slots(Y[cc], so).real - want[cc]).max() < 2.0 ** -18


def layer_attention_case(seed: int, tokens: int, heads: int, T: int, n: int):
    """Synthetic attention block of a decoder layer in the projections' layout: X [tokens][hidden], W_q, W_k, W_v with their
    output columns in channel-major order d * heads + h, W_o with its input rows in that order; the clear pipeline's
    result Z = attention(X W_q, X W_k, X W_v) W_o with the Softmax by doubling of attention_case_from."""
    D = n // (heads * T)
    hidden = heads * D
    g = inputs.rng(seed, 13)
    X = g.uniform(-1.0, 1.0, (tokens, hidden))
    W = {k: g.normal(0.0, 1.0 / np.sqrt(hidden), (hidden, hidden)) for k in "qkvo"}
    split = lambda A: A.reshape(tokens, D, heads).transpose(0, 2, 1)          # [tokens][d * heads + h] -> [tokens][heads][D]
    S = np.einsum("ihd,jhd->hij", split(X @ W["q"]), split(X @ W["k"]))
    W["q"] = W["q"] * (1.9 / np.abs(S).max())                                 # scores within +- 2 (the 1/sqrt(dim) of the model)
    c = attention_case_from(split(X @ W["q"]), split(X @ W["k"]), split(X @ W["v"]), 1)
    Yf = c["out_clear"].transpose(0, 2, 1).reshape(tokens, hidden)
    return X, W, c, Yf @ W["o"]


def test_attention_block_from_projections_to_projection():
    """X -> Q, K, V projections (channel-major output columns) -> operands -> scores, Softmax, values -> shards -> output
    projection, everything in the checker: the decrypted shards hold the clear pipeline's Z = attention(X W_q, X W_k, X W_v) W_o."""
    from oracle.ckks_oracle import ProjDesc
    tokens, heads, E, T, seed = 16, 8, 4, 4, 96
    P = params(10, 18, 6, 3)
    o = P.oracle
    cl = Client(P, seed)
    desc = AttnDesc(tokens, heads, E, 1, T)
    D = P.n // (heads * T)
    hidden, C_ = heads * D, tokens // T
    X, W, c, Z = layer_attention_case(seed, tokens, heads, T, P.n)
    level, scale = 18, 2.0 ** 50
    pd = ProjDesc(hidden, hidden, T, C_, 8)
    rots = set(o.proj_rotations(pd)) | set(sum(o.attention_rotations(desc), [])) | set(o.attention_pack_rotations(desc, 0, D)[0]) | set(o.attention_unpack_rotations(desc, D))
    _, dbl, shift = o.attention_pack_rotations(desc, 1, D)
    rots |= set(dbl) | {r for pair in shift for r in pair if r}
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in rots}
    rlk = cl.relin_key()
    x = np.stack([cl.encrypt_slots(z, scale, level) for z in inputs.pack_feature_major(X, T, P.n)])
    proj = {k: o.linear_proj(pd, x, W[k], keys, scale) for k in "qkv"}
    for k in "qkv":
        assert proj[k][1] == scale
    q = np.ascontiguousarray(o.attention_pack(desc, 0, proj["q"][0], D, keys)[:, :, :level - 3])
    kk = o.attention_pack(desc, 1, proj["k"][0], D, keys)
    v = o.attention_pack(desc, 1, proj["v"][0], D, keys)
    out, so = o.attention(desc, q, kk, v, scale, scale, c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], rlk, keys)
    Y = o.attention_unpack(desc, out, keys)
    z, sz = o.linear_proj(pd, Y, W["o"], keys, so)
    assert z.shape[2] == level - 16
    want = inputs.pack_feature_major(Z, T, P.n)
    for cc in range(C_):
        assert np.abs(cl.decrypt_slots(z[cc], sz).real - want[cc]).max() < 2.0 ** -14
