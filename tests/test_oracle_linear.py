"""Pins for the checker's linear projection: Eq. 5 in the clear for every block
shape, the paper's object counts, and the encrypted composite against X W."""
import os

import numpy as np
import pytest

from oracle.ckks_oracle import Oracle, ProjDesc
from paper_2609_12378_b200 import inputs
from tests.harness import Client, params

GOLD = os.path.join(os.path.dirname(__file__), "golden", "paper_counts.txt")


def _gold():
    out = {}
    for line in open(GOLD):
        line = line.split("#")[0].split()
        if len(line) == 2:
            out[line[0]] = line[1]
    return out


def _clear_projection(o, desc, X, W):
    """The schedule of Oracle.linear_proj with slot vectors in the clear and rotations as rolls."""
    F, ins, outs = o.proj_blocks(desc)
    T, B = desc.tokens_per_shard, desc.baby
    A = W.T
    res = []
    for c in range(desc.nshards):
        xs = []
        for (s0, mi) in ins:
            xs.append(inputs.pack_feature_major(X[c * T:(c + 1) * T, s0:s0 + mi], T, o.n)[0])
        for (o0, mo) in outs:
            total = np.zeros(o.n)
            nds = [min(mi, mo) for (_, mi) in ins]
            for g in range(max(nds) // B):
                acc = np.zeros(o.n)
                for ib, (s0, mi) in enumerate(ins):
                    if g >= nds[ib] // B:
                        continue
                    for b in range(B):
                        d = o.diagonal(A[o0:o0 + mo, s0:s0 + mi], g * B + b, F)
                        acc += np.repeat(np.roll(d, g * B), T) * np.roll(xs[ib], -b * T)
                total += np.roll(acc, -g * B * T)
            f, mi = mo, ins[0][1]
            while f < mi:
                total = total + np.roll(total, -f * T); f *= 2
            res.append(total)
    return res


@pytest.mark.parametrize("d_in,d_out,T,log_n,B", [
    (16, 16, 4, 7, 4),      # square, F = 16
    (16, 4, 4, 7, 2),       # wide (K/V-like): m_out < F, folded
    (16, 40, 4, 7, 4),      # several output blocks + remainder 8 | 16 (gate/up-like)
    (40, 16, 4, 7, 4),      # several input blocks + input remainder (down-like)
    (8, 8, 4, 7, 2),        # block smaller than F on both sides, replicated (toy config)
])
def test_eq5_schedule_in_the_clear(d_in, d_out, T, log_n, B):
    o = Oracle(log_n, [inputs.ntt_primes(log_n, 1)[0]], [], 1)
    F = o.n // T
    g = inputs.rng(61, d_in * 100 + d_out)
    X, W = inputs.activations_normal(g, 2 * T, d_in), inputs.weights_normal(g, d_in, d_out, 1.0)
    desc = ProjDesc(d_in, d_out, T, 2, B)
    Y = X @ W
    res = _clear_projection(o, desc, X, W)
    _, ins, outs = o.proj_blocks(desc)
    for c in range(2):
        for ob, (o0, mo) in enumerate(outs):
            got = res[c * len(outs) + ob].reshape(F, T)          # [feature][token]
            for r in range(F):                                   # output replicated F/mo times
                assert np.allclose(got[r], Y[c * T:(c + 1) * T, o0 + r % mo], atol=1e-9)


def test_paper_object_counts():
    """One plaintext = one 4096-entry diagonal shared by all token shards."""
    gold = _gold()
    h, f, tokens = int(gold["hidden"]), int(gold["ffn"]), int(gold["tokens"])
    kv = 1024
    shapes = {"q": (h, h), "k": (h, kv), "v": (h, kv), "o": (h, h), "gate": (h, f), "up": (h, f), "down": (f, h)}
    P = params(16, 24, 8, 3)
    o = P.oracle
    T = 8
    assert o.n // T == h and tokens // T == 16
    total = 0
    for name, (di, do) in shapes.items():
        F, ins, outs = o.proj_blocks(ProjDesc(di, do, T, tokens // T, 64 if min(di, do) >= 2048 else 32))
        nd = sum(min(mi, mo) for (_, mi) in ins for (_, mo) in outs)
        assert nd == di * do // h
        total += nd
    assert total == 53248 and 8 * total == int(gold["plaintext_weight_objects_per_layer_thor_style"])
    # reuse across the 16 token shards is the paper's 1/16 encode ratio
    num, den = gold["encode_ratio_qkv_gate_up"].split("/")
    assert int(den) // int(num) == tokens // T


def test_rotation_counts_llama_layer():
    """Rotation counts of one decoder layer's seven projections under this schedule."""
    P = params(16, 24, 8, 3)
    o = P.oracle
    T, S = 8, 16
    shapes = [(4096, 4096, 64), (4096, 1024, 32), (4096, 1024, 32), (4096, 4096, 64),
              (4096, 14336, 64), (4096, 14336, 64), (14336, 4096, 64)]
    baby = giant = 0
    for di, do, B in shapes:
        F, ins, outs = o.proj_blocks(ProjDesc(di, do, T, S, B))
        baby += S * len(ins) * (B - 1)
        for (_, mo) in outs:
            G = max(min(mi, mo) for (_, mi) in ins) // B
            folds = {(mi // mo).bit_length() - 1 if mi > mo else 0 for (_, mi) in ins}
            giant += S * (G - 1 + folds.pop())
    assert (baby, giant) == (9056, 11152)


@pytest.mark.parametrize("d_in,d_out,T,B", [(16, 16, 32, 4), (16, 4, 32, 2), (16, 24, 32, 4), (24, 16, 32, 4), (8, 8, 32, 4)])
def test_encrypted_projection_small_ring(d_in, d_out, T, B):
    """N = 2^10 (n = 512, F = 16): decrypt(linear_proj(enc X)) = X W."""
    P = params(10, 4, 2, 2)
    o = P.oracle
    cl = Client(P, 62)
    level, scale = 4, 2.0 ** 40
    g = inputs.rng(63, d_in * 100 + d_out)
    X, W = inputs.activations_uniform(g, 2 * T, d_in), inputs.weights_normal(g, d_in, d_out, 0.05)
    desc = ProjDesc(d_in, d_out, T, 2, B)
    F, ins, outs = o.proj_blocks(desc)
    cts = []
    for c in range(2):
        for (s0, mi) in ins:
            cts.append(cl.encrypt_slots(inputs.pack_feature_major(X[c * T:(c + 1) * T, s0:s0 + mi], T, o.n)[0], scale, level))
    keys = {}
    for r in o.proj_rotations(desc):
        keys[o.galois_element(r)] = cl.rotation_key(o.galois_element(r))
    Yc, out_scale = o.linear_proj(desc, np.stack(cts), W, keys, scale)
    assert out_scale == scale and Yc.shape == (2 * len(outs), 2, level - 1, P.N)
    Y = X @ W
    for c in range(2):
        for ob, (o0, mo) in enumerate(outs):
            got = cl.decrypt_slots(Yc[c * len(outs) + ob], out_scale).real.reshape(F, T)
            for r in range(F):
                assert np.abs(got[r] - Y[c * T:(c + 1) * T, o0 + r % mo]).max() < 2.0 ** -20
    # shard independence: shard 1's output does not depend on shard 0's input
    cts2 = list(cts)
    for i in range(len(ins)):
        cts2[i] = cts[len(ins) + i]
    Yc2, _ = o.linear_proj(desc, np.stack(cts2), W, keys, scale)
    assert np.array_equal(Yc2[len(outs):], Yc[len(outs):]) and np.array_equal(Yc2[:len(outs)], Yc[len(outs):])


@pytest.mark.parametrize("d_in,d_out,T,B", [(16, 16, 32, 4), (16, 4, 32, 2), (24, 16, 32, 4), (16, 16, 32, 16)])
def test_lazy_moddown_projection(d_in, d_out, T, B):
    """Giant steps summed in the extended basis: the same plaintext result (X W) within the same bound; equal to the
    eager schedule bit for bit when there is no giant step to sum, and otherwise within one unit per residue after the
    rescale (the two differ by a few units before the division by q_last, which almost always rounds them away)."""
    P = params(10, 4, 2, 2)
    o = P.oracle
    cl = Client(P, 64)
    level, scale = 4, 2.0 ** 40
    g = inputs.rng(65, d_in * 100 + d_out)
    X, W = inputs.activations_uniform(g, T, d_in), inputs.weights_normal(g, d_in, d_out, 0.05)
    eager, lazy = ProjDesc(d_in, d_out, T, 1, B), ProjDesc(d_in, d_out, T, 1, B, lazy_moddown=True)
    F, ins, outs = o.proj_blocks(eager)
    cts = np.stack([cl.encrypt_slots(inputs.pack_feature_major(X[:, s0:s0 + mi], T, o.n)[0], scale, level) for (s0, mi) in ins])
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in o.proj_rotations(eager)}
    Ye, se = o.linear_proj(eager, cts, W, keys, scale)
    Yl, sl = o.linear_proj(lazy, cts, W, keys, scale)
    assert se == sl and Ye.shape == Yl.shape
    giants = max(min(mi, mo) for (_, mi) in ins for (_, mo) in outs) // B
    if giants == 1:
        assert np.array_equal(Ye, Yl)
    q = np.array(P.q[:level - 1], dtype=np.int64)[None, None, :, None]
    d = (Yl.astype(np.int64) - Ye.astype(np.int64)) % q
    assert np.minimum(d, q - d).max() <= 1
    Y = X @ W
    for ob, (o0, mo) in enumerate(outs):
        got = cl.decrypt_slots(Yl[ob], sl).real.reshape(F, T)
        ref = cl.decrypt_slots(Ye[ob], se).real.reshape(F, T)
        for r in range(F):
            assert np.abs(got[r] - Y[:, o0 + r % mo]).max() < 2.0 ** -20
        assert np.abs(got - ref).max() < 2.0 ** -24


def test_toy_config_projection():
    """Config 1: N = 2^13, 6+1 primes, dnum 6, 32 tokens x 64 features, 64x64 weights, B = G = 8."""
    P = params(13, 6, 1, 6)
    o = P.oracle
    cl = Client(P, 1001)
    level, scale, T = 6, 2.0 ** 40, 32
    g = inputs.rng(1001, 100)
    X, W = inputs.activations_uniform(g, 32, 64), inputs.weights_normal(g, 64, 64)
    desc = ProjDesc(64, 64, T, 1, 8)
    assert len(o.proj_rotations(desc)) == 14
    ct = cl.encrypt_slots(inputs.pack_feature_major(X, T, o.n)[0], scale, level)
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in o.proj_rotations(desc)}
    Yc, out_scale = o.linear_proj(desc, ct[None], W, keys, scale)
    got = cl.decrypt_slots(Yc[0], out_scale).real.reshape(128, T)
    Y = X @ W
    for r in range(128):
        assert np.abs(got[r] - Y[:, r % 64]).max() < 2.0 ** -20
