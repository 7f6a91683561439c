"""GPU parity at the benchmark's full sizes (N = 2^16, L = 24, K = 8, dnum = 3) with real keys and ciphertexts.

The 128-token 4096 x 4096 projection runs in the launch configuration bench.py times (16 shards, B = G = 64,
126 rotation keys).  Every output ciphertext is decrypted and compared with X W in fp64 (bounded by the scheme's
noise), and the first, the last and one seeded middle shard are recomputed by the CPU checker and compared bit for
bit (a shard's output depends only on that shard's input; every key switch is batched over the shards, so both ends of
the batch and an entry inside a chunk are covered).  The other decoder-layer shapes (key/value, gate/up, down) and the
seeded subset of the attention products run the same way.  Minutes of host time: key generation and the checker."""
import numpy as np
import pytest

from oracle.ckks_oracle import ProjDesc
from paper_2609_12378_b200 import binding, inputs
from tests.harness import Client, params

pytestmark = [pytest.mark.gpu, pytest.mark.slow]


def test_llama_shaped_projection_full_size():
    from tests.gpu_util import context, ct_dev, dev, host, key_dev
    P, ctx = params(16, 24, 8, 3), context(16, 24, 8, 3)
    o = P.oracle
    cl = Client(P, 1004)
    level, scale, T, S, B, D = 24, 2.0 ** 40, 8, 16, 64, 4096
    g = inputs.rng(1004, 1)
    X = inputs.activations_normal(g, S * T, D)
    W = inputs.weights_normal(g, D, D, 0.02)
    desc = ProjDesc(D, D, T, S, B)
    rots = o.proj_rotations(desc)
    assert len(rots) == 126 and rots == ctx.linear_proj_rotations(D, D, T, S, B)
    cts = [cl.encrypt_slots(inputs.pack_feature_major(X[c * T:(c + 1) * T], T, o.n)[0], scale, level) for c in range(S)]
    keys, dkeys = {}, []
    for r in rots:
        ge = o.galois_element(r)
        keys[ge] = cl.rotation_key(ge)
        dkeys.append(key_dev(keys[ge], ge))
    dcts = [ct_dev(c, scale) for c in cts]
    outs = ctx.linear_proj(dcts, dev(W), dkeys, D, D, T, S, B)
    assert ctx.device_status() == binding.OK
    Y = X @ W
    got = [host(ct.data) for ct in outs]
    worst = 0.0
    for c in range(S):
        assert outs[c].level == level - 1 and outs[c].scale == scale
        sl = cl.decrypt_slots(got[c], outs[c].scale).real.reshape(D, T)
        worst = max(worst, np.abs(sl - Y[c * T:(c + 1) * T].T).max())
    assert worst < 2.0 ** -16, worst           # two key switches, 4096-term sums and a rescale at Delta = 2^40
    # the first and the last shard of the batch and a seeded one in between, bit for bit (one checker call, so the
    # encoded diagonals are shared)
    c = int(inputs.rng(1004, 2).integers(1, S - 1))
    sel = [0, c, S - 1]
    some = ProjDesc(D, D, T, len(sel), B)
    want, want_scale = o.linear_proj(some, np.stack([cts[i] for i in sel]), W, keys, scale)
    for n, i in enumerate(sel):
        assert want_scale == outs[i].scale
        assert np.array_equal(got[i], want[n]), i
    # the schedule with the giant steps summed before one ModDown: all shards decrypt to X W, the same three shards
    # are the checker's lazy variant bit for bit
    lazy = ctx.linear_proj(dcts, dev(W), dkeys, D, D, T, S, B, lazy_moddown=True)
    assert ctx.device_status() == binding.OK
    for cc in range(S):
        sl = cl.decrypt_slots(host(lazy[cc].data), lazy[cc].scale).real.reshape(D, T)
        assert np.abs(sl - Y[cc * T:(cc + 1) * T].T).max() < 2.0 ** -16
    want_lazy, _ = o.linear_proj(ProjDesc(D, D, T, len(sel), B, lazy_moddown=True), np.stack([cts[i] for i in sel]), W, keys, scale)
    for n, i in enumerate(sel):
        assert np.array_equal(host(lazy[i].data), want_lazy[n]), i
    del lazy
    # the same inputs through the square and a key-shaped (4096 x 1024) matrix in one call with shared baby steps:
    # the square matrix's outputs do not change, the second matrix's decrypt to X Wk (one block, stored four times)
    Wk = inputs.weights_normal(inputs.rng(1004, 3), D, 1024, 0.02)
    both = ctx.linear_proj_multi(dcts, [dev(W), dev(Wk)], dkeys, D, [D, 1024], T, S, B)
    assert ctx.device_status() == binding.OK
    assert len(both[0]) == S and len(both[1]) == S
    for a, b in zip(both[0], got):
        assert np.array_equal(host(a.data), b)
    Yk = X @ Wk
    for cc in (0, c, S - 1):
        sl = cl.decrypt_slots(host(both[1][cc].data), both[1][cc].scale).real.reshape(D, T)
        assert np.abs(sl - np.tile(Yk[cc * T:(cc + 1) * T].T, (4, 1))).max() < 2.0 ** -16


def test_sixty_four_rotations_full_size():
    """64 rotations by 8b slots, b = 1..64: plain and hoisted, four of them bit for bit against the checker,
    all of them after decryption."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(16, 24, 8, 3), context(16, 24, 8, 3)
    o = P.oracle
    cl = Client(P, 1003)
    level, scale = 24, 2.0 ** 40
    z = inputs.rng(1003, 1).uniform(-1, 1, P.n)
    ct = cl.encrypt_slots(z, scale, level)
    dct = ct_dev(ct, scale)
    rots = [8 * b for b in range(1, 65)]
    gals = [o.galois_element(r) for r in rots]
    assert len(set(gals)) == 64
    keys = [cl.rotation_key(g) for g in gals]
    dkeys = [key_dev(k, g) for k, g in zip(keys, gals)]
    hoisted = ctx.rotate_hoisted(dct, dkeys)
    sample = [0, 17, 40, 63]
    want_h = o.rotate_hoisted(ct, [keys[i] for i in sample], [gals[i] for i in sample])
    for n, i in enumerate(sample):
        assert np.array_equal(host(hoisted[i].data), want_h[n]), i
        assert np.array_equal(host(ctx.rotate(dct, dkeys[i]).data), o.rotate(ct, keys[i], gals[i])), i
    for i, r in enumerate(rots):
        zp = cl.decrypt_slots(host(ctx.rotate(dct, dkeys[i]).data), scale).real
        zh = cl.decrypt_slots(host(hoisted[i].data), scale).real
        want = np.roll(z, -r)
        assert np.abs(zp - want).max() < 2.0 ** -17 and np.abs(zh - want).max() < 2.0 ** -17, i


def _full_ring_shape(d_in, d_out, S, B, seed, shards_checked=1, lazy=False):
    """A decoder-layer projection shape at N = 2^16, level 24: decrypt everything, recompute `shards_checked` shards."""
    from tests.gpu_util import context, ct_dev, dev, host, key_dev
    P, ctx = params(16, 24, 8, 3), context(16, 24, 8, 3)
    o = P.oracle
    cl = Client(P, seed)
    level, scale, T = 24, 2.0 ** 40, 8
    g = inputs.rng(seed, 1)
    X = inputs.activations_normal(g, S * T, d_in)
    W = inputs.weights_normal(g, d_in, d_out, 0.02)
    desc = ProjDesc(d_in, d_out, T, S, B, lazy_moddown=lazy)
    F, ins, outs_b = o.proj_blocks(desc)
    rots = o.proj_rotations(desc)
    assert rots == ctx.linear_proj_rotations(d_in, d_out, T, S, B)
    cts = []
    for c in range(S):
        for (s0, mi) in ins:
            cts.append(cl.encrypt_slots(inputs.pack_feature_major(X[c * T:(c + 1) * T, s0:s0 + mi], T, o.n)[0], scale, level))
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in rots}
    outs = ctx.linear_proj([ct_dev(c, scale) for c in cts], dev(W), [key_dev(k, ge) for ge, k in keys.items()], d_in, d_out, T, S, B,
                           lazy_moddown=lazy)
    assert ctx.device_status() == binding.OK
    Y = X @ W
    nib, nob = len(ins), len(outs_b)
    got = [host(ct.data) for ct in outs]
    for c in range(S):
        for ob, (o0, mo) in enumerate(outs_b):
            sl = cl.decrypt_slots(got[c * nob + ob], outs[c * nob + ob].scale).real.reshape(F, T)
            for r in range(0, F, 37):
                assert np.abs(sl[r] - Y[c * T:(c + 1) * T, o0 + r % mo]).max() < 2.0 ** -16, (c, ob, r)
    for c in range(shards_checked):
        one = ProjDesc(d_in, d_out, T, 1, B, lazy_moddown=lazy)
        want, _ = o.linear_proj(one, np.stack(cts[c * nib:(c + 1) * nib]), W, keys, scale)
        for ob in range(nob):
            assert np.array_equal(got[c * nob + ob], want[ob]), (c, ob)


def test_kv_projection_full_ring():
    """K / V shape: 4096 -> 1024 (wide block, folded twice), B = G = 32, giant steps summed before one ModDown."""
    _full_ring_shape(4096, 1024, 4, 32, seed=1005, lazy=True)


def test_gate_up_projection_full_ring():
    """gate / up shape: 4096 -> 14336 = 3 x 4096 + 2048 (three square output blocks and a folded remainder block)."""
    _full_ring_shape(4096, 14336, 2, 64, seed=1006)


def test_down_projection_full_ring():
    """down shape: 14336 -> 4096 (three full input blocks and a repeated remainder block summed before the giant steps)."""
    _full_ring_shape(14336, 4096, 2, 64, seed=1007, lazy=True)


def test_attention_product_batch_full_size():
    """The decoder layer's ciphertext x ciphertext work (QK^T and PV: 2048 + 2048 independent products at level 24,
    128 of them summed per output ciphertext) on a seeded subset: 64 products through the batched entry point, each
    against the checker's single product, and one sum of 128 products with a single relinearisation against the
    checker's sum, bit for bit; the first product and the sum also after decryption."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(16, 24, 8, 3), context(16, 24, 8, 3)
    o = P.oracle
    cl = Client(P, 1005)
    level, scale = 24, 2.0 ** 40
    g = inputs.rng(1005, 9)
    rlk = cl.relin_key()
    drlk = key_dev(rlk, 0)
    # 16 distinct ciphertexts on either side; product i pairs a[i % 16] with b[(5 i + 3 + i / 16) % 16], so all 64 pairs differ
    za, zb = g.uniform(-1, 1, (16, P.n)), g.uniform(-1, 1, (16, P.n))
    a = [cl.encrypt_slots(z, scale, level) for z in za]
    b = [cl.encrypt_slots(z, scale, level) for z in zb]
    da, db = [ct_dev(x, scale) for x in a], [ct_dev(x, scale) for x in b]
    ia, ib = [i % 16 for i in range(64)], [(5 * i + 3 + i // 16) % 16 for i in range(64)]
    assert len(set(zip(ia, ib))) == 64
    outs = ctx.mul_relin_batch([da[i] for i in ia], [db[j] for j in ib], drlk)
    assert ctx.device_status() == binding.OK
    for n, (i, j) in enumerate(zip(ia, ib)):
        assert outs[n].scale == scale * scale
        assert np.array_equal(host(outs[n].data), o.mul_relin(a[i], b[j], rlk)), n
    z0 = cl.decrypt_slots(host(outs[0].data), scale * scale).real
    assert np.abs(z0 - za[ia[0]] * zb[ib[0]]).max() < 2.0 ** -17
    # one output ciphertext of PV: 128 products summed, one key switch
    ja, jb = [i % 16 for i in range(128)], [(3 * i + i // 16) % 16 for i in range(128)]
    tot = ctx.mul_relin_sum([da[i] for i in ja], [db[j] for j in jb], drlk)
    assert ctx.device_status() == binding.OK
    want = o.mul_relin_sum(np.stack([a[i] for i in ja]), np.stack([b[j] for j in jb]), rlk)
    assert np.array_equal(host(tot.data), want)
    zs = cl.decrypt_slots(host(tot.data), scale * scale).real
    assert np.abs(zs - sum(za[i] * zb[j] for i, j in zip(ja, jb))).max() < 2.0 ** -17
