"""GPU parity at the benchmark's full sizes (N = 2^16, L = 24, K = 8, dnum = 3) with real keys and ciphertexts.

The 128-token 4096 x 4096 projection runs in the launch configuration bench.py times (16 shards, B = G = 64,
126 rotation keys).  Every output ciphertext is decrypted and compared with X W in fp64 (bounded by the scheme's
noise), and one sampled shard is recomputed by the CPU checker and compared bit for bit (a shard's output depends
only on that shard's input).  Minutes of host time: key generation and the checker's shard."""
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
    outs = ctx.linear_proj([ct_dev(c, scale) for c in cts], dev(W), dkeys, D, D, T, S, B)
    assert ctx.device_status() == binding.OK
    Y = X @ W
    got = [host(ct.data) for ct in outs]
    worst = 0.0
    for c in range(S):
        assert outs[c].level == level - 1 and outs[c].scale == scale
        sl = cl.decrypt_slots(got[c], outs[c].scale).real.reshape(D, T)
        worst = max(worst, np.abs(sl - Y[c * T:(c + 1) * T].T).max())
    assert worst < 2.0 ** -16, worst           # two key switches, 4096-term sums and a rescale at Delta = 2^40
    # one sampled shard, bit for bit
    c = int(inputs.rng(1004, 2).integers(0, S))
    one = ProjDesc(D, D, T, 1, B)
    want, want_scale = o.linear_proj(one, cts[c][None], W, keys, scale)
    assert want_scale == outs[c].scale
    assert np.array_equal(got[c], want[0])


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
