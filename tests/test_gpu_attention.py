"""GPU parity: attention in the diagonal-block layout (scores, Softmax over rows spread across ciphertexts, probability x
value), every output limb bit-exact against the CPU checker's compositions, stage by stage and in one call."""
import numpy as np
import pytest

from oracle.ckks_oracle import AttnDesc
from paper_2609_12378_b200 import binding, inputs
from tests.harness import Client, attention_case, params

pytestmark = pytest.mark.gpu


def _setup(log_n, L, K, dnum, level, tokens, heads, E, dim, dim_v, seed, rounds=1, Gb=1):
    from tests.gpu_util import context, ct_dev, key_dev
    P, ctx = params(log_n, L, K, dnum), context(log_n, L, K, dnum)
    o = P.oracle
    cl = Client(P, seed)
    desc = AttnDesc(tokens, heads, E, Gb)
    scale = 2.0 ** 50
    c = attention_case(seed, tokens, heads, dim, dim_v, rounds)
    Qs, Ks, Vs = inputs.pack_attention_operands(c["Q"], c["K"], c["V"], E, P.n)
    q = np.stack([cl.encrypt_slots(z, scale, level) for z in Qs])
    k = np.stack([cl.encrypt_slots(z, scale, level) for z in Ks])
    v = np.stack([cl.encrypt_slots(z, scale, level) for z in Vs])
    tok, lad = o.attention_rotations(desc)
    neg = o.attention_query_rotations(desc)
    assert ctx.attention_rotations(tokens, heads, E, Gb) == tok + lad + neg
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in tok + lad + neg}
    rlk = cl.relin_key()
    dev = dict(q=[ct_dev(x, scale) for x in q], k=[ct_dev(x, scale) for x in k], v=[ct_dev(x, scale) for x in v],
               rlk=key_dev(rlk, 0), keys=[key_dev(kk, ge) for ge, kk in keys.items()])
    return P, ctx, o, cl, desc, c, scale, q, k, v, rlk, keys, dev


@pytest.mark.parametrize("log_n,L,K,dnum,level,tokens,heads,E,dim,dim_v", [
    (10, 13, 4, 4, 13, 8, 1, 4, 8, 8),        # one head, two groups of four diagonals
    (10, 13, 4, 4, 13, 16, 2, 4, 4, 3),       # two heads, four groups
    (10, 13, 4, 4, 12, 8, 2, 8, 2, 2),        # a single group: no token rotation, ladder of three; level below L
    (10, 13, 4, 4, 13, 16, 4, 1, 2, 1),       # one diagonal per ciphertext: sixteen groups, no ladder
])
def test_attention_stages_bit_exact(log_n, L, K, dnum, level, tokens, heads, E, dim, dim_v):
    from tests.gpu_util import host
    P, ctx, o, cl, desc, c, scale, q, k, v, rlk, keys, dev = _setup(log_n, L, K, dnum, level, tokens, heads, E, dim, dim_v, 600 + tokens + heads + E)
    a = (tokens, heads, E)
    ss = scale * scale / float(P.q[level - 1])
    S = o.attention_scores(desc, q, k, rlk, keys)
    dS = ctx.attention_scores(dev["q"], dev["k"], dev["rlk"], dev["keys"], *a)
    assert len(dS) == desc.groups()
    for g in range(desc.groups()):
        assert dS[g].scale == ss and dS[g].level == level - 1
        assert np.array_equal(host(dS[g].data), S[g]), g
    Pr, sp = o.softmax_rows(desc, S, ss, c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], rlk, keys)
    dP = ctx.softmax_rows(dS, c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], dev["rlk"], dev["keys"], *a)
    for g in range(desc.groups()):
        assert dP[g].scale == sp and dP[g].level == Pr.shape[2]
        assert np.array_equal(host(dP[g].data), Pr[g]), g
    out = o.attention_values(desc, Pr, v, rlk, keys)
    dO = ctx.attention_values(dP, dev["v"], dev["rlk"], dev["keys"], *a)
    for d in range(dim_v):
        assert np.array_equal(host(dO[d].data), out[d]), d
    # the three steps in one call: the same integers, and the decrypted outputs are Softmax attention
    whole = ctx.attention(dev["q"], dev["k"], dev["v"], c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], dev["rlk"], dev["keys"], *a)
    assert ctx.device_status() == binding.OK
    e, i, h = inputs.attention_slot_index(tokens, heads, E, P.n)
    for d in range(dim_v):
        assert whole[d].scale == dO[d].scale
        arr = host(whole[d].data)
        assert np.array_equal(arr, out[d]), d
        got = cl.decrypt_slots(arr, whole[d].scale).real
        assert np.abs(got - c["out_clear"][i, h, d]).max() < 2.0 ** -19
        assert np.abs(got - c["out_true"][i, h, d]).max() < 0.05


@pytest.mark.parametrize("tokens,heads,E,dim,Gb", [(16, 2, 4, 3, 2), (16, 4, 1, 2, 4), (16, 1, 2, 2, 8), (8, 2, 4, 2, 2)])
def test_attention_scores_with_split_groups_bit_exact(tokens, heads, E, dim, Gb):
    """The score groups split into baby and giant steps (rotated queries, one rotation back per group): every limb equals
    the checker's, the whole block in one call too, and a workspace short of the full size is refused."""
    import ctypes as C

    import torch

    from tests.gpu_util import host
    level = 13
    P, ctx, o, cl, desc, c, scale, q, k, v, rlk, keys, dev = _setup(10, 13, 4, 4, level, tokens, heads, E, dim, 1, 700 + tokens + E + Gb, Gb=Gb)
    a = (tokens, heads, E)
    S = o.attention_scores(desc, q, k, rlk, keys)
    dS = ctx.attention_scores(dev["q"], dev["k"], dev["rlk"], dev["keys"], *a, group_baby=Gb)
    ss = scale * scale / float(P.q[level - 1])
    for g in range(desc.groups()):
        assert dS[g].scale == ss and dS[g].level == level - 1
        assert np.array_equal(host(dS[g].data), S[g]), g
    want, so = o.attention(desc, q, k, v, scale, scale, c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], rlk, keys)
    got = ctx.attention(dev["q"], dev["k"], dev["v"], c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], dev["rlk"], dev["keys"], *a, group_baby=Gb)
    assert ctx.device_status() == binding.OK
    e, i, h = inputs.attention_slot_index(tokens, heads, E, P.n)
    assert got[0].scale == so and np.array_equal(host(got[0].data), want[0])
    assert np.abs(cl.decrypt_slots(host(got[0].data), so).real - c["out_clear"][i, h, 0]).max() < 2.0 ** -19
    d = binding.CAttnDesc(*a, Gb)
    need = binding.load().ckks_attention_scores_workspace_bytes(ctx._h, C.byref(d), level, dim)
    with pytest.raises(binding.CkksError) as err:
        ctx.attention_scores(dev["q"], dev["k"], dev["rlk"], dev["keys"], *a, ws=torch.empty(need - 256, dtype=torch.uint8, device="cuda"), group_baby=Gb)
    assert err.value.code == binding.ERR_WORKSPACE
    if desc.groups() > Gb:
        with pytest.raises(binding.CkksError) as err:
            ctx.attention_scores(dev["q"], dev["k"], dev["rlk"], dev["keys"][:-1], *a, group_baby=Gb)   # a query rotation's key is missing
        assert err.value.code == binding.ERR_NO_KEY
    with pytest.raises(binding.CkksError) as err:
        ctx.attention_rotations(tokens, heads, E, 3)
    assert err.value.code == binding.ERR_UNSUPPORTED


def test_attention_scores_in_passes_and_errors():
    """A workspace that holds one group's rotated operands at a time gives the same scores; missing keys, short
    workspaces, shapes that do not tile the slots and operands at different levels are refused before any launch."""
    import torch

    from tests.gpu_util import host
    P, ctx, o, cl, desc, c, scale, q, k, v, rlk, keys, dev = _setup(10, 13, 4, 4, 5, 16, 2, 4, 3, 1, 640)
    a = (16, 2, 4)
    full = ctx.attention_scores(dev["q"], dev["k"], dev["rlk"], dev["keys"], *a)
    lib = binding.load()
    import ctypes as C
    d = binding.CAttnDesc(*a)
    need = lib.ckks_attention_scores_workspace_bytes(ctx._h, C.byref(d), 5, 3)
    ct = 2 * 5 * P.N * 8
    small = torch.empty(need - 2 * 3 * ct, dtype=torch.uint8, device="cuda")          # room for one group's operands only
    again = ctx.attention_scores(dev["q"], dev["k"], dev["rlk"], dev["keys"], *a, ws=small)
    for x, y in zip(full, again):
        assert np.array_equal(host(x.data), host(y.data))
    launches = binding.kernel_launches()
    with pytest.raises(binding.CkksError) as e:
        ctx.attention_scores(dev["q"], dev["k"], dev["rlk"], dev["keys"][1:], *a)
    assert e.value.code == binding.ERR_NO_KEY
    with pytest.raises(binding.CkksError) as e:
        ctx.attention_scores(dev["q"], dev["k"], dev["rlk"], dev["keys"], *a, ws=torch.empty(1024, dtype=torch.uint8, device="cuda"))
    assert e.value.code == binding.ERR_WORKSPACE
    with pytest.raises(binding.CkksError) as e:
        ctx.attention_scores(dev["q"], dev["k"], dev["rlk"], dev["keys"], 16, 3, 4)        # 4 * 16 * 3 does not divide the slots
    assert e.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.CkksError) as e:
        ctx.attention_rotations(16, 2, 3)
    assert e.value.code == binding.ERR_UNSUPPORTED
    low = binding.Ciphertext(dev["k"][0].data[:, :4].contiguous(), scale)
    with pytest.raises(binding.CkksError) as e:
        ctx.attention_scores(dev["q"], [low] + dev["k"][1:], dev["rlk"], dev["keys"], *a)
    assert e.value.code == binding.ERR_LEVEL
    with pytest.raises(binding.CkksError) as e:
        ctx.softmax_rows(full, c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], dev["rlk"], dev["keys"], *a)   # 4 limbs are too few
    assert e.value.code == binding.ERR_LEVEL
    assert binding.kernel_launches() == launches


@pytest.mark.slow
def test_attention_full_ring():
    """N = 2^16 with the decoder layer's attention shape in the slots (128 tokens, 32 heads, 8 diagonals per ciphertext:
    16 groups split into 4 baby and 4 giant steps, every slot used) and a few channels: bit-exact in one call, and Softmax attention after decryption."""
    from tests.gpu_util import host
    tokens, heads, E, dim, dim_v, level, Gb = 128, 32, 8, 2, 1, 13, 4
    P, ctx, o, cl, desc, c, scale, q, k, v, rlk, keys, dev = _setup(16, 24, 8, 3, level, tokens, heads, E, dim, dim_v, 660, Gb=Gb)
    want, so = o.attention(desc, q, k, v, scale, scale, c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], rlk, keys)
    got = ctx.attention(dev["q"], dev["k"], dev["v"], c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], dev["rlk"], dev["keys"], tokens, heads, E,
                        group_baby=Gb)
    assert ctx.device_status() == binding.OK
    e, i, h = inputs.attention_slot_index(tokens, heads, E, P.n)
    for d in range(dim_v):
        assert got[d].scale == so
        arr = host(got[d].data)
        assert np.array_equal(arr, want[d]), d
        sl = cl.decrypt_slots(arr, so).real
        assert np.abs(sl - c["out_clear"][i, h, d]).max() < 2.0 ** -14
        assert np.abs(sl - c["out_true"][i, h, d]).max() < 0.05


@pytest.mark.parametrize("tokens,heads,E,Ti,dim", [(16, 8, 4, 4, 3), (16, 8, 4, 2, 2), (16, 8, 4, 1, 2), (32, 16, 1, 1, 2)])
def test_pack_and_unpack_bit_exact(tokens, heads, E, Ti, dim):
    """Token-shard ciphertexts in channel-major feature order -> query and key operands -> shards again: every limb equals the
    checker's composition, the rotation lists agree, and the operands decrypt to the clear packings."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    P, ctx = params(10, 6, 2, 3), context(10, 6, 2, 3)
    o = P.oracle
    cl = Client(P, 800 + tokens + E + Ti)
    desc = AttnDesc(tokens, heads, E, 1, Ti)
    D = P.n // (heads * Ti)
    X = inputs.rng(800 + Ti, 3).uniform(-1.0, 1.0, (tokens, heads, D))
    shards = inputs.pack_channel_major_shards(X, Ti, P.n)
    level, scale = 6, 2.0 ** 40
    cts = np.stack([cl.encrypt_slots(z, scale, level) for z in shards])
    a = (tokens, heads, E, Ti)
    move, lad = o.attention_pack_rotations(desc, 0, dim)
    _, dbl, shift = o.attention_pack_rotations(desc, 1, dim)
    back = o.attention_unpack_rotations(desc, dim)
    shifts = [r for pair in shift for r in pair if r]
    assert ctx.attention_pack_rotations(binding.ATTN_QUERY, dim, *a) == move + lad
    assert set(ctx.attention_pack_rotations(binding.ATTN_KEY_VALUE, dim, *a)) == set(move + dbl + shifts)
    assert ctx.attention_pack_rotations(binding.ATTN_TO_SHARDS, dim, *a) == back
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in set(move + lad + dbl + shifts + back)}
    dkeys = [key_dev(kk, ge) for ge, kk in keys.items()]
    dcts = [ct_dev(x, scale) for x in cts]
    Qs, Ks, _ = inputs.pack_attention_operands(X[:, :, :dim], X[:, :, :dim], X[:, :, :dim], E, P.n, Ti)
    q = o.attention_pack(desc, 0, cts, dim, keys)
    dq = ctx.attention_pack(binding.ATTN_QUERY, dcts, dim, dkeys, *a)
    k = o.attention_pack(desc, 1, cts, dim, keys)
    dk = ctx.attention_pack(binding.ATTN_KEY_VALUE, dcts, dim, dkeys, *a)
    for d in range(dim):
        assert dq[d].level == level - 1 and abs(dq[d].scale / scale - 1.0) < 1e-12
        assert np.array_equal(host(dq[d].data), q[d]), d
        assert dk[d].level == k.shape[2] and np.array_equal(host(dk[d].data), k[d]), d
        assert np.abs(cl.decrypt_slots(host(dk[d].data), scale).real - Ks[d]).max() < 2.0 ** -20
    Y = o.attention_unpack(desc, q, keys)
    dY = ctx.attention_pack(binding.ATTN_TO_SHARDS, dq, dim, dkeys, *a)
    assert len(dY) == tokens // Ti
    for c in range(tokens // Ti):
        assert np.array_equal(host(dY[c].data), Y[c]), c
    assert ctx.device_status() == binding.OK
    launches = binding.kernel_launches()
    with pytest.raises(binding.CkksError) as err:
        ctx.attention_pack(binding.ATTN_KEY_VALUE, dcts, dim, dkeys[:1], *a)
    assert err.value.code == binding.ERR_NO_KEY
    with pytest.raises(binding.CkksError) as err:
        ctx.attention_pack(binding.ATTN_QUERY, dcts, dim, dkeys, tokens, heads // 2, E, Ti)        # trailing copies
    assert err.value.code == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.CkksError) as err:
        ctx.attention_pack_rotations(binding.ATTN_QUERY, dim, tokens, heads, E, 3)
    assert err.value.code == binding.ERR_UNSUPPORTED
    assert binding.kernel_launches() == launches


@pytest.mark.slow
def test_pack_full_ring():
    """N = 2^16 with the decoder layer's shape (128 tokens in 16 shards of 8, 32 heads, 8 diagonals per ciphertext) and two
    channels: key operands from the shards bit-exact (block moves, the copy of block 0, fifteen token shifts), and back."""
    from tests.gpu_util import context, ct_dev, host, key_dev
    tokens, heads, E, Ti, dim, level = 128, 32, 8, 8, 2, 6
    P, ctx = params(16, 24, 8, 3), context(16, 24, 8, 3)
    o = P.oracle
    cl = Client(P, 880)
    desc = AttnDesc(tokens, heads, E, 1, Ti)
    D = P.n // (heads * Ti)
    X = inputs.rng(881, 3).uniform(-1.0, 1.0, (tokens, heads, D))
    shards = inputs.pack_channel_major_shards(X, Ti, P.n)
    scale = 2.0 ** 40
    cts = np.stack([cl.encrypt_slots(z, scale, level) for z in shards])
    a = (tokens, heads, E, Ti)
    rots = set(ctx.attention_pack_rotations(binding.ATTN_KEY_VALUE, dim, *a)) | set(ctx.attention_pack_rotations(binding.ATTN_TO_SHARDS, dim, *a))
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in rots}
    dkeys = [key_dev(kk, ge) for ge, kk in keys.items()]
    dcts = [ct_dev(x, scale) for x in cts]
    k = o.attention_pack(desc, 1, cts, dim, keys)
    dk = ctx.attention_pack(binding.ATTN_KEY_VALUE, dcts, dim, dkeys, *a)
    _, Ks, _ = inputs.pack_attention_operands(X[:, :, :dim], X[:, :, :dim], X[:, :, :dim], E, P.n, Ti)
    for d in range(dim):
        arr = host(dk[d].data)
        assert dk[d].level == level - 2 and np.array_equal(arr, k[d]), d
        assert np.abs(cl.decrypt_slots(arr, scale).real - Ks[d]).max() < 2.0 ** -14
    Y = o.attention_unpack(desc, k, keys)               # any ciphertexts in the operands' slots serve as input of the way back
    dY = ctx.attention_pack(binding.ATTN_TO_SHARDS, dk, dim, dkeys, *a)
    for c in (0, 7, 15):
        assert np.array_equal(host(dY[c].data), Y[c]), c
    assert ctx.device_status() == binding.OK


def test_attention_block_from_projections_to_projection_bit_exact():
    """The attention block of a decoder layer through the C ABI on a small ring: query/key/value projections in one call
    (channel-major output columns), operands, scores - Softmax - values, back to shards, output projection.  Every stage's
    limbs equal the checker's, and the decrypted result is the clear pipeline's attention(X W_q, X W_k, X W_v) W_o."""
    import torch

    from oracle.ckks_oracle import ProjDesc
    from tests.gpu_util import context, ct_dev, host, key_dev
    from tests.test_oracle_attention import layer_attention_case
    tokens, heads, E, T, seed = 16, 8, 4, 4, 96
    P, ctx = params(10, 18, 6, 3), context(10, 18, 6, 3)
    o = P.oracle
    cl = Client(P, seed)
    desc = AttnDesc(tokens, heads, E, 1, T)
    D = P.n // (heads * T)
    hidden, C_ = heads * D, tokens // T
    X, W, c, Z = layer_attention_case(seed, tokens, heads, T, P.n)
    level, scale = 18, 2.0 ** 50
    pd = ProjDesc(hidden, hidden, T, C_, 8)
    a = (tokens, heads, E, T)
    rots = set(ctx.linear_proj_rotations(hidden, hidden, T, C_, 8)) | set(ctx.attention_rotations(tokens, heads, E))
    for kind in (binding.ATTN_QUERY, binding.ATTN_KEY_VALUE, binding.ATTN_TO_SHARDS):
        rots |= set(ctx.attention_pack_rotations(kind, D, *a))
    keys = {o.galois_element(r): cl.rotation_key(o.galois_element(r)) for r in rots}
    dkeys = [key_dev(kk, ge) for ge, kk in keys.items()]
    rlk = cl.relin_key()
    drlk = key_dev(rlk, 0)
    x = np.stack([cl.encrypt_slots(z, scale, level) for z in inputs.pack_feature_major(X, T, P.n)])
    dx = [ct_dev(z, scale) for z in x]
    dW = {k: torch.tensor(W[k], dtype=torch.float64, device="cuda").contiguous() for k in "qkvo"}
    # projections
    dproj = ctx.linear_proj_multi(dx, [dW["q"], dW["k"], dW["v"]], dkeys, hidden, [hidden] * 3, T, C_, 8)
    proj = {k: o.linear_proj(pd, x, W[k], keys, scale)[0] for k in "qkv"}
    for i, k in enumerate("qkv"):
        for cc in range(C_):
            assert np.array_equal(host(dproj[i][cc].data), proj[k][cc]), (k, cc)
    # operands
    q = o.attention_pack(desc, 0, proj["q"], D, keys)
    kk = o.attention_pack(desc, 1, proj["k"], D, keys)
    v = o.attention_pack(desc, 1, proj["v"], D, keys)
    dq = ctx.attention_pack(binding.ATTN_QUERY, dproj[0], D, dkeys, *a)
    dk = ctx.attention_pack(binding.ATTN_KEY_VALUE, dproj[1], D, dkeys, *a)
    dv = ctx.attention_pack(binding.ATTN_KEY_VALUE, dproj[2], D, dkeys, *a)
    for d in range(D):
        assert np.array_equal(host(dq[d].data), q[d]) and np.array_equal(host(dk[d].data), kk[d]) and np.array_equal(host(dv[d].data), v[d]), d
    lk = dk[0].level
    dq = [binding.Ciphertext(z.data[:, :lk].contiguous(), z.scale) for z in dq]          # down to the key operands' level
    # attention
    out, so = o.attention(desc, np.ascontiguousarray(q[:, :, :lk]), kk, v, scale, scale, c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], rlk, keys)
    dout = ctx.attention(dq, dk, dv, c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], drlk, dkeys, tokens, heads, E)
    for d in range(D):
        assert np.array_equal(host(dout[d].data), out[d]), d
    # back to shards, output projection
    Y = o.attention_unpack(desc, out, keys)
    dY = ctx.attention_pack(binding.ATTN_TO_SHARDS, dout, D, dkeys, *a)
    z, sz = o.linear_proj(pd, Y, W["o"], keys, so)
    dz = ctx.linear_proj(dY, dW["o"], dkeys, hidden, hidden, T, C_, 8)
    assert ctx.device_status() == binding.OK
    want = inputs.pack_feature_major(Z, T, P.n)
    for cc in range(C_):
        arr = host(dz[cc].data)
        assert np.array_equal(host(dY[cc].data), Y[cc]) and np.array_equal(arr, z[cc]), cc
        assert np.abs(cl.decrypt_slots(arr, dz[cc].scale).real - want[cc]).max() < 2.0 ** -14


def test_lanes_do_not_change_results():
    """The attention entry points spread independent chains over the context's streams (option CKKS_OPT_LANES); one lane
    (the caller's stream only) and four give the same limbs, on the caller's stream in both cases."""
    from tests.gpu_util import host
    P, ctx, o, cl, desc, c, scale, q, k, v, rlk, keys, dev = _setup(10, 13, 4, 4, 13, 16, 2, 4, 4, 3, 641)
    a = (16, 2, 4)
    assert ctx.get_option(binding.OPT_LANES) == 4
    res = {}
    try:
        for lanes in (1, 4, 2):
            ctx.set_option(binding.OPT_LANES, lanes)
            out = ctx.attention(dev["q"], dev["k"], dev["v"], c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], dev["rlk"], dev["keys"], *a)
            res[lanes] = [host(x.data) for x in out]
    finally:
        ctx.set_option(binding.OPT_LANES, 4)
    want, _ = o.attention(desc, q, k, v, scale, scale, c["shift"], 1, c["exp_coeffs"], c["rsqrt_coeffs"], rlk, keys)
    for lanes in (1, 2, 4):
        for d in range(3):
            assert np.array_equal(res[lanes][d], want[d]), (lanes, d)
    with pytest.raises(binding.CkksError):
        ctx.set_option(binding.OPT_LANES, 5)
    assert ctx.device_status() == binding.OK
