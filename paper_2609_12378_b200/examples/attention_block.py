"""Times the attention block of one Llama-3-8B-shaped decoder layer on 128 encrypted tokens (N = 2^16, 24 + 8 primes, dnum 3)
through the public binding, from the projections' token-shard ciphertexts to the input of the output projection:

    16 shard ciphertexts of Q, K, V (8 tokens each, features in channel-major order d * heads + h)
      -> 128 query / key / value operands, one per channel      (attention_pack)
      -> 16 score ciphertexts (groups split 4 x 4)              (attention_scores)
      -> Softmax by doubling over rows spread across them       (softmax_rows, two rounds, degree-4 polynomials)
      -> 128 output channels                                    (attention_values)
      -> 16 shard ciphertexts again                             (attention_pack, ATTN_TO_SHARDS)

Synthetic inputs (uniform residues for ciphertexts and keys, made-up polynomial coefficients): the kernels do the same work on
them as on real ones; the parity tests run the same chain on a small ring with real keys.  Needs one B200-class GPU (about
60 GB: 300 rotation keys of 96 MiB are the largest part).

    python -m paper_2609_12378_b200.examples.attention_block
"""
import torch

from paper_2609_12378_b200 import binding, inputs

LOG_N, L, K, DNUM, LEVEL = 16, 24, 8, 3, 24
N = 1 << LOG_N
TOKENS, HEADS, E, T_SHARD, DIM, GROUP_BABY = 128, 32, 8, 8, 128, 4


def main():
    dev = torch.device("cuda", 0)
    q, p = inputs.prime_chain(LOG_N, L, K)
    allp = [int(x) for x in q] + [int(x) for x in p]
    ctx = binding.Context(LOG_N, q, p, DNUM)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)

    def residues(primes, *lead):
        out = torch.empty((*lead, len(primes), N), dtype=torch.int64, device=dev)
        for i, m in enumerate(primes):
            out[..., i, :] = torch.randint(0, int(m), (*lead, N), generator=gen, device=dev, dtype=torch.int64)
        return out.view(torch.uint64)

    def keys_for(rots):
        return [binding.SwitchKey(residues(allp, DNUM, 2), ctx.galois_element(r)) for r in sorted(set(rots))]

    def timed(name, f):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); out = f(); b.record()
        torch.cuda.synchronize()
        print(f"{name:44s} {a.elapsed_time(b):8.1f} ms")
        return out, a.elapsed_time(b)

    shape = (TOKENS, HEADS, E, T_SHARD)
    rots = set(ctx.attention_rotations(TOKENS, HEADS, E, GROUP_BABY))
    for kind in (binding.ATTN_QUERY, binding.ATTN_KEY_VALUE, binding.ATTN_TO_SHARDS):
        rots |= set(ctx.attention_pack_rotations(kind, DIM, *shape))
    keys = keys_for(rots)
    rlk = binding.SwitchKey(residues(allp, DNUM, 2), 0)
    print(f"{len(keys)} rotation keys, {len(keys) * 96 / 1024:.1f} GiB")
    shards = {k: [binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 50) for _ in range(TOKENS // T_SHARD)] for k in "qkv"}
    poly = [1.0, 0.25, 0.03, 0.002, 0.0001]
    total = 0.0
    qq, ms = timed("query operands", lambda: ctx.attention_pack(binding.ATTN_QUERY, shards["q"], DIM, keys, *shape)); total += ms
    kk, ms = timed("key operands", lambda: ctx.attention_pack(binding.ATTN_KEY_VALUE, shards["k"], DIM, keys, *shape)); total += ms
    vv, ms = timed("value operands", lambda: ctx.attention_pack(binding.ATTN_KEY_VALUE, shards["v"], DIM, keys, *shape)); total += ms
    lk = kk[0].level
    qq = [binding.Ciphertext(x.data[:, :lk].contiguous(), x.scale) for x in qq]          # down to the key operands' level
    S, ms = timed("scores", lambda: ctx.attention_scores(qq, kk, rlk, keys, TOKENS, HEADS, E, group_baby=GROUP_BABY)); total += ms
    P, ms = timed("Softmax over the score rows", lambda: ctx.softmax_rows(S, 3.0, 2, poly, [poly, poly], rlk, keys, TOKENS, HEADS, E)); total += ms
    O, ms = timed("values", lambda: ctx.attention_values(P, vv, rlk, keys, TOKENS, HEADS, E)); total += ms
    Y, ms = timed("outputs back to shards", lambda: ctx.attention_pack(binding.ATTN_TO_SHARDS, O, DIM, keys, *shape)); total += ms
    print(f"{'attention block':44s} {total:8.1f} ms   (levels: operands {lk}, scores {S[0].level}, probabilities {P[0].level}, shards {Y[0].level})")
    assert ctx.device_status() == binding.OK


if __name__ == "__main__":
    main()
