"""Times the seven linear projections of one Llama-3-8B decoder layer on 128 encrypted tokens (N = 2^16, 24 + 8 primes,
dnum 3, 16 token shards of 8, B = 64) through the public binding: query/key/value as one call sharing their baby
steps, output, gate/up as one call, down.  Synthetic inputs (uniform residues for ciphertexts and keys, normal weights):
the kernels do the same work on them as on real ones.  Needs one B200-class GPU (the down projection's workspace is
62.5 GiB with B = 64, next to 11.8 GiB of rotation keys).

    python -m paper_2609_12378_b200.examples.llama_layer_projections [--eager] [--down-baby 32]
"""
import argparse

import torch

from paper_2609_12378_b200 import binding, inputs

LOG_N, L, K, DNUM, LEVEL = 16, 24, 8, 3, 24
N = 1 << LOG_N
HIDDEN, KV, FFN, T_SHARD, SHARDS = 4096, 1024, 14336, 8, 16


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--eager", action="store_true", help="one ModDown per giant-step rotation instead of one per output")
    ap.add_argument("--down-baby", type=int, default=64)
    args = ap.parse_args()
    lazy = not args.eager
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

    def weights(d_in, d_out):
        return (torch.randn((d_in, d_out), generator=gen, device=dev, dtype=torch.float64) * 0.02).contiguous()

    def keys_for(shapes, baby):
        rots = sorted(set(r for d_in, d_out in shapes for r in ctx.linear_proj_rotations(d_in, d_out, T_SHARD, SHARDS, baby)))
        return [binding.SwitchKey(residues(allp, DNUM, 2), ctx.galois_element(r)) for r in rots]

    def timed(f):
        f()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); f(); b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    total = 0.0
    # one input block (hidden -> ...): shared-input calls and the output projection
    cts = [binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 40) for _ in range(SHARDS)]
    for name, d_outs in (("query + key + value", [HIDDEN, KV, KV]), ("output", [HIDDEN]), ("gate + up", [FFN, FFN])):
        keys = keys_for([(HIDDEN, d) for d in d_outs], 64)
        Ws = [weights(HIDDEN, d) for d in d_outs]
        ms = timed(lambda: ctx.linear_proj_multi(cts, Ws, keys, HIDDEN, d_outs, T_SHARD, SHARDS, 64, lazy_moddown=lazy))
        print(f"{name:22s} {ms:8.1f} ms")
        total += ms
        del keys, Ws
        torch.cuda.empty_cache()
    del cts
    # down: four input blocks per shard
    nib = -(-FFN // HIDDEN)
    cts = [binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 40) for _ in range(SHARDS * nib)]
    keys = keys_for([(FFN, HIDDEN)], args.down_baby)
    W = weights(FFN, HIDDEN)
    ctx._ws = None
    torch.cuda.empty_cache()
    ms = timed(lambda: ctx.linear_proj(cts, W, keys, FFN, HIDDEN, T_SHARD, SHARDS, args.down_baby, lazy_moddown=lazy))
    print(f"{'down':22s} {ms:8.1f} ms")
    total += ms
    print(f"{'layer, linear part':22s} {total / 1e3:8.2f} s   ({'lazy' if lazy else 'eager'} giant-step ModDown)")


if __name__ == "__main__":
    main()
