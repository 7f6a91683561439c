#!/usr/bin/env python
"""Benchmark of the CKKS RNS hot path on B200.

One step = one pass of the whole hot path at N = 2^16, L = 24, K = 8, dnum = 3 over
seeded synthetic inputs:
  (a) NTT microbenchmark: 32 x 24 limbs, forward + inverse;
  (b) key switching: 64 plain rotations (distinct Galois elements), the same 64 hoisted
      off one ModUp, one ciphertext x ciphertext multiply with relinearisation;
  (c) the Llama-3-8B-shaped projection: 128 tokens x 4096 features in 16 token-shard
      ciphertexts times a 4096 x 4096 fp64 weight matrix encoded on the fly
      (encode + ct x pt multiply-accumulate + hoisted/plain rotations + rescale).
`value` is seconds per projection (part c); NTT limbs/s and key switches/s (plain rotations,
each a complete key switch) from parts (a) and (b) ride along in `submetrics`, with a roofline
fraction for each of the three paths (`roofline`, `roofline_keyswitch`, `roofline_projection`).  Ciphertexts and keys are uniform residues
(what real ones look like to the kernels); weights N(0, 0.02), fp64.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

With --impl reference the CPU checker is timed on a bounded sample of the same work.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

LOG_N, L, K, DNUM, LEVEL = 16, 24, 8, 3, 24
N = 1 << LOG_N
TOKENS, HIDDEN, T_SHARD, SHARDS, BABY = 128, 4096, 8, 16, 64
NTT_BATCH, NROT = 32, 64
METRIC = "key-switches/s & NTT limbs/s at N=2^16; s per 128-token Llama-3-8B projection"
WORKLOAD = ("one pass of the hot path at N=2^16 L=24 K=8 dnum=3: NTT fwd+inv of 32x24 limbs; 64 plain + 64 hoisted "
            "rotations + 1 mul_relin; 128-token 4096x4096 projection (16 shard ciphertexts, B=G=64, giant steps ")
LAZY = True


def workload():
    return WORKLOAD + ("summed before one ModDown per output)" if LAZY else "with one ModDown each)")


def peaks():
    try:
        return json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json"))), "measured"
    except Exception:
        return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0}, "fallback"


def profile_figure(name, key):
    """A figure recorded in a profiles/ summary as a line `key: number` (None if the file or the key is missing)."""
    import re
    try:
        text = open(os.path.join(ROOT, "profiles", name)).read()
    except OSError:
        return None
    m = re.search(r"^[-* ]*%s\s*[:=]\s*([0-9.eE+-]+)" % re.escape(key), text, re.M)
    return float(m.group(1)) if m else None


# ----------------------------------------------------------------- algorithmic work (what the rooflines count)
BFLY = (N // 2) * LOG_N                 # butterflies of one limb transform
FP64_PER_BFLY, FP64_PER_PAIR = 8, 7     # exact twiddle product + sum and difference; exact product of a conversion / key pair + add
ALPHA = -(-L // DNUM)


def ks_work(level=LEVEL, hoisted=False):
    """Limb transforms and multiply-add pairs (per coefficient products of basis conversion, key inner product and the
    ModDown tail) of one key switch at `level`; hoisted: without the shared inverse transform, ModUp and its transforms."""
    beta, nt = -(-level // ALPHA), level + K
    own = [min(ALPHA, level - j * ALPHA) for j in range(beta)]
    up_ntt = level + sum(nt - d for d in own)
    up_pairs = sum(d * (nt - d) + d for d in own)                  # conversions and the y = d qhat^-1 products
    ip_pairs = beta * 2 * nt
    dn_ntt = 2 * K + 2 * level
    dn_pairs = 2 * (K * level + K) + 2 * level                     # conversions, y products, the (u - conv) P^-1 tail
    ntt = dn_ntt + (0 if hoisted else up_ntt)
    pairs = ip_pairs + dn_pairs + (0 if hoisted else up_pairs)
    return {"limb_ntts": ntt, "pairs_per_coeff": pairs, "fp64_instr": ntt * BFLY * FP64_PER_BFLY + pairs * N * FP64_PER_PAIR,
            "modup": {"limb_ntts": up_ntt, "pairs_per_coeff": up_pairs}, "moddown": {"limb_ntts": dn_ntt, "pairs_per_coeff": dn_pairs},
            "inner": {"pairs_per_coeff": ip_pairs}}


def instr_of(limb_ntts, pairs_per_coeff):
    return limb_ntts * BFLY * FP64_PER_BFLY + pairs_per_coeff * N * FP64_PER_PAIR


def projection_work(lazy, shards=SHARDS):
    """Algorithmic work of the 4096 x 4096 projection: FP64 instructions of everything transform- or conversion-shaped,
    and the multiply-accumulate as the bytes that must cross HBM once (plaintexts, baby ciphertexts, accumulators)."""
    G = HIDDEN // BABY
    ks, ksh = ks_work(), ks_work(hoisted=True)
    limb = 8 * N
    parts = {
        "encode": {"count": HIDDEN, "fp64_instr": HIDDEN * instr_of(LEVEL, 0)},
        "baby_modup": {"count": shards, "fp64_instr": shards * instr_of(**ks["modup"])},
        "baby_hoisted_rotations": {"count": shards * (BABY - 1), "fp64_instr": shards * (BABY - 1) * ksh["fp64_instr"]},
        "rescale": {"count": shards, "fp64_instr": shards * instr_of(2 + 2 * (LEVEL - 1), 2 * (LEVEL - 1))},
        "mac": {"count": HIDDEN * shards,
                "hbm_bytes": HIDDEN * LEVEL * limb + shards * BABY * 2 * LEVEL * limb + shards * G * 2 * LEVEL * limb},
    }
    if lazy:
        term = instr_of(ks["modup"]["limb_ntts"], ks["modup"]["pairs_per_coeff"] + ks["inner"]["pairs_per_coeff"] + 1)
        parts["giant_terms"] = {"count": shards * (G - 1), "fp64_instr": shards * (G - 1) * term}
        parts["giant_moddown"] = {"count": shards, "fp64_instr": shards * instr_of(**ks["moddown"])}
    else:
        parts["giant_rotations"] = {"count": shards * (G - 1), "fp64_instr": shards * (G - 1) * ks["fp64_instr"]}
    return parts


def bound_ms(parts, fp64_peak_t, hbm_gbs):
    """Time the parts would take at the FP64 instruction peak (T instr/s) and, for the multiply-accumulate, at the HBM peak."""
    t = 0.0
    for v in parts.values():
        t += v.get("fp64_instr", 0) / (fp64_peak_t * 1e12) + v.get("hbm_bytes", 0) / (hbm_gbs * 1e9)
    return t * 1e3


# ----------------------------------------------------------------- clock sampling
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "200",
                                          "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except Exception:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass
        sm = [float(r[1]) for r in self.rows if len(r) >= 9 and r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in self.rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 9 and r[5 + i].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


# ----------------------------------------------------------------- CPU checker leg
def oracle_sample(lazy=True):
    """Time the CPU checker on a bounded sample of the projection workload and scale to one projection."""
    import numpy as np

    from oracle.ckks_oracle import Oracle
    from paper_2609_12378_b200 import inputs

    q, p = inputs.prime_chain(LOG_N, L, K)
    orc = Oracle(LOG_N, q, p, DNUM)
    g = inputs.rng(1004, 0)
    allp = list(q) + list(p)
    ct = inputs.uniform_residues(g, q, N, 2)
    keys = [inputs.uniform_residues(g, allp, N, DNUM * 2).reshape(DNUM, 2, L + K, N) for _ in range(3)]
    gals = [orc.galois_element(8), orc.galois_element(512), orc.galois_element(16)]
    z = np.repeat(g.normal(0, 0.02, HIDDEN), T_SHARD)
    t = {}
    t0 = time.perf_counter(); pts = [orc.encode(z, float(q[-1]), LEVEL) for _ in range(2)]; t["encode"] = (time.perf_counter() - t0) / 2
    t0 = time.perf_counter(); acc = orc.mul_plain_acc(ct, pts[0]); acc = orc.mul_plain_acc(ct, pts[1], acc); t["mac"] = (time.perf_counter() - t0) / 2
    t0 = time.perf_counter(); orc.rotate_hoisted(ct, keys[:1], gals[:1]); t["hoisted_1"] = time.perf_counter() - t0
    t0 = time.perf_counter(); orc.rotate_hoisted(ct, keys, gals); t["hoisted_3"] = time.perf_counter() - t0
    t0 = time.perf_counter(); orc.rotate(ct, keys[0], gals[0]); t["rotate"] = time.perf_counter() - t0
    t0 = time.perf_counter(); orc.rotate_sum(np.stack([ct, ct]), keys[:2], gals[:2]); t["rotate_sum_2"] = time.perf_counter() - t0
    t0 = time.perf_counter(); orc.rescale(acc); t["rescale"] = time.perf_counter() - t0
    t0 = time.perf_counter(); x = inputs.uniform_residues(g, q, N, 1); orc.intt(orc.ntt(x)); t["ntt_pair_24"] = time.perf_counter() - t0
    G = HIDDEN // BABY
    # hoisted rotations: three cost the shared ModUp plus three per-rotation parts, one costs the ModUp plus one
    per_h = max(t["hoisted_3"] - t["hoisted_1"], 0.0) / 2
    shared_up = max(t["hoisted_1"] - per_h, 0.0)
    # a two-term rotate_sum is two extended-basis terms and one ModDown, a rotation one term and one ModDown
    term = max(t["rotate_sum_2"] - t["rotate"], 0.0)
    moddown = max(t["rotate"] - term, 0.0)
    giant = (G - 1) * term + moddown if lazy else (G - 1) * t["rotate"]
    proj = (HIDDEN * t["encode"] + HIDDEN * SHARDS * t["mac"] + SHARDS * (shared_up + (BABY - 1) * per_h)
            + SHARDS * giant + SHARDS * t["rescale"])
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    sample = ("2 encodes, 2 ct x pt MACs, hoisted rotations by 1 and by 3 keys, 1 plain rotation, 1 two-term rotate_sum, 1 rescale, "
              "24 NTT round trips at full size; scaled by the projection's counts (4096 encodes, 65536 MACs, 16 ModUps + 1008 hoisted rotations, "
              + ("1008 giant-step terms + 16 ModDowns" if lazy else "1008 plain rotations") + ", 16 rescales)")
    return {"proj_s": proj, "ntt_limbs_per_s": 48 / t["ntt_pair_24"], "key_switches_per_s": 1.0 / t["rotate"],
            "parts_s": t, "cores": cores, "sample": sample}


def oracle_one_shard(lazy=True):
    """One whole token shard of the 4096 x 4096 projection through the checker (all 4096 diagonals encoded, 4096
    multiply-accumulates, 63 hoisted and 63 giant-step rotations, one rescale): seconds."""
    import numpy as np

    from oracle.ckks_oracle import Oracle, ProjDesc
    from paper_2609_12378_b200 import inputs

    q, p = inputs.prime_chain(LOG_N, L, K)
    orc = Oracle(LOG_N, q, p, DNUM)
    g = inputs.rng(1004, 5)
    allp = list(q) + list(p)
    desc = ProjDesc(HIDDEN, HIDDEN, T_SHARD, 1, BABY, lazy_moddown=lazy)
    ct = inputs.uniform_residues(g, q, N, 2)
    W = inputs.weights_normal(g, HIDDEN, HIDDEN, 0.02)
    key = inputs.uniform_residues(g, allp, N, DNUM * 2).reshape(DNUM, 2, L + K, N)      # one key stands in for all 126: same work
    keys = {orc.galois_element(r): key for r in orc.proj_rotations(desc)}
    t0 = time.perf_counter()
    orc.linear_proj(desc, ct[None], W, keys, 2.0 ** 40)
    return time.perf_counter() - t0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    if args.cpu_anchor:
        sec = oracle_one_shard(LAZY)
        print(json.dumps({"impl": "reference", "one_shard_seconds": sec,
                          "cores": int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))}))
        return
    for _ in range(args.warmup if args.warmup < 2 else 1):
        oracle_sample(LAZY)
    vals = [oracle_sample(LAZY) for _ in range(max(1, args.steps))]
    v = statistics.mean(x["proj_s"] for x in vals)
    last = vals[-1]
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": "s/projection", "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": v * 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "u64", "data": "synthetic",
            "config": {"workload": workload(), "note": "CPU checker timed on a bounded sample, scaled by operation counts"},
            "submetrics": {"ntt_limbs_per_s": last["ntt_limbs_per_s"], "key_switches_per_s": last["key_switches_per_s"]},
            "cpu_baseline": {"value": v, "unit": "s/projection", "cores": last["cores"], "kind": "oracle", "sample": last["sample"]},
            "e2e": {"value": v, "unit": "s/projection", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ----------------------------------------------------------------- multi-rank aggregation (replicas: no data-path collective)
def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_metrics(world, a_ms, plain_ms, c_ms, hoisted_ms=None, relin_ms=None):
    """Whole-job figures from the slowest rank's part times: every rank ran the same step on its own replica.
    plain_ms: the NROT plain rotations (each a complete key switch); hoisted_ms: the same NROT off one shared ModUp."""
    limb_ntts = NTT_BATCH * L
    out = {"value": c_ms * 1e-3 / world,                                   # seconds per projection, all ranks together
           "ntt_limbs_per_s": world * 2 * limb_ntts / (a_ms * 1e-3),
           "key_switches_per_s": world * NROT / (plain_ms * 1e-3)}
    if hoisted_ms:
        out["hoisted_rotations_per_s"] = world * NROT / (hoisted_ms * 1e-3)
    if relin_ms:
        out["mul_relin_per_s"] = world / (relin_ms * 1e-3)
    return out


# ----------------------------------------------------------------- CUDA leg
def run_cuda(args):
    import torch
    import torch.distributed as dist

    from paper_2609_12378_b200 import binding, inputs

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    SH = args.shards if args.profile else SHARDS
    q, p = inputs.prime_chain(LOG_N, L, K)
    allp = [int(x) for x in q] + [int(x) for x in p]
    ctx = binding.Context(LOG_N, q, p, DNUM, device=local)
    if args.profile and args.mac_kernel:
        ctx.set_option(binding.OPT_MAC_KERNEL, args.mac_kernel)
    if args.profile and args.conv_kernel >= 0:
        ctx.set_option(binding.OPT_CONV_KERNEL, args.conv_kernel)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1004 + rank)

    def residues(primes, *lead):
        out = torch.empty((*lead, len(primes), N), dtype=torch.int64, device=dev)
        for i, m in enumerate(primes):
            out[..., i, :] = torch.randint(0, int(m), (*lead, N), generator=gen, device=dev, dtype=torch.int64)
        return out.view(torch.uint64)

    # (a) NTT inputs
    polys = residues(allp[:L], NTT_BATCH)
    # keys: the projection's rotation set contains the 64 rotations 8b, b = 1..64, of part (b)
    rots = ctx.linear_proj_rotations(HIDDEN, HIDDEN, T_SHARD, SH, BABY)
    keys = {r: binding.SwitchKey(residues(allp, DNUM, 2), ctx.galois_element(r)) for r in rots}
    rlk = binding.SwitchKey(residues(allp, DNUM, 2), 0)
    rot_keys = [keys[8 * b] for b in range(1, NROT + 1)]
    proj_keys = list(keys.values())
    # (b) ciphertexts
    cta = binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 40)
    ctb = binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 40)
    rot_out = ctx.empty_ct(LEVEL)
    hoist_out = [ctx.empty_ct(LEVEL) for _ in range(NROT)]
    mul_out = ctx.empty_ct(LEVEL)
    # (c) projection inputs
    cts = [binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 40) for _ in range(SH)]
    W = (torch.randn((HIDDEN, HIDDEN), generator=gen, device=dev, dtype=torch.float64) * 0.02).contiguous()
    outs = [ctx.empty_ct(LEVEL - 1) for _ in range(SH)]
    ws = torch.empty(ctx.linear_proj_workspace_bytes(HIDDEN, HIDDEN, T_SHARD, SH, BABY, LEVEL, True), dtype=torch.uint8, device=dev)
    # e2e host buffers (pinned)
    h_cts = [c.data.cpu().pin_memory() for c in cts]
    h_W = W.cpu().pin_memory()
    h_outs = [torch.empty((2, LEVEL - 1, N), dtype=torch.uint64).pin_memory() for _ in range(SH)]

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def part_a():
        ctx.ntt(polys, 0)
        ctx.intt(polys, 0)

    def part_b1():
        for k in rot_keys:
            ctx.rotate(cta, k, out=rot_out)

    def part_b2():
        ctx.rotate_hoisted(cta, rot_keys, outs=hoist_out)

    def part_b3():
        ctx.mul_relin(cta, ctb, rlk, out=mul_out)

    def part_b():
        part_b1(); part_b2(); part_b3()

    def part_c():
        ctx.linear_proj(cts, W, proj_keys, HIDDEN, HIDDEN, T_SHARD, SH, BABY, outs=outs, ws=ws, lazy_moddown=LAZY)

    def step(times=None):
        e = [ev() for _ in range(6)]
        if args.profile:
            for name, f in (("a", part_a), ("b", part_b), ("c", part_c)):
                if name in args.parts:
                    f()
            return
        e[0].record(); part_a(); e[1].record(); part_b1(); e[4].record(); part_b2(); e[5].record(); part_b3(); e[2].record(); part_c(); e[3].record()
        if times is not None:
            times.append(e)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    nwarm = args.warmup if args.profile else max(3, args.warmup)
    for _ in range(nwarm):
        step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = binding.kernel_launches()
    times = []
    t_start, t_end = ev(), ev()
    t_start.record()
    for _ in range(args.steps):
        step(times)
    t_end.record()
    barrier()
    launches = binding.kernel_launches() - launches0
    total_ms = t_start.elapsed_time(t_end)
    clocks = sampler.stop() if rank == 0 else None
    if args.profile:
        print(json.dumps({"profile_run": True, "launches_per_step": launches // max(1, args.steps)}))
        return
    a_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in times)
    b_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in times)
    c_ms = statistics.mean(e[2].elapsed_time(e[3]) for e in times)
    b1_ms = statistics.mean(e[1].elapsed_time(e[4]) for e in times)
    b2_ms = statistics.mean(e[4].elapsed_time(e[5]) for e in times)
    b3_ms = statistics.mean(e[5].elapsed_time(e[2]) for e in times)

    # the other giant-step schedule (one ModDown per rotation if the step timed the lazy form, and the reverse), with the
    # same statistics: the same number of calls, one event pair each, mean
    def part_c_other():
        ctx.linear_proj(cts, W, proj_keys, HIDDEN, HIDDEN, T_SHARD, SH, BABY, outs=outs, ws=ws, lazy_moddown=not LAZY)

    part_c_other()
    torch.cuda.synchronize()
    other = []
    for _ in range(args.steps):
        a_, b_ = ev(), ev()
        a_.record(); part_c_other(); b_.record()
        other.append((a_, b_))
    torch.cuda.synchronize()
    c_other_ms = statistics.mean(a_.elapsed_time(b_) for a_, b_ in other)

    # dominant-kernel roofline leg: the NTT kernel pair timed alone on the launching stream
    s0, s1 = ev(), ev()
    s0.record()
    reps = 5
    for _ in range(reps):
        ctx.ntt(polys, 0)
    s1.record()
    torch.cuda.synchronize()
    ntt_fwd_ms = s0.elapsed_time(s1) / reps
    # the same butterflies on registers only (no global traffic): what the arithmetic alone sustains on this GPU
    probe_scratch = torch.zeros(1 << 20, dtype=torch.int64, device=dev).view(torch.uint64)
    ctx.ntt_butterfly_probe(64, probe_scratch)
    p0, p1 = ev(), ev()
    p0.record()
    probe_bfly = ctx.ntt_butterfly_probe(4096, probe_scratch)
    p1.record()
    torch.cuda.synchronize()
    probe_rate = probe_bfly / (p0.elapsed_time(p1) * 1e-3)          # butterflies per second

    # outside the step, once each after a warm-up call: the composite calls built on the step's primitives
    def once(f):
        f()
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record(); f(); b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    extras = {}
    if rank == 0 and not args.no_extras:
        Wk = (torch.randn((HIDDEN, HIDDEN // 4), generator=gen, device=dev, dtype=torch.float64) * 0.02).contiguous()
        Wv = (torch.randn((HIDDEN, HIDDEN // 4), generator=gen, device=dev, dtype=torch.float64) * 0.02).contiguous()
        douts = [HIDDEN, HIDDEN // 4, HIDDEN // 4]
        extras["qkv_three_calls_ms"] = once(lambda: [ctx.linear_proj(cts, w_, proj_keys, HIDDEN, d_, T_SHARD, SH, BABY, ws=ws) for w_, d_ in zip((W, Wk, Wv), douts)])
        extras["qkv_shared_baby_steps_ms"] = once(lambda: ctx.linear_proj_multi(cts, [W, Wk, Wv], proj_keys, HIDDEN, douts, T_SHARD, SH, BABY, ws=ws))
        pa, pb = [cta, ctb] * 64, [ctb, cta] * 64
        extras["sum_of_128_products_one_relin_ms"] = once(lambda: ctx.mul_relin_sum(pa, pb, rlk, out=mul_out))
        extras["mul_relin_128_calls_ms"] = once(lambda: [ctx.mul_relin(x_, y_, rlk, out=mul_out) for x_, y_ in zip(pa, pb)])
        bouts = [ctx.empty_ct(LEVEL) for _ in range(16)] * 8
        bws = ctx.workspace(ctx.workspace_bytes(binding.OP_MUL_RELIN_BATCH, LEVEL, 128))
        extras["mul_relin_batch_128_ms"] = once(lambda: ctx.mul_relin_batch(pa, pb, rlk, outs=bouts, ws=bws))
        del bouts, bws
        rin, routs = [cta, ctb] * 32, [ctx.empty_ct(LEVEL) for _ in range(16)] * 4
        rws = ctx.workspace(ctx.workspace_bytes(binding.OP_ROTATE_BATCH, LEVEL, 64))
        extras["rotate_64_calls_ms"] = once(lambda: [ctx.rotate(x_, rot_keys[0], out=rot_out) for x_ in rin])
        extras["rotate_batch_64_ms"] = once(lambda: ctx.rotate_batch(rin, rot_keys[0], outs=routs, ws=rws))
        del routs, rws
        # the same 64 independent rotations issued on four streams, a context (tables and scratch) per stream: kernels of
        # single-ciphertext calls fill the GPU for at most one wave, so independent calls overlap
        sctx = [ctx] + [binding.Context(LOG_N, q, p, DNUM, device=local) for _ in range(3)]
        sts = [torch.cuda.Stream() for _ in range(4)]
        souts = [ctx.empty_ct(LEVEL) for _ in range(4)]

        def on_streams():
            cur = torch.cuda.current_stream()
            for s_ in sts:
                s_.wait_stream(cur)
            for i_, x_ in enumerate(rin):
                with torch.cuda.stream(sts[i_ % 4]):
                    sctx[i_ % 4].rotate(x_, rot_keys[0], out=souts[i_ % 4], stream=sts[i_ % 4])
            for s_ in sts:
                cur.wait_stream(s_)

        extras["rotate_64_calls_on_4_streams_ms"] = once(on_streams)
        del sctx, sts, souts
        # a degree-63 polynomial (the paper's SiLU degree per layer) by the power tree and by baby steps / giant steps
        c63 = [1.0 / (1 + k) for k in range(64)]
        extras["poly_degree63_tree_ms"] = once(lambda: ctx.poly_eval_tree(binding.Ciphertext(cta.data, 2.0 ** 50), c63, rlk))
        extras["poly_degree63_bsgs_m8_ms"] = once(lambda: ctx.poly_eval_bsgs(binding.Ciphertext(cta.data, 2.0 ** 50), c63, 8, rlk))
        # Softmax by doubling on 256 rows of 128 scores (one ciphertext), two rounds, degree-4 polynomials: 7 + 2 x 11 products,
        # 14 rotations
        sm_keys = [keys[256 << i] for i in range(7)]
        sm_in = binding.Ciphertext(cta.data, 2.0 ** 50)
        poly = [1.0, 0.25, 0.03, 0.002, 0.0001]
        extras["softmax_256x128_two_rounds_ms"] = once(lambda: ctx.softmax(sm_in, 3.0, 2, 128, poly, [poly, poly], rlk, sm_keys))
        del Wk, Wv

    # e2e: host buffers in, host buffers out, copies inside the timed region
    def e2e_step():
        for c, h in zip(cts, h_cts):
            c.data.copy_(h, non_blocking=True)
        W.copy_(h_W, non_blocking=True)
        part_c()
        for o, h in zip(outs, h_outs):
            h.copy_(o.data, non_blocking=True)

    e2e_step()
    barrier()
    x0, x1 = ev(), ev()
    x0.record()
    for _ in range(args.steps):
        e2e_step()
    x1.record()
    barrier()
    e2e_ms = x0.elapsed_time(x1) / args.steps
    h2d = sum(h.numel() * 8 for h in h_cts) + h_W.numel() * 8
    d2h = sum(h.numel() * 8 for h in h_outs)

    # the same steps with two sets of device buffers and the copies on their own streams: step i + 1's inputs arrive and
    # step i - 1's results leave while step i computes (reported beside the serial figure, which stays the e2e value)
    def pipelined(k):
        cs, hs, ds = torch.cuda.current_stream(), torch.cuda.Stream(), torch.cuda.Stream()
        sets = [(cts, W, outs),
                ([binding.Ciphertext(torch.empty_like(c.data), c.scale) for c in cts], torch.empty_like(W), [ctx.empty_ct(LEVEL - 1) for _ in outs])]
        done, left = [None] * k, [None] * k
        hs.wait_stream(cs); ds.wait_stream(cs)
        for i in range(k):
            ci, wi, oi = sets[i % 2]
            with torch.cuda.stream(hs):
                if i >= 2:
                    hs.wait_event(done[i - 2])
                for c, h in zip(ci, h_cts):
                    c.data.copy_(h, non_blocking=True)
                wi.copy_(h_W, non_blocking=True)
                arrived = torch.cuda.Event(); arrived.record(hs)
            cs.wait_event(arrived)
            if i >= 2:
                cs.wait_event(left[i - 2])
            ctx.linear_proj(ci, wi, proj_keys, HIDDEN, HIDDEN, T_SHARD, SH, BABY, outs=oi, ws=ws, lazy_moddown=LAZY)
            done[i] = torch.cuda.Event(); done[i].record(cs)
            with torch.cuda.stream(ds):
                ds.wait_event(done[i])
                for o, h in zip(oi, h_outs):
                    h.copy_(o.data, non_blocking=True)
                left[i] = torch.cuda.Event(); left[i].record(ds)
        cs.wait_stream(ds); cs.wait_stream(hs)

    pipelined(2)
    barrier()
    y0, y1 = ev(), ev()
    y0.record()
    pipelined(args.steps)
    y1.record()
    barrier()
    e2e_pipe_ms = y0.elapsed_time(y1) / args.steps

    (total_ms, a_ms, b_ms, c_ms, e2e_ms, ntt_fwd_ms, e2e_pipe_ms, b1_ms, b2_ms, b3_ms, c_other_ms) = max_over_ranks(
        [total_ms, a_ms, b_ms, c_ms, e2e_ms, ntt_fwd_ms, e2e_pipe_ms, b1_ms, b2_ms, b3_ms, c_other_ms], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    layer = None
    if not args.no_extras and not args.no_layer:
        # the layer's down projection needs most of the device: keep only the rotation keys (reused) and the context
        del ws, h_cts, h_W, h_outs, hoist_out, polys, probe_scratch, outs, cts, W, rot_out, mul_out, rot_keys, proj_keys
        ctx._ws = None
        torch.cuda.empty_cache()
        layer = layer_submetrics(ctx, residues, allp, gen, dev, args.layer_reps, keys)

    pk, pk_kind = peaks()
    limb_ntts = NTT_BATCH * L
    sm_count = torch.cuda.get_device_properties(local).multi_processor_count
    sm_max = float(pk.get("sm_max_mhz", 1965.0))
    # Every path here is bound by FP64 arithmetic ("alu"): butterflies and exact modular products run on the FP64 pipe.
    # Peak = 64 FP64 instructions per clock per SM (the DFMA rate) x SM count x the maximum SM clock.  Algorithmic work =
    # 8 instructions per butterfly (6 for the exact twiddle product with its quotient, 2 for sum and difference),
    # N/2 log2 N butterflies per limb transform, and 7 per multiply-add pair of a basis conversion or key product.
    fp64_peak = 64.0 * sm_count * sm_max * 1e6 / 1e12          # T instr/s
    peak_kind = "derived: 64 DFMA/clk/SM x %d SMs x %.0f MHz" % (sm_count, sm_max)
    clock_ratio = float(clocks["sm_mhz"]) / sm_max if clocks and clocks.get("sm_mhz") else None

    def alu(instr, ms):
        ach = instr / (ms * 1e-3) / 1e12
        return {"bound": "alu", "achieved": ach, "peak": fp64_peak, "unit": "T FP64 instr/s", "frac": ach / fp64_peak,
                "frac_at_sampled_clock": ach / (fp64_peak * clock_ratio) if clock_ratio else None, "peak_kind": peak_kind}

    # (1) dominant kernel pair: forward transform of 768 limbs, timed alone
    ops = limb_ntts * BFLY * FP64_PER_BFLY
    ntt_bytes = limb_ntts * 2 * 8 * N          # algorithmic bytes: each limb read once and written once
    hbm_achieved = ntt_bytes / (ntt_fwd_ms * 1e-3) / 1e9
    roofline = alu(ops, ntt_fwd_ms)
    roofline.update({
        "kernel": "ntt16_fwd_cols + ntt16_fwd_rows (forward NTT of 768 limbs, one launch each)",
        # ncu, dram read + write bytes of the two launches; None when no capture of the current kernels is recorded
        "traffic": profile_figure("ntt16_384limbs.md", "dram_bytes_per_launch_pair"),
        "ms_per_launch_pair": ntt_fwd_ms,
        "vs_register_resident_butterflies": {
            "achieved_gbfly_s": limb_ntts * BFLY / (ntt_fwd_ms * 1e-3) / 1e9, "peak_gbfly_s": probe_rate / 1e9,
            "frac": limb_ntts * BFLY / (ntt_fwd_ms * 1e-3) / probe_rate,
            "peak_kind": "measured in this run: the transform's radix-16 butterfly groups on registers, 3 CTAs x 256 threads per SM"},
        "hbm": {"achieved": hbm_achieved, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": hbm_achieved / pk["hbm_gbs"],
                "algorithmic_bytes": ntt_bytes, "peak_kind": pk_kind + " copy bandwidth"}})
    # (2) key switching: one plain rotation = one complete key switch; the hoisted form shares the ModUp
    ks, ksh = ks_work(), ks_work(hoisted=True)
    ks_bytes = (2 * LEVEL + DNUM * 2 * (L + K) + 2 * LEVEL) * 8 * N          # ciphertext in, key, ciphertext out
    roofline_ks = alu(ks["fp64_instr"], b1_ms / NROT)
    roofline_ks.update({
        "per": "plain rotation (ckks_rotate, one ciphertext per call)", "us": b1_ms / NROT * 1e3,
        "work": {"limb_ntts": ks["limb_ntts"], "mul_add_pairs": ks["pairs_per_coeff"] * N, "fp64_instr": ks["fp64_instr"]},
        "hbm": {"achieved": ks_bytes / (b1_ms / NROT * 1e-3) / 1e9, "peak": pk["hbm_gbs"], "unit": "GB/s",
                "frac": ks_bytes / (b1_ms / NROT * 1e-3) / 1e9 / pk["hbm_gbs"], "algorithmic_bytes": ks_bytes},
        "hoisted": dict(alu(ksh["fp64_instr"] + instr_of(**ks["modup"]) / NROT, b2_ms / NROT), us=b2_ms / NROT * 1e3,
                        per="rotation off a ModUp shared by %d (ckks_rotate_hoisted)" % NROT),
        "mul_relin": dict(alu(ks["fp64_instr"], b3_ms), us=b3_ms * 1e3)})
    # (3) the projection: everything transform- or conversion-shaped at the FP64 peak, the multiply-accumulate at the
    # HBM peak (its operands and results crossing HBM once); fraction = that time / measured time
    def proj_roofline(lazy, ms):
        parts = projection_work(lazy, SH)
        bnd = bound_ms(parts, fp64_peak, pk["hbm_gbs"])
        return {"bound": "alu + hbm (multiply-accumulate)", "bound_ms": bnd, "measured_ms": ms, "frac": bnd / ms,
                "frac_at_sampled_clock": (bound_ms(parts, fp64_peak * clock_ratio, pk["hbm_gbs"]) / ms) if clock_ratio else None,
                "schedule": "giant steps summed before one ModDown" if lazy else "one ModDown per giant-step rotation",
                "parts_bound_ms": {k: bound_ms({k: v}, fp64_peak, pk["hbm_gbs"]) for k, v in parts.items()},
                "peak_kind": peak_kind + "; " + pk_kind + " copy bandwidth %.0f GB/s" % pk["hbm_gbs"]}
    roofline_proj = proj_roofline(LAZY, c_ms)
    roofline_proj["other_schedule"] = proj_roofline(not LAZY, c_other_ms)

    cpu = oracle_sample(LAZY)
    jm = job_metrics(world, a_ms, b1_ms, c_ms, b2_ms, b3_ms)
    sub = {"ntt_limbs_per_s": jm["ntt_limbs_per_s"], "key_switches_per_s": jm["key_switches_per_s"],
           "hoisted_rotations_per_s": jm["hoisted_rotations_per_s"], "mul_relin_per_s": jm["mul_relin_per_s"],
           "ms": {"ntt_roundtrip": a_ms, "keyswitch_part": b_ms, "plain_rotations_%d" % NROT: b1_ms, "hoisted_rotations_%d" % NROT: b2_ms,
                  "mul_relin": b3_ms, "projection": c_ms,
                  "projection_%s_moddown" % ("eager" if LAZY else "lazy"): c_other_ms}}
    if layer:
        sub["layer"] = layer
    line = {
        "metric": METRIC, "value": jm["value"], "unit": "s/projection", "n_gpus": world, "steps": args.steps,
        "warmup": nwarm, "ms_per_step": total_ms / args.steps, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": workload(), "l2": "inputs larger than L2 (>= 384 MiB per part)", "parallelism": f"replicas x{world}"},
        "extras": extras,
        "submetrics": sub,
        "clocks": clocks,
        "e2e": {"value": e2e_ms * 1e-3 / world, "unit": "s/projection", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "copies_overlapped_value": e2e_pipe_ms * 1e-3 / world},
        "gpu_launches": launches,
        "roofline": roofline,
        "roofline_keyswitch": roofline_ks,
        "roofline_projection": roofline_proj,
        "cpu_baseline": {"value": cpu["proj_s"], "unit": "s/projection", "cores": cpu["cores"], "kind": "oracle",
                         "method": "extrapolated from a timed sample by operation counts", "sample": cpu["sample"],
                         "ntt_limbs_per_s": cpu["ntt_limbs_per_s"], "key_switches_per_s": cpu["key_switches_per_s"],
                         # one whole shard of this projection through the checker, timed once on a B200 host (16 cores) and
                         # recorded with its command: x 16 shards = what the extrapolation should land near
                         "one_shard_anchor_s": profile_figure("oracle_one_shard.md", "one_shard_seconds")},
        # figures copied from ncu captures (profiles/), with the kernels they were taken on: not measured in this run
        "static_notes": {"source": "profiles/bench_step_launch_list.md, profiles/ntt16_384limbs.md",
                         "ntt16_family_share_of_step": profile_figure("bench_step_launch_list.md", "ntt16_family_share"),
                         "mac_share_of_step": profile_figure("bench_step_launch_list.md", "mac_share"),
                         "keyswitch_kernels_share_of_step": profile_figure("bench_step_launch_list.md", "keyswitch_kernels_share"),
                         "fp64_pipe_active_fwd_cols": profile_figure("ntt16_384limbs.md", "fp64_pipe_active_fwd_cols"),
                         "fp64_pipe_active_fwd_rows": profile_figure("ntt16_384limbs.md", "fp64_pipe_active_fwd_rows")},
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------- one decoder layer's linear work and products
def layer_submetrics(ctx, residues, allp, gen, dev, reps, have_keys):
    """CUDA-event means of one Llama-3-8B decoder layer's homomorphic linear work at 128 tokens (16 shards of 8, B = 64,
    giant steps summed before one ModDown): query/key/value as one call sharing their baby steps, output, gate and up as
    one call, down; and the attention products as ciphertext x ciphertext multiplies at level 24: 2048 + 2048 products,
    128 summed per output ciphertext with one relinearisation (ckks_mul_relin_sum), and the same count relinearised one
    by one in batches (ckks_mul_relin_batch).  Synthetic operands (uniform residues, normal weights)."""
    import torch

    from paper_2609_12378_b200 import binding

    KV, FFN = 1024, 14336

    def weights(d_in, d_out):
        return (torch.randn((d_in, d_out), generator=gen, device=dev, dtype=torch.float64) * 0.02).contiguous()

    def keys_for(shapes):
        """Rotation keys of the shapes: the ones the caller already holds (rotation in slots -> key), new ones otherwise."""
        rots = sorted(set(r for d_in, d_out in shapes for r in ctx.linear_proj_rotations(d_in, d_out, T_SHARD, SHARDS, BABY)))
        for r in rots:
            if r not in have_keys:
                have_keys[r] = binding.SwitchKey(residues(allp, DNUM, 2), ctx.galois_element(r))
        return [have_keys[r] for r in rots]

    def timed(f):
        f()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); f(); b.record()
            ts.append((a, b))
        torch.cuda.synchronize()
        return statistics.mean(a.elapsed_time(b) for a, b in ts)

    out = {"reps": reps, "ms": {}}
    cts = [binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 40) for _ in range(SHARDS)]
    for name, d_outs in (("qkv", [HIDDEN, KV, KV]), ("o", [HIDDEN]), ("gate_up", [FFN, FFN])):
        keys = keys_for([(HIDDEN, d) for d in d_outs])
        Ws = [weights(HIDDEN, d) for d in d_outs]
        out["ms"][name] = timed(lambda: ctx.linear_proj_multi(cts, Ws, keys, HIDDEN, d_outs, T_SHARD, SHARDS, BABY, lazy_moddown=True))
        del keys, Ws
        ctx._ws = None
        torch.cuda.empty_cache()
    del cts
    nib = -(-FFN // HIDDEN)
    cts = [binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 40) for _ in range(SHARDS * nib)]
    keys = keys_for([(FFN, HIDDEN)])
    W = weights(FFN, HIDDEN)
    out["ms"]["down"] = timed(lambda: ctx.linear_proj(cts, W, keys, FFN, HIDDEN, T_SHARD, SHARDS, BABY, lazy_moddown=True))
    out["down_workspace_gib"] = ctx.linear_proj_workspace_bytes(FFN, HIDDEN, T_SHARD, SHARDS, BABY, LEVEL, True) / 2 ** 30
    del cts, keys, W
    ctx._ws = None
    torch.cuda.empty_cache()
    out["projections_s"] = sum(out["ms"][k] for k in ("qkv", "o", "gate_up", "down")) * 1e-3
    # attention products: 16 distinct operands, 128 pairs per output ciphertext, 16 outputs for QK^T and 16 for PV
    a = [binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 40) for _ in range(16)]
    b = [binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 40) for _ in range(16)]
    rlk = binding.SwitchKey(residues(allp, DNUM, 2), 0)
    pa, pb = [a[i % 16] for i in range(128)], [b[(3 * i + i // 16) % 16] for i in range(128)]
    acc = ctx.empty_ct(LEVEL)
    out["ms"]["products_2x2048_summed_128_per_output"] = timed(lambda: [ctx.mul_relin_sum(pa, pb, rlk, out=acc) for _ in range(32)])
    bouts = [ctx.empty_ct(LEVEL) for _ in range(16)] * 8
    bws = ctx.workspace(ctx.workspace_bytes(binding.OP_MUL_RELIN_BATCH, LEVEL, 128))
    out["ms"]["products_2x2048_each_relinearised"] = timed(lambda: [ctx.mul_relin_batch(pa, pb, rlk, outs=bouts, ws=bws) for _ in range(32)])
    out["layer_linear_and_products_s"] = out["projections_s"] + out["ms"]["products_2x2048_summed_128_per_output"] * 1e-3
    # the element-wise product of the gate and up branches (SiLU's polynomial not included): 4 blocks x 16 shards of
    # ciphertext pairs at the projections' output level, relinearised in batches of 16
    g1 = [binding.Ciphertext(a[i % 16].data[:, :LEVEL - 1].contiguous(), 2.0 ** 40) for i in range(16)]
    g2 = [binding.Ciphertext(b[i % 16].data[:, :LEVEL - 1].contiguous(), 2.0 ** 40) for i in range(16)]
    ga, gb = [g1[i % 16] for i in range(nib * SHARDS)], [g2[(5 * i + 1) % 16] for i in range(nib * SHARDS)]
    gouts = [ctx.empty_ct(LEVEL - 1) for _ in range(16)] * (nib * SHARDS // 16)
    gws = ctx.workspace(ctx.workspace_bytes(binding.OP_MUL_RELIN_BATCH, LEVEL - 1, nib * SHARDS))
    out["ms"]["gate_times_up_64_products"] = timed(lambda: ctx.mul_relin_batch(ga, gb, rlk, outs=gouts, ws=gws))
    # a degree-63 polynomial (the size the paper's Table 7 gives SiLU) of one gate ciphertext by baby and giant steps of 8,
    # synthetic coefficients; a layer evaluates it on all 64 gate ciphertexts
    pc = [0.5 ** (k // 4) / (1 + k) for k in range(64)]
    xg = binding.Ciphertext(g1[0].data, 2.0 ** 50)
    out["ms"]["polynomial_degree_63_one_ciphertext"] = timed(lambda: ctx.poly_eval_bsgs(xg, pc, 8, rlk))
    xs = [binding.Ciphertext(g1[i % 16].data, 2.0 ** 50) for i in range(nib * SHARDS)]
    out["ms"]["polynomial_degree_63_of_64_ciphertexts"] = timed(lambda: ctx.poly_eval_bsgs_batch(xs, pc, 8, rlk))
    del xg, xs
    del bouts, bws, a, b, acc, g1, g2, ga, gb, gouts, gws
    ctx._ws = None
    torch.cuda.empty_cache()
    # the same products inside the attention entry points (diagonal-block layout: 128 tokens, 32 heads, 8 diagonals per
    # ciphertext, 128 channels): scores with hoisted rotations of the key and query operands (groups split 4 x 4), Softmax by doubling over rows spread
    # across 16 ciphertexts (two rounds, degree-4 polynomials), probability x value with the value operands' rotations
    tokens, heads, E, dim = 128, 32, 8, 128
    GB = 4                                  # score groups split into 4 baby x 4 giant steps
    rots = ctx.attention_rotations(tokens, heads, E, GB)
    akeys = [binding.SwitchKey(residues(allp, DNUM, 2), ctx.galois_element(r)) for r in rots]
    q = [binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 50) for _ in range(dim)]
    k = [binding.Ciphertext(residues(allp[:L], 2), 2.0 ** 50) for _ in range(dim)]
    v = q                                   # same shape and level; the values' content does not matter to the kernels
    poly = [1.0, 0.25, 0.03, 0.002, 0.0001]
    att = {}
    att["scores_every_group_by_itself"] = timed(lambda: ctx.attention_scores(q, k, rlk, akeys, tokens, heads, E))
    ctx._ws = None
    torch.cuda.empty_cache()
    S = ctx.attention_scores(q, k, rlk, akeys, tokens, heads, E, group_baby=GB)
    att["scores"] = timed(lambda: ctx.attention_scores(q, k, rlk, akeys, tokens, heads, E, group_baby=GB))
    P = ctx.softmax_rows(S, 3.0, 2, poly, [poly, poly], rlk, akeys, tokens, heads, E)
    att["softmax_rows"] = timed(lambda: ctx.softmax_rows(S, 3.0, 2, poly, [poly, poly], rlk, akeys, tokens, heads, E))
    att["values"] = timed(lambda: ctx.attention_values(P, v, rlk, akeys, tokens, heads, E))
    att["levels"] = {"operands": LEVEL, "scores": S[0].level, "probabilities": P[0].level, "outputs": P[0].level - 1}
    att["total_s"] = (att["scores"] + att["softmax_rows"] + att["values"]) * 1e-3
    # the conversions around it: 16 token-shard ciphertexts (8 tokens each, channel-major features) -> 128 query operands,
    # 128 key (or value) operands, and 128 outputs at the values' level back to 16 shards; timed once each (one call is
    # 2048 hoisted rotations), with their own rotation keys
    del S, akeys, k
    ctx._ws = None
    torch.cuda.empty_cache()
    TI = 8
    shape = (tokens, heads, E, TI)
    conv = {}
    for name, kind, level in (("query_operands", binding.ATTN_QUERY, LEVEL), ("key_or_value_operands", binding.ATTN_KEY_VALUE, LEVEL),
                              ("outputs_to_shards", binding.ATTN_TO_SHARDS, P[0].level - 1)):
        rots = ctx.attention_pack_rotations(kind, dim, *shape)
        ckeys = [binding.SwitchKey(residues(allp, DNUM, 2), ctx.galois_element(r)) for r in rots]
        nin = dim if kind == binding.ATTN_TO_SHARDS else tokens // TI
        src = [binding.Ciphertext(q[x % dim].data[:, :level].contiguous(), 2.0 ** 40) for x in range(nin)]
        ctx.attention_pack(kind, src, dim, ckeys, *shape)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); ctx.attention_pack(kind, src, dim, ckeys, *shape); b.record()
        torch.cuda.synchronize()
        conv[name] = a.elapsed_time(b)
        conv[name + "_rotation_keys"] = len(rots)
        del ckeys, src
        ctx._ws = None
        torch.cuda.empty_cache()
    conv["q_k_v_and_back_s"] = (conv["query_operands"] + 2 * conv["key_or_value_operands"] + conv["outputs_to_shards"]) * 1e-3
    att["layout_conversions_ms"] = conv
    out["attention_32_heads_128_tokens_dim_128_ms"] = att
    return out


def main():
    global LAZY, NTT_BATCH
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--parts", default="abc", help="with --profile: which parts of the step to run (a: NTT, b: key switching, c: projection)")
    ap.add_argument("--shards", type=int, default=SHARDS, help="with --profile: token shards in the projection (default 16)")
    ap.add_argument("--ntt-batch", type=int, default=NTT_BATCH, help="with --profile: polynomials in the NTT part (default 32)")
    ap.add_argument("--mac-kernel", type=int, default=0, help="with --profile: CKKS_OPT_MAC_KERNEL value (82, 83, 81, 42, 100); 0 = the default")
    ap.add_argument("--conv-kernel", type=int, default=-1, help="with --profile: CKKS_OPT_CONV_KERNEL value (0 = FP64, 1 = tensor cores)")
    ap.add_argument("--eager-moddown", action="store_true",
                    help="one ModDown per giant-step rotation instead of one per output ciphertext")
    ap.add_argument("--no-extras", action="store_true", help="skip the untimed one-off measurements of the composite calls")
    ap.add_argument("--no-layer", action="store_true", help="skip the decoder-layer submetrics (seven projections and the attention products)")
    ap.add_argument("--layer-reps", type=int, default=3, help="timed repetitions of each decoder-layer call")
    ap.add_argument("--cpu-anchor", action="store_true",
                    help="with --impl reference: time the checker on one whole shard of the projection instead of the sample")
    ap.add_argument("--profile", action="store_true",
                    help="for profiler captures: honour --warmup below 3 and skip the e2e and CPU legs (prints no bench line)")
    args = ap.parse_args()
    LAZY = not args.eager_moddown
    if args.profile:
        NTT_BATCH = args.ntt_batch
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
