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
`value` is seconds per projection (part c); NTT limbs/s and key switches/s from parts
(a) and (b) ride along in `submetrics`.  Ciphertexts and keys are uniform residues
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
    keys = [inputs.uniform_residues(g, allp, N, DNUM * 2).reshape(DNUM, 2, L + K, N) for _ in range(2)]
    gals = [orc.galois_element(8), orc.galois_element(512)]
    z = np.repeat(g.normal(0, 0.02, HIDDEN), T_SHARD)
    t = {}
    t0 = time.perf_counter(); pts = [orc.encode(z, float(q[-1]), LEVEL) for _ in range(2)]; t["encode"] = (time.perf_counter() - t0) / 2
    t0 = time.perf_counter(); acc = orc.mul_plain_acc(ct, pts[0]); acc = orc.mul_plain_acc(ct, pts[1], acc); t["mac"] = (time.perf_counter() - t0) / 2
    t0 = time.perf_counter(); orc.rotate_hoisted(ct, keys, gals); t["hoisted_2"] = time.perf_counter() - t0
    t0 = time.perf_counter(); orc.rotate(ct, keys[0], gals[0]); t["rotate"] = time.perf_counter() - t0
    t0 = time.perf_counter(); orc.rotate_sum(np.stack([ct, ct]), keys, gals); t["rotate_sum_2"] = time.perf_counter() - t0
    t0 = time.perf_counter(); orc.rescale(acc); t["rescale"] = time.perf_counter() - t0
    t0 = time.perf_counter(); x = inputs.uniform_residues(g, q, N, 1); orc.intt(orc.ntt(x)); t["ntt_pair_24"] = time.perf_counter() - t0
    G = HIDDEN // BABY
    # a hoisted rotation costs (hoisted_2 - shared ModUp)/2; approximate the shared part by rotate - per-rotation part
    per_h = t["hoisted_2"] / 2
    # a two-term rotate_sum is two extended-basis terms and one ModDown, a rotation one term and one ModDown
    term = max(t["rotate_sum_2"] - t["rotate"], 0.0)
    moddown = max(t["rotate"] - term, 0.0)
    giant = (G - 1) * term + moddown if lazy else (G - 1) * t["rotate"]
    proj = (HIDDEN * t["encode"] + HIDDEN * SHARDS * t["mac"] + SHARDS * (BABY - 1) * per_h
            + SHARDS * giant + SHARDS * t["rescale"])
    cores = int(os.environ.get("OMP_NUM_THREADS", os.cpu_count() or 1))
    sample = ("2 encodes, 2 ct x pt MACs, 2 hoisted + 1 plain rotation, 1 two-term rotate_sum, 1 rescale, 24 NTT round trips at "
              "full size; scaled by the projection's counts (4096 encodes, 65536 MACs, 1008 hoisted rotations, "
              + ("1008 giant-step terms + 16 ModDowns" if lazy else "1008 plain rotations") + ", 16 rescales)")
    return {"proj_s": proj, "ntt_limbs_per_s": 48 / t["ntt_pair_24"], "key_switches_per_s": 1.0 / t["rotate"],
            "parts_s": t, "cores": cores, "sample": sample}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
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


def job_metrics(world, a_ms, b_ms, c_ms):
    """Whole-job figures from the slowest rank's part times: every rank ran the same step on its own replica."""
    limb_ntts = NTT_BATCH * L
    return {"value": c_ms * 1e-3 / world,                                   # seconds per projection, all ranks together
            "ntt_limbs_per_s": world * 2 * limb_ntts / (a_ms * 1e-3),
            "key_switches_per_s": world * (2 * NROT + 1) / (b_ms * 1e-3)}


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

    def part_b():
        for k in rot_keys:
            ctx.rotate(cta, k, out=rot_out)
        ctx.rotate_hoisted(cta, rot_keys, outs=hoist_out)
        ctx.mul_relin(cta, ctb, rlk, out=mul_out)

    def part_c():
        ctx.linear_proj(cts, W, proj_keys, HIDDEN, HIDDEN, T_SHARD, SH, BABY, outs=outs, ws=ws, lazy_moddown=LAZY)

    def step(times=None):
        e = [ev() for _ in range(4)]
        if args.profile:
            for name, f in (("a", part_a), ("b", part_b), ("c", part_c)):
                if name in args.parts:
                    f()
            return
        e[0].record(); part_a(); e[1].record(); part_b(); e[2].record(); part_c(); e[3].record()
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

    # outside the step, once each: the two composite calls that go beyond the scope table's rows
    def once(f):
        f()
        torch.cuda.synchronize()
        a, b = ev(), ev()
        a.record(); f(); b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    extras = {}
    if rank == 0 and not args.no_extras:
        extras["projection_%s_moddown_ms" % ("eager" if LAZY else "lazy")] = once(
            lambda: ctx.linear_proj(cts, W, proj_keys, HIDDEN, HIDDEN, T_SHARD, SH, BABY, outs=outs, ws=ws, lazy_moddown=not LAZY))
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

    total_ms, a_ms, b_ms, c_ms, e2e_ms, ntt_fwd_ms, e2e_pipe_ms = max_over_ranks([total_ms, a_ms, b_ms, c_ms, e2e_ms, ntt_fwd_ms, e2e_pipe_ms], dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk, pk_kind = peaks()
    limb_ntts = NTT_BATCH * L
    # Roofline of the dominant kernel family (the ntt16 kernels: 55 % of the step in the ncu launch list).
    # The butterflies run on the FP64 pipe, which ncu shows to be the busiest unit of the column passes, so the
    # bound is "alu": algorithmic work = 8 FP64 instructions per butterfly (6 for the exact twiddle product with
    # its quotient, 2 for the sum and difference), N/2 * log2 N butterflies per limb; peak = 64 FP64 instructions
    # per clock per SM (the DFMA rate ncu reports for this part) x SM count x the maximum SM clock.
    sm_count = torch.cuda.get_device_properties(local).multi_processor_count
    fp64_peak = 64.0 * sm_count * float(pk.get("sm_max_mhz", 1965.0)) * 1e6 / 1e12          # T instr/s
    ops = limb_ntts * (N // 2) * LOG_N * 8
    achieved = ops / (ntt_fwd_ms * 1e-3) / 1e12
    ntt_bytes = limb_ntts * 2 * 8 * N          # algorithmic bytes: each limb read once and written once
    hbm_achieved = ntt_bytes / (ntt_fwd_ms * 1e-3) / 1e9
    roofline = {"kernel": "ntt16_fwd_cols + ntt16_fwd_rows (forward NTT of 768 limbs, one launch each)", "bound": "alu",
                "achieved": achieved, "peak": fp64_peak, "unit": "T FP64 instr/s", "frac": achieved / fp64_peak,
                "traffic": 1523.0e6,   # ncu: dram read+write of the two launches (profiles/ntt16_768limbs.md), bytes
                "fp64_pipe_active_ncu": {"ntt16_fwd_cols": 0.761, "ntt16_fwd_rows": 0.670},
                "peak_kind": "derived: 64 DFMA/clk/SM x %d SMs x %.0f MHz" % (sm_count, float(pk.get("sm_max_mhz", 1965.0))),
                "ms_per_launch_pair": ntt_fwd_ms,
                # the same fraction against the clock the SMs held under the power cap during the timed steps
                "frac_at_sampled_clock": (achieved / (fp64_peak * float(clocks["sm_mhz"]) / float(pk.get("sm_max_mhz", 1965.0)))
                                          if clocks and clocks.get("sm_mhz") else None),
                "vs_register_resident_butterflies": {
                    "achieved_gbfly_s": limb_ntts * (N // 2) * LOG_N / (ntt_fwd_ms * 1e-3) / 1e9, "peak_gbfly_s": probe_rate / 1e9,
                    "frac": limb_ntts * (N // 2) * LOG_N / (ntt_fwd_ms * 1e-3) / probe_rate,
                    "peak_kind": "measured in this run: the transform's radix-16 butterfly groups on registers, 3 CTAs x 256 threads per SM"},
                "hbm": {"achieved": hbm_achieved, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": hbm_achieved / pk["hbm_gbs"],
                        "algorithmic_bytes": ntt_bytes, "peak_kind": pk_kind + " copy bandwidth"},
                "others": ({"ntt16 family": "49.6 % of the step (profiles/bench_step_launch_list.md)",
                            "mac_mma_kernel": "19.3 % of the step; legacy tensor path 32 % busy, DRAM 51 %, see profiles/mac_mma_projection_8shards.md",
                            "modup + moddown_conv + inner_product(_terms)": "28.3 % of the step; FP64 pipe 67 % (conversions), DRAM 60-72 % (inner products)"}
                           if LAZY else
                           {"ntt16 family": "55.0 % of the step (profiles/bench_step_launch_list.md)",
                            "mac_mma_kernel": "15.0 % of the step; legacy tensor path 32 % busy, DRAM 51 %, see profiles/mac_mma_projection_8shards.md",
                            "modup + moddown_conv + inner_product": "27.8 % of the step; FP64 pipe 67 % (conversions), DRAM 72 % (inner product)"})}
    cpu = oracle_sample(LAZY)
    jm = job_metrics(world, a_ms, b_ms, c_ms)
    line = {
        "metric": METRIC, "value": jm["value"], "unit": "s/projection", "n_gpus": world, "steps": args.steps,
        "warmup": nwarm, "ms_per_step": total_ms / args.steps, "higher_is_better": False, "scaling": "weak",
        "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": workload(), "l2": "inputs larger than L2 (>= 384 MiB per part)", "parallelism": f"replicas x{world}"},
        "extras": extras,
        "submetrics": {"ntt_limbs_per_s": jm["ntt_limbs_per_s"], "key_switches_per_s": jm["key_switches_per_s"],
                       "ms": {"ntt_roundtrip": a_ms, "keyswitch_part": b_ms, "projection": c_ms}},
        "clocks": clocks,
        "e2e": {"value": e2e_ms * 1e-3 / world, "unit": "s/projection", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "copies_overlapped_value": e2e_pipe_ms * 1e-3 / world},
        "gpu_launches": launches,
        "roofline": roofline,
        "cpu_baseline": {"value": cpu["proj_s"], "unit": "s/projection", "cores": cpu["cores"], "kind": "oracle",
                         "sample": cpu["sample"], "ntt_limbs_per_s": cpu["ntt_limbs_per_s"],
                         "key_switches_per_s": cpu["key_switches_per_s"]},
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--parts", default="abc", help="with --profile: which parts of the step to run (a: NTT, b: key switching, c: projection)")
    ap.add_argument("--shards", type=int, default=SHARDS, help="with --profile: token shards in the projection (default 16)")
    ap.add_argument("--eager-moddown", action="store_true",
                    help="one ModDown per giant-step rotation instead of one per output ciphertext")
    ap.add_argument("--no-extras", action="store_true", help="skip the untimed one-off measurements of the composite calls")
    ap.add_argument("--profile", action="store_true",
                    help="for profiler captures: honour --warmup below 3 and skip the e2e and CPU legs (prints no bench line)")
    args = ap.parse_args()
    global LAZY
    LAZY = not args.eager_moddown
    if args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
