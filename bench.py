#!/usr/bin/env python
"""Benchmark of the D2-MHE private gradient update on B200.

One step = one pass of the whole hot path over one batch of synthetic gradients:
encode -> encrypt -> neighbour sums -> decryption shares -> combine (scale-and-round) -> decode,
with every protocol message (ciphertexts, aggregates, shares) written to and read from HBM.
Metric: gradient coefficients per second per full round = K * params / t_round.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config 4] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank runs the same configuration on its
own range of ciphertext indices; nothing is exchanged inside a round (weak scaling).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2207_04604_b200 import workloads as wl  # noqa: E402

METRIC = "gradient coefficients/sec per full MHE round (enc+agg+dec); NTT GB/s vs HBM peak"
UNIT = "coeff/s"
STEP_CALLS = ["encode", "encrypt", "aggregate", "partial_decrypt", "combine_decrypt", "decode"]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index):
        self.rows = []
        self.proc = None
        self.device_index = device_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.device_index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            if len(r) < 8:
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def algorithmic_bytes(cfg, n_cts):
    """Protocol bytes per call for n_cts ciphertext indices of all K users (S = K share holders)."""
    K, S, A = cfg.num_parties, cfg.num_parties, cfg.degree + 1
    P = 8 * cfg.n * cfg.num_limbs
    units = K * n_cts
    return {
        "encode": units * cfg.n * 8,
        "encrypt": units * (4 * cfg.n + 2 * P),
        "aggregate": units * (A * 2 * P + 2 * P),
        "partial_decrypt": units * (P + S * P),
        "combine_decrypt": units * (P + S * P + 4 * cfg.n),
        "decode": units * cfg.n * 8,
    }


# Integer roofline of the transform-bearing kernels.  The scarce unit is the 32-bit integer
# multiply-add pipe.  Its rate is MEASURED in every run by the library's register-only loops
# (d2mhe_debug_int_throughput: mad.lo.u32, mad.wide.u32, mad.hi.u32, and the engine's butterfly)
# and the roofline's peak is the measured mad.lo rate in lane operations ("slots") per second;
# 148 SMs x 64 lanes x 1.965 GHz (unit counts and maximum clock) is printed beside it.  A widening
# or high-half multiply occupies the pipe for two slots (the measured rates say so).  Algorithmic
# slots: one lazy Shoup butterfly = 5 widening/high + 3 low multiplies = 13 slots (the primes of
# every configuration are 2^b - d with small d, which turns a fourth low multiply into a shift);
# a transform = (N/2) log2 N butterflies; a pointwise product = 14; one Philox4x32-10 call = 20
# widening multiplies = 40 slots (one call serves all L limbs).
IMAD_LANES_PER_SM = 64
NUM_SMS = 148
SM_MAX_HZ = 1.965e9
IMAD_PEAK_UNIT_COUNTS = NUM_SMS * IMAD_LANES_PER_SM * SM_MAX_HZ
SLOTS_PER_BUTTERFLY = 13


def algorithmic_mad_slots(cfg, n_cts):
    K, S, L, n = cfg.num_parties, cfg.num_parties, cfg.num_limbs, cfg.n
    transform = SLOTS_PER_BUTTERFLY * (n // 2) * cfg.log2_n   # slots per limb-transform
    units = K * n_cts
    return {
        # NTT(u) + 2 inverse transforms, 2 pointwise products, Lambda*m (10 slots) per limb; 3 samples per coefficient
        "encrypt": units * (L * (3 * transform + n * (2 * 14 + 10)) + 3 * 40 * n),
        # NTT(c1) once, then per share: pointwise product + inverse transform per limb, one sample per coefficient
        "partial_decrypt": units * (L * (transform + S * (transform + 14 * n)) + S * 40 * n),
    }


# dram__bytes_read.sum + dram__bytes_write.sum of the share kernel per (recipient, ciphertext) unit,
# from the ncu captures under profiles/ (taken on a few ciphertext indices of the configuration and
# scaled by the units of a launch: the traffic is the shares written plus c_1 and the noise bytes
# read, all proportional to the units).  None when the kernel has changed since the capture.
NCU_TRAFFIC_BYTES_PER_UNIT = {("resnet18-K50", "partial_decrypt"): (589769984 + 5258257000) / 100.0}


def measure_int_peak(ctx):
    """The integer rates of this GPU, measured now (lane operations per second)."""
    lo = max(ctx.debug_int_throughput(0, 4096) for _ in range(3))
    wide = max(ctx.debug_int_throughput(1, 4096) for _ in range(3))
    hi = max(ctx.debug_int_throughput(2, 4096) for _ in range(3))
    mul_wide = max(ctx.debug_int_throughput(4, 4096) for _ in range(3))
    mul_hi = max(ctx.debug_int_throughput(5, 4096) for _ in range(3))
    out = {"mad_lo_per_s": lo, "mad_wide_per_s": wide, "mad_hi_per_s": hi, "mul_wide_per_s": mul_wide,
           "mul_hi_per_s": mul_hi,
           "slots_per_mad_wide": lo / wide if wide else None, "slots_per_mad_hi": lo / hi if hi else None,
           "slots_per_mul_wide": lo / mul_wide if mul_wide else None, "slots_per_mul_hi": lo / mul_hi if mul_hi else None,
           "unit_count_peak_per_s": IMAD_PEAK_UNIT_COUNTS,
           "mad_lo_warp_instr_per_clk_per_sm_at_max_clock": lo / 32 / NUM_SMS / SM_MAX_HZ}
    try:
        bf = max(ctx.debug_int_throughput(3, 2048) for _ in range(3))
        out["butterflies_per_s_registers_only"] = bf
        out["butterfly_loop_frac_of_peak"] = bf * SLOTS_PER_BUTTERFLY / lo
        out["cycles_per_warp_butterfly_per_scheduler_at_max_clock"] = NUM_SMS * 4 * SM_MAX_HZ / (bf / 32)
    except Exception:  # primes outside the form the probe's butterfly is written for
        pass
    return out


# ----------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands
# ----------------------------------------------------------------------------------


def oracle_round(cfg, seed, ct_first, n_cts, o=None, pk=None):
    from oracle import d2mhe_oracle as orc

    if o is None:
        psi_t = pow(3, (wl.PLAIN_MODULUS - 1) // (2 * cfg.n), wl.PLAIN_MODULUS)
        o = orc.Oracle(cfg.log2_n, cfg.moduli, wl.PLAIN_MODULUS, seed, psi_t=psi_t)
    K = cfg.num_parties
    parties = list(range(K))
    if pk is None:
        pk = o.collective_pk(parties)
    offsets, rows = wl.regular_graph(K, cfg.degree, seed)
    values = wl.gradients(cfg, seed, ct_first, n_cts)
    t0 = time.perf_counter()
    ct = o.encrypt(pk, parties, ct_first, o.encode(values))
    agg = o.aggregate(ct, offsets, rows)
    shares = o.partial_decrypt(agg, parties, parties, ct_first)
    sums = o.decode(o.combine(agg, shares))
    dt = time.perf_counter() - t0
    return dt, sums, values, offsets, rows, o, pk


def coeffs_of(cfg, ct_first, n_cts):
    """Gradient coefficients (of all K users) carried by ciphertext indices ct_first .. ct_first+n_cts-1."""
    lo, hi = ct_first * cfg.n, min(cfg.params, (ct_first + n_cts) * cfg.n)
    return cfg.num_parties * max(0, hi - lo)


def cpu_baseline(cfg, seed, budget_s=15.0):
    """Times the oracle on as many ciphertext indices of the workload as fit the budget."""
    from oracle import d2mhe_oracle as orc

    dt, _, _, _, _, o, pk = oracle_round(cfg, seed, 0, 1)
    n_cts = 1
    if dt < budget_s / 3:
        n_cts = int(max(1, min(cfg.num_cts, budget_s / max(dt, 1e-6))))
        dt, *_ = oracle_round(cfg, seed, 0, n_cts, o, pk)
    return {"value": coeffs_of(cfg, 0, n_cts) / dt, "unit": UNIT, "cores": orc.threads(), "kind": "oracle",
            "sample": "ciphertext indices 0..%d of %d, all %d users and share holders, %.2f s"
                      % (n_cts - 1, cfg.num_cts, cfg.num_parties, dt)}


def config_dict(cfg):
    """The workload's description: the same keys and values in both arms."""
    return {"workload": cfg.name, "K": cfg.num_parties, "N": cfg.n, "L": cfg.num_limbs,
            "cts_per_user": cfg.num_cts, "params_per_user": cfg.params}


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import d2mhe_oracle as orc

    dt1, _, _, _, _, o, pk = oracle_round(cfg, args.seed, 0, 1)
    per_step_budget = 120.0 / max(1, args.steps + args.warmup)
    n_cts = int(max(1, min(cfg.num_cts, per_step_budget / max(dt1, 1e-6))))
    for _ in range(args.warmup):
        oracle_round(cfg, args.seed, 0, n_cts, o, pk)
    total = 0.0
    for _ in range(args.steps):
        dt, *_ = oracle_round(cfg, args.seed, 0, n_cts, o, pk)
        total += dt
    value = coeffs_of(cfg, 0, n_cts) * args.steps / total
    sample = "each step: ciphertext indices 0..%d of %d, all %d users and share holders" % (
        n_cts - 1, cfg.num_cts, cfg.num_parties)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": config_dict(cfg),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------
# the CUDA arm
# ----------------------------------------------------------------------------------


def measure_round(cfg, args, steps, warmup, rank, local_rank, world, detailed, sampler=None, n_cts=None):
    """Times one configuration.  detailed: also the call-by-call pass (per-kernel durations), the
    host-buffer pass (e2e) and the transform micro-benchmark.  n_cts: only the first n_cts
    ciphertext indices of the workload (a labelled slice, for profiling)."""
    import torch

    from paper_2207_04604_b200 import d2mhe, parallel

    dev = torch.device("cuda", local_rank)
    K, L, n = cfg.num_parties, cfg.num_limbs, cfg.n
    C = cfg.num_cts if not n_cts else min(n_cts, cfg.num_cts)
    parties = list(range(K))
    offsets, rows = wl.regular_graph(K, cfg.degree, args.seed)
    ct_first, _ = wl.shard_ct_range(rank, world, C)  # each rank: its own C ciphertext indices
    ctx = d2mhe.Context(cfg.log2_n, cfg.moduli, K, seed=args.seed, device=local_rank)
    stream = torch.cuda.current_stream(dev)

    # Initialization (reported separately, as the paper does): key shares and the collective key.
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    ev1.record(stream)
    ctx.sync()
    init_ms = ev0.elapsed_time(ev1)
    int_peak = measure_int_peak(ctx) if detailed and rank == 0 else None

    values_np = wl.gradients(cfg, args.seed, ct_first, C)
    values = torch.from_numpy(values_np).to(dev)
    sums = torch.empty((K, C, n), dtype=torch.int32, device=dev)
    # chunking: keep all protocol messages of the sub-chunks in flight in HBM at once
    free_b, _ = torch.cuda.mem_get_info(dev)
    per_ct = ctx.round_workspace_bytes(1) - 256
    chunk = int(max(1, min(C, (int(free_b * 0.6)) // per_ct)))
    if args.chunk:
        chunk = min(chunk, args.chunk)
    ws = torch.empty(ctx.round_workspace_bytes(chunk), dtype=torch.uint8, device=dev)
    flush = torch.empty(384 * 1024 * 1024, dtype=torch.uint8, device=dev)  # > 126 MB L2
    idx = [torch.as_tensor(rows[offsets[i]:offsets[i + 1]].astype(np.int64), device=dev) for i in range(K)]

    def sums_are_right(t):
        """Every decrypted sum equals the plaintext neighbour sum (checked on the device)."""
        return all(bool(torch.equal(t[i], values[idx[i]].sum(dim=0, dtype=torch.int32))) for i in range(K))

    def barrier():
        parallel.barrier(dev)

    # ---- timed region: the whole round as one call (sub-chunks overlapped on internal streams) ----
    def step():
        ctx.round_device(values, ct_first, C, offsets, rows, sums, ws)

    for _ in range(warmup):
        flush.zero_()
        step()
    barrier()
    if not sums_are_right(sums):
        raise RuntimeError("decrypted neighbour sums differ from the plaintext sums")

    if sampler is not None:
        sampler.start()
    launches0 = ctx.launch_count()
    step_events = []
    barrier()
    wall0 = time.perf_counter()
    for _ in range(steps):
        flush.zero_()  # evict the previous step's messages from L2 (outside the timed events)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        step()
        e1.record(stream)
        step_events.append((e0, e1))
    barrier()
    wall = time.perf_counter() - wall0
    launches = ctx.launch_count() - launches0
    step_ms = sum(a.elapsed_time(b) for a, b in step_events) / steps
    step_ms_max = parallel.max_over_ranks(step_ms, dev)
    coeffs_per_step = world * coeffs_of(cfg, 0, C)
    res = {"cfg": cfg, "C": C, "chunk": chunk, "ms_per_step": step_ms_max, "value": coeffs_per_step / (step_ms_max * 1e-3),
           "launches": int(launches), "init_ms": init_ms, "wall_ms_per_step_incl_flush": wall * 1e3 / steps,
           "int_peak": int_peak, "sub_chunks": d2mhe.round_plan(C, chunk)[0]}
    if not detailed:
        if sampler is not None:
            res["clocks"] = sampler.stop()
        ctx.close()
        return res

    # ---- the same round call by call on one stream, with an event between the calls: each kernel's
    # launch duration (nothing overlaps here), its share of the step and the roofline entry ----
    # The three large message buffers of this pass are views of the round call's workspace (the two
    # passes never run at the same time); the ragged last chunk uses the same storage.
    def alloc(cc):
        n_ct, n_sh = K * cc * 2 * L * n, K * K * cc * L * n
        words = ws[:8 * (2 * n_ct + n_sh)].view(torch.int64)
        return (torch.empty((K, cc, n), dtype=torch.int32, device=dev), ctx.empty_u32(K, cc, n),
                words[:n_ct].view(K, cc, 2, L, n), words[n_ct:2 * n_ct].view(K, cc, 2, L, n),
                words[2 * n_ct:].view(K, K, cc, L, n),
                ctx.empty_u32(K, cc, n), torch.empty((K, cc, n), dtype=torch.int32, device=dev))

    bufs = {chunk: alloc(chunk)}
    if C % chunk:
        bufs[C % chunk] = alloc(C % chunk)

    def serial_step(events=None):
        for first in range(0, C, chunk):
            cc = min(chunk, C - first)
            v, p, c_, a, s, o_, r = bufs[cc]
            v.copy_(values[:, first:first + cc])
            marks = []

            def mark():
                if events is not None:
                    e = torch.cuda.Event(enable_timing=True)
                    e.record(stream)
                    marks.append(e)

            mark()
            ctx.encode(v, K * cc, p)
            mark()
            ctx.encrypt(parties, ct_first + first, cc, p, c_)
            mark()
            ctx.aggregate(c_, K, cc, offsets, rows, a)
            mark()
            ctx.partial_decrypt(a, parties, parties, ct_first + first, cc, s)
            mark()
            ctx.combine_decrypt(a, s, K, K, cc, o_)
            mark()
            ctx.decode(o_, K * cc, r)
            mark()
            sums[:, first:first + cc].copy_(r)
            if events is not None:
                events.append(marks)

    long_step = step_ms_max > 500.0  # seconds-long rounds: a few steps per extra pass are enough
    serial_steps = 2 if long_step else max(3, min(steps, 50))
    sums.zero_()
    for _ in range(1 if long_step else min(warmup, 3)):
        flush.zero_()
        serial_step()
    if not sums_are_right(sums):
        raise RuntimeError("call-by-call round differs from the plaintext sums")
    chunk_events, serial_events = [], []
    for _ in range(serial_steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        serial_step(chunk_events)
        e1.record(stream)
        serial_events.append((e0, e1))
    torch.cuda.synchronize(dev)
    if sampler is not None:
        res["clocks"] = sampler.stop()
    res["serial_ms"] = sum(a.elapsed_time(b) for a, b in serial_events) / serial_steps
    per_call = {name: 0.0 for name in STEP_CALLS}
    for marks in chunk_events:
        for i, name in enumerate(STEP_CALLS):
            per_call[name] += marks[i].elapsed_time(marks[i + 1])
    res.update(per_call=per_call, serial_steps=serial_steps, n_chunks_total=len(chunk_events))
    bufs.clear()
    torch.cuda.empty_cache()

    # end to end through the host-buffer entry point: H2D of the gradients, the round, D2H of the sums
    hv = torch.from_numpy(values_np).pin_memory()
    hs = torch.zeros((K, C, n), dtype=torch.int32).pin_memory()
    for _ in range(1 if long_step else 2):
        ctx.round_host(hv, ct_first, C, offsets, rows, hs, ws)
    sums.copy_(hs)
    if not sums_are_right(sums):
        raise RuntimeError("host-buffer round differs from the plaintext sums")
    e2e_steps = 3 if long_step else max(3, min(steps, 50))
    barrier()
    e2e_total, e2e_each = 0.0, []
    for _ in range(e2e_steps):
        flush.zero_()
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()  # host clock: the call returns when the sums are in host memory
        ctx.round_host(hv, ct_first, C, offsets, rows, hs, ws)
        e2e_each.append(time.perf_counter() - t0)
        e2e_total += e2e_each[-1]
    barrier()
    e2e_ms_max = parallel.max_over_ranks(e2e_total * 1e3 / e2e_steps, dev)
    res["e2e"] = {"value": coeffs_per_step / (e2e_ms_max * 1e-3), "unit": UNIT, "h2d_bytes_per_step": K * C * n * 4,
                  "d2h_bytes_per_step": K * C * n * 4, "ms_per_step": e2e_ms_max,
                  "ms_per_step_median": float(np.median(e2e_each)) * 1e3, "steps": e2e_steps}
    del hv, hs

    # transform / multiply-add micro-benchmark on this configuration's ring (batch > L2), and the
    # conversion / refresh calls (the paper's own decryption path and its bootstrap) on a few indices
    res["ntt"] = res["convert_bootstrap"] = None
    if rank == 0 and not args.no_extras:
        del ws
        torch.cuda.empty_cache()
        res["ntt"] = ntt_microbench(ctx, cfg, dev, stream, flush)
        torch.cuda.empty_cache()
        res["convert_bootstrap"] = convert_bootstrap_bench(ctx, cfg, dev, stream, flush, offsets, rows, args.seed)
    ctx.close()
    return res


def ntt_microbench(ctx, cfg, dev, stream, flush):
    import torch

    L, n = cfg.num_limbs, cfg.n
    batch = max(1, (384 << 20) // (8 * n * L))
    polys = torch.randint(0, min(cfg.moduli), (batch, L, n), dtype=torch.int64, device=dev)
    other, third, out = polys.clone(), polys.clone(), torch.empty_like(polys)

    def timed(fn, reps=5):
        fn()
        best = None
        for _ in range(reps):
            flush.zero_()
            a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a_.record(stream)
            fn()
            b_.record(stream)
            torch.cuda.synchronize(dev)
            ms = a_.elapsed_time(b_)
            best = ms if best is None else min(best, ms)
        return best

    nbytes = 16.0 * n * L * batch
    f_ms = timed(lambda: ctx.ntt_forward(polys, batch))
    i_ms = timed(lambda: ctx.ntt_inverse(polys, batch))
    m_ms = timed(lambda: ctx.poly_muladd(polys, other, third, out, batch))
    bfly = batch * L * (n // 2) * cfg.log2_n
    return {"shape": [batch, L, n], "forward_GBps": nbytes / 1e9 / (f_ms * 1e-3),
            "inverse_GBps": nbytes / 1e9 / (i_ms * 1e-3), "muladd_GBps": 2 * nbytes / 1e9 / (m_ms * 1e-3),
            "forward_butterflies_per_s": bfly / (f_ms * 1e-3), "inverse_butterflies_per_s": bfly / (i_ms * 1e-3),
            "bytes_per_coeff": {"ntt": 16, "muladd": 32}}


def convert_bootstrap_bench(ctx, cfg, dev, stream, flush, offsets, rows, seed):
    """MBFV.Convert to the recipients' own keys (+ BFV.Decrypt) and MBFV.Bootstrap on the first few
    ciphertext indices of the workload, all K recipients and share holders: CUDA-event time per call
    and the share calls' fraction of the integer roofline (slots counted as for the decryption shares:
    Convert = NTT(c_1) once, then per share NTT(mu_k), two inverse transforms, three pointwise
    products per limb and three samples per coefficient; Bootstrap = NTT(c_1), NTT(alpha) and L
    samples per coefficient once, then per share two inverse transforms, two products and Lambda M_k
    per limb and three samples per coefficient)."""
    import torch

    K, L, n = cfg.num_parties, cfg.num_limbs, cfg.n
    free_b, _ = torch.cuda.mem_get_info(dev)
    per_ct = K * K * 2 * L * n * 8 + 4 * K * 2 * L * n * 8
    cc = int(max(1, min(cfg.num_cts, 4, int(free_b * 0.5) // per_ct)))
    parties = list(range(K))
    values = torch.from_numpy(wl.gradients(cfg, seed, 0, cc)).to(dev)
    plain = ctx.empty_u32(K, cc, n)
    ct, agg = ctx.empty_u64(K, cc, 2, L, n), ctx.empty_u64(K, cc, 2, L, n)
    shares = ctx.empty_u64(K, K, cc, 2, L, n)
    conv, scratch = ctx.empty_u64(K, cc, 2, L, n), ctx.empty_u64(K, cc, L, n)
    out_plain = ctx.empty_u32(K, cc, n)
    sums = torch.empty((K, cc, n), dtype=torch.int32, device=dev)
    ctx.encode(values, K * cc, plain)
    ctx.encrypt(parties, 0, cc, plain, ct)
    ctx.aggregate(ct, K, cc, offsets, rows, agg)
    ctx.user_keygen(parties)

    def timed(fn, reps=3):
        fn()
        best = None
        for _ in range(reps):
            flush.zero_()
            a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a_.record(stream)
            fn()
            b_.record(stream)
            torch.cuda.synchronize(dev)
            ms = a_.elapsed_time(b_)
            best = ms if best is None else min(best, ms)
        return best

    idx = [torch.as_tensor(rows[offsets[i]:offsets[i + 1]].astype(np.int64), device=dev) for i in range(K)]

    def check(what):
        ctx.decode(out_plain, K * cc, sums)
        ok = all(bool(torch.equal(sums[i], values[idx[i]].sum(dim=0, dtype=torch.int32))) for i in range(K))
        if not ok:
            raise RuntimeError(what + ": decrypted sums differ from the plaintext sums")

    t_cs = timed(lambda: ctx.convert_share(agg, parties, parties, 0, cc, shares))
    t_cc = timed(lambda: ctx.convert_combine(agg, shares, K, K, cc, conv))
    t_cd = timed(lambda: ctx.decrypt(parties, conv, cc, scratch, out_plain))
    check("Convert")
    t_bs = timed(lambda: ctx.bootstrap_share(agg, parties, parties, 0, cc, shares))
    t_bc = timed(lambda: ctx.bootstrap_combine(agg, shares, parties, K, 0, cc, out_plain, conv))
    # the refreshed ciphertext decrypts to the same sums through the ordinary collective decryption
    sh1 = shares.view(-1)[:K * K * cc * L * n].view(K, K, cc, L, n)
    ctx.partial_decrypt(conv, parties, parties, 0, cc, sh1)
    ctx.combine_decrypt(conv, sh1, K, K, cc, out_plain)
    check("Bootstrap")
    T = SLOTS_PER_BUTTERFLY * (n // 2) * cfg.log2_n
    units, S = K * cc, K
    slots_conv = units * (L * (T + S * (3 * T + 3 * 14 * n)) + S * 3 * 40 * n)
    slots_boot = units * (L * (2 * T + 40 * n + S * (2 * T + 2 * 14 * n + 10 * n)) + S * 3 * 40 * n)
    return {"cts": cc, "units": units,
            "convert_share_ms": t_cs, "convert_combine_ms": t_cc, "decrypt_ms": t_cd,
            "bootstrap_share_ms": t_bs, "bootstrap_combine_ms": t_bc,
            "convert_share_slots": slots_conv, "bootstrap_share_slots": slots_boot,
            "share_bytes": units * S * 2 * 8 * n * L}


def narrow_round_bench(args, local_rank):
    """The MNIST-shaped round on seven 30-bit limbs (log q = 210 against 216) through the 32-bit-word
    protocol calls, call by call on one stream, and the same parameter set through the 64-bit-word
    calls: a separate, labelled line (the benchmark configurations fix their 54-bit primes)."""
    import torch

    from paper_2207_04604_b200 import d2mhe

    cfg = wl.narrow_round_config()
    dev = torch.device("cuda", local_rank)
    stream = torch.cuda.current_stream(dev)
    K, L, n, C = cfg.num_parties, cfg.num_limbs, cfg.n, cfg.num_cts
    parties = list(range(K))
    offsets, rows = wl.regular_graph(K, cfg.degree, args.seed)
    ctx = d2mhe.Context(cfg.log2_n, cfg.moduli, K, seed=args.seed, device=local_rank)
    ctx.keygen_share(parties)
    ctx.collective_pk(parties)
    values = torch.from_numpy(wl.gradients(cfg, args.seed)).to(dev)
    flush = torch.empty(384 * 1024 * 1024, dtype=torch.uint8, device=dev)
    idx = [torch.as_tensor(rows[offsets[i]:offsets[i + 1]].astype(np.int64), device=dev) for i in range(K)]
    plain, out_plain = ctx.empty_u32(K, C, n), ctx.empty_u32(K, C, n)
    sums = torch.empty((K, C, n), dtype=torch.int32, device=dev)
    names = ["encode", "encrypt", "aggregate", "partial_decrypt", "combine_decrypt", "decode"]

    def run(words32, reps=10):
        mk = ctx.empty_u32 if words32 else ctx.empty_u64
        ct, agg, sh = mk(K, C, 2, L, n), mk(K, C, 2, L, n), mk(K, K, C, L, n)
        calls = [lambda: ctx.encode(values, K * C, plain),
                 (lambda: ctx.encrypt32(parties, 0, C, plain, ct)) if words32 else (lambda: ctx.encrypt(parties, 0, C, plain, ct)),
                 (lambda: ctx.aggregate32(ct, K, C, offsets, rows, agg)) if words32 else (lambda: ctx.aggregate(ct, K, C, offsets, rows, agg)),
                 (lambda: ctx.partial_decrypt32(agg, parties, parties, 0, C, sh)) if words32 else (lambda: ctx.partial_decrypt(agg, parties, parties, 0, C, sh)),
                 (lambda: ctx.combine_decrypt32(agg, sh, K, K, C, out_plain)) if words32 else (lambda: ctx.combine_decrypt(agg, sh, K, K, C, out_plain)),
                 lambda: ctx.decode(out_plain, K * C, sums)]
        per = [0.0] * len(calls)
        total = 0.0
        for it in range(reps + 3):
            flush.zero_()
            marks = [torch.cuda.Event(enable_timing=True) for _ in range(len(calls) + 1)]
            marks[0].record(stream)
            for i, fn in enumerate(calls):
                fn()
                marks[i + 1].record(stream)
            torch.cuda.synchronize(dev)
            if it == 0 and not all(bool(torch.equal(sums[i], values[idx[i]].sum(dim=0, dtype=torch.int32))) for i in range(K)):
                raise RuntimeError("narrow round: decrypted sums differ from the plaintext sums")
            if it >= 3:
                total += marks[0].elapsed_time(marks[-1])
                for i in range(len(calls)):
                    per[i] += marks[i].elapsed_time(marks[i + 1])
        return total / reps, {nm: t / reps for nm, t in zip(names, per)}

    ms32, per32 = run(True)
    ms64, per64 = run(False)
    lo = max(ctx.debug_int_throughput(0, 4096) for _ in range(3))
    t32 = 4 * (n // 2) * cfg.log2_n  # one high and two low multiplies per 32-bit butterfly
    slots_pdec = K * C * (L * (t32 + K * (t32 + 4 * n)) + K * 40 * n)
    coeffs = coeffs_of(cfg, 0, C)
    ctx.close()
    return {"config": config_dict(cfg), "note": "call by call on one stream; not the headline (its primes are not the benchmark's)",
            "words32": {"ms_per_round": ms32, "value": coeffs / (ms32 * 1e-3), "unit": UNIT, "calls_ms": per32,
                        "partial_decrypt_alu_frac": slots_pdec / (per32["partial_decrypt"] * 1e-3) / lo,
                        "slots_per_butterfly": 4},
            "words64_same_primes": {"ms_per_round": ms64, "value": coeffs / (ms64 * 1e-3), "unit": UNIT, "calls_ms": per64}}


def run_cuda(args, cfg):
    import torch

    from paper_2207_04604_b200 import build, parallel

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    rank, local_rank, world = parallel.init()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if rank == 0:
        build.build()
    parallel.barrier(dev)

    sampler = ClockSampler(local_rank) if rank == 0 else None
    res = measure_round(cfg, args, args.steps, args.warmup, rank, local_rank, world, True, sampler, args.cts)
    others = {}
    if rank == 0 and world == 1 and not args.no_other_configs and not args.cts:
        # the smaller round configurations, one short pass each (device-resident value only)
        for i in (1, 2, 3):
            c2 = wl.round_config(i)
            if c2.name == cfg.name:
                continue
            torch.cuda.empty_cache()
            r2 = measure_round(c2, args, 10, 3, 0, local_rank, 1, False)
            others[c2.name] = {"config": config_dict(c2), "ms_per_step": r2["ms_per_step"], "value": r2["value"],
                               "unit": UNIT, "steps": 10, "warmup": 3, "sub_chunks": r2["sub_chunks"],
                               "round_hbm_frac": sum(algorithmic_bytes(c2, c2.num_cts).values()) / 1e9
                               / (r2["ms_per_step"] * 1e-3) / measured_peaks()[0]}

    narrow = None
    if rank == 0 and world == 1 and not args.no_other_configs and not args.cts:
        torch.cuda.empty_cache()
        narrow = narrow_round_bench(args, local_rank)

    if rank == 0:
        K, L, n, C = cfg.num_parties, cfg.num_limbs, cfg.n, res["C"]
        peak, peak_kind = measured_peaks()
        clocks = res.get("clocks") or {}
        mhz = clocks.get("sm_mhz")
        ip = res["int_peak"]
        imad_peak = ip["mad_lo_per_s"]

        def mcycles(ms):  # duration x median sampled SM clock: comparable across clock states
            return ms * mhz * 1e-3 if (mhz and ms is not None) else None

        ab = algorithmic_bytes(cfg, C)
        per_call, serial_steps, n_chunks_total = res["per_call"], res["serial_steps"], res["n_chunks_total"]
        total_ms = sum(per_call.values())
        slots = algorithmic_mad_slots(cfg, C)
        ntt = res["ntt"]
        for k_ in ("forward", "inverse", "muladd") if ntt else ():
            ntt[k_ + "_frac_of_hbm"] = ntt[k_ + "_GBps"] / peak
        for k_ in ("forward", "inverse") if ntt else ():
            ntt[k_ + "_alu_frac"] = ntt[k_ + "_butterflies_per_s"] * SLOTS_PER_BUTTERFLY / imad_peak
        cb = res["convert_bootstrap"]
        for k_ in ("convert", "bootstrap") if cb else ():
            cb[k_ + "_share_alu_frac"] = cb[k_ + "_share_slots"] / (cb[k_ + "_share_ms"] * 1e-3) / imad_peak
            cb[k_ + "_share_GBps"] = cb["share_bytes"] / 1e9 / (cb[k_ + "_share_ms"] * 1e-3)
        kernels = {}
        for name in STEP_CALLS:
            ms = per_call[name] / serial_steps  # per step, summed over chunks
            kernels[name] = {"ms_per_step": ms, "mcycles_per_step": mcycles(ms),
                             "share": per_call[name] / total_ms if total_ms else None,
                             "algorithmic_GB": ab[name] / 1e9, "GBps": ab[name] / 1e9 / (ms * 1e-3) if ms else None,
                             "hbm_frac": ab[name] / 1e9 / (ms * 1e-3) / peak if ms else None}
            if name in slots:
                kernels[name]["alu_frac"] = slots[name] / (ms * 1e-3) / imad_peak if ms else None
        kernels["aggregate"]["note"] = ("algorithmic bytes count every list's read of a ciphertext; the ciphertexts were "
                                        "just written and most of those reads hit L2, so this is not a DRAM roofline fraction")
        dominant = max(STEP_CALLS, key=lambda k_: per_call[k_])
        chunks_per_step = n_chunks_total / serial_steps
        dur_ms = per_call[dominant] / n_chunks_total
        units_per_launch = K * C / chunks_per_step
        achieved = ab[dominant] / chunks_per_step / 1e9 / (dur_ms * 1e-3)
        per_unit = NCU_TRAFFIC_BYTES_PER_UNIT.get((cfg.name, dominant))
        traffic = per_unit * units_per_launch if per_unit else None
        if dominant in slots:  # transform-bearing kernel: bound by the integer multiply-add pipe
            got = slots[dominant] / chunks_per_step / (dur_ms * 1e-3)
            roofline = {"bound": "alu", "kernel": dominant, "achieved": got / 1e12, "peak": imad_peak / 1e12,
                        "unit": "T int32 multiply-add slots/s", "frac": got / imad_peak,
                        "peak_source": "measured in this run: mad.lo.u32 lane operations/s of a register-only loop on "
                                       "all SMs (d2mhe_debug_int_throughput); unit counts x maximum clock give %.2f"
                                       % (IMAD_PEAK_UNIT_COUNTS / 1e12),
                        "frac_of_unit_count_peak": got / IMAD_PEAK_UNIT_COUNTS,
                        "traffic": traffic, "avg_launch_ms": dur_ms, "avg_launch_mcycles": mcycles(dur_ms),
                        "units_per_launch": units_per_launch,
                        "launches_note": "one call = the sampling kernel (about 5 % of the time) followed by the "
                                         "transform kernel; traffic is the transform kernel's, scaled from a capture "
                                         "of a few ciphertext indices by the (recipient, ciphertext) units of a launch",
                        "hbm": {"achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                                "peak_source": "of " + peak_kind}}
        else:
            roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak, "unit": "GB/s",
                        "frac": achieved / peak, "peak_source": "of " + peak_kind, "traffic": traffic,
                        "avg_launch_ms": dur_ms}
        round_bytes = sum(ab.values())
        config = config_dict(cfg)
        if args.cts:
            config["slice"] = "first %d ciphertext indices only (profiling run, not the benchmark)" % C
        line = {
            "metric": METRIC, "value": res["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": res["ms_per_step"], "mcycles_per_step": mcycles(res["ms_per_step"]),
            "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u64", "data": "synthetic",
            "config": config,
            "launch": {"graph_degree": cfg.degree, "share_holders": K, "chunk_cts": res["chunk"],
                       "sub_chunks": res["sub_chunks"],
                       "entry_point": "d2mhe_round_device (sub-chunks overlapped on two internal streams)",
                       "l2": "384 MB buffer written between timed steps (L2 flush)",
                       "parallelism": "ciphertext-index shards, no exchange" if world > 1 else "single GPU"},
            "clocks": clocks,
            "e2e": res["e2e"],
            "gpu_launches": res["launches"],
            "roofline": roofline,
            "integer_peak": ip,
            "round_hbm_frac": round_bytes / 1e9 / (res["ms_per_step"] * 1e-3) / peak,
            "ms_per_step_call_by_call": res["serial_ms"],
            "kernels_note": "per-call durations from a separate pass of the same round, call by call on one stream; "
                            "mcycles = duration x median sampled SM clock",
            "kernels": kernels,
            "ntt": ntt,
            "convert_bootstrap": cb,
            "other_configs": others,
            "narrow_words": narrow,
            "init_ms": res["init_ms"],
            "wall_ms_per_step_incl_flush": res["wall_ms_per_step_incl_flush"],
            "cpu_baseline": cpu_baseline(cfg, args.seed) if world == 1 and not args.no_cpu_baseline else None,
        }
        print(json.dumps(line))
    parallel.finish()


def run_sweep(args):
    """Kernel sweep (configuration 5): batched forward/inverse transforms and the RNS multiply-add over
    N in 2^12..2^16, L in {1,4,8,16,24}, batch in {1,64,1024,4096}, uniform residues mod 60-bit primes
    (50-bit with --sweep-bits 50).  One JSON line with a row per point; GB/s = 16 B (transforms) or 32 B
    (multiply-add) per residue over the CUDA-event time, against the measured HBM copy bandwidth.
    --sweep-bits 30 (or less) runs the 32-bit-word calls instead: 8 and 16 B per residue, N up to 2^14
    for the transforms."""
    import torch

    from paper_2207_04604_b200 import build, d2mhe

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    build.build()
    dev = torch.device("cuda", 0)
    stream = torch.cuda.current_stream(dev)
    peak, peak_kind = measured_peaks()
    flush = torch.empty(384 * 1024 * 1024, dtype=torch.uint8, device=dev)
    free_b, _ = torch.cuda.mem_get_info(dev)
    rows = []
    imad_peak = None  # the mad.lo rate of this GPU, measured with the first context
    only = [int(x) for x in args.sweep_point.split(",")] if args.sweep_point else None  # N, L, batch
    for log2_n in wl.SWEEP_LOG2_N:
        n = 1 << log2_n
        if only and n != only[0]:
            continue
        for L in wl.SWEEP_LIMBS:
            if only and L != only[1]:
                continue
            moduli = wl.sweep_moduli(args.sweep_bits, L)
            ctx = d2mhe.Context(log2_n, moduli, 1, seed=args.seed)
            if imad_peak is None:
                imad_peak = max(ctx.debug_int_throughput(0, 4096) for _ in range(3))
            narrow = args.sweep_bits <= 30
            slots_per_bfly = 4 if narrow else SLOTS_PER_BUTTERFLY
            word = 4 if narrow else 8
            host_tile = wl.random_polys(moduli, log2_n, 1, args.seed)
            tile = torch.from_numpy(host_tile.astype(np.uint32).view(np.int32) if narrow else host_tile.view(np.int64)).to(dev)
            fwd, inv, mad = ((ctx.ntt32_forward, ctx.ntt32_inverse, ctx.poly_muladd32) if narrow
                             else (ctx.ntt_forward, ctx.ntt_inverse, ctx.poly_muladd))
            for batch in ([only[2]] if only else wl.SWEEP_BATCH):
                nbytes = word * n * L * batch
                row = {"N": n, "L": L, "batch": batch, "GiB": nbytes / 2**30}
                if nbytes > 0.6 * free_b:
                    row["skipped"] = "buffer exceeds the memory budget"
                    rows.append(row)
                    continue
                polys = tile.expand(batch, L, n).contiguous()

                def timed(fn, reps=3):
                    fn()
                    best = None
                    for _ in range(reps):
                        flush.zero_()
                        a_, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                        a_.record(stream)
                        fn()
                        b_.record(stream)
                        torch.cuda.synchronize(dev)
                        ms = a_.elapsed_time(b_)
                        best = ms if best is None else min(best, ms)
                    return best

                if not narrow or log2_n <= 14:
                    f_ms = timed(lambda: fwd(polys, batch))
                    i_ms = timed(lambda: inv(polys, batch))
                    row.update({"forward_GBps": 2 * nbytes / 1e9 / (f_ms * 1e-3), "inverse_GBps": 2 * nbytes / 1e9 / (i_ms * 1e-3)})
                if 4 * nbytes <= 0.6 * free_b:
                    b2, c2, d2_ = polys.clone(), polys.clone(), torch.empty_like(polys)
                    m_ms = timed(lambda: mad(polys, b2, c2, d2_, batch))
                    row["muladd_GBps"] = 4 * nbytes / 1e9 / (m_ms * 1e-3)
                    del b2, c2, d2_
                row["in_l2_or_launch_bound"] = bool(nbytes < 2 * 126e6 or batch * L < NUM_SMS)
                for k_ in ("forward", "inverse", "muladd"):
                    if k_ + "_GBps" in row:
                        row[k_ + "_frac_of_hbm"] = row[k_ + "_GBps"] / peak
                for k_ in ("forward", "inverse"):
                    if k_ + "_GBps" in row:  # butterflies/s x slots per butterfly / measured mad.lo rate
                        bfly = row[k_ + "_GBps"] * 1e9 / (2 * word) * log2_n / 2
                        row[k_ + "_alu_frac"] = bfly * slots_per_bfly / imad_peak
                rows.append(row)
                del polys
                torch.cuda.empty_cache()
            ctx.close()
    print(json.dumps({"metric": METRIC, "unit": "GB/s", "config": {"workload": "kernel-sweep", "prime_bits": args.sweep_bits},
                      "hbm_peak_GBps": peak, "peak_source": "of " + peak_kind,
                      "integer_peak_slots_per_s": imad_peak,
                      "integer_peak_source": "mad.lo.u32 rate measured in this run (d2mhe_debug_int_throughput); a "
                                             "butterfly counts %d slots" % (4 if args.sweep_bits <= 30 else SLOTS_PER_BUTTERFLY),
                      "dtype": "u32" if args.sweep_bits <= 30 else "u64", "data": "synthetic", "rows": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--config", type=int, default=4,
                    help="round configuration 1..4 (default 4: ResNet-18-shaped, the largest one); 5 = kernel sweep")
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--chunk", type=int, default=0, help="ciphertext indices per chunk (0: as many as fit)")
    ap.add_argument("--cts", type=int, default=0,
                    help="run only the first CTS ciphertext indices of the workload (a labelled slice, for profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the transform micro-benchmark and the conversion / refresh calls")
    ap.add_argument("--narrow", action="store_true",
                    help="run only the MNIST-shaped round on 30-bit limbs (32-bit-word calls) and print its line")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the short passes over the other round configurations")
    ap.add_argument("--sweep-bits", type=int, default=60, choices=[30, 50, 60])
    ap.add_argument("--sweep-point", default="", help="N,L,batch: run this one point of the sweep (any batch)")
    args = ap.parse_args()
    if args.config == 5:
        return run_sweep(args)
    if args.narrow:
        from paper_2207_04604_b200 import build

        build.build()
        line = narrow_round_bench(args, 0)
        line.update(metric=METRIC, unit=UNIT, dtype="u32", data="synthetic")
        return print(json.dumps(line))
    cfg = wl.round_config(args.config)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_cuda(args, cfg)


if __name__ == "__main__":
    main()
