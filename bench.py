#!/usr/bin/env python
"""Benchmark of the coded-gradient hot path on B200.

One step = one round of the whole path on one batch of synthetic partial gradients:
fused encode + quantise + pack of all n workers (kernel K1), then unpack + dequantise +
straggler-masked decode fused with the parameter update (kernel K2). Metric: gradient
coordinates per second through encode + quantise + decode.

  python bench.py --gpus N --steps K --warmup W [--workload cfg3] [--impl reference]

With N > 1 (launched by torch.distributed.run) every rank runs the same workload on its own
coordinate range (the path shards by coordinate with no exchange), so scaling is weak.
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

METRIC = "coded_gradient_coords_per_s_encode_quantize_decode"
UNIT = "coords/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the encode kernel, from the ncu
# capture summarised under profiles/ (bytes per coordinate of the captured case, scaled to d).
NCU_TRAFFIC_BYTES_PER_COORD = {"cfg3": 142.28}   # bucket-wise encoder, bucket 512
# smsp__inst_executed.sum per (worker, pack block) task of the encode kernel from the same capture:
# the kernel is bound by instruction issue, so the line also reports the issue rate it reaches
# against 4 schedulers x 148 SMs x the SM clock sampled during the run.
NCU_WARP_INST_PER_TASK = {"cfg3": 383.0}


def workload(name):
    from synth import configs as cfgs
    return {"cfg1": cfgs.config1, "cfg2": cfgs.config2, "cfg3": cfgs.config3, "cfg5": cfgs.config5}[name]()


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def k1_algorithmic_bytes(wl, bits, bucket):
    """Partitions read once + packed codes + scales written (per launch)."""
    nblk = (wl.d + 511) // 512
    if bucket == 0:   # global norm: the partial gradients are read twice, one scale per worker
        return 8 * wl.k * wl.d + int(sum(4 * 16 * int(b) * nblk for b in bits)) + 4 * wl.n
    nb = (wl.d + bucket - 1) // bucket
    passes = 2 if bucket > 512 else 1   # buckets of several pack blocks: two passes as well
    return 4 * passes * wl.k * wl.d + int(sum(4 * 16 * int(b) * nblk for b in bits)) + 4 * wl.n * nb


def k2_algorithmic_bytes(wl, bits, bucket, masks_all, p):
    """Average bytes per decode launch: messages and scales of the received workers (of the
    workers with a non-zero effective weight when R realisations are collapsed) read once,
    parameters read and written."""
    nblk = (wl.d + 511) // 512
    nb = (wl.d + bucket - 1) // bucket if bucket else 1
    m = masks_all.cpu().numpy().astype(bool)          # rounds x R x n
    used = m.any(axis=1)                              # rounds x n
    per_worker = np.array([64 * int(b) * nblk + 4 * nb for b in bits], np.float64)
    return float((used * per_worker[None, :]).sum(axis=1).mean()) + 8.0 * wl.d


def issue_rate(wl, bucket, k1_ms, clocks):
    """Second ceiling of the encode kernel: warp instructions issued per second against the
    issue capacity at the sampled SM clock (None where no instruction count was captured)."""
    ipt = NCU_WARP_INST_PER_TASK.get(wl.name) if bucket == 512 else None
    if ipt is None or not clocks or not clocks.get("sm_mhz"):
        return None
    tasks = wl.n * ((wl.d + 511) // 512)
    achieved = ipt * tasks / (k1_ms * 1e-3)
    peak = 148 * 4 * clocks["sm_mhz"] * 1e6
    return {"bound": "alu", "achieved": achieved / 1e9, "peak": peak / 1e9, "unit": "G warp-inst/s",
            "frac": achieved / peak, "warp_inst_per_task": ipt}


class ClockSampler:
    """nvidia-smi clocks and throttle reasons during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.lines, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.th.start()
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        self.th.join(timeout=5)
        sm, smax, power, reasons = [], [], [], set()
        for ln in self.lines:
            f = [t.strip() for t in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); smax.append(float(f[2]))
            except ValueError:
                continue
            try:
                power.append(float(f[3]))
            except ValueError:
                pass
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "samples": len(sm), "reasons": sorted(reasons), "power_w_max": max(power) if power else None}


def oracle_round(orp, code, bits, bucket, seed, t, G, d, mask, lr, beta):
    """One round of the oracle: encode + quantise + pack, then decode + update (returns beta)."""
    rp, ci, a, w = code
    if bucket > 512:
        c, s0, _, _ = orp.encode_quantize_grouped(rp, ci, a, bits, bucket, seed, t, G, d=d)
        s, B = orp.expand_grouped_scales(s0, d, bucket), 512
    elif bucket:
        c, s, _, _ = orp.encode_quantize(rp, ci, a, bits, bucket, seed, t, G, d=d)
        B = bucket
    else:
        c, s0, _, _ = orp.encode_quantize_global(rp, ci, a, bits, seed, t, G, d=d)
        s, B = orp.expand_global_scales(s0, d), 512
    _, beta = orp.decode(d, bits, B, w, mask, c, s, lr=lr, beta=beta, want_ghat=False)
    return beta


def parity_sample(ses, G, wl, code, bits, bucket, blocks=(0, 1, 2, 3)):
    """The messages the GPU produced for the bench's own inputs against the oracle on a few pack
    blocks (first ones and the last): counts of differing code words and scales (expected 0).
    Bucket-wise mode only (the global norm needs the whole vector)."""
    if not bucket or bucket > 512:
        return None
    from oracle import roundpath as orp
    rp, ci, a, w = code
    nblk = (wl.d + 511) // 512
    rnd = 12345
    ses.encode(G, rnd)
    off = orp.worker_word_offsets(wl.d, bits)
    bad_codes = bad_scales = 0
    qs = sorted({q for q in blocks if q < nblk} | {nblk - 1})
    for q in qs:
        m0, m1 = q * 512, min((q + 1) * 512, wl.d)
        blk = np.zeros((wl.k, 512), np.float32)
        blk[:, :m1 - m0] = G[:, m0:m1].cpu().numpy()
        oc, osc, _, _ = orp.encode_block(rp, ci, a, bits, bucket, wl.seed, rnd, q + ses.first_block, blk)
        wb = 0
        for i in range(wl.n):
            b = int(bits[i])
            lo = int(off[i]) + q * 16 * b
            got = ses.codes[lo:lo + 16 * b].cpu().numpy().view(np.uint32)
            bad_codes += int((got != oc[wb:wb + 16 * b]).sum())
            wb += 16 * b
        per = 512 // bucket
        nb = (wl.d + bucket - 1) // bucket
        got_s = ses.scales.view(wl.n, -1)[:, q * per:min((q + 1) * per, nb)].cpu().numpy()
        bad_scales += int((got_s.view(np.uint32) != osc[:, :got_s.shape[1]].view(np.uint32)).sum())
    return {"pack_blocks": qs, "code_words_differ": bad_codes, "scales_differ": bad_scales}


def oracle_sample_rate(wl, code, bits, bucket, target_s=12.0):
    """Time the CPU oracle (as it stands, one thread) on a bounded sample of the workload:
    whole pack blocks through encode + quantise + pack + decode + update."""
    from oracle import roundpath as orp
    from synth import configs as cfgs
    rp, ci, a, w = code
    blocks = 8
    d_s = blocks * 512
    G = cfgs.partials_numpy(wl, 0, d=d_s)
    mask = np.ones((1, wl.n), np.uint8)
    beta = np.zeros(d_s, np.float32)
    lr = np.array([1e-3], np.float32)

    def run(dd):
        t0 = time.perf_counter()
        oracle_round(orp, code, bits, bucket, wl.seed, 0, G[:, :dd], dd, mask, lr, beta[:dd])
        return time.perf_counter() - t0

    t_small = run(d_s)
    blocks = int(max(8, min(1 << 16, blocks * target_s / max(t_small, 1e-6))))
    d_s = blocks * 512
    G = cfgs.partials_numpy(wl, 0, d=d_s)
    beta = np.zeros(d_s, np.float32)
    t = run(d_s)
    return d_s / t, t, d_s


def build_code(agc, wl, bucket):
    """Bits (from the allocator where the workload says so) and code weights. With the global
    norm (bucket 0) the variance dimension of the design is kept at 512, so that the bucket-wise
    and the global-norm runs encode with the same bits and weights."""
    from synth import configs as cfgs
    phi_dim = float(bucket) if bucket else 512.0
    if wl.bits is None:
        bits, _ = agc.agc_bit_allocate(wl.p, wl.z_tot, b_min=2, b_max=wl.bits_range[1], phi_dim=phi_dim)
    else:
        bits = wl.bits
    sup = cfgs.cyclic_support(wl)
    srp = np.arange(0, wl.n * wl.s + 1, wl.s, dtype=np.int32)
    sci = np.array(sum(sup, []), np.int32)
    rp, ci, a, w, _ = agc.agc_code_build(wl.n, wl.k, wl.p, bits, phi_dim, mode=agc.AGC_CODE_SUPPORT,
                                         sup_row_ptr=srp, sup_col_idx=sci)
    return (rp, ci, a, w), np.asarray(bits, np.uint8)


def oracle_build_code(wl, bucket):
    """Bits and code weights of the workload from the oracle's own design code (float64 numpy /
    scipy): Algorithm 1 for the bits, the support-restricted problem (c-SP2) for the weights.
    Used by the reference arm, which must not touch the CUDA library."""
    from oracle import design as od
    phi_dim = float(bucket) if bucket else 512.0
    if wl.bits is None:
        bits, _ = od.bit_allocate_low_complexity(wl.p, wl.z_tot, phi_dim, b_max=wl.bits_range[1])
    else:
        bits = wl.bits
    bits = np.asarray(bits, np.uint8)
    support = od.cyclic_support(wl.n, wl.k, wl.s)
    c = od.c_coeff(wl.p, bits, phi_dim)
    alpha, _ = od.support_restricted_alpha_reference(c, support, wl.k)
    rp, ci, vals = od.alpha_to_csr(alpha, drop=1e-9)
    _, w = od.physical_coefficients(alpha, wl.p)
    return (rp, ci, vals.astype(np.float32), w.astype(np.float32)), bits


def run_reference(args, wl, bucket):
    """Reference arm: the CPU oracle as it stands, on host cores, each step a bounded sample.
    Nothing of the CUDA library is imported here: bits and weights come from oracle/design.py."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import roundpath as orp
    from synth import configs as cfgs
    code, bits = oracle_build_code(wl, bucket)
    rp, ci, a, w = code
    rate0, _, _ = oracle_sample_rate(wl, code, bits, bucket, target_s=2.0)
    # the whole run (warm-up + timed steps) is sized to about two minutes of host time
    per_step_s = min(4.0, 120.0 / max(1, args.steps + args.warmup))
    blocks = int(max(8, min(1 << 15, rate0 * per_step_s / 512)))
    d_s = blocks * 512
    G = cfgs.partials_numpy(wl, 0, d=d_s)
    masks = cfgs.straggler_masks(wl, rounds=min(args.steps + args.warmup, 64), realizations=1)
    beta = np.zeros(d_s, np.float32)
    lr = np.array([1e-3], np.float32)
    times = []
    for t in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        beta = oracle_round(orp, code, bits, bucket, wl.seed, t, G, d_s, masks[t % len(masks)], lr, beta)
        if t >= args.warmup:
            times.append(time.perf_counter() - t0)
    tot = sum(times)
    value = d_s * args.steps / tot
    sample = f"{blocks} pack blocks ({d_s} of {wl.d} coordinates, all {wl.n} workers) per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot / args.steps * (wl.d / d_s),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": workload_config(wl, bits, bucket, "n/a (CPU)"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def workload_config(wl, bits, bucket, l2_note):
    return {"workload": f"{wl.name}: n={wl.n} workers, k={wl.k} partitions, cyclic s={wl.s}, d={wl.d}, "
                        f"{wl.value_model} values, bucket={bucket}",
            "bits": [int(b) for b in bits], "bits_per_coord_total": int(np.sum(bits)),
            "realizations_per_encode": wl.realizations, "l2": l2_note}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg1", "cfg2", "cfg3", "cfg5"])
    ap.add_argument("--bucket", type=int, default=512, help="128, 256, 512 (one pass), 1024, 2048, 4096 or 0 = one norm per worker (two-pass encode)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-two-track", action="store_true")
    ap.add_argument("--d", type=int, default=0, help="override the number of coordinates (profiling on a small case)")
    args = ap.parse_args()
    wl = workload(args.workload)
    if args.d:
        wl.d = args.d
        wl.name += f"@d={args.d}"
    bucket = args.bucket
    if args.impl == "reference":
        run_reference(args, wl, bucket)
        return

    import torch
    import paper_2605_15890_b200 as agc
    from paper_2605_15890_b200 import sharding
    from paper_2605_15890_b200.session import Session
    from synth import configs as cfgs

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    dev = f"cuda:{local_rank}"
    torch.cuda.set_device(dev)

    code, bits = build_code(agc, wl, bucket)
    rp, ci, a, w = code
    flags = agc.AGC_FLAG_ALLOW_1BIT if int(bits.min()) == 1 else 0
    # weak scaling: the job is a gradient of world * nblk pack blocks, rank r holds blocks
    # [r * nblk, (r + 1) * nblk) of it (its own data, same shape), no exchange on the data path
    ses = Session(wl.n, wl.k, wl.d, rp, ci, a, w, wl.p, bits, bucket=bucket, seed=wl.seed, flags=flags, device=dev)
    align = max(512, bucket)                                  # a rank's range starts at a bucket
    per_rank = (wl.d + align - 1) // align * align
    ses.set_first_block(sharding.first_block(world * per_rank, rank, world, align=align))
    wl.seed += 7919 * rank  # the synthetic values of this rank's range
    ld = (wl.d + 3) // 4 * 4
    G = cfgs.partials_torch(wl, dev, ld=ld)
    R = wl.realizations
    total = args.warmup + args.steps
    n_masks = min(total, 64)
    masks_all = torch.from_numpy(cfgs.straggler_masks(wl, rounds=n_masks, realizations=R)).to(dev)
    beta = torch.zeros(wl.d, dtype=torch.float32, device=dev)
    lr = np.full(R, 1e-3, np.float32)
    in_bytes = 4 * wl.k * wl.d
    l2_note = ("inputs (%.2f GB) larger than the 126 MB L2; no flush" % (in_bytes / 1e9)) if in_bytes > 4 * 126e6 \
        else "L2 flushed between steps by writing a 512 MB buffer"
    flush = None if in_bytes > 4 * 126e6 else torch.empty(512 << 20, dtype=torch.uint8, device=dev)

    def step(t, ev=None):
        if flush is not None:
            flush.fill_(t & 0xFF)
        if ev:
            ev[0].record()
        ses.encode(G, t)
        if ev:
            ev[1].record()
        ses.decode(masks_all[t % n_masks], lr=lr, beta=beta)
        if ev:
            ev[2].record()

    for t in range(args.warmup):
        step(t)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    torch.cuda.synchronize()
    for t in range(args.steps):
        step(args.warmup + t, evs[t])
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    if dist:
        dist.barrier()
    k1_ms = sum(e[0].elapsed_time(e[1]) for e in evs) / args.steps
    k2_ms = sum(e[1].elapsed_time(e[2]) for e in evs) / args.steps
    step_ms = k1_ms + k2_ms if flush is not None else evs[0][0].elapsed_time(evs[-1][2]) / args.steps
    status = int(ses.status.item())
    step_ms, k1_ms, k2_ms = sharding.max_over_ranks([step_ms, k1_ms, k2_ms], device=dev)
    value = world * wl.d / (step_ms * 1e-3)

    # the two-track decode + Adam step (Sec. V-E) on the same messages: timed apart, not part of the step
    tt_ms = None
    if R == 1 and not args.no_two_track:
        v2 = agc.agc_two_track_vector(wl.n, wl.k, wl.p, bits, float(bucket) if bucket else 512.0, rp, a)
        m_t = torch.zeros(wl.d, dtype=torch.float32, device=dev)
        u_t = torch.zeros(wl.d, dtype=torch.float32, device=dev)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = 30
        for it in range(reps + 3):
            if it == 3:
                e0.record()
            agc.agc_decode_two_track(ses.plan, ses.codes, ses.scales, masks_all[it % n_masks, 0], v2, None, None,
                                     beta, m_t, u_t, adam=(1e-3, 0.9, 0.999, 1e-8, it + 1), status_dev=ses.status)
        e1.record()
        torch.cuda.synchronize()
        tt_ms = sharding.max_over_ranks([e0.elapsed_time(e1) / reps], device=dev)[0]
        del m_t, u_t

    # end to end through the host-buffer entry point (pinned host memory, copies timed)
    e2e = None
    if not args.no_e2e and in_bytes > 16e9:
        e2e = {"value": None, "unit": UNIT, "skipped": "host staging of %.0f GB of partial gradients not attempted" % (in_bytes / 1e9)}
    elif not args.no_e2e:
        Gh = torch.empty((wl.k, wl.d), dtype=torch.float32).pin_memory()
        Gh.copy_(G[:, :wl.d])
        mh = masks_all[0, 0].cpu().pin_memory()
        gh = torch.empty(wl.d, dtype=torch.float32).pin_memory()
        agc.agc_round_host(ses.plan, Gh, wl.d, 0, mh, gh)
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        t0 = time.perf_counter()
        for t in range(args.e2e_steps):
            agc.agc_round_host(ses.plan, Gh, wl.d, t + 1, mh, gh)
        e2e_s = (time.perf_counter() - t0) / args.e2e_steps
        e2e_s = sharding.max_over_ranks([e2e_s], device=dev)[0]
        e2e = {"value": world * wl.d / e2e_s, "unit": UNIT, "h2d_bytes_per_step": 4 * wl.k * wl.d + wl.n,
               "d2h_bytes_per_step": 4 * wl.d + 4, "ms_per_step": 1e3 * e2e_s, "steps": args.e2e_steps}
        del Gh, gh

    if rank == 0:
        peak, which = measured_hbm_peak()
        k1_bytes = k1_algorithmic_bytes(wl, bits, bucket)
        achieved = k1_bytes / (k1_ms * 1e-3) / 1e9
        tpc = NCU_TRAFFIC_BYTES_PER_COORD.get(wl.name) if bucket == 512 else None
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": workload_config(wl, bits, bucket, l2_note),
                "kernels": {"encode_quantize_ms": k1_ms, "decode_update_ms": k2_ms, "staged_tma": bool(ses.uses_tma),
                            "status_bits": status, "two_track_adam_ms": tt_ms,
                            "decode_GBs": k2_algorithmic_bytes(wl, bits, bucket, masks_all, wl.p) / (k2_ms * 1e-3) / 1e9,
                            "encode_GBs": achieved,
                            "encode_coords_per_s": wl.d / (k1_ms * 1e-3), "decode_coords_per_s": wl.d / (k2_ms * 1e-3),
                            "worker_coords_per_s": world * wl.n * wl.d / (step_ms * 1e-3)},
                "roofline": {"bound": "hbm", "kernel": "agc_encode_staged_kernel" if ses.uses_tma else "agc_encode_direct_kernel",
                             "achieved": achieved, "peak": peak, "peak_source": f"of {which}", "unit": "GB/s",
                             "frac": achieved / peak, "frac_of_8000": achieved / 8000.0,
                             "algorithmic_bytes": k1_bytes,
                             "traffic": None if tpc is None else tpc * wl.d,
                             "issue": issue_rate(wl, bucket, k1_ms, clocks)},
                "clocks": clocks, "e2e": e2e,
                # encode (global norm: first pass, two reduction kernels, second pass; buckets of several
                # pack blocks: first pass, one reduction kernel, second pass), decode, and the
                # effective-weights kernel of a multi-realisation update
                "gpu_launches": args.steps * ((4 if bucket == 0 else 3 if bucket > 512 else 1) + 1 + (1 if R > 1 else 0))}
        if not args.no_cpu_baseline:
            rate, secs, d_s = oracle_sample_rate(wl, code, bits, bucket)
            line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle",
                                    "sample": f"{d_s} of {wl.d} coordinates (whole pack blocks, all {wl.n} workers), "
                                              f"one round, {secs:.1f} s"}
            line["parity_sample"] = parity_sample(ses, G, wl, code, bits, bucket)
        print(json.dumps(line))
    ses.close()
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
