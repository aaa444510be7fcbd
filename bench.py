#!/usr/bin/env python
"""Benchmark of the coded-gradient hot path on B200.

One step = one round of the whole path on one batch of synthetic partial gradients:
fused encode + quantise + pack of all n workers (kernel K1), then unpack + dequantise +
straggler-masked decode fused with the parameter update (kernel K2). Metric: gradient
coordinates per second through encode + quantise + decode.

  python bench.py --gpus N --steps K --warmup W [--workload cfg3] [--code cyclic] [--impl reference]
  python bench.py --study allocators          (the allocator comparison of Sec. VI, host only)

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
# From the ncu captures summarised under profiles/ (per coordinate of the captured case, scaled
# to d; valid for the cyclic cfg3 code with bucket 512 only, and only while the kernel is the
# captured one):
#   dram__bytes_read.sum + dram__bytes_write.sum per launch of the encode kernel
NCU_TRAFFIC_BYTES_PER_COORD = {"cfg3": 143.82}   # captured at d = 16,777,216 (messages larger than L2)
#   smsp__inst_executed.sum per (worker, pack block) task of the encode kernel
NCU_WARP_INST_PER_TASK = {"cfg3": 307.4}


def workload(name):
    from synth import configs as cfgs
    return {"cfg1": cfgs.config1, "cfg2": cfgs.config2, "cfg3": cfgs.config3, "cfg4": cfgs.config4,
            "cfg5": cfgs.config5}[name]()


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


def k2_algorithmic_bytes(wl, bits, bucket, masks_all):
    """Average bytes per decode launch: messages and scales of the received workers (of the
    workers with a non-zero effective weight when R realisations are collapsed) read once,
    parameters read and written."""
    nblk = (wl.d + 511) // 512
    nb = (wl.d + bucket - 1) // bucket if bucket else 1
    m = masks_all.cpu().numpy().astype(bool)          # rounds x R x n
    used = m.any(axis=1)                              # rounds x n
    per_worker = np.array([64 * int(b) * nblk + 4 * nb for b in bits], np.float64)
    return float((used * per_worker[None, :]).sum(axis=1).mean()) + 8.0 * wl.d


def issue_rate(wl, bucket, code_kind, k1_ms, clocks):
    """Second ceiling of the encode kernel: warp instructions issued per second against the
    issue capacity at the sampled SM clock (None where no instruction count was captured)."""
    ipt = NCU_WARP_INST_PER_TASK.get(wl.name) if bucket == 512 and code_kind == "cyclic" else None
    if ipt is None or not clocks or not clocks.get("sm_mhz"):
        return None
    tasks = wl.n * ((wl.d + 511) // 512)
    achieved = ipt * tasks / (k1_ms * 1e-3)
    peak = 148 * 4 * clocks["sm_mhz"] * 1e6
    return {"bound": "alu", "achieved": achieved / 1e9, "peak": peak / 1e9, "unit": "G warp-inst/s",
            "frac": achieved / peak, "warp_inst_per_task": ipt}


class ClockSampler:
    """SM clock, power and throttle reasons during a timed region: NVML polled from a thread about
    every millisecond (the timed steps of the default run last some tens of milliseconds), or, where
    NVML cannot be loaded, nvidia-smi every 50 ms."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    REASONS = ((0x8, "hw_slowdown"), (0x40, "hw_thermal_slowdown"), (0x20, "sw_thermal_slowdown"), (0x4, "sw_power_cap"))

    def __init__(self, index):
        self.index, self.lines, self.proc = index, [], None
        self.nvml, self.handle, self.samples, self.stop_flag, self.th = None, None, [], False, None

    def _nvml_handle(self):
        import pynvml
        pynvml.nvmlInit()
        handle = None
        try:   # the CUDA device's own UUID: CUDA_VISIBLE_DEVICES may renumber the devices
            import torch
            uuid = str(torch.cuda.get_device_properties(self.index).uuid)
            handle = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid).encode())
        except Exception:
            handle = None
        if handle is None:
            handle = pynvml.nvmlDeviceGetHandleByIndex(self.index)
        return pynvml, handle

    def _poll(self):
        nv, h = self.nvml, self.handle
        reasons_fn = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
            getattr(nv, "nvmlDeviceGetCurrentClocksThrottleReasons")
        while not self.stop_flag:
            try:
                self.samples.append((float(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)),
                                     nv.nvmlDeviceGetPowerUsage(h) / 1000.0, int(reasons_fn(h))))
            except Exception:
                break
            time.sleep(0.001)

    def start(self):
        try:
            self.nvml, self.handle = self._nvml_handle()
            self.smax = float(self.nvml.nvmlDeviceGetMaxClockInfo(self.handle, self.nvml.NVML_CLOCK_SM))
            self.stop_flag = False
            self.th = threading.Thread(target=self._poll, daemon=True)
            self.th.start()
            return
        except Exception:
            self.nvml = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=lambda: self.lines.extend(self.proc.stdout), daemon=True)
            self.th.start()
        except OSError:
            self.proc = None

    def stop(self):
        if self.nvml is not None:
            self.stop_flag = True
            self.th.join(timeout=5)
            if self.samples:
                sm = [x[0] for x in self.samples]
                mask = 0
                for x in self.samples:
                    mask |= x[2]
                return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": self.smax, "samples": len(sm),
                        "reasons": sorted(name for bit, name in self.REASONS if mask & bit),
                        "power_w_max": max(x[1] for x in self.samples), "source": "nvml"}
        if self.proc is None and self.nvml is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass
            self.th.join(timeout=5)
        if not self.lines:
            # a region shorter than the sampling period: one reading taken right after it
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-i",
                                      str(self.index)], capture_output=True, text=True, timeout=10).stdout
                self.lines = [ln for ln in out.splitlines() if ln.strip()]
            except (OSError, subprocess.SubprocessError):
                pass
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
                "samples": len(sm), "reasons": sorted(reasons), "power_w_max": max(power) if power else None,
                "source": "nvidia-smi"}


# ------------------------------------------------------------------ oracle legs (CPU)
def oracle_encode(orp, code, bits, bucket, seed, t, G, d):
    rp, ci, a, w = code
    if bucket > 512:
        c, s0, _, _ = orp.encode_quantize_grouped(rp, ci, a, bits, bucket, seed, t, G, d=d)
        return c, orp.expand_grouped_scales(s0, d, bucket), 512
    if bucket:
        c, s, _, _ = orp.encode_quantize(rp, ci, a, bits, bucket, seed, t, G, d=d)
        return c, s, bucket
    c, s0, _, _ = orp.encode_quantize_global(rp, ci, a, bits, seed, t, G, d=d)
    return c, orp.expand_global_scales(s0, d), 512


def oracle_round(orp, code, bits, bucket, seed, t, G, d, mask, lr, beta, times=None):
    """One round of the oracle: encode + quantise + pack, then decode + update (returns beta)."""
    t0 = time.perf_counter()
    c, s, B = oracle_encode(orp, code, bits, bucket, seed, t, G, d)
    t1 = time.perf_counter()
    _, beta = orp.decode(d, bits, B, code[3], mask, c, s, lr=lr, beta=beta, want_ghat=False)
    if times is not None:
        times.append((t1 - t0, time.perf_counter() - t1))
    return beta


def parity_blocks(wl, nblk, count=64):
    """Pack blocks for the bench's own parity sample: first and last ones, the blocks that hold a
    segment boundary of the synthetic gradient (cfg3), seeded random ones."""
    from synth import configs as cfgs
    pick = {0, 1, 2, 3, nblk - 2, nblk - 1}
    if wl.value_model == "segments":
        starts, _, _ = cfgs.segment_table(wl)
        pick |= {int(s) // 512 for s in starts[1:25]}
    pick = {q for q in pick if 0 <= q < nblk}
    rng = np.random.default_rng(12345)
    while len(pick) < min(count, nblk):
        pick.add(int(rng.integers(0, nblk)))
    return sorted(pick)


def parity_sample(ses, G, wl, code, bits, bucket):
    """The messages the GPU produced for the bench's own inputs against the oracle on sampled
    pack blocks: counts of differing code words and scales (expected 0). Bucket-wise mode only
    (the global norm needs the whole vector)."""
    if not bucket or bucket > 512:
        return None
    from oracle import roundpath as orp
    rp, ci, a, w = code
    nblk = (wl.d + 511) // 512
    rnd = 12345
    ses.encode(G, rnd)
    off = orp.worker_word_offsets(wl.d, bits)
    bad_codes = bad_scales = 0
    qs = parity_blocks(wl, nblk)
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
    return {"pack_blocks": len(qs), "first_blocks": qs[:6], "last_block": qs[-1], "code_words_differ": bad_codes,
            "scales_differ": bad_scales}


def sample_size(wl, blocks):
    """Coordinates of a sample of `blocks` whole pack blocks (the whole vector if it is shorter)."""
    return wl.d if blocks * 512 >= wl.d else blocks * 512


def oracle_sample_rate(wl, code, bits, bucket, target_s=12.0, full_s=0.0):
    """Time the CPU oracle (as it stands, one thread) on a bounded sample of the workload: whole
    pack blocks through encode + quantise + pack, then decode + update, the two legs timed apart.
    The sample is the whole vector if that is estimated to take at most full_s seconds, else about
    target_s seconds' worth of pack blocks."""
    from oracle import roundpath as orp
    from synth import configs as cfgs
    mask = np.ones((1, wl.n), np.uint8)
    lr = np.array([1e-3], np.float32)

    def run(dd, times=None):
        G = cfgs.partials_numpy(wl, 0, d=dd)
        t0 = time.perf_counter()
        oracle_round(orp, code, bits, bucket, wl.seed, 0, G, dd, mask, lr, np.zeros(dd, np.float32), times)
        return time.perf_counter() - t0

    blocks = 8
    t_small = run(sample_size(wl, blocks))
    per_block = max(t_small, 1e-6) / blocks
    nblk = (wl.d + 511) // 512
    if full_s and per_block * nblk <= full_s:
        blocks = nblk                      # the whole vector where that stays within the time allowed
    else:
        blocks = int(max(8, min(1 << 16, target_s / per_block)))
    d_s = sample_size(wl, blocks)
    legs = []
    t = run(d_s, legs)
    return {"rate": d_s / t, "seconds": t, "d": d_s, "encode_rate": d_s / legs[0][0], "decode_rate": d_s / legs[0][1]}


# ------------------------------------------------------------------ code builders
def workload_support(wl, code_kind):
    """Column lists of the assignment: the cyclic-s support of the configurations, or a seeded
    scattered one (every worker holds s partitions drawn at random; every partition is held)."""
    from synth import configs as cfgs
    if code_kind == "cyclic":
        return cfgs.cyclic_support(wl)
    rng = np.random.default_rng(np.random.SeedSequence([int(wl.seed), 31]))
    sup = [sorted(int(j) for j in rng.choice(wl.k, size=wl.s, replace=False)) for _ in range(wl.n)]
    for j in range(wl.k):          # a partition nobody drew goes to a worker in place of one held elsewhere too
        if any(j in cols for cols in sup):
            continue
        count = {c: sum(c in cols for cols in sup) for c in range(wl.k)}
        for i in rng.permutation(wl.n):
            spare = [c for c in sup[i] if count[c] > 1]
            if spare:
                sup[i] = sorted((set(sup[i]) - {spare[0]}) | {j})
                break
    return sup


def build_code(agc, wl, bucket, code_kind="cyclic"):
    """Bits (from the allocator where the workload says so) and code weights from the library's
    design calls. With the global norm (bucket 0) the variance dimension of the design is kept at
    512, so that the bucket-wise and the global-norm runs encode with the same bits and weights.
    code_kind: 'cyclic' = the paper's objective on the cyclic-s support of the configuration,
    'scattered' = the same on a seeded scattered support, 'interval' = the paper's own
    construction of Sec. III-A (its support follows from the row sums of Theorem 1)."""
    phi_dim = float(bucket) if bucket else 512.0
    if wl.bits is None:
        bits, _ = agc.agc_bit_allocate(wl.p, wl.z_tot, b_min=2, b_max=wl.bits_range[1], phi_dim=phi_dim)
    else:
        bits = wl.bits
    if code_kind == "interval":
        rp, ci, a, w, _ = agc.agc_code_build(wl.n, wl.k, wl.p, bits, phi_dim, mode=agc.AGC_CODE_INTERVAL)
    else:
        sup = workload_support(wl, code_kind)
        srp = np.zeros(wl.n + 1, np.int32)
        srp[1:] = np.cumsum([len(c) for c in sup])
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


def workload_config(wl, bits, bucket, l2_note, code=None, code_kind="cyclic"):
    cfg = {"workload": f"{wl.name}: n={wl.n} workers, k={wl.k} partitions, {code_kind} code"
                       f"{'' if code_kind == 'interval' else f' s={wl.s}'}, d={wl.d}, {wl.value_model} values, "
                       f"bucket={bucket}",
           "bits": [int(b) for b in bits], "bits_per_coord_total": int(np.sum(bits)),
           "realizations_per_encode": wl.realizations, "l2": l2_note}
    if code is not None:
        nnz = int(len(code[1]))
        cfg["nnz"] = nnz                       # non-zero coefficients of A after the design (zeros dropped)
        cfg["coefficients_per_worker"] = round(nnz / wl.n, 3)
    return cfg


def run_reference(args, wl, bucket):
    """Reference arm: the CPU oracle as it stands, on host cores, each step a bounded sample.
    Nothing of the CUDA library is imported here: bits and weights come from oracle/design.py."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import roundpath as orp
    from synth import configs as cfgs
    code, bits = oracle_build_code(wl, bucket)
    r0 = oracle_sample_rate(wl, code, bits, bucket, target_s=2.0)
    # the whole run (warm-up + timed steps) is sized to about two minutes of host time
    per_step_s = min(4.0, 120.0 / max(1, args.steps + args.warmup))
    blocks = int(max(8, min(1 << 15, r0["rate"] * per_step_s / 512)))
    d_s = sample_size(wl, blocks)
    G = cfgs.partials_numpy(wl, 0, d=d_s)
    masks = cfgs.straggler_masks(wl, rounds=min(args.steps + args.warmup, 64), realizations=1)
    beta = np.zeros(d_s, np.float32)
    lr = np.array([1e-3], np.float32)
    times, legs = [], []
    for t in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        beta = oracle_round(orp, code, bits, bucket, wl.seed, t, G, d_s, masks[t % len(masks)], lr, beta,
                            legs if t >= args.warmup else None)
        if t >= args.warmup:
            times.append(time.perf_counter() - t0)
    tot = sum(times)
    value = d_s * args.steps / tot
    sample = f"{(d_s + 511) // 512} pack blocks ({d_s} of {wl.d} coordinates, all {wl.n} workers) per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot / args.steps * (wl.d / d_s),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
            "data": "synthetic", "config": workload_config(wl, bits, bucket, "n/a (CPU)", code),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "host_cores": os.cpu_count(), "kind": "oracle",
                             "sample": sample,
                             "encode": {"value": d_s * args.steps / sum(x[0] for x in legs), "unit": UNIT},
                             "decode": {"value": d_s * args.steps / sum(x[1] for x in legs), "unit": UNIT}},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def sustained(launch, est_ms, seconds, local_rank, torch):
    """A kernel launched back to back for about `seconds`: mean time per launch with the SM clock
    sampled over that interval (under the power cap the clock settles below its burst value)."""
    reps = int(max(50, min(200000, seconds * 1e3 / max(est_ms, 1e-3))))
    sampler = ClockSampler(local_rank)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    sampler.start()
    e0.record()
    for t in range(reps):
        launch(t)
    e1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / reps
    return ms, reps, clocks


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3", choices=["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"])
    ap.add_argument("--code", default="cyclic", choices=["cyclic", "interval", "scattered"],
                    help="code structure: the configuration's cyclic support, the paper's interval construction, or a seeded scattered support")
    ap.add_argument("--bucket", type=int, default=512, help="128, 256, 512 (one pass), 1024, 2048, 4096 or 0 = one norm per worker (two-pass encode)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--sustain-s", type=float, default=1.2, help="seconds of back-to-back launches per kernel for the sustained figures (0 = off)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-two-track", action="store_true")
    ap.add_argument("--d", type=int, default=0, help="override the number of coordinates (profiling on a small case)")
    ap.add_argument("--study", default=None, choices=["allocators"], help="print the allocator comparison of Sec. VI and exit (host only)")
    args = ap.parse_args()
    if args.study:
        from paper_2605_15890_b200 import allocator_study
        sys.argv = [sys.argv[0], "--markdown"]
        allocator_study.main()
        return
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
    if world > 1 and bucket == 0:
        # every rank of this bench holds its own vector's range; one norm per worker over the whole
        # vector needs the exchange of the split encoder (agc_encode_norm_sums / _with_norms),
        # which this step does not time
        if rank == 0:
            print("bench.py: --bucket 0 (one norm over the whole vector) is timed on one GPU only", file=sys.stderr)
        sys.exit(2)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    dev = f"cuda:{local_rank}"
    torch.cuda.set_device(dev)

    code, bits = build_code(agc, wl, bucket, args.code)
    rp, ci, a, w = code
    flags = agc.AGC_FLAG_ALLOW_1BIT if int(bits.min()) == 1 else 0
    # weak scaling: the job is a gradient of world * nblk pack blocks, rank r holds blocks
    # [r * nblk, (r + 1) * nblk) of it (its own data, same shape), no exchange on the data path
    ses = Session(wl.n, wl.k, wl.d, rp, ci, a, w, wl.p, bits, bucket=bucket, seed=wl.seed, flags=flags, device=dev)
    align = max(512, bucket)                                  # a rank's range starts at a bucket
    per_rank = (wl.d + align - 1) // align * align
    if world > 1:
        ses.set_first_block(sharding.first_block(world * per_rank, rank, world, align=align))
    layout = agc.agc_plan_encode_layout(ses.plan)
    wl.seed += 7919 * rank  # the synthetic values of this rank's range
    ld = (wl.d + 3) // 4 * 4
    R = wl.realizations
    total = args.warmup + args.steps
    n_masks = min(total, 64)
    masks_all = torch.from_numpy(cfgs.straggler_masks(wl, rounds=n_masks, realizations=R)).to(dev)
    beta = torch.zeros(wl.d, dtype=torch.float32, device=dev)
    lr = np.full(R, 1e-3, np.float32)
    in_bytes = 4 * wl.k * wl.d
    graph_mode = wl.name.startswith("cfg4")
    if graph_mode:
        # launch-latency regime: the rounds are recorded in one CUDA graph and replayed; the
        # partial gradients of a round are those of the least-squares problem at w = 0 (a reduced
        # number of rows: the timed path depends on their shape only), in rotating buffers whose
        # total exceeds L2
        n_buf = max(2, int(1.3 * 126e6 / in_bytes) + 1)
        X, y, _ = cfgs.least_squares_problem(wl, dev, rows=wl.k * 256)
        rows_per = X.shape[0] // wl.k
        G0 = torch.stack([-(X[j * rows_per:(j + 1) * rows_per].T @ y[j * rows_per:(j + 1) * rows_per])
                          for j in range(wl.k)])
        del X, y
        Gs = [(G0 * (1.0 + 0.01 * t)).contiguous() for t in range(n_buf)]
        G = Gs[0]
        l2_note = f"{n_buf} rotating input buffers ({n_buf * in_bytes / 1e6:.0f} MB in all, more than the 126 MB L2); no flush"
        flush = None
    else:
        G = cfgs.partials_torch(wl, dev, ld=ld)
        Gs = [G]
        l2_note = ("inputs (%.2f GB) larger than the 126 MB L2; no flush" % (in_bytes / 1e9)) if in_bytes > 4 * 126e6 \
            else "L2 flushed between steps by writing a 512 MB buffer"
        flush = None if in_bytes > 4 * 126e6 else torch.empty(512 << 20, dtype=torch.uint8, device=dev)

    def step(t, ev=None):
        if flush is not None:
            flush.fill_(t & 0xFF)
        if ev:
            ev[0].record()
        ses.encode(Gs[t % len(Gs)], t)
        if ev:
            ev[1].record()
        ses.decode(masks_all[t % n_masks], lr=lr, beta=beta)
        if ev:
            ev[2].record()

    for t in range(args.warmup):
        step(t)
    torch.cuda.synchronize()
    graph = None
    if graph_mode:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for t in range(args.steps):
                step(args.warmup + t)
        graph.replay()                 # one untimed replay
        torch.cuda.synchronize()
    if dist:
        dist.barrier()
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    torch.cuda.synchronize()
    if graph is not None:
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record()
        graph.replay()
        g1.record()
        torch.cuda.synchronize()
        step_ms = g0.elapsed_time(g1) / args.steps
    else:
        for t in range(args.steps):
            step(args.warmup + t, evs[t])
        torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    if dist:
        dist.barrier()
    if graph is not None:
        # per-kernel times from a second, eager pass (events cannot be read out of a replay)
        for t in range(args.steps):
            step(args.warmup + t, evs[t])
        torch.cuda.synchronize()
    k1_ms = sum(e[0].elapsed_time(e[1]) for e in evs) / args.steps
    k2_ms = sum(e[1].elapsed_time(e[2]) for e in evs) / args.steps
    if graph is None:
        step_ms = k1_ms + k2_ms if flush is not None else evs[0][0].elapsed_time(evs[-1][2]) / args.steps
    status = int(ses.status.item())
    step_ms, k1_ms, k2_ms = sharding.max_over_ranks([step_ms, k1_ms, k2_ms], device=dev)
    value = world * wl.d / (step_ms * 1e-3)

    # sustained figures: each kernel alone, back to back for about a second, its own clock samples
    sus = None
    if args.sustain_s > 0 and not graph_mode and flush is None:
        k1s_ms, k1_reps, k1_clk = sustained(lambda t: ses.encode(G, t), k1_ms, args.sustain_s, local_rank, torch)
        k2s_ms, k2_reps, k2_clk = sustained(lambda t: ses.decode(masks_all[t % n_masks], lr=lr, beta=beta), k2_ms,
                                            args.sustain_s, local_rank, torch)
        k1s_ms, k2s_ms = sharding.max_over_ranks([k1s_ms, k2s_ms], device=dev)
        sus = {"k1_ms": k1s_ms, "k1_launches": k1_reps, "k1_clocks": k1_clk, "k2_ms": k2s_ms, "k2_launches": k2_reps,
               "k2_clocks": k2_clk}

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
        k2_bytes = k2_algorithmic_bytes(wl, bits, bucket, masks_all)
        achieved = k1_bytes / (k1_ms * 1e-3) / 1e9
        achieved2 = k2_bytes / (k2_ms * 1e-3) / 1e9
        plain = bucket == 512 and args.code == "cyclic"
        tpc = NCU_TRAFFIC_BYTES_PER_COORD.get(wl.name) if plain else None
        mhz = clocks.get("sm_mhz") if clocks else None
        roof = {"bound": "hbm", "kernel": "agc_encode_staged_kernel" if ses.uses_tma else "agc_encode_direct_kernel",
                "achieved": achieved, "peak": peak, "peak_source": f"of {which}", "unit": "GB/s",
                "frac": achieved / peak, "frac_of_8000": achieved / 8000.0, "algorithmic_bytes": k1_bytes,
                "traffic": None if tpc is None else tpc * wl.d,
                "time_x_mhz": None if not mhz else k1_ms * mhz,
                "issue": issue_rate(wl, bucket, args.code, k1_ms, clocks)}
        roof2 = {"bound": "hbm", "kernel": "agc_decode_ring_kernel", "achieved": achieved2, "peak": peak,
                 "peak_source": f"of {which}", "unit": "GB/s", "frac": achieved2 / peak, "algorithmic_bytes": k2_bytes,
                 "time_x_mhz": None if not mhz else k2_ms * mhz, "traffic": None}
        if sus:
            a1 = k1_bytes / (sus["k1_ms"] * 1e-3) / 1e9
            a2 = k2_bytes / (sus["k2_ms"] * 1e-3) / 1e9
            c1, c2 = sus["k1_clocks"], sus["k2_clocks"]
            roof["sustained"] = {"ms": sus["k1_ms"], "launches": sus["k1_launches"], "achieved": a1, "frac": a1 / peak,
                                 "frac_of_8000": a1 / 8000.0, "clocks": c1,
                                 "time_x_mhz": None if not c1.get("sm_mhz") else sus["k1_ms"] * c1["sm_mhz"]}
            roof2["sustained"] = {"ms": sus["k2_ms"], "launches": sus["k2_launches"], "achieved": a2, "frac": a2 / peak,
                                  "clocks": c2,
                                  "time_x_mhz": None if not c2.get("sm_mhz") else sus["k2_ms"] * c2["sm_mhz"]}
        cfg = workload_config(wl, bits, bucket, l2_note, code, args.code)
        cfg["encoder_layout"] = dict(layout, restaging_factor=round(layout["rows_staged"] / wl.k, 3) if layout["staged"] else None)
        if graph_mode:
            cfg["launch"] = f"{args.steps} rounds recorded in one CUDA graph, one replay timed"
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": cfg,
                "kernels": {"encode_quantize_ms": k1_ms, "decode_update_ms": k2_ms, "staged_tma": bool(ses.uses_tma),
                            "status_bits": status, "two_track_adam_ms": tt_ms,
                            "decode_GBs": achieved2, "encode_GBs": achieved,
                            "encode_coords_per_s": wl.d / (k1_ms * 1e-3), "decode_coords_per_s": wl.d / (k2_ms * 1e-3),
                            "worker_coords_per_s": world * wl.n * wl.d / (step_ms * 1e-3)},
                "roofline": roof, "roofline_k2": roof2, "clocks": clocks, "e2e": e2e,
                # encode (global norm: first pass, two reduction kernels, the scales, second pass; buckets of
                # several pack blocks: first pass, one reduction kernel, second pass), decode, and the
                # effective-weights kernel of a multi-realisation update
                "gpu_launches": args.steps * ((5 if bucket == 0 else 3 if bucket > 512 else 1) + 1 + (1 if R > 1 else 0))}
        if not args.no_cpu_baseline:
            r = oracle_sample_rate(wl, code, bits, bucket, full_s=40.0)
            line["cpu_baseline"] = {"value": r["rate"], "unit": UNIT, "cores": 1, "host_cores": os.cpu_count(),
                                    "kind": "oracle",
                                    "sample": (f"the whole vector ({wl.d} coordinates, all {wl.n} workers), " if r["d"] == wl.d else
                                               f"{r['d']} of {wl.d} coordinates (whole pack blocks, all {wl.n} workers; "
                                               f"the rate extrapolates linearly), ") + f"one round, {r['seconds']:.1f} s",
                                    "encode": {"value": r["encode_rate"], "unit": UNIT},
                                    "decode": {"value": r["decode_rate"], "unit": UNIT}}
            line["parity_sample"] = parity_sample(ses, G, wl, code, bits, bucket)
        print(json.dumps(line))
    ses.close()
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
