#!/usr/bin/env python
"""Benchmark of the double-quantization round on B200.

Default workload ("c5"): the quantiser/packer bandwidth configuration -- M = 8 worker gradient vectors of
d = 2^27 fp32 coordinates (N(0,1) with 0.1 % outliers x100), quantised to b = 4 bits and packed, aggregated
and prox-updated by the master, and the new model requantised to b_x = 8 bits.  One "step" is one such
round: ||v||_inf pass, quantise+pack, master unpack+aggregate+prox (model norm fused), model quantise.
Prints ONE JSON line:
  value / ms_per_step    whole-job rounds/s over exactly --steps steps (CUDA events, max over ranks)
  stages                 per-stage time, algorithmic GB/s and fraction of the HBM peak, twice: over the timed steps
                         (short run: the GPU usually still boosts) and from a loop of >= --sustain-s seconds per stage
                         with the SM clock sampled every 20 ms (where the 1 kW power cap settles the clock)
  roofline               the dominant kernel (quantise+pack) against the measured copy bandwidth
  sweep                  the c5 grid d in {2^24, 2^27} x b in {2,4,8} x sparsify off/on, each point with its own
                         clock record, fractions of the measured peak and of the nominal 8 TB/s
  e2e                    the same round through host buffers (copies inside the timed region)
  cpu_baseline           the CPU oracle on a bounded slice of the workload, threads stated
  training_configs       rounds/s of dq_rounds on c1..c4 and the network, per-stage times of the stage entry
                         points called one by one, bits per round, and the oracle's rate on the same data

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--log2d 27] [--bits 4]

With N > 1 (launched by torch.distributed.run) every rank runs an independent replica of the workload (the
path is single-GPU by definition; there is no exchange step) and the value is the sum over ranks.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "simulated-worker rounds/sec"
UNIT = "rounds/s"
NOMINAL_HBM_GBPS = 8000.0          # the figure the target is worded against
SEED = 1805


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--log2d", type=int, default=27)
    ap.add_argument("--bits", type=int, default=4)
    ap.add_argument("--workers", type=int, default=8)
    ap.add_argument("--sparsify", type=int, default=0)
    ap.add_argument("--sequential", type=int, default=0, help="1: master applies one prox step per message")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--sustain-s", type=float, default=1.5, help="seconds each stage is looped for the sustained-clock figure (0: skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="leave the c5 grid out of the line")
    ap.add_argument("--sweep", action="store_true", help="print only the c5 grid (adds d = 2^20) as one JSON object")
    ap.add_argument("--only-training", action="store_true", help="time only the training configurations of --configs (one JSON object)")
    ap.add_argument("--train-rounds", type=int, default=200, help="rounds timed per training configuration")
    ap.add_argument("--tensor-cores", type=int, default=0, help="training configurations: dq_config.tensor_cores (1: both products of the "
                                                                "dense bf16 gradient as MMAs, 2: the margins only)")
    ap.add_argument("--no-fused", type=int, default=0, help="training configurations: dq_config.no_fused")
    ap.add_argument("--configs", default="c1,c2,c2_tau3,c3,c4,nn", help="training configurations to time with dq_rounds ('' for none)")
    return ap.parse_args()


def workload_config(a):
    d = 1 << a.log2d
    return {"workload": "c5 quantiser/packer sweep point: d=2^%d, M=%d, b=%d, b_x=8, sparsify=%s, lambda1=1e-6, eta=0.1"
                        % (a.log2d, a.workers, a.bits, "on(phi=0.01d)" if a.sparsify else "off"),
            "d": d, "M": a.workers, "b": a.bits, "bx": 8, "sparsify": a.sparsify, "sequential_master": a.sequential,
            "l2_policy": "inputs larger than L2 (%.0f MiB per round)" % (a.workers * d * 4 / 2 ** 20)}


# ---------------------------------------------------------------------------------------------------------------
# CPU oracle leg (cpu_baseline of the main line, and the whole of --impl reference)
# ---------------------------------------------------------------------------------------------------------------
def oracle_codec_round(v, x, g, b, rnd, sparsify, pool=None):
    """One codec round of the oracle as it stands: every worker's message, the master step, the model's codes.
    pool: a thread pool over the M independent workers (the C functions release the interpreter lock)."""
    import numpy as np
    import oracle
    M, ds = v.shape

    def one(w):
        if sparsify:
            r = oracle.sparsify(v[w], 0.01 * ds, SEED, rnd, w)
            return oracle.quantize_survivors(r["beta"], r["Z"], b, SEED, rnd, w)[:2]
        return oracle.quantize(v[w], b, SEED, rnd, w, oracle.STREAM_GRAD)[:2]

    res = list(pool.map(one, range(M))) if pool is not None else [one(w) for w in range(M)]
    raw = np.stack([r[0] for r in res]); delta = np.array([r[1] for r in res], np.float32)
    oracle.master_step(raw, delta, g, x, 0.1, l1=1e-6)
    oracle.quantize(x, 8, SEED, rnd, oracle.MASTER, oracle.STREAM_MODEL)


def oracle_rounds_per_sec(a, steps, warmup, log2_sample, threads):
    """Times the oracle's codec round on a d = 2^log2_sample slice of the workload (same recipe, same M, b, sparsify);
    the work is linear in d, so the full-size rate is the slice's rate times 2^log2_sample / d.  Returns
    (rounds/s at full size, seconds per sampled round, description)."""
    from concurrent.futures import ThreadPoolExecutor
    from paper_1805_10111_b200 import synth
    ls = min(log2_sample, a.log2d)
    ds = 1 << ls
    v, x, g = synth.config5(ds, a.workers)
    x = x.copy()
    pool = ThreadPoolExecutor(threads) if threads > 1 else None
    times = []
    for rnd in range(warmup + steps):
        t0 = time.perf_counter()
        oracle_codec_round(v, x, g, a.bits, rnd, a.sparsify, pool)
        if rnd >= warmup:
            times.append(time.perf_counter() - t0)
    if pool is not None:
        pool.shutdown()
    sec = sum(times) / len(times)
    what = ("oracle codec round on a d=2^%d slice of the workload (%d timed rounds, %d thread%s over the %d workers; master step and "
            "model quantiser single-threaded)%s" % (ls, steps, threads, "" if threads == 1 else "s", a.workers,
                                                     "" if ls == a.log2d else "; rate scaled by 2^%d/d (work is linear in d)" % ls))
    return (1.0 / sec) * ds / (1 << a.log2d), sec, what


def host_threads(M):
    return max(1, min(M, os.cpu_count() or 1))


def run_reference(a):
    """--impl reference: the oracle, as it stands, on the host cores.  Runs exactly --warmup + --steps rounds, each on a
    slice of the workload sized (from one calibration round at d = 2^18) so that the whole run takes about a minute."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = host_threads(a.workers)
    _, sec18, _ = oracle_rounds_per_sec(a, steps=1, warmup=0, log2_sample=min(18, a.log2d), threads=threads)
    budget = 60.0 / max(1, a.steps + a.warmup)                               # seconds per round
    ls = min(18, a.log2d)
    while ls < a.log2d and sec18 * (1 << (ls + 1 - min(18, a.log2d))) <= budget:
        ls += 1
    val, sec, what = oracle_rounds_per_sec(a, a.steps, a.warmup, ls, threads)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": a.gpus, "steps": a.steps,
            "warmup": a.warmup, "ms_per_step": 1000.0 / val, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": workload_config(a),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what,
                             "seconds_per_sampled_round": sec, "extrapolated": ls != a.log2d},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ---------------------------------------------------------------------------------------------------------------
# helpers
# ---------------------------------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi polled every `period_ms` while a timed region runs (read-only queries; no setting is touched)."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index, period_ms=20):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.FIELDS,
                                          "--format=csv,noheader,nounits", "-lms", str(period_ms)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.05)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill(); out, _ = self.proc.communicate()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in out.strip().splitlines():
            p = [t.strip() for t in ln.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0])); smax.append(float(p[1])); power.append(float(p[2]))
            except ValueError:
                continue
            for nm, flag in zip(names, p[3:7]):
                if flag.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_mhz_min": sm[0], "sm_max_mhz": max(smax), "power_w_max": max(power),
                "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(value, dist=None, device="cpu"):
    """The slowest rank's time: every rank must have finished before the job has."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(value)
    import torch
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(world, steps, slowest_ms):
    """Replicas are independent: the job processed world * steps rounds in the slowest rank's time."""
    return world * steps / (slowest_ms / 1000.0)


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return float(json.load(open(p))["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


def kernel_source_hash():
    h = hashlib.sha256()
    for f in ("dq_codec.cu", "dq_common.cuh"):
        h.update(open(os.path.join(ROOT, "paper_1805_10111_b200", "csrc", f), "rb").read())
    return h.hexdigest()[:16]


def recorded_traffic(bits):
    """DRAM bytes per coordinate of quantize_pack_kernel from the committed ncu summary, or None if the kernel
    source has changed since that capture."""
    p = os.path.join(ROOT, "profiles", "quantize_pack_kernel_c5.md")
    if not os.path.exists(p):
        return None
    t = open(p).read()
    m = re.search(r"source_sha256_16:\s*([0-9a-f]{16})", t)
    k = re.search(r"dram_bytes_per_coordinate_b%d:\s*([0-9.]+)" % bits, t)
    if not m or not k or m.group(1) != kernel_source_hash():
        return None
    return float(k.group(1))


STAGE_NAMES = ["norm_inf", "quantize_pack", "master_unpack_aggregate_prox", "quantize_model"]


def codec_alg_bytes(M, d, b, bx, sparsify):
    """Algorithmic bytes per launch of the four codec stages: norm 4 B and quantise+pack 4 + b/8 B per message
    coordinate (8 + b/8 when sparsifying: ||v||_1 must be known before the first mask bit can be drawn, so the vectors
    are read twice), master M b/8 + 12 B and model quantise 4 + b_x/8 B per model coordinate."""
    return [M * d * 4.0, M * d * ((8.0 if sparsify else 4.0) + b / 8.0), d * (M * b / 8.0 + 12.0), d * (4.0 + bx / 8.0)]


def stage_report(ms_list, alg, peak):
    return {n: {"ms": round(ms, 4), "alg_GBps": round(by / ms / 1e6, 1), "frac_of_peak": round(by / ms / 1e6 / peak, 4),
                "frac_of_8TBps": round(by / ms / 1e6 / NOMINAL_HBM_GBPS, 4)}
            for n, ms, by in zip(STAGE_NAMES, ms_list, alg)}


# ---------------------------------------------------------------------------------------------------------------
# whole training rounds (dq_rounds) on the training configurations, and their stages one by one
# ---------------------------------------------------------------------------------------------------------------
TRAIN_CONFIGS = {
    "c1": dict(gen="config1", kw=dict(M=4, B=16, bx=8, b=8, lambda1=1e-4), lr=1.0, theta=0.0, m=200),
    "c2": dict(gen="config2", kw=dict(M=8, B=64, bx=8, b=4, lambda2=1e-5), lr=1.0, theta=0.0, m=200),
    # the same rounds with workers that lag 0..3 rounds behind the master (Algorithm 1 step 11, x_{D(t)}): what delays cost
    "c2_tau3": dict(gen="config2", kw=dict(M=8, B=64, bx=8, b=4, lambda2=1e-5, max_delay=3), lr=1.0, theta=0.0, m=200,
                    delays=[0, 1, 2, 3, 0, 1, 2, 3]),
    # sparse_cap: a message holds at most B * nnz/row = 12,800 entries here; the default capacity (d) would have the
    # round clear 8 MiB of code buffers for a few hundred bytes of codes
    "c3": dict(gen="config3", kw=dict(M=16, B=128, bx=8, b=4, lambda1=1e-6, sparsify=1, phi=0.01 * (1 << 20), msg_format=1,
                                      sparse_cap=1 << 14),
               lr=1.0, theta=0.0, m=200),
    "nn": dict(gen="config_nn", kw=dict(M=8, B=20, bx=8, b=4, lambda2=1e-4, model=1, hidden=100, classes=10), lr=0.1, theta=0.0, m=500),
    "c4": dict(gen="config4", kw=dict(M=32, B=256, bx=8, b=8, box_lo=-10.0, box_hi=10.0, accelerated=1), lr=1e-4,
               theta=0.1, m=200),
}


class _Raw:
    """A device address owned by the library, passed back to it."""
    def __init__(self, ptr):
        self._p = ptr

    def data_ptr(self):
        return self._p


def time_training_stages(dq, ctx, cfg, h, st, eta, theta, peak, reps=60):
    """The four stage entry points called one after the other on the context's own buffers (so the touched-group list
    of sparse gradients is used as in dq_round), CUDA events between them.  dq_round itself merges stages (the model
    quantiser also writes xhat - xsnap and clears accumulators, quantiser and master share a kernel for dense
    messages, small problems run in one cluster kernel), so these are the stages' stand-alone costs."""
    import torch
    _, buf = dq.dq_round_buffers(ctx)
    alpha, ninf = _Raw(buf["alpha"]), _Raw(buf["norm_inf"])
    codes_x, delta_x = _Raw(buf["codes_x"]), _Raw(buf["delta_x"])
    msgs = type("OwnMsgs", (), {"c": buf["msgs"]})()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(reps)]
    for k in range(-3, reps):
        rnd = 100000 + k
        e = ev[k] if k >= 0 else None
        if e: e[0].record()
        dq.ok(dq.dq_quantize_model(ctx, st.x, st.norm_x, rnd, codes_x, delta_x))
        if e: e[1].record()
        dq.ok(dq.dq_worker_grad(ctx, codes_x, delta_x, 0, st, rnd, None, alpha, ninf))
        if e: e[2].record()
        dq.ok(dq.dq_quantize_sparsify_pack(ctx, alpha, ninf, rnd, msgs))
        if e: e[3].record()
        dq.ok(dq.dq_master_unpack_aggregate_prox(ctx, msgs, st, eta, theta))
        if e: e[4].record()
    torch.cuda.synchronize()
    ms = [sorted(ev[k][i].elapsed_time(ev[k][i + 1]) for k in range(reps))[reps // 2] for i in range(4)]
    M, B, d, b, bx = cfg.M, cfg.B, int(cfg.d), cfg.b, cfg.bx
    if cfg.model == 1:
        grad_bytes, grad_what = M * B * h.d * 4.0 + 2 * d * 4.0, "sampled rows (fp32) + both parameter vectors"
    elif h.format == 1:
        nnz_row = float(h.row_ptr[-1]) / h.n
        grad_bytes, grad_what = M * B * nnz_row * 8.0, "8 B per gathered nonzero (%.0f per row)" % nnz_row
    else:
        grad_bytes, grad_what = M * B * h.d * (4.0 if h.format == 0 else 2.0), "sampled rows read once"
    sparse = bool(cfg.sparsify) and cfg.msg_format == 1
    alg = {"quantize_model": d * (4.0 + bx / 8.0), "worker_grad": grad_bytes,
           "quantize_sparsify_pack": None if sparse else M * d * ((8.0 if cfg.sparsify else 4.0) + b / 8.0),
           "master_unpack_aggregate_prox": d * ((0.0 if sparse else M * b / 8.0) + (32.0 if cfg.accelerated else 12.0))}
    out = {}
    for (name, by), t in zip(alg.items(), ms):
        out[name] = {"us": round(t * 1000.0, 2)}
        if by is not None:
            out[name].update(alg_bytes=int(by), alg_GBps=round(by / t / 1e6, 1), frac_of_peak=round(by / t / 1e6 / peak, 4),
                             frac_of_8TBps=round(by / t / 1e6 / NOMINAL_HBM_GBPS, 4))
    out["worker_grad"]["bytes_counted"] = grad_what
    if sparse:
        out["quantize_sparsify_pack"]["note"] = "works on the list of touched groups (KBs): bound by kernel latency, no bandwidth figure"
    out["sum_us"] = round(sum(ms) * 1000.0, 2)
    return out


def time_training_config(name, rounds=200, warmup=20, with_oracle=False, peak=None, extra=None):
    """rounds/s of dq_rounds on one of the training configurations (full size, synthetic data), the stages one by one,
    and the bits the paper's accounting charges per round."""
    import numpy as np
    import torch
    import paper_1805_10111_b200 as dq
    from paper_1805_10111_b200 import synth
    spec = TRAIN_CONFIGS[name]
    h = getattr(synth, spec["gen"])()
    is_nn = spec["kw"].get("model", 0) == 1
    x0 = synth.mlp_init(h.d, spec["kw"]["hidden"], spec["kw"]["classes"], 9) if is_nn else np.zeros(h.d, np.float32)
    cfg = dq.make_config(x0.size, spec["kw"]["M"], seed=SEED, **{k: v for k, v in spec["kw"].items() if k != "M"}, **(extra or {}))
    data = dq.Data(h)
    rc, ctx = dq.dq_create(cfg, data); dq.ok(rc, "dq_create " + name)
    if spec.get("delays"):
        dq.ok(dq.dq_set_delays(ctx, spec["delays"]))
    st = dq.State(x0, n=h.n, accelerated=bool(cfg.accelerated))
    theta = spec["theta"]; eta = spec["lr"] / theta if theta else spec["lr"]
    bits = torch.zeros(2, dtype=torch.int64, device="cuda")
    dq.ok(dq.dq_epoch_begin(ctx, st, theta))
    for r in range(warmup):
        dq.ok(dq.dq_round(ctx, st, r, eta, theta))
    torch.cuda.synchronize()
    sampler = ClockSampler(torch.cuda.current_device())
    l0 = dq.dq_launch_count(ctx)
    # three batches of `rounds` rounds, each one call; the median batch is reported and all three are listed (a process
    # that starts on an idle GPU can see its first milliseconds at a lower clock than the sampler's 20 ms grid shows)
    batch_ms = []
    for k in range(3):
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record()
        dq.ok(dq.dq_rounds(ctx, st, warmup + k * rounds, rounds, eta, theta, bits[0:1], bits[1:2]))      # one call for all rounds of the batch
        e1.record(); torch.cuda.synchronize()
        batch_ms.append(e0.elapsed_time(e1) / rounds)
    clocks = sampler.stop()
    ms = sorted(batch_ms)[1]
    launches = (dq.dq_launch_count(ctx) - l0) / (3 * rounds)
    out = {"rounds_per_s": round(1000.0 / ms, 1), "ms_per_round": round(ms, 4), "ms_per_round_batches": [round(v, 4) for v in batch_ms],
           "n": h.n, "d": int(cfg.d), "M": cfg.M, "B": cfg.B,
           "launches_per_round": launches, "bits_down": int(bits[0].item()),
           "bits_up": int(bits[1].item()), "bits_full_precision": 2 * cfg.M * 32 * int(cfg.d), "clocks": clocks}
    out["stages_one_by_one"] = time_training_stages(dq, ctx, cfg, h, st, eta, theta, peak or measured_peak()[0])
    rc, status = dq.dq_poll_status(ctx)
    out["device_status"] = status
    dq.dq_destroy(ctx)
    if with_oracle and not spec.get("delays"):       # the CPU figure is taken without delays (they change no arithmetic cost there)
        out["cpu_oracle"] = oracle_training_rounds_per_sec(h, spec, x0)
    return out


def oracle_training_rounds_per_sec(h, spec, x0, budget_s=5.0):
    """The CPU oracle on the same data and settings: an epoch boundary, one untimed round, then whole rounds until
    about budget_s seconds have gone (at least two).  Single thread."""
    import numpy as np
    import oracle
    kw = spec["kw"]
    ocfg = oracle.make_config(x0.size, kw["M"], kw["B"], kw["bx"], kw["b"], l1=kw.get("lambda1", 0.0), l2=kw.get("lambda2", 0.0),
                              box_lo=kw.get("box_lo", -np.inf), box_hi=kw.get("box_hi", np.inf), sparsify=kw.get("sparsify", 0),
                              phi=kw.get("phi", 0.0), msg_format=kw.get("msg_format", 0), accelerated=kw.get("accelerated", 0),
                              seed=SEED, model=kw.get("model", 0), hidden=kw.get("hidden", 0), classes=kw.get("classes", 0))
    data = oracle.Dataset(h.format, h.n, h.d, h.values, h.labels, getattr(h, "col_idx", None), getattr(h, "row_ptr", None))
    run = oracle.Run(ocfg, data, x0)
    theta = spec["theta"]; eta = spec["lr"] / theta if theta else spec["lr"]
    run.epoch_begin(theta)
    run.round(0, eta, theta)
    n, t0 = 0, time.perf_counter()
    while n < 2 or time.perf_counter() - t0 < budget_s:
        run.round(1 + n, eta, theta); n += 1
        if n >= 200:
            break
    sec = (time.perf_counter() - t0) / n
    return {"rounds_per_s": round(1.0 / sec, 3), "cores": 1, "kind": "oracle", "sample": "%d whole rounds at full size" % n}


# ---------------------------------------------------------------------------------------------------------------
# the quantiser/packer grid of the c5 configuration: stage times per point, each with its own clock record
# ---------------------------------------------------------------------------------------------------------------
def time_codec_point(dq, vs, x0, gf, M, d, b, bx, sparsify, peak, reps, device_index, eta=0.1):
    """Median stage times of the codec round over `reps` rounds on the vectors vs (a list of [M][d] device arrays that
    the rounds rotate over), with the SM clock sampled meanwhile."""
    import torch
    cfg = dq.make_config(d, M, b=b, bx=bx, seed=SEED, lambda1=1e-6, sparsify=sparsify, phi=0.01 * d if sparsify else 0.0)
    rc, ctx = dq.dq_create(cfg); dq.ok(rc, "dq_create")
    st = dq.State(x0); st.g_full.copy_(gf)
    msgs = dq.Msgs(cfg)
    ninf = torch.zeros(M, device="cuda")
    nbx = dq.dq_packed_bytes(d, bx)
    codes_x = torch.zeros(nbx, dtype=torch.uint8, device="cuda"); delta_x = torch.zeros(1, device="cuda")
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(reps)]
    sampler = None
    for k in range(-3, reps):
        if k == 0:
            torch.cuda.synchronize(); sampler = ClockSampler(device_index)
        vk = vs[k % len(vs)]
        e = ev[k] if k >= 0 else None
        if e: e[0].record()
        dq.ok(dq.dq_norm_inf(ctx, vk, M, ninf))
        if e: e[1].record()
        dq.ok(dq.dq_quantize_sparsify_pack(ctx, vk, ninf, 1000 + k, msgs))
        if e: e[2].record()
        dq.ok(dq.dq_master_unpack_aggregate_prox(ctx, msgs, st, eta))
        if e: e[3].record()
        dq.ok(dq.dq_quantize_model(ctx, st.x, st.norm_x, 1000 + k, codes_x, delta_x))
        if e: e[4].record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    rc, status = dq.dq_poll_status(ctx); assert rc == 0 and status == 0
    ms = [sorted(ev[k][i].elapsed_time(ev[k][i + 1]) for k in range(reps))[reps // 2] for i in range(4)]   # medians
    point = {"log2d": d.bit_length() - 1, "b": b, "sparsify": sparsify, "rounds_per_s": round(1000.0 / sum(ms), 1),
             "stages": stage_report(ms, codec_alg_bytes(M, d, b, bx, sparsify), peak), "clocks": clocks, "reps": reps}
    if sparsify:      # realised density of worker 0's message: nonzero entries of the dequantised vector
        out = torch.empty(d, device="cuda")
        dq.ok(dq.dq_unpack(ctx, msgs, 0, out))
        point["realised_density"] = round(float(torch.count_nonzero(out).item()) / d, 6)
        del out
    dq.dq_destroy(ctx)
    return point


def codec_grid(dq, v, x0, gf, M, bx, peak, device_index, log2ds=(24, 27), with_clean_input=True):
    """d x b x sparsify off/on.  v [M][2^27] holds the workload's vectors; smaller d take a leading part of it (the same
    distribution).  At d = 2^20 one set of inputs would sit in L2, so the rounds rotate over enough copies to exceed it."""
    import torch
    points = []
    flat = v.view(-1)
    for log2d in log2ds:
        d = 1 << log2d
        copies = max(1, min((256 << 20) // (M * d * 4), flat.numel() // (M * d)))
        vs = [flat[c * M * d:(c + 1) * M * d].view(M, d) for c in range(copies)]
        xs, gs = x0[:d].contiguous(), gf[:d].contiguous()
        reps = 200 if log2d <= 20 else (40 if log2d <= 24 else 12)
        for sparsify in (0, 1):
            for b in (2, 4, 8):
                points.append(time_codec_point(dq, vs, xs, gs, M, d, b, bx, sparsify, peak, reps, device_index))
    if with_clean_input:
        # the budget phi = 0.01 d exceeds ||v||_1/||v||_inf on vectors with x100 outliers (Lemma 2's condition clamps it to
        # about 0.2 % density); on plain N(0,1) vectors the same budget is feasible and 1 % density is realised
        d = 1 << 24
        g = torch.Generator(device="cuda"); g.manual_seed(180510111)
        clean = torch.randn((M, d), device="cuda", generator=g)
        p = time_codec_point(dq, [clean], x0[:d].contiguous(), gf[:d].contiguous(), M, d, 4, bx, 1, peak, 40, device_index)
        p["input"] = "N(0,1) without outliers"
        points.append(p)
        del clean
    return points


def time_stage_sustained(fns, min_s, device_index):
    """Each stage alone in a loop of at least min_s seconds (so that the power cap, not the boost clock, sets the pace),
    CUDA events around every call, SM clock sampled every 20 ms.  Returns per stage (median ms, clock record)."""
    import torch
    out = []
    for fn in fns:
        fn(); torch.cuda.synchronize()
        sampler = ClockSampler(device_index)
        times = []
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < min_s:
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(33)]
            ev[0].record()
            for k in range(32):
                fn(); ev[k + 1].record()
            torch.cuda.synchronize()
            times += [ev[k].elapsed_time(ev[k + 1]) for k in range(32)]
        clocks = sampler.stop()
        half = sorted(times[len(times) // 2:])                  # the second half of the loop: the clock has settled
        out.append((half[len(half) // 2], clocks, len(times)))
    return out


# ---------------------------------------------------------------------------------------------------------------
# GPU leg
# ---------------------------------------------------------------------------------------------------------------
def run_ours(a):
    import numpy as np
    import torch
    import paper_1805_10111_b200 as dq
    from paper_1805_10111_b200 import synth

    rank = int(os.environ.get("RANK", "0")); world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dq.lib()

    d, M, b, bx, eta = 1 << a.log2d, a.workers, a.bits, 8, 0.1
    cfg = dq.make_config(d, M, b=b, bx=bx, seed=SEED, lambda1=1e-6, sparsify=a.sparsify, phi=0.01 * d if a.sparsify else 0.0,
                         sequential=a.sequential)
    rc, ctx = dq.dq_create(cfg); dq.ok(rc, "dq_create")

    # seeded synthetic inputs, generated on the host straight into pinned memory (also the e2e source)
    hv = torch.empty((M, d), dtype=torch.float32).pin_memory()
    g = synth.rng(5 + 100 * rank)
    hv_np = hv.numpy()
    for w in range(M):
        row = hv_np[w]
        g.standard_normal(d, dtype=np.float32, out=row)
        row[g.integers(0, d, max(1, d // 1000))] *= np.float32(100.0)
    x0 = synth.normal_vector(d, 6); gf = synth.normal_vector(d, 7)
    v = hv.cuda(non_blocking=False)
    st = dq.State(x0); st.g_full.copy_(torch.from_numpy(gf).cuda())
    msgs = dq.Msgs(cfg)
    ninf = torch.zeros(M, device="cuda")
    nbx = dq.dq_packed_bytes(d, bx)
    codes_x = torch.zeros(nbx, dtype=torch.uint8, device="cuda"); delta_x = torch.zeros(1, device="cuda")

    stage_fns = [lambda rnd=0: dq.ok(dq.dq_norm_inf(ctx, v, M, ninf)),
                 lambda rnd=0: dq.ok(dq.dq_quantize_sparsify_pack(ctx, v, ninf, rnd, msgs)),
                 lambda rnd=0: dq.ok(dq.dq_master_unpack_aggregate_prox(ctx, msgs, st, eta)),
                 lambda rnd=0: dq.ok(dq.dq_quantize_model(ctx, st.x, st.norm_x, rnd, codes_x, delta_x))]

    def step(rnd, ev=None):
        for i, fn in enumerate(stage_fns):
            if ev: ev[i].record()
            fn(rnd)
        if ev: ev[4].record()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    warm = max(3, a.warmup)
    for rnd in range(warm):
        step(rnd)
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(a.steps)]
    barrier()
    sampler = ClockSampler(local)
    launches0 = dq.dq_launch_count(ctx)
    t_begin = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record()
    for k in range(a.steps):
        step(1000 + k, events[k])
    t_end.record()
    barrier()
    clocks = sampler.stop()
    launches = dq.dq_launch_count(ctx) - launches0
    total_ms = t_begin.elapsed_time(t_end)
    rc, status = dq.dq_poll_status(ctx)
    assert rc == 0 and status == 0, "device status %d" % status
    stage_ms = [sum(events[k][i].elapsed_time(events[k][i + 1]) for k in range(a.steps)) / a.steps for i in range(4)]
    total_ms = max_over_ranks(total_ms, dist, "cuda")
    ms_per_step = total_ms / a.steps
    value = whole_job_rate(world, a.steps, total_ms)
    peak, peak_src = measured_peak()
    alg = codec_alg_bytes(M, d, b, bx, a.sparsify)

    # every stage alone, long enough for the clock to settle under the power cap
    sustained = None
    if rank == 0 and world == 1 and a.sustain_s > 0:
        res = time_stage_sustained(stage_fns, a.sustain_s, local)
        sustained = {}
        for n, (ms, ck, calls), by in zip(STAGE_NAMES, res, alg):
            sustained[n] = {"ms": round(ms, 4), "alg_GBps": round(by / ms / 1e6, 1), "frac_of_peak": round(by / ms / 1e6 / peak, 4),
                            "frac_of_8TBps": round(by / ms / 1e6 / NOMINAL_HBM_GBPS, 4), "sm_mhz": ck.get("sm_mhz"),
                            "ms_x_mhz": None if ck.get("sm_mhz") is None else round(ms * ck["sm_mhz"], 1),
                            "power_w_max": ck.get("power_w_max"), "reasons": ck.get("reasons"), "calls": calls}

    # the optional width search of condition (3) on the same model (not part of the default round, mu = 0)
    sel_bits = torch.zeros(1, dtype=torch.int32, device="cuda"); sel_stats = torch.zeros(11, dtype=torch.float64, device="cuda")
    xs_dev = torch.from_numpy(x0).cuda()
    for _ in range(3):
        dq.ok(dq.dq_select_model_bits(ctx, st.x, xs_dev, st.norm_x, 1.0, sel_bits, sel_stats))
    s0 = torch.cuda.Event(enable_timing=True); s1 = torch.cuda.Event(enable_timing=True)
    s0.record()
    for _ in range(20):
        dq.ok(dq.dq_select_model_bits(ctx, st.x, xs_dev, st.norm_x, 1.0, sel_bits, sel_stats))
    s1.record(); torch.cuda.synchronize()
    select_ms = s0.elapsed_time(s1) / 20
    del xs_dev

    # end to end through the host-buffer entry point: H2D of the M gradient vectors, the round, D2H of the model codes
    e2e = None
    if a.e2e_steps > 0:
        dq.ok(dq.dq_codec_host_setup(ctx, x0, gf))
        hcodes = torch.zeros(nbx, dtype=torch.uint8).pin_memory(); hdelta = torch.zeros(1).pin_memory()
        dq.ok(dq.dq_codec_round_host(ctx, hv, 0, eta, hcodes, hdelta))
        barrier()
        t0 = time.perf_counter()
        for k in range(a.e2e_steps):
            dq.ok(dq.dq_codec_round_host(ctx, hv, 2000 + k, eta, hcodes, hdelta))
        torch.cuda.synchronize()
        e2e_s = time.perf_counter() - t0
        e2e_s = max_over_ranks(e2e_s, dist, "cuda")
        e2e = {"value": world * a.e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": M * d * 4,
               "d2h_bytes_per_step": nbx + 4, "steps": a.e2e_steps}

    if rank != 0:
        dq.dq_destroy(ctx)
        if dist is not None:
            dist.destroy_process_group()
        return
    stages = stage_report(stage_ms, alg, peak)
    # the width search is bound by the double-precision pipe: about 63 of its lane-slots per coordinate (ten widths x
    # five operations, two fp32->fp64 conversions at a quarter of the rate, the squared distance) on 64 lanes per SM
    sm_ghz = (clocks.get("sm_mhz") or 1965.0) / 1000.0
    alu_peak = 148 * 64 * sm_ghz * 1e9 / 63.0                      # coordinates per second
    stages["select_model_bits(optional)"] = {"ms": round(select_ms, 4), "alg_GBps": round(d * 8.0 / select_ms / 1e6, 1),
                                              "frac_of_peak": round(d * 8.0 / select_ms / 1e6 / peak, 4), "bound": "alu",
                                              "alu_peak_coordinates_per_s": round(alu_peak, 0),
                                              "frac_of_alu_peak": round(d / (select_ms * 1e-3) / alu_peak, 4)}
    qp = stages["quantize_pack"]
    tr = recorded_traffic(b) if not a.sparsify else None
    roofline = {"kernel": "quantize_pack_kernel<%d>" % b if not a.sparsify else "norm_l1_kernel + sparsify_stage_kernel + sparsify_scatter_dense_kernel<%d>" % b,
                "bound": "hbm", "achieved": qp["alg_GBps"], "peak": peak, "unit": "GB/s",
                "frac": round(qp["alg_GBps"] / peak, 4), "peak_source": peak_src,
                "frac_of_8TBps": qp["frac_of_8TBps"],
                "regime": "timed steps: %d steps, median SM clock %s MHz, reasons %s" % (a.steps, clocks.get("sm_mhz"), clocks.get("reasons")),
                "traffic": None if tr is None else tr * M * d,
                "alg_bytes_per_launch": alg[1]}
    if sustained:
        roofline["sustained"] = {k: sustained["quantize_pack"][k] for k in ("ms", "alg_GBps", "frac_of_peak", "sm_mhz", "reasons")}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": a.steps, "warmup": warm,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "config": workload_config(a), "roofline": roofline,
            "stages": stages, "stages_sustained": sustained, "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "bits_per_round": {"down": M * (32 + bx * d), "up_dense": M * (32 + b * d), "full_precision": 2 * M * 32 * d}}
    dq.dq_destroy(ctx)
    del st, msgs
    if world == 1 and not a.no_sweep and a.log2d >= 27:
        xd = torch.from_numpy(x0).cuda(); gd = torch.from_numpy(gf).cuda()
        line["sweep"] = {"what": "c5 grid: M=%d, b_x=8, lambda1=1e-6, eta=0.1, phi=0.01d when sparsifying; medians over `reps` rounds; "
                                 "fractions of the measured copy peak and of the nominal 8 TB/s" % M,
                         "peak_GBps": peak, "points": codec_grid(dq, v, xd, gd, M, bx, peak, local)}
        below = [(p["log2d"], p["b"], p["sparsify"], n, s["frac_of_peak"]) for p in line["sweep"]["points"]
                 for n, s in p["stages"].items() if n in ("quantize_pack", "master_unpack_aggregate_prox") and s["frac_of_peak"] < 0.70]
        line["sweep"]["below_0.70_of_measured_peak"] = below
        del xd, gd
    del v
    torch.cuda.empty_cache()
    if world == 1 and not a.no_cpu_baseline:
        threads = host_threads(M)
        val, sec, what = oracle_rounds_per_sec(a, steps=2, warmup=0, log2_sample=24, threads=threads)
        line["cpu_baseline"] = {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": what,
                                "seconds_per_sampled_round": round(sec, 3), "extrapolated": a.log2d > 24}
        if threads > 1:
            val1, sec1, _ = oracle_rounds_per_sec(a, steps=1, warmup=0, log2_sample=22, threads=1)
            line["cpu_baseline"]["single_thread_value"] = val1
    del hv
    if world == 1 and a.configs:
        line["training_configs"] = {c: time_training_config(c, with_oracle=not a.no_cpu_baseline, peak=peak)
                                    for c in a.configs.split(",") if c in TRAIN_CONFIGS}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_sweep(a):
    """Only the grid (with d = 2^20 added), on vectors drawn on the device."""
    import torch
    import paper_1805_10111_b200 as dq
    torch.cuda.set_device(0)
    dq.lib()
    peak, peak_src = measured_peak()
    M, d = a.workers, 1 << 27
    g = torch.Generator(device="cuda"); g.manual_seed(180510111 + 27)
    v = torch.randn((M, d), device="cuda", generator=g)
    idx = torch.randint(0, d, (M, max(1, d // 1000)), device="cuda", generator=g)
    v.scatter_(1, idx, v.gather(1, idx) * 100.0)                      # 0.1 % outliers x100
    x0 = torch.randn(d, device="cuda", generator=g); gf = torch.randn(d, device="cuda", generator=g)
    points = codec_grid(dq, v, x0, gf, M, 8, peak, 0, log2ds=(20, 24, 27))
    print(json.dumps({"sweep": "c5 quantiser/packer: M=%d, b_x=8, lambda1=1e-6, eta=0.1, phi=0.01d when sparsifying" % M,
                      "peak_GBps": peak, "peak_source": peak_src, "l2_policy": "inputs rotated over >= 256 MiB", "points": points}))


def run_training_only(a):
    import torch
    import paper_1805_10111_b200 as dq
    torch.cuda.set_device(0)
    dq.lib()
    peak, _ = measured_peak()
    extra = {"tensor_cores": a.tensor_cores, "no_fused": a.no_fused}
    print(json.dumps({"dq_config": extra,
                      "training_configs": {c: time_training_config(c, rounds=a.train_rounds, with_oracle=not a.no_cpu_baseline, peak=peak, extra=extra)
                                           for c in a.configs.split(",") if c in TRAIN_CONFIGS}}))


def main():
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    elif a.only_training:
        run_training_only(a)
    elif a.sweep:
        run_sweep(a)
    else:
        run_ours(a)


if __name__ == "__main__":
    main()
