#!/usr/bin/env python
"""Benchmark of the verify step (one step = one pass of the whole hot path over one batch).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5_K..] [--impl reference]

Prints ONE JSON line.  `value` = verify-steps/s with inputs resident in HBM (CUDA events, max over
ranks); `e2e` = the same metric through the host-buffer entry point (copies inside the timed
region); `roofline` = algorithmic bytes of the logit-streaming kernel / its event-timed duration
against the measured HBM copy peak; `cpu_baseline` = the float64 oracle timed on the host cores.
N > 1 (torchrun): batch rows are independent, so every rank verifies its own batches with no
collective in the data path (weak scaling); only the timing is reduced (max over ranks).
"""
from __future__ import annotations

import argparse
import ctypes
import json
import math
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

L2_BYTES = 126e6
FALLBACK_HBM_GBS = 6650.0


def describe(cfg) -> str:
    return (f"{cfg.name}: B={cfg.B},K={cfg.K},gamma={cfg.gamma},V={cfg.V},{cfg.dtype},T={cfg.temperature},"
            f"alpha={cfg.alpha}")


def algorithmic_bytes(cfg, n_bonus: float) -> dict:
    """Bytes the method must move per verify step (each needed logit exactly once)."""
    s = 2 if cfg.dtype == "bf16" else 4
    B, K, g, V = cfg.B, cfg.K, cfg.gamma, cfg.V
    sweep = 2 * B * K * g * V * s                       # target rows i < gamma and all draft rows
    bonus = n_bonus * V * s                             # target row gamma of fully accepted drafts
    small = B * K * g * (4 + 4) + B * (K * g + 1) * 4 + B * (g + 3) * 4
    return {"sweep": sweep, "step": sweep + bonus + small}


def kernel_traffic(workload: str):
    """DRAM bytes per launch of the logit-streaming kernel from the committed ncu capture
    (profiles/fused_chain_kernel_traffic.txt), or None if there is no capture for this workload or the
    kernel source has changed since the counters were taken."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "fused_chain_kernel_traffic.txt")
    src = os.path.join(ROOT, "paper_2604_25925_b200", "csrc", "sgbv_fused.cu")
    try:
        sha = hashlib.sha256(open(src, "rb").read()).hexdigest()
        vals = {}
        for line in open(path):
            if ":" in line and not line.startswith("#"):
                k, v = line.split(":", 1)
                vals[k.strip()] = v.strip()
        if vals.get("source_sha256") != sha or workload not in vals:
            return None
        return int(vals[workload].split()[0])
    except Exception:
        return None


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clocks/throttle reasons sampled every 100 ms while the timed region runs."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        cmd = ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"]
        if uuid:
            cmd += ["-i", uuid]
        try:
            self.proc = subprocess.Popen(cmd, stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t0: float, t1: float) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        rows = []
        for line in self.tmp.read().splitlines():
            p = [x.strip() for x in line.split(",")]
            if len(p) < 8:
                continue
            try:
                ts = time.mktime(time.strptime(p[0].split(".")[0], "%Y/%m/%d %H:%M:%S")) + float("0." + p[0].split(".")[1])
                rows.append((ts, float(p[1]), float(p[2]), float(p[3]), p[4:8]))
            except Exception:
                continue
        os.unlink(self.tmp.name)
        inside = [r for r in rows if t0 - 0.05 <= r[0] <= t1 + 0.05] or rows
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        sm = sorted(r[1] for r in inside)
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        reasons = [n for j, n in enumerate(names) if any(r[4][j].lower().startswith("active") for r in inside)]
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": inside[0][2], "power_w_max": max(r[3] for r in inside),
                "samples": len(inside), "reasons": reasons}


def time_oracle(cfg, inp_cpu, budget_s: float = 12.0):
    """Oracle on the host cores: whole steps if one fits the budget, else the first batch rows
    of one step, scaled to whole steps.  -> (steps/s, threads, sample text, result, rows or None)"""
    import oracle
    zq = inp_cpu.target_logits.float().numpy()
    zp = inp_cpu.draft_logits.float().numpy()
    tok, u = inp_cpu.draft_tokens.numpy(), inp_cpu.uniforms.numpy()
    cores = os.cpu_count() or 1
    t = time.perf_counter()
    oracle.verify(zq[:1], zp[:1], tok[:1], u[:1], cfg.temperature)
    per_row = time.perf_counter() - t                      # one batch row on one core
    est_step = per_row * math.ceil(cfg.B / min(cores, cfg.B))
    if est_step <= budget_s:
        reps = int(max(1, min(50, budget_s // max(est_step, 1e-3))))
        t = time.perf_counter()
        for _ in range(reps):
            res = oracle.verify(zq, zp, tok, u, cfg.temperature)
        dt = time.perf_counter() - t
        return reps / dt, res.threads, f"{reps} whole step(s) of {cfg.name} (all {cfg.B} batch rows)", res, None
    rows = int(min(cfg.B, max(1, budget_s / per_row) * min(cores, cfg.B)))
    rows = max(min(cores, cfg.B), rows // min(cores, cfg.B) * min(cores, cfg.B))
    t = time.perf_counter()
    res = oracle.verify(zq[:rows], zp[:rows], tok[:rows], u[:rows], cfg.temperature)
    dt = time.perf_counter() - t
    return ((rows / cfg.B) / dt, res.threads,
            f"first {rows} of {cfg.B} batch rows of one {cfg.name} step, scaled to whole steps", res, rows)


def run_reference(args):
    """The oracle as the reference arm: rank 0 only, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from paper_2604_25925_b200 import workloads
    cfg = workloads.get_config(args.workload)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    B_gen = cfg.B if cfg.logit_bytes() < 2e9 else max(8, os.cpu_count() or 8)
    inp = workloads.make_inputs(workloads.with_batch(cfg, min(cfg.B, B_gen)), device=dev).to("cpu")
    import oracle
    zq, zp = inp.target_logits.float().numpy(), inp.draft_logits.float().numpy()
    tok, u = inp.draft_tokens.numpy(), inp.uniforms.numpy()
    t = time.perf_counter()
    res = oracle.verify(zq[:1], zp[:1], tok[:1], u[:1], cfg.temperature)
    per_row = time.perf_counter() - t
    cores = os.cpu_count() or 1
    total = args.steps + args.warmup
    rows = int(min(zq.shape[0], max(1, (120.0 / total) / per_row * min(cores, zq.shape[0]))))
    for _ in range(args.warmup):
        res = oracle.verify(zq[:rows], zp[:rows], tok[:rows], u[:rows], cfg.temperature)
    t = time.perf_counter()
    for _ in range(args.steps):
        res = oracle.verify(zq[:rows], zp[:rows], tok[:rows], u[:rows], cfg.temperature)
    dt = time.perf_counter() - t
    value = args.steps * (rows / cfg.B) / dt
    sample = f"each step = first {rows} of {cfg.B} batch rows of {cfg.name}, scaled to whole steps"
    line = {"impl": "reference", "metric": "verify_steps_per_s", "value": value, "unit": "verify-steps/s",
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": describe(cfg)},
            "cpu_baseline": {"value": value, "unit": "verify-steps/s", "cores": int(res.threads), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "verify-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = args.steps or 3
        args.warmup = args.warmup if args.warmup is not None else 1
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2604_25925_b200 import binding, sharding, workloads

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the verify path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    cfg = workloads.get_config(args.workload)
    set_bytes = cfg.logit_bytes()
    # enough input sets to exceed twice the L2; capped for toy shapes, whose line then says that they stay in L2
    nsets = int(min(512, max(2, math.ceil(2.2 * L2_BYTES / set_bytes))))
    est_ms = max(0.02, set_bytes / 2.5e9)                  # rough step time for choosing defaults
    steps = args.steps if args.steps is not None else int(max(20, min(50000, 4000.0 / est_ms)))
    warmup = args.warmup if args.warmup is not None else max(3, min(50, steps // 10))
    warmup = max(3, warmup)

    sets = [workloads.make_inputs(cfg, device=dev, set_index=rank * 1000 + i) for i in range(nsets)]
    outs = [binding.VerifyOutput(torch.empty(cfg.B, dtype=torch.int32, device=dev),
                                 torch.empty(cfg.B, dtype=torch.int32, device=dev),
                                 torch.empty((cfg.B, cfg.gamma + 1), dtype=torch.int32, device=dev))
            for _ in range(nsets)]
    lib = binding.load()
    fn = lib.sgbv_verify_bf16 if cfg.dtype == "bf16" else lib.sgbv_verify
    stream = torch.cuda.current_stream(dev)
    calls = []
    for inp, out in zip(sets, outs):
        calls.append((inp.target_logits.data_ptr(), inp.draft_logits.data_ptr(), inp.draft_tokens.data_ptr(),
                      inp.uniforms.data_ptr(), cfg.B, cfg.K, cfg.gamma, cfg.V, float(cfg.temperature),
                      out.accept_len.data_ptr(), out.draft_idx.data_ptr(), out.tokens.data_ptr(),
                      stream.cuda_stream))

    def step(i):
        rc = fn(*calls[i % nsets])
        if rc != 0:
            raise binding.SgbvError(rc)

    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        pass
    sampler = ClockSampler(uuid) if rank == 0 else None
    time.sleep(0.25)
    # the warm-up steps run right before the timed ones (the sampler's start-up pause would let the GPU idle)
    for i in range(warmup):
        step(i)
    torch.cuda.synchronize()
    launches_per_step = binding.last_launch_count()
    # event pairs around the streaming kernel on a tenth of the timed steps at most: the records sit between
    # the two kernels of a step and between steps, where they cost the overlap that the launches otherwise have
    nrec = max(1, min(steps // 10, 4000))
    binding.profile_begin(nrec)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    ev0.record(stream)
    for i in range(steps):
        step(i)
    ev1.record(stream)
    torch.cuda.synchronize()
    t1 = time.time()
    if world > 1:
        dist.barrier()
    ms_total = ev0.elapsed_time(ev1)
    kern_ms, kern_n = binding.profile_end()
    ms_total = sharding.max_over_ranks(ms_total, device=dev)   # a step takes as long as its slowest rank
    clocks = sampler.stop(t0, t1) if sampler else None

    # parity-relevant facts of the timed outputs, and the end-to-end / CPU legs (rank 0)
    n_bonus = float(sum(int((o.accept_len == cfg.gamma).sum().item()) for o in outs)) / nsets
    be = float(sum(float((o.accept_len.float() + 1).mean().item()) for o in outs)) / nsets
    if rank == 0:
        ab = algorithmic_bytes(cfg, n_bonus)
        ms_step = ms_total / steps
        value = world * steps / (ms_total * 1e-3)
        peak, which = hbm_peak()
        kern_avg_ms = kern_ms / max(kern_n, 1)
        achieved = ab["sweep"] / (kern_avg_ms * 1e-3) / 1e9 if kern_n else None
        line = {
            "metric": "verify_steps_per_s", "value": value, "unit": "verify-steps/s", "n_gpus": world,
            "steps": steps, "warmup": warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": describe(cfg),
                       "l2": f"{nsets} rotating input sets of {set_bytes / 1e6:.1f} MB "
                             f"({nsets * set_bytes / 1e6:.0f} MB total, L2 is 126 MB)"
                             + ("" if nsets * set_bytes >= 2 * L2_BYTES else ": NOT larger than L2, no flush"),
                       "per_rank_batch": cfg.B},
            "hbm_gbs_step": ab["step"] / (ms_step * 1e-3) / 1e9,
            "algorithmic_bytes_per_step": ab["step"],
            "block_efficiency": be,
            "roofline": {"bound": "hbm", "kernel": binding.last_main_kernel(), "achieved": achieved, "peak": peak,
                         "unit": "GB/s", "frac": (achieved / peak) if achieved else None,
                         "peak_source": f"of {which}", "kernel_ms": kern_avg_ms, "launches_timed": kern_n,
                         "algorithmic_bytes_per_launch": ab["sweep"], "traffic": kernel_traffic(cfg.name)},
            "gpu_launches": launches_per_step * steps,
            "clocks": clocks,
        }
        if not args.no_e2e:
            host = sets[0].to("cpu")
            pinned = [t.pin_memory() for t in (host.target_logits, host.draft_logits, host.draft_tokens,
                                               host.uniforms)]
            hout = binding.VerifyOutput(torch.empty(cfg.B, dtype=torch.int32).pin_memory(),
                                        torch.empty(cfg.B, dtype=torch.int32).pin_memory(),
                                        torch.empty((cfg.B, cfg.gamma + 1), dtype=torch.int32).pin_memory(),
                                        status=torch.empty(cfg.B, dtype=torch.int32).pin_memory())
            e_steps = int(max(3, min(steps, 2.0 / max(set_bytes / 20e9, 1e-4))))
            for _ in range(2):
                binding.sgbv_verify_host(*pinned, cfg.temperature, out=hout, device=local)
            t = time.perf_counter()
            for _ in range(e_steps):
                binding.sgbv_verify_host(*pinned, cfg.temperature, out=hout, device=local)
            dt = time.perf_counter() - t
            h2d = sum(t.numel() * t.element_size() for t in pinned)
            d2h = sum(t.numel() * t.element_size() for t in (hout.accept_len, hout.draft_idx, hout.tokens,
                                                             hout.status))
            line["e2e"] = {"value": world * e_steps / dt, "unit": "verify-steps/s", "h2d_bytes_per_step": h2d,
                           "d2h_bytes_per_step": d2h, "steps": e_steps,
                           "note": "sgbv_verify_host: pinned host buffers, copies and sync inside the timed region"}
        if not args.no_cpu_baseline:
            from oracle.compare import compare
            host = sets[0].to("cpu")
            v, cores, sample, ref, rows = time_oracle(cfg, host)
            line["cpu_baseline"] = {"value": v, "unit": "verify-steps/s", "cores": int(cores), "kind": "oracle",
                                    "sample": sample}
            dx = binding.sgbv_verify_ex(sets[0].target_logits, sets[0].draft_logits, sets[0].draft_tokens,
                                        sets[0].uniforms, cfg.temperature)
            torch.cuda.synchronize()
            sl = slice(None) if rows is None else slice(0, rows)
            rep = compare(ref, dx.accept_len[sl].cpu().numpy(), dx.draft_idx[sl].cpu().numpy(),
                          dx.tokens[sl].cpu().numpy(), dx.h[sl].cpu().numpy(), dx.resmass[sl].cpu().numpy(),
                          dx.status[sl].cpu().numpy())
            line["parity"] = rep.summary()
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
