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
NOMINAL_HBM_GBS = 8000.0        # the nominal peak the fractions are also quoted against


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


def config_dict(cfg, nsets=None, set_bytes=None) -> dict:
    """The `config` object of the JSON line; the same from both arms."""
    d = {"workload": describe(cfg), "per_rank_batch": cfg.B}
    if nsets is not None:
        d["l2"] = (f"{nsets} rotating input sets of {set_bytes / 1e6:.1f} MB ({nsets * set_bytes / 1e6:.0f} MB total, "
                   "L2 is 126 MB)" + ("" if nsets * set_bytes >= 2 * L2_BYTES else ": NOT larger than L2, no flush"))
    return d


def rotating_sets(cfg) -> int:
    """Enough input sets to exceed twice the L2; capped for toy shapes, whose line then says that they stay in L2."""
    return int(min(512, max(2, math.ceil(2.2 * L2_BYTES / cfg.logit_bytes()))))


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
            "config": config_dict(cfg, rotating_sets(cfg), cfg.logit_bytes()),
            "cpu_baseline": {"value": value, "unit": "verify-steps/s", "cores": int(res.threads), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": "verify-steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


class Workload:
    """One configuration resident on the device: rotating input sets, output buffers, prepared C-ABI calls."""

    def __init__(self, cfg, dev, rank):
        import torch
        from paper_2604_25925_b200 import binding, workloads
        self.cfg, self.dev = cfg, dev
        self.nsets = rotating_sets(cfg)
        self.sets = [workloads.make_inputs(cfg, device=dev, set_index=rank * 1000 + i) for i in range(self.nsets)]
        self.outs = [binding.VerifyOutput(torch.empty(cfg.B, dtype=torch.int32, device=dev),
                                          torch.empty(cfg.B, dtype=torch.int32, device=dev),
                                          torch.empty((cfg.B, cfg.gamma + 1), dtype=torch.int32, device=dev))
                     for _ in range(self.nsets)]
        lib = binding.load()
        self.fn = lib.sgbv_verify_bf16 if cfg.dtype == "bf16" else lib.sgbv_verify
        self.stream = torch.cuda.current_stream(dev)
        self.calls = [(i.target_logits.data_ptr(), i.draft_logits.data_ptr(), i.draft_tokens.data_ptr(),
                       i.uniforms.data_ptr(), cfg.B, cfg.K, cfg.gamma, cfg.V, float(cfg.temperature),
                       o.accept_len.data_ptr(), o.draft_idx.data_ptr(), o.tokens.data_ptr(), self.stream.cuda_stream)
                      for i, o in zip(self.sets, self.outs)]
        self.count = 0

    def step(self):
        from paper_2604_25925_b200 import binding
        rc = self.fn(*self.calls[self.count % self.nsets])
        self.count += 1
        if rc != 0:
            raise binding.SgbvError(rc)


def timed_blocks(wl, steps, warmup, world, min_seconds=1.0, max_repeats=400):
    """Blocks of exactly `steps` steps, each bracketed by a barrier and a synchronisation on both sides and timed
    with CUDA events on the launching stream, repeated until `min_seconds` have been timed.  Returns the per-block
    milliseconds (max over ranks), the wall-clock interval, and the kernel launches per step."""
    import torch
    import torch.distributed as dist
    from paper_2604_25925_b200 import binding, sharding
    for _ in range(warmup):
        wl.step()
    torch.cuda.synchronize()
    launches_per_step = binding.last_launch_count()
    blocks, total = [], 0.0
    t0 = time.time()
    while True:
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(wl.stream)
        for _ in range(steps):
            wl.step()
        ev1.record(wl.stream)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        ms = sharding.max_over_ranks(ev0.elapsed_time(ev1), device=wl.dev)   # a block takes as long as its slowest rank
        blocks.append(ms)
        total += ms
        if total >= 1e3 * min_seconds or len(blocks) >= max_repeats:   # (the same decision on every rank: ms is the max)
            break
    return blocks, (t0, time.time()), launches_per_step


def kernel_pass(wl, n):
    """A separate pass of n steps with an event pair around the streaming kernel of every step (the pairs sit between
    the kernels of a step, so this pass is not the one `value` comes from).  -> (mean kernel ms, launches timed)"""
    import torch
    from paper_2604_25925_b200 import binding
    binding.profile_begin(n)
    for _ in range(n):
        wl.step()
    torch.cuda.synchronize()
    ms, cnt = binding.profile_end()
    return ms / max(cnt, 1), cnt


def parity_report(wl, budget_s):
    """Oracle on the host cores against the CUDA path on the first input set (whole batch or its first rows)."""
    import torch
    from oracle.compare import compare
    from paper_2604_25925_b200 import binding
    cfg = wl.cfg
    host = wl.sets[0].to("cpu")
    v, cores, sample, ref, rows = time_oracle(cfg, host, budget_s)
    s0 = wl.sets[0]
    dx = binding.sgbv_verify_ex(s0.target_logits, s0.draft_logits, s0.draft_tokens, s0.uniforms, cfg.temperature)
    torch.cuda.synchronize()
    sl = slice(None) if rows is None else slice(0, rows)
    rep = compare(ref, dx.accept_len[sl].cpu().numpy(), dx.draft_idx[sl].cpu().numpy(), dx.tokens[sl].cpu().numpy(),
                  dx.h[sl].cpu().numpy(), dx.resmass[sl].cpu().numpy(), dx.status[sl].cpu().numpy())
    return rep.summary(), {"value": v, "unit": "verify-steps/s", "cores": int(cores), "kind": "oracle", "sample": sample}


def roofline_of(wl, ab, kern_ms, kern_n):
    from paper_2604_25925_b200 import binding
    peak, which = hbm_peak()
    achieved = ab["sweep"] / (kern_ms * 1e-3) / 1e9 if kern_n else None
    return {"bound": "hbm", "kernel": binding.last_main_kernel(), "achieved": achieved, "peak": peak, "unit": "GB/s",
            "frac": (achieved / peak) if achieved else None, "peak_source": f"of {which}",
            "frac_of_nominal_8000": (achieved / NOMINAL_HBM_GBS) if achieved else None,
            "kernel_ms": kern_ms, "launches_timed": kern_n, "algorithmic_bytes_per_launch": ab["sweep"],
            "traffic": kernel_traffic(wl.cfg.name)}


def block_facts(wl):
    """Mean number of fully accepted batch rows (they cost one more vocabulary row each) and block efficiency."""
    g = wl.cfg.gamma
    used = wl.outs[:min(wl.nsets, max(1, wl.count))]
    n_bonus = float(sum(int((o.accept_len == g).sum().item()) for o in used)) / len(used)
    be = float(sum(float((o.accept_len.float() + 1).mean().item()) for o in used)) / len(used)
    return n_bonus, be


def compare_verifiers(dev):
    """Verification cost of the four verifiers behind the boundary on the paper's operating points (K = 3 drafts of
    L = 12 or 8 tokens, T = 0.4, 32k vocabulary): one prompt and a batch of 64, microseconds per verify call and
    block efficiency.  The single-draft methods (token-level speculative sampling, GBV) see the first draft only."""
    import torch
    from paper_2604_25925_b200 import binding, workloads
    rows = []
    for name in ("paper_l12", "paper_l8"):
        for B in (1, 64):
            cfg = workloads.with_batch(workloads.CONFIGS[name], B)
            nsets = 8 if B == 1 else 4
            sets = [workloads.make_inputs(cfg, device=dev, set_index=500 + i) for i in range(nsets)]
            single = [(i.target_logits[:, 0].contiguous(), i.draft_logits[:, 0].contiguous(),
                       i.draft_tokens[:, 0].contiguous(), i.uniforms[:, :cfg.gamma + 1].contiguous()) for i in sets]
            T = cfg.temperature
            methods = {
                "spectr_gbv": lambda j: binding.sgbv_verify(sets[j].target_logits, sets[j].draft_logits,
                                                            sets[j].draft_tokens, sets[j].uniforms, T).accept_len,
                "spectr_kseq": lambda j: binding.sgbv_verify_kseq(sets[j].target_logits, sets[j].draft_logits,
                                                                  sets[j].draft_tokens, sets[j].uniforms, T).accept_len,
                "gbv_single_draft": lambda j: binding.sgbv_verify_gbv(*single[j], T).accept_len,
                "token_level_sd": lambda j: binding.sgbv_verify_token(*single[j], T).accept_len,
            }
            entry = {"workload": describe(cfg)}
            for mname, fn in methods.items():
                for j in range(nsets):
                    fn(j)
                torch.cuda.synchronize()
                reps = 40
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for r in range(reps):
                    fn(r % nsets)
                e1.record()
                torch.cuda.synchronize()
                be = float(sum(float((fn(j).float() + 1).mean().item()) for j in range(nsets))) / nsets
                entry[mname] = {"us_per_verify": 1e3 * e0.elapsed_time(e1) / reps, "block_efficiency": be}
            rows.append(entry)
            del sets, single
            torch.cuda.empty_cache()
    return rows


def vocab_sharded_leg(dev, n_ranks=8):
    """The vocabulary-sharded form of the step on C4's shape split over `n_ranks` ranges: one rank's four local
    phases timed on this device (every rank does the same amount of work; the three exchanges between the phases
    move the byte counts listed and are not timed here, there being one GPU)."""
    import torch
    from paper_2604_25925_b200 import binding, sharded, workloads
    cfg = workloads.get_config("c4")
    inp = workloads.make_inputs(cfg, device=dev, set_index=700)
    bounds = sharded.shard_bounds(cfg.V, n_ranks)
    shards = [(inp.target_logits[..., lo:hi].contiguous(), inp.draft_logits[..., lo:hi].contiguous(), lo)
              for lo, hi in bounds]
    one = binding.sgbv_verify(inp.target_logits, inp.draft_logits, inp.draft_tokens, inp.uniforms, cfg.temperature)
    tok, u, T = inp.draft_tokens, inp.uniforms, cfg.temperature
    del inp
    torch.cuda.empty_cache()
    outs = sharded.verify_all_ranks_on_one_device(shards, tok, u, T, cfg.V)
    torch.cuda.synchronize()
    agree = float((outs[0].accept_len == one.accept_len).float().mean().item())
    same_tokens = float((outs[0].tokens == one.tokens).all(dim=1).float().mean().item())
    stats_all = torch.stack([binding.sgbv_shard_stats(zq, zp, tok, vb, cfg.V, T) for zq, zp, vb in shards]).contiguous()
    zq, zp, vb = shards[0]
    ws = torch.empty(binding.sgbv_shard_workspace_bytes(cfg.B, cfg.K, cfg.gamma, zq.shape[-1]), dtype=torch.uint8, device=dev)
    wss = [torch.empty_like(ws) for _ in shards]
    sums_all = torch.stack([binding.sgbv_shard_sums(a, b, T, stats_all, wss[r]) for r, (a, b, _) in enumerate(shards)]).contiguous()
    phases = {
        "stats": lambda r: binding.sgbv_shard_stats(shards[r][0], shards[r][1], tok, shards[r][2], cfg.V, T),
        "sums": lambda r: binding.sgbv_shard_sums(shards[r][0], shards[r][1], T, stats_all, wss[r]),
        "decide": lambda r: binding.sgbv_shard_decide(tok, u, shards[r][0].shape[-1], T, stats_all, sums_all, wss[r]),
        "draw": lambda r: binding.sgbv_shard_draw(shards[r][0], shards[r][1], shards[r][2], T, r, wss[r], outs[r].tokens),
    }
    shard_bytes = sum(t.numel() * t.element_size() for t in (zq, zp))
    res = {}
    for name, fn in phases.items():
        for r in range(n_ranks):   # warm-up, and the rotation over the ranks' shards keeps the inputs out of L2
            fn(r)
        torch.cuda.synchronize()
        reps = 3 * n_ranks
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(reps):
            fn(i % n_ranks)
        e1.record()
        torch.cuda.synchronize()
        res[name + "_us"] = 1e3 * e0.elapsed_time(e1) / reps
    total_us = sum(res.values())
    res.update({
        "workload": describe(cfg) + f", vocabulary split over {n_ranks} ranks ({zq.shape[-1]} entries each)",
        "per_rank_us": total_us, "per_rank_shard_bytes": shard_bytes,
        "per_rank_gbs_over_both_sweeps": 2 * shard_bytes / (total_us * 1e-6) / 1e9,
        "exchange_bytes": {"stats_all_gather": stats_all.numel() * 4, "sums_all_gather": sums_all.numel() * 8,
                           "tokens_all_reduce": outs[0].tokens.numel() * 4},
        "agreement_with_one_device": {"accept_len": agree, "whole_rows": same_tokens},
        "note": "phases timed on one device over the ranks' shards in turn; exchanges not timed (one GPU)"})
    return res


PER_CONFIG = ("c2", "c3", "c5_K1_a0.8_T1.0", "c5_K8_a0.8_T1.0")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--sweep-c5", action="store_true",
                    help="instead of the default line: the 24 points of the B=256, gamma=4, V=32000 sweep, one JSON line")
    ap.add_argument("--vocab-sharded", action="store_true",
                    help="instead of the default line: one rank's phases of the vocabulary-sharded form, one JSON line")
    args = ap.parse_args()
    if args.impl == "reference":
        args.steps = args.steps or 3
        args.warmup = args.warmup if args.warmup is not None else 1
        run_reference(args)
        return

    import torch
    import torch.distributed as dist
    from paper_2604_25925_b200 import binding, workloads

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the verify path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    if args.vocab_sharded:
        if world > 1:
            raise RuntimeError("--vocab-sharded times one rank's phases on one GPU")
        print(json.dumps({"metric": "verify_steps_per_s", "n_gpus": 1, "data": "synthetic",
                          "vocab_sharded": vocab_sharded_leg(dev)}))
        return

    if args.sweep_c5:
        if world > 1:
            raise RuntimeError("--sweep-c5 runs on one GPU")
        points = []
        for c in workloads.sweep_c5():
            w = Workload(c, dev, rank)
            c_steps = int(max(20, min(2000, 50.0 / max(0.02, c.logit_bytes() / 4.0e9))))
            bl, _, _ = timed_blocks(w, c_steps, max(3, c_steps // 4), 1, min_seconds=0.3)
            k_ms, k_n = kernel_pass(w, max(20, min(c_steps, 100)))
            nb, c_be = block_facts(w)
            c_ab = algorithmic_bytes(c, nb)
            msb = sorted(bl)[len(bl) // 2]
            r = roofline_of(w, c_ab, k_ms, k_n)
            points.append({"workload": describe(c), "K": c.K, "alpha": c.alpha, "temperature": c.temperature,
                           "value": c_steps / (msb * 1e-3), "ms_per_step": msb / c_steps, "block_efficiency": c_be,
                           "hbm_gbs_step": c_ab["step"] / (msb / c_steps * 1e-3) / 1e9, "kernel_gbs": r["achieved"],
                           "frac": r["frac"], "launches_timed": k_n})
            del w
            torch.cuda.empty_cache()
        print(json.dumps({"metric": "verify_steps_per_s", "unit": "verify-steps/s", "n_gpus": 1, "data": "synthetic",
                          "config": {"workload": "c5 sweep: B=256, gamma=4, V=32000, fp32, K x alpha x temperature"},
                          "points": points}))
        return

    cfg = workloads.get_config(args.workload)
    est_ms = max(0.02, cfg.logit_bytes() / 4.0e9)             # rough step time for choosing defaults
    steps = args.steps if args.steps is not None else int(max(20, min(2000, 50.0 / est_ms)))
    warmup = max(3, args.warmup if args.warmup is not None else min(50, steps // 4))

    wl = Workload(cfg, dev, rank)
    uuid = None
    try:
        uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid)
    except Exception:
        pass
    sampler = ClockSampler(uuid) if rank == 0 else None
    time.sleep(0.25)
    # the warm-up steps run right before the timed ones (the sampler's start-up pause would let the GPU idle)
    blocks, (t0, t1), launches_per_step = timed_blocks(wl, steps, warmup, world)
    clocks = sampler.stop(t0, t1) if sampler else None
    kern_ms, kern_n = kernel_pass(wl, max(20, min(steps, 200)))
    n_bonus, be = block_facts(wl)

    if rank == 0:
        ab = algorithmic_bytes(cfg, n_bonus)
        ms_block = sorted(blocks)[len(blocks) // 2]           # the median block
        ms_step = ms_block / steps
        line = {
            "metric": "verify_steps_per_s", "value": world * steps / (ms_block * 1e-3), "unit": "verify-steps/s",
            "n_gpus": world, "steps": steps, "warmup": warmup, "repeats": len(blocks), "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": config_dict(cfg, wl.nsets, cfg.logit_bytes()),
            "hbm_gbs_step": ab["step"] / (ms_step * 1e-3) / 1e9,
            "algorithmic_bytes_per_step": ab["step"],
            "block_efficiency": be,
            "roofline": roofline_of(wl, ab, kern_ms, kern_n),
            "gpu_launches": launches_per_step * steps,
            "clocks": clocks,
        }
        if not args.no_e2e:
            host = wl.sets[0].to("cpu")
            pinned = [t.pin_memory() for t in (host.target_logits, host.draft_logits, host.draft_tokens,
                                               host.uniforms)]
            hout = binding.VerifyOutput(torch.empty(cfg.B, dtype=torch.int32).pin_memory(),
                                        torch.empty(cfg.B, dtype=torch.int32).pin_memory(),
                                        torch.empty((cfg.B, cfg.gamma + 1), dtype=torch.int32).pin_memory(),
                                        status=torch.empty(cfg.B, dtype=torch.int32).pin_memory())
            e_steps = int(max(3, min(steps, 2.0 / max(cfg.logit_bytes() / 20e9, 1e-4))))
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
            del pinned, host
        if not args.no_cpu_baseline:
            line["parity"], line["cpu_baseline"] = parity_report(wl, 12.0)
        del wl
        torch.cuda.empty_cache()
        # the other configurations the metric is quoted on, measured the same way (one GPU, shorter)
        if world == 1 and not args.no_per_config:
            per = []
            for name in PER_CONFIG:
                if name == cfg.name:
                    continue
                c = workloads.get_config(name)
                w = Workload(c, dev, rank)
                c_steps = int(max(20, min(2000, 50.0 / max(0.02, c.logit_bytes() / 4.0e9))))
                bl, _, _ = timed_blocks(w, c_steps, max(3, c_steps // 4), 1, min_seconds=0.5)
                k_ms, k_n = kernel_pass(w, max(20, min(c_steps, 200)))
                nb, c_be = block_facts(w)
                c_ab = algorithmic_bytes(c, nb)
                msb = sorted(bl)[len(bl) // 2]
                entry = {"workload": describe(c), "value": c_steps / (msb * 1e-3), "ms_per_step": msb / c_steps,
                         "steps": c_steps, "repeats": len(bl), "block_efficiency": c_be,
                         "roofline": roofline_of(w, c_ab, k_ms, k_n)}
                if not args.no_cpu_baseline:
                    entry["parity"], _ = parity_report(w, 2.0)
                per.append(entry)
                del w
                torch.cuda.empty_cache()
            line["per_config"] = per
            line["verifier_comparison"] = compare_verifiers(dev)
            line["vocab_sharded"] = vocab_sharded_leg(dev)
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
