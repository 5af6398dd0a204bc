#!/usr/bin/env python
"""Suffix-rollout benchmark: one step = prefill of the cached prefixes (once per group) plus
batched decode of G suffixes per group over the shared prefix KV, on seeded synthetic inputs.

    python bench.py --gpus 1 --steps 5 --warmup 3            # this library, config 2
    python bench.py --impl reference --steps 2 --warmup 1    # the CPU oracle on a bounded sample

Prints ONE JSON line (rank 0).  value = suffix tokens/s over all ranks with inputs resident in
HBM; e2e = the same through rpo_rollout_host with pinned host buffers.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
import workloads  # noqa: E402

METRIC = "suffix_rollout_tokens_per_sec"
UNIT = "tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"], bf16_sustained=d.get("bf16_tflops_sustained"),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_sustained=1400.0, source="fallback")


def ncu_traffic_per_launch():
    """DRAM bytes per launch of the decode GEMM from the committed ncu capture, or None once the
    kernel source has changed since the counters were taken."""
    import hashlib
    prof = os.path.join(ROOT, "profiles", "decode_step_kernels_cfg2_reduced.txt")
    try:
        vals = dict(l.split(" = ") for l in open(prof).read().splitlines() if " = " in l)
        h = hashlib.sha256()
        for name in ("gemm_tc.cuh", "gemm_tc2.cuh"):
            h.update(open(os.path.join(ROOT, "paper_2601_19404_b200", "csrc", name), "rb").read())
        if vals["gemm_sources_sha256"].strip() != h.hexdigest():
            return None
        return float(vals["gemm_decode_traffic_bytes_per_launch"])
    except Exception:
        return None


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "200",
                                       "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush(); self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        self.f.close(); os.unlink(self.f.name)
        if sm:
            out = dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def algorithmic_decode_bytes(shape, lens, G, S):
    """Bytes one decode step must move: all layer matrices + lm_head once, each group's prefix K/V
    once per group, each sequence's own suffix K/V (mean over the S-1 forward steps)."""
    e = 2 if shape["dtype"] == "bf16" else 4
    d, dh, hq, hkv, F, V, L = (shape[k] for k in ("d_model", "head_dim", "n_q_heads", "n_kv_heads", "d_ffn", "vocab", "n_layers"))
    layer = (hq + 2 * hkv) * dh * d + d * hq * dh + 3 * F * d
    weights = (L * layer + V * d) * e
    kv_tok = 2 * L * hkv * dh * e
    prefix = int(np.sum(lens)) * kv_tok
    suffix = len(lens) * G * (S / 2.0) * kv_tok
    return dict(weights=weights, prefix_kv=prefix, suffix_kv=suffix, total=weights + prefix + suffix)


def prefill_flops(shape, lens):
    d, dh, hq, hkv, F, L = (shape[k] for k in ("d_model", "head_dim", "n_q_heads", "n_kv_heads", "d_ffn", "n_layers"))
    layer = (hq + 2 * hkv) * dh * d + d * hq * dh + 3 * F * d
    T = float(np.sum(lens))
    attn = sum(2 * 2 * (float(p) * p / 2) * dh * hq * L for p in lens)
    return 2 * layer * L * T + attn


def run_reference(args, cfg_name, rank, world):
    """The CPU oracle, as it stands, on a bounded sample of the workload (rank 0 only)."""
    if rank != 0:
        return
    import torch
    from oracle import init as oinit, rollout as orollout, decoder as odecoder
    cfg = workloads.CONFIGS[cfg_name]
    shape = workloads.SHAPES[cfg["shape"]]
    sh = odecoder.Shape(**{k: shape[k] for k in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn",
                                                  "vocab", "rope_base", "rms_eps", "dtype")})
    G = cfg["G"]
    P, S = args.ref_prefix, args.ref_suffix
    w = oinit.init_weights(sh, seed=0, std=0.02)
    toks, off = workloads.prefix_tokens(np.array([P], dtype=np.int32), sh.vocab, seed=0)
    sc = cfg["sampler"]
    ocfg = orollout.SamplerCfg(sc["temperature"], sc["top_p"], sc["greedy"], 0, sc["eos_id"])
    times = []
    for it in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        out = orollout.rollout_group(w, sh, toks, G, S, ocfg, group_id=it, dt=np.float32)
        dt = time.perf_counter() - t0
        if it >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = G * S / (ms / 1e3)
    cores = torch.get_num_threads()
    sample = f"1 group x G={G}, prefix {P} of the config's tokens, {S} suffix tokens, full depth, float32 numpy"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": {"workload": cfg_name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def cpu_baseline(cfg_name, prefix, suffix):
    import torch
    from oracle import init as oinit, rollout as orollout, decoder as odecoder
    cfg = workloads.CONFIGS[cfg_name]
    shape = workloads.SHAPES[cfg["shape"]]
    sh = odecoder.Shape(**{k: shape[k] for k in ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn",
                                                  "vocab", "rope_base", "rms_eps", "dtype")})
    G = cfg["G"]
    w = oinit.init_weights(sh, seed=0, std=0.02)
    toks, _ = workloads.prefix_tokens(np.array([prefix], dtype=np.int32), sh.vocab, seed=0)
    sc = cfg["sampler"]
    t0 = time.perf_counter()
    orollout.rollout_group(w, sh, toks, G, suffix, orollout.SamplerCfg(sc["temperature"], sc["top_p"], sc["greedy"], 0, sc["eos_id"]),
                           dt=np.float32)
    dt = time.perf_counter() - t0
    return {"value": G * suffix / dt, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
            "sample": f"1 group x G={G}, prefix {prefix}, {suffix} suffix tokens, full depth, float32 numpy, {dt:.1f} s"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg2_1p5b_16x8")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-profile", action="store_true")
    ap.add_argument("--chunk", type=int, default=0, help="prefill chunk in tokens (0: 16384, or the longest prefix if longer)")
    ap.add_argument("--ref-prefix", type=int, default=1024)
    ap.add_argument("--ref-suffix", type=int, default=8)
    ap.add_argument("--options", default="", help="comma list name=value passed to rpo_set_option")
    ap.add_argument("--layers", type=int, default=0, help="override n_layers (reduced case for profiler captures)")
    ap.add_argument("--suffix", type=int, default=0, help="override the suffix length (reduced case for profiler captures)")
    ap.add_argument("--groups", type=int, default=0, help="override the number of prompt groups (reduced case)")
    ap.add_argument("--kernel-table", action="store_true", help="print per-kernel event timings of one profiled step on stderr")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, args.config, rank, world)
        return

    import torch
    import torch.distributed as dist
    import paper_2601_19404_b200 as rpo
    from paper_2601_19404_b200 import binding

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    cfg = dict(workloads.CONFIGS[args.config])
    shape = dict(workloads.SHAPES[cfg["shape"]])
    reduced = []
    if args.layers:
        shape["n_layers"] = args.layers; reduced.append(f"layers={args.layers}")
    if args.suffix:
        cfg["suffix"] = args.suffix; reduced.append(f"suffix={args.suffix}")
    if args.groups:
        cfg["n_groups"] = args.groups; reduced.append(f"groups={args.groups}")
    n_g, G, S = cfg["n_groups"], cfg["G"], cfg["suffix"]
    B = n_g * G
    lens = workloads.prefix_lengths(cfg, seed=rank)
    toks, off = workloads.prefix_tokens(lens, shape["vocab"], seed=rank)
    group_ids = workloads.rank_group_ids(n_g, rank)                  # weak scaling: every rank its own groups
    sc = cfg["sampler"]
    smp = rpo.Sampler(sc["temperature"], sc["top_p"], sc["greedy"], sc["eos_id"], seed=0)
    want_lp = bool(cfg.get("logprobs"))

    blocks = int(np.sum(-(-lens // 16))) + B * (-(-S // 16)) + 64
    chunk = args.chunk if args.chunk > 0 else int(min(max(int(lens.max()), 16384), 32768))
    stream = torch.cuda.Stream(device=dev)
    ctx = rpo.Context(binding.shape_from_dict(shape), blocks, max_groups=n_g, max_seqs=B, max_chunk_tokens=chunk,
                      max_positions=int(lens.max()) + S + 1, stream=stream)
    for kv in filter(None, args.options.split(",")):
        k, v = kv.split("=")
        ctx.set_option(k, int(v))
    ctx.init_weights(seed=0, std=0.02)

    d_toks = torch.from_numpy(toks).to(dev)
    d_out = torch.zeros((B, S), dtype=torch.int32, device=dev)
    d_lens = torch.zeros(B, dtype=torch.int32, device=dev)
    d_lp = torch.zeros((B, S), dtype=torch.float32, device=dev)
    d_pol = torch.zeros((B, S), dtype=torch.float32, device=dev)

    def step(timers=None):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        ev[0].record(stream)
        groups = ctx.prefill_prefix(d_toks, off, group_ids)
        ev[1].record(stream)
        ctx.decode_suffix(groups, G, S, smp, d_out, d_lens, d_lp)
        ev[2].record(stream)
        if want_lp:
            ctx.token_logprobs(groups, G, S, d_out, d_lens, d_pol, inv_temperature=1.0 / sc["temperature"])
        ev[3].record(stream)
        ctx.release_groups(groups)
        if timers is not None:
            timers.append(ev)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    launches0 = ctx.counters()[0]
    clocks = ClockSampler(local_rank)
    timers = []
    t_begin = torch.cuda.Event(enable_timing=True); t_end = torch.cuda.Event(enable_timing=True)
    t_begin.record(stream)
    for _ in range(args.steps):
        step(timers)
    t_end.record(stream)
    barrier()
    clk = clocks.stop()
    total_ms = t_begin.elapsed_time(t_end)
    launches = ctx.counters()[0] - launches0
    emitted = int(d_lens.sum().item())
    pre_ms = float(np.mean([e[0].elapsed_time(e[1]) for e in timers]))
    dec_ms = float(np.mean([e[1].elapsed_time(e[2]) for e in timers]))
    lp_ms = float(np.mean([e[2].elapsed_time(e[3]) for e in timers]))
    if world > 1:
        t = torch.tensor([total_ms, pre_ms, dec_ms, lp_ms], device=dev, dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        total_ms, pre_ms, dec_ms, lp_ms = t.tolist()
        em = torch.tensor([emitted], device=dev, dtype=torch.int64)
        dist.all_reduce(em, op=dist.ReduceOp.SUM)
        emitted_all = int(em.item())
    else:
        emitted_all = emitted
    ms_per_step = total_ms / args.steps
    value = emitted_all / (ms_per_step / 1e3)

    # ---- end to end through the host-buffer call (pinned host memory, copies inside the timed region)
    e2e = None
    if not args.no_e2e:
        h_toks = torch.from_numpy(toks).pin_memory()
        h_out = torch.zeros((B, S), dtype=torch.int32).pin_memory()
        h_lens = torch.zeros(B, dtype=torch.int32).pin_memory()
        h_lp = torch.zeros((B, S), dtype=torch.float32).pin_memory()
        h_pol = torch.zeros((B, S), dtype=torch.float32).pin_memory() if want_lp else None

        def e2e_step():
            ctx.rollout_host(h_toks.numpy(), off, G, S, smp, h_out.numpy(), h_lens.numpy(), h_lp.numpy(),
                             None if h_pol is None else h_pol.numpy(), group_ids=group_ids)

        e2e_step()
        barrier()
        e_begin = torch.cuda.Event(enable_timing=True); e_end = torch.cuda.Event(enable_timing=True)
        n_e2e = max(1, min(args.steps, 3))
        e_begin.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        e_end.record(stream)
        barrier()
        e2e_ms = e_begin.elapsed_time(e_end) / n_e2e
        e2e_tokens = int(h_lens.sum().item())
        if world > 1:
            t = torch.tensor([e2e_ms], device=dev, dtype=torch.float64); dist.all_reduce(t, op=dist.ReduceOp.MAX); e2e_ms = t.item()
            em = torch.tensor([e2e_tokens], device=dev, dtype=torch.int64); dist.all_reduce(em, op=dist.ReduceOp.SUM); e2e_tokens = int(em.item())
        h2d = int(toks.nbytes)
        d2h = int(h_out.numel() * 4 + h_lens.numel() * 4 + h_lp.numel() * 4 + (h_pol.numel() * 4 if want_lp else 0))
        e2e = {"value": e2e_tokens / (e2e_ms / 1e3), "unit": UNIT, "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h}

    # ---- roofline: per-kernel event timing in one extra profiled step (graphs off, same kernels)
    peaks = measured_peaks()
    ab = algorithmic_decode_bytes(shape, lens, G, S)
    dec_step_ms = dec_ms / max(S - 1, 1)
    roofline = None
    phases = None
    if not args.no_profile and rank == 0:
        ctx.set_option("profile", 2 if args.kernel_table else 1)
        step()
        prof = ctx.profile_read()
        ctx.set_option("profile", 0)
        phases = {p: {k: {"ms": round(v[0], 3), "launches": v[1]} for k, v in d.items() if v[1]} for p, d in prof.items()}
        gemm_ms, gemm_n = prof["decode"]["gemm"]
        # Dominant kernel of the path: the weight-streaming tensor-core GEMM of the decode step (all
        # layer matrices + lm_head once per step).  Algorithmic bytes per launch = weight bytes a step
        # reads / GEMM launches per step; duration = mean of CUDA-event pairs bracketing every launch
        # of the profiled step (bracketing adds a few microseconds per launch: the fraction is a floor).
        if gemm_n:
            per_launch_bytes = ab["weights"] * (S - 1) / gemm_n
            achieved = per_launch_bytes / (gemm_ms / gemm_n * 1e-3) / 1e9
            esz = 2 if shape["dtype"] == "bf16" else 4
            roofline = {"bound": "hbm", "kernel": "gemm_tc_kernel / gemm_tc2_kernel (decode weight GEMMs)", "achieved": achieved,
                        "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                        "traffic": ncu_traffic_per_launch() if (not reduced and args.config.startswith("cfg2")) else None,
                        "tensor_tflops": 2.0 * B * (ab["weights"] / esz) * (S - 1) / (gemm_ms * 1e-3) / 1e12,
                        "algorithmic_bytes_per_launch": per_launch_bytes, "launches_per_step": gemm_n / max(S - 1, 1),
                        "peak_source": peaks["source"] + " copy bandwidth (MEASURED_PEAKS.json)" if peaks["source"] == "measured" else "fallback",
                        "ms_per_launch": gemm_ms / gemm_n}
    decode_gbs = ab["total"] / (dec_step_ms * 1e-3) / 1e9
    pf = prefill_flops(shape, lens)
    prefill_tfs = pf / (pre_ms * 1e-3) / 1e12

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if shape["dtype"] == "bf16" else "f32", "data": "synthetic",
        "config": {"workload": args.config + ("" if not reduced else " REDUCED(" + ",".join(reduced) + ")"), "shape": cfg["shape"], "n_groups": n_g, "G": G, "prefix_tokens": int(lens.sum()),
                   "suffix": S, "l2": "inputs larger than L2 (weights %.2f GB + KV)" % (ab["weights"] / 1e9),
                   "parallelism": f"groups sharded over {world} rank(s), no collective in the step"},
        "phases_ms": {"prefill": pre_ms, "decode": dec_ms, "logprobs": lp_ms, "decode_per_step": dec_step_ms},
        "decode_hbm": {"algorithmic_bytes_per_step": ab, "achieved_gbs": decode_gbs, "frac_of_measured": decode_gbs / peaks["hbm_gbs"],
                       "frac_of_8tbs": decode_gbs / 8000.0},
        "prefill_tensor": {"flops": pf, "achieved_tflops": prefill_tfs, "frac_of_measured_burst": prefill_tfs / peaks["bf16_tflops"],
                           "frac_of_2250": prefill_tfs / 2250.0},
        "roofline": roofline, "kernel_classes": phases,
        "e2e": e2e,
        "gpu_launches": int(launches), "clocks": clk, "device_status": ctx.device_status(),
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(args.config, args.ref_prefix, args.ref_suffix)
    if rank == 0:
        print(json.dumps(out))
    ctx.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
