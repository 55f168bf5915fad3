#!/usr/bin/env python
"""Benchmark of the QZO hot path: whole optimisation steps (two perturbed forwards + seeded
scale update) on a synthetic int4 Llama-2-7B-shaped model, one B200 per rank.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

Prints ONE JSON line (rank 0).  `value` is steps/s with tokens already resident on the device;
`e2e` is the same step through the host-buffer entry point (token upload and loss read-back
inside the timed region).  `--impl reference` times the CPU oracle on a bounded sample.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

# ncu capture of the dominant kernel on the 4096 x 11008, M = 4096 sweep launch (tracked summary); the
# benchmark reads the DRAM bytes from it.  Remove or rename the file when the kernel changes: `traffic`
# is then null until the capture is retaken.
NCU_PROFILE = os.path.join(ROOT, "profiles", "w4a16_gemm_K4096_N11008_M4096.txt")
NCU_PROFILE_ALGORITHMIC_BYTES = 4096 * 11008 // 2 + 2 * 32 * 11008 + 2 * 4096 * 4096 + 2 * 4096 * 11008
NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 8000.0, 2250.0


def ncu_traffic_ratio():
    """(DRAM bytes read + written) / algorithmic bytes of the captured launch, from the tracked ncu summary."""
    try:
        vals = {}
        for line in open(NCU_PROFILE):
            for key in ("dram__bytes_read.sum ", "dram__bytes_write.sum "):
                if line.startswith(key) and "[Mbyte]" in line:
                    nums = [float(v) for v in line.split("]")[1].split(";")]
                    vals[key.strip()] = sum(nums) / len(nums) * 1e6
        if len(vals) == 2:
            return sum(vals.values()) / NCU_PROFILE_ALGORITHMIC_BYTES
    except (OSError, ValueError):
        pass
    return None


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.file.name)
        if sm:
            sm.sort()
            out = {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm)}
        return out


def oracle_sample(workload, n_seq=2):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: the forward of a model
    truncated to ONE decoder block (embedding, the block, final norm, full lm_head and cross entropy) and
    of the same model with NO block, on n_seq sequences; a whole step is then
    (n_layers x (one-block time - no-block time) + no-block time) x 2 signs x (batch / n_seq).
    Returns (steps_per_s, cores, description)."""
    import numpy as np
    import torch
    from oracle import int4, model as omodel
    from paper_2505_13430_b200 import inputs
    c = inputs.CONFIGS[workload]
    cfg = inputs.model_cfg(workload, n_layers=1)
    raw = inputs.raw_model_tensors(cfg, seed=1000)
    m = {"cfg": dict(cfg), "embed": raw["embed"].float().numpy(), "lm_head": raw["lm_head"].float().numpy(),
         "final_norm_w": raw["final_norm_w"].numpy()}
    if "pos_embed" in raw:
        m["pos_embed"] = raw["pos_embed"].float().numpy()
        m["final_norm_b"] = raw["final_norm_b"].numpy()
    layer = {k: v.float().numpy() for k, v in raw["layers"][0].items() if k != "lin"}
    layer["lin"] = {}
    for name, ent in raw["layers"][0]["lin"].items():
        q, s = int4.quantize_int4(ent["w"].numpy())
        layer["lin"][name] = {"q": q, "s": s}
        if "bias" in ent:
            layer["lin"][name]["bias"] = ent["bias"].numpy()
    m["layers"] = [layer]
    del raw
    n_seq = min(n_seq, c["batch"])
    tok, lab = inputs.tokens_and_labels(cfg, n_seq, c["seq"], seed=7)
    signs = (+1, -1) if n_seq > 1 else (+1,)
    head_only = dict(m, cfg=dict(cfg, n_layers=0), layers=[])
    t0 = time.perf_counter()
    for sign in signs:
        omodel.forward_loss(m, tok.numpy(), lab.numpy(), 42, sign, c["eps"])
    t_one = time.perf_counter() - t0
    t0 = time.perf_counter()
    for sign in signs:
        omodel.forward_loss(head_only, tok.numpy(), lab.numpy(), 42, sign, c["eps"])
    t_head = time.perf_counter() - t0
    t_block = max(t_one - t_head, 0.0)
    step_s = (t_block * c["n_layers"] + t_head) * (2 / len(signs)) * (c["batch"] / n_seq)
    cores = torch.get_num_threads()
    desc = (f"oracle forward on {n_seq} of {c['batch']} sequences (S={c['seq']}), {len(signs)} of 2 signs: one decoder block "
            f"{t_block:.2f} s, embedding + final norm + full lm_head + cross entropy {t_head:.2f} s; whole step = "
            f"({c['n_layers']} x block + head) x {2 // len(signs)} x {c['batch'] // n_seq}, extrapolated linearly")
    return 1.0 / step_s, cores, desc


def gemm_sweep_rows(inputs, peaks):
    """The second half of the metric: the standalone perturbed GEMM on the Llama-2-7B linears' K x N at every
    token count of the sweep (each shape alone after an idle second, median of nine passes of about
    4 ms, operands rotated through more than the L2 capacity), as fractions of
    max(bytes / HBM, flops / dense bf16) against the measured and against the nominal peaks."""
    from paper_2505_13430_b200 import gemm_sweep
    rows = []
    for K, N in ((4096, 4096), (4096, 11008), (11008, 4096)):
        for M in inputs.GEMM_SWEEP_M:
            us, best_us, n_sets = gemm_sweep.run_shape(M, K, N, 50, settle=0.5)
            nbytes, flops = gemm_sweep.gemm_bytes(M, K, N), 2.0 * M * K * N
            roof = max(nbytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)) * 1e6
            roof_nom = max(nbytes / (NOMINAL_HBM_GBS * 1e9), flops / (NOMINAL_BF16_TFLOPS * 1e12)) * 1e6
            rows.append({"K": K, "N": N, "M": M, "us": round(us, 2), "best_pass_us": round(best_us, 2),
                         "bound": "hbm" if nbytes / (peaks["hbm_gbs"] * 1e9) > flops / (peaks["bf16_tflops"] * 1e12) else "tensor",
                         "frac": round(roof / us, 4), "frac_of_nominal": round(roof_nom / us, 4)})
    return {"rows": rows, "min_frac": min(r["frac"] for r in rows), "min_frac_of_nominal": min(r["frac_of_nominal"] for r in rows),
            "peaks": {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops": peaks["bf16_tflops"], "source": peaks["source"],
                      "nominal_hbm_gbs": NOMINAL_HBM_GBS, "nominal_bf16_tflops": NOMINAL_BF16_TFLOPS},
            "method": "qzo_perturbed_gemm through the C ABI, CUDA-graph replays timed with CUDA events, median pass"}


def run_reference(args, workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    cores, desc = 0, ""
    for i in range(args.warmup + args.steps):
        v, cores, desc = oracle_sample(workload, n_seq=1)
        if i >= args.warmup:
            vals.append(v)
    value = sum(vals) / len(vals)
    c = bench_config(workload, args.gpus)
    line = {"impl": "reference", "metric": "qzo_steps_per_s", "value": value, "unit": "steps/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1000.0 / value, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": c,
            "cpu_baseline": {"value": value, "unit": "steps/s", "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": "steps/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def bench_config(workload, n_gpus):
    from paper_2505_13430_b200 import inputs
    c = inputs.CONFIGS[workload]
    return {"workload": f"{workload}: {c['arch']}-shaped random-init int4 model, {c['n_layers']} layers, d={c['d_model']}, "
                        f"{c['n_heads']} heads, FFN {c['d_ffn']}, vocab {c['vocab']}, group-128 bf16 scales; full QZO step "
                        f"(2 perturbed forwards + seeded scale update)",
            "batch_per_gpu": c["batch"], "seq_len": c["seq"], "eps": c["eps"], "lr": c["lr"], "clip": c["clip"],
            "parallelism": f"{n_gpus} independent replica(s), no collective",
            "l2": "inputs larger than L2: every step streams 3.3 GB+ of int4 weights"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="llama7b")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the standalone GEMM rows (roofline.sweep)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    workload = args.workload

    if args.impl == "reference":
        run_reference(args, workload)
        return

    import torch
    import torch.distributed as dist
    from paper_2505_13430_b200 import inputs, qzo, replicas

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    c = inputs.CONFIGS[workload]
    cfg = inputs.model_cfg(workload)
    B, S = c["batch"], c["seq"]
    model_seed, token_seed = replicas.rank_seeds(1000, 7, rank)
    model = qzo.build_random_model_gpu(cfg, B * S, seed=model_seed)
    tok, lab = inputs.tokens_and_labels(cfg, B, S, seed=token_seed)
    tok_pin, lab_pin = tok.contiguous().pin_memory(), lab.contiguous().pin_memory()
    tok_d, lab_d = tok.cuda(), lab.cuda()
    n_gemm = cfg["n_layers"] * len(inputs.linear_shapes(cfg)) * 2
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record(stream)
        for t in range(steps):
            fn(t)
        ev1.record(stream)
        barrier()
        return replicas.max_over_ranks(ev0.elapsed_time(ev1), device="cuda")

    seed0 = 42
    for t in range(args.warmup):
        model.qzo_step(tok_d, lab_d, seed0 + t, c["eps"], c["lr"], c["clip"], read_back=False)
        if t == 0 and model.qzo_device_status() != 0:
            raise SystemExit("device status word set in the first step: a bounded wait expired")
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    launches0 = qzo.qzo_launch_count()
    ms = timed(lambda t: model.qzo_step(tok_d, lab_d, seed0 + 100 + t, c["eps"], c["lr"], c["clip"], read_back=False),
               args.steps)
    launches = qzo.qzo_launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    # second pass of the same length with every perturbed-GEMM launch bracketed by CUDA events on the
    # model's stream: the dominant kernel's launch durations (the brackets cost a little, so `value`
    # comes from the pass above, without them)
    model.qzo_profile_gemms(n_gemm * args.steps)
    ms_bracketed = timed(lambda t: model.qzo_step(tok_d, lab_d, seed0 + 300 + t, c["eps"], c["lr"], c["clip"],
                                                  read_back=False), args.steps)
    n_l, gemm_ms, gemm_flops = model.qzo_profile_read()
    model.qzo_profile_gemms(0)
    status = model.qzo_device_status()
    if status != 0:
        raise SystemExit("device status word set: a bounded wait expired during the benchmark")

    # end to end: host (pinned) tokens in, losses out, every step
    for t in range(2):
        model.qzo_step_host(tok_pin, lab_pin, seed0 + t, c["eps"], c["lr"], c["clip"])
    e2e_ms = timed(lambda t: model.qzo_step_host(tok_pin, lab_pin, seed0 + 200 + t, c["eps"], c["lr"], c["clip"]),
                   args.steps)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # DRAM traffic of the dominant kernel: measured once with ncu on the 4096 x 11008, M = 4096 sweep
    # launch (tracked summary under profiles/) and scaled to this step's mean launch by algorithmic bytes.
    def gemm_bytes(M, K, N):
        return K * N // 2 + 2 * ((K + 127) // 128) * N + 2 * M * K + 2 * M * N
    shapes = inputs.linear_shapes(cfg)
    T = B * S
    launches_per_layer = 4 if cfg["arch"] == "llama" else 4          # qkv, o, (gate+up | fc1), (down | fc2)
    # a step runs its two passes as one forward over both copies of the batch when the token count
    # allows it: then a launch covers 2 T rows (seen from the number of profiled launches)
    passes_per_launch = 2 if n_l <= launches_per_layer * cfg["n_layers"] * args.steps else 1
    mean_bytes = sum(gemm_bytes(passes_per_launch * T, K, N) for _, K, N in shapes) / launches_per_layer
    ratio = ncu_traffic_ratio()
    traffic = ratio * mean_bytes if ratio else None
    peaks = measured_peaks()
    value = replicas.whole_job_rate(args.steps, world, ms)
    e2e = replicas.whole_job_rate(args.steps, world, e2e_ms)
    achieved = gemm_flops / (gemm_ms / 1000.0) / 1e12 if gemm_ms > 0 else 0.0
    # the roofline of a launch is the slower of its bytes over HBM and its flops over the dense bf16 peak
    mean_flops = gemm_flops / n_l if n_l else 0.0
    t_hbm = mean_bytes / (peaks["hbm_gbs"] * 1e9)
    t_mma = mean_flops / (peaks["bf16_tflops"] * 1e12)
    bound = "hbm" if t_hbm > t_mma else "tensor"
    peak = peaks["bf16_tflops"]
    sweep = None if args.no_sweep else gemm_sweep_rows(inputs, peaks)
    line = {"metric": "qzo_steps_per_s", "value": value, "unit": "steps/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic", "config": bench_config(workload, world),
            "clocks": clocks,
            "e2e": {"value": e2e, "unit": "steps/s", "h2d_bytes_per_step": 2 * B * S * 4, "d2h_bytes_per_step": 16},
            "gpu_launches": int(launches),
            "roofline": {"kernel": "w4a16_gemm_kernel (perturbed W4A16 GEMM, all block linears)", "bound": bound,
                         "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                         "peak_source": f"{peaks['source']} dense bf16 (burst, MEASURED_PEAKS.json bf16_tflops)",
                         "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"],
                         "sustained_peak": peaks["bf16_tflops_sustained"],
                         "frac_of_nominal_peak": achieved / NOMINAL_BF16_TFLOPS,
                         "traffic": traffic,
                         "traffic_source": "profiles/w4a16_gemm_K4096_N11008_M4096.txt (one ncu capture of the sweep "
                                           "launch, scaled to this step's mean launch by algorithmic bytes; not measured in this run)",
                         "algorithmic_bytes_per_launch": mean_bytes, "algorithmic_flops_per_launch": mean_flops,
                         "launches": int(n_l), "gemm_share_of_step": gemm_ms / ms_bracketed if ms_bracketed > 0 else None,
                         "ms_per_step_with_event_brackets": ms_bracketed / args.steps,
                         "sweep": sweep}}
    if not args.no_cpu_baseline:
        v, cores, desc = oracle_sample(workload, n_seq=16)
        line["cpu_baseline"] = {"value": v, "unit": "steps/s", "cores": cores, "kind": "oracle", "sample": desc}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
