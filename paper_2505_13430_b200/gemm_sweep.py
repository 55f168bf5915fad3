"""Standalone perturbed W4A16 GEMM sweep (K x N and token counts of the paper-shaped linears).

    python -m paper_2505_13430_b200.gemm_sweep [--shapes KxN,...] [--tokens M,...] [--iters I] [--json]

For every shape it times qzo_perturbed_gemm with CUDA events around replays of a CUDA graph that
holds up to `iters` launches (a pass of about 4 ms, at least one launch per set), rotating through
enough distinct weight / scale / activation sets that every launch streams its operands from HBM
(the rotation exceeds the L2 capacity).  Every shape is timed alone after an idle second, nine
passes one by one; the median pass gives the achieved fraction of the roofline
max(bytes / HBM bandwidth, flops / dense bf16 peak) with
bytes = K N / 2 + 2 ceil(K/128) N + 2 M K + 2 M N and flops = 2 M K N, against the burst peaks
(measured the same way: short runs of one kernel); the best pass is printed beside it.
"""
import argparse
import time
import json
import os

import torch

from . import inputs, qzo

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
L2_BYTES = 126 * 2 ** 20
NOMINAL_HBM_GBS, NOMINAL_BF16_TFLOPS = 8000.0, 2250.0      # datasheet figures, for the second column


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return p["hbm_gbs"], p["bf16_tflops"], "measured"
    return 6650.0, 1590.0, "fallback"


def gemm_bytes(M, K, N):
    return K * N // 2 + 2 * ((K + 127) // 128) * N + 2 * M * K + 2 * M * N


def run_shape(M, K, N, iters, sign=1, reps=9, settle=1.0, pass_ms=4.0, table16=False):
    per_set = gemm_bytes(M, K, N)
    n_sets = max(2, min(64, (2 * L2_BYTES) // per_set + 1))
    sets = []
    for i in range(n_sets):
        x = torch.randn((M, K), device="cuda", dtype=torch.float32).bfloat16()
        words = torch.randint(-2 ** 31, 2 ** 31 - 1, (K // 8, N), device="cuda", dtype=torch.int32)
        s = (torch.rand(((K + 63) // 64 if table16 else (K + 127) // 128, N), device="cuda") * 0.015 + 0.005).bfloat16()
        wq = qzo.qzo_repack_int4(words, K, N)
        y = torch.empty((M, N), device="cuda", dtype=torch.bfloat16)
        sets.append((x, wq, s, y))
        del words
    iters = max(iters, n_sets)
    need = qzo.qzo_gemm_workspace_bytes(M, K, N)
    ws = torch.empty((max(need, 256),), dtype=torch.uint8, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")

    table = [(-1.0 + 2.0 * i / 15.0) ** 3 for i in range(16)]        # any 16 values: the kernel looks them up

    def call(i):
        x, wq, s, y = sets[i % n_sets]
        if table16:
            qzo.qzo_perturbed_gemm_table16(x, wq, s, table, M, K, N, 42, 0, sign, 1e-3, y=y, workspace=ws, status=status)
        else:
            qzo.qzo_perturbed_gemm(x, wq, s, M, K, N, 42, 0, sign, 1e-3, y=y, workspace=ws, status=status)

    for i in range(max(3, n_sets)):
        call(i)
    torch.cuda.synchronize()
    # One launch, timed with events, sizes the timed pass: a pass rotates through every set at least
    # once and lasts about `pass_ms`, short enough to be a burst like the one the peak was taken in.
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    call(0)
    ev1.record()
    torch.cuda.synchronize()
    est_us = max(ev0.elapsed_time(ev1) * 1e3, 1.0)
    iters = max(n_sets, min(iters, int(pass_ms * 1e3 / est_us) + 1))
    # The launches of one timed pass are recorded into a CUDA graph and replayed, so that the
    # figure is device time: at small M a launch from Python costs more than the kernel runs.
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    times = []
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            for i in range(iters):
                call(i)
        graph.replay()
        side.synchronize()
        # Every shape is timed alone, against the burst peaks: an idle moment lets the SM clock recover
        # from the power-capped run of the shape before it; one untimed replay then warms up again.
        time.sleep(settle)
        graph.replay()
        side.synchronize()
        for _ in range(reps):
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record(side)
            graph.replay()
            ev1.record(side)
            side.synchronize()
            times.append(ev0.elapsed_time(ev1) * 1e3 / iters)
    assert int(status.item()) == 0
    times.sort()
    return times[len(times) // 2], times[0], n_sets      # microseconds per launch: median and best pass


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--shapes", default=",".join(f"{k}x{n}" for k, n in inputs.GEMM_SWEEP_KN))
    ap.add_argument("--tokens", default=",".join(str(m) for m in inputs.GEMM_SWEEP_M))
    ap.add_argument("--iters", type=int, default=50)
    ap.add_argument("--settle", type=float, default=1.0, help="idle seconds before each shape is timed")
    ap.add_argument("--json", action="store_true")
    ap.add_argument("--table16", action="store_true",
                    help="time the 16-entry-codebook / block-64 prologue (NF4-style storage) instead of int4 / group 128")
    args = ap.parse_args()
    bw, tf, src = peaks()
    rows = []
    for shape in args.shapes.split(","):
        K, N = (int(v) for v in shape.split("x"))
        for M in (int(v) for v in args.tokens.split(",")):
            us, best_us, n_sets = run_shape(M, K, N, args.iters, settle=args.settle, table16=args.table16)
            t_hbm = gemm_bytes(M, K, N) / (bw * 1e9) * 1e6
            t_mma = 2.0 * M * K * N / (tf * 1e12) * 1e6
            roof = max(t_hbm, t_mma)
            rows.append({"K": K, "N": N, "M": M, "us": us, "roofline_us": roof, "bound": "hbm" if t_hbm > t_mma else "tensor",
                         "frac": roof / us, "tflops": 2.0 * M * K * N / us / 1e6, "gbs": gemm_bytes(M, K, N) / us / 1e3,
                         "best_pass_us": best_us, "rotation_sets": n_sets})
            r = rows[-1]
            roof_nom = max(gemm_bytes(M, K, N) / (NOMINAL_HBM_GBS * 1e9), 2.0 * M * K * N / (NOMINAL_BF16_TFLOPS * 1e12)) * 1e6
            r["frac_of_nominal"] = roof_nom / us
            r["splits"] = qzo.qzo_gemm_workspace_bytes(M, K, N) // (M * N * 4)
            if not args.json:
                print(f"K={K:6d} N={N:6d} M={M:5d}  {us:9.2f} us  roofline {roof:8.2f} us ({r['bound']:6s})  "
                      f"frac {r['frac']:.3f} (of nominal peaks {r['frac_of_nominal']:.3f})  {r['tflops']:8.1f} TFLOP/s  "
                      f"{r['gbs']:8.1f} GB/s  best pass {best_us:8.2f} us  K slices {max(r['splits'], 1)}  sets={n_sets}",
                      flush=True)
    if not args.json:
        print(f"peaks ({src}): HBM {bw:.1f} GB/s, dense bf16 {tf:.1f} TFLOP/s; nominal: {NOMINAL_HBM_GBS:.0f} GB/s, "
              f"{NOMINAL_BF16_TFLOPS:.0f} TFLOP/s; min frac {min(r['frac'] for r in rows):.3f}, "
              f"rows at or above 0.70: {sum(r['frac'] >= 0.70 for r in rows)} of {len(rows)}")
    if args.json:
        print(json.dumps({"peaks": {"hbm_gbs": bw, "bf16_tflops": tf, "source": src}, "rows": rows}))


if __name__ == "__main__":
    main()
