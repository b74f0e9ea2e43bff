"""Small cases of the library's calls for profiler captures and quick CUDA-event timings.

    python -m paper_2302_08545_b200.profile_cases <case> [--iters 5]

Each case allocates a few hundred MB (inputs larger than the 126 MB L2, far below a GB per
buffer), warms the calls up, times them with CUDA events and prints one JSON line.  Run under
`ncu -k regex:<kernel> -c <n>` the same command gives the counters of the kernels named below.

  case              calls (kernels)
  tile14            prepare, compress, aggregate, decompress at B = 2^14 (rht_tile_kernel)
  quantize          thc_quantize_rotated (quantize_rotated_kernel)
  bf16k22           compress, aggregate, decompress for bf16 gradients at B = 2^22, n = 2
                    (thc_pipeline_kernel<bf16, KB = 9>, aggregate_b4w8, thc_pipeline_kernel<decompress>)
  n16               the same calls for n = 16 workers, fp32, B = 2^20 (aggregate_b4w16_kernel)
  b2                n = 4, 2-bit identity table (aggregate_small_w8_kernel<2>)
  ef                thc_error_feedback (thc_pipeline_kernel<error feedback>)
  minmax            thc_prepare_minmax + compress in exact-range mode (thc_pipeline_kernel<range>)
  aggdec            thc_aggregate_decompress (thc_pipeline_kernel<aggregate + decompress>)
  fused             thc_prepare_compress, n = 8 (thc_pipeline_kernel<fused scales + compress>)
  scan              compress and decompress of 4 x 2^26 fp32 coordinates for B = 2^15 .. 2^22 (one line each)
  cfg1 .. cfg4, cfg3b2   the benchmark configurations at full size, inputs generated on the device
                    (per-call times of the round, error feedback and the one-call tail included)
"""
from __future__ import annotations

import argparse
import json

from . import workloads as W


W_PEAK = 6549.8   # GB/s: the machine's measured HBM copy rate (MEASURED_PEAKS.json), for the printed fraction


def _time(fn, iters, torch, stream):
    for _ in range(2):
        fn()
    torch.cuda.synchronize()
    evs = []
    for _ in range(iters):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        fn()
        b.record(stream)
        evs.append((a, b))
    torch.cuda.synchronize()
    ts = sorted(a.elapsed_time(b) for a, b in evs)
    return ts[len(ts) // 2]


def scan(iters: int):
    """Block-size scan: the same 4 x 2^26 coordinates through every two-pass block size."""
    import torch
    from . import runner
    stream = torch.cuda.current_stream()
    for k in range(15, 23):
        w = W.Workload(f"scan_k{k}", n=4, d=1 << 26, log2_block=k, bits=4, granularity=30,
                       table=W.TABLES[(4, 30)], data_seed=5)
        ctx = runner.context_for(w)
        r = runner.Round(ctx, w.n, w.d, w.in_dtype)
        W.fill_torch(w, r.grads)
        r.prepare()
        tc = _time(lambda: r.compress(0), iters, torch, stream)
        r.aggregate()
        td = _time(lambda: r.decompress(0), iters, torch, stream)
        print(json.dumps({"case": "scan", "log2_block": k, "compress_ms": round(tc, 4),
                          "decompress_ms": round(td, 4), "status_flags": ctx.status()}), flush=True)
        del r, ctx
        torch.cuda.empty_cache()


def run(case: str, iters: int):
    import torch
    from . import runner
    if case == "scan":
        return scan(iters)
    stream = torch.cuda.current_stream()
    T = W.TABLES[(4, 30)]
    mk = lambda **kw: W.Workload(f"profile_{case}", table=kw.pop("table", T), bits=kw.pop("bits", 4),
                                 granularity=kw.pop("granularity", 30), data_seed=9, **kw)
    exact = case == "minmax"
    full = {"cfg1": W.config1, "cfg2": W.config2, "cfg3": lambda: W.config3(4), "cfg3b2": lambda: W.config3(2),
            "cfg4": W.config4}
    if case in full:
        w = full[case]()
    elif case == "tile14":
        w = mk(n=4, d=1 << 24, log2_block=14)
    elif case == "bf16k22":
        w = mk(n=2, d=1 << 25, log2_block=22, in_dtype="bf16")
    elif case == "n16":
        w = mk(n=16, d=1 << 23, log2_block=20)
    elif case == "fused":
        w = mk(n=8, d=1 << 24, log2_block=20)
    elif case == "b2":
        w = mk(n=4, d=1 << 24, log2_block=20, bits=2, granularity=3, table=W.TABLES[(2, 3)])
    else:
        w = mk(n=4, d=1 << 24, log2_block=20)
    ctx = runner.context_for(w, exact_range=exact)
    r = runner.Round(ctx, w.n, w.d, w.in_dtype, want_rotated=case in ("quantize",))
    W.fill_torch(w, r.grads)
    out = {}
    if exact:
        r.rotated = None
        prep = lambda: ctx.prepare_minmax(r.grads, w.d, 0, r.scales, r.workspace)
        out["prepare_minmax"] = _time(prep, iters, torch, stream)
    else:
        out["prepare"] = _time(r.prepare, iters, torch, stream)
    out["compress"] = _time(lambda: r.compress(0), iters, torch, stream)
    if case == "fused" or (case in full and r.sz.fused_scales):
        out["prepare_compress"] = _time(lambda: r.prepare_compress(0), iters, torch, stream)
    if case == "quantize":
        out["quantize_rotated"] = _time(lambda: r.quantize_rotated(0), iters, torch, stream)
    out["aggregate"] = _time(r.aggregate, iters, torch, stream)
    out["decompress"] = _time(lambda: r.decompress(0), iters, torch, stream)
    if case == "aggdec" or case in full:
        out["aggregate_decompress"] = _time(lambda: r.aggregate_decompress(0), iters, torch, stream)
    if case == "ef" or (case in full and w.in_dtype == "f32"):
        ef = [torch.zeros(w.d, dtype=torch.float32, device=r.device) for _ in range(w.n)]
        out["error_feedback"] = _time(lambda: ctx.error_feedback(r.grads, r.packed, w.d, 0, r.scales, ef, r.workspace),
                                      iters, torch, stream)
    ab = w.algorithmic_bytes()
    if case in full:
        rnd = out["compress"] + out["aggregate"] + out["decompress"]
        out["round"] = rnd
        out["round_one_call_tail"] = out["compress"] + out["aggregate_decompress"]
    line = {"case": case, "n": w.n, "d": w.d, "log2_block": w.log2_block, "bits": w.bits, "in_dtype": w.in_dtype,
            "acc_bits": w.acc_bits, "ms": {k: round(v, 4) for k, v in out.items()},
            "algorithmic_gbs": {k: round(ab[k] / out[k] / 1e6, 1) for k in out if k in ab},
            "round_frac_of_measured_hbm": (round(ab["round"] / out["round"] / 1e6 / W_PEAK, 4) if "round" in out else None),
            "status_flags": ctx.status()}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("case", choices=["tile14", "quantize", "bf16k22", "n16", "b2", "ef", "minmax", "aggdec", "fused", "scan",
                                     "cfg1", "cfg2", "cfg3", "cfg3b2", "cfg4"])
    ap.add_argument("--iters", type=int, default=5)
    a = ap.parse_args()
    run(a.case, a.iters)


if __name__ == "__main__":
    main()
