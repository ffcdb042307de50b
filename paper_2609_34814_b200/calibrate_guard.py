"""Offline profile behind the skip guard (Section 4.5 of the paper: the thresholds of the
short-sequence and too-sparse tests are fitted to the machine, not derived).

For a grid of sequence lengths (frames of the 720p recipe) and mask densities it times, on the
current device, the attention kernel in natural and in planned row order and the plan itself,
and prints for every point whether planning pays (natural - planned > plan time).  From the
grid it proposes the two integer thresholds the library takes:

  l2_fit_num / l2_fit_den   skip when K+V bytes of one head <= L2 bytes * num / den
  min_density_ppm           skip when the mask is sparser than this

Usage:  python -m paper_2609_34814_b200.calibrate_guard [--heads 40] [--frames 11,21,41,61,101]
                                                        [--densities 0.02,0.04,0.10] [--json out.json]
Inputs are the same seeded synthetic masks and tensors the tests and the bench use; the tool
only calls the library's public entry points.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import statistics
import sys

import numpy as np


def measure(cfg, reps: int):
    import torch
    from . import binding as wb
    from . import inputs as I
    from . import timing as wt

    dev = torch.device("cuda")
    H, S, Sp, D, B, nb = cfg.heads, cfg.seq, cfg.seq_pad, cfg.head_dim, cfg.block, cfg.n_blocks
    masks = [I.make_mask(cfg, h) for h in range(H)]
    bitmap = torch.from_numpy(np.stack([I.mask_to_bitmap(m) for m in masks]).view(np.int64)).to(dev)
    ptr_np, idx_np = I.masks_to_csr(masks)
    ptr, idx = torch.from_numpy(ptr_np).to(dev), torch.from_numpy(idx_np).to(dev)
    pairs = int(ptr_np[-1])
    g = torch.Generator(device=dev)
    g.manual_seed(cfg.tensor_seed)
    q, k, v = (torch.randn((H, Sp, D), device=dev, generator=g).to(torch.bfloat16) for _ in range(3))
    o = torch.empty_like(q)
    pdesc = wb.plan_desc_default(heads=H, n_q_blocks=nb, n_kv_blocks=nb, wave_size=wb.default_wave_size(),
                                 mode=wb.FORCE_REORDER, seed=cfg.plan_seed, kv_bytes_per_head=2 * Sp * D * 2)
    pws = torch.empty((wb.plan_workspace_bytes(pdesc) + 256,), dtype=torch.uint8, device=dev)
    st = torch.zeros((4,), dtype=torch.int32, device=dev)
    adesc = wb.attn_desc(q, k, v, o, S, S, B)
    aws = torch.empty((wb.bsattn_workspace_bytes(adesc),), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def timed(fn):
        fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)

    plan = wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream)
    t_plan = timed(lambda: wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream))
    # the two orders alternate launch by launch (a drifting SM clock then hits both alike); the
    # gain is taken from the median per-pair ratio, and the kernel's own cycle counts give the
    # clock-independent view
    aws_words = aws.view(torch.int32)
    ab = wt.ab_interleaved(
        lambda: wb.bsattn_fwd(adesc, q, k, v, o, ptr, idx, row_order=plan.row_order, workspace=aws, dev_status=st, stream=stream),
        lambda: wb.bsattn_fwd(adesc, q, k, v, o, ptr, idx, row_order=None, workspace=aws, dev_status=st, stream=stream),
        reps, stream, cycles_of=lambda: aws_words[4:5])
    if st.tolist()[0] != 0:
        raise RuntimeError(f"attention kernel reported {st.tolist()}")
    t_reo = ab["a_ms"]
    t_nat = t_reo * ab["b_over_a"]
    return {"frames": cfg.frames, "seq": S, "density": pairs / (H * nb * nb), "pairs": pairs,
            "kv_bytes_per_head": 2 * Sp * D * 2, "natural_ms": t_nat, "planned_ms": t_reo, "plan_ms": t_plan,
            "natural_over_planned": ab["b_over_a"], "ratio_min": ab["b_over_a_min"], "ratio_max": ab["b_over_a_max"],
            "natural_over_planned_cycles": ab.get("b_over_a_cycles"),
            "gain_ms": t_nat - t_reo - t_plan, "pays": bool(t_nat - t_reo > t_plan)}


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__, formatter_class=argparse.RawDescriptionHelpFormatter)
    ap.add_argument("--heads", type=int, default=40,
                    help="heads per call: the plan runs one CTA per head, so its time is flat up to the SM count "
                         "while the attention time grows with the heads - calibrate at the deployment's head count")
    ap.add_argument("--frames", default="11,21,41,61,101")
    ap.add_argument("--densities", default="0.02,0.04,0.10")
    ap.add_argument("--reps", type=int, default=8, help="interleaved launch pairs per grid point")
    ap.add_argument("--recipe", default="long720p", help="config whose mask recipe the grid scales (long720p, wan720p)")
    ap.add_argument("--json", default="")
    args = ap.parse_args(argv)
    import torch
    from . import binding as wb
    from . import inputs as I

    if not torch.cuda.is_available():
        raise RuntimeError("the guard is calibrated on the device it will run on: a CUDA device is required")
    wb.load()
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    base = I.CONFIGS[args.recipe]
    rows = []
    for fr in (int(x) for x in args.frames.split(",")):
        for rho in (float(x) for x in args.densities.split(",")):
            cfg = dataclasses.replace(I.scaled_config(base, fr, heads=args.heads), rho=(rho, rho))
            r = measure(cfg, args.reps)
            r["kv_over_l2"] = r["kv_bytes_per_head"] / l2
            rows.append(r)
            print("frames %4d  seq %7d  density %.3f  K+V/L2 %.2f  natural %8.3f  planned %8.3f  ratio %.3f [%.3f, %.3f] cycles %s  "
                  "plan %6.3f  gain %+7.3f ms  %s"
                  % (fr, r["seq"], r["density"], r["kv_over_l2"], r["natural_ms"], r["planned_ms"], r["natural_over_planned"],
                     r["ratio_min"], r["ratio_max"],
                     "%.3f" % r["natural_over_planned_cycles"] if r["natural_over_planned_cycles"] else "-",
                     r["plan_ms"], r["gain_ms"], "pays" if r["pays"] else "skip"), flush=True)
    # thresholds: the largest K+V/L2 ratio at which planning never paid, and the largest density
    # at which it never paid once K+V no longer fits
    never = [r["kv_over_l2"] for r in rows if not any(x["pays"] for x in rows if x["frames"] == r["frames"])]
    fit = max(never) if never else 0.0
    big = [r for r in rows if r["kv_over_l2"] > fit]
    sparse = [r["density"] for r in big if not r["pays"]]
    dens = max(sparse) if sparse else 0.0
    den = 16
    num = int(fit * den)
    out = {"l2_bytes": l2, "l2_fit_num": num, "l2_fit_den": den, "min_density_ppm": int(round(dens * 1e6)),
           "grid": rows}
    print("proposed: l2_fit %d/%d (planning never paid up to K+V = %.2f x L2), min_density_ppm %d"
          % (num, den, fit, out["min_density_ppm"]))
    if args.json:
        with open(args.json, "w") as f:
            json.dump(out, f, indent=1)
    return out


if __name__ == "__main__":
    main(sys.argv[1:])
