#!/usr/bin/env python
"""Benchmark of the WaveAlign hot path on B200: one step = plan (row counts, guard statistics,
centred subspace iteration, angular sort, per-wave count sort) + block-sparse attention in
the planned row order, over one synthetic video-shaped batch.

    python bench.py --gpus N --steps K --warmup W            # this library
    python bench.py --impl reference ...                      # the CPU oracle, bounded sample

Prints ONE JSON line (rank 0).  metric: TFLOP/s over computed block pairs
(4 * block_q * block_kv * head_dim * #pairs / time).  With N > 1 every rank runs one batch
element of the same shape (heads sharded by batch element, no data-path collective), timing
is the max over ranks and the value is the whole-job aggregate ("weak" scaling).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "block-sparse attn TFLOP/s (computed blocks) & % BF16 peak; L2 hit %, DRAM bytes"
UNIT = "TFLOP/s"


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], bf16=d["bf16_tflops"], bf16_sustained=d.get("bf16_tflops_sustained"),
                    source="measured")
    return dict(hbm=6650.0, bf16=1590.0, bf16_sustained=1400.0, source="fallback")


def ncu_traffic(workload: str):
    """DRAM bytes per launch of the attention kernel from the committed ncu summary, if any."""
    p = os.path.join(ROOT, "profiles", f"k_bsattn_fwd_{workload}.txt")
    if os.path.exists(p):
        for line in open(p):
            if line.startswith("dram_bytes_per_launch_bench_workload:"):
                return float(line.split(":")[1].split()[0])
    return None


class ClockSampler:
    """nvidia-smi clock/throttle samples during the timed region (reading only)."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "20", "-i", str(index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            pass

    def stop(self):
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        rows = [r.strip().split(", ") for r in open(self.f.name) if r.strip()]
        os.unlink(self.f.name)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[3:7]):
                if v.strip().lower().startswith("active"):
                    reasons.add(n)
        busy = sorted(sm)[len(sm) // 2:] if sm else []
        return {"sm_mhz": statistics.median(busy) if busy else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------- oracle legs

def oracle_sample(cfg, target_s=12.0, n_heads=4):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload: the plan
    (NumPy, every step of Algorithm 1/2) of `n_heads` heads and the attention (C twin, OpenMP
    over query tokens) of query blocks drawn from those heads until about `target_s` seconds
    of CPU work are spent.  Returns (TFLOP/s over the sampled pairs, info, seconds)."""
    from oracle import waveal_oracle as wo
    from oracle import c_twin
    from paper_2609_34814_b200 import inputs as I
    import torch
    c_twin.build()
    rng = np.random.default_rng(cfg.tensor_seed)
    heads = sorted(rng.choice(cfg.heads, size=min(n_heads, cfg.heads), replace=False).tolist())
    t_plan = t_attn = 0.0
    pairs = tasks = 0
    data = []
    for h in heads:
        mk = I.make_mask(cfg, h)
        t0 = time.perf_counter()
        wo.plan_head(mk, 148, 5, cfg.plan_seed, h, mode=wo.MODE_FORCE_REORDER)   # T = the library default
        t_plan += time.perf_counter() - t0
        bits = [I.make_head_tensor(cfg, w, h).view(torch.int16).numpy().view(np.uint16) for w in "qkv"]
        data.append((mk, bits, rng.permutation(cfg.n_blocks)))
    scale = 1 / math.sqrt(cfg.head_dim)
    for i in range(cfg.n_blocks):
        for mk, bits, rows in data:
            r = int(rows[i])
            lst = np.nonzero(mk[r])[0]
            t0 = time.perf_counter()
            c_twin.attn_tasks(*bits, cfg.block, cfg.block, cfg.seq, cfg.seq, scale, [r], [lst])
            t_attn += time.perf_counter() - t0
            pairs += len(lst)
            tasks += 1
        if t_plan + t_attn >= target_s:
            break
    flops = 4.0 * cfg.block * cfg.block * cfg.head_dim * pairs
    total = t_plan + t_attn
    info = {"cores": c_twin.threads(), "kind": "oracle",
            "sample": f"{tasks} query blocks ({pairs} block pairs) of {len(heads)} heads: fp64 C attention "
                      f"{t_attn:.2f} s + NumPy plan of those heads {t_plan:.2f} s",
            "seconds": total}
    return flops / total / 1e12, info, total


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals, infos, times = [], None, []
    for i in range(args.warmup + args.steps):
        v, info, t = oracle_sample(cfg, target_s=5.0, n_heads=1)
        if i >= args.warmup:
            vals.append(v); times.append(t); infos = info
    value = float(np.mean(vals))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(times)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg.name, "note": "CPU oracle on a bounded sample of the workload per step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": infos["cores"], "kind": "oracle",
                             "sample": infos["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# --------------------------------------------------------------------------- GPU arm

def run_waveal(args, cfg):
    import torch
    from paper_2609_34814_b200 import binding as wb
    from paper_2609_34814_b200 import dist as wd
    from paper_2609_34814_b200 import inputs as I

    rank, world, local = wd.init("nccl")
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    wb.load()
    H, S, Sp, D, B = cfg.heads, cfg.seq, cfg.seq_pad, cfg.head_dim, cfg.block
    nb = cfg.n_blocks
    # ---- synthetic batch element of this rank: host (pinned) and device copies
    if args.mask == "random20":
        # the unstructured mask of the paper's Table 1 (20 % uniform columns per row): the locality floor
        masks = [I.random_mask(nb, nb, 0.20, cfg.mask_seed * 1000 + h) for h in range(H)]
    elif args.mask == "dense":
        # all block pairs: the dense run behind the gap metric (1/density) / (t_dense / t_sparse)
        masks = [np.ones((nb, nb), dtype=bool) for _ in range(H)]
    else:
        masks = [I.make_mask(cfg, h) for h in range(H)]
    bitmap_h = torch.from_numpy(np.stack([I.mask_to_bitmap(m) for m in masks]).view(np.int64)).pin_memory()
    ptr_np, idx_np = I.masks_to_csr(masks)
    pairs = int(ptr_np[-1])
    flops = 4.0 * B * B * D * pairs
    qkv_h = [torch.empty((H, Sp, D), dtype=torch.bfloat16).pin_memory() for _ in range(3)]
    for h in range(H):
        for t, name in zip(qkv_h, "qkv"):
            t[h].copy_(I.make_head_tensor(cfg, name, h))
    o_h = torch.empty((H, Sp, D), dtype=torch.bfloat16).pin_memory()
    q, k, v = (t.to(dev, non_blocking=True) for t in qkv_h)
    o = torch.zeros_like(q)
    bitmap = bitmap_h.to(dev, non_blocking=True)
    ptr = torch.from_numpy(ptr_np).to(dev)
    idx = torch.from_numpy(idx_np).to(dev)
    W = wb.default_wave_size()
    step_mode = {"reorder": wb.FORCE_REORDER, "natural": wb.FORCE_NATURAL, "auto": wb.AUTO,
                 "stage1": wb.STAGE1_ONLY, "stage2": wb.STAGE2_ONLY}[args.plan_mode]
    pdesc = wb.plan_desc_default(heads=H, n_q_blocks=nb, n_kv_blocks=nb, wave_size=W, mode=step_mode,
                                 seed=cfg.plan_seed, kv_bytes_per_head=2 * Sp * D * 2)
    if args.svd_iters > 0:
        pdesc.svd_iters = args.svd_iters
    pws = torch.empty((wb.plan_workspace_bytes(pdesc) + 256,), dtype=torch.uint8, device=dev)
    adesc = wb.attn_desc(q, k, v, o, S, S, B, args.head_order == "interleaved")
    aws = torch.empty((wb.bsattn_workspace_bytes(adesc),), dtype=torch.uint8, device=dev)
    status = torch.zeros((4,), dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    launches = {"n": 0}

    def step(mode=step_mode, count=False):
        pdesc.mode = mode
        plan = wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream)
        if count:
            launches["n"] += wb.last_launch_count()
        wb.bsattn_fwd(adesc, q, k, v, o, ptr, idx, row_order=plan.row_order, workspace=aws, dev_status=status,
                      stream=stream)
        if count:
            launches["n"] += wb.last_launch_count()
        return plan

    def ev():
        return torch.cuda.Event(enable_timing=True)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    # ---- timed region: K steps, events on the launching stream; the attention kernel of each
    #      step is bracketed by its own events for the roofline figure
    pdesc.mode = step_mode
    attn_ev = []
    wd.barrier()
    torch.cuda.synchronize()
    sampler = ClockSampler(local) if rank == 0 else None
    e0, e1 = ev(), ev()
    e0.record(stream)
    for _ in range(args.steps):
        plan = wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream)
        launches["n"] += wb.last_launch_count()
        a0, a1 = ev(), ev()
        a0.record(stream)
        wb.bsattn_fwd(adesc, q, k, v, o, ptr, idx, row_order=plan.row_order, workspace=aws, dev_status=status,
                      stream=stream)
        a1.record(stream)
        launches["n"] += wb.last_launch_count()
        attn_ev.append((a0, a1))
    e1.record(stream)
    torch.cuda.synchronize()
    wd.barrier()
    clocks = sampler.stop() if sampler else None
    total_ms = wd.max_over_ranks(e0.elapsed_time(e1), dev)
    ms_per_step = total_ms / args.steps
    attn_ms = statistics.mean(a.elapsed_time(b) for a, b in attn_ev)
    if status.tolist()[0] != 0:
        raise RuntimeError(f"device-side failure reported by the attention kernel: {status.tolist()}")
    value = world * flops / (ms_per_step * 1e-3) / 1e12

    # ---- context numbers (outside the timed region): natural order, guard decision, plan alone
    def timed(fn, reps=5):
        ts = []
        for _ in range(reps):
            a, b = ev(), ev()
            a.record(stream); fn(); b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)

    pdesc.mode = wb.FORCE_REORDER
    reo = wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream).row_order
    t_reo = timed(lambda: wb.bsattn_fwd(adesc, q, k, v, o, ptr, idx, row_order=reo, workspace=aws, dev_status=status, stream=stream))
    t_nat = timed(lambda: wb.bsattn_fwd(adesc, q, k, v, o, ptr, idx, row_order=None, workspace=aws, dev_status=status, stream=stream))
    t_plan = timed(lambda: wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream))
    pdesc.mode = wb.AUTO
    auto = wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream)
    torch.cuda.synchronize()
    skipped = int((auto.skip_flags & 1).sum().item())
    t_plan_auto = timed(lambda: wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream))
    pdesc.mode = step_mode
    # the two extra passes of the paper's own deployment (gather Q into the order, scatter O back),
    # which the index-list kernel does not need: pure HBM copies, reported for context
    t_gather = timed(lambda: wb.gather_rows(q, o, reo, B, stream=stream))
    t_scatter = timed(lambda: wb.scatter_rows(q, o, reo, B, stream=stream))
    copy_bytes = 2.0 * H * Sp * D * 2

    # ---- end to end through the public API with host buffers: H2D of Q, K, V and the mask,
    #      index lists built on the device, plan, attention, D2H of O - all inside the timed region.
    #      Heads are independent, so the step runs as groups of heads on three streams (copy in,
    #      compute, copy out): the copies of one group overlap the kernels of another.
    e2e = None
    if not args.no_e2e:
        n_e2e = max(1, min(args.steps, 3))
        G = 4 if H >= 8 else H
        groups = [(g0, min(g0 + G, H)) for g0 in range(0, H, G)]
        s_in, s_c, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
        gdesc = {}
        for g0, g1 in groups:
            gdesc[g0] = wb.plan_desc_default(heads=g1 - g0, n_q_blocks=nb, n_kv_blocks=nb, wave_size=W, mode=step_mode,
                                             seed=cfg.plan_seed, kv_bytes_per_head=2 * Sp * D * 2)
            gdesc[g0].svd_iters = pdesc.svd_iters

        def e2e_step():
            start = ev()
            start.record(stream)
            for st_ in (s_in, s_c, s_out):
                st_.wait_event(start)
            done = []
            for g0, g1 in groups:
                with torch.cuda.stream(s_in):
                    for src, dst in zip(qkv_h, (q, k, v)):
                        dst[g0:g1].copy_(src[g0:g1], non_blocking=True)
                    bitmap[g0:g1].copy_(bitmap_h[g0:g1], non_blocking=True)
                    e_in = ev()
                    e_in.record(s_in)
                with torch.cuda.stream(s_c):
                    s_c.wait_event(e_in)
                    cap = int(ptr_np[g1 * nb] - ptr_np[g0 * nb])
                    p2, i2 = wb.bitmap_to_csr(bitmap[g0:g1], nb, capacity=cap, stream=s_c)
                    pl = wb.plan_bitmap(gdesc[g0], bitmap[g0:g1], workspace=pws, stream=s_c)
                    ad = wb.attn_desc(q[g0:g1], k[g0:g1], v[g0:g1], o[g0:g1], S, S, B, args.head_order == "interleaved")
                    wb.bsattn_fwd(ad, q[g0:g1], k[g0:g1], v[g0:g1], o[g0:g1], p2, i2, row_order=pl.row_order,
                                  workspace=aws, dev_status=status, stream=s_c)
                    e_c = ev()
                    e_c.record(s_c)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(e_c)
                    o_h[g0:g1].copy_(o[g0:g1], non_blocking=True)
                    e_o = ev()
                    e_o.record(s_out)
                done.append(e_o)
            for e_o in done:
                stream.wait_event(e_o)

        e2e_step()
        torch.cuda.synchronize()
        wd.barrier()
        a, b = ev(), ev()
        a.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        b.record(stream)
        torch.cuda.synchronize()
        wd.barrier()
        if status.tolist()[0] != 0:
            raise RuntimeError(f"device-side failure reported by the attention kernel: {status.tolist()}")
        ms = wd.max_over_ranks(a.elapsed_time(b), dev) / n_e2e
        h2d = sum(t.numel() * t.element_size() for t in qkv_h) + bitmap_h.numel() * 8
        e2e = {"value": world * flops / (ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": o_h.numel() * 2,
               "pipeline": "%d groups of %d heads on three streams" % (len(groups), G)}

    pk = peaks()
    if rank != 0:
        wd.shutdown()
        return
    achieved = flops / (attn_ms * 1e-3) / 1e12
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "heads": H, "head_dim": D, "seq": S, "block": B, "block_pairs": pairs,
                   "density": pairs / (H * nb * nb), "wave_size": W, "plan_mode": args.plan_mode,
                   "mask": args.mask, "head_order": args.head_order, "svd_iters": int(pdesc.svd_iters),
                   "step": "plan + attention", "l2": "inputs (Q,K,V,O %.1f GB) larger than L2, no flush" %
                   (4 * H * Sp * D * 2 / 1e9), "batch_elements": world},
        "roofline": {"bound": "tensor", "kernel": "k_bsattn_fwd", "achieved": achieved, "peak": pk["bf16"],
                     "unit": "TFLOP/s", "frac": achieved / pk["bf16"], "peak_source": pk["source"] + " (burst)",
                     "frac_of_sustained": achieved / pk["bf16_sustained"] if pk["bf16_sustained"] else None,
                     "kernel_ms": attn_ms,
                     "traffic": ncu_traffic(cfg.name) if args.mask == "videomask" else None},
        "kernel": {"attn_ms_reordered": t_reo, "attn_ms_natural": t_nat, "speedup_vs_natural": t_nat / t_reo,
                   "tflops_reordered": flops / t_reo / 1e9, "tflops_natural": flops / t_nat / 1e9,
                   "plan_ms": t_plan, "plan_ms_auto": t_plan_auto, "auto_skipped_heads": skipped,
                   "plan_share_of_step": t_plan / (t_plan + t_reo),
                   "paper_gather_q_ms": t_gather, "paper_scatter_o_ms": t_scatter,
                   "gather_gbs": copy_bytes / t_gather / 1e6, "gather_frac_of_hbm_peak": copy_bytes / t_gather / 1e6 / pk["hbm"]},
        "e2e": e2e, "gpu_launches": launches["n"], "clocks": clocks,
    }
    if world == 1 and not args.no_cpu:
        v, info, _ = oracle_sample(cfg)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": info["cores"], "kind": "oracle",
                                "sample": info["sample"]}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    wd.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="waveal", choices=["waveal", "reference"])
    ap.add_argument("--config", default="wan720p")
    ap.add_argument("--heads", type=int, default=0, help="use only the first HEADS heads (profiling / parity cases)")
    ap.add_argument("--plan-mode", default="reorder", choices=["reorder", "natural", "auto", "stage1", "stage2"],
                    help="which stages the plan of the timed step runs (Section 6.5 ablation); the headline is 'reorder'")
    ap.add_argument("--mask", default="videomask", choices=["videomask", "random20", "dense"],
                    help="mask generator: the config's structured recipe, 20 %% uniform columns per row "
                         "(the paper's Random row), or all pairs (dense run for the gap metric)")
    ap.add_argument("--head-order", default="sequential", choices=["sequential", "interleaved"],
                    help="ticket order: all rows of a head before the next head, or position-major over heads")
    ap.add_argument("--svd-iters", type=int, default=0, help="T of Algorithm 1 (0 = the library default)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "waveal" else args.warmup
    from paper_2609_34814_b200 import inputs as I
    cfg = I.CONFIGS[args.config]
    if args.heads:
        import dataclasses
        cfg = dataclasses.replace(cfg, heads=args.heads, name=f"{cfg.name}_h{args.heads}")
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_waveal(args, cfg)


if __name__ == "__main__":
    main()
