#!/usr/bin/env python
"""Benchmark of the WaveAlign hot path on B200: one step = plan (row counts, guard statistics,
centred subspace iteration, angular sort, per-wave count sort) + block-sparse attention in
the planned row order, over one synthetic video-shaped batch.

    python bench.py --gpus N --steps K --warmup W            # this library
    python bench.py --impl reference ...                      # the CPU oracle, bounded sample

Prints ONE JSON line (rank 0).  metric: TFLOP/s over computed block pairs
(4 * block_q * block_kv * head_dim * #pairs / time).  With N > 1 the heads of the one batch
element are split over the ranks (contiguous slices, no data-path collective: heads are planned
and attended independently), timing is the max over ranks and the value is all heads' FLOPs over
that time ("strong" scaling); --replicas gives every rank a whole batch element instead ("weak").
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
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


def ncu_counters(workload: str):
    """Counters of one launch of the attention kernel on this workload, per row order, from the
    committed ncu summary (profiles/k_bsattn_fwd_<workload>.txt, lines `key: value`), if any."""
    p = os.path.join(ROOT, "profiles", f"k_bsattn_fwd_{workload}.txt")
    out = {}
    if os.path.exists(p):
        for line in open(p):
            k, _, v = line.partition(":")
            if k in ("l2_hit_pct_reordered", "l2_hit_pct_natural", "dram_read_bytes_reordered",
                     "dram_write_bytes_reordered", "dram_read_bytes_natural", "dram_write_bytes_natural",
                     "kernel_time_ns_natural", "kernel_time_ns_reordered"):
                try:
                    out[k] = float(v.split()[0])
                except (ValueError, IndexError):
                    pass
    return out


# --------------------------------------------------------------------------- oracle legs

ORACLE_MODES = {"reorder": 1, "natural": 2, "auto": 0, "stage1": 3, "stage2": 4}


def l2_bytes_of_device() -> int:
    """L2 size the guard compares with (the device's when one is visible, else the B200's 126 MB)."""
    try:
        import torch
        if torch.cuda.is_available():
            return int(torch.cuda.get_device_properties(0).L2_cache_size)
    except Exception:
        pass
    return 126 * 1024 * 1024


def oracle_sample(cfg, target_s=12.0, n_heads=4, plan_mode="auto"):
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
        wo.plan_head(mk, 148, 5, cfg.plan_seed, h, mode=ORACLE_MODES[plan_mode],          # T = the library default
                     guard={"kv_bytes_per_head": 2 * cfg.seq_pad * cfg.head_dim * 2, "l2_bytes": l2_bytes_of_device()})
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
        v, info, t = oracle_sample(cfg, target_s=5.0, n_heads=1, plan_mode=args.plan_mode)
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
    from paper_2609_34814_b200 import timing as wt

    rank, world, local = wd.init("nccl")
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU fallback")
    if os.environ.get("WAVEAL_BENCH_ONE_DEVICE"):
        local = 0                                 # functional test: all ranks share cuda:0 (control plane over gloo)
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    wb.load()
    S, Sp, D, B = cfg.seq, cfg.seq_pad, cfg.head_dim, cfg.block
    nb = cfg.n_blocks
    # ---- this rank's heads: all of them at N = 1 or with --replicas, else a contiguous slice
    split = world > 1 and not args.replicas
    my_heads = list(wd.head_slice(rank, world, cfg.heads)) if split else list(range(cfg.heads))
    H = len(my_heads)
    if H == 0:
        raise RuntimeError(f"{cfg.heads} heads cannot be split over {world} ranks")
    # ---- synthetic inputs of those heads: host (pinned) and device copies
    if args.mask == "random20":
        # the unstructured mask of the paper's Table 1 (20 % uniform columns per row): the locality floor
        masks = [I.random_mask(nb, nb, 0.20, cfg.mask_seed * 1000 + h) for h in my_heads]
    elif args.mask == "dense":
        # all block pairs: the dense run behind the gap metric (1/density) / (t_dense / t_sparse)
        masks = [np.ones((nb, nb), dtype=bool) for _ in my_heads]
    else:
        masks = [I.make_mask(cfg, h) for h in my_heads]
    bitmap_h = torch.from_numpy(np.stack([I.mask_to_bitmap(m) for m in masks]).view(np.int64)).pin_memory()
    ptr_np, idx_np = I.masks_to_csr(masks)
    pairs = int(ptr_np[-1])
    flops = 4.0 * B * B * D * pairs                         # this rank's share
    qkv_h = [torch.empty((H, Sp, D), dtype=torch.bfloat16).pin_memory() for _ in range(3)]
    for i, h in enumerate(my_heads):
        for t, name in zip(qkv_h, "qkv"):
            t[i].copy_(I.make_head_tensor(cfg, name, h))
    o_h = torch.empty((H, Sp, D), dtype=torch.bfloat16).pin_memory()
    q, k, v = (t.to(dev, non_blocking=True) for t in qkv_h)
    o = torch.zeros_like(q)
    bitmap = bitmap_h.to(dev, non_blocking=True)
    ptr = torch.from_numpy(ptr_np).to(dev)
    idx = torch.from_numpy(idx_np).to(dev)
    W = args.wave if args.wave > 0 else wb.default_wave_size()
    step_mode = {"reorder": wb.FORCE_REORDER, "natural": wb.FORCE_NATURAL, "auto": wb.AUTO,
                 "stage1": wb.STAGE1_ONLY, "stage2": wb.STAGE2_ONLY}[args.plan_mode]
    ring = wb.RING_CUT_LARGEST_GAP if args.ring_cut else 0
    step_mode |= ring
    pdesc = wb.plan_desc_default(heads=H, n_q_blocks=nb, n_kv_blocks=nb, wave_size=W, mode=step_mode,
                                 seed=cfg.plan_seed, kv_bytes_per_head=2 * Sp * D * 2)
    if args.svd_iters > 0:
        pdesc.svd_iters = args.svd_iters
    pws = torch.empty((wb.plan_workspace_bytes(pdesc) + 256,), dtype=torch.uint8, device=dev)
    adesc = wb.attn_desc(q, k, v, o, S, S, B, args.head_order == "interleaved")
    aws = torch.empty((wb.bsattn_workspace_bytes(adesc),), dtype=torch.uint8, device=dev)
    aws_words = aws.view(torch.int32)
    status = torch.zeros((4,), dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    launches = {"n": 0}

    def attend(order):
        wb.bsattn_fwd(adesc, q, k, v, o, ptr, idx, row_order=order, workspace=aws, dev_status=status, stream=stream)

    def step():
        plan = wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream)
        attend(plan.row_order)
        return plan

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def check_status():
        if status.tolist()[0] != 0:
            raise RuntimeError(f"device-side failure reported by the attention kernel: {status.tolist()}")

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    # ---- timed region: K steps, events on the launching stream; the attention kernel of each
    #      step is bracketed by its own events for the roofline figure
    attn_ev = []
    wd.barrier()
    torch.cuda.synchronize()
    sampler = wt.ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.begin("timed steps")
    e0, e1 = ev(), ev()
    e0.record(stream)
    for i in range(args.steps):
        plan = wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream)
        launches["n"] += wb.last_launch_count()
        a0, a1 = ev(), ev()
        a0.record(stream)
        attend(plan.row_order)
        a1.record(stream)
        launches["n"] += wb.last_launch_count()
        attn_ev.append((a0, a1))
    e1.record(stream)
    torch.cuda.synchronize()
    if sampler:
        sampler.end("timed steps")
    wd.barrier()
    total_ms = wd.max_over_ranks(e0.elapsed_time(e1), dev)
    ms_per_step = total_ms / args.steps
    attn_ms = statistics.mean(a.elapsed_time(b) for a, b in attn_ev)
    step_cycles = int(aws_words[4].item())          # SM cycles of the attention launch of the last timed step
    step_pairs = int(aws_words[6].item())           # query-block pairs that shared a tile in it (64-row blocks)
    step_tiles = int(aws_words[7].item())           # 128-row x 128-key MMA tiles it ran
    check_status()
    flops_all = wd.sum_over_ranks(flops, dev) if world > 1 else flops
    value = flops_all / (ms_per_step * 1e-3) / 1e12

    # ---- context numbers (outside the timed region)
    def timed(fn, reps=5, batch=1):
        """Median over `reps` of the device time of `batch` back-to-back calls, per call (a batch
        keeps the stream busy, so that short kernels are not timed by the host's enqueue rate)."""
        ts = []
        for _ in range(reps):
            a, b = ev(), ev()
            a.record(stream)
            for _ in range(batch):
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b) / batch)
        return statistics.median(ts)

    # planned vs natural row order of the same kernel: interleaved launches, per-pair ratios,
    # and the kernel's own cycle counts (clock-independent)
    pdesc.mode = wb.FORCE_REORDER | ring
    reo = wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream).row_order
    if sampler:
        torch.cuda.synchronize()
        sampler.begin("order comparison")
    ab = wt.ab_interleaved(lambda: attend(reo), lambda: attend(None), args.ab_pairs, stream,
                           cycles_of=lambda: aws_words[4:5])
    if sampler:
        sampler.end("order comparison")
    check_status()
    t_reo, t_nat = ab["a_ms"], ab["b_ms"]
    t_plan = timed(lambda: wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream), batch=8)
    pdesc.mode = wb.AUTO | ring
    auto = wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream)
    torch.cuda.synchronize()
    skipped = int((auto.skip_flags & 1).sum().item())
    t_plan_auto = timed(lambda: wb.plan_bitmap(pdesc, bitmap, workspace=pws, stream=stream), batch=8)
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
        check_status()
        ms = wd.max_over_ranks(a.elapsed_time(b), dev) / n_e2e
        h2d = sum(t.numel() * t.element_size() for t in qkv_h) + bitmap_h.numel() * 8
        e2e = {"value": flops_all / (ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": o_h.numel() * 2,
               "pipeline": "%d groups of %d heads on three streams" % (len(groups), G)}

    # ---- optional: every rank gets the whole O back (one all-gather over the head axis)
    gather_ms = None
    if split and args.gather_o:
        torch.cuda.synchronize()
        wd.barrier()
        a, b = ev(), ev()
        a.record(stream)
        full = wd.gather_heads(o, cfg.heads)
        b.record(stream)
        torch.cuda.synchronize()
        gather_ms = wd.max_over_ranks(a.elapsed_time(b), dev)
        assert full.shape[0] == cfg.heads
        del full

    pk = peaks()
    if rank != 0:
        wd.shutdown()
        return
    achieved = flops / (attn_ms * 1e-3) / 1e12
    ctr = ncu_counters(cfg.name) if args.mask == "videomask" and not split else {}
    traffic = None
    step_skipped = int((plan.skip_flags & 1).sum().item())      # heads the timed steps ran in natural order
    key = "natural" if step_skipped == H else "reordered" if step_skipped == 0 else "mixed"
    if f"dram_read_bytes_{key}" in ctr and f"dram_write_bytes_{key}" in ctr:
        traffic = ctr[f"dram_read_bytes_{key}"] + ctr[f"dram_write_bytes_{key}"]
    for o in ("natural", "reordered"):
        # achieved HBM rate of the captured launch against the measured copy bandwidth
        if all(f"{x}_{o}" in ctr for x in ("dram_read_bytes", "dram_write_bytes", "kernel_time_ns")):
            gbs = (ctr[f"dram_read_bytes_{o}"] + ctr[f"dram_write_bytes_{o}"]) / ctr[f"kernel_time_ns_{o}"]
            ctr[f"hbm_gbs_{o}"] = gbs
            ctr[f"hbm_frac_of_peak_{o}"] = gbs / pk["hbm"]
    clocks = sampler.summary("timed steps")
    clocks_ab = sampler.summary("order comparison")
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if split else "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "heads": cfg.heads, "heads_per_rank": H, "head_dim": D, "seq": S, "block": B,
                   "block_pairs_rank0": pairs,
                   "density": pairs / (H * nb * nb), "wave_size": W, "plan_mode": args.plan_mode, "ring_cut": bool(args.ring_cut), "heads_in_natural_order": step_skipped,
                   "mask": args.mask, "head_order": args.head_order, "svd_iters": int(pdesc.svd_iters),
                   "step": "plan + attention", "l2": "inputs (Q,K,V,O %.1f GB per rank) larger than L2, no flush" %
                   (4 * H * Sp * D * 2 / 1e9),
                   "sharding": ("heads split over ranks, no collective" if split else
                                "one batch element per rank" if world > 1 else "single GPU")},
        "roofline": {"bound": "tensor", "kernel": "k_bsattn_fwd", "achieved": achieved, "peak": pk["bf16"],
                     "unit": "TFLOP/s", "frac": achieved / pk["bf16"], "peak_source": pk["source"] + " (burst)",
                     "frac_of_sustained": achieved / pk["bf16_sustained"] if pk["bf16_sustained"] else None,
                     "frac_of_datasheet_2250": achieved / 2250.0,
                     "kernel_ms": attn_ms, "kernel_sm_cycles": step_cycles, "tiles_shared_by_two_blocks": step_pairs,
                     "mma_tiles": step_tiles, "mma_tile_fill": (pairs * B * B / (step_tiles * 128.0 * 128.0)) if step_tiles else None,
                     "traffic": traffic,
                     "traffic_source": "ncu, one launch of this workload (profiles/)" if traffic else None},
        "counters": {"source": "profiles/k_bsattn_fwd_%s.txt (ncu, one launch per order)" % cfg.name, **ctr} if ctr else None,
        "kernel": {"attn_ms_reordered": t_reo, "attn_ms_natural": t_nat,
                   "speedup_vs_natural": ab["b_over_a"], "speedup_vs_natural_min": ab["b_over_a_min"],
                   "speedup_vs_natural_max": ab["b_over_a_max"],
                   "speedup_vs_natural_cycles": ab.get("b_over_a_cycles"),
                   "speedup_vs_natural_cycles_min": ab.get("b_over_a_cycles_min"),
                   "speedup_vs_natural_cycles_max": ab.get("b_over_a_cycles_max"),
                   "cycles_reordered": ab.get("a_cycles"), "cycles_natural": ab.get("b_cycles"),
                   "comparison": "%d interleaved pairs, median of per-pair ratios" % ab["pairs"],
                   "clocks_during_comparison": clocks_ab,
                   "tflops_reordered": flops / t_reo / 1e9, "tflops_natural": flops / t_nat / 1e9,
                   "plan_ms": t_plan, "plan_ms_auto": t_plan_auto, "auto_skipped_heads": skipped,
                   "plan_share_of_step": t_plan / (t_plan + t_reo),
                   "paper_gather_q_ms": t_gather, "paper_scatter_o_ms": t_scatter,
                   "gather_gbs": copy_bytes / t_gather / 1e6, "gather_frac_of_hbm_peak": copy_bytes / t_gather / 1e6 / pk["hbm"],
                   "all_gather_o_ms": gather_ms},
        "e2e": e2e, "gpu_launches": launches["n"], "clocks": clocks,
    }
    if world == 1 and not args.no_cpu:
        v, info, _ = oracle_sample(cfg, plan_mode=args.plan_mode)
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
    ap.add_argument("--plan-mode", default="auto", choices=["reorder", "natural", "auto", "stage1", "stage2"],
                    help="which stages the plan of the timed step runs (Section 6.5 ablation); the headline is 'auto': "
                         "the guard of Section 4.5 decides per head whether reordering pays")
    ap.add_argument("--mask", default="videomask", choices=["videomask", "random20", "dense"],
                    help="mask generator: the config's structured recipe, 20 %% uniform columns per row "
                         "(the paper's Random row), or all pairs (dense run for the gap metric)")
    ap.add_argument("--head-order", default="sequential", choices=["sequential", "interleaved"],
                    help="ticket order: all rows of a head before the next head, or position-major over heads")
    ap.add_argument("--svd-iters", type=int, default=0, help="T of Algorithm 1 (0 = the library default)")
    ap.add_argument("--wave", type=int, default=0, help="W the plan buckets by (0 = the kernel's tasks in flight, SM count)")
    ap.add_argument("--ring-cut", action="store_true", help="Stage-1 variant: open the angular ring at its largest gap")
    ap.add_argument("--ab-pairs", type=int, default=12, help="interleaved launch pairs of the planned-vs-natural comparison")
    ap.add_argument("--replicas", action="store_true", help="N > 1: every rank runs a whole batch element (weak scaling) "
                                                             "instead of a slice of the heads")
    ap.add_argument("--gather-o", action="store_true", help="N > 1: also time the all-gather that re-assembles O on every rank")
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
