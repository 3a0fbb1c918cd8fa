#!/usr/bin/env python
"""Benchmark of the DAM prefill hot path (mask construction + masked sparse attention) on B200.

One step = one layer of the workload: `dam_build_masks` followed by `dam_sparse_attention`, through
the C ABI.  Default workload: the 32-layer stack of Llama-3-8B-shaped layers at 32768 tokens, PCL 2048
(each step takes the next layer, its own seed and planted-pattern mix), inputs resident in HBM.

Prints ONE JSON line (metric, value, roofline, cpu_baseline, e2e, clocks, ...).  `--impl reference` times the CPU oracle
on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2506_11104_b200 import synth  # noqa: E402

METRIC = "prefill_attn_effective_tflops_active_tiles"
UNIT = "TFLOP/s"
TILE = 128


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16": d["bf16_tflops"], "bf16_sustained": d.get("bf16_tflops_sustained"),
                "which": "measured"}
    return {"hbm_gbs": 6650.0, "bf16": 1590.0, "bf16_sustained": 1400.0, "which": "fallback"}


def workload_name(cfg):
    return {1: "C1: Llama-3-8B-shaped layer, 32q/8kv heads, d128, S=8192, PCL=1024, bf16",
            2: "C2: 32-layer stack of Llama-3-8B-shaped layers (32q/8kv heads, d128), S=32768, PCL=2048, bf16; "
               "one step = one layer",
            3: "C3: one layer, 32q/8kv heads, d128, S=131072, PCL=4096, bf16",
            4: "C4: varlen batch 4096+16384+32768+65536 tokens, 32q/8kv heads, d128, PCL=1024, bf16"}[cfg]


def make_layer(cfg, layer, device):
    if cfg == 1:
        w = synth.llama_layer(8192, 1024, 1, layer, device)
    elif cfg == 2:
        w = synth.config2_layer(layer, device)
    elif cfg == 3:
        w = synth.llama_layer(131072, 4096, 3, layer, device, band_m_choices=(12, 16, 24), max_stripes=8)
    else:
        w = synth.config4(device)
    return w


def layer_ids_for_rank(rank, n_layers):
    """Each rank owns its own layers (independent problems, no data-path collective): seeds differ per rank."""
    return [rank * 1000 + l for l in range(n_layers)]


def aggregate_over_ranks(total_ms, flops, world, device):
    """Whole-job figures: time = MAX over ranks, work = SUM over ranks.  Returns (ms, flops)."""
    if world <= 1:
        return float(total_ms), float(flops)
    import torch.distributed as dist
    t = torch.tensor([total_ms], dtype=torch.float64, device=device)
    f = torch.tensor([flops], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(f, op=dist.ReduceOp.SUM)
    return float(t.item()), float(f.item())


def measured_traffic(kernel, cfg):
    """DRAM bytes per launch of the dominant kernel from the committed ncu capture (profiles/traffic.json)."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    try:
        return json.load(open(p)).get(kernel, {}).get(f"C{cfg}")
    except Exception:
        return None


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index = index
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()

    def run(self):
        q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        while not self._halt.is_set():
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-i",
                                      str(self.index)], capture_output=True, text=True, timeout=5).stdout.strip()
                f = [x.strip() for x in out.split(",")]
                self.samples.append(float(f[0]))
                self.max_mhz = float(f[1])
                for n, v in zip(names, f[2:]):
                    if v.lower().startswith("active"):
                        self.reasons.add(n)
            except Exception:
                pass
            self._halt.wait(0.1)

    def stop(self):
        self._halt.set()
        self.join(timeout=6)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_sample(w, n_rows=96, heads=(0, 13)):
    """Times the CPU oracle as it stands on a bounded sample of one layer: masks of a few heads (complete)
    plus masked attention on `n_rows` rows per head.  Returns (seconds per full layer extrapolated, info)."""
    from oracle import dam_oracle as orc
    Q, K, V = (x.float().cpu().numpy() for x in (w.Q, w.K, w.V))
    cores = orc.num_threads()
    t0 = time.perf_counter()
    masks = orc.build_masks(Q, K, w.cu_seqlens, w.pcl_max, w.tau, w.mu, w.lam, w.eps, heads=heads)
    t_mask = time.perf_counter() - t0
    rng = np.random.default_rng(0)
    t_att, rows_done, rows_total = 0.0, 0, 0
    for b in range(len(w.cu_seqlens) - 1):
        S = w.cu_seqlens[b + 1] - w.cu_seqlens[b]
        rows_total += S * w.num_q_heads
        for h in heads:
            rows = sorted(int(x) for x in rng.choice(S, size=min(S, n_rows), replace=False))
            t1 = time.perf_counter()
            orc.attention(Q, K, V, w.cu_seqlens, b, h, rows, masks[b][h])
            t_att += time.perf_counter() - t1
            rows_done += len(rows)
    nseq = len(w.cu_seqlens) - 1
    layer_s = t_mask / (len(heads) * nseq) * w.num_q_heads * nseq + t_att / rows_done * rows_total
    info = {"cores": cores, "kind": "oracle",
            "sample": f"masks of {len(heads)} of {w.num_q_heads} heads in full + masked attention on {rows_done} "
                      f"rows of {rows_total} (random rows, all keys); layer time extrapolated",
            "sample_seconds": round(t_mask + t_att, 2), "layer_seconds_extrapolated": layer_s}
    return layer_s, info


def decode_leg(dev, num_seqs=64, capacity=32768, pcl=2048, iters=16):
    """Generation-time attention: one token per sequence against a KV cache, keys chosen by the stored patterns.

    Reported beside the headline, not part of it.  Algorithmic bytes = the K and V rows a launch has to read once:
    per (sequence, KV head) the union over its query heads of matched columns and matched diagonals, 2 x 256 B
    each (positions are drawn at or beyond 2 L, where the two sets are disjoint)."""
    from paper_2506_11104_b200 import binding as B
    win, Kc, Vc, q = synth.decode_case(num_seqs, capacity, pcl, dev)
    Hq, Hkv, d = win.num_q_heads, win.num_kv_heads, win.head_dim
    wshape = B.make_shape(win.cu_seqlens, Hq, Hkv, d, torch.bfloat16, dev)
    rule = B.make_rule(pcl, win.tau, win.mu)
    blob, _ = B.dam_build_masks(win.Q, win.K, wshape, rule)
    assert B.dam_poll_status(blob) == 0
    mb = B.MaskBlob(blob)
    g = Hq // Hkv
    keys_all = keys_unique = 0
    for b in range(num_seqs):
        bits = [mb.pattern_bits(b, h) for h in range(Hq)]
        keys_all += sum(int(D.sum()) + int(V.sum()) for D, _, V in bits)
        for kv in range(Hkv):
            uD = np.zeros_like(bits[0][0])
            uV = np.zeros_like(bits[0][2])
            for h in range(kv * g, (kv + 1) * g):
                uD |= bits[h][0]
                uV |= bits[h][2]
            keys_unique += int(uD.sum()) + int(uV.sum())
    cache = B.make_shape([capacity * i for i in range(num_seqs + 1)], Hq, Hkv, d, torch.bfloat16, dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(1)
    poss = [torch.randint(2 * pcl, capacity, (num_seqs,), device=dev, dtype=torch.int32, generator=gen)
            for _ in range(iters + 3)]
    O = torch.empty_like(q)
    lse = torch.empty(num_seqs, Hq, device=dev, dtype=torch.float32)
    scr = torch.zeros(256, dtype=torch.uint8, device=dev)
    for p in poss[:3]:
        B.dam_decode_attention(q, Kc, Vc, blob, cache, p, O=O, lse=lse, scratch=scr)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for p in poss[3:]:
        B.dam_decode_attention(q, Kc, Vc, blob, cache, p, O=O, lse=lse, scratch=scr)
    e1.record()
    torch.cuda.synchronize()
    assert B.dam_poll_status(scr) == 0
    us = e0.elapsed_time(e1) / iters * 1e3
    row_bytes = 2 * d * 2
    pk = peaks()
    peak = pk["hbm_gbs"]
    gbs = keys_unique * row_bytes / (us * 1e-6) / 1e9
    return {"workload": f"{num_seqs} sequences x {capacity}-token KV cache (8 KV heads, d 128, bf16), one token each, "
                        f"positions uniform in [2 PCL, capacity), PCL {pcl}; {Kc.numel() * 4 / 2**30:.1f} GiB of cache, a new "
                        "position vector every launch",
            "us_per_launch": round(us, 1), "tokens_per_s": round(num_seqs / (us * 1e-6)),
            "keys_per_query_head": round(keys_all / (num_seqs * Hq), 1),
            "unique_keys_per_kv_head": round(keys_unique / (num_seqs * Hkv), 1),
            "roofline": {"bound": "hbm", "kernel": "decode_group_kernel", "achieved": round(gbs, 1), "peak": peak,
                         "peak_kind": "copy bandwidth, " + pk["which"], "unit": "GB/s", "frac": round(gbs / peak, 4),
                         "traffic": (lambda t: int(t * num_seqs) if t else None)(
                             (json.load(open(os.path.join(ROOT, "profiles", "traffic.json")))
                              .get("decode_group_kernel", {}).get("per_sequence"))
                             if os.path.exists(os.path.join(ROOT, "profiles", "traffic.json")) else None),
                         "algorithmic_bytes": keys_unique * row_bytes,
                         "requested_gbs": round(keys_all * row_bytes / (us * 1e-6) / 1e9, 1)}}


def per_head_listed_tiles(mask, Hq):
    """Listed (non-padding) entries of tiles[] per query head, read from the blob on the device."""
    from paper_2506_11104_b200 import binding as B
    hdr = np.frombuffer(mask[:256].cpu().numpy().tobytes(), dtype=B._HDR)[0]
    off_tiles, cap_head = int(hdr["off_tiles"]), int(hdr["head_tile_cap"])
    t = mask[off_tiles: off_tiles + 4 * Hq * cap_head].view(torch.int32).view(Hq, cap_head)
    return (t != 0).sum(dim=1).cpu().numpy()


def run_config(cfg, steps, warmup, gather, rank, world, local_rank, dev, pk, B, want_dense, long_warm=True):
    """Times `steps` layers of configuration `cfg` (stage 1 + stage 2 per step) and returns the figures of one
    benchmark line: executed-tile FLOPs over whole-step device time, per-stage times, densities, roofline."""
    import torch.distributed as dist
    n_distinct = {1: 32, 2: 32, 3: 2, 4: 1}[cfg]
    n_layers = min(n_distinct, steps + warmup)
    layers = [make_layer(cfg, l, dev) for l in layer_ids_for_rank(rank, n_layers)]
    w0 = layers[0]
    shape = B.make_shape(w0.cu_seqlens, w0.num_q_heads, w0.num_kv_heads, w0.head_dim, w0.Q.dtype, dev)
    rule = B.make_rule(w0.pcl_max, w0.tau, w0.mu, w0.lam, w0.eps, gather_columns=gather)
    rule_plain = B.make_rule(w0.pcl_max, w0.tau, w0.mu, w0.lam, w0.eps, gather_columns=False)
    mb, sb, ab = B.dam_mask_sizes(shape, rule)
    mbp, sbp, _ = B.dam_mask_sizes(shape, rule_plain)
    mask = torch.empty(max(mb, mbp), dtype=torch.uint8, device=dev)
    bscr = torch.empty(max(sb, sbp), dtype=torch.uint8, device=dev)
    ascr = torch.empty(max(256, ab), dtype=torch.uint8, device=dev)
    O = torch.empty_like(w0.Q)
    lse = torch.empty(w0.num_q_heads, shape.c.total_tokens, dtype=torch.float32, device=dev)

    def step(l, ev=None):
        w = layers[l % n_layers]
        if ev:
            ev[0].record()
        B.dam_build_masks(w.Q, w.K, shape, rule, mask, bscr)
        if ev:
            ev[1].record()
        B.dam_sparse_attention(w.Q, w.K, w.V, mask, shape, True, 0.0, O, lse, ascr)
        if ev:
            ev[2].record()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, warmup)):
        step(i)
    torch.cuda.synchronize()
    assert B.dam_poll_status(mask) == 0 and B.dam_poll_status(ascr) == 0
    sampler = ClockSampler(local_rank)
    sampler.start()
    if long_warm:
        # a longer loaded stretch before the timed region so that the clock sampler sees the GPU under this load
        t_end = time.perf_counter() + 1.0
        i = 0
        while time.perf_counter() < t_end:
            step(i)
            i += 1
            if i % 8 == 0:
                torch.cuda.synchronize()

    # ---- timed region: exactly `steps` steps, device-timed, per-stage events inside
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(steps)]
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    start.record()
    for i in range(steps):
        step(warmup + i, evs[i])
    end.record()
    barrier()
    clocks = sampler.stop()
    total_ms = start.elapsed_time(end)
    assert B.dam_poll_status(mask) == 0 and B.dam_poll_status(ascr) == 0
    s1 = [e[0].elapsed_time(e[1]) for e in evs]
    s2 = [e[1].elapsed_time(e[2]) for e in evs]

    # ---- statistics of the timed layers (outside the timed region: rebuild and read the blob)
    timed = sorted(set((warmup + i) % n_layers for i in range(steps)))
    Hq = w0.num_q_heads
    per_layer, head_exec, head_mask, elem_nnz = {}, [], [], {}
    for l in timed:
        w = layers[l]
        B.dam_build_masks(w.Q, w.K, shape, rule, mask, bscr)
        st = B.dam_mask_stats(mask, shape, active_elements=True)
        elem_nnz[l] = int(st.pop("active_elements").sum().item())
        per_layer[l] = st
        head_exec.append(per_head_listed_tiles(mask, Hq))
        if gather:
            B.dam_build_masks(w.Q, w.K, shape, rule_plain, mask, bscr)      # tiles of the masks themselves, per head
            head_mask.append(per_head_listed_tiles(mask, Hq))
        else:
            head_mask.append(head_exec[-1])
    causal_tiles = per_layer[timed[0]]["causal_tiles"]
    causal_head = causal_tiles / Hq
    hm = np.concatenate(head_mask) / causal_head
    he = np.concatenate(head_exec) / causal_head
    flops_tile = 4.0 * TILE * TILE * w0.head_dim
    step_tiles = [per_layer[(warmup + i) % n_layers]["tiles"] for i in range(steps)]
    step_mask_tiles = [per_layer[(warmup + i) % n_layers]["mask_tiles"] for i in range(steps)]
    total_ms_max, flops_exec = aggregate_over_ranks(total_ms, flops_tile * sum(step_tiles), world, dev)
    _, flops_mask = aggregate_over_ranks(total_ms, flops_tile * sum(step_mask_tiles), world, dev)
    _, flops_elem = aggregate_over_ranks(total_ms, 4.0 * w0.head_dim * sum(elem_nnz[(warmup + i) % n_layers] for i in range(steps)),
                                         world, dev)
    sec = total_ms_max * 1e-3
    causal_elems = sum(S * (S + 1) // 2 for S in shape.lengths) * Hq

    # ---- roofline of the dominant kernel (sparse attention incl. the column gather), from the per-launch events
    attn_ms = sum(s2) / len(s2)
    attn_tflops = flops_tile * (sum(step_tiles) / len(step_tiles)) / (attn_ms * 1e-3) / 1e12
    roof = {"bound": "tensor", "kernel": "attn_sm100_kernel", "achieved": round(attn_tflops, 2), "peak": pk["bf16"],
            "peak_kind": f"cuBLAS bf16 burst, {pk['which']} (the attention call is timed by itself, {attn_ms:.2f} ms per launch)",
            "unit": "TFLOP/s", "frac": round(attn_tflops / pk["bf16"], 4),
            "frac_of_sustained": round(attn_tflops / (pk["bf16_sustained"] or pk["bf16"]), 4),
            "frac_of_nominal_2250": round(attn_tflops / 2250.0, 4),
            "sm_mhz_sampled": clocks.get("sm_mhz"),
            "algorithmic_flops_per_launch": flops_tile * (sum(step_tiles) / len(step_tiles)),
            "traffic": measured_traffic("attn_sm100_kernel", cfg) if gather else None,
            "avg_launch_ms": round(attn_ms, 4)}
    res = {"value": round(flops_exec / sec / 1e12, 3), "ms_per_step": round(total_ms_max / steps, 4),
           "stage1_ms": round(sum(s1) / len(s1), 4), "stage2_ms": round(attn_ms, 4),
           "median_ms": {"stage1": round(statistics.median(s1), 4), "stage2": round(statistics.median(s2), 4),
                         "layer": round(statistics.median([a + b for a, b in zip(s1, s2)]), 4)},
           "value_definition": "4*128*128*d FLOP per tile the attention kernel executed (listed tiles), over the device "
                               "time of the whole steps (stage 1 + stage 2)",
           "effective_mask_tile_tflops": round(flops_mask / sec / 1e12, 3),
           "effective_mask_tile_definition": "4*128*128*d per 128x128 tile of the masks that holds an active cell (more "
                                             "than the kernel executes when matched columns are served by gathered tiles)",
           "element_active_tflops": round(flops_elem / sec / 1e12, 3),
           "element_density": round(sum(elem_nnz.values()) / len(elem_nnz) / causal_elems, 5),
           "tile_density": round(sum(step_mask_tiles) / len(step_mask_tiles) / causal_tiles, 4),
           "executed_tile_density": round(sum(step_tiles) / len(step_tiles) / causal_tiles, 4),
           "tile_density_per_layer_min_max": [round(min(step_mask_tiles) / causal_tiles, 4),
                                              round(max(step_mask_tiles) / causal_tiles, 4)],
           "tile_density_per_head": {"heads": int(hm.size), "min": round(float(hm.min()), 4),
                                     "median": round(float(np.median(hm)), 4), "max": round(float(hm.max()), 4),
                                     "executed_min": round(float(he.min()), 4), "executed_median": round(float(np.median(he)), 4),
                                     "executed_max": round(float(he.max()), 4)},
           "roofline": roof, "clocks": clocks, "distinct_layers": n_layers,
           "gpu_launches": (8 if gather else 7) * steps}      # init, score, counts, match, classify, order, [gather], attention
    if want_dense and rank == 0:
        # the build's own dense causal attention at the same length (all tiles listed as fully active)
        dmb, _, _ = B.dam_mask_sizes(shape, None, True)
        dmask = torch.empty(dmb, dtype=torch.uint8, device=dev)
        B.dam_mask_all_ones(shape, True, dev, dmask)
        for _ in range(2):
            B.dam_sparse_attention(w0.Q, w0.K, w0.V, dmask, shape, True, 0.0, O, lse, ascr)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        nd = 3 if cfg != 3 else 1
        e0.record()
        for i in range(nd):
            w = layers[i % n_layers]
            B.dam_sparse_attention(w.Q, w.K, w.V, dmask, shape, True, 0.0, O, lse, ascr)
        e1.record()
        torch.cuda.synchronize()
        dense_ms = e0.elapsed_time(e1) / nd
        res["dense_causal"] = {"ms": round(dense_ms, 3), "tflops": round(flops_tile * causal_tiles / (dense_ms * 1e-3) / 1e12, 1),
                               "frac_of_burst": round(flops_tile * causal_tiles / (dense_ms * 1e-3) / 1e12 / pk["bf16"], 4),
                               "speedup_sparse_stage2": round(dense_ms / attn_ms, 2),
                               "speedup_sparse_layer": round(dense_ms / (total_ms_max / steps), 2)}
        del dmask
    ctx = dict(layers=layers, shape=shape, rule=rule, w0=w0, lse=lse, per_layer=per_layer, n_layers=n_layers,
               flops_tile=flops_tile, barrier=barrier)
    return res, ctx


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=32)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-dense", action="store_true")
    ap.add_argument("--no-decode", action="store_true", help="skip the generation-time (KV cache) measurement")
    ap.add_argument("--no-configs", action="store_true", help="skip the short runs of the other configurations")
    ap.add_argument("--only-decode", type=int, default=0, metavar="SEQS",
                    help="run only the generation-time measurement on SEQS sequences and print its object (for profiling)")
    ap.add_argument("--no-gather", action="store_true", help="list one tile per matched column stripe instead of gathered-column tiles")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if rank != 0:
            return
        run_reference(args)
        return

    if args.only_decode:
        if rank == 0:
            torch.cuda.set_device(0)
            print(json.dumps({"decode": decode_leg("cuda:0", num_seqs=args.only_decode, iters=4)}))
        return

    import torch.distributed as dist
    from paper_2506_11104_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)
    pk = peaks()
    cfg = args.config
    gather = not args.no_gather
    res, ctx = run_config(cfg, args.steps, args.warmup, gather, rank, world, local_rank, dev, pk, B, not args.no_dense)
    layers, shape, rule, w0, lse = ctx["layers"], ctx["shape"], ctx["rule"], ctx["w0"], ctx["lse"]
    per_layer, n_layers, flops_tile, barrier = ctx["per_layer"], ctx["n_layers"], ctx["flops_tile"], ctx["barrier"]

    out = {"metric": METRIC, "value": res.pop("value"), "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": args.warmup, "ms_per_step": res.pop("ms_per_step"), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
           "config": {"workload": workload_name(cfg), "pcl": w0.pcl_max, "tau": w0.tau, "mu": w0.mu,
                      "l2": "inputs larger than L2: every step reads a different layer's Q/K/V (384 MiB at C2)",
                      "distinct_layers": res.pop("distinct_layers"), "gathered_column_tiles": gather,
                      "tile_density_per_head": res.pop("tile_density_per_head")}}
    out.update(res)

    if rank == 0 and world == 1 and not args.no_decode:
        out["decode"] = decode_leg(dev)

    if not args.no_e2e:
        # end to end through the host-buffer entry point: H2D of Q, K, V and D2H of O, LSE inside the timed region;
        # the layers are the first timed ones, so that their executed-tile counts are the measured ones
        n_e2e = min(args.steps, 4)
        e2e_layers = [(args.warmup + i) % n_layers for i in range(n_e2e)]
        hosts = [tuple(x.cpu().pin_memory() for x in (layers[l].Q, layers[l].K, layers[l].V)) for l in e2e_layers]
        Oh = torch.empty(w0.Q.shape, dtype=w0.Q.dtype).pin_memory()
        lh = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
        nbytes = B.dam_prefill_host(hosts[0][0], hosts[0][1], hosts[0][2], shape, rule, Oh, lh, None, dev)
        ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
        B.dam_prefill_host(hosts[0][0], hosts[0][1], hosts[0][2], shape, rule, Oh, lh, ws, dev)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for q, k, v in hosts:
            B.dam_prefill_host(q, k, v, shape, rule, Oh, lh, ws, dev)
        e1.record()
        barrier()
        e2e_ms, e2e_flops = aggregate_over_ranks(e0.elapsed_time(e1), flops_tile * sum(per_layer[l]["tiles"] for l in e2e_layers),
                                                 world, dev)
        es = w0.Q.element_size()
        out["e2e"] = {"value": round(e2e_flops / (e2e_ms * 1e-3) / 1e12, 3), "unit": UNIT,
                      "ms_per_step": round(e2e_ms / n_e2e, 3), "steps": n_e2e, "layers": e2e_layers,
                      "h2d_bytes_per_step": int((w0.Q.numel() + w0.K.numel() + w0.V.numel()) * es),
                      "d2h_bytes_per_step": int(w0.Q.numel() * es + lse.numel() * 4),
                      "api": "dam_prefill_host (pinned host buffers in and out); executed-tile FLOPs of the layers it ran"}
        del ws, hosts

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        l = args.warmup % n_layers
        layer_s, info = oracle_sample(layers[l], n_rows=6144, heads=tuple(range(w0.num_q_heads)))
        info["value"] = round(flops_tile * per_layer[l]["tiles"] / layer_s / 1e12, 6)
        info["unit"] = UNIT
        out["cpu_baseline"] = info

    del layers, ctx
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and gather and not args.no_configs:
        # the same workload with one listed tile per matched-column stripe (no gathered-column tiles): more tiles, longer
        # lists, a slower layer and a higher rate on the executed tiles
        r, cx = run_config(cfg, 8, 3, False, rank, world, local_rank, dev, pk, B, False, long_warm=False)
        out["no_gather"] = {k: r[k] for k in ("value", "ms_per_step", "stage1_ms", "stage2_ms", "executed_tile_density", "roofline")}
        del cx
        torch.cuda.empty_cache()
    if rank == 0 and world == 1 and not args.no_configs:
        # the other full-size configurations, one short run each, same fields
        others = {}
        for c in (1, 3, 4):
            if c == cfg:
                continue
            r, cx = run_config(c, 8 if c != 3 else 4, 3, gather, rank, world, local_rank, dev, pk, B, c != 3, long_warm=False)
            r["workload"] = workload_name(c)
            others[f"C{c}"] = r
            del cx
            torch.cuda.empty_cache()
        out["configs"] = others

    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def run_reference(args):
    """The CPU oracle, as it stands, on a bounded sample of the same workload (one sample per step)."""
    cfg = args.config
    w = make_layer(cfg, 0, "cpu") if cfg != 3 else synth.llama_layer(131072, 4096, 3, 0, "cpu", band_m_choices=(12, 16, 24), max_stripes=8)
    from oracle import dam_oracle as orc
    # tile count of the layer from the oracle's own masks is expensive; use a tile-density estimate from sampled heads
    times, measured, info = [], [], None
    n = args.warmup + args.steps
    for i in range(n):
        t0 = time.perf_counter()
        layer_s, info = oracle_sample(w, n_rows=256, heads=(i % w.num_q_heads, (i + 16) % w.num_q_heads))
        if i >= args.warmup:
            times.append(layer_s)
            measured.append(time.perf_counter() - t0)
    layer_s = sum(times) / len(times)
    # active tiles of the sampled head, from its oracle mask rows (q-block samples)
    tiles = estimate_tiles(w, orc)
    flops = 4.0 * TILE * TILE * w.head_dim * tiles
    value = flops / layer_s / 1e12
    info.update({"value": round(value, 6), "unit": UNIT})
    out = {"impl": "reference", "metric": METRIC, "value": round(value, 6), "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(sum(measured) / len(measured) * 1e3, 1),
           "step_definition": "one bounded sample of a layer (the masks of two heads in full, masked attention on 256 rows "
                              "of each); ms_per_step is the time a sample took, value the rate of the whole layer "
                              "extrapolated from it",
           "layer_ms_extrapolated": round(layer_s * 1e3, 1), "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": workload_name(cfg), "pcl": w.pcl_max, "tau": w.tau, "mu": w.mu},
           "cpu_baseline": info,
           "e2e": {"value": round(value, 6), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def estimate_tiles(w, orc, heads=(0, 7, 13, 22, 29)):
    """Active 128 x 128 tiles of the layer, estimated from the oracle's masks of a few heads."""
    Q, K = w.Q.float().numpy(), w.K.float().numpy()
    masks = orc.build_masks(Q, K, w.cu_seqlens, w.pcl_max, w.tau, w.mu, w.lam, w.eps, heads=heads)
    tot = 0.0
    for b in range(len(w.cu_seqlens) - 1):
        S = w.cu_seqlens[b + 1] - w.cu_seqlens[b]
        nq = (S + TILE - 1) // TILE
        for h in heads:
            hm = masks[b][h]
            qbs = sorted(set(np.linspace(0, nq - 1, num=min(nq, 16), dtype=int).tolist()))
            per = []
            for qb in qbs:
                rows = hm.rows(list(range(qb * TILE, min(S, qb * TILE + TILE))))
                nk = (S + TILE - 1) // TILE
                pad = np.zeros((rows.shape[0], nk * TILE), np.uint8)
                pad[:, :S] = rows
                per.append(int(pad.reshape(rows.shape[0], nk, TILE).any(axis=(0, 2)).sum()))
            tot += float(np.mean(per)) * nq / len(heads) * w.num_q_heads
    return tot


if __name__ == "__main__":
    main()
