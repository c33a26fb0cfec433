#!/usr/bin/env python
"""Throughput of the large-resolution ViT inference path on B200: images/s of ViT-L/16 at
2048x2048 with neighbouring-block sparse attention and the CLS-score token filter.

One step = one vit_forward over one batch of synthetic tissue-like images (patch embedding, 24
blocks with sparse attention, the filter after block 4, final LayerNorm).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME]
    python bench.py --impl reference ...     # the CPU oracle on a bounded sample of the workload

Prints ONE JSON line.  `value` is measured with the inputs resident in device memory; `e2e`
includes the pinned-host -> device copy of the images and the device -> host read of the output
tokens in every step.  `roofline` describes the kernel class with the largest share of the step,
`breakdown` every class, `cpu_baseline` the oracle timed on this host's cores.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import synth  # noqa: E402

METRIC = "ViT-L/16 images/s at 2048x2048 (sparse attention + token filter)"


def metric_name(wl):
    """The headline metric for the default workload; other workloads are named for what they run."""
    if wl["name"] == DEFAULT_WORKLOAD:
        return METRIC
    arch = "ViT-L/16" if wl["arch"]["patch"] == 16 else "ViT-g/14-style"
    what = "sparse attention + token filter" if wl["cfg"]["filter_layer"] > 0 else "sparse attention"
    return "%s images/s at %dx%d (%s)" % (arch, wl["side"], wl["side"], what)

WORKLOADS = {
    # name: (arch, image side, batch, block, radius, filter_layer, keep, weight seed, image seed)
    "vitl16_2048_b4_sparse_filter": ("l16", 2048, 4, 8, 1, 4, 0.5, 2, 6),
    "vitl16_2048_b4_sparse": ("l16", 2048, 4, 8, 1, 0, 1.0, 2, 6),
    "vitl16_1024_b1_sparse_filter": ("l16", 1024, 1, 8, 1, 4, 0.6, 2, 3),
    "vitl16_1024_b4_sparse_filter": ("l16", 1024, 4, 8, 1, 4, 0.5, 2, 6),
    "vitl16_448_b4_sparse_filter": ("l16", 448, 4, 8, 1, 4, 0.5, 2, 6),
    # ViT-g/14-style: 40 layers, d 1536, 24 heads, SwiGLU 4096; 146x146 grid, 5x5 block neighbourhood
    "vitg14_2044_b1_sparse_filter": ("g14", 2044, 1, 8, 2, 8, 0.5, 4, 5),
}
DEFAULT_WORKLOAD = "vitl16_2048_b4_sparse_filter"


def workload_config(name):
    arch_name, side, batch, block, radius, fl, keep, wseed, iseed = WORKLOADS[name]
    arch = synth.vit_l16() if arch_name == "l16" else synth.vit_g14()
    grid = side // arch["patch"]
    cfg = dict(arch, attn_mode=synth.ATTN_SPARSE, block=block, radius=radius, filter_layer=fl, keep_ratio=keep)
    return dict(name=name, arch=arch, cfg=cfg, side=side, grid=grid, batch=batch, wseed=wseed, iseed=iseed)


# --------------------------------------------------------------------------------------------
# algorithmic work (counting only; none of the method's arithmetic)
# --------------------------------------------------------------------------------------------
def attention_pairs(grid_h, grid_w, block, radius, n_global, positions=None):
    """(patch-query pairs incl. global key columns, global-query pairs) of one image and head."""
    pos = np.arange(grid_h * grid_w) if positions is None else np.asarray(positions)
    nby, nbx = -(-grid_h // block), -(-grid_w // block)
    cnt = np.zeros((nby, nbx), dtype=np.int64)
    np.add.at(cnt, ((pos // grid_w) // block, (pos % grid_w) // block), 1)
    integ = np.zeros((nby + 1, nbx + 1), dtype=np.int64)
    integ[1:, 1:] = cnt.cumsum(0).cumsum(1)
    by, bx = np.meshgrid(np.arange(nby), np.arange(nbx), indexing="ij")
    y0, y1 = np.maximum(by - radius, 0), np.minimum(by + radius, nby - 1) + 1
    x0, x1 = np.maximum(bx - radius, 0), np.minimum(bx + radius, nbx - 1) + 1
    nsum = integ[y1, x1] - integ[y0, x1] - integ[y1, x0] + integ[y0, x0]
    n_p = int(cnt.sum())
    return int((cnt * nsum).sum()) + n_p * n_global, n_global * (n_global + n_p)


def forward_flops(wl, kept_positions):
    """Useful FLOP of one step: GEMMs (2MNK) and attention (4*64 per allowed pair and head)."""
    a, c, g, B = wl["arch"], wl["cfg"], wl["grid"], wl["batch"]
    D, HID, H, G = a["dim"], a["mlp_hidden"], a["heads"], a["n_global"]
    n0 = G + g * g
    per_tok = 2 * D * (3 * D) + 2 * D * D + 2 * D * HID * (3 if a["mlp_kind"] == synth.MLP_SWIGLU else 2)
    gemm = 2.0 * B * g * g * (3 * a["patch"] ** 2) * D
    attn_patch = attn_glob = 0.0
    fl = c["filter_layer"]
    pre_p, pre_g = attention_pairs(g, g, c["block"], c["radius"], G)
    n_pre = a["layers"] if fl == 0 else fl
    gemm += n_pre * B * n0 * per_tok
    attn_patch += n_pre * B * 4.0 * 64 * H * pre_p
    attn_glob += n_pre * B * 4.0 * 64 * H * pre_g
    for b in range(B if fl > 0 else 0):
        pp, pg = attention_pairs(g, g, c["block"], c["radius"], G, kept_positions[b])
        n_post = a["layers"] - fl
        gemm += n_post * (G + len(kept_positions[b])) * per_tok
        attn_patch += n_post * 4.0 * 64 * H * pp
        attn_glob += n_post * 4.0 * 64 * H * pg
    return dict(gemm=gemm, attn_patch=attn_patch, attn_global=attn_glob)


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per GEMM launch, averaged over the 104
# GEMM launches of one step, from one ncu capture (profiles/gemm_dram_vitl16_2048_b4.md).  Valid
# only for the kernel source it was taken with: reported as null once gemm.cu has changed.
GEMM_TRAFFIC = {"vitl16_2048_b4_sparse_filter": (375.5e6, "39d36c0b6203")}


def gemm_traffic(workload):
    import hashlib
    ent = GEMM_TRAFFIC.get(workload)
    if ent is None:
        return None
    src = os.path.join(ROOT, "paper_2601_12150_b200", "csrc", "gemm.cu")
    try:
        sha = hashlib.sha1(open(src, "rb").read()).hexdigest()[:12]
    except OSError:
        return None
    return ent[0] if sha == ent[1] else None


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm=float(p["hbm_gbs"]), tensor=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    tensor_burst=float(p["bf16_tflops"]), source="measured")
    return dict(hbm=6650.0, tensor=1400.0, tensor_burst=1590.0, source="fallback")


# --------------------------------------------------------------------------------------------
# clocks
# --------------------------------------------------------------------------------------------
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.proc = None
        self.gpu = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
            out, _ = self.proc.communicate()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), reasons=sorted(reasons), samples=len(sm))


# --------------------------------------------------------------------------------------------
# CPU oracle leg
# --------------------------------------------------------------------------------------------
def oracle_sample(wl, rows, seed=11):
    """Time the oracle, as it stands, on a bounded sample of the workload and extrapolate to
    images/s.  Sample: `rows` token rows of every per-token operation of one block (LayerNorm,
    QKV / out / MLP linears, activation, residual adds) plus `rows` query rows of the sparse
    attention against all keys, once at the full token count and once at the post-filter count
    (a spatially coherent kept set); plus `rows` rows of the patch-embedding linear.  Every cost
    is linear in rows at a fixed token count, so
      T_image = N (t_embed + f (t_tok + t_attn_full)) + N' (L - f) (t_tok + t_attn_kept)  per row.
    """
    import oracle
    a, c, g = wl["arch"], wl["cfg"], wl["grid"]
    D, HID, H, G, L = a["dim"], a["mlp_hidden"], a["heads"], a["n_global"], a["layers"]
    rng = np.random.Generator(np.random.PCG64(seed))
    one = dict(a, layers=1)
    w = synth.vit_weights(wl["wseed"], one, 2, 2, pos_base=2)
    lw = w["layers"][0]
    np0 = g * g
    n0 = G + np0
    fl = c["filter_layer"]
    k = oracle.keep_count(np0, c["keep_ratio"]) if fl > 0 else np0
    n1 = G + k
    rows = min(rows, n0)
    x = rng.standard_normal((rows, D), dtype=np.float32)
    cols = synth.round_bf16(rng.standard_normal((rows, 3 * a["patch"] ** 2), dtype=np.float32))
    t = {}
    t0 = time.perf_counter()
    oracle.linear(cols, w["w_pe"], w["b_pe"])
    t["embed"] = time.perf_counter() - t0

    def per_token():
        h = oracle.layernorm(x, lw["ln1_g"], lw["ln1_b"], a["ln_eps"])
        oracle.linear(h, lw["w_qkv"], lw["b_qkv"])
        y = x + lw.get("ls1", 1.0) * oracle.linear(h, lw["w_o"], lw["b_o"])
        h = oracle.layernorm(y, lw["ln2_g"], lw["ln2_b"], a["ln_eps"])
        u = oracle.linear(h, lw["w_fc1"], lw["b_fc1"])
        if a["mlp_kind"] == synth.MLP_SWIGLU:
            u = oracle.silu_mul_n(u, oracle.linear(h, lw["w_fc3"], lw["b_fc3"]))
        else:
            u = oracle.gelu_n(u)
        return y + lw.get("ls2", 1.0) * oracle.linear(u, lw["w_fc2"], lw["b_fc2"])

    t0 = time.perf_counter()
    per_token()
    t["tok"] = time.perf_counter() - t0

    def attn(n_tok, positions):
        q, kk, v = synth.attention_qkv(seed + n_tok, 1, n_tok, H, D // H)
        qrows = np.sort(rng.choice(n_tok, size=rows, replace=rows > n_tok)).astype(np.int32)
        pp = None if positions is None else positions[None].astype(np.int32)
        t0 = time.perf_counter()
        oracle.attention(q, kk, v, g, g, c["block"], c["radius"], n_global=G, patch_pos=pp, rows=qrows)
        return time.perf_counter() - t0

    t["attn_full"] = attn(n0, None)
    if fl > 0:
        bg = synth.background_mask(rng, g, g, 1.0 - k / np0).reshape(-1)
        kept = np.flatnonzero(~bg)[:k]
        if kept.size < k:
            kept = np.sort(np.concatenate([kept, np.flatnonzero(bg)[:k - kept.size]]))
        t["attn_kept"] = attn(n1, kept)
    else:
        t["attn_kept"] = t["attn_full"]
    f = fl if fl > 0 else L
    t_image = (n0 * (t["embed"] + f * (t["tok"] + t["attn_full"])) + n1 * (L - f) * (t["tok"] + t["attn_kept"])) / rows
    total = sum(t.values())
    return dict(images_per_s=1.0 / t_image, sample_seconds=total, rows=rows, cores=oracle.num_threads(),
                parts={k_: round(v_, 4) for k_, v_ in t.items()})


def run_reference(args, wl, rank):
    if rank != 0:
        return
    rows = 512
    for _ in range(args.warmup):
        oracle_sample(wl, rows)
    times, rates, last = [], [], None
    for _ in range(args.steps):
        last = oracle_sample(wl, rows)
        times.append(last["sample_seconds"])
        rates.append(last["images_per_s"])
    value = statistics.mean(rates)
    sample = (f"{rows} token rows of each per-token op of one block + {rows} attention query rows at the full and "
              f"post-filter token counts + {rows} patch-embedding rows of one {wl['side']}x{wl['side']} image, "
              "extrapolated linearly in rows to a whole image")
    print(json.dumps({
        "impl": "reference", "metric": metric_name(wl), "value": value, "unit": "images/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * statistics.mean(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl["name"], "l2": "inputs larger than L2"},
        "cpu_baseline": {"value": value, "unit": "images/s", "cores": last["cores"], "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# --------------------------------------------------------------------------------------------
# multi-rank bookkeeping (replicas only: the path has no exchange step, so the only collective is
# this reduction of the timings)
# --------------------------------------------------------------------------------------------
def max_over_ranks(values, world, device):
    """Element-wise maximum of a list of floats over all ranks (identity when world == 1)."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist
    tt = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return tt.tolist()


def whole_job_rate(units_per_rank, world, ms):
    """Units per second of the whole job: every rank processed `units_per_rank` in `ms` (max over ranks)."""
    return units_per_rank * world / (ms * 1e-3)


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
def run_gpu(args, wl, rank, world):
    import torch
    import torch.distributed as dist
    import paper_2601_12150_b200 as spv

    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    ctx = spv.Context(local)
    a, c, g, B = wl["arch"], wl["cfg"], wl["grid"], wl["batch"]
    side = wl["side"]

    w = synth.vit_weights(wl["wseed"], a, g, g)
    dw = ctx.make_vit_weights(w)
    del w
    img_host = torch.from_numpy(synth.tissue_batch(wl["iseed"] + rank, B, side, side,
                                                   background_range=(0.3, 0.6))).pin_memory()
    img = img_host.to(dev)
    k = spv.filter_keep_count(g * g, c["keep_ratio"]) if c["filter_layer"] > 0 else g * g
    out = torch.empty((B, a["n_global"] + k, a["dim"]), dtype=torch.bfloat16, device=dev)
    out_host = torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()
    stream = torch.cuda.current_stream()

    def step():
        return ctx.vit_forward(c, dw, img, g, g, out=out)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    torch.cuda.reset_peak_memory_stats()
    n_warm = max(args.warmup, 1) if args.quick else max(args.warmup, 3)
    for _ in range(n_warm):
        _, kept = step()
    ctx.check()
    kept_host = kept.cpu().numpy() if kept is not None else None

    # ---- timed region: device-resident inputs.  K steps timed as a whole give `value`; the same K
    # steps are then repeated with the library's per-launch CUDA events switched on, which gives the
    # per-class times of the roofline figures (the events cost a little, so they stay out of `value`).
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
    barrier()
    sampler.start()
    launches0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    launches = ctx.launch_count() - launches0
    ctx.profile(True)
    for _ in range(args.steps):
        step()
    prof = ctx.profile_read()
    ctx.profile(False)
    ctx.check()
    clocks = sampler.stop()
    peak_bytes = torch.cuda.max_memory_allocated()

    # ---- end to end: pinned host images in, output tokens back to the host, every step.  The way a
    # user of the library would run a stream of batches: copies on their own streams, double-buffered,
    # so that the copy of batch i+1 and the read-back of batch i-1 overlap the forward of batch i.
    # Every byte of every step is copied inside the timed region.
    ms_e2e = float("nan")
    if not args.quick:
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        imgs = [img, torch.empty_like(img)]
        outs = [out, torch.empty_like(out)]
        outs_host = [out_host, torch.empty(out.shape, dtype=torch.bfloat16).pin_memory()]
        in_ready = [torch.cuda.Event() for _ in range(2)]
        comp_done = [torch.cuda.Event() for _ in range(2)]
        out_done = [torch.cuda.Event() for _ in range(2)]

        def e2e_run(n):
            for i in range(n):
                bsel = i & 1
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(comp_done[bsel])          # the forward that read this buffer is done
                    imgs[bsel].copy_(img_host, non_blocking=True)
                    in_ready[bsel].record(s_in)
                stream.wait_event(in_ready[bsel])
                if i >= 2:
                    stream.wait_event(out_done[bsel])             # its previous result has been read back
                ctx.vit_forward(c, dw, imgs[bsel], g, g, out=outs[bsel])
                comp_done[bsel].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(comp_done[bsel])
                    outs_host[bsel].copy_(outs[bsel], non_blocking=True)
                    out_done[bsel].record(s_out)
            stream.wait_event(out_done[0])
            stream.wait_event(out_done[1])

        e2e_run(2)
        barrier()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        e2e_run(args.steps)
        f1.record(stream)
        barrier()
        ms_e2e = f0.elapsed_time(f1)
        ctx.check()

    ms, ms_e2e = max_over_ranks([ms, ms_e2e], world, dev)
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    images = B * args.steps * world
    value = whole_job_rate(B * args.steps, world, ms)
    fl = forward_flops(wl, kept_host)
    steps = args.steps
    tot_ms = sum(v["ms"] for v in prof.values()) or 1.0
    brk = {}
    for name, v in prof.items():
        if v["launches"] == 0:
            continue
        e = dict(launches_per_step=v["launches"] / steps, ms_per_step=v["ms"] / steps, share=v["ms"] / tot_ms)
        sec = v["ms"] * 1e-3
        if name == "gemm":
            e.update(bound="tensor", achieved=v["work"] / sec / 1e12, unit="TFLOP/s", peak=pk["tensor"])
        elif name == "attn_patch":
            e.update(bound="tensor", achieved=fl["attn_patch"] * steps / sec / 1e12, unit="useful TFLOP/s",
                     peak=pk["tensor"])
        elif name in ("layernorm", "filter_gather", "filter_select"):
            e.update(bound="hbm", achieved=v["work"] / sec / 1e9, unit="GB/s", peak=pk["hbm"])
        if "achieved" in e:
            e["frac"] = e["achieved"] / e["peak"]
        brk[name] = e
    top = max(brk, key=lambda n: brk[n]["share"])
    roof = {"kernel": top, "bound": brk[top].get("bound"), "achieved": brk[top].get("achieved"),
            "peak": brk[top].get("peak"), "unit": "TFLOP/s" if brk[top].get("bound") == "tensor" else "GB/s",
            "frac": brk[top].get("frac"),
            "traffic": gemm_traffic(wl["name"]) if top == "gemm" else None,
            "peak_source": f"of {pk['source']} (sustained bf16 figure: the kernel is timed inside a long step)"}
    total_flops = fl["gemm"] + fl["attn_patch"] + fl["attn_global"]
    line = {
        "metric": metric_name(wl), "value": value, "unit": "images/s", "n_gpus": world, "steps": steps, "warmup": n_warm,
        "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": wl["name"], "image": f"{side}x{side}", "batch_per_gpu": B, "grid": f"{g}x{g}",
                   "tokens": a["n_global"] + g * g, "block": c["block"], "radius": c["radius"],
                   "filter_layer": c["filter_layer"], "keep_ratio": c["keep_ratio"], "kept": k,
                   "parallelism": "replicas" if world > 1 else "single GPU",
                   "l2": "inputs larger than L2 (activations of one step exceed 126 MB)"},
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": images / (ms_e2e * 1e-3), "unit": "images/s",
                "h2d_bytes_per_step": img_host.numel() * 4, "d2h_bytes_per_step": out_host.numel() * 2},
        "roofline": roof, "breakdown": brk,
        "useful_tflops": total_flops * steps * world / (ms * 1e-3) / 1e12,
        "peak_hbm_bytes": peak_bytes,
    }
    if world == 1 and not args.no_cpu and not args.quick:
        cb = oracle_sample(wl, args.cpu_rows)
        line["cpu_baseline"] = {
            "value": cb["images_per_s"], "unit": "images/s", "cores": cb["cores"], "kind": "oracle",
            "sample": (f"{cb['rows']} token rows of each per-token op of one block, {cb['rows']} attention query "
                       f"rows at the full and post-filter token counts and {cb['rows']} patch-embedding rows of one "
                       f"image ({cb['sample_seconds']:.1f} s of CPU work), extrapolated linearly in rows"),
            "parts_s": cb["parts"]}
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------
# resolution sweep (ViT-L/16, batch 4): dense attention, neighbour-block sparse, sparse + filter
# --------------------------------------------------------------------------------------------
def run_sweep(args):
    """One JSON line per (image side, mode): images/s, peak HBM bytes, useful TFLOP/s and its fraction
    of the measured bf16 peak.  Dense attention is the same kernel with a radius that covers the grid."""
    import torch
    import paper_2601_12150_b200 as spv
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = spv.Context(0)
    pk = peaks()
    arch = synth.vit_l16()
    B = 4
    sides = [int(x) for x in args.sweep_sides.split(",")]
    for side in sides:
        g = side // arch["patch"]
        w = synth.vit_weights(2, arch, g, g)
        dw = ctx.make_vit_weights(w)
        del w
        img = torch.from_numpy(synth.tissue_batch(6, B, side, side, background_range=(0.3, 0.6))).to(dev)
        for mode in ("dense", "sparse", "sparse_filter"):
            cfg = dict(arch, attn_mode=synth.ATTN_DENSE if mode == "dense" else synth.ATTN_SPARSE, block=8, radius=1,
                       filter_layer=4 if mode == "sparse_filter" else 0, keep_ratio=0.5 if mode == "sparse_filter" else 1.0)
            wl = dict(name=f"vitl16_{side}_b{B}_{mode}", arch=arch, cfg=cfg, side=side, grid=g, batch=B)
            torch.cuda.empty_cache()
            torch.cuda.reset_peak_memory_stats()
            steps = args.steps if side <= 2048 else max(1, args.steps // 3)
            kept = None
            for _ in range(2 if side <= 2048 else 1):
                _, kept = ctx.vit_forward(cfg, dw, img, g, g)
            ctx.check()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for _ in range(steps):
                ctx.vit_forward(cfg, dw, img, g, g)
            e1.record()
            torch.cuda.synchronize()
            ctx.check()
            ms = e0.elapsed_time(e1) / steps
            fl = forward_flops(dict(wl, cfg=dict(cfg, radius=g if mode == "dense" else 1)),
                               None if kept is None else kept.cpu().numpy())
            useful = fl["gemm"] + fl["attn_patch"] + fl["attn_global"]
            print(json.dumps({"workload": wl["name"], "image": f"{side}x{side}", "tokens": 1 + g * g, "mode": mode,
                              "batch": B, "ms_per_step": ms, "images_per_s": B / (ms * 1e-3),
                              "useful_tflops": useful / (ms * 1e-3) / 1e12,
                              "frac_of_bf16_peak": useful / (ms * 1e-3) / 1e12 / pk["tensor"],
                              "attention_density": fl["attn_patch"] / max(1.0, forward_flops(
                                  dict(wl, cfg=dict(cfg, radius=g, filter_layer=0)), None)["attn_patch"]),
                              "peak_hbm_bytes": torch.cuda.max_memory_allocated(), "steps": steps}), flush=True)
        del dw, img


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--cpu-rows", type=int, default=16384, help="rows of the CPU-oracle sample")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--quick", action="store_true",
                    help="profiling aid: exactly --warmup warm-up steps, no end-to-end and no CPU leg")
    ap.add_argument("--sweep", action="store_true",
                    help="resolution sweep (dense / sparse / sparse+filter), one JSON line per point")
    ap.add_argument("--sweep-sides", default="224,448,1024,2048,3072,4096")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    wl = workload_config(args.workload)
    if args.impl == "reference":
        run_reference(args, wl, rank)
    else:
        run_gpu(args, wl, rank, world)


if __name__ == "__main__":
    main()
