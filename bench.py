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


def config_of(wl, world):
    a, c, g = wl["arch"], wl["cfg"], wl["grid"]
    k = g * g
    if c["filter_layer"] > 0:
        k = int(np.ceil(c["keep_ratio"] * g * g - 1e-9))
    return {"workload": wl["name"], "image": f"{wl['side']}x{wl['side']}", "batch_per_gpu": wl["batch"], "grid": f"{g}x{g}",
            "tokens": a["n_global"] + g * g, "block": c["block"], "radius": c["radius"],
            "filter_layer": c["filter_layer"], "keep_ratio": c["keep_ratio"], "kept": k,
            "parallelism": "replicas" if world > 1 else "single GPU",
            "l2": "inputs larger than L2 (activations of one step exceed 126 MB)"}


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


# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per GEMM launch, averaged over the 100 GEMM
# launches of one step: four ncu captures, one per GEMM shape of a block at M = 65540 (two launches each),
# weighted by the step's launch counts, the half-size launches after the filter scaled by their rows
# (profiles/gemm_dram_by_shape_m65540.md).  Valid only for the kernel source it was taken with: reported as
# null once gemm.cu has changed.
GEMM_TRAFFIC = {"vitl16_2048_b4_sparse_filter": (393.6e6, "3ed141e24586")}


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
    rows = args.cpu_rows           # the same sample as the cpu_baseline leg of the GPU arm
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
        "config": config_of(wl, int(os.environ.get("WORLD_SIZE", "1"))),
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

    # ---- the same steps with a spatially coherent kept set: random weights scatter the kept tokens over the
    # blocks, the worst case for the block-sparse kernel; a trained backbone drops background.  forced_keep =
    # the k darkest patches of each image (the tissue).
    coh = None
    if c["filter_layer"] > 0 and not args.quick:
        fk_host = tissue_kept(img_host.numpy(), a["patch"], k)
        fk = torch.from_numpy(fk_host).to(dev)
        for _ in range(2):
            ctx.vit_forward(c, dw, img, g, g, out=out, forced_keep=fk)
        ctx.check()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        g0.record(stream)
        for _ in range(args.steps):
            ctx.vit_forward(c, dw, img, g, g, out=out, forced_keep=fk)
        g1.record(stream)
        barrier()
        ms_coh = g0.elapsed_time(g1)
        ctx.profile(True)
        for _ in range(args.steps):
            ctx.vit_forward(c, dw, img, g, g, out=out, forced_keep=fk)
        prof_coh = ctx.profile_read()
        ctx.profile(False)
        ctx.check()
        fl_coh = forward_flops(wl, fk_host)
        coh = {"kept": "the k darkest patches of each image (tissue), given as forced_keep",
               "images_per_s": B * args.steps / (ms_coh * 1e-3), "ms_per_step": ms_coh / args.steps,
               "attn_patch_ms_per_step": prof_coh["attn_patch"]["ms"] / args.steps,
               "attn_patch_useful_tflops": fl_coh["attn_patch"] * args.steps / (prof_coh["attn_patch"]["ms"] * 1e-3) / 1e12}

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
        "config": config_of(wl, world),
        "clocks": clocks, "gpu_launches": launches,
        "e2e": {"value": images / (ms_e2e * 1e-3), "unit": "images/s",
                "h2d_bytes_per_step": img_host.numel() * 4, "d2h_bytes_per_step": out_host.numel() * 2},
        "roofline": roof, "breakdown": brk,
        "useful_tflops": total_flops * steps * world / (ms * 1e-3) / 1e12,
        "peak_hbm_bytes": peak_bytes,
    }
    if coh is not None:
        coh["attn_patch_frac"] = coh["attn_patch_useful_tflops"] / pk["tensor"]
        line["coherent_kept"] = coh
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
# single-operation workloads: the hot-path kernels timed alone through the C ABI
# --------------------------------------------------------------------------------------------
def coherent_kept(seed, grid, keep):
    """A spatially coherent kept set (what Sec. 3.3 leaves on a real slide: background goes, tissue stays):
    the complement of a low-frequency background mask, exactly ceil(keep * grid^2) positions, ascending."""
    rng = np.random.Generator(np.random.PCG64(seed))
    n = grid * grid
    k = int(np.ceil(keep * n - 1e-9))
    bg = synth.background_mask(rng, grid, grid, 1.0 - k / n, cell=32).reshape(-1)   # regions a few blocks wide
    kept = np.flatnonzero(~bg)[:k]
    if kept.size < k:
        kept = np.sort(np.concatenate([kept, np.flatnonzero(bg)[:k - kept.size]]))
    return kept.astype(np.int32)


def tissue_kept(images, patch, k):
    """[B, k] ascending positions of the k darkest patches of each image (mean of the green channel; ties to the
    lower index): on these images that is the tissue, i.e. the spatially coherent set a trained backbone's CLS
    scores would keep (Sec. 3.3 reports that the pruned tokens are background).  images: fp32 [B, 3, S, S]."""
    B, _, S, _ = images.shape
    g = S // patch
    m = images[:, 1].reshape(B, g, patch, g, patch).mean(axis=(2, 4)).reshape(B, g * g)
    order = np.argsort(m, axis=1, kind="stable")[:, :k]
    return np.sort(order, axis=1).astype(np.int32)


def block_major(pos, grid, block):
    """Positions reordered by (block row, block column, position): the order vit_forward keeps internally."""
    return pos[np.lexsort((pos, (pos % grid) // block, (pos // grid) // block))]


OP_WORKLOADS = {
    # attention: (grid, block, radius, batch, heads, kept, pattern)
    "attn_28x28_b1": ("attn", dict(grid=28, block=7, radius=1, batch=1, heads=16)),
    "attn_28x28_b64": ("attn", dict(grid=28, block=7, radius=1, batch=64, heads=16)),
    "attn_128x128_b4_r1": ("attn", dict(grid=128, block=8, radius=1, batch=4, heads=16)),
    "attn_128x128_b4_r2": ("attn", dict(grid=128, block=8, radius=2, batch=4, heads=16)),
    "attn_128x128_b4_r3": ("attn", dict(grid=128, block=8, radius=3, batch=4, heads=16)),
    "attn_128x128_b2_dense": ("attn", dict(grid=128, block=8, radius=16, batch=2, heads=16)),
    "attn_128x128_b4_keep50_scattered": ("attn", dict(grid=128, block=8, radius=1, batch=4, heads=16, keep=0.5,
                                                      pattern="scattered")),
    "attn_128x128_b4_keep50_coherent": ("attn", dict(grid=128, block=8, radius=1, batch=4, heads=16, keep=0.5,
                                                     pattern="coherent")),
    # 16x16-patch blocks, same 3x3 neighbourhood: a 128-row query tile lies inside one block (no warp-tile without
    # keys) and streams three times as many key tiles per CTA as with 8x8 blocks
    "attn_128x128_b4_block16_r1": ("attn", dict(grid=128, block=16, radius=1, batch=4, heads=16)),
    "attn_128x128_b4_block16_keep50_scattered": ("attn", dict(grid=128, block=16, radius=1, batch=4, heads=16, keep=0.5,
                                                              pattern="scattered")),
    # filter: (grid, batch, heads, dim, keep, cold L2)
    "filter_64x64_b1": ("filter", dict(grid=64, batch=1, heads=16, dim=1024, keep=0.5, cold=False)),
    "filter_64x64_b1_cold": ("filter", dict(grid=64, batch=1, heads=16, dim=1024, keep=0.5, cold=True)),
    "filter_256x256_b4": ("filter", dict(grid=256, batch=4, heads=16, dim=1024, keep=0.5, cold=False)),
    # GEMMs of one ViT-L/16 block at 2048x2048, batch 4 (M = 4 * 16385 rows)
    "gemm_qkv_65540": ("gemm", dict(m=65540, n=3072, k=1024, epi="bias")),
    "gemm_out_65540": ("gemm", dict(m=65540, n=1024, k=1024, epi="resid")),
    "gemm_fc1_65540": ("gemm", dict(m=65540, n=4096, k=1024, epi="gelu")),
    "gemm_fc2_65540": ("gemm", dict(m=65540, n=1024, k=4096, epi="resid")),
    # LayerNorm at the full and post-filter row counts
    "ln_65540x1024": ("ln", dict(rows=65540, dim=1024)),
    "ln_32772x1024": ("ln", dict(rows=32772, dim=1024)),
}


def time_op(torch, fn, iters, flush=None):
    """Mean device time of fn() in ms over `iters` calls (CUDA events on the current stream, after three
    warm-up calls).  With `flush` (a buffer larger than L2) every call is preceded by a write of that buffer
    and timed by its own event pair, so that the operands come from HBM."""
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    if flush is None:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters
    tot = 0.0
    for _ in range(iters):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        tot += e0.elapsed_time(e1)
    return tot / iters


def run_op(args, name):
    """One JSON line for a single-operation workload: the rate in the roofline's unit, the roofline object
    (useful FLOP or algorithmic bytes / CUDA-event time / measured peak) and the oracle timed on the same
    operation (a bounded sample of it)."""
    import torch
    import oracle
    import paper_2601_12150_b200 as spv
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = spv.Context(0)
    pk = peaks()
    kind, o = OP_WORKLOADS[name]
    iters = max(args.steps, 1) * 5
    launches0 = ctx.launch_count()
    cfg = {"workload": name}
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
    sampler.start()
    if kind == "attn":
        g, b, r, B, H = o["grid"], o["block"], o["radius"], o["batch"], o["heads"]
        pos_dev, pos_host, order = None, None, spv.TOKENS_ROW_MAJOR
        if "keep" in o:
            rows = []
            for i in range(B):
                if o["pattern"] == "scattered":
                    rng = np.random.Generator(np.random.PCG64(100 + i))
                    kept = np.sort(rng.choice(g * g, size=int(np.ceil(o["keep"] * g * g - 1e-9)), replace=False)).astype(np.int32)
                else:
                    kept = coherent_kept(200 + i, g, o["keep"])
                rows.append(block_major(kept, g, b))
            pos_host = np.stack(rows)
            pos_dev = torch.from_numpy(pos_host).to(dev)
            order = spv.TOKENS_BLOCK_MAJOR
            n_patch = pos_host.shape[1]
        else:
            n_patch = g * g
            if g >= 64:          # the layout vit_forward uses: block-major tokens inside the fused QKV buffer
                order = spv.TOKENS_BLOCK_MAJOR
                pos_host = np.stack([block_major(np.arange(g * g, dtype=np.int32), g, b)] * B)
                pos_dev = torch.from_numpy(pos_host).to(dev)
        n = 1 + n_patch
        gen = torch.Generator(device=dev).manual_seed(1)
        qkv = torch.randn((B, n, 3, H, 64), device=dev, generator=gen).to(torch.bfloat16)
        q, k, v = qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2]
        out = torch.empty_strided(q.shape, q.stride(), dtype=q.dtype, device=dev)
        ctx.spatial_block_attention(q, k, v, g, g, b, r, patch_pos=pos_dev, token_order=order, want_scores=False, out=out)
        ctx.check()
        ctx.profile(True)
        for _ in range(iters):
            ctx.spatial_block_attention(q, k, v, g, g, b, r, patch_pos=pos_dev, token_order=order, want_scores=False, out=out)
        prof = ctx.profile_read()
        ctx.profile(False)
        ctx.check()
        ms_patch = prof["attn_patch"]["ms"] / iters
        ms_all = sum(p_["ms"] for p_ in prof.values()) / iters
        pairs = sum(attention_pairs(g, g, b, r, 1, None if pos_host is None else pos_host[i])[0] for i in range(B))
        flop = 4.0 * 64 * H * pairs
        achieved = flop / (ms_patch * 1e-3) / 1e12
        cfg.update(grid=f"{g}x{g}", block=b, radius=r, batch=B, heads=H, tokens=n,
                   token_order="block-major" if order == spv.TOKENS_BLOCK_MAJOR else "row-major",
                   l2="inputs larger than L2" if qkv.numel() * 2 > 126e6 else "warm L2 (Q, K, V fit in L2)",
                   ms_patch_kernel=ms_patch, ms_whole_call=ms_all,
                   mean_tokens_per_block=n_patch / (-(-g // b)) ** 2)
        value, unit = achieved, "useful TFLOP/s (patch-query kernel)"
        roof = dict(kernel="attn_patch_kernel", bound="tensor", achieved=achieved, peak=pk["tensor_burst"], unit="TFLOP/s",
                    frac=achieved / pk["tensor_burst"], traffic=None,
                    peak_source=f"of {pk['source']} (burst bf16 figure: the kernel is timed alone)",
                    frac_of_sustained=achieved / pk["tensor"])
        # oracle: sampled query rows of image 0
        nrow = min(n, 256 if n > 4096 else 785)
        qh, kh, vh = (x_[:1].float().cpu().numpy() for x_ in (q, k, v))
        rows = np.unique(np.linspace(0, n - 1, nrow).astype(np.int32))
        t0 = time.perf_counter()
        oracle.attention(qh, kh, vh, g, g, b, r, patch_pos=None if pos_host is None else pos_host[:1], rows=rows)
        dt = time.perf_counter() - t0
        cpu_rate = (flop / B) * (rows.size / n) / dt / 1e12
        cpu = dict(value=cpu_rate, unit="useful TFLOP/s", cores=oracle.num_threads(), kind="oracle",
                   sample=f"{rows.size} query rows of image 0, all heads ({dt:.1f} s)")
    elif kind == "filter":
        g, B, H, D, keep = o["grid"], o["batch"], o["heads"], o["dim"], o["keep"]
        NP = g * g
        sc_h = synth.filter_scores(1, B, H, g, g)
        tok_h = synth.token_rows(1, B, 1 + NP, D) if B * NP <= 65536 else None      # uint16 bf16 bit patterns
        sc = torch.from_numpy(sc_h).to(dev)
        if tok_h is not None:
            tok = torch.from_numpy(tok_h.view(np.int16)).to(dev).view(torch.bfloat16)
        else:
            tok = torch.randn((B, 1 + NP, D), device=dev, generator=torch.Generator(device=dev).manual_seed(2)).to(torch.bfloat16)
        kk = spv.filter_keep_count(NP, keep)
        out = torch.empty((B, 1 + kk, D), dtype=torch.bfloat16, device=dev)
        kept = torch.empty((B, kk), dtype=torch.int32, device=dev)
        fn = lambda: ctx.cls_score_topk_filter(sc, tok, 1, keep, tokens_out=out, kept_idx=kept)
        flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if o["cold"] else None
        ms = time_op(torch, fn, iters, flush)
        ctx.check()
        ctx.profile(True)
        for _ in range(iters):
            if flush is not None:
                flush.zero_()
            fn()
        prof = ctx.profile_read()
        ctx.profile(False)
        nbytes = B * (H * NP * 4 + 2 * (1 + kk) * D * 2 + kk * 4)
        achieved = nbytes / (ms * 1e-3) / 1e9
        gather_gbs = prof["filter_gather"]["work"] / (prof["filter_gather"]["ms"] * 1e-3) / 1e9
        cfg.update(grid=f"{g}x{g}", batch=B, heads=H, dim=D, keep_ratio=keep, kept=kk, algorithmic_bytes=nbytes,
                   l2=("L2 flushed before every call (256 MB written)" if o["cold"] else
                       ("inputs larger than L2" if nbytes > 126e6 else "warm L2 (the operands fit in L2)")),
                   ms_select=prof["filter_select"]["ms"] / iters, ms_gather=prof["filter_gather"]["ms"] / iters,
                   gather_gbs=gather_gbs)
        value, unit = achieved, "GB/s (whole call: head mean + select + gather)"
        roof = dict(kernel="filter_gather", bound="hbm", achieved=gather_gbs, peak=pk["hbm"], unit="GB/s",
                    frac=gather_gbs / pk["hbm"], traffic=None, peak_source=f"of {pk['source']}")
        t0 = time.perf_counter()
        oracle.token_filter(sc_h[:1], None if tok_h is None else tok_h[:1], n_global=1, keep_ratio=keep)
        dt = time.perf_counter() - t0
        per_img = nbytes / B if tok_h is not None else H * NP * 4 + kk * 4
        cpu = dict(value=per_img / dt / 1e9, unit="GB/s", cores=oracle.num_threads(), kind="oracle",
                   sample=f"image 0 ({'ranking and row gather' if tok_h is not None else 'ranking only'}, {dt:.2f} s)")
    elif kind == "gemm":
        M, N, K = o["m"], o["n"], o["k"]
        gen = torch.Generator(device=dev).manual_seed(3)
        a = (torch.randn((M, K), device=dev, generator=gen)).to(torch.bfloat16)
        w = (torch.randn((N, K), device=dev, generator=gen) * 0.02).to(torch.bfloat16)
        bias = torch.randn(N, device=dev, generator=gen)
        if o["epi"] == "resid":
            outb = torch.zeros((M, N), dtype=torch.float32, device=dev)
            scale = torch.full((N,), 0.1, device=dev)
            fn = lambda: ctx.gemm_bf16(a, w, outb, spv.EPI_BIAS_SCALE_RESID, bias=bias, scale=scale)
            out_bytes = M * N * 4 * 2
        else:
            outb = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
            epi = spv.EPI_BIAS_GELU if o["epi"] == "gelu" else spv.EPI_BIAS
            fn = lambda: ctx.gemm_bf16(a, w, outb, epi, bias=bias)
            out_bytes = M * N * 2
        ms = time_op(torch, fn, iters)
        ctx.check()
        flop = 2.0 * M * N * K
        achieved = flop / (ms * 1e-3) / 1e12
        cfg.update(m=M, n=N, k=K, epilogue=o["epi"], l2="operands and output larger than L2",
                   algorithmic_bytes=2 * (M * K + N * K) + out_bytes)
        value, unit = achieved, "TFLOP/s"
        roof = dict(kernel="gemm_bf16_kernel", bound="tensor", achieved=achieved, peak=pk["tensor_burst"], unit="TFLOP/s",
                    frac=achieved / pk["tensor_burst"], traffic=None,
                    peak_source=f"of {pk['source']} (burst bf16 figure: the kernel is timed alone)",
                    frac_of_sustained=achieved / pk["tensor"])
        rows = 256
        ah = a[:rows].float().cpu().numpy()
        wh = w.float().cpu().numpy()
        oracle.linear(ah[:8], wh, None)
        t0 = time.perf_counter()
        oracle.linear(ah, wh, bias.cpu().numpy())
        dt = time.perf_counter() - t0
        cpu = dict(value=2.0 * rows * N * K / dt / 1e12, unit="TFLOP/s", cores=oracle.num_threads(), kind="oracle",
                   sample=f"{rows} rows of A against the whole weight ({dt:.2f} s), without the activation")
    else:
        R, D = o["rows"], o["dim"]
        gen = torch.Generator(device=dev).manual_seed(4)
        x = torch.randn((R, D), device=dev, generator=gen)
        gam = torch.randn(D, device=dev, generator=gen)
        bet = torch.randn(D, device=dev, generator=gen)
        y = torch.empty((R, D), dtype=torch.bfloat16, device=dev)
        fn = lambda: ctx.layernorm(x, gam, bet, 1e-6, out=y)
        ms = time_op(torch, fn, iters)
        ctx.check()
        nbytes = R * D * 6
        achieved = nbytes / (ms * 1e-3) / 1e9
        cfg.update(rows=R, dim=D, algorithmic_bytes=nbytes, l2="input + output larger than L2")
        value, unit = achieved, "GB/s"
        roof = dict(kernel="layernorm_kernel", bound="hbm", achieved=achieved, peak=pk["hbm"], unit="GB/s",
                    frac=achieved / pk["hbm"], traffic=None, peak_source=f"of {pk['source']}")
        rows = min(R, 16384)
        xh = x[:rows].cpu().numpy()
        t0 = time.perf_counter()
        oracle.layernorm(xh, gam.cpu().numpy(), bet.cpu().numpy(), 1e-6)
        dt = time.perf_counter() - t0
        cpu = dict(value=rows * D * 6 / dt / 1e9, unit="GB/s", cores=oracle.num_threads(), kind="oracle",
                   sample=f"{rows} rows ({dt:.2f} s)")
    clocks = sampler.stop()
    print(json.dumps({"metric": name, "value": value, "unit": unit, "n_gpus": 1, "steps": iters, "warmup": 3,
                      "higher_is_better": True, "dtype": "bf16", "data": "synthetic", "config": cfg, "clocks": clocks,
                      "gpu_launches": ctx.launch_count() - launches0, "roofline": roof, "cpu_baseline": cpu}))


def run_microbench(args):
    """The hardware rates the attention kernel's design is argued from, one JSON line per probe."""
    import torch
    import paper_2601_12150_b200 as spv
    torch.cuda.set_device(0)
    ctx = spv.Context(0)

    def emit(name, r, unit, **extra):
        sm = r["sm_count"]
        print(json.dumps(dict(probe=name, per_clk_per_sm=r["units"] / r["cycles"] / sm, unit=unit + " / clk / SM",
                              per_second=r["units"] / (r["ms"] * 1e-3), sm_mhz=r["cycles"] / r["ms"] / 1e3,
                              ms=r["ms"], **extra)), flush=True)
    for cps, thr in ((1, 128), (1, 512), (2, 1024)):
        emit(f"ex2 ctas/SM={cps} threads={thr}", ctx.microbench("ex2", ctas_per_sm=cps, threads=thr, iters=4000), "ex2")
    for poly in (0, 2, 4):
        for cps, thr in ((2, 128), (3, 128), (2, 256)):
            emit(f"softmax_body poly={poly}/8 ctas/SM={cps} threads={thr}",
                 ctx.microbench("softmax_body", ctas_per_sm=cps, threads=thr, iters=500, poly_per_8=poly), "score")
    for kind in ("mma_ss", "mma_ts"):
        for m, n in ((128, 64), (64, 64), (128, 128), (128, 256)):
            for iss in (1, 2, 4):
                if iss * n + 32 > 512:
                    continue
                r = ctx.microbench(kind, m=m, n=n, iters=2000, issuers=iss)
                emit(f"{kind} m={m} n={n} k=16 issuing warps={iss}", r, "FLOP",
                     cycles_per_instruction_per_issuer=r["cycles"] / 8000)
    for cps in (1, 2):
        for rows, st in ((64, 4), (128, 4), (256, 2)):
            emit(f"l2_tma ctas/SM={cps} box={rows}x128B stages={st}",
                 ctx.microbench("l2_tma", ctas_per_sm=cps, box_rows=rows, stages=st, iters=4000), "byte")
    ctx.check()


# --------------------------------------------------------------------------------------------
# ablation axes of the paper (Tables 2, 3, 5) as throughput sweeps: pruning ratio, window (block) size,
# neighbourhood radius, number of global tokens, and filtering in two stages
# --------------------------------------------------------------------------------------------
def run_ablation(args):
    """ViT-L/16 at 2048x2048, batch 4, one factor varied at a time around (block 8, radius 1, keep 0.5 after
    block 4, one global token).  One JSON line per point: images/s, time and useful TFLOP/s of the patch-query
    attention kernel, and the mean number of surviving tokens per spatial block after the filter."""
    import torch
    import paper_2601_12150_b200 as spv
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    ctx = spv.Context(0)
    pk = peaks()
    side, B = args.ablation_side, 4
    base_arch = synth.vit_l16()
    g = side // base_arch["patch"]
    img = torch.from_numpy(synth.tissue_batch(6, B, side, side, background_range=(0.3, 0.6))).to(dev)
    points = [("keep_ratio", kr, dict(keep=kr)) for kr in (0.6, 0.5, 0.4, 0.3, 0.2)]
    points += [("block", b, dict(block=b)) for b in (2, 8, 16, 64)]
    points += [("radius", r, dict(radius=r)) for r in (0, 1, 2, 3)]
    points += [("n_global", G, dict(G=G)) for G in (1, 5, 9)]
    points += [("filters", "4:0.7,12:0.7", dict(filters=[(4, 0.7), (12, 0.7)])),
               ("filters", "4:0.5", dict(filters=[(4, 0.5)])),
               ("unfused_filter", 1, dict(unfused=1)), ("unfused_filter", 0, dict(unfused=0))]
    weights = {}
    for axis, val, o in points:
        G = o.get("G", 1)
        arch = dict(base_arch, n_global=G)
        if G not in weights:
            weights.clear()
            torch.cuda.empty_cache()
            weights[G] = ctx.make_vit_weights(synth.vit_weights(2, arch, g, g))
        dw = weights[G]
        stages = o.get("filters", [(4, o.get("keep", 0.5))])
        cfg = dict(arch, attn_mode=synth.ATTN_SPARSE, block=o.get("block", 8), radius=o.get("radius", 1), filters=stages,
                   unfused_filter=o.get("unfused", 0))
        wl = dict(name="ablation", arch=arch, cfg=dict(cfg, filter_layer=stages[0][0], keep_ratio=stages[0][1]),
                  side=side, grid=g, batch=B)
        kept = None
        for _ in range(2):
            _, kept = ctx.vit_forward(cfg, dw, img, g, g)
        ctx.check()
        steps = max(1, args.steps // 2)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            ctx.vit_forward(cfg, dw, img, g, g)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        ctx.profile(True)
        for _ in range(steps):
            ctx.vit_forward(cfg, dw, img, g, g)
        prof = ctx.profile_read()
        ctx.profile(False)
        ctx.check()
        kept_h = kept.cpu().numpy()
        # useful attention FLOP of one step: stage boundaries split the layers
        counts, cur = [], g * g
        for _, ratio in stages:
            cur = spv.filter_keep_count(cur, ratio)
            counts.append(cur)
        H = arch["heads"]
        flop, prev_layer, off = 0.0, 0, 0
        pos_sets = [None]
        for c in counts:
            pos_sets.append([kept_h[b, off:off + c] for b in range(B)])
            off += c
        bounds = [l for l, _ in stages] + [arch["layers"]]
        for si, upto in enumerate(bounds):
            n_layers = upto - prev_layer
            prev_layer = upto
            for b in range(B):
                pp, _ = attention_pairs(g, g, cfg["block"], cfg["radius"], G, None if pos_sets[si] is None else pos_sets[si][b])
                flop += n_layers * 4.0 * 64 * H * pp
        nblocks = (-(-g // cfg["block"])) ** 2
        attn_ms = prof["attn_patch"]["ms"] / steps
        print(json.dumps({"axis": axis, "value": val, "image": f"{side}x{side}", "batch": B, "block": cfg["block"],
                          "radius": cfg["radius"], "n_global": G, "filters": stages, "kept_final": counts[-1],
                          "mean_survivors_per_block": counts[-1] / nblocks, "ms_per_step": ms,
                          "images_per_s": B / (ms * 1e-3), "attn_patch_ms_per_step": attn_ms,
                          "attn_useful_tflops": flop / (attn_ms * 1e-3) / 1e12,
                          "attn_frac_of_sustained_bf16": flop / (attn_ms * 1e-3) / 1e12 / pk["tensor"],
                          "gemm_ms_per_step": prof["gemm"]["ms"] / steps,
                          "filter_select_ms_per_step": prof["filter_select"]["ms"] / steps,
                          "attn_global_ms_per_step": prof["attn_global"]["ms"] / steps, "steps": steps}), flush=True)


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
            # small images are bound by the ~240 launches of a forward: the same call captured once in a
            # CUDA graph and replayed (vit_forward only enqueues work on its stream)
            ms_graph = None
            if side <= args.sweep_graph_max_side:
                out, _ = ctx.vit_forward(cfg, dw, img, g, g)
                st = torch.cuda.Stream()
                st.wait_stream(torch.cuda.current_stream())
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(st):
                    with torch.cuda.graph(graph, stream=st):
                        ctx.vit_forward(cfg, dw, img, g, g, out=out, stream=st)
                graph.replay()
                torch.cuda.synchronize()
                e0.record()
                for _ in range(steps):
                    graph.replay()
                e1.record()
                torch.cuda.synchronize()
                ctx.check()
                ms_graph = e0.elapsed_time(e1) / steps
                del graph
            fl = forward_flops(dict(wl, cfg=dict(cfg, radius=g if mode == "dense" else 1)),
                               None if kept is None else kept.cpu().numpy())
            useful = fl["gemm"] + fl["attn_patch"] + fl["attn_global"]
            print(json.dumps({"workload": wl["name"], "image": f"{side}x{side}", "tokens": 1 + g * g, "mode": mode,
                              "batch": B, "ms_per_step": ms, "images_per_s": B / (ms * 1e-3),
                              "ms_per_step_graph_replay": ms_graph,
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
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS) + sorted(OP_WORKLOADS))
    ap.add_argument("--microbench", action="store_true", help="hardware rate probes, one JSON line each")
    ap.add_argument("--sweep-ablation", action="store_true",
                    help="keep ratio / block / radius / global tokens / two filter stages, one JSON line per point")
    ap.add_argument("--ablation-side", type=int, default=2048)
    ap.add_argument("--cpu-rows", type=int, default=8192, help="rows of the CPU-oracle sample (both arms)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle leg")
    ap.add_argument("--quick", action="store_true",
                    help="profiling aid: exactly --warmup warm-up steps, no end-to-end and no CPU leg")
    ap.add_argument("--sweep", action="store_true",
                    help="resolution sweep (dense / sparse / sparse+filter), one JSON line per point")
    ap.add_argument("--sweep-sides", default="224,448,1024,2048,3072,4096")
    ap.add_argument("--sweep-graph-max-side", type=int, default=2048,
                    help="largest image side of the sweep that is also timed as a CUDA-graph replay")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.microbench:
        run_microbench(args)
        return
    if args.sweep_ablation:
        run_ablation(args)
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus != world:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE is {world}: launch N > 1 with "
                         "python -m torch.distributed.run --nproc-per-node N bench.py --gpus N")
    if args.workload in OP_WORKLOADS:
        if args.impl == "reference" or world > 1:
            raise SystemExit("single-operation workloads run on one GPU with --impl ours")
        run_op(args, args.workload)
        return
    wl = workload_config(args.workload)
    if args.impl == "reference":
        run_reference(args, wl, rank)
    else:
        run_gpu(args, wl, rank, world)


if __name__ == "__main__":
    main()
