#!/usr/bin/env python
"""Throughput of the IPGS carve path (TokenCarve Sec. 3.3) on synthetic LLaVA-1.5-shaped inputs.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one tc_carve over a batch of images (score -> prune -> match -> merge -> gather).
For N > 1 launch under torch.distributed.run; every rank carves its own batch (images are
independent, so there is no collective on the path) and rank 0 prints one JSON line.
`--impl reference` times the float64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2503_10501_b200 import inputs, sharding  # noqa: E402

METRIC = "IPGS carve images/s (N=576,d=4096,fp16,keep 128)"
UNIT = "images/s"


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            m = json.load(f)
        return {"hbm_gbs": float(m["hbm_gbs"]), "bf16_tflops": float(m["bf16_tflops"]),
                "bf16_tflops_sustained": float(m.get("bf16_tflops_sustained", m["bf16_tflops"])),
                "sm_max_mhz": float(m.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
            "sm_max_mhz": 1965.0, "source": "fallback"}


CONFIG_KEYS = {"cfg1": "cfg1_single_f32", "cfg2": "cfg2_llava7b_f16", "cfg3": "cfg3_llava13b_f16",
               "cfg4": "cfg4_anyres_f16", "cfg5": "cfg5_sweep_f16"}


def workload(args, rank=0):
    """The metric's workload (cfg5 at B=64, T=128, keep=128) unless --config names another of
    the five; --batch / --n-query / --keep override the named configuration's own values."""
    base = inputs.CONFIGS[CONFIG_KEYS[args.config]]
    if args.config == "cfg5":
        cfg = base.with_(batch=args.batch or 64, n_query=args.n_query or 128, keep=args.keep or 128)
    else:
        cfg = base.with_(batch=args.batch or base.batch, n_query=args.n_query or base.n_query,
                         keep=args.keep or base.keep)
    if args.rank_cap >= 0:
        cfg = cfg.with_(rank_cap=args.rank_cap)   # 0 = the full solve (no rank hint)
    name = (f"{cfg.name} B={cfg.batch} N={cfg.n_tokens} d={cfg.d_model} T={cfg.n_query} "
            f"keep={cfg.keep} rank_cap={cfg.rank_cap}")
    return cfg, name


def uses_tensor_products(cfg):
    """Whether the subspace solve of this configuration runs its products on the tensor cores
    (the library's own rule: a rank hint of 128, 144, 160 or 192 and N a multiple of 4)."""
    return cfg.rank_cap in (128, 144, 160, 192) and cfg.n_tokens % 4 == 0 and cfg.d_model * 4 <= 48 * 1024


def product_peak(pk):
    """float32-equivalent peak of the three-product TF32 kernel: the measured sustained bf16
    tensor throughput x 1/2 (nominal TF32 : bf16 ratio) / 3 (products per term)."""
    return pk["bf16_tflops_sustained"] * 0.5 / 3.0


def algorithmic_bytes_per_image(cfg, P):
    """O and A read once; P rows of X, K, V read and keep rows written."""
    e = 2 if cfg.dtype == "f16" else 4
    N, d, H, dh, T = cfg.n_tokens, cfg.d_model, cfg.n_heads, cfg.head_dim, cfg.n_query
    row = (d + 2 * H * dh) * e
    return N * d * e + H * T * N * e + (P + cfg.keep) * row


# ----------------------------------------------------------------------------- CPU oracle leg
def time_oracle(cfg, n_images, first_image=0, single_thread=False):
    """Seconds per image of the float64 oracle as it stands, and the BLAS threads it used."""
    from oracle import ipgs_oracle as orc
    import contextlib
    limit = contextlib.nullcontext()
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
        threads = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
        if single_thread:
            limit, threads = threadpool_limits(limits=1), 1
    except Exception:
        threads = os.cpu_count() or 1
    ims = [inputs.make_image(cfg, first_image + b) for b in range(n_images)]
    with limit:
        t0 = time.perf_counter()
        for im in ims:
            orc.carve(im["O"].astype(np.float64), im["A"].astype(np.float64), im["X"], im["K"], im["V"],
                      cfg.keep, cfg.rho, cfg.lam, cfg.rank_tol, "none")
        dt = time.perf_counter() - t0
    return dt / n_images, threads


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg, name = workload(args)
    n = args.cpu_images
    for _ in range(max(0, min(args.warmup, 1))):
        time_oracle(cfg, 1)
    per = []
    for s in range(args.steps):
        sec, threads = time_oracle(cfg, n, first_image=s * n)
        per.append(sec)
    sec = float(np.mean(per))
    val = 1.0 / sec
    sample = f"{n} images per step of the {cfg.batch}-image batch, float64 oracle (LAPACK SVD + loops)"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * n * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": name, "sample_images_per_step": n},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------------- clocks sampler
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self.stop = threading.Event()
        self.th = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        while not self.stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                      "--format=csv,noheader,nounits"], capture_output=True,
                                     text=True, timeout=5).stdout.strip()
                if out:
                    self.rows.append([c.strip() for c in out.split(",")])
            except Exception:
                pass
            self.stop.wait(0.2)

    def __enter__(self):
        self.th.start()
        return self

    def __exit__(self, *a):
        self.stop.set()
        self.th.join(timeout=6)

    def summary(self):
        sm = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names)
                   if any(len(r) > 3 + i and r[3 + i].lower().startswith("active") for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(self.rows)}


# ----------------------------------------------------------------------------- the CUDA arm
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2503_10501_b200 import binding as tcb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the carve path")
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    tcb.lib()
    use_graph = not args.no_graph
    cfg, name = workload(args)
    # concurrent image groups: measured best under graph replay is 16 at 64 images (8 at 16
    # images), the library's 4 otherwise
    groups = args.groups if args.groups else ((16 if cfg.batch >= 64 else 8) if use_graph else 4)
    tcb.tc_set_groups(groups)
    M, P, nA, nB = 0, 0, 0, 0
    p = tcb.Params(batch=cfg.batch, n_tokens=cfg.n_tokens, d_model=cfg.d_model, n_heads=cfg.n_heads,
                   head_dim=cfg.head_dim, n_query=cfg.n_query, keep=cfg.keep, rho=cfg.rho,
                   lam=cfg.lam, rank_tol=cfg.rank_tol, dtype=cfg.dtype, rank_cap=cfg.rank_cap)
    M, P, nA, nB = tcb.tc_counts(p)
    # each rank carves its own images (weak scaling): image numbers rank*B .. rank*B + B - 1
    batch = inputs.make_batch(cfg, images=sharding.image_range(rank, world, cfg.batch))
    hostin = {k: torch.from_numpy(v).pin_memory() for k, v in batch.items()}
    devin = {k: v.cuda(non_blocking=True) for k, v in hostin.items()}
    dt = p.torch_dtype
    mk = lambda *s, dtype=dt: torch.empty(*s, dtype=dtype, device="cuda")
    out = (mk(p.batch, p.keep, p.d_model), mk(p.batch, p.n_heads, p.keep, p.head_dim),
           mk(p.batch, p.n_heads, p.keep, p.head_dim), mk(p.batch, p.keep, dtype=torch.int32),
           mk(p.batch, dtype=torch.int32))
    hout = tuple(torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in out)
    ws = tcb.workspace(p, host=True)
    torch.cuda.synchronize()

    def step():
        tcb.tc_carve(p, devin["O"], devin["A"], devin["X"], devin["K"], devin["V"], ws, out)

    def step_host():
        tcb.tc_carve_host(p, hostin["O"], hostin["A"], hostin["X"], hostin["K"], hostin["V"], hout, ws)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        """Milliseconds for `steps` calls between one pair of events (max over ranks), and this
        rank's per-step times from an event after every call."""
        barrier()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record()
        for i in range(steps):
            fn()
            ev[i + 1].record()
        barrier()
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        return sharding.max_over_ranks(ev[0].elapsed_time(ev[steps]), device="cuda"), per

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    status = out[4].cpu().numpy()
    if status.any():
        raise SystemExit(f"carve reported per-image status {status.tolist()}")

    # The timed step replays a CUDA graph of one tc_carve call (same kernels, same streams: the
    # fork/join of the library's internal streams is captured as graph dependencies), which
    # takes the ~25 dependent launches of a group's chain off the host (a few per cent of the
    # step against plain calls, --no-graph).
    eager_step = step
    graph = None
    if use_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            eager_step()
        step = graph.replay
        for _ in range(2):
            step()
        torch.cuda.synchronize()
        status = out[4].cpu().numpy()
        if status.any():
            raise SystemExit(f"graph replay reported per-image status {status.tolist()}")

    # nvidia-smi is sampled (every 0.2 s) over the timed region and the two passes after it,
    # which run the same kernels: one timed region alone is shorter than a sampling period
    with ClockSampler(local) as cs:
        ms, per_step = timed(step, args.steps)
        launches0 = tcb.tc_launch_count()
        eager_step()
        launches = (tcb.tc_launch_count() - launches0) * args.steps  # same kernels per step

        # per-kernel-class device time (CUDA events on the launching stream), same steps again,
        # with the image groups run one after the other so that no two kernels share the GPU
        tcb.tc_set_groups(1)
        eager_step()
        tcb.tc_profile_begin()
        for _ in range(args.steps):
            eager_step()
        prof = tcb.tc_profile_end()
        tcb.tc_set_groups(groups)

        # end to end through the host-buffer entry point
        for _ in range(min(args.warmup, 2)):
            step_host()
        ms_host, _ = timed(step_host, args.steps)

        # Extra figure, not the headline: the same K steps with two of them in flight (two
        # graphs with a workspace and outputs each, replayed on alternating streams), as a
        # server with a queue of batches would run them.  One carve of 64 images is bound by
        # the latency of its dependent chain; the second batch fills the SMs it leaves idle.
        pipelined = None
        nfl = args.inflight
        if use_graph and world == 1 and nfl >= 2 and args.steps >= nfl:
            sA = torch.cuda.current_stream()
            lanes = [(graph, sA, out)]
            for _ in range(nfl - 1):
                wsx = tcb.workspace(p, host=True)
                outx = tuple(torch.empty_like(t) for t in out)
                sx = torch.cuda.Stream()
                sx.wait_stream(sA)
                with torch.cuda.stream(sx):   # warm-up outside capture
                    tcb.tc_carve(p, devin["O"], devin["A"], devin["X"], devin["K"], devin["V"], wsx, outx)
                sA.wait_stream(sx)
                torch.cuda.synchronize()
                gx = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gx):
                    tcb.tc_carve(p, devin["O"], devin["A"], devin["X"], devin["K"], devin["V"], wsx, outx)
                lanes.append((gx, sx, outx, wsx))

            def run_lanes(n):
                e0 = torch.cuda.Event(enable_timing=True)
                ends = [torch.cuda.Event(enable_timing=True) for _ in lanes]
                torch.cuda.synchronize()
                e0.record(sA)
                for ln in lanes[1:]:
                    ln[1].wait_event(e0)
                for i in range(n):
                    g_, s_ = lanes[i % nfl][0], lanes[i % nfl][1]
                    with torch.cuda.stream(s_):
                        g_.replay()
                for ln, e in zip(lanes, ends):
                    e.record(ln[1])
                torch.cuda.synchronize()
                return max(e0.elapsed_time(e) for e in ends)

            run_lanes(2 * nfl)
            ms2 = run_lanes(args.steps)
            same = all(torch.equal(a_, b_) for ln in lanes[1:] for a_, b_ in zip(out, ln[2]))
            pipelined = {"steps_in_flight": nfl, "value": cfg.batch * args.steps / (ms2 * 1e-3),
                         "unit": "images/s", "ms_per_step": ms2 / args.steps,
                         "outputs_equal_single": bool(same)}
    clocks = cs.summary()

    images = cfg.batch * world * args.steps
    value = images / (ms * 1e-3)
    e2e = images / (ms_host * 1e-3)
    nbytes = lambda ts: int(sum(t.numel() * t.element_size() for t in ts))
    pk = peaks()

    # roofline of the kernel class that takes the most device time per step
    k = p.rank_cap if p.rank_cap else p.n_tokens
    N = cfg.n_tokens
    alg_bytes_img = algorithmic_bytes_per_image(cfg, P)
    kfr = kernel_fractions(cfg, P, k, prof, args.steps, pk)
    top_name = max((n for n in prof if prof[n][1] and n in kfr), key=lambda n: prof[n][0])
    roof = {"kernel": top_name}
    roof.update({f: kfr[top_name][f] for f in ("bound", "achieved", "peak", "unit", "frac", "peak_source")})
    # DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of
    # this kernel at B=16, scaled by the batch: the traffic of these kernels grows in proportion);
    # null for a kernel that changed after its counters were taken
    ncu_dram_per_image = {"gram": (75.58e6 + 3.49e6) / 16, "attn_colsum": (75.52e6 + 1.38e6) / 16,
                          "compact": (75.56e6 + 18.61e6) / 16, "eig": 1.396e6 / 16,
                          "sketch": (75.51e6 + 1.85e6) / 16}
    same_shape = (cfg.n_tokens, cfg.d_model, cfg.n_query, cfg.keep, k, cfg.dtype) == \
        (576, 4096, 128, 128, 144, "f16")
    roof["traffic"] = (ncu_dram_per_image[top_name] * cfg.batch
                       if same_shape and top_name in ncu_dram_per_image else None)
    # the whole path against the slower of its HBM bytes and its Gram flops
    t_hbm = alg_bytes_img / (pk["hbm_gbs"] * 1e9)
    t_tensor = 2.0 * cfg.n_tokens ** 2 * cfg.d_model / (pk["bf16_tflops_sustained"] * 1e12)
    t_roof = max(t_hbm, t_tensor)
    us_img = ms * 1e3 / (cfg.batch * args.steps)
    path = {"roofline_us_per_image": t_roof * 1e6, "achieved_us_per_image": us_img,
            "frac": t_roof * 1e6 / us_img, "bound": "hbm" if t_hbm >= t_tensor else "tensor",
            "algorithmic_bytes_per_image": alg_bytes_img}

    if rank == 0:
        cpu = None
        if world == 1 and args.cpu_images > 0:
            sec, threads = time_oracle(cfg, args.cpu_images)
            n1 = max(1, args.cpu_images // 4)
            sec1, _ = time_oracle(cfg, n1, single_thread=True)
            cpu = {"value": 1.0 / sec, "unit": UNIT, "cores": threads, "kind": "oracle",
                   "sample": f"{args.cpu_images} images of the {cfg.batch}-image batch, "
                             "float64 oracle (LAPACK SVD + loops)",
                   "single_thread": {"value": 1.0 / sec1, "unit": UNIT, "cores": 1,
                                     "sample": f"{n1} images, BLAS limited to one thread"}}
        line = {"metric": METRIC if args.config == "cfg5" else "IPGS carve images/s", "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": name, "images_per_gpu": cfg.batch, "rank_cap": p.rank_cap,
                           "rank_tol": p.rank_tol, "lambda": p.lam, "rho": p.rho,
                           "l2": f"inputs ({nbytes(devin.values()) / 1e9:.2f} GB per step) "
                                 + ("exceed the 126 MB L2" if nbytes(devin.values()) > 126e6
                                    else "fit the 126 MB L2: cold-cache figures need a larger batch"),
                           "solver": ("full Jacobi / tridiagonal solve" if not p.rank_cap else
                                      "subspace solve, products on the tensor cores"
                                      if uses_tensor_products(cfg) else "subspace solve, float32 ALU products"),
                           "image_groups": groups,
                           "launch": "CUDA graph replay of one tc_carve" if use_graph else "plain calls"},
                "us_per_image": us_img,
                "ms_per_step_median": float(np.median(per_step)), "ms_per_step_min": float(min(per_step)),
                "e2e": {"value": e2e, "unit": UNIT,
                        "h2d_bytes_per_step": nbytes(hostin.values()),
                        "d2h_bytes_per_step": nbytes(hout)},
                "gpu_launches": int(launches), "clocks": clocks, "roofline": roof,
                "path_roofline": path,
                "kernel_ms_per_step": {k_: round(v[0] / args.steps, 4) for k_, v in prof.items() if v[1]},
                "kernel_roofline": kfr,
                "cpu_baseline": cpu}
        if pipelined is not None:
            line["steps_in_flight"] = pipelined
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------- sweep
def kernel_fractions(cfg, P, k, prof, steps, pk):
    """Roofline fraction of every profiled kernel class: algorithmic bytes (or flops) per launch
    over its event-timed duration, against the peak that bounds it: measured HBM copy bandwidth,
    measured sustained bf16 tensor throughput (scaled for the three-product TF32 kernel), or the
    FP32-ALU peak derived as 148 SMs x 128 lanes x 2 x the maximum SM clock."""
    e = 2 if cfg.dtype == "f16" else 4
    B, N, d, H, dh, T = cfg.batch, cfg.n_tokens, cfg.d_model, cfg.n_heads, cfg.head_dim, cfg.n_query
    src = pk["source"]
    hbm = (pk["hbm_gbs"] * 1e9, "hbm", 1e9, "GB/s", src)
    alu = (148 * 128 * 2 * pk["sm_max_mhz"] * 1e6, "alu", 1e12, "TFLOP/s",
           "derived: 148 SMs x 128 lanes x 2 x max SM clock")
    tens = (pk["bf16_tflops_sustained"] * 1e12, "tensor", 1e12, "TFLOP/s", src + " (sustained bf16)")
    tcp = uses_tensor_products(cfg)
    prod = (product_peak(pk) * 1e12, "tensor", 1e12, "TFLOP/s",
            src + " sustained bf16 x 1/2 (TF32) / 3 (products per float32 term)") if tcp else alu
    nt = (N + 127) // 128
    gram_tiles = nt * (nt + 1) // 2 if cfg.dtype == "f16" else nt * nt
    work = {  # class -> (algorithmic amount per launch, peak)
        "attn_colsum": (B * H * T * N * e, hbm),
        "sketch": (B * N * d * e, hbm),
        "compact": (B * (P + cfg.keep) * (d + 2 * H * dh) * e, hbm),
        "gram": (B * 2.0 * N * N * d, tens),
        "gemm_f32_GQ": (B * 2.0 * N * N * k, prod),
        "gemm_f32_YtY": (B * 1.0 * N * k * (k + 1), prod),  # symmetric result: upper triangle
        # Y R^-1 (R^-1 triangular: N k^2 per launch) x passes, plus one full back-transformation
        "gemm_f32_YRinv": (B * N * k * k * ((3 * 1.0 + 2.0) / 4 if tcp else 2.0 * 11.0 / 15.0), prod),
        "chol_inv": (B * (2.0 / 3.0) * k ** 3, alu),
        "eig": (B * (14.0 / 3.0) * k ** 3, alu),
    }
    out = {}
    for name, (ms_total, launches) in prof.items():
        if not launches or name not in work:
            continue
        amount, (peak, bound, scale, unit, psrc) = work[name]
        # a class launched several times per step (the products, chol_inv) does `amount` per
        # launch; its time per launch is the class total over its launches
        per_launch_s = ms_total * 1e-3 / launches
        if name == "sketch":  # one amount per step: the sketch kernel and the transposition after it
            per_launch_s = ms_total * 1e-3 / steps
        out[name] = {"bound": bound, "frac": round(amount / per_launch_s / peak, 4),
                     "achieved": round(amount / per_launch_s / scale, 3), "peak": round(peak / scale, 3),
                     "unit": unit, "peak_source": psrc, "ms_per_step": round(ms_total / steps, 4)}
        if name == "gram" and cfg.dtype == "f16":
            # the kernel issues the 128 x 128 tiles on or below the diagonal; the dense count
            # above credits it with the mirror images it only stores
            issued = B * gram_tiles * 2.0 * 128 * 128 * d
            out[name]["frac_issued"] = round(issued / per_launch_s / peak, 4)
            out[name]["achieved_issued"] = round(issued / per_launch_s / scale, 3)
            out[name]["frac"] = out[name]["frac_issued"]
            out[name]["achieved"] = out[name]["achieved_issued"]
            out[name]["frac_dense_equivalent"] = round(amount / per_launch_s / peak, 4)
    return out


def run_sweep(args):
    """One JSON line per point of the throughput sweep: text tokens T in {32,128,512} x keep in
    {64,128,192,288} at the bench batch; images/s and the roofline fraction of every kernel."""
    import torch
    from paper_2503_10501_b200 import binding as tcb

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the carve path")
    torch.cuda.set_device(0)
    tcb.lib()
    groups = args.groups if args.groups else 4
    tcb.tc_set_groups(groups)
    pk = peaks()
    base = inputs.CONFIGS["cfg5_sweep_f16"].with_(batch=args.batch or 64)
    if args.rank_cap >= 0:
        base = base.with_(rank_cap=args.rank_cap)
    dev = {k: torch.from_numpy(v).cuda() for k, v in inputs.make_batch(base, want="OXKV").items()}
    for T in (32, 128, 512):
        cfgT = base.with_(n_query=T)
        A = torch.from_numpy(inputs.make_batch(cfgT, want="A")["A"]).cuda()
        for keep in (64, 128, 192, 288):
            cfg = cfgT.with_(keep=keep)
            p = tcb.Params(batch=cfg.batch, n_tokens=cfg.n_tokens, d_model=cfg.d_model,
                           n_heads=cfg.n_heads, head_dim=cfg.head_dim, n_query=T, keep=keep,
                           rho=cfg.rho, lam=cfg.lam, rank_tol=cfg.rank_tol, dtype=cfg.dtype,
                           rank_cap=cfg.rank_cap)
            M, P, nA, nB = tcb.tc_counts(p)
            dt = p.torch_dtype
            mk = lambda *s, dtype=dt: torch.empty(*s, dtype=dtype, device="cuda")
            out = (mk(p.batch, keep, p.d_model), mk(p.batch, p.n_heads, keep, p.head_dim),
                   mk(p.batch, p.n_heads, keep, p.head_dim), mk(p.batch, keep, dtype=torch.int32),
                   mk(p.batch, dtype=torch.int32))
            ws = tcb.workspace(p)

            def step():
                tcb.tc_carve(p, dev["O"], A, dev["X"], dev["K"], dev["V"], ws, out)

            for _ in range(args.warmup):
                step()
            torch.cuda.synchronize()
            status = out[4].cpu().numpy()
            if status.any():
                raise SystemExit(f"T={T} keep={keep}: per-image status {status.tolist()}")
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(args.steps):
                step()
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            tcb.tc_set_groups(1)
            step()
            tcb.tc_profile_begin()
            for _ in range(args.steps):
                step()
            prof = tcb.tc_profile_end()
            tcb.tc_set_groups(groups)
            k = p.rank_cap if p.rank_cap else p.n_tokens
            alg = algorithmic_bytes_per_image(cfg, P)
            t_roof = max(alg / (pk["hbm_gbs"] * 1e9),
                         2.0 * cfg.n_tokens ** 2 * cfg.d_model / (pk["bf16_tflops_sustained"] * 1e12))
            us_img = ms * 1e3 / (cfg.batch * args.steps)
            print(json.dumps({
                "sweep_point": {"T": T, "keep": keep, "P": P, "M": M, "batch": cfg.batch},
                "images_per_s": round(cfg.batch * args.steps / (ms * 1e-3), 1),
                "us_per_image": round(us_img, 3), "ms_per_step": round(ms / args.steps, 4),
                "path_roofline_frac": round(t_roof * 1e6 / us_img, 4),
                "algorithmic_bytes_per_image": alg, "peak_source": pk["source"],
                "kernels": kernel_fractions(cfg, P, k, prof, args.steps, pk)}), flush=True)
            del out, ws
        del A
        torch.cuda.empty_cache()


# ----------------------------------------------------------------------------- the two side entries
def run_extras(args):
    """One JSON line each for tc_rank and tc_reassemble at the bench point (event-timed, inputs
    resident): the information-quantity curve of Sec. 3.2 at three token counts, and the
    re-assembled sequence of the layers after the compression."""
    import torch
    from paper_2503_10501_b200 import binding as tcb

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the carve path")
    torch.cuda.set_device(0)
    tcb.lib()
    pk = peaks()
    cfg, name = workload(args)
    p = tcb.Params(batch=cfg.batch, n_tokens=cfg.n_tokens, d_model=cfg.d_model, n_heads=cfg.n_heads,
                   head_dim=cfg.head_dim, n_query=cfg.n_query, keep=cfg.keep, rho=cfg.rho,
                   lam=cfg.lam, rank_tol=1e-2, dtype=cfg.dtype, rank_cap=cfg.rank_cap)
    batch = inputs.make_batch(cfg)
    dev = {k: torch.from_numpy(v).cuda() for k, v in batch.items()}
    out = tcb.tc_carve(p, dev["O"], dev["A"], dev["X"], dev["K"], dev["V"])
    Xo, kept = out[0], out[3]

    def timed(fn):
        for _ in range(args.warmup):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / args.steps

    e = 2 if cfg.dtype == "f16" else 4
    g = torch.Generator().manual_seed(1)
    for label, idx in (("all 576 tokens", None), ("the 128 kept tokens", kept),
                       ("288 random tokens", torch.stack([torch.randperm(cfg.n_tokens, generator=g)[:288]
                                                          for _ in range(cfg.batch)]).int().cuda())):
        n_sub = cfg.n_tokens if idx is None else idx.shape[1]
        ws = torch.empty(tcb.tc_rank_workspace_bytes(p, n_sub), dtype=torch.uint8, device="cuda")
        res = tcb.tc_rank(p, dev["O"], idx, ws)
        torch.cuda.synchronize()
        ms = timed(lambda: tcb.tc_rank(p, dev["O"], idx, ws))
        print(json.dumps({"entry": "tc_rank", "workload": name, "token_set": label,
                          "ms_per_call": round(ms, 4), "images_per_s": round(cfg.batch / (ms * 1e-3), 1),
                          "rank_of_image_0": int(res["rank"][0]), "status_any": bool(res["img_status"].any()),
                          "bytes_read_per_call": cfg.batch * n_sub * cfg.d_model * e}), flush=True)
    n_sys, n_text = 35, cfg.n_query
    L = n_sys + cfg.n_tokens + n_text
    Hs = torch.randn(cfg.batch, L, cfg.d_model, device="cuda").to(dev["X"].dtype)
    ms = timed(lambda: tcb.tc_reassemble(p, n_sys, n_text, Hs, Xo, kept))
    moved = 2 * cfg.batch * (n_sys + cfg.keep + n_text) * cfg.d_model * e
    print(json.dumps({"entry": "tc_reassemble", "workload": name, "n_sys": n_sys, "n_text": n_text,
                      "ms_per_call": round(ms, 4), "bytes_per_call": moved,
                      "roofline": {"bound": "hbm", "achieved": round(moved / (ms * 1e-3) / 1e9, 1),
                                   "peak": pk["hbm_gbs"], "unit": "GB/s",
                                   "frac": round(moved / (ms * 1e-3) / 1e9 / pk["hbm_gbs"], 4),
                                   "note": "the call also allocates its two outputs"}}), flush=True)


def run_probe(args):
    """One JSON line for the layer-2 probe (tc_probe) at the LLaVA-1.5 layout of the bench point:
    35 system + 576 visual + 64 prompt tokens, 32 heads x 128, the prompt rows probing; event-timed
    with the inputs resident (Q, K, V of a 64-image batch are 1.06 GB, larger than L2)."""
    import torch
    from paper_2503_10501_b200 import binding as tcb

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the probe")
    torch.cuda.set_device(0)
    tcb.lib()
    pk = peaks()
    B, H, dh, n_sys, N, n_text = args.batch or 64, 32, 128, 35, 576, 64
    L = n_sys + N + n_text
    g = torch.Generator(device="cuda").manual_seed(7)
    Q, K, V = (torch.randn(B, H, L, dh, device="cuda", generator=g).half() for _ in range(3))
    p = tcb.Params(batch=B, n_tokens=N, d_model=H * dh, n_heads=H, head_dim=dh, n_query=n_text, keep=128,
                   dtype="f16")
    n = __import__("ctypes").c_size_t(0)
    cp = p.c()
    tcb.lib().tc_probe_workspace_bytes(__import__("ctypes").byref(cp), n_sys, n_text, __import__("ctypes").byref(n))
    ws = torch.empty(int(n.value), dtype=torch.uint8, device="cuda")
    out = (torch.empty(B, N, H * dh, dtype=torch.float16, device="cuda"),
           torch.empty(B, H, n_text, N, dtype=torch.float16, device="cuda"),
           torch.empty(B, dtype=torch.int32, device="cuda"))

    def step():
        tcb.tc_probe(p, n_sys, n_text, n_sys + N, Q, K, V, ws=ws, out=out)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    if int(out[2].abs().sum()):
        raise SystemExit("probe reported a per-image status")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    # algorithmic flops: row i sees i + 1 keys; Q K^T and P V, 2 flops per multiply-add
    vis = sum(i + 1 for i in range(n_sys, n_sys + N))
    prb = sum(i + 1 for i in range(n_sys + N, L))
    flops = B * H * (4.0 * vis * dh + 2.0 * 2 * prb * dh)
    # issued: 128 x 128 key blocks up to the last row of each 128-row tile
    tiles = sum(((min(N, (t + 1) * 128) + n_sys - 1) // 128 + 1) for t in range((N + 127) // 128))
    issued = B * H * tiles * 2 * 2.0 * 128 * 128 * dh
    byts = (3 * Q.numel() + out[0].numel() + out[1].numel()) * 2 + 2 * V.numel() * 2
    print(json.dumps({
        "entry": "tc_probe", "workload": f"B={B} H={H} dh={dh} n_sys={n_sys} N={N} n_text={n_text} f16",
        "ms_per_call": round(ms, 4), "images_per_s": round(B / (ms * 1e-3), 1),
        "roofline": {"bound": "tensor", "achieved": round(flops / (ms * 1e-3) / 1e12, 2),
                     "achieved_issued": round(issued / (ms * 1e-3) / 1e12, 2),
                     "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s",
                     "frac": round(flops / (ms * 1e-3) / 1e12 / pk["bf16_tflops_sustained"], 4),
                     "peak_source": pk["source"] + " (sustained bf16)"},
        "hbm_bytes_per_call": byts,
        "hbm_frac": round(byts / (ms * 1e-3) / 1e9 / pk["hbm_gbs"], 4)}), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="cfg5", choices=sorted(CONFIG_KEYS),
                    help="which of the five named workloads (default: the metric's, cfg5)")
    ap.add_argument("--batch", type=int, default=0, help="images per GPU per step (0 = the configuration's)")
    ap.add_argument("--n-query", type=int, default=0)
    ap.add_argument("--keep", type=int, default=0)
    ap.add_argument("--rank-cap", type=int, default=-1,
                    help="override the workload's rank_cap; 0 = full solve without a rank hint")
    ap.add_argument("--graph", action="store_true", help="(the default; kept for old command lines)")
    ap.add_argument("--no-graph", action="store_true",
                    help="time plain tc_carve calls instead of the replay of a CUDA graph of one call")
    ap.add_argument("--groups", type=int, default=0, help="concurrent image groups (0 = library default)")
    ap.add_argument("--inflight", type=int, default=2,
                    help="extra figure: the timed steps again with this many of them in flight (0 = skip)")
    ap.add_argument("--cpu-images", type=int, default=12,
                    help="images the CPU oracle is timed on (0 = skip)")
    ap.add_argument("--sweep", action="store_true",
                    help="one line per point of the T x keep sweep instead of the bench line")
    ap.add_argument("--probe", action="store_true",
                    help="time the layer-2 probe (tc_probe) at the bench point's layout instead of the bench line")
    ap.add_argument("--extras", action="store_true",
                    help="time tc_rank and tc_reassemble at the bench point instead of the bench line")
    args = ap.parse_args()
    if args.probe:
        run_probe(args)
    elif args.extras:
        run_extras(args)
    elif args.sweep:
        run_sweep(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
