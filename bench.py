#!/usr/bin/env python
"""Benchmark of the AB-Training hot path on B200.

A step is one pass of the whole path over one batch of synthetic input at the ViT-B/16 MLP
shapes (W1 3072x768, W2 768x3072, rank 192, 50,432 token rows, bf16 storage / fp32
accumulation, K = 4 group copies):
  chain : ab_layer_forward + ab_layer_backward (dX, dA, dB) of both layers,
  sync  : ab_group_sync of both layers (mean of the K copies, W = Abar Bbar, truncated-SVD split).
`value` is the chain's algorithmic TFLOP/s, 6 N r (m+n) per layer, over the chain's share of
the timed steps (CUDA events inside every step); the sync is reported beside it as ms per
step.  `ms_per_step` covers both.  One process per GPU; ranks take independent batches (weak
scaling, no collective on the data path).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--rows R]
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "AB layer fwd+bwd TFLOP/s"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
R = 192
LAYERS = ((3072, 768), (768, 3072))
K_GROUPS = 4
# dram__bytes_read.sum + dram__bytes_write.sum of one chain_kernel launch (forward of W1, 50,432 rows), from the
# ncu capture summarised under profiles/; None until the kernel of that capture is current.
ROW_CHAIN_DRAM_BYTES_PER_LAUNCH = 352.5e6   # 79.5 MB read + 273.0 MB written


def chain_flops(N, layers=LAYERS, r=R):
    return sum(6.0 * N * r * (m + n) for m, n in layers)


def chain_bytes(N, layers=LAYERS):
    # every activation once: x in forward and backward, y out, dY in, dX out (bf16)
    return sum(2.0 * N * (3 * n + 2 * m) for m, n in layers)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm=d["hbm_gbs"], tc_burst=d["bf16_tflops"], tc_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, tc_burst=1590.0, tc_sustained=1400.0, source="fallback")


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.stop_flag, self.sm, self.reasons, self.max_sm = index, False, [], set(), None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_sm = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
                     0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}
            while not self.stop_flag:
                self.sm.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                bits = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                for b, nm in names.items():
                    if bits & b:
                        self.reasons.add(nm)
                time.sleep(0.002)
        except Exception as e:  # clocks are evidence, not a dependency of the measurement
            self.reasons.add(f"nvml_unavailable:{type(e).__name__}")

    def summary(self):
        return dict(sm_mhz=float(np.median(self.sm)) if self.sm else None, sm_max_mhz=self.max_sm,
                    reasons=sorted(self.reasons), samples=len(self.sm))


def make_inputs(rank, N):
    """Host-side synthetic inputs of both layers for one rank (seed depends on the rank)."""
    from paper_2405_01067_b200 import synth
    out = []
    for li in (1, 2):
        d = synth.vit_mlp(li, seed=rank_seed(rank), N=N, K=K_GROUPS)
        d["A_copies"] = synth.group_copies(d["A"], d["noise_A"], bf16=True)
        d["B_copies"] = synth.group_copies(d["B"], d["noise_B"], bf16=True)
        out.append(d)
    return out


def cpu_baseline(inputs, rows, sync_scale=8):
    """The CPU checker, as it stands, on a bounded sample: chain on the first `rows` rows of both
    layers; the group sync of a 1/sync_scale-size copy of the recipe (timed separately)."""
    from oracle import ab_oracle as orc
    from paper_2405_01067_b200 import synth
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count() or 1])
    except Exception:
        cores = os.cpu_count() or 1
    t0 = time.perf_counter()
    for d in inputs:
        x, dY = d["x"][:rows], d["dY"][:rows]
        orc.forward(x, d["A"], d["B"])
        orc.backward(x, dY, d["A"], d["B"])
    t_chain = time.perf_counter() - t0
    t0 = time.perf_counter()
    for i, (m, n) in enumerate(LAYERS):
        s = synth.vit_sync_matrix(1, i, m, n, K=K_GROUPS, scale=sync_scale)
        orc.group_sync(synth.group_copies(s["A"], s["noise_A"]), synth.group_copies(s["B"], s["noise_B"]), s["r"], 0.0)
    t_sync = time.perf_counter() - t0
    # for scale: the library SVD (LAPACK, float64) of one full-size recombined matrix of each shape
    lapack = {}
    rng = np.random.default_rng(0)
    for (m, n) in ((768, 768), (3072, 768)):
        W = rng.standard_normal((m, n // 4)) @ rng.standard_normal((n // 4, n))
        t0 = time.perf_counter()
        np.linalg.svd(W, full_matrices=False)
        lapack[f"{m}x{n}"] = time.perf_counter() - t0
    return dict(value=chain_flops(rows) / t_chain / 1e12, unit=UNIT, cores=int(cores), kind="oracle",
                sample=f"chain: first {rows} of 50432 rows of both layers, float64, {t_chain:.2f} s; "
                       f"sync: both matrices at 1/{sync_scale} scale, own Jacobi SVD, {t_sync:.2f} s; "
                       f"LAPACK SVD of one full-size matrix: 768x768 {lapack['768x768']:.2f} s, "
                       f"3072x768 {lapack['3072x768']:.2f} s",
                chain_s=t_chain, sync_sample_s=t_sync)


def run_reference(args):
    """--impl reference: the CPU checker timed on the host cores, same metric and config."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = args.ref_rows
    inputs = make_inputs(0, rows)
    for _ in range(args.warmup):
        cpu_baseline(inputs, min(rows, 512))
    t0 = time.perf_counter()
    last = None
    for _ in range(args.steps):
        last = cpu_baseline(inputs, rows)
    dt = (time.perf_counter() - t0) / args.steps
    chain_s = last["chain_s"]
    v = chain_flops(rows) / chain_s / 1e12
    line = dict(impl="reference", metric=METRIC, value=v, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=dt * 1e3, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="f64", data="synthetic",
                config=dict(workload="vit_b16_mlp_pair_r192 (bounded sample)", rows=rows, K=K_GROUPS, r=R,
                            same_config=False,
                            sample=f"first {rows} of 50432 rows of both layers per step (a rate: FLOP of the sample "
                                   "over its time); the GPU arm runs all 50432 rows"),
                cpu_baseline=dict(value=v, unit=UNIT, cores=last["cores"], kind="oracle", sample=last["sample"]),
                e2e=dict(value=v, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0), gpu_launches=0)
    print(json.dumps(line))


def rank_seed(rank):
    """Every rank draws its own batch: the path shards by independent batches (weak scaling)."""
    return 1 + 100 * rank


def max_over_ranks(values, device, world):
    """Slowest rank's times: element-wise MAX all-reduce (the only collective, outside the timed region)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_tflops(N, world, steps, chain_ms):
    """Aggregate chain throughput of all ranks: every rank does chain_flops(N) per step."""
    return chain_flops(N) * world * steps / (chain_ms * 1e-3) / 1e12


def vit_model_sync(ab, torch, steps=5):
    """Second part of the metric: group sync of a whole ViT-B/16 (72 matrices, fp32 factors, rank 25 %,
    K = 8 noisy copies in one packed arena per group, cutoff 0.1).  Returns ms per model for the mean
    alone (one streaming call over the arena) and for the whole sync, with the mean's HBM figures."""
    from paper_2405_01067_b200 import synth
    K = 8
    shapes = synth.vit_sync_shapes(12)
    sizes = [(m * min(m, n) // 4, min(m, n) // 4 * n) for m, n in shapes]
    total = sum(a + b for a, b in sizes)
    arena = torch.empty((K, total), dtype=torch.float32, device="cuda")
    off, views = 0, []
    cache = {}
    for i, (m, n) in enumerate(shapes):
        if (m, n) not in cache:            # one recipe per shape and block position keeps set-up short
            cache[(m, n)] = synth.vit_sync_matrix(3, len(cache), m, n, K=K)
        d = cache[(m, n)]
        r = d["r"]
        a_sz, b_sz = m * r, r * n
        for k in range(K):
            arena[k, off:off + a_sz] = torch.from_numpy(d["A"] + d["noise_A"][k]).reshape(-1).cuda()
            arena[k, off + a_sz:off + a_sz + b_sz] = torch.from_numpy(d["B"] + d["noise_B"][k]).reshape(-1).cuda()
        views.append((arena[:, off:off + a_sz].view(K, m, r), arena[:, off + a_sz:off + a_sz + b_sz].view(K, r, n)))
        off += a_sz + b_sz
    mean_out = torch.empty((total,), dtype=torch.float32, device="cuda")

    # the copies of a matrix are views into the arena: copy k sits one arena row further on
    plan = ab.SyncPlan([v[0] for v in views], [v[1] for v in views], 0.1, want_W=True, strided=True)

    def ev():
        return torch.cuda.Event(enable_timing=True)
    res = {}
    plan_now = ab.SyncPlan([v[0] for v in views], [v[1] for v in views], 0.1, want_W=False, strided=True)
    for name, fn in (("mean", lambda: ab.ab_group_average(arena, out=mean_out)), ("sync", lambda: ab.ab_group_sync(plan)),
                     ("sync_now", lambda: ab.ab_group_sync(plan_now))):
        for _ in range(2):
            fn()
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        res[name] = e0.elapsed_time(e1) / steps
    bad = int(plan.status.abs().sum().item())
    # the same model through the dense route (W formed, block Jacobi at short side 768): what a decomposition
    # costs when W is not of rank <= r any more; one warm-up, one timed call
    ab.ab_group_sync(plan_now, path=ab.AB_SYNC_DENSE)
    torch.cuda.synchronize()
    e0, e1 = ev(), ev()
    e0.record()
    ab.ab_group_sync(plan_now, path=ab.AB_SYNC_DENSE)
    e1.record()
    torch.cuda.synchronize()
    res["dense"] = e0.elapsed_time(e1)
    bad += int(plan_now.status.abs().sum().item())
    pk = measured_peaks()
    mean_bytes = (K + 1) * 4.0 * total
    return dict(workload="vit_b16_full_sync_72_matrices_fp32_K8_cutoff0.1", ms_per_model=res["sync"],
                ms_per_model_without_W=res["sync_now"], ms_per_model_dense_route=res["dense"], ms_per_matrix=res["sync"] / len(shapes),
                mean_ms=res["mean"], mean_gbs=mean_bytes / (res["mean"] * 1e-3) / 1e9,
                mean_frac_of_measured_hbm=mean_bytes / (res["mean"] * 1e-3) / 1e9 / pk["hbm"],
                mean_frac_of_nominal_8tbs=mean_bytes / (res["mean"] * 1e-3) / 1e9 / 8000.0,
                kept_ranks=sorted(set(plan.r_out.tolist())), device_status_errors=bad)


def other_workloads(ab, torch, iters=10):
    """The remaining layer shapes of the evaluation, one line each: forward + backward (dX, dA, dB) of one
    factorised layer, event-timed after warm-up, with the algorithmic FLOP and the minimum HBM bytes
    (each activation once: x twice, dY, y, dX) and the ceiling those give: min(tensor peak, intensity x HBM
    peak).  ResNet-50 layer3 3x3 conv as GEMM on materialised im2col rows; VGG16 512 x 4608 at ranks 8..64
    (the skinny, HBM-bound regime); the small fp32 layer (launch-latency bound, reported in us)."""
    from paper_2405_01067_b200 import synth
    pk = measured_peaks()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters

    def layer(d, bf16):
        dt = torch.bfloat16 if bf16 else torch.float32
        g = {k: torch.from_numpy(np.ascontiguousarray(d[k], dtype=np.float32)).to(dt).cuda() for k in ("x", "dY", "A", "B")}
        N, n = g["x"].shape
        m, r = g["A"].shape
        code = ab.AB_BF16 if bf16 else ab.AB_F32
        ws_f = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_LAYER_FORWARD, N, m, n, r, 1, code), "cuda")
        ws_b = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_LAYER_BACKWARD, N, m, n, r, 1, code), "cuda")
        y = torch.empty((N, m), dtype=dt, device="cuda")
        T = torch.empty((N, r), dtype=dt, device="cuda")
        dX = torch.empty((N, n), dtype=dt, device="cuda")
        dA = torch.empty((m, r), dtype=torch.float32, device="cuda")
        dB = torch.empty((r, n), dtype=torch.float32, device="cuda")

        def fn():
            ab.ab_layer_forward(g["x"], g["A"], g["B"], y=y, T_save=T, ws=ws_f)
            ab.ab_layer_backward(g["x"], g["dY"], g["A"], g["B"], T_saved=T, dX=dX, dA=dA, dB=dB, ws=ws_b)
        ms = timed(fn)
        flop = 6.0 * N * r * (m + n)
        nbytes = (2.0 if bf16 else 4.0) * N * (3 * n + 2 * m)
        tf = flop / (ms * 1e-3) / 1e12
        ceil_tf = min(pk["tc_burst"], flop / nbytes * pk["hbm"] / 1e3)
        return dict(N=N, m=m, n=n, r=r, ms=ms, tflops=tf, algorithmic_gbs=nbytes / (ms * 1e-3) / 1e9,
                    ceiling_tflops=ceil_tf, frac_of_ceiling=tf / ceil_tf,
                    bound="hbm" if ceil_tf < pk["tc_burst"] else "tensor")

    out = {}
    d = synth.resnet_conv(2)
    out["resnet50_layer3_conv3x3_r128"] = layer(d, True)
    A32, B32 = torch.from_numpy(d["A"]).cuda(), torch.from_numpy(d["B"]).cuda()
    W = ab.ab_recombine(A32, B32)
    ms = timed(lambda: ab.ab_svd_split(W, d["r"], 0.0))
    out["resnet50_layer3_conv3x3_r128"]["recombined_W_split_ms"] = ms
    del d, A32, B32, W
    out["vgg16_512x4608"] = {}
    for r in (8, 16, 32, 64):
        out["vgg16_512x4608"][f"r{r}"] = layer(synth.vgg_conv(r, 4), True)
        torch.cuda.empty_cache()
    d = synth.linear_fp32(0)
    A, B, _, _, _ = ab.ab_svd_split(torch.from_numpy(d["W"]).cuda(), d["r"], 0.0)   # its factors are the split of its W
    d["A"], d["B"] = A.cpu().numpy(), B.cpu().numpy()
    one = layer(d, False)
    out["linear_256x512_fp32_r32"] = dict(N=one["N"], us_fwd_bwd=one["ms"] * 1e3, note="launch-latency bound")
    return out


def conv_workloads(ab, torch, iters=10):
    """The two convolution shapes through the implicit-im2col entry points (NHWC activation in, no 9x inflated
    rows in memory): forward + backward (dX with col2im folded in, dA, dB).  Bytes are counted against the
    un-inflated activation: x in forward and backward, dX out, y out, dY in (bf16)."""
    pk = measured_peaks()
    out = {}
    bf = torch.bfloat16
    for name, (B, H, W, C, m, r) in (("resnet50_layer3_conv3x3_r128", (128, 14, 14, 256, 256, 128)),
                                     ("vgg16_512_4x4_r8", (1024, 4, 4, 512, 512, 8)),
                                     ("vgg16_512_4x4_r16", (1024, 4, 4, 512, 512, 16)),
                                     ("vgg16_512_4x4_r32", (1024, 4, 4, 512, 512, 32)),
                                     ("vgg16_512_4x4_r64", (1024, 4, 4, 512, 512, 64))):
        g = torch.Generator(device="cuda").manual_seed(5)
        x = torch.randn((B, H, W, C), device="cuda", generator=g).abs().to(bf)
        dY = torch.randn((B, H, W, m), device="cuda", generator=g).to(bf)
        A = (torch.randn((m, r), device="cuda", generator=g) * 0.05).to(bf)
        Bf = (torch.randn((r, 9 * C), device="cuda", generator=g) * 0.05).to(bf)
        y = torch.empty((B, H, W, m), dtype=bf, device="cuda")
        T = torch.empty((B * H * W, r), dtype=bf, device="cuda")
        dX = torch.empty_like(x)
        dA = torch.empty((m, r), device="cuda")
        dB = torch.empty((r, 9 * C), device="cuda")
        ws = ab.workspace(ab.ab_conv3x3_workspace_bytes(B, H, W, C, m, r), "cuda")

        def fn():
            ab.ab_conv3x3_forward(x, A, Bf, y=y, T_save=T, ws=ws)
            ab.ab_conv3x3_backward(x, dY, A, Bf, T_saved=T, dX=dX, dA=dA, dB=dB, ws=ws)
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        N = B * H * W
        flop = 6.0 * N * r * (m + 9 * C)
        nbytes = 2.0 * N * (3 * C + 2 * m)
        out[name] = dict(batch=B, H=H, W=W, C=C, m=m, r=r, ms=ms, tflops=flop / (ms * 1e-3) / 1e12,
                         activation_gbs=nbytes / (ms * 1e-3) / 1e9, frac_of_hbm=nbytes / (ms * 1e-3) / 1e9 / pk["hbm"],
                         bytes_vs_materialised_rows=nbytes / (2.0 * N * (3 * 9 * C + 2 * m)),
                         device_status=ab.workspace_status(ws))
    return out


def training_cycle(ab, torch, N=256 * 197, n_ab=4, n_dense=1, K=K_GROUPS):
    """One whole cycle of Algorithm 1 on one GPU for the ViT-B/16 MLP pair, every step through the library:
    decomposition of the dense weights (ab_svd_split, rank 192) -> n_ab factorised steps (forward, backward,
    AdamW on A and B) -> group synchronisation of K copies (mean, W = Abar Bbar, written) -> n_dense full-rank
    steps (dense forward, backward, AdamW on W) -> decomposition again.  The paper's ratio of factorised to
    rebound steps is 4 : 1.  Event-timed per phase; the K copies are the trained factors plus N(0, 1e-3) noise."""
    from paper_2405_01067_b200 import synth
    bf = torch.bfloat16
    w = synth.vit_mlp_weights(seed=1)
    layers = []
    for li, (m, n) in enumerate(LAYERS):
        d = synth.vit_mlp(li + 1, seed=7, N=N, K=K)
        g = dict(m=m, n=n, W=torch.from_numpy(w["W1" if li == 0 else "W2"]).cuda(),
                 x=torch.from_numpy(d["x"]).to(bf).cuda(), dY=torch.from_numpy(d["dY"]).to(bf).cuda(),
                 noise_A=torch.from_numpy(np.stack(d["noise_A"])).cuda(), noise_B=torch.from_numpy(np.stack(d["noise_B"])).cuda(),
                 y=torch.empty((N, m), dtype=bf, device="cuda"), T=torch.empty((N, R), dtype=bf, device="cuda"),
                 dX=torch.empty((N, n), dtype=bf, device="cuda"), dA=torch.empty((m, R), device="cuda"),
                 dB=torch.empty((R, n), device="cuda"), dW=torch.empty((m, n), device="cuda"),
                 W_lp=torch.empty((m, n), dtype=bf, device="cuda"), A_lp=torch.empty((m, R), dtype=bf, device="cuda"),
                 B_lp=torch.empty((R, n), dtype=bf, device="cuda"))
        for nm, shape in (("A", (m, R)), ("B", (R, n)), ("W", (m, n))):
            g["m_" + nm] = torch.zeros(shape, device="cuda")
            g["v_" + nm] = torch.zeros(shape, device="cuda")
        g["ws_f"] = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_LAYER_FORWARD, N, m, n, R, 1, ab.AB_BF16), "cuda")
        g["ws_b"] = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_LAYER_BACKWARD, N, m, n, R, 1, ab.AB_BF16), "cuda")
        g["ws_df"] = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_DENSE_FORWARD, N, m, n, 0, 1, ab.AB_BF16), "cuda")
        g["ws_db"] = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_DENSE_BACKWARD, N, m, n, 0, 1, ab.AB_BF16), "cuda")
        g["ws_s"] = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_SVD_SPLIT, 0, m, n, R, 1, ab.AB_F32), "cuda")
        layers.append(g)

    def decompose():
        for g in layers:
            g["A"], g["B"], g["sigma"], g["r_out"], g["st"] = ab.ab_svd_split(g["W"], R, 0.0, ws=g["ws_s"])
            ab.ab_group_average(g["A"][None], out=g["A_lp"])        # the bf16 copies the chain reads (a mean of one)
            ab.ab_group_average(g["B"][None], out=g["B_lp"])

    def ab_steps():
        for step in range(1, n_ab + 1):
            lr = 1e-3 * ab.ab_lr_rebound_factor(step, 2, 0.05)
            for g in layers:
                ab.ab_layer_forward(g["x"], g["A_lp"], g["B_lp"], y=g["y"], T_save=g["T"], ws=g["ws_f"])
                ab.ab_layer_backward(g["x"], g["dY"], g["A_lp"], g["B_lp"], T_saved=g["T"], dX=g["dX"], dA=g["dA"], dB=g["dB"],
                                     ws=g["ws_b"])
                ab.ab_adamw_step(g["A"], g["dA"], g["m_A"], g["v_A"], lr, step, param_bf16=g["A_lp"])
                ab.ab_adamw_step(g["B"], g["dB"], g["m_B"], g["v_B"], lr, step, param_bf16=g["B_lp"])

    def sync():
        copies_A = [g["A"][None] + g["noise_A"] for g in layers]      # input assembly: the K groups' copies
        copies_B = [g["B"][None] + g["noise_B"] for g in layers]
        plan = ab.SyncPlan(copies_A, copies_B, 0.0, want_W=True)
        return plan

    def sync_run(plan):
        ab.ab_group_sync(plan)
        for g, Wn in zip(layers, plan.W_out):
            g["W"] = Wn
            ab.ab_group_average(Wn[None], out=g["W_lp"])

    def dense_steps():
        for step in range(1, n_dense + 1):
            lr = 1e-3 * ab.ab_lr_rebound_factor(step, 2, 0.05)
            for g in layers:
                ab.ab_dense_forward(g["x"], g["W_lp"], y=g["y"], ws=g["ws_df"])
                ab.ab_dense_backward(g["x"], g["dY"], g["W_lp"], dX=g["dX"], dW=g["dW"], ws=g["ws_db"])
                ab.ab_adamw_step(g["W"], g["dW"], g["m_W"], g["v_W"], lr, step, param_bf16=g["W_lp"])

    def timed(fn):
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    decompose()                      # warm-up of every kernel on the way
    ab_steps()
    plan = sync()
    sync_run(plan)
    dense_steps()
    out = dict(workload="vit_b16_mlp_pair, one cycle", rows=N, n_ab_steps=n_ab, n_dense_steps=n_dense, K=K)
    out["decompose_ms"] = timed(decompose)
    out["ab_steps_ms"] = timed(ab_steps)
    plan = sync()
    out["sync_ms"] = timed(lambda: sync_run(plan))
    out["dense_steps_ms"] = timed(dense_steps)
    out["decompose_again_ms"] = timed(decompose)
    out["cycle_ms"] = sum(out[k] for k in ("decompose_ms", "ab_steps_ms", "sync_ms", "dense_steps_ms"))
    out["device_status"] = [int(g["st"].item()) for g in layers] + [int(plan.status.abs().sum().item())]
    return out


def fused_mean_recombine(ab, torch, iters=10):
    """Mean of K = 8 copies and W = Abar Bbar for one ViT-B/16 matrix of each shape: the one-kernel form (the mean
    as the product's operand prologue, ab_recombine_mean) against the separate calls (ab_group_average twice,
    then ab_recombine on the tensor cores)."""
    out = {}
    K, r = 8, 192
    for (m, n) in ((768, 768), (3072, 768), (768, 3072)):
        Ak = torch.randn((K, m, r), device="cuda")
        Bk = torch.randn((K, r, n), device="cuda")
        W = torch.empty((m, n), device="cuda")
        Ab, Bb = torch.empty((m, r), device="cuda"), torch.empty((r, n), device="cuda")
        ws = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_RECOMBINE, 0, m, n, r, 1, ab.AB_F32), "cuda")

        def separate():
            ab.ab_group_average(Ak, out=Ab)
            ab.ab_group_average(Bk, out=Bb)
            ab.ab_recombine(Ab, Bb, W=W, ws=ws)

        def fused():
            ab.ab_recombine_mean(Ak, Bk, W=W, Abar=Ab, Bbar=Bb)
        res = {}
        for name, fn in (("separate_us", separate), ("one_kernel_us", fused)):
            for _ in range(3):
                fn()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(iters):
                fn()
            e1.record()
            torch.cuda.synchronize()
            res[name] = e0.elapsed_time(e1) / iters * 1e3
        out[f"{m}x{n}"] = res
    return out


def dense_split_times(ab, torch, iters=3):
    """The decomposition Algorithm 1 runs after the full-rank rebound phase: W is dense and no longer of rank
    <= r, so the factored route does not apply.  ab_svd_split (r_max 192, fixed rank) of one matrix of each
    ViT-B/16 shape, W = 0.02 G + P diag(0.9^i) Q^T, event-timed; LAPACK's float64 time on the host beside it."""
    from paper_2405_01067_b200 import synth
    out = {}
    w = synth.vit_mlp_weights(seed=1)
    st = synth.streams(11, ["g", "p"])
    sq = synth.normal(st["g"], (768, 768), 0.02) + synth.planted_matrix(st["p"], 768, 768, 0.9 ** np.arange(768))
    for name, W in (("768x768", sq), ("3072x768", w["W1"]), ("768x3072", w["W2"])):
        Wd = torch.from_numpy(W).cuda()
        m, n = W.shape
        ws = ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_SVD_SPLIT, 0, m, n, 192, 1, ab.AB_F32), "cuda")
        res = ab.ab_svd_split(Wd, 192, 0.0, ws=ws)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            res = ab.ab_svd_split(Wd, 192, 0.0, ws=ws)
        e1.record()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        np.linalg.svd(W.astype(np.float64), full_matrices=False)
        out[name] = dict(ms=e0.elapsed_time(e1) / iters, device_status=int(res[4].item()),
                         lapack_f64_host_ms=(time.perf_counter() - t0) * 1e3)
    return out


def optimizer_step(ab, torch, iters=10):
    """AdamW update of a whole ViT-B/16 factor set (31.85 M fp32 master values, moments in fp32, bf16 copy
    written): a pure HBM stream of 30 bytes per value."""
    count = 31850496
    p = torch.randn(count, device="cuda")
    g = torch.randn(count, device="cuda")
    m = torch.zeros(count, device="cuda")
    v = torch.zeros(count, device="cuda")
    lp = torch.empty(count, dtype=torch.bfloat16, device="cuda")
    for k in range(3):
        ab.ab_adamw_step(p, g, m, v, 1e-3, k + 1, param_bf16=lp)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for k in range(iters):
        ab.ab_adamw_step(p, g, m, v, 1e-3, k + 4, param_bf16=lp)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    gbs = 30.0 * count / (ms * 1e-3) / 1e9
    return dict(values=count, ms=ms, gbs=gbs, frac_of_measured_hbm=gbs / measured_peaks()["hbm"])


def backward_variants(ab, torch, layers, N, iters=10):
    """The two frozen-factor steps of the method on the same workload: a B-group trains B (forward, then
    dT, dX and dB; A frozen, no dA), an A-group trains A (forward with T kept, then dA only -- its dX is
    counted with the B-side variant of the layer below in a real model, and is not computed here).
    Returns ms per step (both layers) and the algorithmic TFLOP/s of what each variant computes."""
    def ev():
        return torch.cuda.Event(enable_timing=True)

    def b_group():
        for L in layers:
            g = L["g"]
            ab.ab_layer_forward(g["x"], g["A"], g["B"], y=g["y"], ws=g["ws_f"])
            ab.ab_layer_backward(g["x"], g["dY"], g["A"], g["B"], want=("dX", "dB"), dX=g["dX"], dB=g["dB"], ws=g["ws_b"])

    def a_group():
        for L in layers:
            g = L["g"]
            ab.ab_layer_forward(g["x"], g["A"], g["B"], y=g["y"], T_save=g["T"], ws=g["ws_f"])
            ab.ab_layer_backward(g["x"], g["dY"], g["A"], g["B"], T_saved=g["T"], want=("dA",), dA=g["dA"], ws=g["ws_b"])

    out = {}
    for name, fn in (("b_group", b_group), ("a_group", a_group)):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        flop = 0.0
        for L in layers:
            m, r = L["g"]["A"].shape
            n = L["g"]["B"].shape[1]
            fwd = 2.0 * N * r * (m + n)
            flop += fwd + (2.0 * N * r * (m + n) + 2.0 * N * r * n if name == "b_group" else 2.0 * N * r * m)
        out[name] = dict(ms_per_step=ms, tflops=flop / (ms * 1e-3) / 1e12,
                         computes="forward, dT, dX, dB" if name == "b_group" else "forward (T kept), dA")
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2405_01067_b200 import binding as ab

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    ab.lib()
    N = args.rows
    inputs = make_inputs(rank, N)
    bf = torch.bfloat16

    def pinned(a):
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(bf).pin_memory()

    layers = []
    for d in inputs:
        m, n = d["m"], d["n"]
        h = {k: pinned(d[k]) for k in ("x", "dY", "A", "B", "A_copies", "B_copies")}
        g = {k: v.cuda() for k, v in h.items()}
        g.update(y=torch.empty((N, m), dtype=bf, device="cuda"), T=torch.empty((N, R), dtype=bf, device="cuda"),
                 dX=torch.empty((N, n), dtype=bf, device="cuda"),
                 dA=torch.empty((m, R), dtype=torch.float32, device="cuda"),
                 dB=torch.empty((R, n), dtype=torch.float32, device="cuda"),
                 ws_f=ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_LAYER_FORWARD, N, m, n, R, 1, ab.AB_BF16), "cuda"),
                 ws_b=ab.workspace(ab.ab_workspace_bytes(ab.AB_OP_LAYER_BACKWARD, N, m, n, R, 1, ab.AB_BF16), "cuda"))
        hout = dict(dA=torch.empty((m, R), dtype=torch.float32).pin_memory(),
                    dB=torch.empty((R, n), dtype=torch.float32).pin_memory(),
                    A=torch.empty((m, R), dtype=bf).pin_memory(), B=torch.empty((R, n), dtype=bf).pin_memory(),
                    sigma=torch.empty((R,), dtype=torch.float32).pin_memory())
        layers.append(dict(m=m, n=n, h=h, g=g, hout=hout))
    plan = ab.SyncPlan([L["g"]["A_copies"] for L in layers], [L["g"]["B_copies"] for L in layers], 0.0, want_W=True)

    def ev():
        return torch.cuda.Event(enable_timing=True)

    fwd_events = []        # (start, stop) around every forward call of the timed steps

    def chain(record=False):
        for L in layers:
            g = L["g"]
            if record:
                f0, f1 = ev(), ev()
                f0.record()
            ab.ab_layer_forward(g["x"], g["A"], g["B"], y=g["y"], T_save=g["T"], ws=g["ws_f"])
            if record:
                f1.record()
                fwd_events.append((f0, f1))
            ab.ab_layer_backward(g["x"], g["dY"], g["A"], g["B"], T_saved=g["T"], dX=g["dX"], dA=g["dA"], dB=g["dB"],
                                 ws=g["ws_b"])

    def step(marks=None):
        if marks is not None:
            marks[0].record()
        chain(record=marks is not None)
        if marks is not None:
            marks[1].record()
        ab.ab_group_sync(plan)
        if marks is not None:
            marks[2].record()

    def e2e_step(with_sync=False):
        for L in layers:
            L["g"]["x"].copy_(L["h"]["x"], non_blocking=True)
            L["g"]["dY"].copy_(L["h"]["dY"], non_blocking=True)
        chain()
        for i, L in enumerate(layers):
            L["hout"]["dA"].copy_(L["g"]["dA"], non_blocking=True)
            L["hout"]["dB"].copy_(L["g"]["dB"], non_blocking=True)
        if with_sync:
            ab.ab_group_sync(plan)
            for i, L in enumerate(layers):
                L["hout"]["A"].copy_(plan.A_out[i], non_blocking=True)
                L["hout"]["B"].copy_(plan.B_out[i], non_blocking=True)
                L["hout"]["sigma"].copy_(plan.sigma[i], non_blocking=True)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    marks = [[ev(), ev(), ev()] for _ in range(args.steps)]
    launches0 = ab.ab_launch_count()
    t_begin, t_end = ev(), ev()
    t_begin.record()
    for i in range(args.steps):
        step(marks[i])
    t_end.record()
    barrier()
    sampler.stop_flag = True
    launches = ab.ab_launch_count() - launches0
    total_ms = t_begin.elapsed_time(t_end)
    chain_each = sorted(mk[0].elapsed_time(mk[1]) for mk in marks)
    chain_ms = sum(chain_each)
    sync_ms = sum(mk[1].elapsed_time(mk[2]) for mk in marks)
    fwd_ms = sum(a.elapsed_time(b) for a, b in fwd_events) / max(len(fwd_events), 1)   # per forward launch
    if int(plan.status.abs().sum().item()) != 0:
        raise SystemExit("group sync reported a device-side error status")

    # the chain alone, steps queued back to back (as between two synchronisations of a training cycle)
    barrier()
    b0, b1 = ev(), ev()
    b0.record()
    for _ in range(args.steps):
        chain()
    b1.record()
    barrier()
    b2b_ms = b0.elapsed_time(b1)

    # end to end: inputs start in pinned host memory, results end there
    for _ in range(2):
        e2e_step()
    barrier()
    e0, e1 = ev(), ev()
    e0.record()
    for _ in range(args.steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e0.record()
    for _ in range(args.steps):
        e2e_step(with_sync=True)
    e1.record()
    barrier()
    e2e_sync_ms = e0.elapsed_time(e1)

    total_ms, chain_ms, sync_ms, e2e_ms, e2e_sync_ms, b2b_ms = max_over_ranks(
        [total_ms, chain_ms, sync_ms, e2e_ms, e2e_sync_ms, b2b_ms], "cuda", world)
    sampler.join(timeout=2.0)
    if rank == 0:
        pk = measured_peaks()
        K = args.steps
        flops_step = chain_flops(N) * world
        value = whole_job_tflops(N, world, K, chain_ms)
        # the metric's work (the chain) from pinned host inputs to pinned host gradients
        e2e_value = flops_step * K / (e2e_ms * 1e-3) / 1e12
        h2d = sum(L["h"]["x"].numel() + L["h"]["dY"].numel() for L in layers) * 2
        d2h = sum(sum(L["hout"][k].numel() * L["hout"][k].element_size() for k in ("dA", "dB")) for L in layers)
        per_gpu = value / world
        # dominant kernel of the chain: chain_kernel (every forward call is exactly one launch of
        # it; backward launches it once more).  Algorithmic work of a forward launch: 2 N r (m+n) FLOP
        # (both layers have m+n = 3840), 2 N (m+n) bytes.
        fwd_flops = 2.0 * N * R * 3840
        fwd_bytes = 2.0 * N * 3840
        fwd_tflops = fwd_flops / (fwd_ms * 1e-3) / 1e12
        fwd_gbs = fwd_bytes / (fwd_ms * 1e-3) / 1e9
        # which roof binds a forward launch: the tensor peak (burst figure: the launch is timed by itself,
        # 0.1 ms at full clocks) or its intensity times the HBM peak
        hbm_ceiling_tflops = fwd_flops / fwd_bytes * pk["hbm"] / 1e3
        hbm_bound = hbm_ceiling_tflops < pk["tc_burst"]
        kernel = "chain_kernel (one launch = ab_layer_forward of one layer at this size)"
        common = dict(kernel=kernel, traffic=ROW_CHAIN_DRAM_BYTES_PER_LAUNCH, us_per_launch=fwd_ms * 1e3,
                      tflops=fwd_tflops, algorithmic_gbs=fwd_gbs, hbm_peak_gbs=pk["hbm"], tensor_peak_tflops=pk["tc_burst"],
                      frac_of_tensor_burst=fwd_tflops / pk["tc_burst"], frac_of_hbm=fwd_gbs / pk["hbm"],
                      frac_of_nominal_2250=fwd_tflops / NOMINAL_BF16_TFLOPS,
                      whole_chain=dict(tflops=per_gpu, frac_of_measured_burst=per_gpu / pk["tc_burst"],
                                       frac_of_nominal_2250=per_gpu / NOMINAL_BF16_TFLOPS,
                                       algorithmic_gbs=chain_bytes(N) * K / (chain_ms * 1e-3) / 1e9,
                                       frac_of_hbm=chain_bytes(N) * K / (chain_ms * 1e-3) / 1e9 / pk["hbm"]))
        if hbm_bound:
            roof = dict(bound="hbm", achieved=fwd_gbs, peak=pk["hbm"], unit="GB/s", frac=fwd_gbs / pk["hbm"],
                        peak_source=f"hbm_gbs of {pk['source']}", **common)
        else:
            roof = dict(bound="tensor", achieved=fwd_tflops, peak=pk["tc_burst"], unit="TFLOP/s",
                        frac=fwd_tflops / pk["tc_burst"], peak_source=f"bf16_tflops (burst) of {pk['source']}", **common)
        line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=K, warmup=args.warmup,
                    ms_per_step=total_ms / K, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="bf16", data="synthetic",
                    config=dict(workload="vit_b16_mlp_pair_r192", rows=N, layers=[list(s) for s in LAYERS], r=R,
                                K=K_GROUPS, sync="mean + recombine (W written) + truncated-SVD split of both layers every step, factored route",
                                l2="inputs larger than L2 (about 0.8 GB of activations read per step)"),
                    chain_ms_per_step=chain_ms / K, chain_ms_median=chain_each[len(chain_each) // 2],
                    chain_ms_min=chain_each[0], group_sync_ms_per_step=sync_ms / K,
                    chain_back_to_back=dict(ms_per_step=b2b_ms / K, tflops=flops_step * K / (b2b_ms * 1e-3) / 1e12,
                                            note="chain steps queued one after the other, no group sync between them"),
                    pct_of_nominal_bf16_peak=100.0 * per_gpu / NOMINAL_BF16_TFLOPS,
                    e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                             ms_per_step=e2e_ms / K, ms_per_step_with_group_sync=e2e_sync_ms / K),
                    gpu_launches=int(launches), clocks=sampler.summary(), roofline=roof)
        if world == 1:
            line["frozen_factor_variants"] = backward_variants(ab, torch, layers, N)
        if world == 1 and not args.no_model_sync:
            del layers, plan
            torch.cuda.empty_cache()
            line["group_sync_model"] = vit_model_sync(ab, torch)
        if world == 1 and not args.no_other_workloads:
            line["other_workloads"] = other_workloads(ab, torch)
            line["adamw_update_vit_factors"] = optimizer_step(ab, torch)
            line["dense_split_ms"] = dense_split_times(ab, torch)
            line["fused_mean_recombine"] = fused_mean_recombine(ab, torch)
            line["implicit_conv"] = conv_workloads(ab, torch)
            torch.cuda.empty_cache()
            line["training_cycle"] = training_cycle(ab, torch)
        if world == 1 and not args.no_cpu_baseline:
            cb = cpu_baseline(inputs, min(N, args.baseline_rows), sync_scale=4)    # about 10 s of host work
            line["cpu_baseline"] = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(n):
    """`python bench.py --gpus N` outside torchrun: start the N ranks (one process per GPU, rendezvous on
    127.0.0.1) with the same arguments and hand their exit status back.  Rank 0 prints the JSON line."""
    import socket
    import subprocess
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--rows", type=int, default=256 * 197, help="token rows per layer (default: batch 256 x 197)")
    ap.add_argument("--ref-rows", type=int, default=8192,
                    help="rows of the CPU checker's bounded sample per step of --impl reference")
    ap.add_argument("--baseline-rows", type=int, default=32768,
                    help="rows of the CPU checker's bounded sample timed once beside the GPU run (cpu_baseline)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-model-sync", action="store_true", help="skip the full-ViT group-sync measurement")
    ap.add_argument("--only-model-sync", action="store_true",
                    help="run only the full-ViT group-sync measurement and print its figures (for profiling that part)")
    ap.add_argument("--no-other-workloads", action="store_true",
                    help="skip the ResNet-50 / VGG16 / small fp32 layer measurements")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        raise SystemExit(spawn_ranks(args.gpus))
    if args.only_model_sync:
        import torch
        from paper_2405_01067_b200 import binding as ab
        print(json.dumps(dict(group_sync_model=vit_model_sync(ab, torch, steps=args.steps))))
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
