#!/usr/bin/env python
"""Benchmark of the NVFP4 W4A4+RAC MoE layer forward on B200.

  python bench.py --gpus N --steps K --warmup W [--workload prefill|decode|large]
                  [--variant both|w13|plain] [--impl reference]

A step is one pass of the whole hot path (activation amax, routing + dispatch,
RAC statistics / selection / residual quantize, both grouped GEMMs with their
fused epilogues, combine) over one batch of seeded synthetic input.  Rank 0
prints ONE JSON line.  With N > 1 (torchrun) every rank runs its own replica of
the layer on its own batch (no data-path collective; weak scaling).
`--impl reference` times the CPU oracle on a bounded sample of the same
workload on the host cores."""
import argparse
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "moe_layer_tokens_per_s"
UNIT = "tokens/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="prefill", choices=["prefill", "decode", "large"])
    ap.add_argument("--variant", default="both", choices=["both", "w13", "plain"])
    ap.add_argument("--no-aux", action="store_true", help="skip the auxiliary quantize / fake-quant / decode numbers")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--fake-quant-only", action="store_true",
                    help="time only the fake-quant + pack of 16 expert weight tensors [3072, 4096] (a small case for profiling)")
    ap.add_argument("--ref-budget-s", type=float, default=0.0,
                    help="seconds of oracle work per step for --impl reference (0: derived from --steps)")
    return ap.parse_args()


def nsel_of(shape, variant):
    n13 = 0 if variant == "plain" else shape.H // 2
    n2 = shape.I // 2 if variant == "both" else 0
    return n13, n2


def workload_config(shape, variant, extra=None):
    n13, n2 = nsel_of(shape, variant)
    cfg = {"workload": "moe_%s_T%d_H%d_E%d_top%d_I%d" % (shape.name, shape.T, shape.H, shape.E, shape.topk, shape.I),
           "variant": {"both": "RAC 50% at W13 and W2 inputs", "w13": "RAC 50% at W13 input only",
                       "plain": "plain W4A4"}[variant],
           "rac_nsel_13": n13, "rac_nsel_2": n2, "tokens": shape.T,
           "skew": "experts 0..%d get %.0f%% of assignments" % (shape.hot_experts - 1, shape.hot_share * 100)
           if shape.hot_experts else "none",
           "l2": "between timed iterations a 256 MB buffer is written (L2 flushed) and a second 256 MB buffer is read, "
                 "so that the timed kernels start on a cold L2 without inheriting the write-back of the flush's dirty lines"}
    if extra:
        cfg.update(extra)
    return cfg


# ----------------------------------------------------------------------- CPU oracle arm
def oracle_sample(shape, variant, budget_s):
    """Prepare a bounded sample of the workload for the CPU oracle: the first
    T_s tokens of the batch (all dims of the layer unchanged).  Returns a
    callable running one oracle step and the sample description."""
    import numpy as np
    import torch
    from oracle import formats as F
    from oracle import moe as M
    from oracle import nvfp4 as Q
    from paper_2607_15810_b200 import synth

    n13, n2 = nsel_of(shape, variant)
    # the oracle dequantizes each expert it meets (~0.15 s each at these sizes)
    n_exp = max(8, min(shape.E, int(budget_s / 0.2)))
    T_s = max(1, n_exp // shape.topk)
    x, _ = synth.activations(shape)
    lg = synth.router_logits(shape)
    x = x[:T_s].to(torch.float32).numpy()
    lg = lg[:T_s].numpy()
    ids, _ = M.route(lg, shape.topk, True)
    experts = sorted(set(int(e) for e in ids.reshape(-1)))
    I, H, E = shape.I, shape.H, shape.E
    w13 = dict(codes=np.zeros((E, 2 * I, H), np.uint8), sf=np.zeros((E, 2 * I, H // 16), np.uint8),
               gs=np.ones(E, np.float32))
    w2 = dict(codes=np.zeros((E, H, I), np.uint8), sf=np.zeros((E, H, I // 16), np.uint8), gs=np.ones(E, np.float32))
    for e in experts:                                     # untimed set-up, like the GPU's weight packing
        for which, dst in (("w13", w13), ("w2", w2)):
            w = synth.expert_weights(shape, which, [e]).to(torch.float32).numpy()
            _, q, sf, gs = Q.fake_quant_weights(w)
            dst["codes"][e], dst["sf"][e], dst["gs"][e] = F.unpack_nibbles(q[0]), sf[0], gs[0]
    a2 = np.float32(synth.H_GLOBAL_SCALE[shape.name])

    def step():
        return M.moe_forward(x, lg, w13, w2, shape.topk, n13, n2, a2)

    desc = "first %d tokens of the %s batch (%d experts hit), full layer dims, weights pre-packed" % (
        T_s, shape.name, len(experts))
    return step, T_s, desc


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2607_15810_b200 import synth
    shape = synth.MOE_SHAPES[args.workload]
    budget = args.ref_budget_s if args.ref_budget_s > 0 else max(1.5, min(20.0, 150.0 / max(1, args.steps + args.warmup)))
    step, T_s, desc = oracle_sample(shape, args.variant, budget)
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    value = T_s / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(shape, args.variant, {"sample": desc}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ----------------------------------------------------------------------- CUDA arm
class ClockSampler:
    """Polls SM clock and throttle reasons through NVML from a host thread while
    the timed regions run (reading only; no setting is changed)."""

    def __init__(self, index, period_s=0.004):
        import threading
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml as nv
            nv.nvmlInit()
            self.nv = nv
            self.h = nv.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(nv.nvmlDeviceGetMaxClockInfo(self.h, nv.NVML_CLOCK_SM))
        except Exception:
            self.nv = None
            return
        self.period = period_s
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def _run(self):
        nv = self.nv
        bits = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for name, bit in bits.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def pcie(self):
        """Current PCIe link generation and width (the bound of the end-to-end number), read only."""
        try:
            nv = self.nv
            return {"gen": int(nv.nvmlDeviceGetCurrPcieLinkGeneration(self.h)), "width": int(nv.nvmlDeviceGetCurrPcieLinkWidth(self.h)),
                    "max_gen": int(nv.nvmlDeviceGetMaxPcieLinkGeneration(self.h)), "max_width": int(nv.nvmlDeviceGetMaxPcieLinkWidth(self.h))}
        except Exception:
            return None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        if self._thread is None:
            return out
        self._stop.set()
        self._thread.join(timeout=2)
        if self.samples:
            s = sorted(self.samples)
            out.update(sm_mhz=s[len(s) // 2], samples=len(s))
        out["reasons"] = sorted(self.reasons)
        return out


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def kernel_source_digest():
    """SHA-256 over the sources of the grouped GEMM (what an ncu capture of it depends on)."""
    import hashlib
    h = hashlib.sha256()
    for name in ("gemm.cu", "tcgen05.cuh", "kernels.cuh", "common.cuh"):
        with open(os.path.join(ROOT, "paper_2607_15810_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(summary_name):
    """(bytes per launch, note) from the `traffic_bytes_per_launch:` / `kernel_source_digest:` lines of an
    ncu summary under profiles/; (None, why) when the summary is missing or was taken on other sources."""
    path = os.path.join(ROOT, "profiles", summary_name)
    try:
        with open(path) as fh:
            text = fh.read()
    except OSError:
        return None, "no ncu summary"
    vals = {}
    for ln in text.splitlines():
        for key in ("traffic_bytes_per_launch", "kernel_source_digest"):
            if ln.strip().startswith(key + ":"):
                vals[key] = ln.split(":", 1)[1].strip()
    if "traffic_bytes_per_launch" not in vals:
        return None, "summary has no traffic line"
    if vals.get("kernel_source_digest") != kernel_source_digest():
        return None, "ncu summary predates the current kernel sources (digest %s, now %s)" % (
            vals.get("kernel_source_digest"), kernel_source_digest())
    return int(vals["traffic_bytes_per_launch"]), "profiles/" + summary_name


def pipe_probe(B, torch, dev):
    """Measured dense-FP4 rate of the tensor pipe: the library's probe kernel (operands resident in shared
    memory, no global traffic), about 20 ms per mode so that clocks settle under the power cap."""
    n = B.lib.quads_fp4_pipe_probe_operand_bytes()
    g = torch.Generator(device=dev).manual_seed(1)
    ops = torch.randint(0, 256, (n,), dtype=torch.uint8, device=dev, generator=g)
    ops[4 * 16384:] = torch.randint(0x30, 0x40, (n - 4 * 16384,), dtype=torch.uint8, device=dev, generator=g)
    st = torch.zeros(1, dtype=torch.int32, device=dev)
    out = {}
    for mode, name, steps in ((0, "mma_only", 200000), (1, "rac_mix_2mma_4copies", 100000), (2, "plain_mix_1mma_3copies", 200000)):
        B.fp4_pipe_probe(mode, 2000, ops, st)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        flop = B.fp4_pipe_probe(mode, steps, ops, st)
        e1.record()
        torch.cuda.synchronize()
        out[name] = flop / (e0.elapsed_time(e1) * 1e-3) / 1e12
    assert st.item() == 0, "the probe's bounded wait gave up"
    return out


def run_fake_quant_only(args):
    """16 experts' W13 of the AQAT workload through quads_fake_quant_weights: 403 MB in, 516 MB out."""
    import torch
    from paper_2607_15810_b200 import binding as B
    dev = torch.device("cuda", 0)
    peaks = measured_peaks()
    w = (torch.randn(16, 3072, 4096, device=dev) * 0.015).to(torch.bfloat16)
    outs = (torch.empty_like(w), torch.empty(16, 3072, 2048, dtype=torch.uint8, device=dev),
            torch.empty(16, 3072, 256, dtype=torch.uint8, device=dev), torch.empty(16, dtype=torch.float32, device=dev))
    ws = torch.empty(B.lib.quads_fake_quant_workspace_bytes(16), dtype=torch.uint8, device=dev)
    times = []
    for i in range(args.warmup + args.steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        B.fake_quant_weights(w, out=outs, workspace=ws)
        e1.record()
        torch.cuda.synchronize()
        if i >= args.warmup:
            times.append(e0.elapsed_time(e1))
    ms = sum(times) / len(times)
    gbs = w.numel() * 4.5625 / (ms * 1e-3) / 1e9
    print(json.dumps({"metric": "fake_quant_gbs", "value": gbs, "unit": "GB/s", "ms_per_step": ms, "steps": args.steps,
                      "warmup": args.warmup, "frac_of_hbm": gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
                      "config": {"workload": "fake-quant + pack, 16 x [3072, 4096] bf16", "l2": "919 MB per call, larger than L2"}}))


def run_ours(args):
    import torch
    from paper_2607_15810_b200 import binding as B
    from paper_2607_15810_b200 import synth
    if args.fake_quant_only:
        return run_fake_quant_only(args)

    from paper_2607_15810_b200 import dist_util as D
    world, rank, local = D.env_world()
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    D.init("nccl", dev)

    def barrier():
        D.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(v):
        return D.max_over_ranks(v, dev)

    shape = synth.MOE_SHAPES[args.workload]
    n13, n2 = nsel_of(shape, args.variant)
    T, H, I, E, topk = shape.T, shape.H, shape.I, shape.E, shape.topk

    def pack_weights(sh):
        out = {}
        for which in ("w13", "w2"):
            parts = []
            for e0 in range(0, sh.E, 16):
                w = synth.expert_weights(sh, which, range(e0, min(sh.E, e0 + 16)))
                parts.append(B.fake_quant_weights(w.to(dev), want_fq=False, sf_layout=B.SF_TILED))
            out[which] = {k: torch.cat([p[k] for p in parts]) for k in ("q", "sf", "gs")}
        return out["w13"], out["w2"]

    gw13, gw2 = pack_weights(shape)
    x_h, _ = synth.activations(shape)
    lg_h = synth.router_logits(shape)
    x_h, lg_h = x_h.pin_memory(), lg_h.pin_memory()
    x_d, lg_d = x_h.to(dev), lg_h.to(dev)
    a2 = torch.tensor([synth.H_GLOBAL_SCALE[shape.name]], dtype=torch.float32, device=dev)
    ws = torch.empty(B.moe_workspace_bytes(T, H, I, E, topk), dtype=torch.uint8, device=dev)
    out_d = torch.empty(T, H, dtype=torch.bfloat16, device=dev)
    out_h = torch.empty(T, H, dtype=torch.bfloat16).pin_memory()
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    flush_rd = torch.zeros(64 << 20, dtype=torch.int32, device=dev)        # 256 MB

    def flush_l2():
        # write a buffer larger than L2 (evicts everything), then read another one: the written lines
        # are still dirty in L2, and the kernels under test would otherwise pay for their write-back
        flush.fill_(1)
        flush_rd.max()

    def step():
        B.moe_w4a4_rac(x_d, lg_d, gw13, gw2, topk, n13, n2, a2, workspace=ws, out=out_d)

    def timed(fn, k, with_flush=True):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(k)]
        for s, e in evs:
            if with_flush:
                flush_l2()
            s.record()
            fn()
            e.record()
        torch.cuda.synchronize()
        return [s.elapsed_time(e) for s, e in evs]

    for _ in range(max(3, args.warmup)):
        flush_l2()
        step()
    torch.cuda.synchronize()
    assert B.moe_async_status(ws) == 0, "device-side wait timed out"
    launches_per_step = B.last_launch_count()

    sampler = ClockSampler(local) if rank == 0 else None
    barrier()
    wall0 = time.perf_counter()
    times = timed(step, args.steps)
    barrier()
    wall = time.perf_counter() - wall0
    ms = max_over_ranks(sum(times) / len(times))
    value = D.whole_job_rate(world, T, ms)

    # end to end: pinned host input -> device, the call, result back to pinned host memory
    def e2e_step():
        x_d.copy_(x_h, non_blocking=True)
        lg_d.copy_(lg_h, non_blocking=True)
        step()
        out_h.copy_(out_d, non_blocking=True)

    for _ in range(2):
        e2e_step()
    barrier()
    e2e_times = timed(e2e_step, args.steps)
    barrier()
    e2e_ms = max_over_ranks(sum(e2e_times) / len(e2e_times))

    # the same end-to-end work pipelined across steps, as a serving loop runs it: every step still
    # copies its own inputs from pinned host memory and its own result back, but on copy streams
    # of their own (two device buffers each way), so a step's transfers overlap its neighbours' compute
    s_in, s_out, s_cmp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
    xin = [torch.empty_like(x_d) for _ in range(2)]
    lgin = [torch.empty_like(lg_d) for _ in range(2)]
    outb = [torch.empty_like(out_d) for _ in range(2)]

    def pipelined(k):
        ev_in = [torch.cuda.Event() for _ in range(k)]
        ev_cmp = [torch.cuda.Event() for _ in range(k)]
        ev_out = [torch.cuda.Event() for _ in range(k)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s_in.wait_stream(s_cmp)
        s_out.wait_stream(s_cmp)
        t0.record(s_in)
        for i in range(k):
            b = i & 1
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_cmp[i - 2])          # the input buffer has been consumed
                xin[b].copy_(x_h, non_blocking=True)
                lgin[b].copy_(lg_h, non_blocking=True)
                ev_in[i].record(s_in)
            s_cmp.wait_event(ev_in[i])
            if i >= 2:
                s_cmp.wait_event(ev_out[i - 2])             # the output buffer has been read back
            flush_l2()
            B.moe_w4a4_rac(xin[b], lgin[b], gw13, gw2, topk, n13, n2, a2, workspace=ws, out=outb[b])
            ev_cmp[i].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[i])
                out_h.copy_(outb[b], non_blocking=True)
                ev_out[i].record(s_out)
        t1.record(s_out)
        torch.cuda.synchronize()
        return t0.elapsed_time(t1) / k

    pipelined(4)
    barrier()
    e2e_pipe_ms = max_over_ranks(pipelined(args.steps))
    barrier()
    pcie = sampler.pcie() if sampler else None
    clocks = sampler.stop() if sampler else None

    # per-kernel time of the two grouped GEMMs (events recorded by the library on the launch stream)
    B.moe_set_kernel_timing(True)
    g1, g2 = [], []
    for _ in range(max(5, min(args.steps, 20))):
        flush_l2()
        step()
        a, b = B.moe_last_kernel_ms()
        g1.append(a)
        g2.append(b)
    B.moe_set_kernel_timing(False)
    g1_ms, g2_ms = sum(g1) / len(g1), sum(g2) / len(g2)
    # per-stage times (events after every stage; separate pass, not the headline timing)
    B.moe_set_stage_trace(True)
    stage_acc = {}
    flush_l2()
    step()                      # kernels that only the traced (serialised) path uses load on their first launch
    for _ in range(5):
        flush_l2()
        step()
        for name, t in B.moe_get_stage_trace():
            stage_acc.setdefault(name, []).append(t)
    B.moe_set_stage_trace(False)
    stages_us = {k: round(1e3 * sum(v) / len(v), 1) for k, v in stage_acc.items()}

    if rank != 0:
        D.shutdown()
        return

    peaks = measured_peaks()
    A = T * topk
    f_model = 6.0 * A * H * I
    f_alg1 = 2.0 * A * H * 2 * I * (1.0 + n13 / H)
    f_alg2 = 2.0 * A * I * H * (1.0 + n2 / I)
    fp4_peak = peaks["bf16_tflops"] * 4.0
    ach = f_alg1 / (g1_ms * 1e-3) / 1e12
    roofline = {"kernel": "gemm_kernel<SwiGLU> (grouped W13 GEMM + RAC + SwiGLU + requantize)", "bound": "tensor",
                "achieved": ach, "peak": fp4_peak, "unit": "TFLOP/s", "frac": ach / fp4_peak,
                "peak_source": "%s bf16 burst %.1f TFLOP/s x 4 (nominal FP4:bf16 ratio)" % (peaks["source"], peaks["bf16_tflops"]),
                "traffic": None, "ms": g1_ms,
                "gemm2": {"ms": g2_ms, "achieved": f_alg2 / (g2_ms * 1e-3) / 1e12, "frac": f_alg2 / (g2_ms * 1e-3) / 1e12 / fp4_peak},
                "frac_of_nominal_9pf": ach / 9000.0}
    # what the tensor pipe executes for those algorithmic flops: the masked residual product runs at full K
    # (2 MMAs per K step at a compensated site) and every expert's rows are padded to whole 128-row tiles
    res_x = B.moe_w4a4_rac(x_d, lg_d, gw13, gw2, topk, n13, n2, a2, workspace=ws, out=out_d, export=True)
    offs = res_x["offsets"].cpu().numpy().astype("int64")
    counts = offs[1:] - offs[:-1]
    padded_rows = int((((counts + 127) // 128) * 128).sum())
    f_exec1 = 2.0 * padded_rows * H * 2 * I * (2.0 if n13 > 0 else 1.0)
    roofline["executed"] = {"tflops": f_exec1 / (g1_ms * 1e-3) / 1e12, "frac_of_peak": f_exec1 / (g1_ms * 1e-3) / 1e12 / fp4_peak,
                            "padded_rows": padded_rows, "dispatched_rows": int(A),
                            "note": "MMAs issued (residual product at full K, padding rows included); not a roofline claim"}
    del res_x
    # dram__bytes_read.sum + dram__bytes_write.sum of one GEMM-1 launch: taken from the ncu summary of this
    # workload, and only while the kernel's sources still are the ones that capture ran (else null)
    if args.workload == "prefill" and args.variant == "both":
        roofline["traffic"], roofline["traffic_source"] = ncu_traffic("gemm_kernel_moe_prefill_ncu_full.md")
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "fp4 (e2m1 x e2m1, ue4m3 block scales, fp32 accumulate)",
            "data": "synthetic", "config": workload_config(shape, args.variant),
            "clocks": clocks, "wall_s_timed_region": wall,
            "e2e": {"value": D.whole_job_rate(world, T, e2e_pipe_ms), "unit": UNIT, "ms_per_step": e2e_pipe_ms,
                    "h2d_bytes_per_step": x_h.numel() * 2 + lg_h.numel() * 4, "d2h_bytes_per_step": out_h.numel() * 2,
                    "how": "every step copies its inputs from pinned host memory and its result back; copies run on "
                           "their own streams with two device buffers each way, so they overlap neighbouring steps",
                    "serial_value": D.whole_job_rate(world, T, e2e_ms), "serial_ms_per_step": e2e_ms,
                    "pcie_link": pcie},
            "gpu_launches": launches_per_step * args.steps,
            "tflops": {"model": f_model / (ms * 1e-3) / 1e12, "algorithmic": (f_alg1 + f_alg2) / (ms * 1e-3) / 1e12,
                       "frac_of_fp4_peak": (f_alg1 + f_alg2) / (ms * 1e-3) / 1e12 / fp4_peak},
            "roofline": roofline, "stages_us": stages_us}

    if not args.no_aux:
        aux = {}
        # measured dense-FP4 rate of the tensor pipe (block-scaled tcgen05.mma issue loop, no global traffic)
        probe = pipe_probe(B, torch, dev)
        aux["fp4_pipe_peak_tflops"] = probe["mma_only"]
        aux["fp4_pipe_probe_tflops"] = probe
        aux["fp4_pipe_note"] = ("executed TFLOP/s of 128x256x64 block-scaled MMAs issued from shared memory by one thread per SM, "
                                "~20 ms per mode under the power cap; the RAC mix executes 4/3 of its algorithmic flops")
        roofline["measured_pipe_peak"] = probe["mma_only"]
        roofline["frac_of_measured_pipe_peak"] = ach / probe["mma_only"]
        # quantize GB/s on the activation tensor of this workload (ring of 8 inputs > L2)
        ring = [torch.randn(T, H, device=dev).to(torch.bfloat16) for _ in range(8)]
        q = torch.empty(T, H // 2, dtype=torch.uint8, device=dev)
        sf = torch.empty(T, H // 16, dtype=torch.uint8, device=dev)
        g = torch.empty(1, dtype=torch.float32, device=dev)
        qws = torch.empty(B.lib.quads_quantize_workspace_bytes(), dtype=torch.uint8, device=dev)
        it = [0]

        def qstep():
            B.quantize_nvfp4(ring[it[0] % 8], out=(q, sf, g), workspace=qws)
            it[0] += 1
        for _ in range(8):
            qstep()
        tq = timed(qstep, 40, with_flush=False)
        aux["quantize_eager_gbs"] = T * H * 2.5625 / (sum(tq) / len(tq) * 1e-3) / 1e9
        # at this size a call is shorter on the GPU than its launches are on the host: the device-side number
        # is the same sequence (ring of 8 inputs, 268 MB, larger than L2) replayed from a CUDA graph
        qgraph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(qgraph):
            for _ in range(8):
                qstep()
        qgraph.replay()
        tg_q = timed(qgraph.replay, 20, with_flush=False)
        q_ms = sum(tg_q) / len(tg_q) / 8
        aux["quantize_gbs"] = T * H * 2.5625 / (q_ms * 1e-3) / 1e9
        aux["quantize_frac_of_hbm"] = aux["quantize_gbs"] / peaks["hbm_gbs"]
        aux["quantize_note"] = ("%.1f MB activation, scale derived on the device (two launches: partial maxima, then "
                                "quantization out of L2); device time per call from a CUDA-graph replay of 8 calls on a ring "
                                "of inputs; `quantize_eager_gbs` is the same with one host launch sequence per call"
                                % (T * H * 2 / 1e6))
        del ring
        # the same call on an activation large enough for bandwidth to matter (65536 x 4096, 537 MB)
        big = torch.randn(65536, 4096, device=dev).to(torch.bfloat16)
        qb = torch.empty(65536, 2048, dtype=torch.uint8, device=dev)
        sb = torch.empty(65536, 256, dtype=torch.uint8, device=dev)

        def qbig():
            B.quantize_nvfp4(big, out=(qb, sb, g), workspace=qws)
        for _ in range(3):
            qbig()
        tb = timed(qbig, 10)
        aux["quantize_large_gbs"] = big.numel() * 2.5625 / (sum(tb) / len(tb) * 1e-3) / 1e9
        aux["quantize_large_frac_of_hbm"] = aux["quantize_large_gbs"] / peaks["hbm_gbs"]
        # and with a caller-supplied (static) per-tensor scale: one pass, no amax read
        gstat = torch.tensor([4.0 / 2688.0], dtype=torch.float32, device=dev)

        def qbig_static():
            B.quantize_nvfp4(big, gs=gstat, out=(qb, sb, g), workspace=qws)
        for _ in range(3):
            qbig_static()
        ts = timed(qbig_static, 10)
        aux["quantize_large_static_scale_gbs"] = big.numel() * 2.5625 / (sum(ts) / len(ts) * 1e-3) / 1e9
        aux["quantize_large_static_scale_frac_of_hbm"] = aux["quantize_large_static_scale_gbs"] / peaks["hbm_gbs"]
        del big, qb, sb
        # fake-quant + pack GB/s: 16 experts' W13 of the AQAT workload (403 MB in, 516 MB out)
        w = (torch.randn(16, 3072, 4096, device=dev) * 0.015).to(torch.bfloat16)
        outs = (torch.empty_like(w), torch.empty(16, 3072, 2048, dtype=torch.uint8, device=dev),
                torch.empty(16, 3072, 256, dtype=torch.uint8, device=dev), torch.empty(16, dtype=torch.float32, device=dev))
        fws = torch.empty(B.lib.quads_fake_quant_workspace_bytes(16), dtype=torch.uint8, device=dev)

        def fstep():
            B.fake_quant_weights(w, out=outs, workspace=fws)
        for _ in range(3):
            fstep()
        tf = timed(fstep, 20)
        aux["fake_quant_gbs"] = w.numel() * 4.5625 / (sum(tf) / len(tf) * 1e-3) / 1e9
        aux["fake_quant_frac_of_hbm"] = aux["fake_quant_gbs"] / peaks["hbm_gbs"]
        aux["hbm_peak_gbs"] = peaks["hbm_gbs"]
        # decode of those packed tensors back to bf16 (the rollout's weight load / a W4A16 operand): 0.5625 B in, 2 B out
        dq_out = outs[0]

        def dstep_():
            B.dequantize_nvfp4(outs[1], outs[2], outs[3], 3072, 4096, out=dq_out)
        for _ in range(3):
            dstep_()
        tdq = timed(dstep_, 20)
        aux["dequantize_gbs"] = w.numel() * 2.5625 / (sum(tdq) / len(tdq) * 1e-3) / 1e9
        aux["dequantize_frac_of_hbm"] = aux["dequantize_gbs"] / peaks["hbm_gbs"]
        del w, outs, dq_out
        # one whole layer of the AQAT + weight-sync workload: 128 experts x (W13 [3072, 4096] + W2 [4096, 1536]),
        # 2.416 G elements = 4.83 GB in, 6.19 GB out; the 48-layer job is this 48 times over one reused buffer
        torch.cuda.empty_cache()
        n_e = 128
        w13l = torch.empty(n_e, 3072, 4096, dtype=torch.bfloat16, device=dev)
        w2l = torch.empty(n_e, 4096, 1536, dtype=torch.bfloat16, device=dev)
        for wl in (w13l, w2l):
            for e0 in range(0, n_e, 16):
                wl[e0:e0 + 16].copy_((torch.randn(16, *wl.shape[1:], device=dev) * 0.015).to(torch.bfloat16))
        outs13 = (torch.empty_like(w13l), torch.empty(n_e, 3072, 2048, dtype=torch.uint8, device=dev),
                  torch.empty(n_e, 3072, 256, dtype=torch.uint8, device=dev), torch.empty(n_e, dtype=torch.float32, device=dev))
        outs2 = (torch.empty_like(w2l), torch.empty(n_e, 4096, 768, dtype=torch.uint8, device=dev),
                 torch.empty(n_e, 4096, 96, dtype=torch.uint8, device=dev), torch.empty(n_e, dtype=torch.float32, device=dev))
        lws = torch.empty(B.lib.quads_fake_quant_workspace_bytes(n_e), dtype=torch.uint8, device=dev)

        def layer_step():
            B.fake_quant_weights(w13l, out=outs13, workspace=lws)
            B.fake_quant_weights(w2l, out=outs2, workspace=lws)
        layer_step()
        tl = timed(layer_step, 3, with_flush=False)
        lms = sum(tl) / len(tl)
        n_el = w13l.numel() + w2l.numel()
        aux["aqat_layer_ms"] = lms
        aux["aqat_layer_gbs"] = n_el * 4.5625 / (lms * 1e-3) / 1e9
        aux["aqat_layer_frac_of_hbm"] = aux["aqat_layer_gbs"] / peaks["hbm_gbs"]
        aux["aqat_48_layers_s_extrapolated"] = 48 * lms * 1e-3
        del w13l, w2l, outs13, outs2
        # the same for the layer this benchmark's MoE workload is taken from (H=2048, I=768):
        # 128 experts x (W13 [1536, 2048] + W2 [2048, 768]), 0.604 G elements
        ws13 = (torch.randn(n_e, 1536, 2048, device=dev) * 0.015).to(torch.bfloat16)
        ws2 = (torch.randn(n_e, 2048, 768, device=dev) * 0.015).to(torch.bfloat16)
        os13 = (torch.empty_like(ws13), torch.empty(n_e, 1536, 1024, dtype=torch.uint8, device=dev),
                torch.empty(n_e, 1536, 128, dtype=torch.uint8, device=dev), torch.empty(n_e, dtype=torch.float32, device=dev))
        os2 = (torch.empty_like(ws2), torch.empty(n_e, 2048, 384, dtype=torch.uint8, device=dev),
               torch.empty(n_e, 2048, 48, dtype=torch.uint8, device=dev), torch.empty(n_e, dtype=torch.float32, device=dev))

        def small_layer_step():
            B.fake_quant_weights(ws13, out=os13, workspace=lws)
            B.fake_quant_weights(ws2, out=os2, workspace=lws)
        small_layer_step()
        tsl = timed(small_layer_step, 5)
        sms_ = sum(tsl) / len(tsl)
        aux["aqat_layer_h2048_ms"] = sms_
        aux["aqat_layer_h2048_frac_of_hbm"] = (ws13.numel() + ws2.numel()) * 4.5625 / (sms_ * 1e-3) / 1e9 / peaks["hbm_gbs"]
        del ws13, ws2, os13, os2
        torch.cuda.empty_cache()
        # a dense (single-expert) W4A4 + RAC projection at model scale: 8192 tokens, 4096 -> 4096, 50 % of the
        # input channels compensated; all rows belong to one weight matrix, so the CTA-pair GEMM is used
        Td, Kd, Nd = 8192, 4096, 4096
        xd = torch.randn(Td, Kd, device=dev).to(torch.bfloat16)
        wd = B.fake_quant_weights((torch.randn(1, Nd, Kd, device=dev) * 0.02).to(torch.bfloat16), want_fq=False,
                                  sf_layout=B.SF_TILED)
        wsd = torch.empty(B.moe_workspace_bytes(Td, Kd, 0, 1, 1, Nd), dtype=torch.uint8, device=dev)

        def dense_step():
            B.dense_w4a4_rac(xd, wd, Kd // 2, workspace=wsd)
        for _ in range(3):
            dense_step()
        tdn = timed(dense_step, 20)
        dms = sum(tdn) / len(tdn)
        aux["dense_linear_ms"] = dms
        aux["dense_linear_tflops_algorithmic"] = 2.0 * Td * Kd * Nd * 1.5 / (dms * 1e-3) / 1e12
        aux["dense_linear_note"] = "T=%d, %d -> %d, RAC on %d channels, activation quantized online, whole call" % (Td, Kd, Nd, Kd // 2)
        del xd, wd
        # the layer-wise mismatch ||Y_rollout - Y_learner|| / ||Y_learner|| of that projection as a function of the
        # share of compensated channels (the paper's ratios): Y_learner = QDQ_W(W) x in float32 with bf16 activations
        # (the asymmetric-QAT learner), Y_rollout = this library's W4A4 + RAC output; activations with 2 % heavy
        # channels (x25), which is where activation quantization error concentrates
        gen = torch.Generator(device=dev).manual_seed(77)
        xe = torch.randn(Td, Kd, device=dev, generator=gen)
        heavy = torch.randperm(Kd, device=dev, generator=gen)[: Kd // 50]
        xe[:, heavy] *= 25.0
        xe = xe.to(torch.bfloat16)
        we = B.fake_quant_weights((torch.randn(1, Nd, Kd, device=dev, generator=gen) * 0.02).to(torch.bfloat16),
                                  want_fq=True, sf_layout=B.SF_TILED)
        tf32 = torch.backends.cuda.matmul.allow_tf32
        torch.backends.cuda.matmul.allow_tf32 = False
        y_learner = xe.to(torch.float32) @ we["w_fq"][0].to(torch.float32).t()
        torch.backends.cuda.matmul.allow_tf32 = tf32
        ref_norm = torch.linalg.norm(y_learner).item()
        sweep = {}
        for pct in (0.0, 12.5, 25.0, 50.0, 75.0, 100.0):
            y = B.dense_w4a4_rac(xe, we, int(Kd * pct / 100.0), workspace=wsd)["out"]
            sweep["%g%%" % pct] = torch.linalg.norm(y.to(torch.float32) - y_learner).item() / ref_norm
        aux["rac_mismatch_vs_ratio"] = sweep
        # Eq. linear-mismatch on the device with the library's own modes and norms: the mismatch of each rollout
        # mode against the unquantized projection (W16A16) and against the asymmetric-QAT learner (W4A16)
        wbf = (torch.randn(Nd, Kd, device=dev, generator=gen) * 0.02).to(torch.bfloat16)
        wqq = B.fake_quant_weights(wbf.unsqueeze(0), want_fq=False, sf_layout=B.SF_TILED)
        y16 = B.dense_one_sided(xe, B.W16A16, w_bf16=wbf, workspace=wsd)["out"]
        ymodes = {"W4A16": B.dense_one_sided(xe, B.W4A16, w=wqq, workspace=wsd)["out"],
                  "W16A4": B.dense_one_sided(xe, B.W16A4, w_bf16=wbf, workspace=wsd)["out"],
                  "W4A4": B.dense_w4a4_rac(xe, wqq, 0, workspace=wsd)["out"],
                  "W4A4+RAC50%": B.dense_w4a4_rac(xe, wqq, Kd // 2, workspace=wsd)["out"]}

        def rel_(a_, b_):
            n_ = B.mismatch_norms(a_, b_).cpu().numpy()
            return float((n_[0] / n_[2]) ** 0.5)
        aux["linear_mismatch"] = {"vs_unquantized": {k_: rel_(v_, y16) for k_, v_ in ymodes.items()},
                                  "vs_w4a16_learner": {k_: rel_(v_, ymodes["W4A16"]) for k_, v_ in ymodes.items() if k_ != "W4A16"},
                                  "note": "||Y_mode - Y_ref||_F / ||Y_ref||_F for one projection (T=%d, %d -> %d), all on the "
                                          "device: W16A4 isolates the activation term, W4A16 the weight term" % (Td, Kd, Nd)}
        scores = B.rac_channel_scores(xe)
        top = torch.topk(scores, Kd // 50).indices
        aux["residual_bands"] = {"heavy_channels_among_top_2pct_scores": int(torch.isin(top // 16, heavy // 16).sum().item()),
                                 "top_2pct": Kd // 50,
                                 "score_share_of_top_2pct": float(scores[top].sum() / scores.sum())}
        del wbf, wqq, y16, ymodes
        aux["rac_mismatch_note"] = ("relative Frobenius mismatch of the W4A4 + RAC projection (T=%d, %d -> %d) against the "
                                    "learner's QDQ_W(W) x (float32 accumulate, bf16 activations), per share of compensated "
                                    "channels; output rounding to bf16 included" % (Td, Kd, Nd))
        del xe, we, y_learner, wsd
        # decode-sized batch on the same layer (the prefill and decode workloads share their weights):
        # weights cold (L2 flushed between iterations); roofline = streaming the 340 MB of weights once
        # the benchmark's own step replayed from a CUDA graph: what the eager launches and cross-stream events cost
        pgraph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(pgraph):
            step()
        for _ in range(3):
            flush_l2()
            pgraph.replay()
        tpg = timed(pgraph.replay, 20)
        aux["step_graph_ms"] = sum(tpg) / len(tpg)
        aux["step_graph_tokens_per_s"] = T / (aux["step_graph_ms"] * 1e-3)
        del pgraph
        # the paper's comparison arm on the same layer: FP8 W8A8 (E4M3, power-of-two scales per 1x128 activation /
        # 128x128 weight tile) through the library's own block-scaled FP8 grouped GEMMs; and plain W4A4 for the
        # RAC overhead.  The paper's figures (~1.3x plain W4A4 over FP8, 5-9 % RAC slowdown, +16 % QUADS over FP8)
        # are end-to-end decode throughput on its rollout engine; these are one MoE layer.
        def pack_fp8(sh):
            out = {}
            for which in ("w13", "w2"):
                parts = []
                for e0 in range(0, sh.E, 16):
                    parts.append(B.fp8_quantize_weights(synth.expert_weights(sh, which, range(e0, min(sh.E, e0 + 16))).to(dev)))
                out[which] = {k: torch.cat([p_[k] for p_ in parts]) for k in ("q", "exps", "atoms")}
            return out["w13"], out["w2"]

        f13, f2 = pack_fp8(shape)
        fws = torch.empty(B.moe_fp8_workspace_bytes(T, H, I, E, topk), dtype=torch.uint8, device=dev)

        def fp8_step():
            B.moe_fp8_w8a8(x_d, lg_d, f13, f2, topk, workspace=fws, out=out_d)

        def plain_step():
            B.moe_w4a4_rac(x_d, lg_d, gw13, gw2, topk, 0, 0, a2, workspace=ws, out=out_d)

        def w13_step():
            B.moe_w4a4_rac(x_d, lg_d, gw13, gw2, topk, H // 2, 0, a2, workspace=ws, out=out_d)
        cmp_ms = {}
        for name_, fn_ in (("fp8_w8a8", fp8_step), ("nvfp4_plain", plain_step), ("nvfp4_rac_w13", w13_step), ("nvfp4_rac_both", step)):
            for _ in range(3):
                flush_l2()
                fn_()
            tt = timed(fn_, 20)
            cmp_ms[name_] = sum(tt) / len(tt)
        assert B.moe_async_status(fws) == 0
        # how well each arm's first projection uses its own tensor-core peak (FP8 = 2 x, FP4 = 4 x the measured bf16 rate):
        # the FP8 kernels here are single-CTA 128 x 256 tiles, which need twice the bytes per MMA cycle of the FP4 ones
        B.moe_set_kernel_timing(True)
        kt = {}
        for name_, fn_ in (("fp8_w8a8", fp8_step), ("nvfp4_plain", plain_step)):
            acc_ = []
            for _ in range(5):
                flush_l2()
                fn_()
                acc_.append(B.moe_last_kernel_ms())
            kt[name_] = [sum(v[i] for v in acc_) / len(acc_) for i in (0, 1)]
        B.moe_set_kernel_timing(False)
        f1_plain = 2.0 * A * H * 2 * I
        f2_plain = 2.0 * A * I * H
        fp8_peak = 2.0 * peaks["bf16_tflops"]
        # the FP8 layer if its two GEMMs ran at the fraction of the FP8 peak that the plain-W4A4 GEMMs reach of the FP4 peak
        eq1 = f1_plain / (f1_plain / (kt["nvfp4_plain"][0] * 1e-3) / fp4_peak * fp8_peak) * 1e3
        eq2 = f2_plain / (f2_plain / (kt["nvfp4_plain"][1] * 1e-3) / fp4_peak * fp8_peak) * 1e3
        fp8_equal_ms = cmp_ms["fp8_w8a8"] - kt["fp8_w8a8"][0] - kt["fp8_w8a8"][1] + eq1 + eq2
        aux["fp8_comparison_%s" % shape.name] = {
            "fp8_ms_at_equal_gemm_efficiency": fp8_equal_ms,
            "ratios_at_equal_gemm_efficiency": {"plain_w4a4_over_fp8": fp8_equal_ms / cmp_ms["nvfp4_plain"],
                                                "rac_w13_over_fp8": fp8_equal_ms / cmp_ms["nvfp4_rac_w13"],
                                                "rac_both_over_fp8": fp8_equal_ms / cmp_ms["nvfp4_rac_both"]},
            "gemm_ms": kt,
            "gemm1_frac_of_own_peak": {"fp8_w8a8": f1_plain / (kt["fp8_w8a8"][0] * 1e-3) / 1e12 / (2.0 * peaks["bf16_tflops"]),
                                       "nvfp4_plain": f1_plain / (kt["nvfp4_plain"][0] * 1e-3) / 1e12 / fp4_peak},
            "fairness": "gemm1_frac_of_own_peak says how much of its own tensor-core peak (FP8 = 2 x, FP4 = 4 x the measured "
                        "bf16 rate) each arm's first projection reaches; fp8_ms_at_equal_gemm_efficiency re-scales the FP8 GEMMs to "
                        "the FP4 kernels' fraction, so the ratios can be read either way",
            "ms_per_layer": cmp_ms,
            "plain_w4a4_over_fp8": cmp_ms["fp8_w8a8"] / cmp_ms["nvfp4_plain"],
            "rac_w13_over_fp8": cmp_ms["fp8_w8a8"] / cmp_ms["nvfp4_rac_w13"],
            "rac_both_over_fp8": cmp_ms["fp8_w8a8"] / cmp_ms["nvfp4_rac_both"],
            "rac_w13_slowdown_vs_plain": 1.0 - cmp_ms["nvfp4_plain"] / cmp_ms["nvfp4_rac_w13"],
            "paper": {"plain_w4a4_over_fp8": 1.3, "quads_over_fp8": 1.16, "rac_slowdown_vs_plain": "5-9 %",
                      "what": "end-to-end decode tokens/s on the paper's rollout engine (context, other hardware)"}}
        del fws
        if args.workload == "prefill":
            dsh = synth.MOE_SHAPES["decode"]
            dn13, dn2 = nsel_of(dsh, args.variant)
            dx, _ = synth.activations(dsh)
            dlg = synth.router_logits(dsh)
            dx, dlg = dx.to(dev), dlg.to(dev)
            da2 = torch.tensor([synth.H_GLOBAL_SCALE[dsh.name]], dtype=torch.float32, device=dev)
            dws = torch.empty(B.moe_workspace_bytes(dsh.T, dsh.H, dsh.I, dsh.E, dsh.topk), dtype=torch.uint8, device=dev)
            dout = torch.empty(dsh.T, dsh.H, dtype=torch.bfloat16, device=dev)

            def dstep():
                B.moe_w4a4_rac(dx, dlg, gw13, gw2, dsh.topk, dn13, dn2, da2, workspace=dws, out=dout)
            for _ in range(5):
                flush_l2()
                dstep()
            td = timed(dstep, 50)
            dms = sum(td) / len(td)
            wbytes = sum(t.numel() * t.element_size() for g in (gw13, gw2) for t in g.values())
            aux["decode_ms_per_step"] = dms
            aux["decode_tokens_per_s"] = dsh.T / (dms * 1e-3)
            aux["decode_weight_stream_gbs"] = wbytes / (dms * 1e-3) / 1e9
            aux["decode_frac_of_hbm"] = aux["decode_weight_stream_gbs"] / peaks["hbm_gbs"]
            aux["decode_note"] = "T=%d on the same layer, cold weights (%.0f MB streamed per step)" % (dsh.T, wbytes / 1e6)
            # FP8 and plain W4A4 on the decode batch (the paper's throughput comparison is a decode one)
            dfws = torch.empty(B.moe_fp8_workspace_bytes(dsh.T, dsh.H, dsh.I, dsh.E, dsh.topk), dtype=torch.uint8, device=dev)

            def d_fp8():
                B.moe_fp8_w8a8(dx, dlg, f13, f2, dsh.topk, workspace=dfws, out=dout)

            def d_plain():
                B.moe_w4a4_rac(dx, dlg, gw13, gw2, dsh.topk, 0, 0, da2, workspace=dws, out=dout)

            def d_w13():
                B.moe_w4a4_rac(dx, dlg, gw13, gw2, dsh.topk, dsh.H // 2, 0, da2, workspace=dws, out=dout)
            dcmp = {"nvfp4_rac_both": dms}
            for name_, fn_ in (("fp8_w8a8", d_fp8), ("nvfp4_plain", d_plain), ("nvfp4_rac_w13", d_w13)):
                for _ in range(3):
                    flush_l2()
                    fn_()
                tt = timed(fn_, 30)
                dcmp[name_] = sum(tt) / len(tt)
            fbytes = sum(t.numel() for g_ in (f13, f2) for t in (g_["q"], g_["atoms"]))
            aux["fp8_comparison_decode"] = {
                "ms_per_layer": dcmp, "plain_w4a4_over_fp8": dcmp["fp8_w8a8"] / dcmp["nvfp4_plain"],
                "rac_w13_over_fp8": dcmp["fp8_w8a8"] / dcmp["nvfp4_rac_w13"],
                "rac_both_over_fp8": dcmp["fp8_w8a8"] / dcmp["nvfp4_rac_both"],
                "rac_w13_slowdown_vs_plain": 1.0 - dcmp["nvfp4_plain"] / dcmp["nvfp4_rac_w13"],
                "weight_bytes": {"fp8": fbytes, "nvfp4": wbytes},
                "note": "T=%d, cold weights; the FP8 path runs 128-row tiles (no operand-swapped kernel for it)" % dsh.T}
            del dfws
            # the same call replayed from a CUDA graph (what a decode loop does)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                dstep()
            for _ in range(3):
                flush_l2()
                graph.replay()
            tg = timed(graph.replay, 50)
            aux["decode_graph_ms_per_step"] = sum(tg) / len(tg)
            aux["decode_graph_tokens_per_s"] = dsh.T / (aux["decode_graph_ms_per_step"] * 1e-3)
            # a 48-layer stack of such layers (each with its own weights, 16 GB in all), static activation
            # scales, every layer's output feeding the next, captured once and replayed as one CUDA graph
            n_layers = 48
            layers = []
            for l in range(n_layers):
                g13 = {k: (v.clone() if l else v) for k, v in gw13.items()}
                g2 = {k: (v.clone() if l else v) for k, v in gw2.items()}
                layers.append((g13, g2, (dlg + 0.37 * l).contiguous()))
            a13 = torch.tensor([float(dx.abs().max()) / 2688.0], dtype=torch.float32, device=dev)
            hbuf = [torch.empty_like(dx), torch.empty_like(dx)]

            def stack():
                cur = dx
                for l, (g13, g2, lg_l) in enumerate(layers):
                    nxt = hbuf[l & 1]
                    B.moe_w4a4_rac(cur, lg_l, g13, g2, dsh.topk, dn13, dn2, da2, a13_gs=a13, workspace=dws, out=nxt)
                    cur = nxt
            stack()
            torch.cuda.synchronize()
            g48 = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g48):
                stack()
            for _ in range(2):
                g48.replay()
            t48 = timed(g48.replay, 10, with_flush=False)
            ms48 = sum(t48) / len(t48)
            aux["decode_48_layers_graph_ms"] = ms48
            aux["decode_48_layers_tokens_per_s"] = dsh.T / (ms48 * 1e-3)
            aux["decode_48_layers_weight_stream_gbs"] = n_layers * wbytes / (ms48 * 1e-3) / 1e9
            aux["decode_48_layers_note"] = ("%d MoE layers x %.0f MB of weights, T=%d, static activation scales, one graph "
                                            "replay per step") % (n_layers, wbytes / 1e6, dsh.T)
            del layers
            # the large layer (T=4096, H=4096, I=1536, 128 experts, ~256 rows per expert: the size
            # where weight streaming and the tensor pipe are about level), weights drawn on the device
            lsh = synth.MOE_SHAPES["large"]
            gl = torch.Generator(device=dev)
            gl.manual_seed(lsh.seed)

            def pack_large(rows, cols):
                parts = []
                for e0 in range(0, lsh.E, 16):
                    w = (torch.randn(16, rows, cols, generator=gl, device=dev) * lsh.w_std).to(torch.bfloat16)
                    parts.append(B.fake_quant_weights(w, want_fq=False, sf_layout=B.SF_TILED))
                    del w
                return {k: torch.cat([p[k] for p in parts]) for k in ("q", "sf", "gs")}
            l13, l2 = pack_large(2 * lsh.I, lsh.H), pack_large(lsh.H, lsh.I)
            lx, _ = synth.activations(lsh)
            llg = synth.router_logits(lsh)
            lx, llg = lx.to(dev), llg.to(dev)
            la2 = torch.tensor([synth.H_GLOBAL_SCALE[lsh.name]], dtype=torch.float32, device=dev)
            lws = torch.empty(B.moe_workspace_bytes(lsh.T, lsh.H, lsh.I, lsh.E, lsh.topk), dtype=torch.uint8, device=dev)
            lout = torch.empty(lsh.T, lsh.H, dtype=torch.bfloat16, device=dev)
            large = {}
            for vname, (v13, v2) in (("rac_both", (lsh.H // 2, lsh.I // 2)), ("rac_w13", (lsh.H // 2, 0)), ("plain", (0, 0))):
                def lstep(v13=v13, v2=v2):
                    B.moe_w4a4_rac(lx, llg, l13, l2, lsh.topk, v13, v2, la2, workspace=lws, out=lout)
                for _ in range(3):
                    flush_l2()
                    lstep()
                tl = timed(lstep, 20)
                lms = sum(tl) / len(tl)
                A_l = lsh.T * lsh.topk
                f_alg = 6.0 * A_l * lsh.H * lsh.I * (1.0 + (2.0 / 3.0) * v13 / lsh.H + (1.0 / 3.0) * v2 / lsh.I)
                large[vname] = {"ms_per_step": lms, "tokens_per_s": lsh.T / (lms * 1e-3),
                                "algorithmic_tflops": f_alg / (lms * 1e-3) / 1e12,
                                "frac_of_fp4_peak": f_alg / (lms * 1e-3) / 1e12 / fp4_peak}
            assert B.moe_async_status(lws) == 0
            lbytes = sum(t.numel() * t.element_size() for g_ in (l13, l2) for t in g_.values())
            large["weight_bytes"] = lbytes
            large["weight_stream_floor_ms"] = lbytes / (peaks["hbm_gbs"] * 1e9) * 1e3
            large["note"] = ("T=%d, H=%d, I=%d, E=%d, top-%d; cold weights, L2 flushed between steps; weights N(0, %.3f) "
                             "drawn on the device" % (lsh.T, lsh.H, lsh.I, lsh.E, lsh.topk, lsh.w_std))
            aux["large_layer"] = large
            del l13, l2, lws
        line["aux"] = aux

    if world == 1 and not args.no_cpu_baseline:
        step_o, T_s, desc = oracle_sample(shape, args.variant, 52.0)   # ~32 tokens: ~10 s of oracle work
        t0 = time.perf_counter()
        step_o()
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": T_s / dt, "unit": UNIT, "cores": cpu_threads(), "kind": "oracle",
                                "sample": desc, "seconds": dt}
    else:
        line["cpu_baseline"] = None
    print(json.dumps(line))
    D.shutdown()


def main():
    args = parse()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
