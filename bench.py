"""Benchmark of the VeLoRA linear forward + backward path on B200.

Workload (``config.workload``): the seven projections of one LLaMA-7B-shaped block
(q/k/v/o 4096->4096, up/gate 4096->11008, down 11008->4096), a batch of 4 x 2048 = 8192 tokens,
sub-token length 64, bf16 data with fp32 accumulation, seeded synthetic activations and gradients.
One step = for every layer: velora_linear_forward (Y = X W^T and Z = compress(X, v)) followed by
velora_linear_backward (dX = dY W and the factored weight gradient).  The metric is tokens per second
through that fwd+bwd pass.  Every tensor set is several times larger than L2, so nothing is served
from cache between steps.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints one JSON line (rank 0).  ``--impl reference`` times the fp64 CPU oracle on a bounded sample.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "velora_linear_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"
CONFIG_DEFAULT = 5
CONFIG_INDEX = CONFIG_DEFAULT
DSUB = 64
DSUB_SWEEP = 256                # the second sub-token length of configuration 5 (kernel table rows only)
CPU_SAMPLE_TOKENS = 128         # oracle leg of the default run: tokens per layer, all host threads, one pass (about 30 s)
CPU_SINGLE_TOKENS = 4           # the same with one thread (about 10 s)
REF_SAMPLE_TOKENS = 32          # --impl reference: tokens per layer and step (23 passes stay within a few minutes)
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
GEMM_TRAFFIC_RATIO = 1.10       # ncu dram bytes / algorithmic bytes of the fused forward gemm_pair_kernel on the q layer


def peaks():
    """Measured peaks of this machine's B200s if present, else the stated fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.005):
        self.index, self.period = index, period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _names(self, mask: int):
        nv = self.nv
        table = {
            "sw_power_cap": getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4),
            "hw_slowdown": getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40),
            "hw_power_brake_slowdown": getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80),
        }
        return [k for k, bit in table.items() if mask & bit]

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                self.reasons.update(self._names(int(mask)))
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)

    def summary(self):
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


# ------------------------------------------------------------------ multi-rank helpers (host logic)
def aggregate_over_ranks(elapsed_ms_local: float, tokens_local: int, dist=None, device=None):
    """MAX of the elapsed time and SUM of the tokens over all ranks (identity without a process group)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return elapsed_ms_local, tokens_local
    import torch
    t = torch.tensor([elapsed_ms_local], dtype=torch.float64, device=device)
    n = torch.tensor([tokens_local], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), int(n.item())


def layer_flops(N, D, O, M):
    """Algorithmic flops: the two dense products and the factored weight gradient."""
    return {"fwd": 2.0 * N * D * O, "dx": 2.0 * N * D * O, "dw": 2.0 * N * O * M + O * D}


# ------------------------------------------------------------------ CPU oracle leg
def oracle_prepare(cfg, sample_tokens: int):
    """Inputs of the oracle sample: the first ``sample_tokens`` tokens of every layer, widened to fp64."""
    import oracle
    import velora_inputs as vi
    layers = []
    for li, layer in enumerate(cfg.layers):
        X = vi.make_X(cfg, li, N=sample_tokens).f64()
        W = vi.make_W(cfg, li).f64()
        dY = vi.make_dY(cfg, li, N=sample_tokens).f64()
        v = oracle.init_v(X + 0.01, DSUB)
        layers.append((X, W, dY, v, layer.D))
    return layers


def set_oracle_threads(n: int) -> bool:
    """Number of OpenMP threads the (unchanged) oracle library runs with from now on; False if the
    OpenMP runtime cannot be reached."""
    import ctypes
    try:
        ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))
        return True
    except OSError:
        return False


def oracle_step(layers):
    """One pass of the oracle, as it stands: forward product, compress, input gradient and the weight
    gradient by its plain definition, for every layer."""
    import oracle
    for X, W, dY, v, D in layers:
        oracle.linear_forward(X, W)
        Z = oracle.compress(X, v)
        oracle.input_grad(dY, W)
        oracle.weight_grad(dY, Z, v, D)


def cpu_sample_text(tokens: int) -> str:
    return ("first %d of the %%d tokens of every layer, each layer in full (forward product, compress, input "
            "gradient, weight gradient by its plain definition); tokens/s = %d / time of one pass, i.e. "
            "extrapolated linearly in tokens" % (tokens, tokens))


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    import velora_inputs as vi
    cfg = vi.CONFIGS[CONFIG_INDEX]
    oracle.build()
    layers = oracle_prepare(cfg, REF_SAMPLE_TOKENS)
    for _ in range(args.warmup):
        oracle_step(layers)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(layers)
    per_step = (time.perf_counter() - t0) / max(args.steps, 1)
    value = REF_SAMPLE_TOKENS / per_step
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(cfg),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(oracle.threads(), REF_SAMPLE_TOKENS), "kind": "oracle",
                         "sample": cpu_sample_text(REF_SAMPLE_TOKENS) % cfg.N},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def workload_config(cfg):
    if cfg.index == 5:
        layers = "7 projections (q,k,v,o 4096x4096; up,gate 4096x11008; down 11008x4096)"
        l2 = "inputs larger than L2 (each step touches > 2 GB)"
    else:
        layers = "%d projections (%s)" % (len(cfg.layers), ", ".join("%s %dx%d" % (l.name, l.D, l.O) for l in cfg.layers))
        step_bytes = sum(cfg.N * (l.D + l.O) * 4 + l.O * l.D * 4 for l in cfg.layers)
        l2 = "each step touches %.0f MB (L2 is 126 MB): %s" % (step_bytes / 1e6, "larger than L2" if step_bytes > 126e6 else "partly L2-resident")
    return {"workload": "config %d: %s, N=%d tokens, %s, Dsub=%d" % (cfg.index, cfg.name, cfg.N, layers, DSUB),
            "tokens": cfg.N, "Dsub": DSUB, "z_dtype": "f32", "dw": "factored", "l2": l2}


# ------------------------------------------------------------------ GPU leg
def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2405_17991_b200 as vl
    import velora_inputs as vi

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    vl.lib()

    cfg = vi.CONFIGS[CONFIG_INDEX]
    N = cfg.N
    pk = peaks()

    # ---- inputs: generated once on the host (seeded), pinned, then resident in HBM
    full = cfg.index == CONFIG_DEFAULT            # kernel table and the end-to-end leg belong to the headline workload
    pad8 = lambda n: -(-n // 8) * 8                # row pitch a multiple of 16 bytes (config 4: 5461 -> 5464)
    L = []
    for li, layer in enumerate(cfg.layers):
        Xa, dYa, Wa = vi.make_X(cfg, li), vi.make_dY(cfg, li), vi.make_W(cfg, li)
        hX = Xa.torch("cpu").pin_memory() if full else None
        hdY = dYa.torch("cpu").pin_memory() if full else None
        W = Wa.torch(dev, ld=pad8(layer.D))
        X, dY = Xa.torch(dev, ld=pad8(layer.D)), dYa.torch(dev, ld=pad8(layer.O))
        M = vl.num_subtokens(layer.D, DSUB)
        v = vl.velora_init_v(X, DSUB)
        L.append({
            "name": layer.name, "D": layer.D, "O": layer.O, "M": M, "hX": hX, "hdY": hdY, "X": X, "dY": dY, "W": W,
            "v": v, "Y": torch.empty((N, pad8(layer.O)), dtype=torch.bfloat16, device=dev)[:, :layer.O],
            "Z": torch.empty((N, M), dtype=torch.float32, device=dev),
            "dX": torch.empty((N, pad8(layer.D)), dtype=torch.bfloat16, device=dev)[:, :layer.D],
            "dW": torch.empty((layer.O, pad8(layer.D)), dtype=torch.bfloat16, device=dev)[:, :layer.D],
        })
    ws_bytes = max(vl.velora_workspace_bytes(vl.OP_LINEAR_BACKWARD_FACTORED, N, l["D"], l["O"], DSUB) for l in L)
    ws = vl.velora_workspace_alloc(ws_bytes, dev)

    def step(events=None):
        for l in L:
            if events is not None:
                e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
                e0.record()
            vl.velora_linear_forward(l["X"], l["W"], l["v"], Y=l["Y"], Z=l["Z"], ws=ws)
            if events is not None:
                e1.record()
            vl.velora_linear_backward(l["dY"], l["W"], l["Z"], l["v"], dX=l["dX"], dW=l["dW"], ws=ws)
            if events is not None:
                e2.record()
                events.append((l, e0, e1, e2))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    launches0 = vl.velora_launch_count()
    events = []
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        barrier()
        start.record()
        for _ in range(args.steps):
            step(events)
        end.record()
        barrier()
    elapsed_ms = start.elapsed_time(end)
    launches = vl.velora_launch_count() - launches0
    graph_ms = None
    if args.graph:
        # The same step captured once into a CUDA graph and replayed: what a launch-bound configuration gains
        # when the host submits one graph instead of 4-5 kernels per layer.  Reported beside the plain figure.
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            step()
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            step()
        for _ in range(3):
            g.replay()
        barrier()
        gs, ge = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        gs.record()
        for _ in range(args.steps):
            g.replay()
        ge.record()
        barrier()
        graph_ms = gs.elapsed_time(ge) / args.steps
    # ---- the same layers WITHOUT the method (what the paper calls full fine-tuning): Y = X W^T keeping X,
    # dX = dY W, dW = dY^T X as a dense product.  Same tensor-core kernels, same buffers, same number of steps.
    def plain_step():
        for l in L:
            vl.velora_dense_product(vl.PRODUCT_A_BT, l["X"], l["W"], C=l["Y"], ws=ws)
            vl.velora_dense_product(vl.PRODUCT_A_B, l["dY"], l["W"], C=l["dX"], ws=ws)
            vl.velora_dense_product(vl.PRODUCT_AT_B, l["dY"], l["X"], C=l["dW"], ws=ws)

    for _ in range(3):
        plain_step()
    barrier()
    ps, pe = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ps.record()
    for _ in range(args.steps):
        plain_step()
    pe.record()
    barrier()
    plain_ms = ps.elapsed_time(pe) / args.steps
    status = vl.velora_workspace_status(ws)
    if status != 0:
        raise RuntimeError("device status %d (%s) after the timed region" % (status, vl.velora_status_string(status)))
    total_ms, total_tokens = aggregate_over_ranks(elapsed_ms, N * args.steps, dist if world > 1 else None, dev)
    value = total_tokens / (total_ms * 1e-3)

    # ---- roofline of the dominant kernel (the forward tensor-core GEMM), from the events of the timed region
    fwd_ms = sum(e0.elapsed_time(e1) for (_, e0, e1, _) in events)
    bwd_ms = sum(e1.elapsed_time(e2) for (_, _, e1, e2) in events)
    fwd_flops = sum(layer_flops(N, l["D"], l["O"], l["M"])["fwd"] for (l, _, _, _) in events)
    achieved = fwd_flops / (fwd_ms * 1e-3) / 1e12
    # Which measured peak applies: the burst figure unless the timed region is seconds long (only then has the
    # power cap pulled the clocks down to where the sustained figure was taken).
    region_s = elapsed_ms * 1e-3
    long_region = region_s >= 2.0
    peak = pk["bf16_tflops_sustained"] if long_region else pk["bf16_tflops"]
    clk = clocks.summary()
    clock_scaled = None
    if clk.get("sm_mhz") and clk.get("sm_max_mhz"):
        # what the same kernel would reach if the clock had stayed at its maximum: lets boxes be compared
        clock_scaled = {"achieved_at_max_clock": achieved * clk["sm_max_mhz"] / clk["sm_mhz"],
                        "sm_mhz_median": clk["sm_mhz"], "sm_max_mhz": clk["sm_max_mhz"]}
    # DRAM traffic per launch: ncu on the q-layer launch of this kernel (compress riding along) read + wrote
    # 187 MB = 1.10 x the 169.9 MB of algorithmic bytes X + W + Y + Z (every operand crosses HBM about once);
    # the other layers of the step run the same kernel with the same tile walk and are scaled by their
    # algorithmic bytes.
    fwd_bytes = sum((N * l["D"] + l["O"] * l["D"] + N * l["O"]) * 2 + N * l["M"] * 4 for (l, _, _, _) in events)
    traffic = GEMM_TRAFFIC_RATIO * fwd_bytes / max(len(events), 1)
    roofline = {"kernel": "velora_linear_forward (tensor-core GEMM Y = X W^T with compress)", "bound": "tensor",
                "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                "peak_source": "%s, %s bf16 GEMM (timed region %.2f s)" % (pk["source"], "sustained" if long_region else "burst", region_s),
                "frac_burst": achieved / pk["bf16_tflops"], "frac_sustained": achieved / pk["bf16_tflops_sustained"],
                "frac_nominal": achieved / NOMINAL_BF16_TFLOPS, "clock_scaled": clock_scaled,
                "traffic": traffic,
                "traffic_unit": "bytes per launch (average over the 7 layers; q-layer ncu capture, scaled)",
                "launches": len(events), "avg_launch_ms": fwd_ms / max(len(events), 1),
                "fwd_ms_per_step": fwd_ms / args.steps, "bwd_ms_per_step": bwd_ms / args.steps}
    overhead = {"velora_ms_per_step": elapsed_ms / args.steps, "plain_ms_per_step": plain_ms,
                "velora_over_plain": (elapsed_ms / args.steps) / plain_ms,
                "plain": "the same layers without the method: Y = X W^T, dX = dY W, dW = dY^T X (dense), X kept",
                "paper": "Table 7 reports VeLoRA 4-9 % slower than full fine-tuning (other hardware, whole model)"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": workload_config(cfg), "clocks": clk,
        "gpu_launches": int(launches), "roofline": roofline, "overhead_vs_plain": overhead,
    }
    if graph_ms is not None:
        line["cuda_graph"] = {"ms_per_step": graph_ms, "value": N * world / (graph_ms * 1e-3), "unit": UNIT,
                              "note": "the same step replayed from one captured graph (this rank's time)"}

    if not full:                                   # a parity-test configuration timed on request: the step only
        # These configurations fit (partly) in L2, so the figure above is a WARM one: every step reads what the
        # step before left in the cache.  The COLD figure rotates through enough copies of all buffers that a
        # step finds none of its operands in L2 (the copies together hold more than twice the L2's 126 MB).
        step_bytes = sum((N * (l["D"] + l["O"]) * 2 + l["O"] * l["D"] * 2) * 2 + N * l["M"] * 4 for l in L)
        copies = int(min(16, max(2, -(-2 * 126e6 // step_bytes) + 1)))
        sets = [L]
        for _ in range(copies - 1):
            # copies keep the row pitch of the originals (a plain clone would pack the padded rows)
            sets.append([{k: (torch.empty_strided(v.shape, v.stride(), dtype=v.dtype, device=v.device).copy_(v)
                              if isinstance(v, torch.Tensor) and v.is_cuda else v) for k, v in l.items()} for l in L])

        def step_on(Ls):
            for l in Ls:
                vl.velora_linear_forward(l["X"], l["W"], l["v"], Y=l["Y"], Z=l["Z"], ws=ws)
                vl.velora_linear_backward(l["dY"], l["W"], l["Z"], l["v"], dX=l["dX"], dW=l["dW"], ws=ws)

        def time_steps(pick):
            for Ls in sets:
                step_on(Ls)
            barrier()
            cs, ce = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            cs.record()
            for i in range(args.steps):
                step_on(pick(i))
            ce.record()
            barrier()
            return cs.elapsed_time(ce) / args.steps

        warm_ms = time_steps(lambda i: sets[0])        # both without the per-layer events of the headline loop
        cold_ms = time_steps(lambda i: sets[i % copies])
        line["l2"] = {"warm_ms_per_step": warm_ms, "warm_tokens_per_s": N * world / (warm_ms * 1e-3),
                      "cold_ms_per_step": cold_ms, "cold_tokens_per_s": N * world / (cold_ms * 1e-3),
                      "copies_rotated": copies, "bytes_per_step": step_bytes,
                      "note": "warm = one set of buffers step after step (partly L2-resident, like value / ms_per_step, which "
                              "also carry three event records per layer); cold = the same step rotating through copies of "
                              "every buffer so that nothing is found in L2"}
        if rank == 0:
            line["roofline"]["traffic"] = None         # the capture behind the ratio was taken on configuration 5
            print(json.dumps(line))
        if world > 1:
            dist.destroy_process_group()
        return
    if rank == 0:
        line["kernels"] = kernel_table(vl, torch, L, N, ws, pk)
        # the metric's other two quantities (and reconstruct), per shape, inside the roofline object
        def pick(prefix):
            rows = []
            for r in line["kernels"]:
                if r["kernel"].startswith(prefix):
                    row = {"shape": r["shape"], "Dsub": r["Dsub"], "bytes": r["bytes"], "us": r["us"], "GB/s": r["GB/s"],
                           "frac": r["frac_measured"], "frac_nominal_8TBs": r["GB/s"] / NOMINAL_HBM_GBS}
                    for k_src, k_dst in (("us_back_to_back", "us_back_to_back"), ("frac_measured_back_to_back", "frac_back_to_back"),
                                         ("us_graph", "us_graph"), ("frac_measured_graph", "frac_graph"),
                                         ("TFLOP/s", "TFLOP/s"), ("roofline_TFLOP/s", "roofline_TFLOP/s")):
                        if k_src in r:
                            row[k_dst] = r[k_src]
                    rows.append(row)
            return rows
        line["roofline"]["hbm_peak_GB/s"] = pk["hbm_gbs"]
        floor = line["kernels"][0]
        line["roofline"]["timing_floor_us"] = {
            "per_call": floor["us"], "back_to_back": floor["us_back_to_back"], "graph": floor["us_graph"],
            "note": "device time of the smallest compress (one CTA) timed the same three ways: `us` = one call between its own "
                    "pair of CUDA events, `us_back_to_back` = calls queued behind one another inside one pair of events, "
                    "`us_graph` = the same calls replayed from a CUDA graph. A kernel of 10-30 us cannot show more than "
                    "t_min / (t_min + per_call floor) in the per-call column."}
        line["roofline"]["compress"] = pick("compress")
        line["roofline"]["reconstruct"] = pick("reconstruct")
        line["roofline"]["weight_grad_factored"] = pick("weight_grad factored")

    # ---- end to end: host buffers in, gradients out, through velora_linear_step_host.  Three streams, each
    # with its own staging area and workspace, take the layers in turn, so that one layer's copies from and
    # to the host overlap the neighbouring layers' kernels (the copies dominate: 1.28 GB in, 0.40 GB out).
    e2e_steps = max(1, min(args.steps, 5))
    n_streams = 3
    staging_bytes = max(vl.velora_host_step_staging_bytes(N, l["D"], l["O"], DSUB) for l in L)
    lanes = []
    for _ in range(n_streams):
        w = vl.velora_workspace_alloc(ws.numel(), dev)
        lanes.append({"stream": torch.cuda.Stream(device=dev), "staging": torch.empty(staging_bytes, dtype=torch.uint8, device=dev),
                      "ws": w, "done": torch.cuda.Event()})
    for l in L:
        l["hdW"] = torch.empty((l["O"], l["D"]), dtype=torch.bfloat16).pin_memory()
    torch.cuda.synchronize(dev)

    def host_steps(count):
        """`count` steps; returns after the current stream has been made to wait for all of them."""
        start = torch.cuda.Event()
        start.record()
        for ln in lanes:
            ln["stream"].wait_event(start)
        i = 0
        for _ in range(count):
            for l in L:
                ln = lanes[i % n_streams]
                i += 1
                vl.velora_linear_step_host(l["hX"], l["hdY"], l["W"], l["v"], ln["staging"], ln["ws"], hdW=l["hdW"],
                                           stream=ln["stream"])
        for ln in lanes:
            ln["done"].record(ln["stream"])
            torch.cuda.current_stream().wait_event(ln["done"])

    host_steps(1)
    barrier()
    s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s2.record()
    host_steps(e2e_steps)
    e2.record()
    barrier()
    for ln in lanes:
        if vl.velora_workspace_status(ln["ws"]) != 0:
            raise RuntimeError("device status raised during the end-to-end steps")
    e2e_ms, e2e_tokens = aggregate_over_ranks(s2.elapsed_time(e2), N * e2e_steps, dist if world > 1 else None, dev)
    line["e2e"] = {
        "value": e2e_tokens / (e2e_ms * 1e-3), "unit": UNIT, "steps": e2e_steps,
        "h2d_bytes_per_step": int(sum(N * (l["D"] + l["O"]) * 2 for l in L)),
        "d2h_bytes_per_step": int(sum(l["O"] * l["D"] * 2 for l in L)),
        "api": "velora_linear_step_host (pinned host X, dY in; dW out), layers dealt round-robin to %d streams" % n_streams,
    }

    if rank == 0:
        import oracle
        threads = oracle.threads()
        layers = oracle_prepare(cfg, CPU_SAMPLE_TOKENS)
        t0 = time.perf_counter()
        oracle_step(layers)
        t_cpu = time.perf_counter() - t0
        line["cpu_baseline"] = {
            "value": CPU_SAMPLE_TOKENS / t_cpu, "unit": UNIT, "cores": min(threads, CPU_SAMPLE_TOKENS), "kind": "oracle",
            "sample": cpu_sample_text(CPU_SAMPLE_TOKENS) % N + "; one pass, %.1f s" % t_cpu,
        }
        if set_oracle_threads(1):
            single = [tuple(a[:CPU_SINGLE_TOKENS] if i in (0, 2) else a for i, a in enumerate(t)) for t in layers]
            t0 = time.perf_counter()
            oracle_step(single)
            t_one = time.perf_counter() - t0
            set_oracle_threads(threads)
            line["cpu_baseline"]["single_thread"] = {
                "value": CPU_SINGLE_TOKENS / t_one, "unit": UNIT, "cores": 1,
                "sample": cpu_sample_text(CPU_SINGLE_TOKENS) % N + "; one pass, %.1f s" % t_one}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def kernel_table(vl, torch, L, N, ws, pk):
    """Per-kernel device times (CUDA events, inputs rotated so that every launch misses L2)."""
    dev = L[0]["X"].device
    by = {l["name"]: l for l in L}
    out = []

    def timed(fn_list, reps=7):
        """Median device time of one call (ms): every call is bracketed by its own pair of CUDA events."""
        for f in fn_list:
            f()
        torch.cuda.synchronize()
        # Keep the GPU busy for ~2 ms first, so that every call below is already queued when its turn
        # comes: the event pairs then time device work only, not the host's submission latency.
        torch.cuda._sleep(4_000_000)
        pairs = []
        for _ in range(reps):
            for f in fn_list:
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                f()
                b.record()
                pairs.append((a, b))
        torch.cuda.synchronize()
        times = sorted(a.elapsed_time(b) for a, b in pairs)
        return times[len(times) // 2]

    def timed_b2b(fn_list, reps=7):
        """Device time per call (ms) of reps x len(fn_list) calls queued back to back inside ONE pair of
        events: what a call costs inside a long step, where the next launch is already waiting when a kernel
        ends.  (A pair of events around a single short kernel also times 6-7 us of launch and completion
        latency: the compress kernel's own first-CTA-start to last-CTA-end span on the 67 MB input is 12.6 us
        when the events around it read 19.5 us.)"""
        torch.cuda.synchronize()
        torch.cuda._sleep(4_000_000)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            for f in fn_list:
                f()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (reps * len(fn_list))

    def timed_graph(fn_list, rounds=5, reps=5):
        """Device time per call (ms) when rounds x len(fn_list) calls are captured once into a CUDA graph and
        the graph is replayed: no host submission at all between the kernels, so this is what a call costs the
        GPU inside a captured step (kernel, launch gap and drain), free of the event pair's own latency and of
        the host's submission rate, which bounds the back-to-back figure of the shortest kernels."""
        torch.cuda.synchronize()
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for f in fn_list:
                f()
        torch.cuda.current_stream().wait_stream(side)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            for _ in range(rounds):
                for f in fn_list:
                    f()
        g.replay()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            g.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / (rounds * reps * len(fn_list))

    def hbm(name, shape, ms, nbytes, ms_b2b=None, dsub=DSUB, ms_graph=None):
        gbs = nbytes / (ms * 1e-3) / 1e9
        row = {"kernel": name, "shape": shape, "Dsub": dsub, "bytes": nbytes, "us": ms * 1e3, "GB/s": gbs, "bound": "hbm",
               "frac_measured": gbs / pk["hbm_gbs"], "frac_nominal_8TBs": gbs / NOMINAL_HBM_GBS}
        if ms_b2b is not None:
            g2 = nbytes / (ms_b2b * 1e-3) / 1e9
            row.update({"us_back_to_back": ms_b2b * 1e3, "GB/s_back_to_back": g2,
                        "frac_measured_back_to_back": g2 / pk["hbm_gbs"], "frac_nominal_8TBs_back_to_back": g2 / NOMINAL_HBM_GBS})
        if ms_graph is not None:
            g3 = nbytes / (ms_graph * 1e-3) / 1e9
            row.update({"us_graph": ms_graph * 1e3, "GB/s_graph": g3, "frac_measured_graph": g3 / pk["hbm_gbs"]})
        out.append(row)

    def tensor(name, shape, ms, flops, nbytes=None, dsub=DSUB):
        tf = flops / (ms * 1e-3) / 1e12
        row = {"kernel": name, "shape": shape, "Dsub": dsub, "us": ms * 1e3, "TFLOP/s": tf, "bound": "tensor",
               "frac_measured_burst": tf / pk["bf16_tflops"], "frac_nominal": tf / NOMINAL_BF16_TFLOPS}
        if nbytes is not None:                         # factored dW: HBM-bound, graded on bytes
            gbs = nbytes / (ms * 1e-3) / 1e9
            ai = flops / nbytes
            row.update({"bound": "hbm", "bytes": nbytes, "GB/s": gbs, "frac_measured": gbs / pk["hbm_gbs"],
                        "roofline_TFLOP/s": min(pk["bf16_tflops"], ai * pk["hbm_gbs"] / 1e3)})
        out.append(row)

    # What the three ways of timing cost by themselves: the smallest compress (8 tokens of 64 columns, one CTA).
    tx = torch.zeros((8, 64), dtype=torch.bfloat16, device=dev)
    tv = torch.ones(64, dtype=torch.float32, device=dev)
    tz = torch.empty((8, 1), dtype=torch.float32, device=dev)
    tiny = [lambda: vl.velora_compress(tx, tv, Z=tz)]
    out.append({"kernel": "timing floor: compress of 8 tokens x 64 columns (one CTA)", "shape": "N=8 D=64", "Dsub": 64,
                "bound": "latency", "us": timed(tiny, reps=21) * 1e3, "us_back_to_back": timed_b2b(tiny, reps=50) * 1e3,
                "us_graph": timed_graph(tiny, rounds=20) * 1e3})

    # The second sub-token length of the configuration: its own v and Z per layer.
    for l in L:
        l["M2"] = vl.num_subtokens(l["D"], DSUB_SWEEP)
        l["v2"] = vl.velora_init_v(l["X"], DSUB_SWEEP)
        l["Z2"] = torch.empty((N, l["M2"]), dtype=torch.float32, device=dev)
        vl.velora_compress(l["X"], l["v2"], Z=l["Z2"])
    variants = ((DSUB, "v", "Z", "M"), (DSUB_SWEEP, "v2", "Z2", "M2"))

    # streaming kernels: the four 4096-wide inputs rotate (4 x 67 MB), the 11008-wide one is 180 MB alone
    small = [by[n] for n in ("q", "k", "v", "o")]
    big = by["down"]
    for dsub, kv, kz, km in variants:
        for group, label in ((small, "N=%d D=4096" % N), ([big], "N=%d D=11008" % N)):
            D, M = group[0]["D"], group[0][km]
            fns = [(lambda l=l: vl.velora_compress(l["X"], l[kv], Z=l[kz])) for l in group]
            hbm("compress", label, timed(fns), N * D * 2 + N * M * 4, timed_b2b(fns), dsub, timed_graph(fns))
            fns = [(lambda l=l: vl.velora_reconstruct(l[kz], l[kv], D, Xhat=l["dX"])) for l in group]
            hbm("reconstruct", label, timed(fns), N * D * 2 + N * M * 4, timed_b2b(fns), dsub, timed_graph(fns))
            if dsub == DSUB:
                ms = timed([(lambda l=l: vl.velora_init_v(l["X"], DSUB, v=l["v"], ws=ws)) for l in group])
                hbm("init_v (incl. the stream sync that reads the degenerate flag)", label, ms, N * D * 2)
                svec = torch.empty(DSUB, dtype=torch.float32, device=dev)
                fns = [(lambda l=l: vl.velora_subtoken_sum(l["X"], DSUB, s=svec, ws=ws)) for l in group]
                hbm("subtoken_sum (init_v's two kernels, no sync)", label, timed(fns), N * D * 2, timed_b2b(fns), DSUB, timed_graph(fns))
    # context only: torch's own fill and reduction on the same 180 MB buffer (pure write / pure read ceilings)
    big_x = big["dX"]
    hbm("reference: torch zero_ (pure write, library kernel)", "N=%d D=11008" % N, timed([lambda: big_x.zero_()]),
        N * big["D"] * 2)
    big_i = big["X"].view(torch.int16)
    hbm("reference: torch max (pure read, library kernel)", "N=%d D=11008" % N, timed([lambda: big_i.max()]),
        N * big["D"] * 2)
    # weight gradient, factored: rotate over layers of equal shape
    for dsub, kv, kz, km in variants:
        for names in (("q", "k", "v", "o"), ("up", "gate"), ("down",)):
            group = [by[n] for n in names]
            l0 = group[0]
            fns = [(lambda l=l: vl.velora_weight_grad(l["dY"], l[kz], l[kv], l["D"], dW=l["dW"], ws=ws)) for l in group]
            ms = timed(fns)
            fl = layer_flops(N, l0["D"], l0["O"], l0[km])["dw"]
            nb = N * l0["O"] * 2 + N * l0[km] * 4 + l0["O"] * l0["D"] * 2
            tensor("weight_grad factored", "%dx%d -> dW[%d,%d]" % (N, l0["O"], l0["O"], l0["D"]), ms, fl, nb, dsub)
            ms2, ms3 = timed_b2b(fns), timed_graph(fns)
            out[-1].update({"us_back_to_back": ms2 * 1e3, "GB/s_back_to_back": nb / (ms2 * 1e-3) / 1e9,
                            "frac_measured_back_to_back": nb / (ms2 * 1e-3) / 1e9 / pk["hbm_gbs"],
                            "us_graph": ms3 * 1e3, "GB/s_graph": nb / (ms3 * 1e-3) / 1e9,
                            "frac_measured_graph": nb / (ms3 * 1e-3) / 1e9 / pk["hbm_gbs"]})
    # the same with Z stored in bf16 (read in place by the tensor map: no conversion launch)
    for l in L:
        l["Zb"] = l["Z"].to(torch.bfloat16)
    for names in (("q", "k", "v", "o"), ("up", "gate"), ("down",)):
        group = [by[n] for n in names]
        l0 = group[0]
        fns = [(lambda l=l: vl.velora_weight_grad(l["dY"], l["Zb"], l["v"], l["D"], dW=l["dW"], ws=ws)) for l in group]
        fl = layer_flops(N, l0["D"], l0["O"], l0["M"])["dw"]
        nb = N * l0["O"] * 2 + N * l0["M"] * 2 + l0["O"] * l0["D"] * 2
        tensor("weight_grad factored, Z stored in bf16", "%dx%d -> dW[%d,%d]" % (N, l0["O"], l0["O"], l0["D"]), timed(fns), fl, nb)
        ms2, ms3 = timed_b2b(fns), timed_graph(fns)
        out[-1].update({"us_back_to_back": ms2 * 1e3, "frac_measured_back_to_back": nb / (ms2 * 1e-3) / 1e9 / pk["hbm_gbs"],
                        "us_graph": ms3 * 1e3, "frac_measured_graph": nb / (ms3 * 1e-3) / 1e9 / pk["hbm_gbs"]})
    # dense contractions
    for names in (("q", "k", "v", "o"), ("up", "gate"), ("down",)):
        group = [by[n] for n in names]
        l0 = group[0]
        fl = 2.0 * N * l0["D"] * l0["O"]
        for dsub, kv, kz, km in variants:
            ms = timed([(lambda l=l: vl.velora_linear_forward(l["X"], l["W"], l[kv], Y=l["Y"], Z=l[kz], ws=ws)) for l in group])
            tensor("linear_forward (GEMM + compress)", "%dx%dx%d" % (N, l0["D"], l0["O"]), ms, fl, dsub=dsub)
        ms = timed([(lambda l=l: vl.velora_dense_product(vl.PRODUCT_A_BT, l["X"], l["W"], C=l["Y"], ws=ws)) for l in group])
        tensor("plain forward product Y = X W^T (no compress)", "%dx%dx%d" % (N, l0["D"], l0["O"]), ms, fl, dsub=None)
        ms = timed([(lambda l=l: vl.velora_linear_backward(l["dY"], l["W"], l["Z"], l["v"], dX=l["dX"], need_dW=False, ws=ws))
                    for l in group])
        tensor("input_grad GEMM dX = dY W", "%dx%dx%d" % (N, l0["O"], l0["D"]), ms, fl, dsub=None)
        ms = timed([(lambda l=l: vl.velora_dense_product(vl.PRODUCT_AT_B, l["dY"], l["X"], C=l["dW"], ws=ws)) for l in group])
        tensor("plain weight gradient dW = dY^T X (dense)", "%dx%dx%d" % (l0["O"], N, l0["D"]), ms, fl, dsub=None)
    l0 = by["q"]
    ws_ex = vl.velora_workspace_alloc(vl.velora_workspace_bytes(vl.OP_WEIGHT_GRAD_EXPLICIT, N, l0["D"], l0["O"], DSUB), dev)
    ms = timed([(lambda l=l: vl.velora_weight_grad(l["dY"], l["Z"], l["v"], l["D"], dW=l["dW"], mode=vl.WG_EXPLICIT, ws=ws_ex))
                for l in [by[n] for n in ("q", "k", "v", "o")]])
    tensor("weight_grad explicit (reconstruct + GEMM dY^T Xhat)", "%dx%dx%d" % (l0["O"], N, l0["D"]), ms,
           2.0 * N * l0["D"] * l0["O"])
    # adapter-shaped layer on the same inputs (rank-16 down-projection of an adapter on the 4096-wide stream):
    # everything is bound by the one pass over X (forward) or over dX (input gradient)
    R = 16
    group = [by[n] for n in ("q", "k", "v", "o")]
    D, M = group[0]["D"], group[0]["M"]
    Wa = group[0]["W"][:R]                               # the first R rows of a projection serve as the adapter's A
    Ya = torch.empty((N, R), dtype=torch.bfloat16, device=dev)
    dYa = [l["dY"][:, :R].contiguous() for l in group]
    dWa = torch.empty((R, D), dtype=torch.bfloat16, device=dev)
    ws_a = vl.velora_workspace_alloc(vl.velora_workspace_bytes(vl.OP_LINEAR_BACKWARD_FACTORED, N, D, R, DSUB), dev)
    fns = [(lambda l=l: vl.velora_linear_forward(l["X"], Wa, l["v"], Y=Ya, Z=l["Z"], ws=ws_a)) for l in group]
    hbm("adapter forward, rank 16 (Y and Z in one pass over X)", "N=%d D=%d" % (N, D), timed(fns),
        N * D * 2 + R * D * 2 + N * R * 2 + N * M * 4, timed_b2b(fns))
    fns = [(lambda l=l, y=y: vl.velora_weight_grad(y, l["Z"], l["v"], D, dW=dWa, ws=ws_a)) for l, y in zip(group, dYa)]
    hbm("adapter weight_grad factored, rank 16", "N=%d D=%d" % (N, D), timed(fns),
        N * R * 2 + N * M * 4 + R * D * 2, timed_b2b(fns))
    fns = [(lambda l=l, y=y: vl.velora_linear_backward(y, Wa, l["Z"], l["v"], dX=l["dX"], need_dW=False, ws=ws_a))
           for l, y in zip(group, dYa)]
    hbm("adapter input_grad, rank 16 (dX = dY A)", "N=%d D=%d" % (N, D), timed(fns), N * D * 2 + N * R * 2 + R * D * 2,
        timed_b2b(fns))
    return out


def run_profile(args):
    """A few launches of one entry point on one config-5 layer: the small, self-ending case for ncu."""
    import torch

    import paper_2405_17991_b200 as vl
    import velora_inputs as vi

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    cfg = vi.CONFIGS[CONFIG_INDEX]
    name = {"compress": "down", "reconstruct": "down", "init_v": "down", "weight_grad": "up",
            "weight_grad_q": "q", "weight_grad_down": "down",
            "forward": "q", "input_grad": "q", "weight_grad_explicit": "q", "adapter_forward": "q",
            "adapter_weight_grad": "q", "adapter_input_grad": "q"}[args.profile]
    li = [l.name for l in cfg.layers].index(name)
    layer = cfg.layers[li]
    N = cfg.N
    X = vi.make_X(cfg, li).torch(dev)
    v = vl.velora_init_v(X, DSUB)
    Z = vl.velora_compress(X, v)
    ws = vl.velora_workspace_alloc(
        max(vl.velora_workspace_bytes(op, N, layer.D, layer.O, DSUB)
            for op in (vl.OP_INIT_V, vl.OP_LINEAR_BACKWARD_FACTORED, vl.OP_WEIGHT_GRAD_EXPLICIT)), dev)
    if args.profile in ("compress", "reconstruct", "init_v"):
        Xhat = torch.empty_like(X)
        fn = {"compress": lambda: vl.velora_compress(X, v, Z=Z),
              "reconstruct": lambda: vl.velora_reconstruct(Z, v, layer.D, Xhat=Xhat),
              "init_v": lambda: vl.velora_init_v(X, DSUB, v=v, ws=ws)}[args.profile]
    elif args.profile in ("adapter_forward", "adapter_weight_grad", "adapter_input_grad"):   # rank-16 adapter on the q input
        Wa = vi.make_W(cfg, li).torch(dev)[:16]
        dYa = vi.make_dY(cfg, li).torch(dev)[:, :16].contiguous()
        Ya = torch.empty((N, 16), dtype=torch.bfloat16, device=dev)
        dWa = torch.empty((16, layer.D), dtype=torch.bfloat16, device=dev)
        dXa = torch.empty_like(X)
        fn = {"adapter_forward": lambda: vl.velora_linear_forward(X, Wa, v, Y=Ya, Z=Z, ws=ws),
              "adapter_input_grad": lambda: vl.velora_linear_backward(dYa, Wa, Z, v, dX=dXa, need_dW=False, ws=ws),
              "adapter_weight_grad": lambda: vl.velora_weight_grad(dYa, Z, v, layer.D, dW=dWa, ws=ws)}[args.profile]
    else:
        W = vi.make_W(cfg, li).torch(dev)
        dY = vi.make_dY(cfg, li).torch(dev)
        Y = torch.empty((N, layer.O), dtype=torch.bfloat16, device=dev)
        dX = torch.empty_like(X)
        dW = torch.empty_like(W)
        wg = lambda: vl.velora_weight_grad(dY, Z, v, layer.D, dW=dW, ws=ws)
        fn = {"weight_grad": wg, "weight_grad_q": wg, "weight_grad_down": wg,
              "weight_grad_explicit": lambda: vl.velora_weight_grad(dY, Z, v, layer.D, dW=dW, mode=vl.WG_EXPLICIT, ws=ws),
              "forward": lambda: vl.velora_linear_forward(X, W, v, Y=Y, Z=Z, ws=ws),
              "input_grad": lambda: vl.velora_linear_backward(dY, W, Z, v, dX=dX, need_dW=False, ws=ws)}[args.profile]
    for _ in range(4):
        fn()
    torch.cuda.synchronize()
    print(json.dumps({"profile": args.profile, "layer": name, "N": N, "D": layer.D, "O": layer.O,
                      "status": vl.velora_workspace_status(ws)}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--profile", default=None,
                    choices=["compress", "reconstruct", "init_v", "weight_grad", "weight_grad_q", "weight_grad_down", "weight_grad_explicit",
                             "forward", "input_grad", "adapter_forward", "adapter_weight_grad", "adapter_input_grad"],
                    help="run four launches of one entry point on one layer (for ncu) and exit")
    ap.add_argument("--config", type=int, default=CONFIG_DEFAULT, choices=[2, 3, 4, 5],
                    help="time the step of another configuration (its first sub-token length); the headline line, "
                         "the kernel table and the end-to-end leg are configuration 5's")
    ap.add_argument("--graph", action="store_true",
                    help="also time the step replayed from a CUDA graph (an extra key; the headline stays the plain step)")
    args = ap.parse_args()
    global CONFIG_INDEX, DSUB
    if args.config != CONFIG_DEFAULT:
        import velora_inputs as vi
        CONFIG_INDEX, DSUB = args.config, vi.CONFIGS[args.config].Dsubs[0]
    if args.profile:
        run_profile(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
