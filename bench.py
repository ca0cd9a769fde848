"""Benchmark of the routed FP4 mixture-of-experts layer on B200.

A step is one pass of the whole hot path (moe_route -> moe_permute -> moe_expert_ffn -> moe_combine)
over one batch of seeded synthetic input.  For a handful of tokens (decode_c1) the library runs that path
as ONE kernel launch behind moe_forward; the step is then that call, and the four calls are timed beside
it.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

N > 1 (launched by torch.distributed.run, one rank per GPU) runs independent replicas: the layer
does not shard in this build, so there is no data-path collective; the barrier and the max over
ranks are the only communication.  --impl reference times the CPU oracle (rank 0 only).
"""
import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "MoE FP4 layer tokens/s"
DECODE = ("decode_c1", "decode_c64")

# dram__bytes_read.sum + dram__bytes_write.sum per moe_expert_ffn call from one ncu capture of the
# workload (see profiles/); None until captured.
NCU_TRAFFIC_BYTES = {
    "decode_c1_one_launch": 110440700,  # ffn_native_kernel<true>, the whole layer: 107.14 MB read + 3.30 MB written (mean of two launches)
    "decode_c1": 111216000,      # ffn_native_kernel<false>: 107.19 MB read + 4.03 MB written (profiles/ffn_native_decode.md)
    "decode_c64": 3064384880,    # 3057.9 MB read + 6.5 MB written
    "prefill_8k": 5611119000,    # ffn_umma_kernel<true> 2.882 + 0.263 GB, <false> 1.431 + 1.034 GB (profiles/ffn_umma_prefill_8k.md)
}


def expert_weight_bytes(H, I):
    return 3 * H * I // 2 + 3 * H * I // 32


def ffn_algorithmic_bytes(wl, n_touched):
    """Bytes moe_expert_ffn must move: each touched expert's packed codes and scale bytes once, the
    sorted activations in, the bf16 intermediate out and back in, the fp32 per-slot rows out."""
    S = wl.T * wl.k
    return n_touched * expert_weight_bytes(wl.H, wl.I) + S * wl.H * 2 + 2 * S * wl.I * 2 + S * wl.H * 4


def layer_algorithmic_bytes(wl, n_touched):
    """Bytes the whole layer must move when nothing between its steps is materialised: each touched
    expert's packed codes and scale bytes once, logits and token rows in, the output rows out."""
    return n_touched * expert_weight_bytes(wl.H, wl.I) + wl.T * wl.E * 4 + 2 * wl.T * wl.H * 2


def ffn_flops(wl):
    return wl.T * wl.k * 6 * wl.I * wl.H


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm=float(p["hbm_gbs"]), tensor_burst=float(p["bf16_tflops"]),
                    tensor_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), source="measured")
    return dict(hbm=6650.0, tensor_burst=1590.0, tensor_sustained=1400.0, source="fallback")


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index, period=0.02):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def sample(self):
        if not self.ok:
            return
        nv = self.nv
        try:
            self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
            r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)) if hasattr(
                nv, "nvmlDeviceGetCurrentClocksEventReasons") else int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            names = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}
            for bit, name in names.items():
                if r & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def run(self):
        while not self._stop_evt.is_set():
            self.sample()
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        self.sample()
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def physical_gpu_index(local_index):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


def max_over_ranks(value, world):
    """Max of a float over all ranks (identity when not distributed)."""
    if world == 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device="cuda" if dist.get_backend() == "nccl" else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def oracle_sample(wl, inputs, n_tokens, seed0=1000, weights=None):
    """Time the CPU oracle, as it stands, on n_tokens tokens of the workload (per-token definition).
    `weights`: the full host arrays if the caller has them; else the touched experts are generated here."""
    from oracle import moe_oracle as O
    logits = inputs.make_logits(max(wl.T, 1), wl.E, seed0, wl.skew)
    x = inputs.make_x(max(wl.T, 1), wl.H, seed0)
    if n_tokens > wl.T:
        logits = np.concatenate([inputs.make_logits(wl.T, wl.E, seed0 + i, wl.skew) for i in range(n_tokens)])[:n_tokens]
        x = np.concatenate([inputs.make_x(wl.T, wl.H, seed0 + i) for i in range(n_tokens)])[:n_tokens]
    tokens = np.arange(min(n_tokens, logits.shape[0]), dtype=np.int32)
    ids, _, _ = O.route(logits, wl.k)
    if weights is not None:
        w13, s13, w2, s2 = weights
    else:
        need = sorted(set(ids[tokens].ravel().tolist()))
        w13, s13, w2, s2 = inputs.make_expert_weights(wl.H, wl.I, wl.E, seed=0, experts=need)
    t0 = time.perf_counter()
    O.forward_tokens(logits, x, w13, s13, w2, s2, wl.k, tokens)
    dt = time.perf_counter() - t0
    return len(tokens) / dt, dt, len(tokens), O.num_threads()


def run_reference(args, wl, inputs):
    """The CPU oracle as the reference arm: each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_tok = {"tiny": 16, "decode_c1": 1, "decode_c64": 8}.get(wl.name, 4)
    for _ in range(args.warmup):
        oracle_sample(wl, inputs, n_tok)
    rates, total_t = [], 0.0
    cores = 1
    for i in range(args.steps):
        r, dt, n, cores = oracle_sample(wl, inputs, n_tok, seed0=2000 + i)
        rates.append(r)
        total_t += dt
    value = n_tok * args.steps / total_t
    sample = "%d token(s) of %s per step, per-token definition, weights of the touched experts only" % (n_tok, wl.name)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "T": wl.T, "H": wl.H, "I": wl.I, "E": wl.E, "k": wl.k},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="decode_c1")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="decode workloads: launch the calls eagerly instead of replaying CUDA graphs")
    ap.add_argument("--four-calls", action="store_true", help="time the four calls even where moe_forward is one launch")
    ap.add_argument("--raw-weights", action="store_true", help="read the weights in the checkpoint's row layout instead of moe_prepack's tiles")
    args = ap.parse_args()

    from paper_2609_15627_b200 import inputs
    wl = inputs.WORKLOADS[args.workload]
    decode = wl.name in DECODE or wl.name == "tiny"
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 5
        args.warmup = args.warmup if args.warmup is not None else 1
        run_reference(args, wl, inputs)
        return
    if args.steps is None:
        args.steps = 2000 if decode else 10
    if args.warmup is None:
        args.warmup = 20 if decode else 3
    args.warmup = max(args.warmup, 3)

    import torch
    from paper_2609_15627_b200 import build_ext, moe

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build_ext.build()
    if world > 1:
        torch.distributed.barrier()
    moe.lib()

    # ---- resident inputs: weights once, a cycle of seeded (logits, x) batches -------------------------
    def dev(a):
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(a).cuda()

    weights_host = inputs.make_expert_weights(wl.H, wl.I, wl.E, seed=0)
    weights = tuple(dev(a) for a in weights_host)
    # One-time load transform (untimed, as in the paper's load path): the same bytes in tiles that are contiguous in
    # memory.  The row-layout tensors are dropped afterwards: one copy of the weights is resident.
    packed = None
    if not args.raw_weights:
        packed = moe.moe_prepack(*weights, moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k))
        torch.cuda.synchronize()
        weights = None
    n_cycle = 32 if decode else 2
    batches_host = [(inputs.make_logits(wl.T, wl.E, 7000 + rank * 100 + i, wl.skew), inputs.make_x(wl.T, wl.H, 7000 + rank * 100 + i))
                    for i in range(n_cycle)]
    batches = [(dev(l), dev(x)) for l, x in batches_host]
    sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
    buf = moe.LayerBuffers(sh)
    stream = torch.cuda.current_stream()

    # experts touched per batch of the cycle (from the library's own routing), for the byte count
    touched = []
    for l, x in batches:
        moe.moe_route(l, wl.k, buf.topk_ids, buf.topk_w, buf.expert_offsets, buf.ws)
        off = buf.expert_offsets.cpu().numpy()
        touched.append(int(np.count_nonzero(np.diff(off))))

    # Does moe_forward run this shape as one launch?  (Asked of the library: one call, then the name of its kernel.)
    fws = moe.alloc_forward_workspace(sh)
    def forward(l, x, st):
        if packed is not None:
            moe.moe_forward_packed(l, x, packed, sh, buf.out, None, None, buf.status, fws, st)
        else:
            moe.moe_forward(l, x, *weights, sh, buf.out, None, None, buf.status, fws, st)

    def expert_ffn(b, st):
        if packed is not None:
            moe.moe_expert_ffn_packed(b.x_perm, b.expert_offsets, packed, sh, b.y_perm, b.status, b.ws, st)
        else:
            moe.moe_expert_ffn(b.x_perm, b.expert_offsets, *weights, sh, b.y_perm, b.status, b.ws, st)

    forward(batches[0][0], batches[0][1], stream)
    torch.cuda.synchronize()
    one_launch = moe.moe_last_kernel_name().startswith("layer_one_launch") and not args.four_calls

    def step4(i, ev=None, st=stream):
        """The four C-ABI calls on batch i of the cycle (st=None: torch's current stream, used during capture)."""
        l, x = batches[i % n_cycle]
        moe.moe_route(l, wl.k, buf.topk_ids, buf.topk_w, buf.expert_offsets, buf.ws, st)
        moe.moe_permute(x, buf.topk_ids, buf.expert_offsets, sh, buf.x_perm, buf.perm, buf.inv_perm, buf.ws, st)
        if ev is not None:
            ev[0].record(st)
        expert_ffn(buf, st)
        if ev is not None:
            ev[1].record(st)
        moe.moe_combine(buf.y_perm, buf.inv_perm, buf.topk_w, sh, buf.out, st)

    def step1(i, ev=None, st=stream):
        """The same path as one call (one kernel launch for this shape)."""
        l, x = batches[i % n_cycle]
        forward(l, x, st)

    step = step1 if one_launch else step4

    def barrier():
        if world > 1:
            torch.distributed.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    barrier()

    # Decode-sized steps are a handful of short kernels: like the paper's decode tiers they are replayed as CUDA
    # graphs (the four C-ABI calls captured as they are).  A serving graph holds many layers back to back; here a
    # graph holds kGraphSteps consecutive batches of the cycle (one layer call each), plus one single-step graph per
    # batch for a step count that is not a multiple of kGraphSteps.
    use_graph = decode and not args.no_graph
    kGraphSteps = 8
    graphs, multi_graphs, launches_per_step = [], [], None
    if use_graph:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            for i in range(3):
                step(i, st=None)
        stream.wait_stream(side)
        barrier()
        for i in range(n_cycle):
            g = torch.cuda.CUDAGraph()
            c0 = moe.moe_launch_count()
            with torch.cuda.graph(g):
                step(i, st=None)
            launches_per_step = moe.moe_launch_count() - c0
            graphs.append(g)
        for i0 in range(0, n_cycle, kGraphSteps):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(i0, i0 + kGraphSteps):
                    step(i, st=None)
            multi_graphs.append(g)
        for i in range(max(args.warmup, 3)):
            graphs[i % n_cycle].replay()
        for g in multi_graphs:
            g.replay()
        barrier()

    # ---- timed region: exactly K steps ---------------------------------------------------------------------
    n_inner = min(args.steps, 256)  # steps whose expert-FFN call is bracketed by its own events
    inner = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_inner)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(physical_gpu_index(local))
    launches0 = moe.moe_launch_count()
    barrier()
    sampler.start()
    e0.record(stream)
    if use_graph:
        n_multi = args.steps // kGraphSteps
        for i in range(n_multi):
            multi_graphs[i % len(multi_graphs)].replay()
        for i in range(n_multi * kGraphSteps, args.steps):
            graphs[i % n_cycle].replay()
    else:
        for i in range(args.steps):
            step(i, inner[i] if i < n_inner and not one_launch else None)
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = launches_per_step * args.steps if use_graph else moe.moe_launch_count() - launches0
    assert int(buf.status.item()) == 0, "device-side wait timed out"
    ms_total = max_over_ranks(e0.elapsed_time(e1), world)
    ms_step = ms_total / args.steps
    value = wl.T * world / (ms_step * 1e-3)
    eager_ms_step = None
    if use_graph or one_launch:
        # the expert-FFN call cannot be bracketed by events inside a graph (nor inside the one-launch layer): time it
        # in a second region of eager steps of the four calls on the same batches, right after the timed one
        for i in range(3):
            step4(i)
        barrier()
        ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ee0.record(stream)
        for i in range(n_inner):
            step4(i, inner[i])
        ee1.record(stream)
        barrier()
        eager_ms_step = ee0.elapsed_time(ee1) / n_inner

    # ---- one-launch workloads: the four calls, graph-replayed the same way, for comparison -----------------------
    four_calls_ms_step = None
    if one_launch and use_graph:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            for i in range(3):
                step4(i, st=None)
        stream.wait_stream(side)
        barrier()
        mg4 = []
        for i0 in range(0, n_cycle, kGraphSteps):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(i0, i0 + kGraphSteps):
                    step4(i, st=None)
            mg4.append(g)
        for g in mg4:
            g.replay()
        barrier()
        n4 = max(len(mg4), min(args.steps // kGraphSteps, 64))
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        g0.record(stream)
        for i in range(n4):
            mg4[i % len(mg4)].replay()
        g1.record(stream)
        barrier()
        four_calls_ms_step = g0.elapsed_time(g1) / (n4 * kGraphSteps)

    # ---- the expert-FFN call alone, graph-replayed like the step (calls shorter than 100 us) -------------------------
    # Eager launches of kernels this short leave the GPU idle between the event and the launch, which the bracketing
    # events count.  So such a call is also captured alone, one graph per batch of the cycle on that batch's own routed
    # and permuted inputs, and the replays are timed back to back: consecutive calls touch different experts, as in
    # the step.  Longer calls keep the time between their events inside the eager steps.
    ffn_graph_ms, n_ffn = None, 0
    if use_graph and float(np.mean([a.elapsed_time(b) for a, b in inner])) < 0.1:
        fbufs = []
        for i in range(n_cycle):
            b = moe.LayerBuffers(sh)
            l, x = batches[i]
            moe.moe_route(l, wl.k, b.topk_ids, b.topk_w, b.expert_offsets, b.ws, stream)
            moe.moe_permute(x, b.topk_ids, b.expert_offsets, sh, b.x_perm, b.perm, b.inv_perm, b.ws, stream)
            fbufs.append(b)
        barrier()

        def ffn_only(b, st=stream):
            expert_ffn(b, st)

        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            ffn_only(fbufs[0], None)
        stream.wait_stream(side)
        barrier()
        fgraphs = []
        for b in fbufs:
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                ffn_only(b, None)
            fgraphs.append(g)
        for i in range(max(args.warmup, 3)):
            fgraphs[i % n_cycle].replay()
        barrier()
        n_ffn = max(n_cycle, min(args.steps, 512))
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(stream)
        for i in range(n_ffn):
            fgraphs[i % n_cycle].replay()
        f1.record(stream)
        barrier()
        ffn_graph_ms = f0.elapsed_time(f1) / n_ffn
        assert all(int(b.status.item()) == 0 for b in fbufs), "device-side wait timed out"

    # ---- roofline of the dominant call (the expert FFN) --------------------------------------------------------
    ffn_eager_ms = float(np.mean([a.elapsed_time(b) for a, b in inner]))
    ffn_ms = ffn_graph_ms if ffn_graph_ms is not None else ffn_eager_ms
    n_avg = n_ffn if ffn_graph_ms is not None else n_inner
    mean_touched = float(np.mean([touched[i % n_cycle] for i in range(n_avg)]))
    peaks = load_peaks()
    if decode:
        alg = ffn_algorithmic_bytes(wl, mean_touched)
        achieved = alg / (ffn_ms * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm"], "unit": "GB/s", "frac": achieved / peaks["hbm"],
                "traffic": NCU_TRAFFIC_BYTES.get(wl.name), "algorithmic_bytes": alg}
    else:
        fl = ffn_flops(wl)
        achieved = fl / (ffn_ms * 1e-3) / 1e12
        roof = {"bound": "tensor", "achieved": achieved, "peak": peaks["tensor_sustained"], "unit": "TFLOP/s",
                "frac": achieved / peaks["tensor_sustained"], "traffic": NCU_TRAFFIC_BYTES.get(wl.name),
                "algorithmic_flops": fl}
    roof.update({"kernel": "moe_expert_ffn",
                 "ms": ffn_ms, "peak_source": peaks["source"], "experts_touched": mean_touched,
                 "timed_in": ("graph replays of the call alone, one graph per batch of the cycle, right after the timed region"
                              if ffn_graph_ms is not None else
                              ("eager steps right after the graph-replayed region" if use_graph or one_launch else "the timed region")),
                 "ms_between_events_in_eager_steps": ffn_eager_ms})
    if one_launch:
        # the dominant kernel is the step itself: one launch per step, timed by the events of the timed region
        touched_steps = float(np.mean([touched[i % n_cycle] for i in range(args.steps)]))
        alg = layer_algorithmic_bytes(wl, touched_steps)
        achieved = alg / (ms_step * 1e-3) / 1e9
        roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm"], "unit": "GB/s", "frac": achieved / peaks["hbm"],
                "traffic": NCU_TRAFFIC_BYTES.get(wl.name + "_one_launch"), "algorithmic_bytes": alg,
                "kernel": "moe_forward (route, term split, expert FFN and combine in one launch)", "ms": ms_step,
                "peak_source": peaks["source"], "experts_touched": touched_steps, "timed_in": "the timed region",
                "four_calls": {"ms_per_step": four_calls_ms_step, "eager_ms_per_step": eager_ms_step, "expert_ffn": roof}}

    # ---- read-only ceiling: the decode kernel's load mechanism alone over the resident gate/up weights ------------
    # (2.1 GB at the production shape, larger than L2; context for the HBM-bound workloads, not the denominator)
    probe_src = packed if packed is not None else weights[0]
    if decode and probe_src.numel() >= (1 << 28):
        sink = torch.empty(4096, dtype=torch.int32, device="cuda")
        for _ in range(2):
            moe.moe_debug_read_probe(probe_src, sink, buf.status, stream)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record(stream)
        for _ in range(5):
            moe.moe_debug_read_probe(probe_src, sink, buf.status, stream)
        p1.record(stream)
        barrier()
        read_gbs = 5 * probe_src.numel() / (p0.elapsed_time(p1) * 1e-3) / 1e9
        roof["read_only_stream_gbs"] = read_gbs
        roof["frac_of_read_only_stream"] = roof["achieved"] / read_gbs

    # ---- end to end through the host-buffer entry point ---------------------------------------------------------
    e2e = None
    if not args.no_e2e:
        ws_h = moe.alloc_workspace(sh, host_path=True)
        lh = [torch.from_numpy(l).pin_memory() for l, _ in batches_host]
        xh = [torch.from_numpy(x.view(np.int16)).pin_memory() for _, x in batches_host]
        oh = torch.empty((wl.T, wl.H), dtype=torch.int16).pin_memory()
        n_e2e = max(3, min(args.steps, 200 if decode else 5))
        def forward_host(i):
            if packed is not None:
                moe.moe_forward_host_packed(lh[i % n_cycle], xh[i % n_cycle], packed, sh, oh, buf.status, ws_h, stream)
            else:
                moe.moe_forward_host(lh[i % n_cycle], xh[i % n_cycle], *weights, sh, oh, buf.status, ws_h, stream)

        for i in range(3):
            forward_host(i)
        barrier()
        t0 = time.perf_counter()
        for i in range(n_e2e):
            forward_host(i)
        dt = max_over_ranks(time.perf_counter() - t0, world)
        e2e = {"value": wl.T * world * n_e2e / dt, "unit": "tokens/s",
               "h2d_bytes_per_step": wl.T * wl.E * 4 + wl.T * wl.H * 2, "d2h_bytes_per_step": wl.T * wl.H * 2,
               "steps": n_e2e, "call": "%s (pinned host logits/x in, bf16 out back, weights resident)"
                       % ("moe_forward_host_packed" if packed is not None else "moe_forward_host")}

    # ---- the oracle on the host cores (rank 0, N = 1 only) ----------------------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # about 10-20 s of host work at the production shape (the oracle does roughly 50 tokens/s on 16 cores)
        n_tok = {"tiny": 4096}.get(wl.name, 640)
        v, dt, n, cores = oracle_sample(wl, inputs, n_tok, weights=weights_host)
        cpu = {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle",
               "sample": "%d tokens with the %s shape and routing distribution, per-token definition, %.1f s" % (n, wl.name, dt)}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "T": wl.T, "H": wl.H, "I": wl.I, "E": wl.E, "k": wl.k,
                       "parallelism": "replicas only" if world > 1 else "1 GPU",
                       "call": ("moe_forward%s (one kernel launch per step)" if one_launch else
                                "moe_route, moe_permute, moe_expert_ffn%s, moe_combine") % ("_packed" if packed is not None else ""),
                       "weights": ("moe_prepack's tile-contiguous layout (one-time transform, same bytes)" if packed is not None
                                   else "checkpoint row layout"),
                       "launch": "cuda graph replay, %d consecutive batches of the cycle per graph" % kGraphSteps if use_graph else "eager",
                       "eager_ms_per_step": None if one_launch else eager_ms_step,
                       "l2": "inputs cycle over %d seeded batches; %.2f GB of expert weights resident (larger than L2)"
                             % (n_cycle, wl.E * expert_weight_bytes(wl.H, wl.I) / 1e9)},
            "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches, "clocks": clocks,
            "kernels": moe.moe_last_kernel_name(),
        }))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
