"""Benchmark of the routed FP4 mixture-of-experts layer on B200.

A step is one pass of the whole hot path (moe_route -> moe_permute -> moe_expert_ffn -> moe_combine)
over one batch of seeded synthetic input.  For a single token (decode_c1) the library runs that path
as ONE kernel launch behind moe_forward; the step is then that call, and the four calls are timed beside
it.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

With no --workload the line's headline keys describe decode_c1 (exactly K timed steps) and a top-level
`workloads` object carries all four production workloads - decode_c1, decode_c64, prefill_8k,
prefill_32k_skewed - timed in the same process on the same resident weights, each over regions of at least
100 ms (three rounds, median reported, every round kept), each with its own roofline, end-to-end figure and
clock record.  --workload NAME times that one workload only.

N > 1 (launched by torch.distributed.run, one rank per GPU) runs independent replicas: the layer
does not shard in this build, so there is no data-path collective; the barrier and the max over
ranks are the only communication.  --impl reference times the CPU oracle (rank 0 only).
"""
import argparse
import json
import math
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
PRODUCTION = ("decode_c1", "decode_c64", "prefill_8k", "prefill_32k_skewed")
HEADLINE = "decode_c1"
QUANT_WORKLOADS = ("decode_c64", "prefill_8k", "prefill_32k_skewed")  # also timed with moe_expert_ffn_q
MIN_REGION_MS = 100.0   # a timed round of a decode workload lasts at least this long
MIN_REGION_MS_PREFILL = 40.0  # prefill rounds: at least this long and at least 3 steps - a burst-length region, to go with
                              # the burst bf16 peak they are divided by (a single sub-millisecond GEMM, best of ten)
COOLDOWN_S = 1.0        # idle time before every round: each round starts with the board below its power limit
ROUNDS = 3
GRAPH_STEPS = 32  # decode steps per CUDA graph: the whole cycle of seeded batches (a serving graph holds dozens of layer calls)

# dram__bytes_read.sum + dram__bytes_write.sum per launch (or per two-launch call) from one ncu capture of the
# workload; which capture, at which commit, is stated in the file under profiles/ named beside each figure.
NCU_TRAFFIC_BYTES = {
    "decode_c1_one_launch": 111113000,  # decode_one_kernel, the whole layer (profiles/decode_one_kernel_decode_c1.md)
    "decode_c1": 111216000,             # ffn_native_kernel<false> (profiles/ffn_native_decode.md)
    "decode_c64": 3064384880,           # ffn_native_kernel<false> (profiles/ffn_native_decode.md)
    "prefill_8k": 5611119000,           # ffn_umma_kernel<true> + <false> (profiles/ffn_umma_prefill_8k.md)
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


def tensor_roofline(flops, ms, region_ms, peaks):
    """Fraction of the dense bf16 peak: the burst figure for a region shorter than a second (the board has not
    reached its power limit yet), the sustained one otherwise; both fractions are printed."""
    achieved = flops / (ms * 1e-3) / 1e12
    sustained = region_ms >= 1000.0
    peak = peaks["tensor_sustained"] if sustained else peaks["tensor_burst"]
    return {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
            "peak_used": "bf16_tflops_sustained" if sustained else "bf16_tflops",
            "frac_of_burst": achieved / peaks["tensor_burst"], "frac_of_sustained": achieved / peaks["tensor_sustained"],
            "algorithmic_flops": flops, "ms": ms, "peak_source": peaks["source"]}


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


def steps_for_region(ms_per_step, min_ms=MIN_REGION_MS, multiple=1, at_least=1):
    """Steps that make a timed round last at least min_ms, rounded up to a multiple (whole graphs)."""
    n = max(at_least, int(math.ceil(min_ms / max(ms_per_step, 1e-6))))
    return (n + multiple - 1) // multiple * multiple


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


class Bench:
    """The resident model state (one copy of the expert weights) and the timing of one workload on it."""

    def __init__(self, args, rank, world, local):
        import torch
        from paper_2609_15627_b200 import inputs, moe
        self.torch, self.inputs, self.moe = torch, inputs, moe
        self.args, self.rank, self.world, self.local = args, rank, world, local
        self.stream = torch.cuda.current_stream()
        self.peaks = load_peaks()
        self._weights_key = None
        self.weights_host = self.weights = self.packed = self.raw = None
        self.read_only_gbs = None

    # ---- plumbing ---------------------------------------------------------------------------------------------
    def dev(self, a):
        torch = self.torch
        if a.dtype == np.uint16:
            return torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16)
        return torch.from_numpy(a).cuda()

    def barrier(self):
        if self.world > 1:
            self.torch.distributed.barrier()
        self.torch.cuda.synchronize()

    def events(self):
        return self.torch.cuda.Event(enable_timing=True), self.torch.cuda.Event(enable_timing=True)

    def hold(self):
        """Keep the GPU busy for about 100 us, so that the event and the launches enqueued behind it are already
        queued when it ends: the region then measures device time, not the host's launch latency."""
        self.torch.cuda._sleep(200000)

    def load_weights(self, wl, keep_raw=False):
        """Weights are model state: generated once per (H, I, E), moved to the device, re-laid by moe_prepack (the
        one-time load transform, untimed) unless --raw-weights, after which the row-layout tensors are dropped
        (keep_raw: not yet - the FFN-block timing, which takes the row layout, runs first and drops them)."""
        key = (wl.H, wl.I, wl.E)
        if self._weights_key == key:
            return
        torch, moe = self.torch, self.moe
        self.weights = self.packed = None
        torch.cuda.empty_cache()
        self.weights_host = self.inputs.make_expert_weights(wl.H, wl.I, wl.E, seed=0)
        self.weights = tuple(self.dev(a) for a in self.weights_host)
        if not self.args.raw_weights:
            self.packed = moe.moe_prepack(*self.weights, moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k))
            torch.cuda.synchronize()
            if keep_raw:
                self.raw = self.weights
            self.weights = None
        self._weights_key = key
        self.read_only_gbs = None

    def run_block(self, wl, min_ms=50.0):
        """The FFN block around the routed path (moe_ffn_block: router projection, routed experts, shared expert, join)
        on the same routed weights in the checkpoint's row layout, seeded router and shared-expert weights, a cycle of
        seeded token batches: one round of at least min_ms, CUDA events, graphs of GRAPH_STEPS steps for decode."""
        torch, moe, inputs = self.torch, self.moe, self.inputs
        stream = self.stream
        decode = wl.name in DECODE
        routed = self.raw if self.raw is not None else self.weights
        sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
        n_cycle = 32 if decode else 2
        xs = [self.dev(inputs.make_x(wl.T, wl.H, 7000 + self.rank * 100 + i)) for i in range(n_cycle)]
        w_router = self.dev(inputs.f32_to_bf16_bits(inputs.bf16_bits_to_f32(inputs.make_x(wl.E, wl.H, 31)) * np.float32(0.03)))
        shared = tuple(self.dev(a) for a in inputs.make_expert_weights(wl.H, wl.I, 1, seed=21))
        ws = moe.alloc_block_workspace(sh)
        out = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device="cuda")
        status = torch.zeros(1, dtype=torch.int32, device="cuda")

        def step(i, st=stream):
            moe.moe_ffn_block(xs[i % n_cycle], w_router, routed, shared, sh, out, None, None, status, ws, st)

        c0 = moe.moe_launch_count()
        step(0)
        launches_per_step = moe.moe_launch_count() - c0
        for i in range(3):
            step(i)
        self.barrier()
        graphs = []
        if decode:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                step(0, None)
            stream.wait_stream(side)
            self.barrier()
            for i0 in range(0, n_cycle, GRAPH_STEPS):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    for i in range(i0, i0 + GRAPH_STEPS):
                        step(i, None)
                graphs.append(g)
            for g in graphs:
                g.replay()
            self.barrier()

        def play(n):
            if decode:
                for i in range(n // GRAPH_STEPS):
                    graphs[i % len(graphs)].replay()
            else:
                for i in range(n):
                    step(i)

        def timed(n):
            e0, e1 = self.events()
            self.barrier()
            self.hold()
            e0.record(stream)
            play(n)
            e1.record(stream)
            self.barrier()
            return max_over_ranks(e0.elapsed_time(e1), self.world)

        pilot_n = GRAPH_STEPS if decode else 2
        pilot = timed(pilot_n) / pilot_n
        n = steps_for_region(pilot, min_ms, multiple=GRAPH_STEPS if decode else 1, at_least=3)
        time.sleep(COOLDOWN_S)
        ms = timed(n) / n
        assert int(status.item()) == 0, "device-side wait timed out"
        del graphs, xs, ws, shared
        torch.cuda.empty_cache()
        return {"ms_per_step": ms, "value": wl.T * self.world / (ms * 1e-3), "unit": "tokens/s", "steps": n,
                "gpu_launches_per_step": launches_per_step, "call": "moe_ffn_block (row-layout weights)",
                "launch": ("cuda graph replay, %d steps per graph" % GRAPH_STEPS) if decode else "eager"}

    def run_quant(self, wl, min_ms=50.0):
        """The quantised-activation variant (moe_expert_ffn_q in place of moe_expert_ffn in the four calls) on the weights
        already resident: one round of at least min_ms of whole steps, and the FFN call between its own events in eager
        steps.  Roofline of the call: HBM bytes for decode batches; for prefill batches the FP4 tensor peak (the
        measured bf16 peak times the nominal ratio of 4)."""
        torch, moe, inputs = self.torch, self.moe, self.inputs
        stream = self.stream
        decode = wl.name in DECODE
        weights = self.packed if self.packed is not None else self.weights
        sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
        n_cycle = 32 if decode else 2
        batches = [(self.dev(inputs.make_logits(wl.T, wl.E, 7000 + self.rank * 100 + i, wl.skew)),
                    self.dev(inputs.make_x(wl.T, wl.H, 7000 + self.rank * 100 + i))) for i in range(n_cycle)]
        buf = moe.LayerBuffers(sh)
        qws = moe.alloc_ffn_q_workspace(sh)
        touched = []
        for l, x in batches:
            moe.moe_route(l, wl.k, buf.topk_ids, buf.topk_w, buf.expert_offsets, buf.ws)
            touched.append(int(np.count_nonzero(np.diff(buf.expert_offsets.cpu().numpy()))))

        def step(i, ev=None, st=stream):
            l, x = batches[i % n_cycle]
            moe.moe_route(l, wl.k, buf.topk_ids, buf.topk_w, buf.expert_offsets, buf.ws, st)
            moe.moe_permute(x, buf.topk_ids, buf.expert_offsets, sh, buf.x_perm, buf.perm, buf.inv_perm, buf.ws, st)
            if ev is not None:
                ev[0].record(st)
            moe.moe_expert_ffn_q(buf.x_perm, buf.expert_offsets, weights, sh, buf.y_perm, buf.status, qws, st)
            if ev is not None:
                ev[1].record(st)
            moe.moe_combine(buf.y_perm, buf.inv_perm, buf.topk_w, sh, buf.out, st)

        c0 = moe.moe_launch_count()
        step(0)
        launches_per_step = moe.moe_launch_count() - c0
        for i in range(3):
            step(i)
        self.barrier()
        graphs = []
        if decode:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                step(0, None, None)
            stream.wait_stream(side)
            self.barrier()
            for i0 in range(0, n_cycle, GRAPH_STEPS):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g):
                    for i in range(i0, i0 + GRAPH_STEPS):
                        step(i, None, None)
                graphs.append(g)
            for g in graphs:
                g.replay()
            self.barrier()

        def timed(n, inner=None):
            e0, e1 = self.events()
            self.barrier()
            self.hold()
            e0.record(stream)
            if decode and inner is None:
                for i in range(n // GRAPH_STEPS):
                    graphs[i % len(graphs)].replay()
            else:
                for i in range(n):
                    step(i, inner[i] if inner is not None else None)
            e1.record(stream)
            self.barrier()
            return max_over_ranks(e0.elapsed_time(e1), self.world)

        pilot_n = GRAPH_STEPS if decode else 2
        pilot = timed(pilot_n) / pilot_n
        n = steps_for_region(pilot, min_ms, multiple=GRAPH_STEPS if decode else 1, at_least=3)
        time.sleep(COOLDOWN_S)
        ms = timed(n) / n
        n_e = min(n, 64)
        inner = [self.events() for _ in range(n_e)]
        timed(n_e, inner)
        ffn_ms = float(np.mean([a.elapsed_time(b) for a, b in inner]))
        assert int(buf.status.item()) == 0, "device-side wait timed out"
        peaks = self.peaks
        mean_touched = float(np.mean(touched))
        if decode:
            # weights of the touched experts once, token rows in, fp32 rows out; the quantised rows are 1/4 of the bf16 ones
            alg = ffn_algorithmic_bytes(wl, mean_touched)
            achieved = alg / (ffn_ms * 1e-3) / 1e9
            roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm"], "unit": "GB/s", "frac": achieved / peaks["hbm"],
                    "traffic": None, "algorithmic_bytes": alg, "ms": ffn_ms, "peak_source": peaks["source"]}
        else:
            achieved = ffn_flops(wl) / (ffn_ms * 1e-3) / 1e12
            peak = 4.0 * peaks["tensor_burst"]
            roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": None, "ms": ffn_ms,
                    "peak_source": "4 x the measured bf16 burst peak (nominal FP4 : bf16 ratio); " + peaks["source"]}
        roof.update({"kernel": "moe_expert_ffn_q", "experts_touched": mean_touched,
                     "timed_in": "CUDA events around the call in eager steps right after the timed round"})
        kernels = moe.moe_last_kernel_name()
        del graphs, batches, buf, qws
        torch.cuda.empty_cache()
        return {"ms_per_step": ms, "value": wl.T * self.world / (ms * 1e-3), "unit": "tokens/s", "steps": n,
                "gpu_launches_per_step": launches_per_step, "roofline": roof,
                "call": "moe_route, moe_permute, moe_expert_ffn_q, moe_combine",
                "launch": ("cuda graph replay, %d steps per graph" % GRAPH_STEPS) if decode else "eager",
                "numerics": "E2M1 activations with one E8M0 scale per 32 elements: a different result from the bf16-activation "
                            "workloads (its own oracle), about 0.2 of the output norm away"}

    def run_ep_emulated(self, wl, world=8, min_ms=20.0):
        """Expert-parallel sharding, ONE rank's step as this GPU would run it in a job of `world` GPUs: routing and sort of
        all tokens, the row table, the rank's experts (their down projection storing through the table - here into
        buffers on the same GPU, so the links are not in the figure), the combine of the rank's tokens.  Row-layout
        weights of the rank's experts; CUDA graph of eight steps for decode."""
        torch, moe, inputs = self.torch, self.moe, self.inputs
        from paper_2609_15627_b200 import ep
        stream = self.stream
        decode = wl.name in DECODE
        sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
        e0, e1, _, _, _ = ep.partition(wl.T, wl.E, world, 0)
        w_local = tuple(self.dev(np.ascontiguousarray(a[e0:e1]))
                        for a in inputs.make_expert_weights(wl.H, wl.I, wl.E, seed=0, experts=range(e0, e1)))
        n_cycle = 8 if decode else 2
        batches = [(self.dev(inputs.make_logits(wl.T, wl.E, 7000 + i, wl.skew)), self.dev(inputs.make_x(wl.T, wl.H, 7000 + i)))
                   for i in range(n_cycle)]
        ranks = [ep.RankBuffers(torch, moe, sh, world, 0)]
        others = [torch.empty_like(ranks[0].y_own) for _ in range(world - 1)]  # the other ranks' buffers (never read here)
        ptrs = torch.tensor([ranks[0].y_own.data_ptr()] + [t.data_ptr() for t in others], dtype=torch.int64, device="cuda")
        ranks[0].owner_y.copy_(ptrs)
        out = torch.empty((wl.T, wl.H), dtype=torch.bfloat16, device="cuda")
        b = ranks[0]

        def step(i, st=stream):
            l, x = batches[i % n_cycle]
            ep.compute(moe, b, l, x, w_local, st)
            ep.finish(moe, b, out, st)

        for i in range(3):
            step(i)
        self.barrier()
        g = None
        if decode:
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                step(0, None)
            stream.wait_stream(side)
            self.barrier()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in range(n_cycle):
                    step(i, None)
            g.replay()
            self.barrier()

        def timed(n):
            e_0, e_1 = self.events()
            self.barrier()
            self.hold()
            e_0.record(stream)
            for i in range(n):
                if g is not None:
                    g.replay()
                else:
                    step(i)
            e_1.record(stream)
            self.barrier()
            return e_0.elapsed_time(e_1) / (n * (n_cycle if g is not None else 1))

        pilot = timed(2)
        n = max(3, int(min_ms / max(pilot * (n_cycle if g is not None else 1), 1e-3)))
        ms = timed(n)
        assert int(b.layer.status.item()) == 0, "device-side wait timed out"
        del g, ranks, others, batches, w_local
        torch.cuda.empty_cache()
        return {"world": world, "rank_ms_per_step": ms, "experts_per_rank": e1 - e0,
                "note": "one rank's step on one GPU; the stores that would cross the links land in local buffers"}

    def read_only_stream(self, status):
        """Read-only ceiling: the decode kernel's load mechanism alone over the resident gate/up weights (2.1 GB at
        the production shape, larger than L2).  Context for the HBM-bound workloads, not the denominator."""
        if self.read_only_gbs is not None:
            return self.read_only_gbs
        torch, moe = self.torch, self.moe
        src = self.packed if self.packed is not None else self.weights[0]
        if src.numel() < (1 << 28):
            return None
        sink = torch.empty(4096, dtype=torch.int32, device="cuda")
        for _ in range(2):
            moe.moe_debug_read_probe(src, sink, status, self.stream)
        p0, p1 = self.events()
        p0.record(self.stream)
        for _ in range(5):
            moe.moe_debug_read_probe(src, sink, status, self.stream)
        p1.record(self.stream)
        self.barrier()
        self.read_only_gbs = 5 * src.numel() / (p0.elapsed_time(p1) * 1e-3) / 1e9
        return self.read_only_gbs

    # ---- one workload -------------------------------------------------------------------------------------------
    def run(self, wl, exact_steps=None, warmup=3, e2e=True):
        """Times `wl`.  exact_steps: also time one region of exactly that many steps (the headline's K).
        Returns the per-workload record; with exact_steps its 'exact' entry holds that region."""
        torch, moe, inputs, args = self.torch, self.moe, self.inputs, self.args
        rank, world, stream = self.rank, self.world, self.stream
        decode = wl.name in DECODE or wl.name == "tiny"
        self.load_weights(wl)
        packed, weights = self.packed, self.weights
        sh = moe.shape(wl.T, wl.H, wl.I, wl.E, wl.k)
        n_cycle = 32 if decode else 2
        batches_host = [(inputs.make_logits(wl.T, wl.E, 7000 + rank * 100 + i, wl.skew),
                         inputs.make_x(wl.T, wl.H, 7000 + rank * 100 + i)) for i in range(n_cycle)]
        batches = [(self.dev(l), self.dev(x)) for l, x in batches_host]
        buf = moe.LayerBuffers(sh)
        fws = moe.alloc_forward_workspace(sh)

        # experts touched per batch of the cycle (from the library's own routing), for the byte count
        touched = []
        for l, x in batches:
            moe.moe_route(l, wl.k, buf.topk_ids, buf.topk_w, buf.expert_offsets, buf.ws)
            touched.append(int(np.count_nonzero(np.diff(buf.expert_offsets.cpu().numpy()))))

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

        # Does moe_forward run this shape as one launch?  (Asked of the library: one call, then the name of its kernel.)
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
        for i in range(max(warmup, 3)):
            step(i)
        self.barrier()

        # Decode-sized steps are a handful of short kernels: like the paper's decode tiers they are replayed as CUDA
        # graphs (the C-ABI calls captured as they are).  A serving graph holds many layers back to back; here a graph
        # holds GRAPH_STEPS consecutive batches of the cycle (one layer call each); a step count that is not a multiple of
        # GRAPH_STEPS ends with one graph of the remaining steps.
        use_graph = decode and not args.no_graph

        def capture(fn, idx):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                for i in idx:
                    fn(i, st=None)
            return g

        def warm_side(fn):
            side = torch.cuda.Stream()
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                for i in range(3):
                    fn(i, st=None)
            stream.wait_stream(side)
            self.barrier()

        graphs, multi_graphs, launches_per_step = [], [], None
        if use_graph:
            warm_side(step)
            c0 = moe.moe_launch_count()
            graphs = [capture(step, [0])]
            launches_per_step = moe.moe_launch_count() - c0
            multi_graphs = [capture(step, range(i0, i0 + GRAPH_STEPS)) for i0 in range(0, n_cycle, GRAPH_STEPS)]
            for g in graphs + multi_graphs:
                g.replay()
            self.barrier()

        rem_graphs, whole_graphs = {}, {}

        def prepare(n, whole=False):
            """A step count that is not a multiple of GRAPH_STEPS ends with ONE graph of the remaining steps (captured
            here, before the timed region).  whole: the region of exactly --steps steps is ONE graph of all its steps
            (up to 4096), so that no gap between graph launches falls inside a region of a few hundred microseconds."""
            if use_graph and whole and n <= 4096:
                if n not in whole_graphs:
                    whole_graphs[n] = capture(step, range(n))
                    whole_graphs[n].replay()
                    self.barrier()
                return
            r = n % GRAPH_STEPS
            if use_graph and r and r not in rem_graphs:
                i0 = (n // GRAPH_STEPS) * GRAPH_STEPS
                rem_graphs[r] = capture(step, range(i0, i0 + r))
                rem_graphs[r].replay()
                self.barrier()

        def play(n, inner=None, whole=False):
            """Enqueue n consecutive steps of the cycle."""
            if use_graph and whole and n in whole_graphs:
                whole_graphs[n].replay()
            elif use_graph:
                n_multi = n // GRAPH_STEPS
                for i in range(n_multi):
                    multi_graphs[i % len(multi_graphs)].replay()
                if n % GRAPH_STEPS:
                    rem_graphs[n % GRAPH_STEPS].replay()
            else:
                for i in range(n):
                    step(i, inner[i] if inner is not None and i < len(inner) and not one_launch else None)

        def region(n, inner=None, whole=False):
            """One timed region of exactly n steps: barrier + synchronize on both sides, CUDA events on the launching
            stream, max over ranks.  Returns (ms of the region, clock record, launches of the library's kernels)."""
            prepare(n, whole)
            if whole and use_graph:
                # a region this short is over before the clocks have come up from idle: run about 20 ms of the same
                # steps, untimed, right in front of it
                for _ in range(max(1, int(20.0 / max(n * 0.03, 0.01)))):
                    play(n, None, whole)
            e0, e1 = self.events()
            sampler = ClockSampler(physical_gpu_index(self.local))
            c0 = moe.moe_launch_count()
            self.barrier()
            sampler.start()
            self.hold()
            e0.record(stream)
            play(n, inner, whole)
            e1.record(stream)
            self.barrier()
            clocks = sampler.stop()
            launches = launches_per_step * n if use_graph else moe.moe_launch_count() - c0
            assert int(buf.status.item()) == 0, "device-side wait timed out"
            return max_over_ranks(e0.elapsed_time(e1), world), clocks, launches

        # ---- the headline's region: exactly K steps -------------------------------------------------------------
        rec = {}
        if exact_steps is not None:
            ms, clocks, launches = region(exact_steps, whole=True)
            rec["exact"] = {"steps": exact_steps, "ms_total": ms, "ms_per_step": ms / exact_steps, "clocks": clocks,
                            "gpu_launches": launches,
                            "experts_touched": float(np.mean([touched[i % n_cycle] for i in range(exact_steps)]))}

        # ---- rounds of at least MIN_REGION_MS ---------------------------------------------------------------------
        pilot_n = GRAPH_STEPS if use_graph else 2
        pilot_ms = region(pilot_n)[0] / pilot_n
        n_steps = steps_for_region(pilot_ms, MIN_REGION_MS if decode else MIN_REGION_MS_PREFILL,
                                   multiple=GRAPH_STEPS if use_graph else 1, at_least=3)
        n_inner = 0 if (use_graph or one_launch) else n_steps
        inner = [self.events() for _ in range(n_inner)]
        rounds, clock_rounds, reasons, launches = [], [], set(), 0
        ffn_round_ms = []
        for _ in range(ROUNDS):
            time.sleep(COOLDOWN_S)
            ms, clocks, launches = region(n_steps, inner if n_inner else None)
            rounds.append(ms / n_steps)
            clock_rounds.append(clocks["sm_mhz"])
            reasons.update(clocks["reasons"])
            if n_inner:
                ffn_round_ms.append(float(np.mean([a.elapsed_time(b) for a, b in inner])))
        ms_step = float(np.median(rounds))
        region_ms = ms_step * n_steps
        mean_touched = float(np.mean([touched[i % n_cycle] for i in range(n_steps)]))
        rec.update({"ms_per_step": ms_step, "value": wl.T * world / (ms_step * 1e-3), "unit": "tokens/s",
                    "steps": n_steps, "rounds_ms_per_step": rounds, "region_ms": region_ms,
                    "gpu_launches": launches,
                    "clocks": {"sm_mhz": int(np.median([c for c in clock_rounds if c is not None])) if any(
                        c is not None for c in clock_rounds) else None, "sm_max_mhz": clocks["sm_max_mhz"],
                        "reasons": sorted(reasons), "sm_mhz_rounds": clock_rounds},
                    "call": ("moe_forward%s (one kernel launch per step)" if one_launch else
                             "moe_route, moe_permute, moe_expert_ffn%s, moe_combine") % ("_packed" if packed is not None else ""),
                    "launch": ("cuda graph replay, %d consecutive batches of the cycle per graph (the region of exactly --steps "
                               "steps: one graph of all its steps)" % GRAPH_STEPS) if use_graph else "eager",
                    "experts_touched": mean_touched})

        # ---- the expert-FFN call inside eager steps (decode: a second region right after the graph-replayed one) ---
        ffn_eager_ms, eager_ms_step = (float(np.median(ffn_round_ms)) if ffn_round_ms else None), None
        if use_graph or one_launch:
            n_e = min(n_steps, 256)
            inner_e = [self.events() for _ in range(n_e)]
            for i in range(3):
                step4(i)
            self.barrier()
            ee0, ee1 = self.events()
            ee0.record(stream)
            for i in range(n_e):
                step4(i, inner_e[i])
            ee1.record(stream)
            self.barrier()
            eager_ms_step = ee0.elapsed_time(ee1) / n_e
            ffn_eager_ms = float(np.mean([a.elapsed_time(b) for a, b in inner_e]))

        # ---- one-launch workloads: the four calls, graph-replayed the same way, for comparison -----------------------
        four_calls_ms_step = None
        if one_launch and use_graph:
            warm_side(step4)
            mg4 = [capture(step4, range(i0, i0 + GRAPH_STEPS)) for i0 in range(0, n_cycle, GRAPH_STEPS)]
            for g in mg4:
                g.replay()
            self.barrier()
            n4 = max(len(mg4), min(n_steps // GRAPH_STEPS, 128))
            g0, g1 = self.events()
            self.hold()
            g0.record(stream)
            for i in range(n4):
                mg4[i % len(mg4)].replay()
            g1.record(stream)
            self.barrier()
            four_calls_ms_step = g0.elapsed_time(g1) / (n4 * GRAPH_STEPS)
            del mg4

        # ---- the expert-FFN call alone, graph-replayed like the step (calls shorter than 100 us) -------------------------
        # Eager launches of kernels this short leave the GPU idle between the event and the launch, which the bracketing
        # events count.  So such a call is also captured alone, one graph per batch of the cycle on that batch's own routed
        # and permuted inputs, and the replays are timed back to back: consecutive calls touch different experts, as in
        # the step.  Longer calls keep the time between their events inside the eager steps.
        ffn_graph_ms, n_ffn = None, 0
        if use_graph and ffn_eager_ms is not None and ffn_eager_ms < 0.1:
            fbufs = []
            for i in range(n_cycle):
                b = moe.LayerBuffers(sh)
                l, x = batches[i]
                moe.moe_route(l, wl.k, b.topk_ids, b.topk_w, b.expert_offsets, b.ws, stream)
                moe.moe_permute(x, b.topk_ids, b.expert_offsets, sh, b.x_perm, b.perm, b.inv_perm, b.ws, stream)
                fbufs.append(b)
            self.barrier()

            def ffn_only(i, st=stream):
                expert_ffn(fbufs[i % n_cycle], st)

            warm_side(ffn_only)
            fgraphs = [capture(ffn_only, [i]) for i in range(n_cycle)]
            for i in range(3):
                fgraphs[i].replay()
            self.barrier()
            n_ffn = max(n_cycle, min(n_steps, 1024))
            f0, f1 = self.events()
            self.hold()
            f0.record(stream)
            for i in range(n_ffn):
                fgraphs[i % n_cycle].replay()
            f1.record(stream)
            self.barrier()
            ffn_graph_ms = f0.elapsed_time(f1) / n_ffn
            assert all(int(b.status.item()) == 0 for b in fbufs), "device-side wait timed out"
            del fgraphs, fbufs

        # ---- roofline of the dominant call (the expert FFN), and of the whole step ---------------------------------
        peaks = self.peaks
        ffn_ms = ffn_graph_ms if ffn_graph_ms is not None else ffn_eager_ms
        timed_in = ("graph replays of the call alone, one graph per batch of the cycle, right after the timed rounds"
                    if ffn_graph_ms is not None else
                    ("eager steps right after the graph-replayed rounds" if use_graph or one_launch else
                     "CUDA events around the call inside every step of the timed rounds"))
        if decode:
            alg = ffn_algorithmic_bytes(wl, mean_touched)
            achieved = alg / (ffn_ms * 1e-3) / 1e9
            roof = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm"], "unit": "GB/s", "frac": achieved / peaks["hbm"],
                    "traffic": NCU_TRAFFIC_BYTES.get(wl.name), "algorithmic_bytes": alg, "ms": ffn_ms,
                    "peak_source": peaks["source"]}
            alg_step = layer_algorithmic_bytes(wl, mean_touched)
            step_roof = {"bound": "hbm", "achieved": alg_step / (ms_step * 1e-3) / 1e9, "peak": peaks["hbm"], "unit": "GB/s",
                         "frac": alg_step / (ms_step * 1e-3) / 1e9 / peaks["hbm"], "algorithmic_bytes": alg_step, "ms": ms_step,
                         "peak_source": peaks["source"],
                         "traffic": NCU_TRAFFIC_BYTES.get(wl.name + "_one_launch") if one_launch else None}
        else:
            roof = tensor_roofline(ffn_flops(wl), ffn_ms, region_ms, peaks)
            roof["traffic"] = NCU_TRAFFIC_BYTES.get(wl.name)
            step_roof = tensor_roofline(ffn_flops(wl), ms_step, region_ms, peaks)
        roof.update({"kernel": "moe_expert_ffn", "experts_touched": mean_touched, "timed_in": timed_in,
                     "ms_between_events_in_eager_steps": ffn_eager_ms})
        step_roof.update({"kernel": "the whole step (%s)" % rec["call"], "timed_in": "the timed rounds"})
        if one_launch:
            # the dominant kernel is the step itself: one launch per step, timed by the events of the timed rounds
            step_roof["four_calls"] = {"ms_per_step": four_calls_ms_step, "eager_ms_per_step": eager_ms_step, "expert_ffn": roof}
            rec["roofline"] = step_roof
        else:
            rec["roofline"] = roof
            rec["roofline_step"] = step_roof
            rec["eager_ms_per_step"] = eager_ms_step
        if decode:
            gbs = self.read_only_stream(buf.status)
            if gbs is not None:
                rec["roofline"]["read_only_stream_gbs"] = gbs
                rec["roofline"]["frac_of_read_only_stream"] = rec["roofline"]["achieved"] / gbs

        # ---- end to end through the host-buffer entry point ---------------------------------------------------------
        if e2e and not args.no_e2e:
            ws_h = moe.alloc_workspace(sh, host_path=True)
            lh = [torch.from_numpy(l).pin_memory() for l, _ in batches_host]
            xh = [torch.from_numpy(x.view(np.int16)).pin_memory() for _, x in batches_host]
            oh = torch.empty((wl.T, wl.H), dtype=torch.int16).pin_memory()
            n_e2e = max(3, min(exact_steps if exact_steps is not None else n_steps, 200 if decode else 5))

            # one call object per batch of the cycle, arguments marshalled once (the buffers are reused every step)
            calls = [moe.bind_forward_host(lh[i], xh[i], packed if packed is not None else weights, sh, oh, buf.status, ws_h, stream)
                     for i in range(n_cycle)]

            def forward_host(i):
                calls[i % n_cycle]()

            for i in range(3):
                forward_host(i)
            self.barrier()
            t0 = time.perf_counter()
            for i in range(n_e2e):
                forward_host(i)
            dt = max_over_ranks(time.perf_counter() - t0, world)
            rec["e2e"] = {"value": wl.T * world * n_e2e / dt, "unit": "tokens/s",
                          "h2d_bytes_per_step": wl.T * wl.E * 4 + wl.T * wl.H * 2, "d2h_bytes_per_step": wl.T * wl.H * 2,
                          "steps": n_e2e, "call": "%s (pinned host logits/x in, bf16 out back, weights resident)"
                                  % ("moe_forward_host_packed" if packed is not None else "moe_forward_host")}
            del calls, ws_h, lh, xh, oh
        rec["kernels"] = moe.moe_last_kernel_name()
        rec["one_launch"] = one_launch
        rec["n_cycle"] = n_cycle
        del graphs, multi_graphs, whole_graphs, rem_graphs, batches, buf, fws
        torch.cuda.empty_cache()
        return rec


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default=None, help="time this workload only (default: all four production workloads, headline decode_c1)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="decode workloads: launch the calls eagerly instead of replaying CUDA graphs")
    ap.add_argument("--no-block", action="store_true", help="skip the timing of moe_ffn_block")
    ap.add_argument("--no-quant", action="store_true", help="skip the quantised-activation variant (moe_expert_ffn_q)")
    ap.add_argument("--only-quant", action="store_true", help="time only the quantised-activation variant of --workload")
    ap.add_argument("--min-ms", type=float, default=50.0, help="with --only-quant: length of the timed round")
    ap.add_argument("--four-calls", action="store_true", help="time the four calls even where moe_forward is one launch")
    ap.add_argument("--raw-weights", action="store_true", help="read the weights in the checkpoint's row layout instead of moe_prepack's tiles")
    args = ap.parse_args()

    from paper_2609_15627_b200 import inputs
    head = inputs.WORKLOADS[args.workload or HEADLINE]
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 5
        args.warmup = args.warmup if args.warmup is not None else 1
        run_reference(args, head, inputs)
        return
    head_decode = head.name in DECODE or head.name == "tiny"
    if args.steps is None:
        args.steps = 2000 if head_decode else 10
    if args.warmup is None:
        args.warmup = 20 if head_decode else 3
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

    bench = Bench(args, rank, world, local)
    if args.only_quant:
        # the variant alone (for a profiler capture: nothing else launches before it but the routing and the load transform)
        assert world == 1 and head.name in QUANT_WORKLOADS
        bench.load_weights(head)
        print(json.dumps({"quantised_activations": {head.name + "_q": bench.run_quant(head, min_ms=args.min_ms)}}))
        return
    # every rank times the same list, in the same order (the barriers pair up)
    # (replicas, N > 1: the headline workload only - the scaling figure is the headline's)
    names = [args.workload] if args.workload else [HEADLINE] + ([n for n in PRODUCTION if n != HEADLINE] if world == 1 else [])
    # the FFN block around the routed path (router projection, shared expert, join), beside the headline (N = 1, default run)
    block = None
    if world == 1 and not args.workload and not args.raw_weights and not args.no_block:
        bench.load_weights(head, keep_raw=True)
        block = {n: bench.run_block(inputs.WORKLOADS[n]) for n in ("decode_c1", "decode_c64", "prefill_8k")}
        bench.raw = None
        torch.cuda.empty_cache()
    records, quant = {}, {}
    for name in names:
        wl = inputs.WORKLOADS[name]
        records[name] = bench.run(wl, exact_steps=args.steps if name == head.name else None, warmup=args.warmup)
        # the quantised-activation variant of the same workload, on the weights this workload has just loaded
        if world == 1 and not args.no_quant and name in QUANT_WORKLOADS:
            quant[name + "_q"] = bench.run_quant(wl)
    # expert-parallel sharding: one emulated rank of eight (N = 1, default run)
    ep_emulated = None
    packed_layout = bench.packed is not None
    if world == 1 and not args.workload and not args.no_block:
        bench.weights = bench.packed = None
        torch.cuda.empty_cache()
        ep_emulated = {n: bench.run_ep_emulated(inputs.WORKLOADS[n]) for n in ("decode_c64", "prefill_8k")}
    hr = records[head.name]
    ex = hr.pop("exact")

    # ---- the headline: exactly K steps of the headline workload ------------------------------------------------
    ms_step = ex["ms_per_step"]
    value = head.T * world / (ms_step * 1e-3)
    peaks = bench.peaks
    roof = dict(hr["roofline"])
    if hr["one_launch"]:
        alg = layer_algorithmic_bytes(head, ex["experts_touched"])
        achieved = alg / (ms_step * 1e-3) / 1e9
        roof.update({"achieved": achieved, "frac": achieved / peaks["hbm"], "algorithmic_bytes": alg, "ms": ms_step,
                     "experts_touched": ex["experts_touched"], "timed_in": "the timed region"})
        if "read_only_stream_gbs" in roof:
            roof["frac_of_read_only_stream"] = achieved / roof["read_only_stream_gbs"]

    # ---- the oracle on the host cores (rank 0, N = 1 only) ----------------------------------------------------------
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        # about 10-20 s of host work at the production shape (the oracle does roughly 50 tokens/s on 16 cores)
        n_tok = {"tiny": 4096}.get(head.name, 640)
        v, dt, n, cores = oracle_sample(head, inputs, n_tok, weights=bench.weights_host)
        cpu = {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle",
               "sample": "%d tokens with the %s shape and routing distribution, per-token definition, %.1f s" % (n, head.name, dt)}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": head.name, "T": head.T, "H": head.H, "I": head.I, "E": head.E, "k": head.k,
                       "parallelism": "replicas only" if world > 1 else "1 GPU", "call": hr["call"],
                       "weights": ("moe_prepack's tile-contiguous layout (one-time transform, same bytes)"
                                   if packed_layout else "checkpoint row layout"),
                       "launch": hr["launch"],
                       "l2": "inputs cycle over %d seeded batches; %.2f GB of expert weights resident (larger than L2)"
                             % (hr["n_cycle"], head.E * expert_weight_bytes(head.H, head.I) / 1e9)},
            "roofline": roof, "cpu_baseline": cpu, "e2e": hr.get("e2e"), "gpu_launches": ex["gpu_launches"],
            "clocks": ex["clocks"], "kernels": hr["kernels"],
            "workloads": {n: {k: v for k, v in r.items() if k not in ("one_launch", "n_cycle")} for n, r in records.items()},
            "ffn_block": block,
            "quantised_activations": quant or None,
            "expert_parallel_emulated": ep_emulated,
            "protocol": ("headline: one region of exactly --steps steps; workloads: %d rounds of at least %d ms (decode) / %d ms "
                         "(prefill) each, %.1f s idle before every round, median reported, every round kept; every region is "
                         "bracketed by a barrier and a synchronize, timed by CUDA events on the launching stream behind a "
                         "100 us hold kernel, max over ranks") % (ROUNDS, MIN_REGION_MS, MIN_REGION_MS_PREFILL, COOLDOWN_S),
        }
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
