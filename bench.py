#!/usr/bin/env python3
"""Benchmark of the sparse-bitmap codec hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic
activations shaped like a ResNet-18 at batch 32 (17 post-ReLU tensors, fp32,
about half zeros): in forward order every layer is stashed twice -- once with
bt_compress (from the post-ReLU activation) and once with bt_relu_fwd_compress
(from the pre-activation) -- and in reverse order every layer is restored with
bt_decompress and its ReLU gradient formed with bt_relu_bwd_from_bitmap.  The
metric is dense-equivalent GB/s: the dense bytes of every tensor an entry point
consumed or produced (N * sizeof(dtype) per call), summed over the step,
divided by the step time.  The step is one CUDA graph of eight independent chains
(plain codec / fused pair, layers by index mod 4) on eight streams; each compress
launch is limited to a share of the SMs (bt_set_max_ctas) so that the chains'
cooperative launches are resident side by side.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank
runs the same batch shard on its own GPU -- data-parallel replicas compress
their own activations, there is no data-path collective -- and the value is the
sum over ranks divided by the slowest rank's time (weak scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "codec_dense_equivalent_throughput"
UNIT = "GB/s"
WORKLOAD = "cfg2_resnet18_b32_f32"
OPS = ("bt_compress", "bt_relu_fwd_compress", "bt_decompress", "bt_relu_bwd_from_bitmap")


def parse_args():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=200)
    p.add_argument("--warmup", type=int, default=5)
    p.add_argument("--impl", choices=("ours", "reference"), default="ours")
    p.add_argument("--batch", type=int, default=32, help="batch of the ResNet-18-shaped set (32 = the named config)")
    p.add_argument("--no-cpu-baseline", action="store_true")
    p.add_argument("--no-large", action="store_true", help="skip the per-kernel runs on 1 GiB tensors")
    p.add_argument("--no-e2e", action="store_true")
    p.add_argument("--chains", type=int, choices=(1, 2, 4, 8), default=8,
                   help="independent chains of the step's graph: 2 = plain codec / fused pair on two streams, "
                        "4 = each of them split into even and odd layers, 8 = into layers by index mod 4")
    p.add_argument("--cta-budget", default="24,74",
                   help="CTAs per compress launch when the step runs as several chains: 'small,large' for layers "
                        "of at most / more than 800 tiles of 8192 elements (0 = one CTA per SM); see bt_set_max_ctas")
    return p.parse_args()


# ------------------------------------------------------------------------------------------
# clocks: read-only NVML sampling in a thread while the timed region runs
class ClockSampler:
    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples = []          # (host time, sm MHz, reasons bitmask)
        self.period = period_s
        self._stop = threading.Event()
        self.ok = False
        self.sm_max = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = self._handle(index)
            self.sm_max = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False
        self.thread = threading.Thread(target=self._run, daemon=True)

    def _handle(self, index):
        import torch
        try:
            uuid = str(torch.cuda.get_device_properties(index).uuid)
            uuid = uuid if uuid.startswith("GPU-") else "GPU-" + uuid
            return self.nv.nvmlDeviceGetHandleByUUID(uuid)
        except Exception:
            return self.nv.nvmlDeviceGetHandleByIndex(index)

    def _run(self):
        while not self._stop.is_set():
            try:
                mhz = int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
                try:
                    r = int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                self.samples.append((time.time(), mhz, r))
            except Exception:
                pass
            self._stop.wait(self.period)

    def start(self):
        if self.ok:
            self.thread.start()

    def stop(self):
        self._stop.set()
        if self.ok and self.thread.is_alive():
            self.thread.join(timeout=1.0)

    def summary(self, t0: float, t1: float) -> dict:
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        note = "sampled during the timed region"
        if not inside:
            inside = self.samples[-3:]
            note = "timed region shorter than the sampling period: nearest samples"
        if not inside:
            return {"sm_mhz": None, "sm_max_mhz": self.sm_max, "reasons": [], "note": "NVML unavailable"}
        mask = 0
        for s in inside:
            mask |= s[2]
        reasons = [name for bit, name in self.REASONS.items() if mask & bit and name != "gpu_idle"]
        return {"sm_mhz": statistics.median(s[1] for s in inside), "sm_max_mhz": self.sm_max,
                "reasons": reasons, "samples": len(inside), "note": note}


# ------------------------------------------------------------------------------------------
# DRAM bytes per launch (read + write) of the dominant kernel class over one step of this workload, from the ncu
# capture summarised in profiles/bench_cfg2_launch_list.md (bytes; None where no capture exists)
NCU_TRAFFIC_PER_LAUNCH = {"bt_compress": 20.57e6, "bt_relu_fwd_compress": 20.61e6, "bt_decompress": 13.88e6}


def max_over_ranks(ms: float, world: int, device) -> float:
    """Slowest rank's time: the job is as fast as its slowest GPU."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(dense_bytes_per_rank_step: int, world: int, ms_per_step: float) -> float:
    """Dense-equivalent GB/s of the whole job: every rank processes its own batch shard (weak scaling)."""
    return world * dense_bytes_per_rank_step / (ms_per_step * 1e-3) / 1e9


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def algorithmic_bytes(op: str, n: int, nnz: int, es: int, with_y: bool = False) -> int:
    """Bytes the method itself must move for one call (dense tensor, bitmap, packed values, prefix)."""
    compressed = 4 * ((n + 31) // 32) + nnz * es + 8 * ((n + 4095) // 4096)
    if op in ("bt_compress", "bt_decompress"):
        return n * es + compressed
    if op == "bt_relu_fwd_compress":
        return n * es + compressed + (n * es if with_y else 0)
    if op == "bt_relu_bwd_from_bitmap":
        return 2 * n * es + 4 * ((n + 31) // 32)
    raise ValueError(op)


class Cfg2Step:
    """Device-resident state of one step over the ResNet-18-shaped activation set."""

    def __init__(self, dev, batch: int):
        import torch
        from paper_2110_15362_b200 import binding as B
        from paper_2110_15362_b200 import workloads as W
        self.B, self.torch = B, torch
        self.shapes = W.resnet18_shapes(batch)
        self.layers = []
        n_max = max(W.numel(s) for s in self.shapes)
        for i, shape, n in W.iter_layers(self.shapes):
            pre = W.cfg2_preact(i, shape, dev).reshape(-1)
            act = torch.clamp_min(pre, 0.0)                     # == W.cfg2_layer(i, shape): same seed
            grad = W.cfg2_grad(i, shape, dev).reshape(-1)
            self.layers.append(dict(n=n, pre=pre, act=act, grad=grad,
                                    stash_a=B.Stash(n, torch.float32, dev), stash_b=B.Stash(n, torch.float32, dev)))
        # one output buffer and one workspace per chain (at most eight chains); chain 0 restores the activations
        self.outs = [torch.empty(n_max, dtype=torch.float32, device=dev) for _ in range(8)]
        self.wss = [B.new_workspace(n_max, dev) for _ in range(8)]
        self.restored, self.gin, self.ws = self.outs[0], self.outs[1], self.wss[0]
        self.total_elems = sum(l["n"] for l in self.layers)
        self.dense_bytes_per_step = len(OPS) * 4 * self.total_elems
        self.launches_per_step = len(OPS) * len(self.layers)
        # CTAs per compress launch (small layers, large layers); (0, 0) = one CTA per SM.  A cooperative launch
        # starts only when all its CTAs fit, so chains that are to overlap get a share of the SMs each.
        self.cta_budget = (0, 0)

    def cta_limit(self, n: int) -> int:
        if len(self.cta_budget) == 5:                        # experiments: one limit per layer size, smallest first
            tiles = (n + 8191) // 8192
            return self.cta_budget[sum(tiles > t for t in (100, 200, 400, 800))]
        return self.cta_budget[0] if n <= 800 * 8192 else self.cta_budget[1]

    def run(self, only_op=None, only_layer=None, streams=None):
        """One step (forward over the layers, backward in reverse).  `only_op` / `only_layer` restrict it to
        one operation and / or one layer, for the per-operation timing passes.  With `streams` (a list of 2,
        4 or 8 streams, the first being the current one) the step runs as independent chains -- the plain codec
        (compress ... decompress) and the fused pair (fused forward ... ReLU backward), each optionally split
        into even and odd layers or into layers by index mod 4 -- every chain with its own stream, workspace and output buffer, so that one
        chain's launch latency hides behind another's kernels."""
        B = self.B
        k = 1 if not streams else len(streams)

        def chain(family, i):                       # family 0: plain codec, 1: fused pair
            if k == 1:
                return 0
            return family if k == 2 else (2 * family + (i & 1) if k == 4 else 4 * family + (i & 3))

        def want(op, i):
            return (only_op is None or op == only_op) and (only_layer is None or i == only_layer)

        for i, l in enumerate(self.layers):
            a, b = l["stash_a"], l["stash_b"]
            B.bt_set_max_ctas(self.cta_limit(l["n"]))
            if want("bt_compress", i):
                c = chain(0, i)
                B.bt_compress(l["act"], a.bitmap, a.values, a.chunk_prefix, a.nnz_out, self.wss[c], a.dev_status,
                              stream=streams[c] if streams else None)
            if want("bt_relu_fwd_compress", i):
                c = chain(1, i)
                B.bt_relu_fwd_compress(l["pre"], None, b.bitmap, b.values, b.chunk_prefix, b.nnz_out, self.wss[c],
                                       b.dev_status, stream=streams[c] if streams else None)
        B.bt_set_max_ctas(0)
        for i in range(len(self.layers) - 1, -1, -1):
            l = self.layers[i]
            a, b = l["stash_a"], l["stash_b"]
            n = l["n"]
            if want("bt_decompress", i):
                c = chain(0, i)
                B.bt_decompress(a.bitmap, a.values, a.chunk_prefix, self.outs[c if k > 1 else 0][:n],
                                stream=streams[c] if streams else None)
            if want("bt_relu_bwd_from_bitmap", i):
                c = chain(1, i)
                B.bt_relu_bwd_from_bitmap(b.bitmap, l["grad"], self.outs[c if k > 1 else 1][:n],
                                          stream=streams[c] if streams else None)

    def check(self):
        """After a step: device status words are clean and both stashes of a layer agree."""
        torch = self.torch
        for l in self.layers:
            a, b = l["stash_a"], l["stash_b"]
            assert a.status == 0 and b.status == 0, "device status not BT_OK"
            assert a.nnz == b.nnz, "the two stashes of a layer disagree"
        last = self.layers[0]
        assert torch.equal(self.restored[:last["n"]].view(torch.int32), last["act"].view(torch.int32)), \
            "round trip is not bit exact"

    def nnz(self):
        return [l["stash_a"].nnz for l in self.layers]


def per_kernel_pass(step: Cfg2Step, steps: int, chains: int = 1):
    """Device time of each operation: the step's launches of ONE operation (all 17 layers, in the step's
    order and launch configuration: with four or eight chains the operation's own two or four chains on their
    streams, with the step's CTA budget) captured as a CUDA graph of their own and replayed `steps` times between two CUDA
    events on the launching stream, so the figure holds what the whole-step graph holds for that operation
    (kernel time, the device's launch latency between dependent kernels, the overlap of the operation's own
    two chains) and no host overhead.  The inputs of one such pass (0.3 GB and more) exceed the L2.  The
    largest layer is timed on its own, one launch with one CTA per SM, the L2 flushed before every replay."""
    import torch
    dev = step.restored.device
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    per_op, per_layer = {}, {}
    side = torch.cuda.Stream()
    branches = [torch.cuda.Stream() for _ in range(chains - 1)] if chains >= 4 else []
    budget = step.cta_budget
    for op in OPS:
        graphs = []
        for only in (None, 0):
            g = torch.cuda.CUDAGraph()
            step.cta_budget = budget if only is None else (0, 0)
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                step.run(only_op=op, only_layer=only)          # warm-up outside the capture
            torch.cuda.current_stream().wait_stream(side)
            with torch.cuda.graph(g):
                if branches and only is None:
                    main_stream = torch.cuda.current_stream()
                    for b in branches:
                        b.wait_stream(main_stream)
                    step.run(only_op=op, streams=[main_stream] + branches)
                    for b in branches:
                        main_stream.wait_stream(b)
                else:
                    step.run(only_op=op, only_layer=only)
            graphs.append(g)
        step.cta_budget = budget
        whole, big = graphs
        for _ in range(3):
            whole.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            whole.replay()
        e1.record()
        torch.cuda.synchronize()
        per_op[op] = {"ms": e0.elapsed_time(e1), "launches": steps * len(step.layers)}
        times = []
        for _ in range(max(5, min(steps, 20))):
            flush.fill_(1)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            big.replay()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        per_layer[(op, 0)] = times
    return per_op, per_layer


def large_tensor_kernels(dev, peak_gbs: float):
    """Every kernel alone on a 1 GiB fp32 tensor (2^28 elements, half zeros) and on the largest
    VGG-16-shaped bf16 tensor: the sizes at which the kernels are held to the HBM roofline."""
    import torch
    from paper_2110_15362_b200 import binding as B
    from paper_2110_15362_b200 import workloads as W
    out = {}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def time_call(fn, reps=10):
        best = []
        for _ in range(3):
            fn()
        for _ in range(reps):
            flush.fill_(1)                       # evict L2 between timed launches
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            best.append(e0.elapsed_time(e1))
        return statistics.median(best), min(best)

    for label, kind, n in (("f32_2^28_s0.5", "f32", 1 << 28), ("bf16_64x64x224x224", "bf16", 64 * 64 * 224 * 224),
                           ("f64_2^27_s0.5", "f64", 1 << 27)):
        if kind == "f32":
            x = W.cfg3_iid(n, 0.5, 2, dev)
            pre = x
        elif kind == "f64":
            x = W.cfg3_iid(n, 0.5, 3, dev).double()
            pre = x
        else:
            pre = W.cfg4_preact(0, (n,), kind, dev)
            x = torch.relu(pre)
        es = x.element_size()
        st = B.Stash(n, x.dtype, dev)
        ws = B.new_workspace(n, dev)
        dense = torch.empty_like(x)
        res = {}
        ms, best = time_call(lambda: B.bt_compress(x, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, ws,
                                                   st.dev_status))
        nnz = st.nnz
        res["bt_compress"] = (ms, best, algorithmic_bytes("bt_compress", n, nnz, es))
        ms, best = time_call(lambda: B.bt_decompress(st.bitmap, st.values, st.chunk_prefix, dense))
        iv = {2: torch.int16, 4: torch.int32, 8: torch.int64}[es]
        assert torch.equal(dense.view(iv), x.view(iv))
        res["bt_decompress"] = (ms, best, algorithmic_bytes("bt_decompress", n, nnz, es))
        ms, best = time_call(lambda: B.bt_relu_fwd_compress(pre, None, st.bitmap, st.values, st.chunk_prefix,
                                                            st.nnz_out, ws, st.dev_status))
        res["bt_relu_fwd_compress"] = (ms, best, algorithmic_bytes("bt_relu_fwd_compress", n, st.nnz, es))
        ms, best = time_call(lambda: B.bt_relu_fwd_compress(pre, dense, st.bitmap, st.values, st.chunk_prefix,
                                                            st.nnz_out, ws, st.dev_status))
        res["bt_relu_fwd_compress+y"] = (ms, best, algorithmic_bytes("bt_relu_fwd_compress", n, st.nnz, es, True))
        ms, best = time_call(lambda: B.bt_relu_bwd_from_bitmap(st.bitmap, x, dense))
        res["bt_relu_bwd_from_bitmap"] = (ms, best, algorithmic_bytes("bt_relu_bwd_from_bitmap", n, 0, es))
        # ReLU6 pair (a "next" row): fused forward, stash only, and the backward that consults the stashed values
        ms, best = time_call(lambda: B.bt_relu6_fwd_compress(pre, None, st.bitmap, st.values, st.chunk_prefix,
                                                             st.nnz_out, ws, st.dev_status))
        nnz6 = st.nnz
        res["bt_relu6_fwd_compress"] = (ms, best, algorithmic_bytes("bt_relu_fwd_compress", n, nnz6, es))
        ms, best = time_call(lambda: B.bt_relu6_bwd_from_stash(st.bitmap, st.values, st.chunk_prefix, x, dense))
        res["bt_relu6_bwd_from_stash"] = (ms, best, 2 * n * es + 4 * ((n + 31) // 32) + 8 * ((n + 4095) // 4096) + nnz6 * es)
        if kind == "f32":
            # down-cast on stash (a "next" row): float32 tensor, 16-bit stashed values
            for to, tdt in (("f16", torch.float16), ("bf16", torch.bfloat16)):
                v16 = torch.empty(n, dtype=tdt, device=dev)
                ms, best = time_call(lambda: B.bt_compress_narrow(x, st.bitmap, v16, st.chunk_prefix, st.nnz_out, ws,
                                                                  st.dev_status))
                by16 = n * es + 4 * ((n + 31) // 32) + 8 * ((n + 4095) // 4096) + st.nnz * 2
                res["bt_compress_narrow_" + to] = (ms, best, by16)
                ms, best = time_call(lambda: B.bt_prune_fwd_compress_narrow(pre, 0.0, None, st.bitmap, v16, st.chunk_prefix,
                                                                            st.nnz_out, ws, st.dev_status))
                res["bt_prune_fwd_compress_narrow_" + to] = (ms, best, by16)
                ms, best = time_call(lambda: B.bt_decompress_widen(st.bitmap, v16, st.chunk_prefix, dense))
                res["bt_decompress_widen_" + to] = (ms, best, by16)
                del v16
        # double-mask form (a "next" row): the stash of x masks a dense tensor of the same shape
        B.bt_compress(x, st.bitmap, st.values, st.chunk_prefix, st.nnz_out, ws, st.dev_status)
        nnz = st.nnz
        masked_vals = torch.empty(nnz, dtype=x.dtype, device=dev)
        by = n * es + 4 * ((n + 31) // 32) + 8 * ((n + 4095) // 4096) + nnz * es
        ms, best = time_call(lambda: B.bt_mask_compress(pre, st.bitmap, st.chunk_prefix, None, masked_vals))
        res["bt_mask_compress"] = (ms, best, by)
        ms, best = time_call(lambda: B.bt_mask_compress(pre, st.bitmap, st.chunk_prefix, dense, masked_vals))
        res["bt_mask_compress+y"] = (ms, best, by + n * es)
        del masked_vals
        out[label] = {op: {"ms_median": round(ms, 4), "ms_best": round(best, 4),
                           "moved_gbs": round(by / ms / 1e6, 1),
                           "dense_equiv_gbs": round(n * es / ms / 1e6, 1),
                           "frac_of_measured_copy": round(by / ms / 1e6 / peak_gbs, 3),
                           "frac_of_8000": round(by / ms / 1e6 / 8000.0, 3)}
                      for op, (ms, best, by) in res.items()}
        del x, pre, st, ws, dense
        torch.cuda.empty_cache()

    # activation pruning fused with the stash (the next row of the scope after the hot path): one pass
    # over 2^28 close-to-zero fp32 pre-activations per threshold of the paper's study
    n = 1 << 28
    pre = W.prune_preact(n, dev)
    st = B.Stash(n, pre.dtype, dev)
    ws = B.new_workspace(n, dev)
    rows = {}
    for tau in W.PRUNE_THRESHOLDS:
        ms, best = time_call(lambda: B.bt_prune_fwd_compress(pre, tau, None, st.bitmap, st.values, st.chunk_prefix,
                                                             st.nnz_out, ws, st.dev_status))
        nnz = st.nnz
        by = algorithmic_bytes("bt_relu_fwd_compress", n, nnz, 4)
        rows["tau=%g" % tau] = {"ms_median": round(ms, 4), "ms_best": round(best, 4),
                                "zero_fraction": round(1.0 - nnz / n, 4),
                                "stash_bytes_over_dense": round(B.bt_compressed_bytes(n, nnz, pre.dtype) / (4.0 * n), 4),
                                "moved_gbs": round(by / ms / 1e6, 1),
                                "frac_of_measured_copy": round(by / ms / 1e6 / peak_gbs, 3),
                                "frac_of_8000": round(by / ms / 1e6 / 8000.0, 3)}
    out["f32_2^28_bt_prune_fwd_compress_N(0,0.15)"] = rows
    del pre, st, ws
    torch.cuda.empty_cache()

    # max pooling with winner codes (a "next" row): the first pooling layer of a VGG-16 at batch 32
    rows = {}
    for label, dt in (("f32", torch.float32), ("bf16", torch.bfloat16)):
        x = torch.clamp_min(torch.randn(32, 64, 224, 224, device=dev, generator=torch.Generator(device=dev).manual_seed(900)),
                            0).to(dt)
        no, es = x.numel() // 4, x.element_size()
        y = torch.empty(32, 64, 112, 112, dtype=dt, device=dev)
        codes = torch.empty((no + 15) // 16, dtype=torch.int32, device=dev)
        gin = torch.empty_like(x)
        by = 5 * no * es + 4 * ((no + 15) // 16)
        pooled_bitmap = torch.randint(-2 ** 31, 2 ** 31 - 1, ((no + 31) // 32,), dtype=torch.int32, device=dev)
        for op, fn in (("bt_maxpool2x2_fwd", lambda: B.bt_maxpool2x2_fwd(x, y, codes)),
                       ("bt_maxpool2x2_bwd", lambda: B.bt_maxpool2x2_bwd(codes, y, gin)),
                       ("bt_maxpool2x2_bwd_masked", lambda: B.bt_maxpool2x2_bwd_masked(codes, pooled_bitmap, y, gin))):
            ms, best = time_call(fn)
            rows[label + "_" + op] = {"ms_median": round(ms, 4), "ms_best": round(best, 4), "moved_gbs": round(by / ms / 1e6, 1),
                                      "frac_of_measured_copy": round(by / ms / 1e6 / peak_gbs, 3),
                                      "frac_of_8000": round(by / ms / 1e6 / 8000.0, 3)}
        del x, y, codes, gin, pooled_bitmap
        torch.cuda.empty_cache()
    out["maxpool2x2_[32,64,224,224]"] = rows
    return out


# ------------------------------------------------------------------------------------------
def oracle_step(layers_np, indices):
    """The CPU oracle on the given layers, same four operations per layer; returns seconds."""
    from oracle import bt_oracle as O
    t0 = time.perf_counter()
    stashes = []
    for i in indices:
        act, pre, grad = layers_np[i]
        a = O.compress(act)
        _, b = O.relu_fwd_compress(pre, "f32", want_y=False)
        stashes.append((i, a, b))
    for i, a, b in reversed(stashes):
        O.decompress(a)
        O.relu_bwd_from_bitmap(b.bitmap, layers_np[i][2])
    return time.perf_counter() - t0


def host_layers(batch, indices):
    import torch
    from paper_2110_15362_b200 import workloads as W
    shapes = W.resnet18_shapes(batch)
    out = {}
    for i in indices:
        pre = W.cfg2_preact(i, shapes[i], "cpu")
        out[i] = (W.raw_numpy(torch.clamp_min(pre, 0.0)), W.raw_numpy(pre), W.raw_numpy(W.cfg2_grad(i, shapes[i], "cpu")))
    return out, shapes


def run_reference(args):
    """The oracle, as it stands, on host cores; each step is a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from paper_2110_15362_b200 import workloads as W
    sample = [1]                                                # one [B,64,56,56] layer per step
    layers, shapes = host_layers(args.batch, sample)
    elems = sum(W.numel(shapes[i]) for i in sample)
    for _ in range(min(args.warmup, 1)):
        oracle_step(layers, sample)
    t = [oracle_step(layers, sample) for _ in range(args.steps)]
    total = sum(t)
    value = len(OPS) * 4 * elems * args.steps / total / 1e9
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": min(args.warmup, 1), "ms_per_step": round(1e3 * total / args.steps, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "batch": args.batch,
                       "ops_per_layer": list(OPS)},
            "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": "layer 1 of 17 ([%d,64,56,56], %d elements) per step, all four operations; "
                                       "host has %d cores" % (args.batch, elems, os.cpu_count())},
            "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2110_15362_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the codec has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    B.lib()
    peak, peak_kind = measured_peak_gbs()

    step = Cfg2Step(dev, args.batch)
    if args.chains > 1:
        step.cta_budget = tuple(int(v) for v in args.cta_budget.split(","))
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        for _ in range(max(args.warmup, 3)):
            step.run()
    torch.cuda.synchronize()
    step.check()
    nnz = step.nnz()

    # the whole step as one CUDA graph: 68 kernel launches replayed without host work in between
    graph = torch.cuda.CUDAGraph()
    branches = [torch.cuda.Stream() for _ in range(args.chains - 1)]
    with torch.cuda.graph(graph):
        if args.chains > 1:
            main_stream = torch.cuda.current_stream()
            for b in branches:
                b.wait_stream(main_stream)               # fork
            step.run(streams=[main_stream] + branches)
            for b in branches:
                main_stream.wait_stream(b)               # join
        else:
            step.run()
    for _ in range(max(args.warmup, 3)):
        graph.replay()
    torch.cuda.synchronize()

    sampler = ClockSampler(local)
    sampler.start()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.time()
    e0.record()
    for _ in range(args.steps):
        graph.replay()
    e1.record()
    barrier()
    t1 = time.time()
    ms_total = e0.elapsed_time(e1)
    step.check()
    clocks = sampler.summary(t0, t1)

    # per-operation device time: one CUDA graph per operation, replayed between two events
    per_op, per_layer = per_kernel_pass(step, min(args.steps, 20), args.chains)

    # end to end: inputs start in pinned host memory, results end in host memory, every step
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(step, graph, min(args.steps, 10), world)
    sampler.stop()

    ms_total = max_over_ranks(ms_total, world, dev)
    if e2e is not None:
        e2e["ms"] = max_over_ranks(e2e["ms"], world, dev)

    if rank == 0:
        ms_step = ms_total / args.steps
        value = whole_job_value(step.dense_bytes_per_step, world, ms_step)
        # roofline of the dominant kernel class
        dom = max(per_op, key=lambda k: per_op[k]["ms"])
        alg = sum(algorithmic_bytes(dom, l["n"], z, 4) for l, z in zip(step.layers, nnz))
        launches = per_op[dom]["launches"]
        avg_ms = per_op[dom]["ms"] / launches
        achieved = (alg / len(step.layers)) / (avg_ms * 1e-3) / 1e9
        # the largest layer alone (98 MiB dense), the launch closest to the sizes the roofline bar is set for
        big_ms = statistics.median(per_layer[(dom, 0)])
        big_alg = algorithmic_bytes(dom, step.layers[0]["n"], nnz[0], 4)
        # all four operations together: the bytes the method must move in one step over the step's time
        step_alg = sum(algorithmic_bytes(op, l["n"], z, 4) for op in OPS for l, z in zip(step.layers, nnz))
        line = {
            "metric": METRIC, "value": round(value, 2), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": round(ms_step, 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": WORKLOAD, "batch": args.batch, "layers": len(step.layers),
                       "elements_per_step": step.total_elems, "zero_fraction": round(
                           1.0 - sum(nnz) / step.total_elems, 4),
                       "ops_per_layer": list(OPS),
                       "launch": "one CUDA graph per step" + (", %d independent chains on %d streams (plain codec / fused "
                                                              "pair%s)" % (args.chains, args.chains, ", even / odd layers" if args.chains == 4
                                                                           else ", layers by index mod 4" if args.chains == 8 else "")
                                                              if args.chains > 1 else ""),
                       "cta_budget": (("compress launches limited to %d CTAs (layers of at most 800 tiles) / %d CTAs "
                                       "(larger layers; 0 = one per SM) so that the chains' cooperative launches are "
                                       "resident side by side" % step.cta_budget) if len(step.cta_budget) == 2
                                      else "CTAs per compress launch by layer size: %s" % (step.cta_budget,))
                       if any(step.cta_budget) else "one CTA per SM",
                       "l2": "per-step working set %.2f GB exceeds the 126 MB L2; no flush between steps"
                             % (7 * 4 * step.total_elems / 1e9),
                       "parallelism": "dp%d" % world if world > 1 else "single"},
            "clocks": clocks,
            "gpu_launches": step.launches_per_step * args.steps,
            "roofline": {"bound": "hbm", "kernel": dom, "achieved": round(achieved, 1), "peak": peak,
                         "unit": "GB/s", "frac": round(achieved / peak, 4), "peak_kind": peak_kind,
                         "traffic": NCU_TRAFFIC_PER_LAUNCH.get(dom),
                         "algorithmic_bytes_per_launch": round(alg / len(step.layers)),
                         "avg_launch_ms": round(avg_ms, 5), "launches_timed": launches,
                         "largest_layer": {"elements": step.layers[0]["n"], "ms": round(big_ms, 5),
                                           "achieved": round(big_alg / big_ms / 1e6, 1),
                                           "frac": round(big_alg / big_ms / 1e6 / peak, 4)},
                         "per_op_ms_per_step": {k: round(v["ms"] / max(1, v["launches"]) * len(step.layers), 5)
                                                for k, v in per_op.items()},
                         "whole_step": {"algorithmic_bytes": step_alg,
                                        "achieved": round(step_alg / (ms_step * 1e-3) / 1e9, 1),
                                        "frac": round(step_alg / (ms_step * 1e-3) / 1e9 / peak, 4)},
                         "how": "avg_launch_ms = time of the step's launches of this operation, in the step's launch "
                                "configuration (its own chains on their streams, the CTA budget), over their "
                                "number; largest_layer = one launch alone, one CTA per SM, L2 flushed"},
        }
        if e2e is not None:
            e2e_ms = e2e["ms"] / e2e["steps"]
            line["e2e"] = {"value": round(whole_job_value(step.dense_bytes_per_step, world, e2e_ms), 3),
                           "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                           "ms_per_step": round(e2e_ms, 3), "steps": e2e["steps"],
                           "api": "bt_*_host entry points, pinned host buffers, %d host threads" % e2e["workers"]}
        if world == 1 and not args.no_large:
            line["large_tensor_kernels"] = large_tensor_kernels(dev, peak)
        if world == 1 and not args.no_cpu_baseline:
            idx = list(range(len(step.layers)))
            layers, _ = host_layers(args.batch, idx)
            secs = oracle_step(layers, idx)
            line["cpu_baseline"] = {"value": round(step.dense_bytes_per_step / secs / 1e9, 4), "unit": UNIT,
                                    "cores": 1, "kind": "oracle",
                                    "sample": "one full step (17 layers, %d elements, four operations each), "
                                              "single thread; host has %d cores" % (step.total_elems, os.cpu_count()),
                                    "seconds": round(secs, 2)}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_e2e(step: Cfg2Step, graph, steps: int, world: int, workers: int = int(os.environ.get("BT_E2E_WORKERS", "4"))):
    """The same step through the host-buffer entry points of the C ABI: every tensor the step consumes
    starts in pinned host memory and every tensor it produces (both stashes, the restored activation, the
    input gradient) ends there; the host<->device copies happen inside the calls, inside the timed region.

    The calls are synchronous, so a few host threads (each with its own stream, staging area and output
    buffers) work on different layers at once: one call's host->device copy overlaps another's
    device->host copy and kernels.  All forward calls of a step finish before its backward calls start."""
    import queue
    from concurrent.futures import ThreadPoolExecutor
    import torch
    B = step.B
    dev = step.restored.device
    n_max = step.restored.numel()
    host = []
    h2d = d2h = 0
    for l in step.layers:
        n = l["n"]
        h = dict(act=l["act"].cpu().pin_memory(), pre=l["pre"].cpu().pin_memory(), grad=l["grad"].cpu().pin_memory())
        for tag in ("a", "b"):
            h["bitmap_" + tag] = torch.empty((n + 31) // 32, dtype=torch.int32).pin_memory()
            h["values_" + tag] = torch.empty(n, dtype=torch.float32).pin_memory()
            h["prefix_" + tag] = torch.empty((n + 4095) // 4096, dtype=torch.int64).pin_memory()
            h["nnz_" + tag] = torch.zeros(1, dtype=torch.int64).pin_memory()
        host.append(h)
    for l, z in zip(step.layers, step.nnz()):
        n = l["n"]
        comp = B.bt_compressed_bytes(n, z, torch.float32)
        h2d += 4 * n + 4 * n + comp + (4 * ((n + 31) // 32) + 4 * n)      # compress, fused forward, decompress, backward
        d2h += (comp + 8) + (comp + 8) + 4 * n + 4 * n

    # per-thread resources, handed out through a queue
    pool = queue.SimpleQueue()
    for _ in range(workers):
        pool.put(dict(stream=torch.cuda.Stream(device=dev),
                      staging=torch.empty(B.bt_host_staging_bytes(n_max, torch.float32), dtype=torch.uint8, device=dev),
                      restored=torch.empty(n_max, dtype=torch.float32).pin_memory(),
                      gin=torch.empty(n_max, dtype=torch.float32).pin_memory()))
    check = {}

    def call(task):
        kind, i = task
        r = pool.get()
        try:
            torch.cuda.set_device(dev)
            h, s, n = host[i], r["stream"], step.layers[i]["n"]
            if kind == "compress":
                B.bt_compress_host(h["act"], h["bitmap_a"], h["values_a"], h["prefix_a"], h["nnz_a"], r["staging"], stream=s)
            elif kind == "fused":
                B.bt_relu_fwd_compress_host(h["pre"], None, h["bitmap_b"], h["values_b"], h["prefix_b"], h["nnz_b"],
                                            r["staging"], stream=s)
            elif kind == "decompress":
                B.bt_decompress_host(h["bitmap_a"], h["values_a"], h["prefix_a"], int(h["nnz_a"].item()),
                                     r["restored"][:n], r["staging"], stream=s)
                if i == 0:
                    check["ok"] = torch.equal(r["restored"][:n].view(torch.int32), h["act"].view(torch.int32))
            else:
                B.bt_relu_bwd_from_bitmap_host(h["bitmap_b"], h["grad"], r["gin"][:n], r["staging"], stream=s)
        finally:
            pool.put(r)

    order = sorted(range(len(step.layers)), key=lambda i: -step.layers[i]["n"])     # large layers first
    fwd = [(k, i) for i in order for k in ("compress", "fused")]
    bwd = [(k, i) for i in order for k in ("decompress", "backward")]
    with ThreadPoolExecutor(max_workers=workers) as ex:
        def one():
            list(ex.map(call, fwd))
            list(ex.map(call, bwd))
        one()
        torch.cuda.synchronize()
        assert check.get("ok"), "end-to-end round trip is not bit exact"
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            one()
        # every call has synchronised its own stream before returning; the closing event follows them all
        e1.record()
        torch.cuda.synchronize()
    return {"ms": e0.elapsed_time(e1), "steps": steps, "h2d": h2d, "d2h": d2h, "workers": workers}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
