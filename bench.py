#!/usr/bin/env python
"""Benchmark of the BOF4 hot path on B200.

One *step* is one pass of the whole path over the largest single-GPU workloads, every component
called through the C ABI (the ctypes binding) with device-resident inputs:

    EM iteration, MSE        one bof4_fit_codebook(iters=1) over the 224 Llama-7B-shaped matrices
    EM iteration, MAE        the same with the weighted-median centroid        (12.95 GB, bf16)
    quantise                 bof4_quantize_batch   of the 224 Llama-3-8B-shaped matrices (13.96 GB)
    dequantise               bof4_dequantize_batch of the same set, back to bf16
    OPQ quantise             bof4_quantize_opq  of one Llama-70B-shaped layer      (1.71 GB)
    OPQ dequantise           bof4_dequantize with outlier write-back of that layer

Every component streams inputs far larger than L2 (126 MB), so no flush is needed between
components.  Each component is captured once into a CUDA graph (the same binding calls, on the
capturing stream) so that its several hundred launches are not limited by Python call overhead;
the graphs are replayed and timed with CUDA events.  Prints ONE JSON line.

`--impl reference` times the CPU oracle (test infrastructure, never tuned) on the host cores
with the same metric, each step on a bounded sample of the same workloads.
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

import numpy as np
import torch

import workloads

I = 64
Q = 0.95
WORKLOAD = ("EM iteration (MSE, MAE; BOF4-S, block 64) over 32 layers x {4 x 4096x4096, 3 x 4096x11008} bf16 "
            "(sigma ~ U[0.01,0.04] per matrix); quantize + dequantize over 32 layers x {4096x4096, 1024x4096 x2, "
            "4096x4096, 14336x4096 x2, 4096x14336} bf16 N(0,0.02^2); OPQ quantize + dequantize of one layer "
            "{8192x8192, 1024x8192 x2, 8192x8192, 28672x8192 x2, 8192x28672} bf16 N(0,0.015^2) + 0.01% outliers")
METRIC = ("hot-path Gweights/s (weights passed through a component per second, summed over the step's "
          "components); components: EM-iteration Gweights/s and quant/dequant HBM GB/s")
# algorithmic bytes per weight of each component (bf16 in, block 64)
BYTES_EM = 2.0
BYTES_QUANT = 2.0 + 0.5 + 2.0 / I
BYTES_DEQUANT = 0.5 + 2.0 / I + 2.0
BYTES_GEMV = 0.5 + 2.0 / I            # 4-bit codes + bf16 block constants; x and y are negligible
# data passes of one MAE iteration that carry the selection (the max-|w| pass of the call, which
# exists only for the fixed-point sample weights, is not counted as algorithmic work)
MAE_SELECTION_PASSES = 2
FALLBACK_HBM_GBS = 6650.0
OPQ_OUTLIER_FRACTION = 2.2e-3         # list capacity n / 64 leaves a 7x margin over the expected rate

# dram__bytes_read.sum + dram__bytes_write.sum per weight of the dominant component's kernels,
# from the committed ncu captures (profiles/), taken on a two-layer slice and scaled by the number
# of weights (traffic is proportional to it); None once the kernels have changed since.
TRAFFIC_PER_WEIGHT = {
    # max-|w| pass 812.9 MB + first pass 813.9 MB + collecting pass 839.0 MB (candidate lists written:
    # 13.1 MB of it) + two empty passes 0.14 MB + the candidate lists read once more by the resolve
    # kernel (at most the 13.1 MB written) over 404,750,336 weights (profiles/mae_*_c3_2layer_slice.md)
    "em_mae": (812913664 + 813880064 + 839011328 + 140544 + 13076224) / 404750336.0,
    "em_mse": (810906368 + 4438272) / 404750336.0,      # profiles/em_mse32_kernel_c3_2layer_slice.md
}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# --------------------------------------------------------------------------- clocks


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if vis:
                try:
                    phys = int(vis.split(",")[index])
                except Exception:
                    phys = index
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "sw_power_cap": 0x4, "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self.nv is not None:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()

    def stop(self):
        self._stop.set()
        if self._thr is not None:
            self._thr.join()
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------- workloads on the device


def fit_set(dev, seed_offset=0, layers=32):
    """The Llama-7B-shaped set of the fitting sweep (per-matrix sigma), generated on `dev`."""
    sig = workloads.config3_sigmas()
    out = []
    for i, (r, c) in enumerate(workloads.llama7b_shapes()[: layers * 7]):
        out.append(workloads.gaussian(r * c, sig[i], 2_000_000 + 1000 * seed_offset + i, torch.bfloat16, dev))
    return out


def quant_set(dev, seed_offset=0, layers=32):
    """The Llama-3-8B-shaped set of the quantise / dequantise throughput run."""
    return [workloads.gaussian(r * c, 0.02, 3_000_000 + 1000 * seed_offset + i, torch.bfloat16, dev)
            for i, (r, c) in enumerate(workloads.llama3_8b_shapes()[: layers * 7])]


def opq_layer(dev, seed_offset=0, layer=0):
    """One Llama-70B-shaped layer with injected outliers."""
    return workloads.config5_layer(layer + 80 * seed_offset, device=dev)


class Step:
    """Device buffers and the component calls of one step."""

    def __init__(self, bof4, dev, seed_offset: int = 0, layers: int = 32, sets=None):
        b = self.b = bof4
        self.dev = dev
        if sets is None:
            sets = (fit_set(dev, seed_offset, layers), quant_set(dev, seed_offset, layers),
                    opq_layer(dev, seed_offset))
        self.w_fit, self.w_q, self.w_opq = sets
        self.n_fit = sum(w.numel() for w in self.w_fit)
        self.n_q = sum(w.numel() for w in self.w_q)
        self.n_opq = sum(w.numel() for w in self.w_opq)
        self.lv0, self.mask = b.bof4_default_init(b.NORM_SIGNED)
        self.cb0 = torch.tensor(self.lv0, device=dev)
        # levels the quantiser uses: the printed BOF4-S (MSE) codebook for block size 64 (Tab. 6)
        self.cb_q = torch.tensor(np.array(workloads.BOF4S_MSE_I64, np.float32), device=dev)
        self.tau = float(np.float32(b.bof4_opq_threshold(Q, I)))
        nmax = max(max(w.numel() for w in s) for s in sets)
        self.ws_em = torch.empty(b.bof4_workspace_bytes(b.OP_EM, self.n_fit, I, b.METRIC_MAE), dtype=torch.uint8, device=dev)
        self.ws_opq = torch.empty(b.bof4_workspace_bytes(b.OP_OPQ, nmax, I, 0), dtype=torch.uint8, device=dev)
        u8, bf = torch.uint8, torch.bfloat16
        self.q_out = [(torch.empty(w.numel() // 2, dtype=u8, device=dev),
                       torch.empty(w.numel() // I, dtype=bf, device=dev)) for w in self.w_q]
        self.q_deq = [torch.empty(w.numel(), dtype=bf, device=dev) for w in self.w_q]
        self.o_out = []
        for w in self.w_opq:
            n, cap = w.numel(), w.numel() // 64
            self.o_out.append((torch.empty(n // 2, dtype=u8, device=dev), torch.empty(n // I, dtype=bf, device=dev),
                               torch.empty(cap, dtype=torch.int32, device=dev), torch.empty(cap, dtype=bf, device=dev),
                               torch.zeros(1, dtype=torch.int64, device=dev)))
        self.o_deq = [torch.empty(w.numel(), dtype=bf, device=dev) for w in self.w_opq]
        # result buffers of the two fits (levels, error log): no allocation inside the timed region
        self.fit_out = [(self.cb0.clone(), torch.zeros(1, dtype=torch.float64, device=dev)) for _ in range(2)]
        self.only = None
        self.graphs = {}

    # ---- the six components (binding calls only).  The two fits continue from their own previous
    # result (the levels buffer is both input and output), so that successive steps are successive
    # Lloyd iterations of one fit, as in a 30-iteration run, rather than the first iteration over
    # and over.
    def em_mse(self):
        b = self.b
        b.bof4_fit_codebook(self.w_fit, I, b.NORM_SIGNED, b.METRIC_MSE, self.fit_out[0][0], self.mask, 1,
                            workspace=self.ws_em, sync=False, out=self.fit_out[0])

    def em_mae(self):
        b = self.b
        b.bof4_fit_codebook(self.w_fit, I, b.NORM_SIGNED, b.METRIC_MAE, self.fit_out[1][0], self.mask, 1,
                            workspace=self.ws_em, sync=False, out=self.fit_out[1])

    def quant(self):
        b = self.b
        b.bof4_quantize_batch(self.w_q, I, b.NORM_SIGNED, self.cb_q,
                              out=([c for c, _ in self.q_out], [s for _, s in self.q_out]))

    def dequant(self):
        b = self.b
        b.bof4_dequantize_batch([c for c, _ in self.q_out], [s for _, s in self.q_out],
                                [w.numel() for w in self.w_q], I, self.cb_q, b.BF16, out=self.q_deq)

    def opq_quant(self):
        b = self.b
        for w, out in zip(self.w_opq, self.o_out):
            b.bof4_quantize_opq(w, I, b.NORM_SIGNED, self.cb_q, self.tau, out[2].numel(), workspace=self.ws_opq, out=out)

    def opq_dequant(self):
        b = self.b
        for (codes, scales, idx, val, cnt), out in zip(self.o_out, self.o_deq):
            b.bof4_dequantize(codes, scales, I, self.cb_q, b.BF16, (idx, val, cnt), out=out)

    # ---- consumers of the quantised matrix (profiling runs, `--only gemv,gemm_tc`): the two
    # 28672 x 8192 matrices of the OPQ layer in turn (235 MB of codes, larger than L2)
    def consumer_setup(self):
        if hasattr(self, "cons"):
            return
        b = self.b
        self.cons = []
        for w in self.w_opq[4:6]:
            codes, scales = b.bof4_quantize(w, I, b.NORM_SIGNED, self.cb_q)
            self.cons.append((codes, scales, 28672, 8192))
        self.cons_x = workloads.gaussian(64 * 8192, 1.0, 77, torch.bfloat16, self.dev).reshape(64, 8192)
        self.cons_y = torch.empty(28672, dtype=torch.float32, device=self.dev)
        self.cons_ws = torch.empty(8 * 28672 * 64 * 4, dtype=torch.uint8, device=self.dev)

    def gemv(self):
        b = self.b
        for codes, scales, r, c in self.cons:
            b.bof4_gemv(codes, scales, r, c, I, self.cb_q, self.cons_x[0], out=self.cons_y)

    def gemm_tc(self):
        b = self.b
        for codes, scales, r, c in self.cons:
            b.bof4_gemm_tc(codes, scales, r, c, I, self.cb_q, self.cons_x, workspace=self.cons_ws)

    def components(self):
        """(name, call, weights per call, algorithmic bytes per weight, kernels launched per call)"""
        b = self.b.binding
        nt, nq, no = len(self.w_fit), len(self.w_q), len(self.w_opq)
        if self.only and (self.only & {"gemv", "gemm_tc"}):
            self.consumer_setup()
            nc = 2 * 28672 * 8192
            extra = [("gemv", self.gemv, nc, BYTES_GEMV, 2), ("gemm_tc", self.gemm_tc, nc, BYTES_GEMV, 2)]
            return [c for c in extra if c[0] in self.only]
        comps = [("em_mse", self.em_mse, self.n_fit, BYTES_EM, b.mse_launches_per_iteration(nt)),
                 ("em_mae", self.em_mae, self.n_fit, BYTES_EM * MAE_SELECTION_PASSES,
                  b.mae_launches_per_call(nt, self.n_fit, 1)),
                 ("quantize", self.quant, self.n_q, BYTES_QUANT, -(-nq // b.TENSORS_PER_LAUNCH)),
                 ("dequantize", self.dequant, self.n_q, BYTES_DEQUANT, -(-nq // b.TENSORS_PER_LAUNCH)),
                 ("opq_quantize", self.opq_quant, self.n_opq, BYTES_QUANT + 6 * OPQ_OUTLIER_FRACTION / 2.2, 2 * no),
                 ("opq_dequantize", self.opq_dequant, self.n_opq, BYTES_DEQUANT + 6 * OPQ_OUTLIER_FRACTION / 2.2, 2 * no)]
        if self.only:
            comps = [c for c in comps if c[0] in self.only]
        return comps

    def capture(self):
        """Captures every component into its own CUDA graph (after it has run once eagerly, so that
        one-time set-up such as shared-memory attributes is done before the capture)."""
        for name, fn, *_ in self.components():
            fn()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                fn()
            self.graphs[name] = g

    def run_timed(self):
        """One step; returns {component: (start, end)} CUDA events on the current stream."""
        times = {}
        for name, fn, *_ in self.components():
            s = torch.cuda.Event(enable_timing=True)
            e = torch.cuda.Event(enable_timing=True)
            s.record()
            g = self.graphs.get(name)
            if g is not None:
                g.replay()
            else:
                fn()
            e.record()
            times[name] = (s, e)
        return times


def rank_env():
    """(rank, local_rank, world_size) as the launcher exports them (1 process per GPU)."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def workload_seed_offset(rank: int) -> int:
    """Every rank works on its own, independent problem: the path shards by blocks and needs
    no exchange, so the ranks' workloads differ only by their seed."""
    return rank


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a group)."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_gweights_per_s(world: int, n_per_rank: int, ms_per_step: float) -> float:
    """All ranks' weights per step over the slowest rank's step time."""
    return world * n_per_rank / ms_per_step / 1e6


# --------------------------------------------------------------------------- end to end (host buffers)


class E2E:
    """The same component calls fed from pinned host memory and read back to it, on a bounded slice
    of the step's workloads (the first `layers` layers of the two 32-layer sets and the whole OPQ
    layer), two slices in flight on two streams so that one upload overlaps the other download.
    quantize_only: weights up, quantise / OPQ quantise, codes + scales + outlier lists down."""

    def __init__(self, bof4, dev, full: Step, layers: int, quantize_only: bool):
        self.quantize_only = quantize_only
        k = layers * 7
        sets = (full.w_fit[:k], full.w_q[:k], full.w_opq)
        self.used = (1, 2) if quantize_only else (0, 1, 2)     # which sets travel
        self.host_in = [[w.cpu().pin_memory() for w in s] if i in self.used else [] for i, s in enumerate(sets)]
        self.slots = []
        for _ in range(2):
            dsets = tuple([torch.empty_like(w) for w in s] if i in self.used else s for i, s in enumerate(sets))
            st = Step(bof4, dev, sets=dsets)
            outs = [t for pair in st.q_out for t in pair] + [t for o in st.o_out for t in o]
            if not quantize_only:
                outs += [st.fit_out[0][0], st.fit_out[0][1], st.fit_out[1][0], st.fit_out[1][1]]
                outs += st.q_deq + st.o_deq
            host_out = [torch.empty_like(t, device="cpu").pin_memory() for t in outs]
            self.slots.append((st, dsets, outs, host_out))
        st = self.slots[0][0]
        self.weights_per_step = (st.n_q + st.n_opq) if quantize_only else 2 * (st.n_fit + st.n_q + st.n_opq)
        self.h2d = sum(w.numel() * 2 for i in self.used for w in sets[i])
        self.d2h = sum(t.numel() * t.element_size() for t in self.slots[0][3])

    def one(self, slot):
        st, dsets, outs, host_out = self.slots[slot]
        for i in self.used:
            for h, d in zip(self.host_in[i], dsets[i]):
                d.copy_(h, non_blocking=True)
        if self.quantize_only:
            st.quant()
            st.opq_quant()
        else:
            for _, fn, *_ in st.components():
                fn()
        for d, h in zip(outs, host_out):
            h.copy_(d, non_blocking=True)

    def run(self, count, streams):
        main = torch.cuda.current_stream()
        for sm in streams:
            sm.wait_stream(main)
        for i in range(count):
            with torch.cuda.stream(streams[i & 1]):
                self.one(i & 1)
        for sm in streams:
            main.wait_stream(sm)


def time_e2e(e2e: E2E, steps: int, dist, dev):
    streams = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]
    e2e.run(2, streams)
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    s = torch.cuda.Event(enable_timing=True)
    e = torch.cuda.Event(enable_timing=True)
    s.record()
    e2e.run(steps, streams)
    e.record()
    torch.cuda.synchronize()
    return s.elapsed_time(e)


# --------------------------------------------------------------------------- GPU arm


def run_gpu(args):
    rank, local, world = rank_env()
    import __graft_entry__ as entry
    if local == 0:
        entry.build()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the hot path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1 or "TORCHELASTIC_RUN_ID" in os.environ:  # launched by torch.distributed.run
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()
    import paper_2505_06653_b200 as bof4
    from paper_2505_06653_b200 import binding
    binding.lib()

    st = Step(bof4, dev, seed_offset=workload_seed_offset(rank), layers=args.layers)  # no data-path collective
    if args.only:
        st.only = set(args.only.split(","))
        args.no_e2e = args.no_cpu_baseline = True
    K, W = args.steps, args.warmup
    if not args.no_graphs:
        st.capture()
    for _ in range(W):
        st.run_timed()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    sampler = ClockSampler(local)
    sampler.start()
    torch.cuda.synchronize()
    recs = [st.run_timed() for _ in range(K)]
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    comp_ms = {name: [s.elapsed_time(e) for s, e in (r[name] for r in recs)] for name in recs[0]}
    total_ms = sum(sum(v) for v in comp_ms.values())
    clocks = sampler.stop()

    # one 30-iteration MAE and MSE fit per call, as the fitting sweep runs them: the per-call
    # max-|w| pass of the MAE fit is then shared by 30 iterations (reported beside the step)
    fit30 = {}
    if not args.only:
        b = bof4
        for name, metric in (("mse", b.METRIC_MSE), ("mae", b.METRIC_MAE)):
            log = torch.zeros(30, dtype=torch.float64, device=dev)
            cb = torch.empty(16, dtype=torch.float32, device=dev)
            s = torch.cuda.Event(enable_timing=True)
            e = torch.cuda.Event(enable_timing=True)
            s.record()
            b.bof4_fit_codebook(st.w_fit, I, b.NORM_SIGNED, metric, st.cb0, st.mask, 30, workspace=st.ws_em,
                                sync=False, out=(cb, log))
            e.record()
            torch.cuda.synchronize()
            fit30[name] = s.elapsed_time(e) / 30.0

    # ---- end to end: pinned host buffers in and out, through the same calls
    e2e_ms = e2eq_ms = 0.0
    Ke = 0 if args.no_e2e else 3
    e2e = e2eq = None
    if Ke:
        el = min(args.e2e_layers, args.layers)
        e2e = E2E(bof4, dev, st, el, quantize_only=False)
        e2e_ms = time_e2e(e2e, Ke, dist, dev)
        del e2e.slots
        e2eq = E2E(bof4, dev, st, el, quantize_only=True)
        e2eq_ms = time_e2e(e2eq, Ke, dist, dev)
        del e2eq.slots

    total_ms, e2e_ms, e2eq_ms = max_over_ranks([total_ms, e2e_ms, e2eq_ms], dist, dev)
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms / K
    peak, peak_kind = measured_peak()
    avg = {k: sum(v) / len(v) for k, v in comp_ms.items()}
    comp, launches, weights_per_step = {}, 0, 0
    info = {c[0]: c for c in st.components()}
    for name, ms in avg.items():
        _, _, n, bpw, nk = info[name]
        comp[name + "_ms"] = ms
        comp[name + "_gweights_s"] = n / ms / 1e6
        comp[name + "_gbs"] = bpw * n / ms / 1e6
        comp[name + "_frac_of_%s_hbm" % peak_kind] = bpw * n / ms / 1e6 / peak
        launches += nk
        weights_per_step += n
    if fit30:
        comp["em_mse_ms_per_iteration_in_a_30_iteration_fit"] = fit30["mse"]
        comp["em_mae_ms_per_iteration_in_a_30_iteration_fit"] = fit30["mae"]
        comp["em_mae_gbs_in_a_30_iteration_fit"] = BYTES_EM * MAE_SELECTION_PASSES * st.n_fit / fit30["mae"] / 1e6
    # dominant component = the one with the largest share of the step
    dom = max(avg, key=avg.get)
    _, _, dn, dbpw, _ = info[dom]
    achieved = dbpw * dn / avg[dom] / 1e6
    tpw = TRAFFIC_PER_WEIGHT.get(dom)
    line = {
        "metric": METRIC, "value": whole_job_gweights_per_s(world, weights_per_step, ms_per_step),
        "unit": "Gweights/s", "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "layers": args.layers,
                   "weights_per_gpu": {"fit_set": st.n_fit, "quantize_set": st.n_q, "opq_layer": st.n_opq},
                   "weight_passes_per_step": weights_per_step, "block_size": I, "opq_q": Q,
                   "l2": "inputs larger than L2 (12.95 GB / 13.96 GB / 1.71 GB per component): no flush",
                   "launch": "one CUDA graph per component" if not args.no_graphs else "eager binding calls",
                   "multi_gpu": "independent problem per rank, no collective",
                   "e2e": "first %d layers of the two 32-layer sets and the whole OPQ layer from pinned host memory, "
                          "all results (incl. dequantised tensors) back; two slices in flight on two streams"
                          % min(args.e2e_layers, args.layers)},
        "components": comp,
        "clocks": clocks,
        "e2e": {"value": (world * e2e.weights_per_step * Ke / e2e_ms / 1e6) if Ke else None, "unit": "Gweights/s",
                "h2d_bytes_per_step": e2e.h2d if Ke else 0, "d2h_bytes_per_step": e2e.d2h if Ke else 0, "steps": Ke},
        "e2e_quantize_only": {"value": (world * e2eq.weights_per_step * Ke / e2eq_ms / 1e6) if Ke else None,
                              "unit": "Gweights/s", "h2d_bytes_per_step": e2eq.h2d if Ke else 0,
                              "d2h_bytes_per_step": e2eq.d2h if Ke else 0, "steps": Ke,
                              "what": "weights up, quantise / OPQ quantise, codes + scales + outlier lists down"},
        "gpu_launches": launches * K,
        "roofline": {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": (tpw * dn) if tpw else None},
    }
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline()
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


# --------------------------------------------------------------------------- CPU arm (oracle)


def oracle_sample(rows: int = 256):
    """A bounded sample of the step's workloads for the CPU legs: the first matrix of each set
    cut to its first `rows` rows (CPU generator, same recipe)."""
    sig = workloads.config3_sigmas()
    r, c = workloads.llama7b_shapes()[0]
    fit = workloads.gaussian(min(rows, r) * c, sig[0], 2_000_000, torch.bfloat16)
    r, c = workloads.llama3_8b_shapes()[0]
    qs = workloads.gaussian(min(rows, r) * c, 0.02, 3_000_000, torch.bfloat16)
    r, c = workloads.llama70b_layer_shapes()[0]
    op = workloads.inject_outliers(workloads.gaussian(min(rows // 2, r) * c, 0.015, 4_000_000, torch.bfloat16),
                                   0.015, 1e-4, 10.0, 40.0, 4_000_008)
    return fit, qs, op


def oracle_step(oracle, sample, lv0, lvq, mask, tau):
    """The same six components computed by the CPU oracle on fp32-widened weights; returns the
    number of weight passes."""
    fit, qs, op = sample
    oracle.fit(fit, I, oracle.NORM_SIGNED, oracle.METRIC_MSE, lv0, mask, 1)
    oracle.fit(fit, I, oracle.NORM_SIGNED, oracle.METRIC_MAE, lv0, mask, 1)
    codes, scales = oracle.quantize(qs, I, oracle.NORM_SIGNED, lvq)
    oracle.dequantize(codes, scales, I, lvq)
    clean, idx, val, k = oracle.opq_split(op, I, tau)
    codes, scales = oracle.quantize(clean, I, oracle.NORM_SIGNED, lvq)
    out = oracle.dequantize(codes, scales, I, lvq)
    oracle.opq_restore(out, idx, val)
    return 2 * (fit.size + qs.size + op.size)


def _oracle_setup(rows):
    import oracle
    oracle.build()
    sample = tuple(oracle.as_f32(t) for t in oracle_sample(rows))
    lv0 = np.array(workloads.init_levels_7_0_8(), np.float32)
    lvq = np.array(workloads.BOF4S_MSE_I64, np.float32)
    tau = float(np.float32(oracle.opq_threshold(Q, I)))
    return oracle, sample, lv0, lvq, tau


def omp_set_threads(n: int):
    """Thread count of the OpenMP runtime the oracle's library is linked against (the oracle itself
    is left as it stands)."""
    import ctypes
    ctypes.CDLL("libgomp.so.1").omp_set_num_threads(int(n))


def cpu_baseline(rows: int = 1024, reps: int = 2):
    """The oracle on all host cores, and on one core, on a bounded sample of the step."""
    oracle, sample, lv0, lvq, tau = _oracle_setup(rows)
    t0 = time.time()
    for _ in range(reps):
        passes = oracle_step(oracle, sample, lv0, lvq, workloads.FIXED_BOF4S, tau)
    dt = (time.time() - t0) / reps
    out = {"value": passes / dt / 1e9, "unit": "Gweights/s", "cores": oracle.n_threads(), "kind": "oracle",
           "sample": "first %d rows of the first matrix of each of the three sets (%.1e weight passes per step), "
                     "%d steps" % (rows, passes, reps)}
    # single-threaded, on a quarter of that sample
    _, small, _, _, _ = _oracle_setup(rows // 4)
    all_cores = oracle.n_threads()
    omp_set_threads(1)
    t0 = time.time()
    p1 = oracle_step(oracle, small, lv0, lvq, workloads.FIXED_BOF4S, tau)
    dt1 = time.time() - t0
    omp_set_threads(all_cores)
    out["single_thread"] = {"value": p1 / dt1 / 1e9, "unit": "Gweights/s", "cores": 1,
                            "sample": "first %d rows, 1 step" % (rows // 4)}
    return out


def run_reference(args):
    rank = rank_env()[0]
    if rank != 0:
        return None
    rows = 512
    oracle, sample, lv0, lvq, tau = _oracle_setup(rows)
    for _ in range(args.warmup):
        oracle_step(oracle, sample, lv0, lvq, workloads.FIXED_BOF4S, tau)
    t0 = time.time()
    passes = 0
    for _ in range(args.steps):
        passes += oracle_step(oracle, sample, lv0, lvq, workloads.FIXED_BOF4S, tau)
    dt = time.time() - t0
    val = passes / dt / 1e9
    what = "first %d rows of the first matrix of each of the three sets per step" % rows
    desc = {"value": val, "unit": "Gweights/s", "cores": oracle.n_threads(), "kind": "oracle", "sample": what}
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "Gweights/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / max(args.steps, 1) * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": what, "weight_passes_per_step": passes // max(args.steps, 1),
                   "block_size": I, "opq_q": Q},
        "cpu_baseline": desc,
        "e2e": {"value": val, "unit": "Gweights/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer legs (profiling runs)")
    ap.add_argument("--no-graphs", action="store_true", help="call the binding eagerly instead of replaying graphs")
    ap.add_argument("--layers", type=int, default=32, help="layers of the two 32-layer sets (fewer: profiling "
                    "runs on a slice; the JSON line is then not a bench result)")
    ap.add_argument("--e2e-layers", type=int, default=4, help="layers of the 32-layer sets in the host-buffer legs")
    ap.add_argument("--only", default="", help="comma list of components to run (profiling runs only; "
                    "the JSON line is then not a bench result)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.impl == "reference":
        run_reference(args)
    else:
        if args.warmup < 3:
            args.warmup = 3
        run_gpu(args)


if __name__ == "__main__":
    main()
