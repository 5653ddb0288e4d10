#!/usr/bin/env python
"""Benchmark of the BOF4 hot path on B200.

One *step* is one pass of the whole path over one batch of synthetic weights (the BOF4-S
workload: 2^26 bf16 weights, 99 % N(0, 0.02^2) + 1 % heavy-tailed, block size 64):
    EM iteration (MSE)  ->  EM iteration (MAE)  ->  OPQ split + quantise  ->  dequantise with
    outlier write-back,
every component called through the C ABI with device-resident inputs.  L2 is flushed before
every component (a 256 MiB write), so each one streams its inputs from HBM; the step time is
the sum of the components' CUDA-event times.  Prints ONE JSON line.

`--impl reference` times the CPU oracle (test infrastructure, never tuned) on the host cores
with the same metric, each step on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
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
N_WEIGHTS = workloads.C2_N
WORKLOAD = "BOF4-S: 2^26 bf16 weights, 99% N(0,0.02^2) + 1% 0.02*t(nu=4), block 64, signed absmax"
METRIC = ("hot-path step Gweights/s (EM iteration MSE + MAE, OPQ quantize, dequantize); "
          "components: EM-iteration Gweights/s and quant/dequant HBM GB/s")
# algorithmic bytes per weight of each component (bf16 in, block 64)
BYTES_EM = 2.0
BYTES_QUANT = 2.0 + 0.5 + 2.0 / I
BYTES_DEQUANT = 0.5 + 2.0 / I + 2.0
BYTES_GEMV = 0.5 + 2.0 / I            # 4-bit codes + bf16 block constants; x and y are negligible
# data passes of one MAE iteration that stream all weights on this workload: the max-|w| pass
# and two selection passes (the rest of the selection runs on the candidate lists)
MAE_DATA_PASSES = 3
FALLBACK_HBM_GBS = 6650.0


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


# --------------------------------------------------------------------------- GPU arm


class Step:
    """Device buffers and the component calls of one step."""

    # kernels launched by each component (accumulate + finalise; selection passes; ...)
    def __init__(self, bof4, dev, seed_offset: int = 0, w_host=None):
        self.b = bof4
        self.dev = dev
        n = N_WEIGHTS
        self.n = n
        self.w_host = w_host if w_host is not None else workloads.gaussian_student_mixture(
            n, 0.02, 0.01, 4, 1 + seed_offset, torch.bfloat16).pin_memory()
        self.w = self.w_host.to(dev)
        self.lv0, self.mask = bof4.bof4_default_init(bof4.NORM_SIGNED)
        self.cb0 = torch.tensor(self.lv0, device=dev)
        self.tau = float(np.float32(bof4.bof4_opq_threshold(Q, I)))
        self.cap = n // 64
        self.ws_em = torch.empty(bof4.bof4_workspace_bytes(bof4.OP_EM, n, I, bof4.METRIC_MAE),
                                 dtype=torch.uint8, device=dev)
        self.ws_opq = torch.empty(bof4.bof4_workspace_bytes(bof4.OP_OPQ, n, I, 0), dtype=torch.uint8,
                                  device=dev)
        self.codes = torch.empty(n // 2, dtype=torch.uint8, device=dev)
        self.scales = torch.empty(n // I, dtype=torch.bfloat16, device=dev)
        self.idx = torch.empty(self.cap, dtype=torch.int32, device=dev)
        self.val = torch.empty(self.cap, dtype=torch.bfloat16, device=dev)
        self.cnt = torch.zeros(1, dtype=torch.int64, device=dev)
        self.out = torch.empty(n, dtype=torch.bfloat16, device=dev)
        self.flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
        self.flush_src = torch.zeros(64 << 20, dtype=torch.float32, device=dev)  # 256 MiB, only ever read
        # result buffers of the two fits (levels, error log): no allocation inside the timed region
        self.fit_out = [(torch.empty(16, dtype=torch.float32, device=dev),
                         torch.zeros(1, dtype=torch.float64, device=dev)) for _ in range(2)]
        self.cb_mse = self.cb_mae = self.cb0
        self.log_mse = torch.zeros(1, dtype=torch.float64, device=dev)
        self.have_mae = True
        self.only = None
        # the decode-side product y = W_q x sees the same codes as a square matrix (profiling runs only)
        self.gemv_rows = self.gemv_cols = int(round(n ** 0.5))
        self.x = workloads.gaussian(self.gemv_cols, 1.0, 5 + seed_offset, torch.bfloat16).to(dev)
        self.y = torch.empty(self.gemv_rows, dtype=torch.float32, device=dev)

    def flush_l2(self):
        # a write larger than L2, then a read of another buffer of the same size: the read pushes
        # the dirty lines of the write out, so that the timed kernel starts on a cold cache
        # without having to write somebody else's lines back
        self.flush_buf.zero_()
        self.flush_sink = self.flush_src.sum()

    def em_mse(self):
        b = self.b
        self.cb_mse, self.log_mse = b.bof4_fit_codebook([self.w], I, b.NORM_SIGNED, b.METRIC_MSE, self.cb0,
                                                        self.mask, 1, workspace=self.ws_em, sync=False,
                                                        out=self.fit_out[0])

    def em_mae(self):
        b = self.b
        self.cb_mae, self.log_mae = b.bof4_fit_codebook([self.w], I, b.NORM_SIGNED, b.METRIC_MAE, self.cb0,
                                                        self.mask, 1, workspace=self.ws_em, sync=False,
                                                        out=self.fit_out[1])

    def quant(self):
        b = self.b
        b.bof4_quantize_opq(self.w, I, b.NORM_SIGNED, self.cb_mse, self.tau, self.cap,
                            workspace=self.ws_opq,
                            out=(self.codes, self.scales, self.idx, self.val, self.cnt))

    def quant_plain(self):
        b = self.b
        b.bof4_quantize(self.w, I, b.NORM_SIGNED, self.cb_mse, out=(self.codes, self.scales))

    def dequant(self):
        b = self.b
        b.bof4_dequantize(self.codes, self.scales, I, self.cb_mse, b.BF16, (self.idx, self.val, self.cnt),
                          out=self.out)

    def gemv(self):
        b = self.b
        b.bof4_gemv(self.codes, self.scales, self.gemv_rows, self.gemv_cols, I, self.cb_mse, self.x,
                    (self.idx, self.val, self.cnt), out=self.y)

    def components(self):
        comps = [("em_mse", self.em_mse, 2), ("em_mae", self.em_mae, None), ("quantize_opq", self.quant, 4),
                 ("dequantize", self.dequant, 2)]
        comps = [c for c in comps if c[0] != "em_mae" or self.have_mae]
        if self.only:
            comps.append(("quantize", self.quant_plain, 1))  # profiling runs only
            comps.append(("gemv", self.gemv, 2))
            comps = [c for c in comps if c[0] in self.only]
        return comps

    def run_timed(self):
        """One step; returns {component: ms} from CUDA events on the current stream."""
        times = {}
        for name, fn, _ in self.components():
            self.flush_l2()
            s = torch.cuda.Event(enable_timing=True)
            e = torch.cuda.Event(enable_timing=True)
            s.record()
            fn()
            e.record()
            times[name] = (s, e)
        return times

    def run_e2e(self, host_out):
        """The same step from pinned host memory and back (copies inside the timed region)."""
        self.w.copy_(self.w_host, non_blocking=True)
        for _, fn, _ in self.components():
            fn()
        k = 0
        for name in ("codes", "scales", "idx", "val", "cnt", "out"):
            host_out[name].copy_(getattr(self, name), non_blocking=True)
        host_out["cb_mse"].copy_(self.cb_mse, non_blocking=True)
        host_out["log_mse"].copy_(self.log_mse, non_blocking=True)


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


def mae_launches(bof4) -> int:
    return getattr(bof4.binding, "MAE_LAUNCHES_PER_ITERATION", 0)


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

    st = Step(bof4, dev, seed_offset=workload_seed_offset(rank))  # no data-path collective
    st.have_mae = hasattr(binding, "MAE_LAUNCHES_PER_ITERATION")
    if args.only:
        st.only = set(args.only.split(","))
        args.no_e2e = args.no_cpu_baseline = True
        if "gemv" in st.only:
            assert st.gemv_rows * st.gemv_cols == st.n
            st.quant()  # the matrix the product reads
    K, W = args.steps, args.warmup
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
    # keep the device busy a little longer so that the clock sampler sees the loaded state
    t_end = time.time() + 0.3
    while time.time() < t_end:
        st.run_timed()
    torch.cuda.synchronize()
    clocks = sampler.stop()

    # ---- end to end: pinned host buffers in and out, through the same calls.  Two steps are in
    # flight on two streams with their own device and host buffers, so that one step's upload
    # overlaps the previous step's download (the copy engines work in both directions at once);
    # every step still uploads its weights and downloads all of its results inside the timed region.
    def make_host_out(step):
        h = {k: torch.empty_like(getattr(step, k), device="cpu").pin_memory()
             for k in ("codes", "scales", "idx", "val", "cnt", "out")}
        h["cb_mse"] = torch.empty(16, dtype=torch.float32).pin_memory()
        h["log_mse"] = torch.empty(1, dtype=torch.float64).pin_memory()
        return h

    Ke = 0 if args.no_e2e else max(2, min(K, 10))
    host_out = make_host_out(st)
    e2e_ms = 0.0
    if Ke:
        st2 = Step(bof4, dev, seed_offset=workload_seed_offset(rank), w_host=st.w_host)
        st2.have_mae = st.have_mae
        sets, outs = [st, st2], [host_out, make_host_out(st2)]
        streams = [torch.cuda.Stream(dev), torch.cuda.Stream(dev)]

        def e2e_steps(count):
            main = torch.cuda.current_stream()
            for sm in streams:
                sm.wait_stream(main)
            for i in range(count):
                with torch.cuda.stream(streams[i & 1]):
                    sets[i & 1].run_e2e(outs[i & 1])
            for sm in streams:
                main.wait_stream(sm)

        e2e_steps(2)
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        s = torch.cuda.Event(enable_timing=True)
        e = torch.cuda.Event(enable_timing=True)
        s.record()
        e2e_steps(Ke)
        e.record()
        torch.cuda.synchronize()
        e2e_ms = s.elapsed_time(e)
    h2d = st.w_host.numel() * 2
    d2h = sum(t.numel() * t.element_size() for t in host_out.values())

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dist, dev)
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    n = st.n
    ms_per_step = total_ms / K
    peak, peak_kind = measured_peak()
    avg = {k: sum(v) / len(v) for k, v in comp_ms.items()}
    bytes_per_w = {"em_mse": BYTES_EM, "em_mae": None, "quantize_opq": BYTES_QUANT, "dequantize": BYTES_DEQUANT,
                   "quantize": BYTES_QUANT, "gemv": BYTES_GEMV}
    # em_mae: the iteration's kernels + the call's max-|w| pass
    kernels = {"em_mse": 1, "em_mae": mae_launches(bof4) + 1, "quantize_opq": 2, "dequantize": 2, "quantize": 1,
               "gemv": 2}
    comp, launches = {}, 0
    for name, ms in avg.items():
        comp[name + "_ms"] = ms
        if name.startswith("em_"):
            comp[name + "_gweights_s"] = n / ms / 1e6
        if bytes_per_w[name]:
            comp[name + "_gbs"] = bytes_per_w[name] * n / ms / 1e6
        launches += kernels[name]
    for k in list(comp):
        if k.endswith("_gbs"):
            comp[k.replace("_gbs", "_frac_of_%s_hbm" % peak_kind)] = comp[k] / peak
    # dominant component = the one with the largest share of the step
    dom = max(avg, key=avg.get)
    dom_bytes = {"em_mse": BYTES_EM, "em_mae": BYTES_EM * MAE_DATA_PASSES, "quantize_opq": BYTES_QUANT,
                 "dequantize": BYTES_DEQUANT, "quantize": BYTES_QUANT, "gemv": BYTES_GEMV}[dom] * n
    achieved = dom_bytes / avg[dom] / 1e6
    line = {
        "metric": METRIC, "value": whole_job_gweights_per_s(world, n, ms_per_step), "unit": "Gweights/s",
        "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": WORKLOAD, "n_weights_per_gpu": n, "block_size": I,
                   "opq_q": Q, "l2": "flushed before every component (256 MiB write, then 256 MiB read: no dirty lines left)",
                   "multi_gpu": "independent problem per rank, no collective",
                   "e2e": "two steps in flight on two streams (upload of one overlaps download of the other)"},
        "components": comp,
        "clocks": clocks,
        "e2e": {"value": (world * n * Ke / e2e_ms / 1e6) if Ke else None, "unit": "Gweights/s",
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": Ke},
        "gpu_launches": launches * K,
        "roofline": {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak,
                     "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": TRAFFIC.get(dom)},
    }
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(st.w_host, have_mae=st.have_mae)
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum of the dominant component's data-carrying kernels
# per step, from the committed ncu captures (profiles/); None for a component whose kernels have
# changed since the counters were taken
TRAFFIC = {"em_mae": 414.4e6,   # max-|w| pass 137.3 MB + first pass 138.8 MB + collecting pass 138.3 MB
           "em_mse": 138.3e6}


# --------------------------------------------------------------------------- CPU arm (oracle)


def oracle_step(oracle, w32, lv0, mask, tau, have_mae=True):
    """The same step computed by the CPU oracle on fp32-widened weights."""
    cb, _ = oracle.fit(w32, I, oracle.NORM_SIGNED, oracle.METRIC_MSE, lv0, mask, 1)
    if have_mae:
        oracle.fit(w32, I, oracle.NORM_SIGNED, oracle.METRIC_MAE, lv0, mask, 1)
    clean, idx, val, k = oracle.opq_split(w32, I, tau)
    codes, scales = oracle.quantize(clean, I, oracle.NORM_SIGNED, cb)
    out = oracle.dequantize(codes, scales, I, cb)
    oracle.opq_restore(out, idx, val)
    return out


def cpu_baseline(w_host, have_mae=True, sample=1 << 25, reps=2):
    import oracle
    oracle.build()
    w32 = oracle.as_f32(w_host[:sample])
    lv0 = np.array(workloads.init_levels_7_0_8(), np.float32)
    tau = float(np.float32(oracle.opq_threshold(Q, I)))
    t0 = time.time()
    for _ in range(reps):
        oracle_step(oracle, w32, lv0, workloads.FIXED_BOF4S, tau, have_mae)
    dt = (time.time() - t0) / reps
    return {"value": sample / dt / 1e9, "unit": "Gweights/s", "cores": oracle.n_threads(),
            "kind": "oracle", "sample": "first 2^%d weights of the workload, %d steps" %
            (int(np.log2(sample)), reps)}


def run_reference(args):
    rank = rank_env()[0]
    if rank != 0:
        return None
    import oracle
    oracle.build()
    sample = 1 << 24
    w = workloads.gaussian_student_mixture(sample, 0.02, 0.01, 4, 1, torch.bfloat16)
    w32 = oracle.as_f32(w)
    lv0 = np.array(workloads.init_levels_7_0_8(), np.float32)
    tau = float(np.float32(oracle.opq_threshold(Q, I)))
    for _ in range(args.warmup):
        oracle_step(oracle, w32, lv0, workloads.FIXED_BOF4S, tau)
    t0 = time.time()
    for _ in range(args.steps):
        oracle_step(oracle, w32, lv0, workloads.FIXED_BOF4S, tau)
    dt = time.time() - t0
    val = sample * args.steps / dt / 1e9
    desc = {"value": val, "unit": "Gweights/s", "cores": oracle.n_threads(), "kind": "oracle",
            "sample": "2^24 weights of the workload per step"}
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "Gweights/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "n_weights_per_step": sample, "block_size": I, "opq_q": Q},
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
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
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
