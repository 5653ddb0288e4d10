"""ctypes binding of ``libbof4.so``: argument marshalling only.

Every function here has the name of the C entry point it calls (see ``include/bof4.h``) and
does nothing but turn torch CUDA tensors into device pointers, allocate the outputs with torch
(device memory and streams are the only things torch is used for) and check the status code.
All arithmetic of the method runs in the CUDA kernels; there is no CPU fallback: if the shared
library is missing or no CUDA device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbof4.so")

F32, BF16 = 0, 1
NORM_ABS, NORM_SIGNED = 0, 1
METRIC_MSE, METRIC_MAE = 0, 1
METRIC_MSE_NORMALIZED, METRIC_MAE_NORMALIZED = 2, 3  # App. D: errors of the normalised weights
OP_EM, OP_OPQ = 0, 1
LEVELS = 16

# kernels one MAE iteration enqueues: setup, 2 x (data pass + bin selection), then 2 data passes
# that carry their own selection and the level update
MAE_LAUNCHES_PER_ITERATION = 7

TENSORS_PER_LAUNCH = 64  # tensors of a multi-tensor fit that one accumulation launch covers


def mse_launches_per_iteration(n_tensors: int) -> int:
    """Kernels one MSE iteration enqueues (the M step rides in the last accumulation launch)."""
    return max(1, -(-n_tensors // TENSORS_PER_LAUNCH))


def mae_launches_per_call(n_tensors: int, n_total: int, iters: int) -> int:
    """Kernels a MAE fit of `iters` iterations enqueues: the max-|w| pass of the call, then per
    iteration the set-up, four data passes and the selection kernels of the passes that do not
    carry their own selection (two up to 2^26 weights, three beyond)."""
    chunks = max(1, -(-n_tensors // TENSORS_PER_LAUNCH))
    cap = min(max(n_total // 1024, 1 << 16), 1 << 23)      # candidate entries per level of the default workspace
    small = n_total // 1024 <= cap
    return chunks + iters * (1 + 4 * chunks + (2 if small else 3))


EXPORTS = ("bof4_workspace_bytes", "bof4_em_step", "bof4_fit_codebook", "bof4_quantize",
           "opq_split", "opq_split_static", "bof4_quantize_opq", "bof4_dequantize", "bof4_opq_threshold",
           "bof4_default_init", "bof4_last_error", "bof4_theoretical_codebook", "bof4_theoretical_codebook_batch",
           "bof4_gemv", "bof4_outlier_count", "bof4_scales_compress", "bof4_scales_expand",
           "bof4_theoretical_codebook_general", "bof4_quantize_batch", "bof4_dequantize_batch", "bof4_m_step", "bof4_gemm_tc")


class Bof4Error(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__("bof4 error %d: %s" % (code, msg))
        self.code = code


class EmStats(ctypes.Structure):
    """Mirror of ``bof4_em_stats``."""
    _fields_ = [("s1", ctypes.c_double * LEVELS), ("s0", ctypes.c_double * LEVELS),
                ("count", ctypes.c_uint64 * LEVELS), ("err_sum", ctypes.c_double),
                ("n_total", ctypes.c_int64), ("median", ctypes.c_float * LEVELS)]


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded shared library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("%s not found: run `python -m paper_2505_06653_b200.build`" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
        L.bof4_workspace_bytes.restype = sz
        L.bof4_workspace_bytes.argtypes = [i32, i64, i32, i32]
        L.bof4_em_step.restype = i32
        L.bof4_em_step.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, vp, vp, sz, vp]
        L.bof4_fit_codebook.restype = i32
        L.bof4_fit_codebook.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, ctypes.c_uint32, i32,
                                        vp, vp, sz, vp]
        L.bof4_quantize.restype = i32
        L.bof4_quantize.argtypes = [vp, i32, i64, i32, i32, vp, vp, vp, i32, vp]
        L.opq_split.restype = i32
        L.opq_split.argtypes = [vp, i32, i64, i32, ctypes.c_float, vp, vp, vp, i64, vp, vp, sz, vp]
        L.opq_split_static.restype = i32
        L.opq_split_static.argtypes = [vp, i32, i64, i32, ctypes.c_float, vp, vp, vp, i64, vp, vp]
        L.bof4_quantize_opq.restype = i32
        L.bof4_quantize_opq.argtypes = [vp, i32, i64, i32, i32, vp, ctypes.c_float, vp, vp, i32,
                                        vp, vp, i64, vp, vp, sz, vp]
        L.bof4_dequantize.restype = i32
        L.bof4_dequantize.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp, vp, i64, vp, i32, vp]
        L.bof4_gemv.restype = i32
        L.bof4_gemv.argtypes = [vp, vp, i32, i64, i64, i32, vp, vp, i32, vp, vp, vp, i64, vp, vp]
        L.bof4_theoretical_codebook.restype = i32
        L.bof4_theoretical_codebook.argtypes = [i32, i32, i32, vp, ctypes.c_uint32, i32, vp, sz, vp]
        L.bof4_theoretical_codebook_batch.restype = i32
        L.bof4_theoretical_codebook_batch.argtypes = [i32, vp, vp, vp, vp, vp, i32, vp, sz, vp]
        L.bof4_theoretical_codebook_general.restype = i32
        L.bof4_theoretical_codebook_general.argtypes = [i32, i32, i32, vp, i32, ctypes.c_double, vp, ctypes.c_uint32,
                                                        i32, vp, sz, vp]
        L.bof4_outlier_count.restype = i32
        L.bof4_outlier_count.argtypes = [vp, i64, vp, vp]
        L.bof4_quantize_batch.restype = i32
        L.bof4_quantize_batch.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, i32, vp]
        L.bof4_dequantize_batch.restype = i32
        L.bof4_dequantize_batch.argtypes = [vp, vp, i32, vp, i32, i32, vp, vp, i32, vp]
        L.bof4_gemm_tc.restype = i32
        L.bof4_gemm_tc.argtypes = [vp, vp, i32, i64, i64, i32, vp, vp, i32, vp, vp, vp, i64, vp, vp, vp, sz, vp]
        L.bof4_m_step.restype = i32
        L.bof4_m_step.argtypes = [vp, i32, i32, vp, ctypes.c_uint32, vp, vp, vp]
        L.bof4_scales_compress.restype = i32
        L.bof4_scales_compress.argtypes = [vp, i32, i64, i32, vp, vp, vp, vp]
        L.bof4_scales_expand.restype = i32
        L.bof4_scales_expand.argtypes = [vp, vp, vp, i64, vp, vp]
        L.bof4_opq_threshold.restype = ctypes.c_double
        L.bof4_opq_threshold.argtypes = [ctypes.c_double, i32]
        L.bof4_default_init.restype = i32
        L.bof4_default_init.argtypes = [i32, vp, vp]
        L.bof4_last_error.restype = ctypes.c_char_p
        L.bof4_last_error.argtypes = []
        _lib = L
    return _lib


def _check(rc: int):
    if rc != 0:
        raise Bof4Error(rc, lib().bof4_last_error().decode())


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError("weights must be float32 or bfloat16, got %s" % t.dtype)


def _torch_dt(code: int):
    return torch.float32 if code == F32 else torch.bfloat16


def _dev(t: torch.Tensor, name: str) -> torch.Tensor:
    if not t.is_cuda:
        raise ValueError("%s must be a CUDA tensor (there is no CPU path)" % name)
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    return t


_allocator = None


def set_output_allocator(fn) -> None:
    """Routes every buffer this binding allocates (outputs and workspaces) through
    ``fn(numel, dtype, device, zero) -> tensor``; None restores plain torch allocation.  A test
    harness uses it to surround each buffer with guard bands."""
    global _allocator
    _allocator = fn


def _new(numel: int, dtype, device, zero: bool = False) -> torch.Tensor:
    if _allocator is not None:
        return _allocator(int(numel), dtype, torch.device(device), zero)
    return (torch.zeros if zero else torch.empty)(int(numel), dtype=dtype, device=device)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _codebook(levels, device) -> torch.Tensor:
    if isinstance(levels, torch.Tensor):
        cb = levels.to(device=device, dtype=torch.float32).contiguous()
    else:
        cb = torch.tensor(np.asarray(levels, dtype=np.float32), device=device)
    if cb.numel() != LEVELS:
        raise ValueError("a codebook has 16 levels")
    return cb


def _workspace(op: int, n_max: int, block_size: int, metric: int, device) -> torch.Tensor:
    nbytes = lib().bof4_workspace_bytes(op, n_max, block_size, metric)
    if nbytes == 0:
        raise Bof4Error(-2, "bof4_workspace_bytes rejected the arguments")
    return _new(nbytes, torch.uint8, device)  # torch allocations are 512-B aligned


# --------------------------------------------------------------------------- host helpers


def bof4_workspace_bytes(op: int, n_max: int, block_size: int, metric: int = METRIC_MSE) -> int:
    return int(lib().bof4_workspace_bytes(op, n_max, block_size, metric))


def bof4_opq_threshold(q: float, block_size: int) -> float:
    return float(lib().bof4_opq_threshold(q, block_size))


def bof4_default_init(norm: int) -> Tuple[np.ndarray, int]:
    lv = np.zeros(LEVELS, np.float32)
    mask = ctypes.c_uint32(0)
    _check(lib().bof4_default_init(norm, lv.ctypes.data_as(ctypes.c_void_p), ctypes.byref(mask)))
    return lv, int(mask.value)


def bof4_last_error() -> str:
    return lib().bof4_last_error().decode()


# --------------------------------------------------------------------------- EM


def _tensor_list(ws: Sequence[torch.Tensor]):
    if isinstance(ws, torch.Tensor):
        ws = [ws]
    ws = [_dev(w, "weights").reshape(-1) for w in ws]
    if not ws:
        raise ValueError("empty tensor list")
    dt = _dt(ws[0])
    if any(_dt(w) != dt for w in ws):
        raise TypeError("all tensors of one call must share a dtype")
    ptrs = (ctypes.c_void_p * len(ws))(*[w.data_ptr() for w in ws])
    sizes = (ctypes.c_int64 * len(ws))(*[w.numel() for w in ws])
    return ws, dt, ptrs, sizes


def bof4_em_step(weights, block_size: int, norm: int, metric: int, levels,
                 workspace: Optional[torch.Tensor] = None) -> dict:
    """One accumulation pass; returns the ``bof4_em_stats`` record as a dict of numpy arrays."""
    ws, dt, ptrs, sizes = _tensor_list(weights)
    dev = ws[0].device
    cb = _codebook(levels, dev)
    wsp = workspace if workspace is not None else _workspace(
        OP_EM, sum(w.numel() for w in ws), block_size, metric, dev)
    stats = _new(ctypes.sizeof(EmStats), torch.uint8, dev, zero=True)
    with torch.cuda.device(dev):
        _check(lib().bof4_em_step(ptrs, sizes, len(ws), dt, block_size, norm, metric, _ptr(cb),
                                  _ptr(stats), _ptr(wsp), wsp.numel(), _stream()))
    rec = EmStats.from_buffer_copy(stats.cpu().numpy().tobytes())
    return dict(s1=np.array(rec.s1), s0=np.array(rec.s0), count=np.array(rec.count, dtype=np.uint64),
                err_sum=float(rec.err_sum), n=int(rec.n_total), median=np.array(rec.median, dtype=np.float32))


def em_step_record(weights, block_size: int, norm: int, metric: int, levels: torch.Tensor,
                   workspace: Optional[torch.Tensor] = None) -> torch.Tensor:
    """bof4_em_step with the record left on the device (uint8[sizeof(bof4_em_stats)]); `levels` is a
    device tensor fp32[16].  Nothing waits for the stream."""
    ws, dt, ptrs, sizes = _tensor_list(weights)
    dev = ws[0].device
    cb = _codebook(levels, dev)
    wsp = workspace if workspace is not None else _workspace(
        OP_EM, sum(w.numel() for w in ws), block_size, metric, dev)
    stats = _new(ctypes.sizeof(EmStats), torch.uint8, dev, zero=True)
    with torch.cuda.device(dev):
        _check(lib().bof4_em_step(ptrs, sizes, len(ws), dt, block_size, norm, metric, _ptr(cb),
                                  _ptr(stats), _ptr(wsp), wsp.numel(), _stream()))
    return stats


def gather_records(record: torch.Tensor, group=None) -> torch.Tensor:
    """The records of all ranks of `group`, concatenated in rank order (the record itself without a
    process group).  The one exchange of a joint fit: 432 bytes per rank and iteration."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return record
    world = dist.get_world_size(group)
    out = torch.empty(world * record.numel(), dtype=record.dtype, device=record.device)
    dist.all_gather_into_tensor(out, record.contiguous(), group=group)
    return out


def bof4_m_step(records: torch.Tensor, metric: int, codebook: torch.Tensor, fixed_mask: int,
                err_slot: Optional[torch.Tensor] = None) -> None:
    """Sums the gathered records in rank order and updates `codebook` (device fp32[16]) in place."""
    records = _dev(records, "records")
    n = records.numel() // ctypes.sizeof(EmStats)
    if records.dtype != torch.uint8 or n * ctypes.sizeof(EmStats) != records.numel():
        raise ValueError("records must be whole bof4_em_stats records as uint8")
    cb = _dev(codebook, "codebook")
    if cb.dtype != torch.float32 or cb.numel() != LEVELS:
        raise ValueError("codebook must be a device tensor float32[16]")
    with torch.cuda.device(cb.device):
        _check(lib().bof4_m_step(_ptr(records), n, metric, _ptr(cb), fixed_mask,
                                 _ptr(err_slot) if err_slot is not None else None, None, _stream()))


def bof4_fit_codebook_joint(weights, block_size: int, norm: int, metric: int, levels, fixed_mask: int,
                            iters: int, group=None):
    """Joint fit over the shards of all ranks of `group` (one process per GPU): every iteration is
    one bof4_em_step on the local shard, one all-gather of the 432-byte records and one bof4_m_step,
    so that every rank ends with the same levels.  MSE metrics.  -> (levels, err_log) on the device."""
    ws, _, _, _ = _tensor_list(weights)
    dev = ws[0].device
    cb = _codebook(levels, dev).clone()
    log = _new(max(iters, 1), torch.float64, dev, zero=True)
    wsp = _workspace(OP_EM, sum(w.numel() for w in ws), block_size, metric, dev)
    for t in range(iters):
        rec = em_step_record(ws, block_size, norm, metric, cb, workspace=wsp)
        bof4_m_step(gather_records(rec, group), metric, cb, fixed_mask, log[t:t + 1])
    torch.cuda.current_stream(dev).synchronize()
    return cb, log[:iters]


def bof4_fit_codebook(weights, block_size: int, norm: int, metric: int, levels, fixed_mask: int,
                      iters: int, workspace: Optional[torch.Tensor] = None,
                      sync: bool = True, out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None):
    """``iters`` Lloyd iterations; returns (levels, err_log) as device tensors (fp32[16],
    fp64[iters]).  With sync=False nothing waits for the stream.  `out` = (fp32[16], fp64[>= iters])
    device tensors to hold the results instead of fresh allocations."""
    ws, dt, ptrs, sizes = _tensor_list(weights)
    dev = ws[0].device
    if out is not None:
        cb, log = _dev(out[0], "out[0]"), _dev(out[1], "out[1]")
        if cb.dtype != torch.float32 or cb.numel() != LEVELS or log.dtype != torch.float64 or log.numel() < iters:
            raise ValueError("out must be (float32[16], float64[>= iters])")
        src = _codebook(levels, dev)
        if src.data_ptr() != cb.data_ptr():  # levels may be the output buffer itself: continue in place
            cb.copy_(src)
    else:
        cb = _codebook(levels, dev).clone()
        log = _new(max(iters, 1), torch.float64, dev, zero=True)
    wsp = workspace if workspace is not None else _workspace(
        OP_EM, sum(w.numel() for w in ws), block_size, metric, dev)
    with torch.cuda.device(dev):
        _check(lib().bof4_fit_codebook(ptrs, sizes, len(ws), dt, block_size, norm, metric, _ptr(cb),
                                       fixed_mask, iters, _ptr(log), _ptr(wsp), wsp.numel(), _stream()))
    if sync:
        torch.cuda.current_stream(dev).synchronize()
    return cb, log[:iters]


def bof4_theoretical_codebook(block_size: int, norm: int, metric: int, levels, fixed_mask: int,
                              iters: int, device="cuda") -> torch.Tensor:
    """Data-free Gaussian codebook: `iters` Lloyd iterations with theoretical centroids.
    -> levels fp32[16] on the device."""
    dev = torch.device(device)
    cb = _codebook(levels, dev).clone()
    ws = _new(256, torch.uint8, dev)
    with torch.cuda.device(dev):
        _check(lib().bof4_theoretical_codebook(block_size, norm, metric, _ptr(cb), fixed_mask, iters,
                                               _ptr(ws), ws.numel(), _stream()))
    return cb


def bof4_theoretical_codebook_general(block_size: int, norm: int, metric: int, pdf, w_max: float, levels,
                                      fixed_mask: int, iters: int, device="cuda") -> torch.Tensor:
    """Data-free codebook for a symmetric density given as samples pdf[j] = p_W(j * w_max / (len - 1)).
    -> levels fp32[16] on the device."""
    dev = torch.device(device)
    cb = _codebook(levels, dev).clone()
    tab = torch.as_tensor(np.ascontiguousarray(pdf, dtype=np.float64)).to(dev) if not isinstance(pdf, torch.Tensor) \
        else _dev(pdf.to(torch.float64), "pdf")
    n = tab.numel()
    ws = _new(256 + 24 * n, torch.uint8, dev)
    with torch.cuda.device(dev):
        _check(lib().bof4_theoretical_codebook_general(block_size, norm, metric, _ptr(tab), n, float(w_max), _ptr(cb),
                                                       fixed_mask, iters, _ptr(ws), ws.numel(), _stream()))
        torch.cuda.current_stream(dev).synchronize()   # the table is a temporary of this call
    return cb


def bof4_theoretical_codebook_batch(block_sizes, norms, metrics, levels, fixed_masks, iters: int,
                                    device="cuda") -> torch.Tensor:
    """The same for several problems at once; `levels` is [n, 16] (or [16], used for every
    problem).  -> levels fp32[n, 16] on the device."""
    dev = torch.device(device)
    n = len(block_sizes)
    if not (len(norms) == len(metrics) == len(fixed_masks) == n):
        raise ValueError("one block size, norm, metric and mask per problem")
    lv = torch.as_tensor(np.asarray(levels.cpu() if isinstance(levels, torch.Tensor) else levels, dtype=np.float32))
    if lv.dim() == 1:
        lv = lv.expand(n, LEVELS)
    if tuple(lv.shape) != (n, LEVELS):
        raise ValueError("levels must be [n, 16] or [16]")
    cb = lv.contiguous().to(dev).clone()
    ws = _new(256 * max(n, 1), torch.uint8, dev)
    arr = lambda v, t: (t * max(n, 1))(*[int(x) for x in v])
    with torch.cuda.device(dev):
        _check(lib().bof4_theoretical_codebook_batch(
            n, arr(block_sizes, ctypes.c_int), arr(norms, ctypes.c_int), arr(metrics, ctypes.c_int),
            arr(fixed_masks, ctypes.c_uint32), _ptr(cb), iters, _ptr(ws), ws.numel(), _stream()))
    return cb


# --------------------------------------------------------------------------- quantise / dequantise


def bof4_quantize(w: torch.Tensor, block_size: int, norm: int, levels,
                  scale_dtype: Optional[int] = None,
                  out: Optional[Tuple[torch.Tensor, torch.Tensor]] = None):
    """-> (codes uint8[n/2], scales [n/block_size])."""
    w = _dev(w, "w").reshape(-1)
    n, dt = w.numel(), _dt(w)
    sd = dt if scale_dtype is None else scale_dtype
    cb = _codebook(levels, w.device)
    if out is None:
        codes = _new((n + 1) // 2, torch.uint8, w.device)
        scales = _new(-(-n // max(block_size, 1)), _torch_dt(sd), w.device)
    else:
        codes, scales = out
    with torch.cuda.device(w.device):
        _check(lib().bof4_quantize(_ptr(w), dt, n, block_size, norm, _ptr(cb), _ptr(codes),
                                   _ptr(scales), sd, _stream()))
    return codes, scales


def bof4_dequantize(codes: torch.Tensor, scales: torch.Tensor, block_size: int, levels,
                    out_dtype: int, outliers: Optional[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]] = None,
                    out: Optional[torch.Tensor] = None, n: Optional[int] = None) -> torch.Tensor:
    """-> dequantised tensor [n]; `outliers` = (idx int32, val bf16, n_out int64[1]) for OPQ.
    `n` = number of weights when it is odd (default: twice the number of code bytes)."""
    codes = _dev(codes, "codes")
    scales = _dev(scales, "scales")
    n = codes.numel() * 2 if n is None else int(n)
    if (n + 1) // 2 != codes.numel():
        raise ValueError("codes must hold (n + 1) // 2 bytes")
    cb = _codebook(levels, codes.device)
    if out is None:
        out = _new(n, _torch_dt(out_dtype), codes.device)
    idx = val = cnt = None
    cap = 0
    if outliers is not None:
        idx, val, cnt = outliers
        cap = idx.numel()
    with torch.cuda.device(codes.device):
        _check(lib().bof4_dequantize(_ptr(codes), _ptr(scales), _dt(scales), n, block_size, _ptr(cb),
                                     _ptr(idx), _ptr(val), _ptr(cnt), cap, _ptr(out), out_dtype,
                                     _stream()))
    return out


def bof4_gemv(codes: torch.Tensor, scales: torch.Tensor, rows: int, cols: int, block_size: int, levels,
              x: torch.Tensor, outliers: Optional[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]] = None,
              out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """-> y fp32 [rows] = W_q x for the rows x cols matrix held as (codes, scales[, outliers])."""
    codes = _dev(codes, "codes")
    scales = _dev(scales, "scales")
    x = _dev(x, "x")
    if codes.numel() * 2 != rows * cols or x.numel() != cols:
        raise ValueError("codes must hold rows * cols weights and x cols values")
    cb = _codebook(levels, codes.device)
    if out is None:
        out = _new(rows, torch.float32, codes.device)
    idx = val = cnt = None
    cap = 0
    if outliers is not None:
        idx, val, cnt = outliers
        cap = idx.numel()
    with torch.cuda.device(codes.device):
        _check(lib().bof4_gemv(_ptr(codes), _ptr(scales), _dt(scales), rows, cols, block_size, _ptr(cb),
                               _ptr(x), _dt(x), _ptr(idx), _ptr(val), _ptr(cnt), cap, _ptr(out), _stream()))
    return out


def opq_split(w: torch.Tensor, block_size: int, tau: float, capacity: int,
              want_clean: bool = True, workspace: Optional[torch.Tensor] = None):
    """-> (w_clean or None, idx int32[capacity], val bf16[capacity], n_out int64[1])."""
    w = _dev(w, "w").reshape(-1)
    n, dt = w.numel(), _dt(w)
    dev = w.device
    wsp = workspace if workspace is not None else _workspace(OP_OPQ, n, block_size, 0, dev)
    clean = _new(w.numel(), w.dtype, w.device).view(w.shape) if want_clean else None
    idx = _new(capacity, torch.int32, dev)
    val = _new(capacity, torch.bfloat16, dev)
    cnt = _new(1, torch.int64, dev, zero=True)
    with torch.cuda.device(dev):
        _check(lib().opq_split(_ptr(w), dt, n, block_size, tau, _ptr(clean), _ptr(idx), _ptr(val),
                               capacity, _ptr(cnt), _ptr(wsp), wsp.numel(), _stream()))
    return clean, idx, val, cnt


def bof4_gemm_tc(codes: torch.Tensor, scales: torch.Tensor, rows: int, cols: int, block_size: int, levels,
                 x: torch.Tensor, workspace: Optional[torch.Tensor] = None, split: bool = True,
                 outliers: Optional[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]] = None):
    """Y fp32 [rows, n_rhs] = W_q X^T on the tensor cores for x bf16 [n_rhs, cols].
    -> (y, status int32[1]); status 0 unless a bounded wait inside the kernel ran out."""
    codes = _dev(codes, "codes")
    scales = _dev(scales, "scales")
    x = _dev(x, "x")
    if x.dtype != torch.bfloat16 or x.dim() != 2 or x.shape[1] != cols or codes.numel() * 2 != rows * cols:
        raise ValueError("x must be bf16 [n_rhs, cols] and codes must hold rows * cols weights")
    n_rhs = x.shape[0]
    cb = _codebook(levels, codes.device)
    y = _new(rows * n_rhs, torch.float32, codes.device).view(rows, n_rhs)
    status = _new(1, torch.int32, codes.device, zero=True)
    ws = workspace if workspace is not None else (_new(8 * rows * n_rhs * 4, torch.uint8, codes.device) if split else None)
    with torch.cuda.device(codes.device):
        idx = val = cnt = None
        cap = 0
        if outliers is not None:
            idx, val, cnt = (_dev(t, "outliers") for t in outliers)
            cap = idx.numel()
        _check(lib().bof4_gemm_tc(_ptr(codes), _ptr(scales), _dt(scales), rows, cols, block_size, _ptr(cb), _ptr(x),
                                  n_rhs, _ptr(idx), _ptr(val), _ptr(cnt), cap, _ptr(y), _ptr(status), _ptr(ws),
                                  ws.numel() if ws is not None else 0, _stream()))
    return y, status


def bof4_outlier_count(n_out: torch.Tensor, capacity: int) -> int:
    """Waits for the current stream and returns the true outlier count; raises Bof4Error
    (BOF4_ERR_CAPACITY) when it exceeds `capacity`, i.e. when outliers were dropped."""
    n_out = _dev(n_out, "n_out")
    if n_out.dtype != torch.int64 or n_out.numel() != 1:
        raise ValueError("n_out must be the int64[1] count tensor of an OPQ call")
    host = ctypes.c_int64(0)
    with torch.cuda.device(n_out.device):
        _check(lib().bof4_outlier_count(_ptr(n_out), int(capacity), ctypes.byref(host), _stream()))
    return int(host.value)


def _ptr_array(tensors):
    return (ctypes.c_void_p * len(tensors))(*[t.data_ptr() for t in tensors])


def bof4_quantize_batch(weights, block_size: int, norm: int, levels, scale_dtype: Optional[int] = None, out=None):
    """bof4_quantize over a list of tensors in few launches -> (list of codes, list of scales).
    `out` = (codes list, scales list) to write into instead of fresh allocations."""
    ws, dt, ptrs, sizes = _tensor_list(weights)
    dev = ws[0].device
    cb = _codebook(levels, dev)
    sd = dt if scale_dtype is None else scale_dtype
    if out is not None:
        codes, scales = [_dev(c, "codes") for c in out[0]], [_dev(s, "scales") for s in out[1]]
    else:
        codes = [_new((w.numel() + 1) // 2, torch.uint8, dev) for w in ws]
        scales = [_new(-(-w.numel() // max(block_size, 1)), _torch_dt(sd), dev) for w in ws]
    for w, c, sc in zip(ws, codes, scales):
        if c.numel() != (w.numel() + 1) // 2 or sc.numel() != -(-w.numel() // max(block_size, 1)) or _dt(sc) != sd:
            raise ValueError("out buffers do not match the tensors")
    with torch.cuda.device(dev):
        _check(lib().bof4_quantize_batch(ptrs, sizes, len(ws), dt, block_size, norm, _ptr(cb), _ptr_array(codes),
                                         _ptr_array(scales), sd, _stream()))
    return codes, scales


def bof4_dequantize_batch(codes, scales, sizes, block_size: int, levels, out_dtype: int = BF16, out=None):
    """bof4_dequantize (no outlier list) over a list of tensors in few launches -> list of outputs."""
    codes = [_dev(c, "codes") for c in codes]
    scales = [_dev(s, "scales") for s in scales]
    dev = codes[0].device
    cb = _codebook(levels, dev)
    outs = [_dev(o, "out") for o in out] if out is not None else [_new(int(n), _torch_dt(out_dtype), dev) for n in sizes]
    ns = (ctypes.c_int64 * len(codes))(*[int(n) for n in sizes])
    for c, sc, o, n in zip(codes, scales, outs, sizes):
        if c.numel() != (n + 1) // 2 or sc.numel() != -(-n // max(block_size, 1)) or o.numel() != n \
                or _dt(o) != out_dtype or _dt(sc) != _dt(scales[0]):
            raise ValueError("buffers do not match the sizes")
    with torch.cuda.device(dev):
        _check(lib().bof4_dequantize_batch(_ptr_array(codes), _ptr_array(scales), _dt(scales[0]), ns, len(codes),
                                           block_size, _ptr(cb), _ptr_array(outs), out_dtype, _stream()))
    return outs


def bof4_scales_compress(scales: torch.Tensor, norm: int):
    """Double quantisation of block constants -> (q uint8[B], group fp32[ceil(B/256)], sign uint8[ceil(B/8)] or None)."""
    scales = _dev(scales, "scales")
    B = scales.numel()
    dev = scales.device
    q = _new(B, torch.uint8, dev)
    g = _new((B + 255) // 256, torch.float32, dev)
    sign = _new((B + 7) // 8, torch.uint8, dev) if norm == NORM_SIGNED else None
    with torch.cuda.device(dev):
        _check(lib().bof4_scales_compress(_ptr(scales), _dt(scales), B, norm, _ptr(q), _ptr(g),
                                          _ptr(sign) if sign is not None else None, _stream()))
    return q, g, sign


def bof4_scales_expand(q: torch.Tensor, group: torch.Tensor, sign: Optional[torch.Tensor]) -> torch.Tensor:
    """The decoder's fp32 block constants from their double-quantised form."""
    q = _dev(q, "q")
    out = _new(q.numel(), torch.float32, q.device)
    with torch.cuda.device(q.device):
        _check(lib().bof4_scales_expand(_ptr(q), _ptr(_dev(group, "group")),
                                        _ptr(_dev(sign, "sign")) if sign is not None else None, q.numel(),
                                        _ptr(out), _stream()))
    return out


def bof4_quantize_opq(w: torch.Tensor, block_size: int, norm: int, levels, tau: float,
                      capacity: int, scale_dtype: Optional[int] = None,
                      workspace: Optional[torch.Tensor] = None, out=None):
    """-> (codes, scales, idx int32[capacity], val bf16[capacity], n_out int64[1])."""
    w = _dev(w, "w").reshape(-1)
    n, dt = w.numel(), _dt(w)
    dev = w.device
    sd = dt if scale_dtype is None else scale_dtype
    cb = _codebook(levels, dev)
    wsp = workspace if workspace is not None else _workspace(OP_OPQ, n, block_size, 0, dev)
    if out is None:
        codes = _new((n + 1) // 2, torch.uint8, dev)
        scales = _new(-(-n // max(block_size, 1)), _torch_dt(sd), dev)
        idx = _new(capacity, torch.int32, dev)
        val = _new(capacity, torch.bfloat16, dev)
        cnt = _new(1, torch.int64, dev, zero=True)
    else:
        codes, scales, idx, val, cnt = out
    with torch.cuda.device(dev):
        _check(lib().bof4_quantize_opq(_ptr(w), dt, n, block_size, norm, _ptr(cb), tau, _ptr(codes),
                                       _ptr(scales), sd, _ptr(idx), _ptr(val), capacity, _ptr(cnt),
                                       _ptr(wsp), wsp.numel(), _stream()))
    return codes, scales, idx, val, cnt
